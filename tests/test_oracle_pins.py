"""Pins for the fp64 oracle: things fixed by the mathematics, not by the oracle itself.

Eq. 1 (with dt, scalar A per head and the D skip) is checked against: a linear-attention closed
form (A=0, dt=1), a hand-worked scalar case, a geometric series, the fully unrolled sum written
with Python loops, central finite differences for every gradient, block-length invariance of the
Algorithm-2 backward, and a few symmetries.
"""
import math
import os

import numpy as np
import pytest

from oracle import ssd_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rand_problem(rng, B=2, L=12, H=4, P=3, N=5, G=2, h0=True, dhf=True):
    d = dict(
        x=rng.standard_normal((B, L, H, P)),
        dt=np.log1p(np.exp(rng.standard_normal((B, L, H)) * 0.5 - 1.0)),
        A=-np.exp(rng.uniform(0, math.log(16), H)),
        Bm=rng.standard_normal((B, L, G, N)) / math.sqrt(N),
        Cm=rng.standard_normal((B, L, G, N)) / math.sqrt(N),
        D=rng.standard_normal(H),
        h0=rng.standard_normal((B, H, P, N)) * 0.3 if h0 else None,
        dy=rng.standard_normal((B, L, H, P)),
        dh_final=rng.standard_normal((B, H, P, N)) if dhf else None,
    )
    return d


def fwd(d, seg=0):
    return orc.ssd_fwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], seg=seg)


def bwd(d, blk=256):
    return orc.ssd_bwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], d["dy"],
                       d["dh_final"], blk=blk)


def loss(d):
    y, hf, _ = fwd(d)
    val = float(np.sum(y * d["dy"]))
    if d["dh_final"] is not None:
        val += float(np.sum(hf * d["dh_final"]))
    return val


# ---------------------------------------------------------------- pin 1: linear attention
def test_closed_form_linear_attention():
    rng = np.random.default_rng(1)
    d = rand_problem(rng, B=2, L=37, H=4, P=3, N=5, G=2)
    d["A"] = np.zeros(4)
    d["dt"] = np.ones_like(d["dt"])
    y, hf, _ = fwd(d)
    B, L, H, P = d["x"].shape
    G = d["Bm"].shape[2]
    mask = np.tril(np.ones((L, L)))
    for b in range(B):
        for h in range(H):
            g = h // (H // G)
            scores = (d["Cm"][b, :, g] @ d["Bm"][b, :, g].T) * mask            # [t, s]
            ref = scores @ d["x"][b, :, h] + d["Cm"][b, :, g] @ d["h0"][b, h].T \
                + d["D"][h] * d["x"][b, :, h]
            np.testing.assert_allclose(y[b, :, h], ref, rtol=0, atol=1e-12)
            ref_h = d["h0"][b, h] + d["x"][b, :, h].T @ d["Bm"][b, :, g]
            np.testing.assert_allclose(hf[b, h], ref_h, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- pin 2: hand case
def _gold():
    vals = {}
    for line in open(os.path.join(GOLD, "hand_case.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        vals[k] = np.array([eval(s, {"LN2": math.log(2.0)}) for s in v], dtype=np.float64)
    return vals


def test_hand_case():
    gold = _gold()
    one = np.ones((1, 3, 1, 1))
    d = dict(x=np.array([1.0, 2.0, 3.0]).reshape(1, 3, 1, 1), dt=np.ones((1, 3, 1)),
             A=np.array([-math.log(2.0)]), Bm=one.copy(), Cm=one.copy(), D=np.array([1.0]),
             h0=None, dy=one.copy(), dh_final=None)
    y, hf, bd = fwd(d, seg=1)
    np.testing.assert_allclose(y.ravel(), gold["y"], atol=1e-15)
    assert hf.ravel()[0] == gold["h"][2]
    # boundary[k] is the state ENTERING segment k: 0, h1, h2
    np.testing.assert_allclose(bd.ravel(), [0.0, gold["h"][0], gold["h"][1]], atol=1e-15)
    for blk in (1, 2, 3, 100):
        g = bwd(d, blk=blk)
        for k in ("dx", "dB", "dC", "ddt", "dA", "dD", "dh0"):
            np.testing.assert_allclose(g[k].ravel(), gold[k], rtol=0, atol=1e-14, err_msg=k)


# ---------------------------------------------------------------- pin 3: geometric series
def test_time_invariant_scalar():
    L, a, dtv, h0v = 50, -0.7, 0.3, 1.7
    alpha = math.exp(dtv * a)
    d = dict(x=np.ones((1, L, 1, 1)), dt=np.full((1, L, 1), dtv), A=np.array([a]),
             Bm=np.ones((1, L, 1, 1)), Cm=np.ones((1, L, 1, 1)), D=np.array([0.0]),
             h0=np.full((1, 1, 1, 1), h0v), dy=None, dh_final=None)
    y, hf, _ = fwd(d)
    t = np.arange(1, L + 1)
    ref = alpha ** t * h0v + dtv * (1 - alpha ** t) / (1 - alpha)
    np.testing.assert_allclose(y.ravel(), ref, rtol=1e-13)
    assert abs(hf.ravel()[0] - ref[-1]) < 1e-13


# ---------------------------------------------------------------- pin 4: unrolled sum, python loops
def test_unrolled_bruteforce():
    rng = np.random.default_rng(4)
    d = rand_problem(rng, B=1, L=7, H=2, P=2, N=3, G=1)
    y, hf, bd = fwd(d, seg=3)
    B, L, H, P = d["x"].shape
    N = d["Bm"].shape[3]
    for h in range(H):
        a = d["dt"][0, :, h] * d["A"][h]
        for t in range(L):
            for p in range(P):
                acc = d["D"][h] * d["x"][0, t, h, p]
                for n in range(N):
                    acc += math.exp(sum(a[:t + 1])) * d["Cm"][0, t, 0, n] * d["h0"][0, h, p, n]
                for s in range(t + 1):
                    dec = math.exp(sum(a[s + 1:t + 1]))
                    cb = sum(d["Cm"][0, t, 0, n] * d["Bm"][0, s, 0, n] for n in range(N))
                    acc += cb * dec * d["dt"][0, s, h] * d["x"][0, s, h, p]
                assert abs(acc - y[0, t, h, p]) < 1e-13
        # the boundary entering segment k is the state after token 3k-1
        for k in range(3):
            tb = 3 * k
            for p in range(P):
                for n in range(N):
                    st = math.exp(sum(a[:tb])) * d["h0"][0, h, p, n]
                    for s in range(tb):
                        st += math.exp(sum(a[s + 1:tb])) * d["dt"][0, s, h] * d["x"][0, s, h, p] \
                            * d["Bm"][0, s, 0, n]
                    assert abs(st - bd[0, k, h, p, n]) < 1e-13


# ---------------------------------------------------------------- pin 5: finite differences
@pytest.mark.parametrize("blk", [5, 64])
def test_finite_differences_all_gradients(blk):
    rng = np.random.default_rng(5)
    d = rand_problem(rng, B=2, L=12, H=4, P=3, N=5, G=2)
    g = bwd(d, blk=blk)
    names = dict(dx="x", ddt="dt", dA="A", dB="Bm", dC="Cm", dD="D", dh0="h0")
    eps = 1e-6
    for gk, ik in names.items():
        arr = d[ik]
        flat = arr.reshape(-1)
        idxs = rng.choice(flat.size, size=min(flat.size, 25), replace=False)
        num = np.empty(len(idxs))
        for j, i in enumerate(idxs):
            keep = flat[i]
            flat[i] = keep + eps
            lp = loss(d)
            flat[i] = keep - eps
            lm = loss(d)
            flat[i] = keep
            num[j] = (lp - lm) / (2 * eps)
        ana = g[gk].reshape(-1)[idxs]
        scale = max(1.0, np.max(np.abs(ana)))
        assert np.max(np.abs(num - ana)) / scale < 1e-7, (gk, num, ana)


# ---------------------------------------------------------------- pin 6: block invariance
def test_block_length_invariance_and_boundaries():
    rng = np.random.default_rng(6)
    d = rand_problem(rng, B=2, L=45, H=4, P=3, N=5, G=2)
    ref = bwd(d, blk=45)
    for blk in (1, 7, 16, 44, 1000):
        g = bwd(d, blk=blk)
        for k in ("dx", "dB", "dC", "ddt", "dh0"):
            assert np.array_equal(g[k], ref[k]), (k, blk)
        for k in ("dA", "dD"):
            np.testing.assert_allclose(g[k], ref[k], rtol=1e-13)
    # Markov property: running the tail from a stored boundary state reproduces the tail.
    y, hf, bd = fwd(d, seg=16)
    assert bd.shape[1] == 3
    tail = {k: (v[:, 32:] if k in ("x", "dt", "Bm", "Cm", "dy") else v) for k, v in d.items()}
    tail["h0"] = bd[:, 2]
    y2, hf2, _ = fwd(tail)
    assert np.array_equal(y2, y[:, 32:]) and np.array_equal(hf2, hf)
    assert np.array_equal(bd[:, 0], d["h0"])
    # chained backward over two halves equals the one-shot backward (nabla_h hand-off of Alg. 2)
    head = {k: (v[:, :32] if k in ("x", "dt", "Bm", "Cm", "dy") else v) for k, v in d.items()}
    gt = bwd(tail, blk=8)
    head["dh_final"] = gt["dh0"]
    gh = bwd(head, blk=8)
    np.testing.assert_allclose(np.concatenate([gh["dx"], gt["dx"]], 1), ref["dx"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(np.concatenate([gh["dB"], gt["dB"]], 1), ref["dB"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(gh["dh0"], ref["dh0"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(gh["dA"] + gt["dA"], ref["dA"], rtol=1e-12)


# ---------------------------------------------------------------- pin 8: symmetries
def test_symmetries():
    rng = np.random.default_rng(8)
    d = rand_problem(rng, B=1, L=20, H=4, P=3, N=5, G=2)
    y, hf, _ = fwd(d)
    # scaling B by c and C by 1/c (with h0 scaled by c) leaves y unchanged
    d2 = dict(d, Bm=d["Bm"] * 3.0, Cm=d["Cm"] / 3.0, h0=d["h0"] * 3.0)
    y2, hf2, _ = fwd(d2)
    np.testing.assert_allclose(y2, y, rtol=0, atol=1e-13)
    np.testing.assert_allclose(hf2, hf * 3.0, rtol=0, atol=1e-13)
    # y is linear in (x, h0)
    d3 = dict(d, x=d["x"] * -2.0, h0=d["h0"] * -2.0)
    np.testing.assert_allclose(fwd(d3)[0], -2.0 * y, rtol=0, atol=1e-13)
    # swapping the two heads of group 0 swaps their outputs
    perm = [1, 0, 2, 3]
    d4 = dict(d, x=d["x"][:, :, perm], dt=d["dt"][:, :, perm], A=d["A"][perm], D=d["D"][perm],
              h0=d["h0"][:, perm])
    assert np.array_equal(fwd(d4)[0], y[:, :, perm])
    # dt -> 0: y -> C_t h0 + D x_t
    d5 = dict(d, dt=np.zeros_like(d["dt"]))
    y5, hf5, _ = fwd(d5)
    ref = np.einsum("btgn,bgjpn->btgjp", d["Cm"], d["h0"].reshape(1, 2, 2, 3, 5)).reshape(1, 20, 4, 3) \
        + d["D"][None, None, :, None] * d["x"]
    np.testing.assert_allclose(y5, ref, rtol=0, atol=1e-13)
    assert np.array_equal(hf5, d["h0"])


def test_threads_reported():
    assert orc.threads() >= 1
