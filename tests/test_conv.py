"""Depthwise causal conv (width 4) + SiLU with its three-input state across segment cuts: the oracle is pinned by a
brute-force loop, by finite differences and by segment invariance; the CUDA kernels are compared with it."""
import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc


def _case(B=2, L=11, C=8, seed=0):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((B, L, C)), rng.standard_normal((C, 4)) * 0.5, rng.standard_normal(C) * 0.1,
            rng.standard_normal((B, 3, C)), rng.standard_normal((B, L, C)))


def test_oracle_conv_equals_brute_force_loop():
    u, w, bias, st, _ = _case()
    out, pre, so = orc.conv_fwd(u, w, bias, st)
    B, L, C = u.shape
    for b in range(B):
        for t in range(L):
            for c in range(C):
                acc = bias[c]
                for k in range(4):
                    tt = t - 3 + k
                    acc += w[c, k] * (u[b, tt, c] if tt >= 0 else st[b, 3 + tt, c])
                assert abs(pre[b, t, c] - acc) < 1e-12
                assert abs(out[b, t, c] - acc / (1 + np.exp(-acc))) < 1e-12
    assert np.array_equal(so, u[:, -3:])


def test_oracle_conv_backward_matches_finite_differences():
    u, w, bias, st, g = _case(B=1, L=7, C=8, seed=1)
    du, dst, dw, db = orc.conv_bwd(u, w, bias, st, g)
    loss = lambda uu, ww, bb, ss: float(np.sum(orc.conv_fwd(uu, ww, bb, ss)[0] * g))
    eps = 1e-6
    rng = np.random.default_rng(2)
    for arr, grad in ((u, du), (w, dw), (bias, db), (st, dst)):
        for _ in range(6):
            idx = tuple(rng.integers(0, n) for n in arr.shape)
            hi, lo = arr.copy(), arr.copy()
            hi[idx] += eps
            lo[idx] -= eps
            args_hi = [hi if a is arr else a for a in (u, w, bias, st)]
            args_lo = [lo if a is arr else a for a in (u, w, bias, st)]
            fd = (loss(*args_hi) - loss(*args_lo)) / (2 * eps)
            assert abs(fd - grad[idx]) < 1e-6 * max(1.0, abs(fd)), (idx, fd, grad[idx])


def test_oracle_conv_is_invariant_to_segmentation():
    u, w, bias, st, g = _case(B=2, L=12, C=8, seed=3)
    out, _, _ = orc.conv_fwd(u, w, bias, st)
    du, dst, dw, db = orc.conv_bwd(u, w, bias, st, g)
    # forward in segments of 5, 4, 3 tokens with the carried state; backward right to left with dstate -> dtail
    cuts = [(0, 5), (5, 9), (9, 12)]
    states = [st]
    for a, b in cuts:
        o, _, s_out = orc.conv_fwd(u[:, a:b], w, bias, states[-1])
        assert np.allclose(o, out[:, a:b], atol=1e-13)
        states.append(s_out)
    dtail, dw_acc, db_acc = None, 0.0, 0.0
    for (a, b), s_in in reversed(list(zip(cuts, states[:-1]))):
        du_s, dtail, dw_s, db_s = orc.conv_bwd(u[:, a:b], w, bias, s_in, g[:, a:b], dtail)
        assert np.allclose(du_s, du[:, a:b], atol=1e-12)
        dw_acc, db_acc = dw_acc + dw_s, db_acc + db_s
    assert np.allclose(dtail, dst, atol=1e-12) and np.allclose(dw_acc, dw, atol=1e-12) and np.allclose(db_acc, db, atol=1e-12)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,B,L,C", [("fp32", 2, 300, 40), ("bf16", 2, 300, 40), ("bf16", 1, 1024, 5376),
                                         ("bf16", 6, 1536, 2560)])   # the last: 88 tokens (11 ring stages) per backward CTA
def test_conv_matches_oracle_whole_and_segmented(dtype, B, L, C):
    from paper_2411_19460_b200 import libssd
    from tests.parity_util import TOL, relerr

    tol = TOL[dtype]
    td = torch.float32 if dtype == "fp32" else torch.bfloat16
    gen = torch.Generator().manual_seed(11)
    u = torch.randn(B, L, C, generator=gen).to(td).cuda()
    g = torch.randn(B, L, C, generator=gen).to(td).cuda()
    st = torch.randn(B, 3, C, generator=gen).to(td).cuda()
    w = (torch.randn(C, 4, generator=gen) * 0.5).cuda()
    bias = (torch.randn(C, generator=gen) * 0.1).cuda()
    f64 = lambda t: t.detach().double().cpu().numpy()
    out_ref, _, so_ref = orc.conv_fwd(f64(u), f64(w), f64(bias), f64(st))
    du_ref, dst_ref, dw_ref, db_ref = orc.conv_bwd(f64(u), f64(w), f64(bias), f64(st), f64(g))

    out, so = libssd.ssd_conv_fwd(u, w, bias, st)
    du, dst, dw, db = libssd.ssd_conv_bwd(u, w, bias, st, g)
    torch.cuda.synchronize()
    assert torch.equal(so, u[:, -3:])
    errs = dict(out=relerr(out, out_ref), du=relerr(du, du_ref), dstate=relerr(dst, dst_ref), dw=relerr(dw, dw_ref),
                dbias=relerr(db, db_ref))
    assert all(v <= tol for v in errs.values()), errs

    # the same through three segments (ragged, not multiples of the token tile), B = 1 slices so that rows stay dense
    if B == 1:
        cuts = [(0, 400), (400, 777), (777, L)]
        state, outs = st, []
        states = [st]
        for a, b in cuts:
            o, state = libssd.ssd_conv_fwd(u[:, a:b], w, bias, state)
            outs.append(o)
            states.append(state)
        assert torch.equal(torch.cat(outs, dim=1), out)           # same arithmetic per token: same bits
        dtail, dus = None, []
        dw2 = torch.zeros_like(dw)
        db2 = torch.zeros_like(db)
        for (a, b), s_in in reversed(list(zip(cuts, states[:-1]))):
            du_s, dtail, _, _ = libssd.ssd_conv_bwd(u[:, a:b], w, bias, s_in, g[:, a:b], dtail, dw=dw2, dbias=db2,
                                                    accumulate=True)
            dus.insert(0, du_s)
        torch.cuda.synchronize()
        assert relerr(torch.cat(dus, dim=1), du_ref) <= tol and relerr(dtail, dst_ref) <= tol
        assert relerr(dw2, dw_ref) <= tol and relerr(db2, db_ref) <= tol


@pytest.mark.gpu
def test_conv_rejects_bad_arguments():
    from paper_2411_19460_b200 import libssd

    u = torch.zeros(1, 2, 8, device="cuda")
    w = torch.zeros(8, 4, device="cuda")
    bias = torch.zeros(8, device="cuda")
    with pytest.raises(libssd.SSDError):
        libssd.ssd_conv_fwd(u, w, bias)                            # L < 3
    with pytest.raises(libssd.SSDError):
        libssd.ssd_conv_fwd(torch.zeros(1, 8, 12, device="cuda"), torch.zeros(12, 4, device="cuda"),
                            torch.zeros(12, device="cuda"))       # C % 8
