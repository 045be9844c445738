"""Single-token step of Eq. 1 (forward-only streaming): the oracle's step is pinned to the sequence oracle
and to a hand-computed case; the CUDA step is compared with it, alone and continuing ssd_fwd's state."""
import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc
from paper_2411_19460_b200.inputs import CONFIGS, make_inputs, to_f64_numpy


def test_oracle_step_by_hand():
    # B=H=P=1, N=2: h = e^{dt A} h + dt x B ; y = C.h + D x
    y, h = orc.decode_step(np.array([[[2.0]]]), np.array([[0.5]]), np.array([-1.0]), np.array([[[1.0, -3.0]]]),
                           np.array([[[4.0, 0.25]]]), np.array([0.125]), np.array([[[[1.0, 2.0]]]]))
    a = np.exp(-0.5)
    h_ref = np.array([a * 1.0 + 0.5 * 2.0 * 1.0, a * 2.0 + 0.5 * 2.0 * -3.0])
    assert np.allclose(h[0, 0, 0], h_ref, rtol=0, atol=1e-15)
    assert np.isclose(y[0, 0, 0], 4.0 * h_ref[0] + 0.25 * h_ref[1] + 0.125 * 2.0, rtol=0, atol=1e-15)


def test_oracle_steps_reproduce_the_sequence_oracle():
    cfg = CONFIGS[0].scaled(B=2, L=24, H=4, G=2, chunk=8, seg=8, h0_std=0.1)
    d = to_f64_numpy(make_inputs(cfg, "cpu"))
    y_seq, h_fin, _ = orc.ssd_fwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], seg=8)
    h = d["h0"].copy()
    for t in range(cfg.L):
        y, h = orc.decode_step(d["x"][:, t], d["dt"][:, t], d["A"], d["Bm"][:, t], d["Cm"][:, t], d["D"], h)
        assert np.allclose(y, y_seq[:, t], rtol=1e-12, atol=1e-12), t
    assert np.allclose(h, h_fin, rtol=1e-12, atol=1e-12)


@pytest.mark.gpu
@pytest.mark.parametrize("which,G,N", [(0, 1, 128), (1, 1, 128), (0, 2, 64), (1, 2, 64)])
def test_decode_step_matches_oracle_and_continues_ssd_fwd(which, G, N):
    from paper_2411_19460_b200 import libssd
    from tests.parity_util import TOL, relerr

    base = CONFIGS[which]
    cfg = base.scaled(B=2, L=512 + 5, H=8, G=G, N=N, seg=256, h0_std=0.1)
    tol = TOL[cfg.dtype]
    inp = make_inputs(cfg, "cuda")
    d = to_f64_numpy({k: (v.cpu() if v is not None else None) for k, v in inp.items()})
    Lp = 512                                                      # prefix by the chunked kernels
    pre = {k: inp[k][:, :Lp].contiguous() for k in ("x", "dt", "Bm", "Cm")}
    y_pre, h = libssd.ssd_fwd(pre["x"], pre["dt"], inp["A"], pre["Bm"], pre["Cm"], inp["D"], inp["h0"],
                              chunk=cfg.chunk, seg=cfg.seg)
    # the oracle walks the same 517 tokens one by one from h0
    h_ref = d["h0"].copy()
    ys_ref = []
    for t in range(cfg.L):
        y_t, h_ref = orc.decode_step(d["x"][:, t], d["dt"][:, t], d["A"], d["Bm"][:, t], d["Cm"][:, t], d["D"], h_ref)
        ys_ref.append(y_t)
        if t == Lp - 1:
            assert relerr(h, h_ref) <= tol
            h_at_prefix = h_ref.copy()
    # (a) one step from the oracle's own state: isolates the step kernel
    h_one = torch.tensor(h_at_prefix, dtype=torch.float32, device="cuda")
    h_before = h_one.double().cpu().numpy()                       # the step updates h_one in place
    y_one = libssd.ssd_decode_step(inp["x"][:, Lp:Lp + 1], inp["dt"][:, Lp:Lp + 1], inp["A"], inp["Bm"][:, Lp:Lp + 1],
                                   inp["Cm"][:, Lp:Lp + 1], inp["D"], h_one)
    y1, h1 = orc.decode_step(d["x"][:, Lp], d["dt"][:, Lp], d["A"], d["Bm"][:, Lp], d["Cm"][:, Lp], d["D"], h_before)
    assert relerr(y_one[:, 0], y1) <= tol and relerr(h_one, h1) <= 1e-6
    # (b) the tail of the sequence token by token from ssd_fwd's state, slices of the long tensors
    for t in range(Lp, cfg.L):
        y_t = libssd.ssd_decode_step(inp["x"][:, t:t + 1], inp["dt"][:, t:t + 1], inp["A"], inp["Bm"][:, t:t + 1],
                                     inp["Cm"][:, t:t + 1], inp["D"], h)
        assert relerr(y_t[:, 0], ys_ref[t]) <= tol, t
    assert relerr(h, h_ref) <= tol


@pytest.mark.gpu
def test_decode_step_rejects_bad_arguments():
    from paper_2411_19460_b200 import libssd

    cfg = CONFIGS[0].scaled(B=1, L=256, H=4)
    inp = make_inputs(cfg, "cuda")
    h = torch.zeros(1, cfg.H, cfg.P, cfg.N, device="cuda")
    with pytest.raises(ValueError):
        libssd.ssd_decode_step(inp["x"][:, :2], inp["dt"][:, :2], inp["A"], inp["Bm"][:, :2], inp["Cm"][:, :2], inp["D"], h)
    shape = libssd.SSDShape(1, 2, cfg.H, cfg.P, cfg.N, cfg.G, 0, 0, libssd.SSD_DTYPE_F32, 0, 0, 0, 0)
    import ctypes
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    rc = libssd.lib().ssd_decode_step(ctypes.byref(shape), p(inp["x"]), p(inp["dt"]), p(inp["A"]), p(inp["Bm"]),
                                      p(inp["Cm"]), p(inp["D"]), p(h), p(inp["x"]), None)
    assert rc == libssd.SSD_EINVAL
