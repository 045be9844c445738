"""Gated RMS normalisation behind the SSD layer: the oracle is pinned by a brute-force loop and by finite differences; the
CUDA kernels are compared with it (whole-row and grouped normalisation, both dtypes, several group widths)."""
import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc


def test_oracle_gated_norm_equals_brute_force_loop():
    rng = np.random.default_rng(0)
    y, z = rng.standard_normal((3, 12)), rng.standard_normal((3, 12))
    gamma = rng.standard_normal(12)
    for group in (12, 4):
        out, _, _ = orc.gated_norm_fwd(y, z, gamma, group, eps=1e-3)
        for r in range(3):
            for g0 in range(0, 12, group):
                v = [y[r, c] * z[r, c] / (1 + np.exp(-z[r, c])) for c in range(g0, g0 + group)]
                ms = sum(a * a for a in v) / group
                for j, c in enumerate(range(g0, g0 + group)):
                    assert abs(out[r, c] - v[j] / np.sqrt(ms + 1e-3) * gamma[c]) < 1e-12


def test_oracle_gated_norm_backward_matches_finite_differences():
    rng = np.random.default_rng(1)
    y, z = rng.standard_normal((2, 8)), rng.standard_normal((2, 8))
    gamma, g = rng.standard_normal(8), rng.standard_normal((2, 8))
    for group in (8, 4):
        dy, dz, dg = orc.gated_norm_bwd(y, z, gamma, g, group, eps=1e-3)
        loss = lambda a, b, c: float(np.sum(orc.gated_norm_fwd(a, b, c, group, eps=1e-3)[0] * g))
        eps = 1e-6
        for arr, grad, pos in ((y, dy, 0), (z, dz, 1), (gamma, dg, 2)):
            for idx in np.ndindex(arr.shape):
                hi, lo = arr.copy(), arr.copy()
                hi[idx] += eps
                lo[idx] -= eps
                args_hi = [y, z, gamma]
                args_lo = [y, z, gamma]
                args_hi[pos], args_lo[pos] = hi, lo
                fd = (loss(*args_hi) - loss(*args_lo)) / (2 * eps)
                assert abs(fd - grad[idx]) < 1e-6 * max(1.0, abs(fd)), (group, pos, idx)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,rows,D,group", [("fp32", 37, 512, 512), ("bf16", 37, 512, 128), ("bf16", 300, 5120, 5120),
                                                 ("bf16", 100, 5120, 640), ("fp32", 20, 8192, 8192)])
def test_gated_norm_matches_oracle(dtype, rows, D, group):
    from paper_2411_19460_b200 import libssd
    from tests.parity_util import TOL, relerr

    tol = TOL[dtype]
    td = torch.float32 if dtype == "fp32" else torch.bfloat16
    gen = torch.Generator().manual_seed(5)
    y = torch.randn(rows, D, generator=gen).to(td).cuda()
    z = torch.randn(rows, D, generator=gen).to(td).cuda()
    g = torch.randn(rows, D, generator=gen).to(td).cuda()
    gamma = (1.0 + 0.1 * torch.randn(D, generator=gen)).cuda()
    f64 = lambda t: t.detach().double().cpu().numpy()
    out_ref, _, _ = orc.gated_norm_fwd(f64(y), f64(z), f64(gamma), group)
    dy_ref, dz_ref, dg_ref = orc.gated_norm_bwd(f64(y), f64(z), f64(gamma), f64(g), group)
    out = libssd.ssd_gated_norm_fwd(y, z, gamma, group=group)
    dy, dz, dg = libssd.ssd_gated_norm_bwd(y, z, gamma, g, group=group)
    # in two row ranges with accumulation: the same values
    dg2 = torch.zeros_like(dg)
    half = rows // 2
    libssd.ssd_gated_norm_bwd(y[:half], z[:half], gamma, g[:half], group=group, dgamma=dg2, accumulate=True)
    libssd.ssd_gated_norm_bwd(y[half:], z[half:], gamma, g[half:], group=group, dgamma=dg2, accumulate=True)
    torch.cuda.synchronize()
    errs = dict(out=relerr(out, out_ref), dy=relerr(dy, dy_ref), dz=relerr(dz, dz_ref), dgamma=relerr(dg, dg_ref),
                dgamma_split=relerr(dg2, dg_ref))
    assert all(v <= tol for v in errs.values()), errs


@pytest.mark.gpu
def test_gated_norm_rejects_bad_arguments():
    from paper_2411_19460_b200 import libssd

    y = torch.zeros(4, 24, device="cuda")
    gamma = torch.ones(24, device="cuda")
    with pytest.raises(libssd.SSDError):
        libssd.ssd_gated_norm_fwd(y, y, gamma, group=10)              # D % group
    with pytest.raises(libssd.SSDError):
        libssd.ssd_gated_norm_fwd(y, y, gamma, group=6)               # group % 4
