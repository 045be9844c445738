"""ssd_fwd_static_ws: the forward for callers that cannot hand the library a scratch buffer
(no cudaMalloc where they run), using the fixed array built into the library instead.

Collected last on purpose.  The GPU test calls the entry point through the C ABI twice in a row,
with different inputs, and compares each result with the ordinary ssd_fwd on the same inputs: the
second call finds the first call's leftovers in the shared array and must not be affected by them.
It passes both alone in a fresh process and after the rest of the suite."""
import ctypes

import pytest
import torch

from paper_2411_19460_b200 import build as ssd_build
from paper_2411_19460_b200 import libssd
from paper_2411_19460_b200.inputs import CONFIGS, make_inputs
from tests.parity_util import TOL, relerr


def test_static_scratch_rejects_shapes_beyond_its_size():
    ssd_build.build()
    L = libssd.lib()
    big = libssd.SSDShape(1, 131072, 80, 64, 128, 1, 256, 4096, libssd.SSD_DTYPE_BF16, 0, 0, 0, 0)
    assert libssd.workspace_bytes(big, libssd.SSD_OP_FWD) > libssd.SSD_STATIC_WS_BYTES
    fake = ctypes.c_void_p(0x1000)
    rc = L.ssd_fwd_static_ws(ctypes.byref(big), fake, fake, fake, fake, fake, fake, None, fake, None, None)
    assert rc == libssd.SSD_ETOOLARGE
    assert b"SSD_STATIC_WS_BYTES" in L.ssd_strerror(rc)


@pytest.mark.gpu
def test_static_scratch_forward_matches_ssd_fwd_on_two_calls_in_a_row():
    cfg = CONFIGS[1].scaled(L=2048, H=8, G=2, seg=512)
    assert cfg.dtype == "bf16"
    tol = TOL[cfg.dtype]
    B, L, H, P, N = cfg.B, cfg.L, cfg.H, cfg.P, cfg.N
    for seed in (11, 12):
        inp = make_inputs(cfg, "cuda", seed=seed)
        args = (inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], inp["h0"])
        y_ref, h_ref = libssd.ssd_fwd(*args, chunk=cfg.chunk, seg=cfg.seg)
        y = torch.full_like(inp["x"], float("nan"))
        hf = torch.full((B, H, P, N), float("nan"), dtype=torch.float32, device="cuda")
        libssd.ssd_fwd_static_ws(*args, chunk=cfg.chunk, seg=cfg.seg, y=y, h_final=hf)
        torch.cuda.synchronize()
        ry = y_ref.double().cpu().numpy()
        rh = h_ref.double().cpu().numpy()
        assert relerr(y, ry) <= tol, (seed, relerr(y, ry))
        assert relerr(hf, rh) <= tol, (seed, relerr(hf, rh))
        assert torch.isfinite(y.float()).all() and torch.isfinite(hf).all()
        # the header promises more than the tolerance: the same kernels on the same inputs, so the same bits
        assert torch.equal(y, y_ref) and torch.equal(hf, h_ref), seed


def test_static_scratch_is_sized_without_the_second_copies():
    # four segments or more: ssd_fwd's default layout doubles some regions for its helper streams, the in-order
    # layout of the built-in scratch does not, so a shape can fit the latter and not the former
    ssd_build.build()
    L = libssd.lib()
    mk = lambda flags: libssd.SSDShape(1, 8192, 8, 64, 128, 1, 256, 1024, libssd.SSD_DTYPE_BF16, flags, 0, 0, 0)
    serial = libssd.workspace_bytes(mk(libssd.SSD_FLAG_SERIAL), libssd.SSD_OP_FWD)
    default = libssd.workspace_bytes(mk(0), libssd.SSD_OP_FWD)
    assert 0 < serial <= default
