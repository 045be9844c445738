"""Host-side checks that need no GPU: the C-ABI library builds, loads, exports every symbol the
header declares, sizes workspaces sensibly and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2411_19460_b200 import build as ssd_build
from paper_2411_19460_b200 import libssd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    ssd_build.build()
    return libssd.lib()


def shape(**kw):
    base = dict(B=1, L=1024, H=4, P=64, N=128, G=1, chunk=256, seg=512, dtype=1, flags=0,
                x_bstride=0, dt_bstride=0, bc_bstride=0)
    base.update(kw)
    return libssd.SSDShape(**base)


def test_exports_match_header(L):
    hdr = open(os.path.join(ROOT, "include", "ssd.h")).read()
    declared = set(re.findall(r"\b(ssd_[a-z_0-9]+)\s*\(", hdr))
    assert declared == set(libssd.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name
    assert L.ssd_version() == int(re.search(r"#define SSD_VERSION (\d+)", hdr).group(1))


def test_struct_layout_matches_header():
    assert ctypes.sizeof(libssd.SSDShape) == 10 * 4 + 3 * 8


def test_workspace_scales_with_segment_not_length(L):
    w = lambda **kw: libssd.workspace_bytes(shape(**kw), libssd.SSD_OP_BWD_SEG)
    assert w(seg=256) < w(seg=512) < w(seg=1024)
    # doubling L at fixed seg adds only the per-chunk dA/dD partial sums
    a, b = w(L=1024, seg=256), w(L=2048, seg=256)
    assert 0 <= b - a <= 4 * (2048 // 256) * 4 * 8
    f = libssd.workspace_bytes(shape(), libssd.SSD_OP_FWD_SEG)
    assert 0 < f < w()
    assert libssd.boundary_bytes(shape(L=1280, seg=512)) == 3 * 4 * 64 * 128 * 4
    assert libssd.boundary_bytes(shape(seg=0)) == 4 * 64 * 128 * 4


@pytest.mark.parametrize("kw,code", [
    (dict(H=3, G=2), libssd.SSD_EINVAL),
    (dict(L=1000), libssd.SSD_EINVAL),
    (dict(seg=300), libssd.SSD_EINVAL),
    (dict(B=0), libssd.SSD_EINVAL),
    (dict(P=32), libssd.SSD_EUNSUPPORTED),
    (dict(N=96), libssd.SSD_EUNSUPPORTED),
    (dict(chunk=32, seg=64, L=64), libssd.SSD_EUNSUPPORTED),
    (dict(dtype=7), libssd.SSD_EUNSUPPORTED),
    (dict(x_bstride=1024 * 4 * 64 + 3), libssd.SSD_EALIGN),
])
def test_bad_shapes_rejected_on_host(L, kw, code):
    s = shape(**kw)
    assert libssd.workspace_bytes(s, libssd.SSD_OP_FWD) == 0
    fake = ctypes.c_void_p(0x1000)
    rc = L.ssd_fwd(ctypes.byref(s), fake, fake, fake, fake, fake, fake, None, fake, None, fake, 1 << 30, None)
    assert rc == code, L.ssd_strerror(rc)


def test_null_misaligned_and_small_workspace(L):
    s = shape()
    ok = ctypes.c_void_p(0x1000)
    bad = ctypes.c_void_p(0x1004)
    big = 1 << 40
    assert L.ssd_fwd(ctypes.byref(s), None, ok, ok, ok, ok, ok, None, ok, None, ok, big, None) == libssd.SSD_EINVAL
    assert L.ssd_fwd(ctypes.byref(s), bad, ok, ok, ok, ok, ok, None, ok, None, ok, big, None) == libssd.SSD_EALIGN
    assert L.ssd_fwd(ctypes.byref(s), ok, ok, ok, ok, ok, ok, None, ok, None, ok, 16, None) == libssd.SSD_EWORKSPACE
    assert L.ssd_fwd(ctypes.byref(s), ok, ok, ok, ok, ok, ok, None, ok, None, ctypes.c_void_p(0x1010), big,
                     None) == libssd.SSD_EWORKSPACE
    # segmented forward requires the boundary buffer
    assert L.ssd_fwd_segmented(ctypes.byref(s), ok, ok, ok, ok, ok, ok, None, ok, None, None, ok, big,
                               None) == libssd.SSD_EINVAL
    assert L.ssd_bwd_segmented(ctypes.byref(s), ok, ok, ok, ok, ok, ok, None, ok, None, ok, ok, ok, ok, ok, ok,
                               None, ok, big, None) == libssd.SSD_EINVAL
    assert b"workspace" in L.ssd_strerror(libssd.SSD_EWORKSPACE)
    assert L.ssd_poll_status(None) == libssd.SSD_EINVAL


@pytest.mark.gpu
def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    """The failure path of the device-side waits, made on purpose in the only harmless way: a barrier that nothing
    arrives on, waited for a few thousand cycles by one warp with nothing else in flight.  The kernel must return by
    itself, the status word must read SSD_ETIMEOUT, and an ordinary call afterwards must work and poll clean."""
    import torch
    from paper_2411_19460_b200.inputs import CONFIGS, make_inputs
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    libssd.selftest_wait_timeout(ws, 5000)
    torch.cuda.synchronize()
    assert libssd.poll_status(ws) == libssd.SSD_ETIMEOUT
    waited = int(ws[256:264].view(torch.int64).item())
    assert 5000 < waited < 50_000_000, waited          # gave up after the limit, and soon after it
    # the context is intact: a normal forward on the same stream, with its own scratch, runs and polls clean
    cfg = CONFIGS[1].scaled(L=1024, H=4, seg=512)
    inp = make_inputs(cfg, "cuda")
    y, hf, bd = libssd.ssd_fwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], inp["h0"],
                                         chunk=cfg.chunk, seg=cfg.seg)
    torch.cuda.synchronize()
    assert torch.isfinite(y.float()).all()
    libssd.selftest_wait_timeout(ws, 0)                 # limit 0: gives up at the first check
    torch.cuda.synchronize()
    assert libssd.poll_status(ws) == libssd.SSD_ETIMEOUT
