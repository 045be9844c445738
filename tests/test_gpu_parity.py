"""GPU parity: libssd (through the C ABI) against the fp64 oracle, element by element, on seeded
inputs that span several chunks, several segments, a ragged last segment, both dtypes, several
chunk lengths, G > 1 and B > 1."""
import pytest
import torch

from paper_2411_19460_b200 import libssd
from paper_2411_19460_b200.inputs import CONFIGS, make_inputs, to_f64_numpy
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

SIMT = libssd.SSD_FLAG_FORCE_SIMT


def small(dtype="bf16", **kw):
    base = dict(name="small", dtype=dtype, B=1, L=1024, H=4, P=64, N=128, G=1, chunk=256, seg=512,
                h0_std=0.1, dh_std=0.1)
    base.update(kw)
    return CONFIGS[0].scaled(**base)


CASES = {
    "cfg0_fp32": CONFIGS[0],
    "fp32_n128_q128_dh": small("fp32", chunk=128, seg=256, L=768, G=2, B=2),
    "fp32_q256": small("fp32", chunk=256, seg=512, L=1280),                # ragged last segment
    "bf16_base": small("bf16"),
    "bf16_ragged_g2_b2": small("bf16", L=1280, G=2, B=2),
    "bf16_n64_q64": small("bf16", N=64, chunk=64, seg=128, L=448),
    "bf16_q128_h8": small("bf16", chunk=128, seg=384, L=1152, H=8, G=4),
    "bf16_stiff": small("bf16", a_max=64.0, dt_lo=1e-4, dt_hi=1.0, L=2048, seg=1024, H=8, G=2),
    "bf16_one_segment": small("bf16", seg=1024),
    # head counts of the other two model sizes of Appendix C's table (d_inner 2048 and 4096: 32 and 64 heads)
    "bf16_h32": small("bf16", H=32, L=512, seg=256),
    "bf16_h64_g8": small("bf16", H=64, G=8, L=512, seg=512),
}


@pytest.mark.parametrize("name", list(CASES))
def test_parity_simt(name):
    errs = pu.full_parity(CASES[name], flags=SIMT)
    print(name, errs)


@pytest.mark.parametrize("name", [n for n in CASES if CASES[n].dtype == "bf16"])
def test_parity_default_path(name):
    errs = pu.full_parity(CASES[name], flags=0)
    print(name, errs)


@pytest.mark.parametrize("name", ["bf16_base", "bf16_ragged_g2_b2", "bf16_stiff"])
def test_parity_two_kernel_dB_dC_path(name):
    """SSD_FLAG_SPLIT_BC: dB and dC by the two separate tensor-core kernels (the cross-check of the fused one)."""
    cfg = CASES[name]
    pu.full_parity(cfg, flags=libssd.SSD_FLAG_SPLIT_BC)


@pytest.mark.parametrize("name", ["bf16_ragged_g2_b2", "bf16_stiff", "bf16_h64_g8"])
def test_tensor_core_path_against_cuda_core_path(name):
    """The two GPU paths on the same bf16 inputs, at half the oracle tolerance: both round their outputs to bf16
    (or sum bf16 products in fp32), so they differ by a rounding step at most, wherever a head is large or small."""
    cfg = CASES[name]
    inp = make_inputs(cfg, "cuda")
    tc = pu.run_gpu(cfg, inp, flags=0)
    cc = pu.run_gpu(cfg, inp, flags=SIMT)
    errs = {}
    for k in ("y", "h_final", "dx", "ddt", "dA", "dB", "dC", "dD", "dh0"):
        ref = cc[k].detach().to("cpu", torch.float64).numpy()
        errs[k] = pu.relerr(tc[k], ref)
        if k in pu.HEAD_AXIS:
            errs[k + "/head"] = pu.relerr_per_head(tc[k], ref, pu.HEAD_AXIS[k])
    bad = {k: v for k, v in errs.items() if not (v <= 1e-2)}
    assert not bad, "paths disagree (limit 1e-2): %s | all %s" % (bad, errs)
    print(name, errs)


@pytest.mark.parametrize("flags", [SIMT, 0, libssd.SSD_FLAG_SPLIT_BC])
@pytest.mark.parametrize("name", ["cfg0_fp32", "bf16_ragged_g2_b2", "bf16_stiff"])
def test_segmented_backward_bit_exact_vs_unsegmented(name, flags):
    """The gradients must not depend on the segment length (seg == L is the unsegmented run)."""
    cfg = CASES[name]
    if cfg.dtype == "fp32" and flags == 0:
        flags = SIMT
    inp = make_inputs(cfg, "cuda")
    a = pu.run_gpu(cfg, inp, seg=cfg.seg, flags=flags)
    b = pu.run_gpu(cfg, inp, seg=cfg.L, flags=flags)
    c = pu.run_gpu(cfg, inp, seg=cfg.chunk, flags=flags)
    for k in ("y", "h_final", "dx", "ddt", "dA", "dB", "dC", "dD", "dh0"):
        assert torch.equal(a[k], b[k]), k
        assert torch.equal(a[k], c[k]), k
    assert torch.equal(a["boundary"][:, 0], b["boundary"][:, 0])


def test_deterministic_run_to_run():
    cfg = CASES["bf16_ragged_g2_b2"]
    inp = make_inputs(cfg, "cuda")
    a = pu.run_gpu(cfg, inp)
    b = pu.run_gpu(cfg, inp)
    for k in a:
        assert torch.equal(a[k], b[k]), k


def test_ssd_fwd_equals_segmented_forward():
    cfg = CASES["bf16_base"]
    inp = make_inputs(cfg, "cuda")
    y1, h1 = libssd.ssd_fwd(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], inp["h0"],
                            chunk=cfg.chunk)
    y2, h2, _ = libssd.ssd_fwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"],
                                         inp["h0"], chunk=cfg.chunk, seg=cfg.seg)
    torch.cuda.synchronize()
    assert torch.equal(y1, y2) and torch.equal(h1, h2)


def test_null_h0_and_null_dh():
    cfg = small("bf16", h0_std=0.0, dh_std=0.0)
    errs = pu.full_parity(cfg)
    print(errs)


def test_status_word_clean():
    cfg = CASES["bf16_base"]
    inp = make_inputs(cfg, "cuda")
    shape = libssd.make_shape(inp["x"], inp["Bm"], cfg.chunk, cfg.seg)
    ws = libssd.alloc_workspace(shape, libssd.SSD_OP_FWD_SEG, "cuda")
    libssd.ssd_fwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], inp["h0"],
                             chunk=cfg.chunk, seg=cfg.seg, ws=ws)
    torch.cuda.synchronize()
    assert libssd.poll_status(ws) == libssd.SSD_OK


@pytest.mark.gpu
@pytest.mark.parametrize("seg", [512, 768, 1024, 2048])   # 4 segments (second scratch copies), 3 (ragged), 2, 1
def test_helper_streams_change_no_bit_and_respect_caller_stream(seg):
    """The backward's forked helper streams (default) against SSD_FLAG_SERIAL: the same bits, also when the
    caller's stream is not the default one and is the only thing the caller synchronises."""
    cfg = small(B=2, L=2048, H=8, G=2, seg=seg)
    inp = make_inputs(cfg, "cuda")
    ref = pu.run_gpu(cfg, inp, flags=libssd.SSD_FLAG_SERIAL)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        g = libssd.ssd_bwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], ref["boundary"],
                                     inp["dy"], inp["dh_final"], chunk=cfg.chunk, seg=cfg.seg, stream=s)
    s.synchronize()                                   # only the caller's stream
    for k, v in g.items():
        if v is not None:
            assert torch.equal(v, ref[k]), k
    # the forward with its state chain one segment ahead on a helper stream, same check
    with torch.cuda.stream(s):
        y, h_final, boundary = libssd.ssd_fwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"],
                                                        inp["h0"], chunk=cfg.chunk, seg=cfg.seg, stream=s)
    s.synchronize()
    assert torch.equal(y, ref["y"]) and torch.equal(h_final, ref["h_final"]) and torch.equal(boundary, ref["boundary"])


@pytest.mark.gpu
def test_two_caller_streams_from_one_thread_share_the_helper_streams():
    """Two calls issued back to back by one host thread on two caller streams: the library's helper streams and
    events belong to the (thread, device), so the second call's forks queue behind the first call's work on them.
    That serialises the two calls against each other but must not mix them up: each result equals the result of
    the same call made alone, bit for bit."""
    cfg = small(B=1, L=2048, H=8, G=2, seg=256)           # eight segments: every helper stream and twin copy in use
    inps = [make_inputs(cfg, "cuda", seed=s) for s in (21, 22)]
    refs = [pu.run_gpu(cfg, i) for i in inps]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for st in streams:
        st.wait_stream(torch.cuda.current_stream())
    got = []
    for i, st in zip(inps, streams):                       # no synchronisation between the two calls
        with torch.cuda.stream(st):
            y, hf, bd = libssd.ssd_fwd_segmented(i["x"], i["dt"], i["A"], i["Bm"], i["Cm"], i["D"], i["h0"],
                                                 chunk=cfg.chunk, seg=cfg.seg, stream=st)
            g = libssd.ssd_bwd_segmented(i["x"], i["dt"], i["A"], i["Bm"], i["Cm"], i["D"], bd, i["dy"], i["dh_final"],
                                         chunk=cfg.chunk, seg=cfg.seg, stream=st)
        got.append(dict(y=y, h_final=hf, boundary=bd, **g))
    for st in streams:
        st.synchronize()
    for ref, out in zip(refs, got):
        for k, v in out.items():
            if v is not None:
                assert torch.equal(v, ref[k]), k


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_skip_gradient_flag_adds_dy_to_dx(dtype):
    """SSD_FLAG_SKIP_GRAD: dx = (plain dx) + dy with one rounding; every other output unchanged."""
    cfg = small(dtype=dtype, B=2, L=1024, H=8, G=2, seg=512) if dtype == "bf16" else CASES["fp32_q256"]
    inp = make_inputs(cfg, "cuda")
    ref = pu.run_gpu(cfg, inp)
    g = libssd.ssd_bwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], ref["boundary"],
                                 inp["dy"], inp["dh_final"], chunk=cfg.chunk, seg=cfg.seg, flags=libssd.SSD_FLAG_SKIP_GRAD)
    torch.cuda.synchronize()
    want = ref["dx"].float() + inp["dy"].float()
    err = (g["dx"].float() - want).abs().max().item() / want.abs().max().item()
    assert err <= (8e-3 if dtype == "bf16" else 1e-6), err
    for k, v in g.items():
        if v is not None and k != "dx":
            assert torch.equal(v, ref[k]), k
