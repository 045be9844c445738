"""Helpers for the GPU parity tests: run libssd through its C ABI on seeded inputs and compare with
the fp64 oracle element by element.  Error measure (per output tensor): max|gpu - ref| / max|ref|,
limit 1e-4 in fp32 mode and 2e-2 in bf16 mode (the oracle consumes the already-rounded inputs)."""
import numpy as np
import torch

from oracle import ssd_oracle as orc
from paper_2411_19460_b200 import libssd
from paper_2411_19460_b200.inputs import make_inputs, to_f64_numpy

TOL = {"fp32": 1e-4, "bf16": 2e-2}


def relerr(gpu, ref):
    g = gpu.detach().to("cpu", torch.float64).numpy() if isinstance(gpu, torch.Tensor) else np.asarray(gpu)
    den = max(float(np.max(np.abs(ref))), 1e-30)
    return float(np.max(np.abs(g - ref))) / den


# Outputs that belong to one head each, with the axis that indexes the head.  For these the error is also measured
# head by head, max over heads of max|gpu_h - ref_h| / max(max|ref_h|, HEAD_FLOOR * max|ref|): with stiff decays the
# heads differ by orders of magnitude, and a wrong result in a small head would vanish in the whole-tensor measure.
# The floor keeps a head whose reference is (almost) zero from turning rounding noise into a large ratio.
HEAD_AXIS = {"y": 2, "dx": 2, "ddt": 2, "h_final": 1, "dh0": 1, "boundary": 2}
HEAD_FLOOR = 0.05


def relerr_per_head(gpu, ref, axis):
    g = gpu.detach().to("cpu", torch.float64).numpy() if isinstance(gpu, torch.Tensor) else np.asarray(gpu)
    other = tuple(i for i in range(ref.ndim) if i != axis)
    den = np.maximum(np.max(np.abs(ref), axis=other), HEAD_FLOOR * max(float(np.max(np.abs(ref))), 1e-30))
    return float(np.max(np.max(np.abs(g - ref), axis=other) / den))


def run_gpu(cfg, inp, seg=None, flags=0, want=("fwd", "bwd")):
    seg = cfg.seg if seg is None else seg
    out = {}
    y, hf, bd = libssd.ssd_fwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"],
                                         inp["h0"], chunk=cfg.chunk, seg=seg, flags=flags)
    out.update(y=y, h_final=hf, boundary=bd)
    if "bwd" in want:
        g = libssd.ssd_bwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], bd,
                                     inp["dy"], inp["dh_final"], chunk=cfg.chunk, seg=seg, flags=flags)
        out.update(g)
    torch.cuda.synchronize()
    return out


def run_oracle(d, seg, want_bwd=True, blk=256):
    y, hf, bd = orc.ssd_fwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], seg=seg)
    ref = dict(y=y, h_final=hf, boundary=bd)
    if want_bwd:
        ref.update(orc.ssd_bwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], d["dy"],
                               d["dh_final"], blk=blk))
    return ref


def check_all(cfg, gpu, ref, keys=None, tol=None):
    tol = TOL[cfg.dtype] if tol is None else tol
    keys = [k for k in ref if k in gpu] if keys is None else keys
    errs = {k: relerr(gpu[k], ref[k]) for k in keys}
    errs.update({k + "/head": relerr_per_head(gpu[k], ref[k], HEAD_AXIS[k]) for k in keys if k in HEAD_AXIS})
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, "parity failure (limit %g): %s  | all: %s" % (tol, bad, errs)
    return errs


def full_parity(cfg, flags=0, seg=None, device="cuda"):
    inp = make_inputs(cfg, device)
    gpu = run_gpu(cfg, inp, seg=seg, flags=flags)
    ref = run_oracle(to_f64_numpy(inp), cfg.seg if seg is None else seg)
    return check_all(cfg, gpu, ref)
