#!/usr/bin/env python
"""Benchmark of libssd: segmented SSD forward + backward (MA-GC along the sequence axis).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--seg S] [--impl ours|reference]

One "step" = ssd_fwd_segmented + ssd_bwd_segmented over one batch of seeded synthetic input.
Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every rank runs an
independent replica on its own GPU: the path has no cross-GPU step, so no data-path collective is
used; only the barrier and the max-over-ranks of the timing go through torch.distributed.

`--impl reference` times the fp64 CPU oracle (oracle/), as it stands, on the host cores, on a
bounded sample of the same workload.
"""
import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2411_19460_b200.inputs import CONFIGS, make_inputs, to_f64_numpy  # noqa: E402

METRIC = "ssd_fwd_bwd_segmented_tokens_per_s"
# With no --config the line is that of the largest single-layer workload that fits one GPU (the million-token one),
# and the 2.7B-dimension layer at 131072 tokens and the small fp32 case ride along under "also", device-timed.
HEADLINE_CONFIG = 4
ALSO_CONFIGS = (2, 0)
UNIT = "tokens/s"


# ----------------------------------------------------------------------------- analytic model
def kappa(Q):
    return (Q + 1) / (2.0 * Q)


def kind_model(cfg):
    """Algorithmic flops and bytes per token for each kernel kind (one launch processes
    B * segment-length tokens).  Only the lower triangle of the Q x Q products counts; elementwise
    work and exponentials are not counted; e = bytes per I/O element."""
    H, P, N, G, Q = cfg.H, cfg.P, cfg.N, cfg.G, cfg.chunk
    e = 2 if cfg.dtype == "bf16" else 4
    k = kappa(Q)
    HPN = H * P * N
    st = 4.0 * HPN / Q                       # one fp32 chunk state per Q tokens
    return {
        # kind: (bound, flops/token, bytes/token)
        "chunk_cumsum": ("hbm", 0.0, 12.0 * H),
        "chunk_state": ("tensor", 2.0 * HPN, e * (H * P + G * N) + st),
        "state_pass_fwd": ("hbm", 0.0, 2.0 * st),
        "chunk_scan_fwd": ("tensor", 2.0 * HPN + 2 * k * Q * (G * N + H * P), e * (2 * H * P + 2 * G * N) + st),
        "dstate_contrib": ("tensor", 2.0 * HPN, e * (H * P + G * N) + st),
        "state_pass_bwd": ("hbm", 0.0, 3.0 * st),
        "bwd_dx": ("tensor", 2.0 * HPN + 2 * k * Q * (G * N + H * P), e * (3 * H * P + 2 * G * N) + st),
        "bwd_dC": ("tensor", 2.0 * HPN + 2 * k * Q * (G * N + H * P), e * (2 * H * P + 2 * G * N) + st),
        "bwd_dB": ("tensor", 2.0 * HPN + 2 * k * Q * (G * N), e * (2 * H * P + 2 * G * N) + st),
        # dB and dC from one masked tile: scores once, the two products of the head-summed tile, two state terms
        "bwd_dBdC": ("tensor", 4.0 * HPN + 2 * k * Q * (H * P + 2 * G * N), e * (2 * H * P + 2 * G * N) + 2 * st),
        "bwd_finish": ("hbm", 0.0, 16.0 * H),
        "reduce_dBdC": ("hbm", 0.0, 2.0 * e * G * N),
        "final_dAdD": ("hbm", 0.0, 0.0),
    }


def step_model(cfg, seg):
    """Whole-step algorithmic flops / bytes per token (forward + recompute + backward)."""
    H, P, N, G, Q = cfg.H, cfg.P, cfg.N, cfg.G, cfg.chunk
    e = 2 if cfg.dtype == "bf16" else 4
    k = kappa(Q)
    HPN = H * P * N
    flops = (4 * HPN + 2 * k * Q * (G * N + H * P)) + 2 * HPN + (8 * HPN + 2 * k * Q * (3 * G * N + 2 * H * P))
    byts = e * (6 * H * P + 7 * G * N) + 16 * H + 2 * 4.0 * HPN / seg
    return flops, byts


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------- DRAM traffic from ncu
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the `ncu --set full` capture summarised in
# profiles/ncu_full_all_kernels_cfg2_geometry.txt, taken at workload 2's launch geometry (one launch = 4096 tokens x
# 80 heads).  A figure is used only while the kernel's source file still has the hash it had when the counters were
# taken; for the other workloads it is scaled by tokens x heads per launch (the traffic of these kernels grows in
# proportion).
NCU_TRAFFIC = {
    # kernel kind: (bytes per launch, source file, sha256 of that file at capture time)
    "bwd_dBdC": (139.4e6, "ssd_tc_bcf.cu", "dea27dee76a18e163bad504ab1ea872d692421f290753dcb7e87928a10f9f10c"),
    "bwd_dx": (165.8e6, "ssd_tc_scan.cu", "8456e62e2f5db54b7c0b95e493eead1031cbb85dbd1e34e93385165c68151b98"),
    "chunk_scan_fwd": (89.2e6, "ssd_tc_scan.cu", "8456e62e2f5db54b7c0b95e493eead1031cbb85dbd1e34e93385165c68151b98"),
    "chunk_state": (47.8e6, "ssd_tc.cu", "443a66c3f770fd0077e43b67055287dd8166d54e8c90b99a3bedc785227b7f08"),
    "dstate_contrib": (70.9e6, "ssd_tc.cu", "443a66c3f770fd0077e43b67055287dd8166d54e8c90b99a3bedc785227b7f08"),
    "state_pass_fwd": (45.4e6, "ssd_simt.cu", "701070c9421ce252f39d2b71218181c3ccaac7433187a73effa60c6cfa5de8f7"),
    "state_pass_bwd": (68.4e6, "ssd_simt.cu", "701070c9421ce252f39d2b71218181c3ccaac7433187a73effa60c6cfa5de8f7"),
}
NCU_UNITS = 4096 * 80


def ncu_traffic(kind, tokens_per_launch, heads):
    ent = NCU_TRAFFIC.get(kind)
    if not ent:
        return None
    import hashlib
    nbytes, src, sha = ent
    path = os.path.join(ROOT, "paper_2411_19460_b200", "csrc", src)
    try:
        cur = hashlib.sha256(open(path, "rb").read()).hexdigest()
    except OSError:
        return None
    if cur != sha:
        return None
    return nbytes * (tokens_per_launch * heads) / NCU_UNITS


# ----------------------------------------------------------------------------- clocks sampling
class ClockSampler:
    """SM clock and clock-event reasons sampled DURING the timed region: an NVML polling thread (a sample
    every few milliseconds, the first one at once), falling back to `nvidia-smi -lms` when NVML's Python
    binding is missing.  Read-only: nothing about the GPU is changed."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASON_BITS = (("sw_power_cap", 0x4), ("hw_slowdown", 0x8), ("sw_thermal_slowdown", 0x20),
                   ("hw_thermal_slowdown", 0x40))

    def __init__(self, device, period_s=0.002):
        self.proc = None
        self.path = None
        self.thread = None
        self.sm, self.mx, self.reasons = [], [], set()
        self._stop = threading.Event()
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
        except Exception:
            return
        try:
            import pynvml
            pynvml.nvmlInit()
            handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            mx = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            get_reasons = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(pynvml, "nvmlDeviceGetCurrentClocksThrottleReasons")

            def poll():
                while True:
                    try:
                        self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(handle, pynvml.NVML_CLOCK_SM)))
                        self.mx.append(mx)
                        bits = int(get_reasons(handle))
                        for name, bit in self.REASON_BITS:
                            if bits & bit:
                                self.reasons.add(name)
                    except Exception:
                        pass
                    if self._stop.wait(period_s):
                        return

            self.thread = threading.Thread(target=poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "--id=" + uuid, "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
            if self.sm:
                out.update(sm_mhz=statistics.median(self.sm), sm_max_mhz=max(self.mx), samples=len(self.sm),
                           source="nvml")
            out["reasons"] = sorted(self.reasons)
            return out
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [s.strip() for s in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[4:8]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm), source="nvidia-smi")
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------- the GPU arm
def run_ours(args):
    from paper_2411_19460_b200 import libssd

    from paper_2411_19460_b200.replicas import Replicas

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    rep = Replicas(backend="nccl", device=dev)
    rank, world = rep.rank, rep.world
    if args.gpus != world:
        raise SystemExit("bench.py: --gpus %d but %d rank(s) were launched (WORLD_SIZE); start it with "
                         "python -m torch.distributed.run --nproc-per-node %d" % (args.gpus, world, args.gpus))
    headline = args.config is None
    if headline:
        args.config = HEADLINE_CONFIG
    cfg = CONFIGS[args.config]
    if args.heads:
        cfg = cfg.scaled(H=args.heads, name="%s_h%d" % (cfg.name, args.heads))
        CONFIGS[args.config] = cfg
    if args.len:
        cfg = cfg.scaled(L=args.len, name="%s_L%d" % (cfg.name, args.len))
        CONFIGS[args.config] = cfg
    if args.stream_len:
        return run_stream(args, rep, dev)
    if args.conv:
        return run_conv(args, rep, dev)
    if args.gated_norm:
        return run_gated_norm(args, rep, dev)
    if cfg.layers != 1:
        return run_stack(args, rep, dev)
    line = measure_layer(args, rep, dev, cfg, full=True)
    if headline:
        # the other single-layer workloads from the same run, device-timed only, so that rounds stay comparable
        also = {}
        for ci in ALSO_CONFIGS:
            torch.cuda.empty_cache()
            sub = measure_layer(args, rep, dev, CONFIGS[ci], full=False)
            if sub is not None:
                also[sub["config"]["workload"]] = {k: sub[k] for k in ("value", "unit", "ms_per_step", "dtype",
                                                                         "config", "step_roofline", "gpu_launches")}
        if line is not None:
            line["also"] = also
    if line is not None:
        print(json.dumps(line))
    rep.close()


def measure_layer(args, rep, dev, cfg, full=True):
    """One single-layer workload: the device-resident timing of the step and its roofline; with `full` also the
    per-kernel-kind table, the end-to-end leg through host buffers and the CPU baseline.  Returns the JSON line as a
    dict on rank 0, None elsewhere."""
    from paper_2411_19460_b200 import libssd

    rank, world = rep.rank, rep.world
    seg = args.seg or cfg.seg
    flags = (libssd.SSD_FLAG_FORCE_SIMT if args.simt else 0) | (libssd.SSD_FLAG_SERIAL if args.serial else 0)
    inp = make_inputs(cfg, dev, seed=cfg.seed + rank)
    x, dt, A, Bm, Cm, D, h0, dy = (inp[k] for k in ("x", "dt", "A", "Bm", "Cm", "D", "h0", "dy"))
    B, L, H, P = x.shape
    N = Bm.shape[3]
    tokens = B * L

    shape = libssd.make_shape(x, Bm, cfg.chunk, seg, flags)
    ws_f = libssd.alloc_workspace(shape, libssd.SSD_OP_FWD_SEG, dev)
    ws_b = libssd.alloc_workspace(shape, libssd.SSD_OP_BWD_SEG, dev)
    nseg = (L + seg - 1) // seg
    y = torch.empty_like(x)
    hf = torch.empty(B, H, P, N, dtype=torch.float32, device=dev)
    bd = torch.empty(B, nseg, H, P, N, dtype=torch.float32, device=dev)
    out = dict(dx=torch.empty_like(x), ddt=torch.empty_like(dt), dA=torch.empty(H, device=dev),
               dB=torch.empty_like(Bm), dC=torch.empty_like(Cm), dD=torch.empty(H, device=dev),
               dh0=torch.empty(B, H, P, N, dtype=torch.float32, device=dev))
    stream = torch.cuda.current_stream()

    def step(src=None, dst=None):
        s = inp if src is None else src
        d = dict(y=y, h_final=hf, out=out) if dst is None else dst
        libssd.ssd_fwd_segmented(s["x"], s["dt"], s["A"], s["Bm"], s["Cm"], s["D"], s["h0"],
                                 chunk=cfg.chunk, seg=seg, flags=flags, y=d["y"], h_final=d["h_final"], boundary=bd,
                                 ws=ws_f, stream=stream)
        libssd.ssd_bwd_segmented(s["x"], s["dt"], s["A"], s["Bm"], s["Cm"], s["D"], bd, s["dy"], None,
                                 chunk=cfg.chunk, seg=seg, flags=flags, out=d["out"], ws=ws_b, stream=stream)

    barrier = rep.barrier
    max_over_ranks = rep.max_over_ranks

    # ---- device-resident timing
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    run_step = step
    graph = None
    if args.graph:
        # the whole step (several hundred launches) captured once and replayed: the library only enqueues
        # on the caller's stream, so it can be captured as it is
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            stream_g = torch.cuda.current_stream()
            def step_on_side():
                libssd.ssd_fwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], inp["h0"],
                                         chunk=cfg.chunk, seg=seg, flags=flags, y=y, h_final=hf, boundary=bd,
                                         ws=ws_f, stream=stream_g)
                libssd.ssd_bwd_segmented(inp["x"], inp["dt"], inp["A"], inp["Bm"], inp["Cm"], inp["D"], bd, inp["dy"],
                                         None, chunk=cfg.chunk, seg=seg, flags=flags, out=out, ws=ws_b, stream=stream_g)
            step_on_side()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            nc0 = libssd.launch_count()
            with torch.cuda.graph(graph, stream=side):
                step_on_side()
            launches_per_replay = libssd.launch_count() - nc0      # kernel nodes of the captured step
        torch.cuda.synchronize()
        run_step = graph.replay
        for _ in range(3):
            run_step()
        barrier()
    torch.cuda.reset_peak_memory_stats(dev)
    sampler = ClockSampler(dev) if rank == 0 else None
    n0 = libssd.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        run_step()
    e1.record(stream)
    barrier()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    launches = libssd.launch_count() - n0
    if graph is not None:
        launches = launches_per_replay * args.steps
    clocks = sampler.stop() if sampler else None
    peak_mem = torch.cuda.max_memory_allocated(dev)
    assert libssd.poll_status(ws_f) == 0 and libssd.poll_status(ws_b) == 0, "device-side wait timed out"
    ms_per_step = ms_total / args.steps
    value = world * tokens / (ms_per_step * 1e-3)

    fl, by = step_model(cfg, seg)
    peaks = load_peaks()
    if cfg.dtype == "bf16":
        t_roof = max(fl * tokens / (peaks["bf16_tflops"] * 1e12), by * tokens / (peaks["hbm_gbs"] * 1e9))
        step_roof = dict(flops_per_token=fl, bytes_per_token=by, roofline_ms=t_roof * 1e3,
                         frac=t_roof * 1e3 / ms_per_step, peaks="bf16 tensor (burst) and HBM copy, " + peaks["source"])
    else:
        # fp32 mode runs on the CUDA cores (TF32 cannot hold 1e-4): its flop roof is the plain FFMA rate, measured here
        ffma = measure_ffma_tflops(dev)
        t_roof = max(fl * tokens / (ffma * 1e12), by * tokens / (peaks["hbm_gbs"] * 1e9))
        step_roof = dict(flops_per_token=fl, bytes_per_token=by, roofline_ms=t_roof * 1e3,
                         frac=t_roof * 1e3 / ms_per_step, ffma_tflops=ffma,
                         peaks="fp32 FFMA rate measured by an fp32 matrix product with TF32 off, and HBM copy",
                         note="%d tokens: the roofline time is a few microseconds, below the cost of launching the "
                              "step's kernels; the configuration is launch-bound" % tokens)
    if not full:
        del graph
        if rank != 0:
            return None
        return {"value": value, "unit": UNIT, "ms_per_step": ms_per_step,
                "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
                "config": {"workload": cfg.name, "B": B, "L": L, "H": H, "P": P, "N": N, "G": cfg.G,
                           "chunk": cfg.chunk, "seg": seg, "nseg": nseg,
                           "launch": "cuda graph replay" if args.graph else "stream launches"},
                "step_roofline": step_roof, "gpu_launches": int(launches)}

    # ---- per-kernel-kind timing (CUDA events on the launch stream, separate pass of the same steps)
    prof_steps = min(args.steps, 3)
    libssd.profile(True)
    for _ in range(prof_steps):
        step()
    torch.cuda.synchronize()
    prof = libssd.profile_read()
    libssd.profile(False)

    # ---- end to end: pinned host buffers -> device -> C ABI -> results back to pinned host, every step.
    # The three legs of a step run on three streams (copy in | the library's calls | copy out) over two sets of
    # device buffers, so that consecutive steps overlap the way an input pipeline does: PCIe carries step i+1's
    # inputs in while step i's results go out (the link is full duplex) and the kernels run under both.
    e2e = None
    if not args.no_e2e:
        names_in = [k for k in ("x", "dt", "A", "Bm", "Cm", "D", "h0", "dy") if inp[k] is not None]
        host_in = {k: torch.empty(inp[k].shape, dtype=inp[k].dtype, pin_memory=True).copy_(inp[k])
                   for k in names_in}
        dev_in = []
        for _ in range(2):
            di = {k: torch.empty_like(inp[k]) for k in names_in}
            di["h0"] = di.get("h0")
            dev_in.append(di)
        dsts = [dict(y=y, h_final=hf, out=out),
                dict(y=torch.empty_like(y), h_final=torch.empty_like(hf), out={k: torch.empty_like(v) for k, v in out.items()})]
        flat = lambda d: dict(y=d["y"], h_final=d["h_final"], **d["out"])
        host_out = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in flat(dsts[0]).items()}
        bi = sum(t.numel() * t.element_size() for t in host_in.values())
        bo = sum(t.numel() * t.element_size() for t in host_out.values())
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_done = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def e2e_run(nsteps):
            s_in.wait_stream(stream)
            s_out.wait_stream(stream)
            for i in range(nsteps):
                b = i & 1
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_done[b])        # step i-2 has consumed this set of inputs
                    for k in names_in:
                        dev_in[b][k].copy_(host_in[k], non_blocking=True)
                    ev_in[b].record(s_in)
                stream.wait_event(ev_in[b])
                if i >= 2:
                    stream.wait_event(ev_out[b])           # step i-2's results have left this set of outputs
                step(dev_in[b], dsts[b])
                ev_done[b].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_done[b])
                    for k, v in flat(dsts[b]).items():
                        host_out[k].copy_(v, non_blocking=True)
                    ev_out[b].record(s_out)
            stream.wait_stream(s_out)                      # the last results are in host memory

        e2e_steps = max(1, min(args.steps, 6))
        e2e_run(2)
        barrier()
        e0.record(stream)
        e2e_run(e2e_steps)
        e1.record(stream)
        barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
        e2e = dict(value=world * tokens / (ms_e2e * 1e-3), unit=UNIT, h2d_bytes_per_step=bi,
                   d2h_bytes_per_step=bo, ms_per_step=ms_e2e, steps=e2e_steps,
                   pipeline="copy-in, compute and copy-out streams over two sets of device buffers")
        del host_in, host_out, dev_in, dsts

    if rank != 0:
        return None

    model = kind_model(cfg)
    # dominant kernel kind = largest share of device time
    total_prof = sum(v[0] for v in prof.values()) or 1.0
    dom = max(prof, key=lambda k: prof[k][0])
    dom_ms, dom_n = prof[dom]
    bound, fl_tok, by_tok = model[dom]
    tok_per_launch = tokens * prof_steps / max(dom_n, 1)
    avg_s = dom_ms * 1e-3 / max(dom_n, 1)
    peak_kind = "HBM copy"
    if bound == "tensor" and cfg.dtype != "bf16":
        # the fp32 mode runs these contractions on the CUDA cores: plain-ALU bound, against the measured FFMA rate
        bound = "alu"
        achieved = fl_tok * tok_per_launch / avg_s / 1e12
        peak = measure_ffma_tflops(dev)
        unit = "TFLOP/s"
        peak_kind = "fp32 FFMA (fp32 matrix product, TF32 off)"
    elif bound == "tensor":
        achieved = fl_tok * tok_per_launch / avg_s / 1e12
        peak = peaks["bf16_tflops"]        # a launch timed by itself with CUDA events: the burst figure
        unit = "TFLOP/s"
        peak_kind = "bf16 matmul, burst"
    else:
        achieved = by_tok * tok_per_launch / avg_s / 1e9
        peak = peaks["hbm_gbs"]
        unit = "GB/s"
    roofline = dict(kernel=dom, bound=bound if bound in ("tensor", "alu") else "hbm", achieved=achieved, peak=peak,
                    unit=unit, frac=achieved / peak, traffic=ncu_traffic(dom, tok_per_launch, H),
                    peak_source=peaks["source"],
                    peak_kind=peak_kind,
                    avg_launch_us=avg_s * 1e6, launches=dom_n, share_of_device_time=dom_ms / total_prof)
    kinds = {k: dict(ms_per_step=v[0] / prof_steps, launches_per_step=v[1] / prof_steps,
                     share=v[0] / total_prof) for k, v in prof.items() if v[1]}

    cpu = None
    if not args.no_cpu:
        cpu = cpu_baseline(cfg, inp, sample_tokens=args.cpu_tokens)

    io_bytes = sum(t.numel() * t.element_size() for t in (x, dt, Bm, Cm, dy, y, out["dx"], out["ddt"],
                                                         out["dB"], out["dC"]))
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
        "data": "synthetic", "impl": "ours",
        "config": {"workload": cfg.name, "B": B, "L": L, "H": H, "P": P, "N": N, "G": cfg.G,
                   "chunk": cfg.chunk, "seg": seg, "nseg": nseg, "l2": "inputs larger than L2",
                   "path": "simt" if (args.simt or cfg.dtype == "fp32") else "default",
                   "launch": "cuda graph replay" if args.graph else "stream launches",
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "step_roofline": step_roof, "kernels": kinds,
        "memory": {"peak_allocated_bytes": int(peak_mem), "workspace_fwd_bytes": ws_f.numel(),
                   "workspace_bwd_bytes": ws_b.numel(), "boundary_bytes": bd.numel() * 4,
                   "io_bytes": int(io_bytes)},
        "cpu_baseline": cpu,
    }
    return line


_FFMA = {}


def measure_ffma_tflops(dev):
    """fp32 multiply-add rate of the CUDA cores: the best of five 4096^3 fp32 matrix products with TF32 disabled."""
    if dev in _FFMA:
        return _FFMA[dev]
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        n = 4096
        a = torch.randn(n, n, device=dev)
        b = torch.randn(n, n, device=dev)
        best = float("inf")
        for _ in range(6):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch.matmul(a, b)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        _FFMA[dev] = 2.0 * n ** 3 / (best * 1e-3) / 1e12
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old
    return _FFMA[dev]


# ----------------------------------------------------------------------------- the stacked configuration
def run_stack(args, rep, dev):
    """Config 3: 64 stacked layers under MA-GC (layer inputs + segment-boundary states kept), one step =
    Algorithm 1 forward + Algorithm 2 backward of the whole stack.  At layer interval 1 the literal
    L = 262144 needs 175 GB of layer inputs alone, so it is run at --stack-len (default 131072) and the line
    says so; with --layer-interval 2 or more (Eq. 4's l) the literal length fits and is the default."""
    from paper_2411_19460_b200 import libssd
    from paper_2411_19460_b200.inputs import make_stack_params
    from paper_2411_19460_b200.stack import LayerStack
    from paper_2411_19460_b200.memory_model import layer_stack_bytes

    base = CONFIGS[args.config]
    L = args.stack_len or (131072 if args.layer_interval == 1 else base.L)
    cfg = base.scaled(L=L, seg=args.seg or base.seg, layers=args.layers or base.layers)
    inp = make_inputs(cfg, dev, seed=cfg.seed + rep.rank)
    sp = make_stack_params(cfg, dev)
    st = LayerStack(inp["x"], inp["dt"], inp["Bm"], inp["Cm"], sp["A"], sp["D"], sp["W"], chunk=cfg.chunk, seg=cfg.seg,
                    layer_interval=args.layer_interval, flags=(libssd.SSD_FLAG_SERIAL if args.serial else 0))
    for j in range(cfg.layers):          # every layer starts from its own N(0, h0_std^2) state, as the workload says
        st.set_h0(j, sp["h0"][j])
    out = dict(dx0=torch.empty_like(inp["x"]), dA=torch.zeros(cfg.layers, cfg.H, device=dev),
               dD=torch.zeros(cfg.layers, cfg.H, device=dev))
    stream = torch.cuda.current_stream()

    def step():
        out["dA"].zero_()
        out["dD"].zero_()
        st.forward()
        st.backward(inp["dy"], out=out)

    for _ in range(max(args.warmup, 1)):
        step()
    rep.barrier()
    torch.cuda.reset_peak_memory_stats(dev)
    sampler = ClockSampler(dev) if rep.rank == 0 else None
    n0 = libssd.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rep.barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    rep.barrier()
    ms = rep.max_over_ranks(e0.elapsed_time(e1)) / args.steps
    launches = libssd.launch_count() - n0
    clocks = sampler.stop() if sampler else None
    peak_mem = torch.cuda.max_memory_allocated(dev)
    if rep.rank != 0:
        rep.close()
        return
    peaks = load_peaks()
    fl, by = step_model(cfg, cfg.seg)
    glue_bytes = 2 * (3 + 2) * cfg.H * cfg.P              # forward x, y -> x_next; backward g -> dz (dx += dz is folded into the dx kernel)
    t_roof = cfg.layers * cfg.L * max(fl / (peaks["bf16_tflops"] * 1e12), (by + glue_bytes) / (peaks["hbm_gbs"] * 1e9))
    value = rep.world * cfg.L / (ms * 1e-3)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": rep.world, "steps": args.steps,
        "warmup": max(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "impl": "ours",
        "config": {"workload": cfg.name, "B": cfg.B, "L": cfg.L, "L_in_definition": base.L, "layers": cfg.layers,
                   "H": cfg.H, "P": cfg.P, "N": cfg.N, "G": cfg.G, "chunk": cfg.chunk, "seg": cfg.seg, "layer_interval": args.layer_interval,
                   "layer_tokens_per_s": value * cfg.layers, "l2": "inputs larger than L2",
                   "parallelism": "replicas" if rep.world > 1 else "single"},
        "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
        "step_roofline": {"roofline_ms": t_roof * 1e3, "frac": t_roof * 1e3 / ms},
        "memory": dict(peak_allocated_bytes=int(peak_mem), **st.checkpoint_bytes()),
        "memory_model": layer_stack_bytes(cfg.layers, cfg.L, args.layer_interval, cfg.seg, cfg.H, cfg.P, cfg.N),
    }
    print(json.dumps(line))
    rep.close()


def run_stream(args, rep, dev):
    """Forward-only streaming over --stream-len tokens (default 2^21) of the configuration's layer: ssd_fwd
    segment by segment with only the state carried, then single-token steps on the same state.  Scratch is
    one segment's; nothing grows with the length but the input and output themselves."""
    from paper_2411_19460_b200 import libssd

    base = CONFIGS[args.config]
    L = args.stream_len
    seg = args.seg or 16384
    cfg = base.scaled(L=L, seg=seg)
    inp = make_inputs(cfg, dev, seed=cfg.seed + rep.rank)
    x, dt, A, Bm, Cm, D = (inp[k] for k in ("x", "dt", "A", "Bm", "Cm", "D"))
    B, _, H, P = x.shape
    N = Bm.shape[3]
    y = torch.empty_like(x)
    h = torch.zeros(B, H, P, N, dtype=torch.float32, device=dev)
    h2 = torch.zeros_like(h)
    cell = libssd.make_shape(x[:, :seg], Bm[:, :seg], cfg.chunk, seg, 0)
    ws = libssd.alloc_workspace(cell, libssd.SSD_OP_FWD, dev)
    assert B == 1, "slices of the sequence are passed as offset pointers: batch 1"
    nseg = L // seg
    views = [(x[:, k * seg:(k + 1) * seg], dt[:, k * seg:(k + 1) * seg], Bm[:, k * seg:(k + 1) * seg],
              Cm[:, k * seg:(k + 1) * seg], y[:, k * seg:(k + 1) * seg]) for k in range(nseg)]
    stream = torch.cuda.current_stream()

    def step():
        hin, hout = None, h
        for xs, dts, Bs, Cs, ys in views:
            libssd.ssd_fwd(xs, dts, A, Bs, Cs, D, hin, chunk=cfg.chunk, seg=seg, y=ys, h_final=hout, ws=ws, stream=stream)
            hin, hout = hout, (h2 if hout is h else h)

    for _ in range(max(args.warmup, 1)):
        step()
    rep.barrier()
    torch.cuda.reset_peak_memory_stats(dev)
    sampler = ClockSampler(dev) if rep.rank == 0 else None
    n0 = libssd.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rep.barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    rep.barrier()
    ms = rep.max_over_ranks(e0.elapsed_time(e1)) / args.steps
    launches = libssd.launch_count() - n0
    clocks = sampler.stop() if sampler else None
    peak_mem = torch.cuda.max_memory_allocated(dev)
    assert libssd.poll_status(ws) == 0
    # single-token steps, captured in a graph of 64 so that launch latency is the GPU's, not Python's
    tok = [(x[:, t:t + 1].contiguous(), dt[:, t:t + 1].contiguous(), Bm[:, t:t + 1].contiguous(),
            Cm[:, t:t + 1].contiguous(), torch.empty(B, 1, H, P, dtype=x.dtype, device=dev)) for t in range(64)]
    side = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(side):
        sg = torch.cuda.current_stream()
        for xt, dtt, Bt, Ct, yt in tok[:2]:
            libssd.ssd_decode_step(xt, dtt, A, Bt, Ct, D, h, y=yt, stream=sg)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for xt, dtt, Bt, Ct, yt in tok:
                libssd.ssd_decode_step(xt, dtt, A, Bt, Ct, D, h, y=yt, stream=sg)
    torch.cuda.synchronize()
    for _ in range(3):
        g.replay()
    e0.record(stream)
    for _ in range(20):
        g.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    us_per_token = e0.elapsed_time(e1) * 1e3 / (20 * 64)
    if rep.rank != 0:
        rep.close()
        return
    peaks = load_peaks()
    state_bytes = 2 * B * H * P * N * 4
    e = x.element_size()
    fwd_bytes = (2 * H * P + 2 * cfg.G * N) * e + 4 * H            # per token: x, y, B, C, dt
    line = {
        "metric": "ssd_fwd_stream_tokens_per_s", "value": rep.world * L / (ms * 1e-3), "unit": UNIT, "n_gpus": rep.world,
        "steps": args.steps, "warmup": max(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if e == 2 else "f32", "data": "synthetic", "impl": "ours",
        "config": {"workload": cfg.name + "_forward_stream", "B": B, "L": L, "H": H, "P": P, "N": N, "G": cfg.G,
                   "chunk": cfg.chunk, "seg": seg, "l2": "inputs larger than L2",
                   "parallelism": "replicas" if rep.world > 1 else "single"},
        "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": fwd_bytes * L / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": fwd_bytes * L / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                     "peak_source": peaks["source"]},
        "decode_step": {"us_per_token": us_per_token, "state_bytes_per_token": state_bytes,
                        "achieved_gbs": state_bytes / (us_per_token * 1e-6) / 1e9, "launch": "cuda graph of 64 steps"},
        "memory": {"peak_allocated_bytes": int(peak_mem), "workspace_bytes": ws.numel(), "state_bytes": h.numel() * 4,
                   "io_bytes": int(sum(t.numel() * t.element_size() for t in (x, dt, Bm, Cm, y)))},
    }
    print(json.dumps(line))
    rep.close()


def run_conv(args, rep, dev):
    """The depthwise causal conv + SiLU stage in front of the SSD layer, forward and backward segment by segment with
    its three-input state carried across the cuts (channels = d_inner + 2 G N of the configuration)."""
    from paper_2411_19460_b200 import libssd

    cfg = CONFIGS[args.config]
    seg = args.seg or cfg.seg
    B, L, C = cfg.B, cfg.L, cfg.H * cfg.P + 2 * cfg.G * cfg.N
    td = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    gen = torch.Generator(device=dev).manual_seed(cfg.seed + rep.rank)
    u = torch.randn(B, L, C, generator=gen, device=dev, dtype=torch.float32).to(td)
    g = torch.randn(B, L, C, generator=gen, device=dev, dtype=torch.float32).to(td)
    w = torch.randn(C, 4, generator=gen, device=dev) * 0.5
    bias = torch.randn(C, generator=gen, device=dev) * 0.1
    out, du = torch.empty_like(u), torch.empty_like(u)
    nseg = L // seg
    assert B == 1 and L % seg == 0, "segments are passed as offset pointers: batch 1, L a multiple of seg"
    states = torch.zeros(nseg + 1, B, 3, C, dtype=td, device=dev)
    dst = torch.zeros(2, B, 3, C, dtype=torch.float32, device=dev)
    dw, db = torch.zeros(C, 4, device=dev), torch.zeros(C, device=dev)
    ws = torch.empty(int(libssd.lib().ssd_conv_workspace_bytes(B, seg, C)), dtype=torch.uint8, device=dev)
    sl = [(u[:, k * seg:(k + 1) * seg], g[:, k * seg:(k + 1) * seg], out[:, k * seg:(k + 1) * seg],
           du[:, k * seg:(k + 1) * seg]) for k in range(nseg)]
    stream = torch.cuda.current_stream()

    def step():
        for k in range(nseg):
            libssd.ssd_conv_fwd(sl[k][0], w, bias, states[k], out=sl[k][2], state_out=states[k + 1], stream=stream)
        dw.zero_()
        db.zero_()
        for k in range(nseg - 1, -1, -1):
            cur = (nseg - 1 - k) & 1
            libssd.ssd_conv_bwd(sl[k][0], w, bias, states[k], sl[k][1], None if k == nseg - 1 else dst[cur],
                                du=sl[k][3], dstate=dst[1 - cur], dw=dw, dbias=db, accumulate=True, ws=ws, stream=stream)

    for _ in range(max(args.warmup, 3)):
        step()
    rep.barrier()
    run_step, per_replay = step, None
    if args.graph:
        # the per-segment calls are short: replay them from a CUDA graph so that the host does not pace them
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            stream = torch.cuda.current_stream()
            step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            nc0 = libssd.launch_count()
            with torch.cuda.graph(graph, stream=side):
                step()
            per_replay = libssd.launch_count() - nc0
        stream = torch.cuda.current_stream()
        torch.cuda.synchronize()
        run_step = graph.replay
        for _ in range(3):
            run_step()
    sampler = ClockSampler(dev) if rep.rank == 0 else None
    n0 = libssd.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rep.barrier()
    e0.record(stream)
    for _ in range(args.steps):
        run_step()
    e1.record(stream)
    rep.barrier()
    ms = rep.max_over_ranks(e0.elapsed_time(e1)) / args.steps
    launches = per_replay * args.steps if per_replay is not None else libssd.launch_count() - n0
    clocks = sampler.stop() if sampler else None
    if rep.rank != 0:
        rep.close()
        return
    peaks = load_peaks()
    e = u.element_size()
    byts = 5 * e * C                       # fwd: u in, out out; bwd: u, dout in, du out
    ach = byts * B * L / (ms * 1e-3) / 1e9
    line = {
        "metric": "conv1d_fwd_bwd_segmented_tokens_per_s", "value": rep.world * B * L / (ms * 1e-3), "unit": UNIT,
        "n_gpus": rep.world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "impl": "ours",
        "config": {"workload": cfg.name + "_conv1d", "B": B, "L": L, "channels": C, "width": 4, "seg": seg, "nseg": nseg,
                   "launch": "cuda graph replay" if args.graph else "stream launches", "l2": "inputs larger than L2", "parallelism": "replicas" if rep.world > 1 else "single"},
        "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
        "roofline": {"kernel": "conv1d fwd+bwd", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"]},
    }
    print(json.dumps(line))
    rep.close()


def run_gated_norm(args, rep, dev):
    """The gated RMS normalisation behind the SSD layer, forward and backward segment by segment (token-local: nothing
    is carried across the cuts; dgamma is summed over the segments)."""
    from paper_2411_19460_b200 import libssd

    cfg = CONFIGS[args.config]
    seg = args.seg or cfg.seg
    B, L, D = cfg.B, cfg.L, cfg.H * cfg.P
    group = D // cfg.G
    td = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    gen = torch.Generator(device=dev).manual_seed(cfg.seed + rep.rank)
    y = torch.randn(B * L, D, generator=gen, device=dev, dtype=torch.float32).to(td)
    z = torch.randn(B * L, D, generator=gen, device=dev, dtype=torch.float32).to(td)
    g = torch.randn(B * L, D, generator=gen, device=dev, dtype=torch.float32).to(td)
    gamma = 1.0 + 0.1 * torch.randn(D, generator=gen, device=dev)
    out, dy, dz = torch.empty_like(y), torch.empty_like(y), torch.empty_like(y)
    dg = torch.zeros(D, device=dev)
    rows = B * seg
    nseg = (B * L) // rows
    ws = torch.empty(int(libssd.lib().ssd_gated_norm_workspace_bytes(rows, D)), dtype=torch.uint8, device=dev)
    sl = [slice(k * rows, (k + 1) * rows) for k in range(nseg)]
    stream = torch.cuda.current_stream()

    def step():
        for k in range(nseg):
            libssd.ssd_gated_norm_fwd(y[sl[k]], z[sl[k]], gamma, group=group, out=out[sl[k]], stream=stream)
        dg.zero_()
        for k in range(nseg - 1, -1, -1):
            libssd.ssd_gated_norm_bwd(y[sl[k]], z[sl[k]], gamma, g[sl[k]], group=group, dy=dy[sl[k]], dz=dz[sl[k]], dgamma=dg,
                                      accumulate=True, ws=ws, stream=stream)

    for _ in range(max(args.warmup, 3)):
        step()
    rep.barrier()
    run_step, per_replay = step, None
    if args.graph:
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            stream = torch.cuda.current_stream()
            step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            nc0 = libssd.launch_count()
            with torch.cuda.graph(graph, stream=side):
                step()
            per_replay = libssd.launch_count() - nc0
        stream = torch.cuda.current_stream()
        torch.cuda.synchronize()
        run_step = graph.replay
        for _ in range(3):
            run_step()
    sampler = ClockSampler(dev) if rep.rank == 0 else None
    n0 = libssd.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rep.barrier()
    e0.record(stream)
    for _ in range(args.steps):
        run_step()
    e1.record(stream)
    rep.barrier()
    ms = rep.max_over_ranks(e0.elapsed_time(e1)) / args.steps
    launches = per_replay * args.steps if per_replay is not None else libssd.launch_count() - n0
    clocks = sampler.stop() if sampler else None
    if rep.rank != 0:
        rep.close()
        return
    peaks = load_peaks()
    e = y.element_size()
    ach = 8 * e * D * B * L / (ms * 1e-3) / 1e9           # fwd: y, z in, out out; bwd: y, z, dout in, dy, dz out
    line = {
        "metric": "gated_norm_fwd_bwd_segmented_tokens_per_s", "value": rep.world * B * L / (ms * 1e-3), "unit": UNIT,
        "n_gpus": rep.world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "impl": "ours",
        "config": {"workload": cfg.name + "_gated_norm", "B": B, "L": L, "channels": D, "group": group, "seg": seg,
                   "nseg": nseg, "launch": "cuda graph replay" if args.graph else "stream launches",
                   "l2": "inputs larger than L2", "parallelism": "replicas" if rep.world > 1 else "single"},
        "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
        "roofline": {"kernel": "gated_norm fwd+bwd", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"]},
    }
    print(json.dumps(line))
    rep.close()


# ----------------------------------------------------------------------------- the CPU oracle legs
def _oracle_sample(cfg, inp, sample_tokens):
    """fp64 host copies of the first `sample_tokens` tokens (all heads) of the workload."""
    Ls = min(cfg.L, sample_tokens)
    sub = {k: (v[:, :Ls] if (v is not None and k in ("x", "dt", "Bm", "Cm", "dy")) else v)
           for k, v in inp.items()}
    return to_f64_numpy(sub), Ls


def _time_oracle(d):
    from oracle import ssd_oracle as orc
    t0 = time.perf_counter()
    y, hf, bd = orc.ssd_fwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], seg=1024)
    orc.ssd_bwd(d["x"], d["dt"], d["A"], d["Bm"], d["Cm"], d["D"], d["h0"], d["dy"], None, blk=256)
    return time.perf_counter() - t0


def cpu_baseline(cfg, inp, sample_tokens):
    from oracle import ssd_oracle as orc
    d, Ls = _oracle_sample(cfg, inp, sample_tokens)
    secs = _time_oracle(d)
    return dict(value=cfg.B * Ls / secs, unit=UNIT, cores=orc.threads(), kind="oracle",
                sample="first %d of %d tokens, all %d heads, fwd+bwd once (%.1f s)" % (Ls, cfg.L, cfg.H, secs))


def run_reference(args):
    """The oracle as the reference arm: each step is fwd+bwd over a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ssd_oracle as orc
    cfg = CONFIGS[HEADLINE_CONFIG if args.config is None else args.config]
    seg = args.seg or cfg.seg
    Ls = min(cfg.L, args.ref_tokens)
    small = cfg.scaled(L=Ls)
    inp = make_inputs(small, "cpu")
    d = to_f64_numpy(inp)
    for _ in range(args.warmup):
        _time_oracle(d)
    t = [_time_oracle(d) for _ in range(args.steps)]
    secs = sum(t) / len(t)
    value = cfg.B * Ls / secs
    sample = "first %d of %d tokens, all %d heads, per step" % (Ls, cfg.L, cfg.H)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
        "config": {"workload": cfg.name, "B": cfg.B, "L": cfg.L, "H": cfg.H, "P": cfg.P, "N": cfg.N,
                   "G": cfg.G, "chunk": cfg.chunk, "seg": seg, "sampled_tokens": Ls},
        "cpu_baseline": dict(value=value, unit=UNIT, cores=orc.threads(), kind="oracle", sample=sample),
        "e2e": dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=6)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None, help="index into the five workloads (default: the largest "
                    "single-layer one, 4, with workloads 2 and 0 reported beside it)")
    ap.add_argument("--seg", type=int, default=0, help="override the segment length")
    ap.add_argument("--simt", action="store_true", help="force the CUDA-core kernels")
    ap.add_argument("--layer-interval", type=int, default=1, help="config 3: keep the input of every l-th layer")
    ap.add_argument("--stack-len", type=int, default=0, help="config 3: sequence length (default 131072 at layer interval 1, else the configuration's own)")
    ap.add_argument("--stream-len", type=int, default=0, help="forward-only streaming over this many tokens "
                    "(e.g. 2097152) instead of the training step")
    ap.add_argument("--conv", action="store_true", help="time the depthwise conv + SiLU stage (forward + backward, "
                    "segment by segment) instead of the SSD step")
    ap.add_argument("--gated-norm", action="store_true", help="time the gated RMS normalisation stage (forward + backward, "
                    "segment by segment) instead of the SSD step")
    ap.add_argument("--heads", type=int, default=0, help="override the head count (32 / 64: the 370M / 1.3B model sizes)")
    ap.add_argument("--len", type=int, default=0, help="override the sequence length (a short prefix of the workload, "
                    "e.g. for a profiler capture of one kernel at the workload's launch geometry)")
    ap.add_argument("--layers", type=int, default=0, help="config 3: number of layers (default 64)")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="time plain stream launches instead of the replay of the step captured in a CUDA graph")
    ap.add_argument("--serial", action="store_true", help="no helper streams: every kernel of the forward and the backward in order on one stream")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-tokens", type=int, default=32768, help="tokens in the cpu_baseline sample")
    ap.add_argument("--ref-tokens", type=int, default=8192, help="tokens per step of --impl reference")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
