"""Seeded synthetic inputs for the SSD layer: the only module shared by the CUDA path's
tests/bench and the CPU oracle's tests.  It holds shapes and random draws, none of the
method's arithmetic.

The tensors stand in for the video-token workload of the paper (1 frame/s x 144 tokens per
frame fed to a Mamba-2 backbone, Section 3.4; Mamba-2 370M/1.3B/2.7B head dimensions as
implied by the constants of Appendix C).  No dataset or trained weight is involved.

Recipe (drawn in this fixed order from one torch.Generator seeded with `seed`):
  x, Bm, Cm, dy ~ N(0,1) (Bm, Cm scaled by 1/sqrt(N));  z ~ N(0, 0.5^2) per (b,t,h);
  A_h = -exp(U(0, ln a_max));  u_h = exp(U(ln dt_lo, ln dt_hi)),
  bias_h = softplus^{-1}(u_h),  dt = softplus(z + bias_h) (fp32);
  D ~ N(0,1);  h0 ~ N(0, h0_std^2) (or zeros);  dh_final ~ N(0, dh_std^2) (zeros by default).
x, Bm, Cm, dy are then cast to the I/O dtype (bf16 or fp32); the cast values are what both
the GPU and the oracle consume.
"""
from dataclasses import dataclass, replace
import math

import torch


@dataclass(frozen=True)
class SSDConfig:
    name: str
    dtype: str          # "fp32" | "bf16": I/O type of x, Bm, Cm, y, dy, dx, dB, dC
    B: int
    L: int
    H: int
    P: int
    N: int
    G: int
    chunk: int
    seg: int
    a_max: float = 16.0     # A = -exp(U(0, ln a_max))
    dt_lo: float = 1e-3
    dt_hi: float = 1e-1
    h0_std: float = 0.0
    dh_std: float = 0.0
    seed: int = 0
    layers: int = 1

    @property
    def nseg(self) -> int:
        return (self.L + self.seg - 1) // self.seg

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def scaled(self, **kw) -> "SSDConfig":
        return replace(self, **kw)


# The five workloads named by the benchmark definition (index = config number).
CONFIGS = [
    SSDConfig("cfg0_fp32_small", "fp32", 1, 1024, 4, 64, 64, 1, 64, 256),
    SSDConfig("cfg1_130m_bf16", "bf16", 1, 16384, 24, 64, 128, 1, 256, 2048, h0_std=0.1),
    SSDConfig("cfg2_2p7b_bf16", "bf16", 1, 131072, 80, 64, 128, 1, 256, 4096, h0_std=0.1),
    SSDConfig("cfg3_2p7b_stack64_bf16", "bf16", 1, 262144, 80, 64, 128, 1, 256, 4096,
              h0_std=0.1, layers=64),
    SSDConfig("cfg4_million_bf16", "bf16", 1, 1048576, 80, 64, 128, 8, 256, 8192,
              a_max=64.0, dt_lo=1e-4, dt_hi=1.0, h0_std=0.1),
]


def make_inputs(cfg: SSDConfig, device="cpu", seed=None):
    """Returns a dict of tensors on `device`: x, dt, A, Bm, Cm, D, h0 (None when h0_std == 0),
    dy, dh_final (None when dh_std == 0)."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(cfg.seed if seed is None else seed)
    io = cfg.torch_dtype
    B, L, H, P, N, G = cfg.B, cfg.L, cfg.H, cfg.P, cfg.N, cfg.G

    def randn(*shape):
        return torch.randn(*shape, generator=g, device=dev, dtype=torch.float32)

    def rand(*shape):
        return torch.rand(*shape, generator=g, device=dev, dtype=torch.float32)

    x = randn(B, L, H, P).to(io)
    Bm = (randn(B, L, G, N) / math.sqrt(N)).to(io)
    Cm = (randn(B, L, G, N) / math.sqrt(N)).to(io)
    dy = randn(B, L, H, P).to(io)
    z = randn(B, L, H) * 0.5
    A = -torch.exp(rand(H) * math.log(cfg.a_max))
    u = torch.exp(math.log(cfg.dt_lo) + rand(H) * (math.log(cfg.dt_hi) - math.log(cfg.dt_lo)))
    bias = u + torch.log(-torch.expm1(-u))
    dt = torch.nn.functional.softplus(z + bias)
    del z
    D = randn(H)
    h0 = randn(B, H, P, N) * cfg.h0_std if cfg.h0_std > 0 else None
    dh_final = randn(B, H, P, N) * cfg.dh_std if cfg.dh_std > 0 else None
    return dict(x=x, dt=dt.contiguous(), A=A, Bm=Bm, Cm=Cm, D=D, h0=h0, dy=dy, dh_final=dh_final)


def to_f64_numpy(inp, heads=None, groups=None):
    """Host float64 copies of (optionally a head/group subset of) the generated tensors, for the
    oracle.  `heads` is a list of head indices, `groups` the matching list of group indices."""
    import numpy as np

    def cv(t):
        return None if t is None else t.detach().to("cpu", torch.float64).numpy()

    if heads is None:
        return {k: cv(v) for k, v in inp.items()}
    hi = torch.as_tensor(heads, device=inp["x"].device)
    gi = torch.as_tensor(groups, device=inp["x"].device)
    out = dict(
        x=cv(inp["x"].index_select(2, hi)), dt=cv(inp["dt"].index_select(2, hi)),
        A=cv(inp["A"].index_select(0, hi)), D=cv(inp["D"].index_select(0, hi)),
        Bm=cv(inp["Bm"].index_select(2, gi)), Cm=cv(inp["Cm"].index_select(2, gi)),
        dy=cv(inp["dy"].index_select(2, hi)),
        h0=None if inp["h0"] is None else cv(inp["h0"].index_select(1, hi)),
        dh_final=None if inp["dh_final"] is None else cv(inp["dh_final"].index_select(1, hi)),
    )
    return {k: (None if v is None else np.ascontiguousarray(v)) for k, v in out.items()}


def make_stack_params(cfg: SSDConfig, device="cpu", scale=None):
    """Per-layer A, D (seed + layer) and the fixed mixing matrix W of the stacked configuration.

    W = scale * Q0 with Q0 the orthogonal factor of a seeded Gaussian P x P matrix, rounded to bf16
    so that both sides use the same numbers; `scale` defaults to 0.5, which keeps the RMS of the layer
    inputs of order one over 64 layers for D ~ N(0,1) (y + x has about (1 + D_h^2)^(1/2) times the RMS
    of x).  B, C and dt are shared by all layers (those of make_inputs).  Every layer has its own initial
    state h0 ~ N(0, h0_std^2), as the single-layer workloads do."""
    dev = torch.device(device)
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.seed + 7919)
    q0, _ = torch.linalg.qr(torch.randn(cfg.P, cfg.P, generator=g, dtype=torch.float64))
    W = ((0.5 if scale is None else scale) * q0).to(torch.bfloat16).to(torch.float32).to(dev)
    A, D, h0 = [], [], []
    for layer in range(cfg.layers):
        gl = torch.Generator(device="cpu")
        gl.manual_seed(cfg.seed + 1 + layer)
        A.append((-torch.exp(torch.rand(cfg.H, generator=gl) * math.log(cfg.a_max))).to(dev))
        D.append(torch.randn(cfg.H, generator=gl).to(dev))
        h0.append((torch.randn(cfg.B, cfg.H, cfg.P, cfg.N, generator=gl) * cfg.h0_std).to(dev))
    return dict(W=W.contiguous(), A=A, D=D, h0=h0)
