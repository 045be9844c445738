"""ctypes/numpy front end of the C oracle (oracle/ssd_oracle.c). TEST INFRASTRUCTURE ONLY.

Every array is converted to contiguous float64 before the call; the C code holds all of the
arithmetic (Eq. 1 forward; Algorithm 2 backward along the sequence axis).
"""
import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        dp = ctypes.POINTER(ctypes.c_double)
        lib.ssd_oracle_fwd.restype = ctypes.c_int
        lib.ssd_oracle_fwd.argtypes = [ctypes.c_int] * 7 + [dp] * 10
        lib.ssd_oracle_bwd.restype = ctypes.c_int
        lib.ssd_oracle_bwd.argtypes = [ctypes.c_int] * 7 + [dp] * 16
        lib.ssd_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of host threads the oracle's (batch, head) loops use."""
    return int(_load().ssd_oracle_threads())


def _f64(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a):
    dp = ctypes.POINTER(ctypes.c_double)
    return ctypes.cast(None, dp) if a is None else a.ctypes.data_as(dp)


def _dims(x, Bm):
    B, L, H, P = x.shape
    G, N = Bm.shape[2], Bm.shape[3]
    return B, L, H, P, N, G


def ssd_fwd(x, dt, A, Bm, Cm, D, h0=None, seg=0):
    """Eq. 1, one step at a time. Returns (y, h_final, boundary) with boundary[:,k] the state
    entering segment k (None when seg == 0)."""
    x, dt, A, Bm, Cm, D, h0 = map(_f64, (x, dt, A, Bm, Cm, D, h0))
    B, L, H, P, N, G = _dims(x, Bm)
    assert dt.shape == (B, L, H) and A.shape == (H,) and D.shape == (H,)
    assert Bm.shape == (B, L, G, N) and Cm.shape == (B, L, G, N)
    assert h0 is None or h0.shape == (B, H, P, N)
    y = np.empty((B, L, H, P))
    hf = np.empty((B, H, P, N))
    bd = None
    if seg > 0:
        bd = np.empty((B, (L + seg - 1) // seg, H, P, N))
    rc = _load().ssd_oracle_fwd(B, L, H, P, N, G, int(seg), _p(x), _p(dt), _p(A), _p(Bm), _p(Cm),
                                _p(D), _p(h0), _p(y), _p(hf), _p(bd))
    if rc != 0:
        raise RuntimeError("ssd_oracle_fwd failed: %d" % rc)
    return y, hf, bd


def ssd_bwd(x, dt, A, Bm, Cm, D, h0, dy, dh_final=None, blk=256):
    """Reverse-mode derivative of ssd_fwd for Loss = <y,dy> + <h_final,dh_final>, walking blocks of
    `blk` steps in reverse with recompute from the block-entry state (Algorithm 2).
    Returns dict(dx, ddt, dA, dB, dC, dD, dh0)."""
    x, dt, A, Bm, Cm, D, h0, dy, dh_final = map(_f64, (x, dt, A, Bm, Cm, D, h0, dy, dh_final))
    B, L, H, P, N, G = _dims(x, Bm)
    assert dy.shape == x.shape
    out = dict(dx=np.empty_like(x), ddt=np.empty((B, L, H)), dA=np.empty(H),
               dB=np.empty((B, L, G, N)), dC=np.empty((B, L, G, N)), dD=np.empty(H),
               dh0=np.empty((B, H, P, N)))
    rc = _load().ssd_oracle_bwd(B, L, H, P, N, G, int(blk), _p(x), _p(dt), _p(A), _p(Bm), _p(Cm),
                                _p(D), _p(h0), _p(dy), _p(dh_final), _p(out["dx"]), _p(out["ddt"]),
                                _p(out["dA"]), _p(out["dB"]), _p(out["dC"]), _p(out["dD"]),
                                _p(out["dh0"]))
    if rc != 0:
        raise RuntimeError("ssd_oracle_bwd failed: %d" % rc)
    return out


def glue_fwd(x, y, W):
    """Hand-over between two stacked layers: x_next[b,t,h,:] = W (y + x)[b,t,h,:] (fp64)."""
    x, y, W = map(_f64, (x, y, W))
    return np.einsum("ij,bthj->bthi", W, y + x)


def glue_bwd(g_next, W):
    """dz = W^T g_next: gradient of (y + x) given the gradient of x_next (fp64)."""
    g_next, W = map(_f64, (g_next, W))
    return np.einsum("ij,bthi->bthj", W, g_next)


def decode_step(x, dt, A, Bm, Cm, D, h):
    """One token of Eq. 1 written out (fp64): returns (y [B,H,P], h_new [B,H,P,N]) for x [B,H,P], dt [B,H],
    Bm/Cm [B,G,N], state h [B,H,P,N]; head hh uses group hh // (H // G)."""
    x, dt, A, Bm, Cm, D, h = map(_f64, (x, dt, A, Bm, Cm, D, h))
    Bsz, H, P = x.shape
    G = Bm.shape[1]
    grp = np.arange(H) // (H // G)
    Bh, Ch = Bm[:, grp], Cm[:, grp]                                   # [B,H,N]
    alpha = np.exp(dt * A[None, :])                                   # [B,H]
    h_new = alpha[:, :, None, None] * h + (dt[:, :, None] * x)[:, :, :, None] * Bh[:, :, None, :]
    y = np.einsum("bhn,bhpn->bhp", Ch, h_new) + D[None, :, None] * x
    return y, h_new


def conv_fwd(u, w, bias, state_in=None):
    """Depthwise causal convolution of width 4 + SiLU written out (fp64): pre[t,c] = bias[c] + sum_k w[c,k] u[t-3+k,c]
    with u[-3..-1] = state_in (zeros without one); returns (out [B,L,C], pre, state_out = the last three inputs)."""
    u, w, bias = map(_f64, (u, w, bias))
    Bsz, L, C = u.shape
    st = np.zeros((Bsz, 3, C)) if state_in is None else _f64(state_in)
    ext = np.concatenate([st, u], axis=1)                       # ext[:, t+3] = u[:, t]
    pre = np.broadcast_to(bias[None, None, :], (Bsz, L, C)).copy()
    for k in range(4):
        pre += w[None, None, :, k] * ext[:, k:k + L, :]
    out = pre / (1.0 + np.exp(-pre))
    return out, pre, ext[:, L:L + 3, :].copy()


def conv_bwd(u, w, bias, state_in, dout, dtail=None):
    """Gradients of Loss = <out, dout> (+ dtail on the last three inputs): du, dstate (to the three inputs in front),
    dw [C,4], dbias [C] (fp64)."""
    u, w, bias, dout = map(_f64, (u, w, bias, dout))
    Bsz, L, C = u.shape
    _, pre, _ = conv_fwd(u, w, bias, state_in)
    st = np.zeros((Bsz, 3, C)) if state_in is None else _f64(state_in)
    ext = np.concatenate([st, u], axis=1)
    sg = 1.0 / (1.0 + np.exp(-pre))
    dpre = dout * sg * (1.0 + pre * (1.0 - sg))
    dext = np.zeros_like(ext)
    dw = np.zeros((C, 4))
    for k in range(4):
        dext[:, k:k + L, :] += w[None, None, :, k] * dpre
        dw[:, k] = np.einsum("blc,blc->c", dpre, ext[:, k:k + L, :])
    du = dext[:, 3:, :].copy()
    if dtail is not None:
        du[:, L - 3:, :] += _f64(dtail)
    return du, dext[:, :3, :].copy(), dw, dpre.sum(axis=(0, 1))


def gated_norm_fwd(y, z, gamma, group=None, eps=1e-5):
    """v = y * silu(z); out = v / sqrt(mean(v^2 over each group of `group` channels) + eps) * gamma (fp64).
    Returns (out, v, rstd [..., D/group])."""
    y, z, gamma = map(_f64, (y, z, gamma))
    D = y.shape[-1]
    group = D if group is None else group
    v = y * z / (1.0 + np.exp(-z))
    vg = v.reshape(v.shape[:-1] + (D // group, group))
    rstd = 1.0 / np.sqrt((vg * vg).mean(axis=-1) + eps)
    out = (vg * rstd[..., None]).reshape(v.shape) * gamma
    return out, v, rstd


def gated_norm_bwd(y, z, gamma, dout, group=None, eps=1e-5):
    """Gradients of Loss = <out, dout>: dy, dz, dgamma (fp64)."""
    y, z, gamma, dout = map(_f64, (y, z, gamma, dout))
    D = y.shape[-1]
    group = D if group is None else group
    _, v, rstd = gated_norm_fwd(y, z, gamma, group, eps)
    sh = v.shape[:-1] + (D // group, group)
    xh = v.reshape(sh) * rstd[..., None]
    dvh = (dout * gamma).reshape(sh)
    dv = (rstd[..., None] * (dvh - xh * (dvh * xh).mean(axis=-1, keepdims=True))).reshape(v.shape)
    sg = 1.0 / (1.0 + np.exp(-z))
    dy = dv * z * sg
    dz = dv * y * sg * (1.0 + z * (1.0 - sg))
    dgamma = (dout * xh.reshape(v.shape)).reshape(-1, D).sum(axis=0)
    return dy, dz, dgamma
