"""ctypes binding of libssd (include/ssd.h).  Argument marshalling only: every step of the path
runs in the library's CUDA kernels.  torch is used for device memory and streams, nothing else.
There is no CPU fallback: if the shared library has not been built, loading raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libssd.so")

SSD_DTYPE_F32, SSD_DTYPE_BF16 = 0, 1
SSD_FLAG_FORCE_SIMT = 1
SSD_FLAG_ACCUM_PARAM_GRADS = 2
SSD_FLAG_SERIAL = 4
SSD_FLAG_SPLIT_BC = 8
SSD_FLAG_SKIP_GRAD = 16
SSD_OP_FWD, SSD_OP_FWD_SEG, SSD_OP_BWD_SEG = 0, 1, 2
SSD_OK, SSD_EINVAL, SSD_EUNSUPPORTED, SSD_EALIGN = 0, -1, -2, -3
SSD_EWORKSPACE, SSD_EDEVICE, SSD_ECUDA, SSD_ETIMEOUT = -4, -5, -6, -7
SSD_ETOOLARGE = -8
SSD_STATIC_WS_BYTES = 8 * 1024 * 1024

EXPORTS = ["ssd_workspace_bytes", "ssd_boundary_bytes", "ssd_fwd", "ssd_fwd_segmented",
           "ssd_bwd_segmented", "ssd_poll_status", "ssd_strerror", "ssd_version",
           "ssd_last_cuda_error", "ssd_launch_count", "ssd_kernel_kinds", "ssd_kernel_name",
           "ssd_profile", "ssd_profile_read", "ssd_fwd_static_ws", "ssd_glue_fwd", "ssd_glue_bwd",
           "ssd_glue_residual", "ssd_decode_step", "ssd_conv_fwd", "ssd_conv_bwd",
           "ssd_conv_workspace_bytes", "ssd_gated_norm_fwd", "ssd_gated_norm_bwd", "ssd_gated_norm_workspace_bytes",
           "ssd_selftest_wait_timeout"]


class SSDShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "L", "H", "P", "N", "G", "chunk", "seg", "dtype", "flags")] + \
               [(n, ctypes.c_int64) for n in ("x_bstride", "dt_bstride", "bc_bstride")]


class SSDError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = lib().ssd_strerror(code).decode()
        if code == SSD_ECUDA:
            msg += " [cudaError %d]" % lib().ssd_last_cuda_error()
        super().__init__("%s: %s (%d)" % (where, msg, code))


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libssd.so is not built: run `python -m paper_2411_19460_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, fp, sp = ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(SSDShape)
        L.ssd_workspace_bytes.restype = ctypes.c_size_t
        L.ssd_workspace_bytes.argtypes = [sp, ctypes.c_int]
        L.ssd_boundary_bytes.restype = ctypes.c_size_t
        L.ssd_boundary_bytes.argtypes = [sp]
        L.ssd_fwd.restype = ctypes.c_int
        L.ssd_fwd.argtypes = [sp, vp, fp, fp, vp, vp, fp, fp, vp, fp, vp, ctypes.c_size_t, vp]
        L.ssd_fwd_static_ws.restype = ctypes.c_int
        L.ssd_fwd_static_ws.argtypes = [sp, vp, fp, fp, vp, vp, fp, fp, vp, fp, vp]
        L.ssd_fwd_segmented.restype = ctypes.c_int
        L.ssd_fwd_segmented.argtypes = [sp, vp, fp, fp, vp, vp, fp, fp, vp, fp, fp, vp, ctypes.c_size_t, vp]
        L.ssd_bwd_segmented.restype = ctypes.c_int
        L.ssd_bwd_segmented.argtypes = [sp, vp, fp, fp, vp, vp, fp, fp, vp, fp,
                                        vp, fp, fp, vp, vp, fp, fp, vp, ctypes.c_size_t, vp]
        L.ssd_glue_fwd.restype = ctypes.c_int
        L.ssd_glue_fwd.argtypes = [sp, vp, vp, fp, vp, vp]
        L.ssd_glue_bwd.restype = ctypes.c_int
        L.ssd_glue_bwd.argtypes = [sp, vp, fp, vp, vp]
        ci, ll = ctypes.c_int, ctypes.c_longlong
        L.ssd_conv_workspace_bytes.restype = ctypes.c_size_t
        L.ssd_conv_workspace_bytes.argtypes = [ci, ci, ci]
        L.ssd_conv_fwd.restype = ctypes.c_int
        L.ssd_conv_fwd.argtypes = [ci, ci, ci, ci, vp, ll, fp, fp, vp, vp, vp, vp]
        L.ssd_conv_bwd.restype = ctypes.c_int
        L.ssd_conv_bwd.argtypes = [ci, ci, ci, ci, vp, ll, fp, fp, vp, vp, fp, vp, fp, fp, fp, ci, vp, ctypes.c_size_t, vp]
        cf = ctypes.c_float
        L.ssd_gated_norm_workspace_bytes.restype = ctypes.c_size_t
        L.ssd_gated_norm_workspace_bytes.argtypes = [ll, ci]
        L.ssd_gated_norm_fwd.restype = ctypes.c_int
        L.ssd_gated_norm_fwd.argtypes = [ll, ci, ci, ci, vp, vp, fp, cf, vp, vp]
        L.ssd_gated_norm_bwd.restype = ctypes.c_int
        L.ssd_gated_norm_bwd.argtypes = [ll, ci, ci, ci, vp, vp, fp, cf, vp, vp, vp, fp, ci, vp, ctypes.c_size_t, vp]
        L.ssd_decode_step.restype = ctypes.c_int
        L.ssd_decode_step.argtypes = [sp, vp, fp, fp, vp, vp, fp, fp, vp, vp]
        L.ssd_glue_residual.restype = ctypes.c_int
        L.ssd_glue_residual.argtypes = [sp, vp, vp, vp]
        L.ssd_poll_status.restype = ctypes.c_int
        L.ssd_poll_status.argtypes = [vp]
        L.ssd_selftest_wait_timeout.restype = ctypes.c_int
        L.ssd_selftest_wait_timeout.argtypes = [vp, ctypes.c_size_t, ctypes.c_longlong, vp]
        L.ssd_strerror.restype = ctypes.c_char_p
        L.ssd_strerror.argtypes = [ctypes.c_int]
        L.ssd_version.restype = ctypes.c_int
        L.ssd_last_cuda_error.restype = ctypes.c_int
        L.ssd_launch_count.restype = ctypes.c_longlong
        L.ssd_kernel_kinds.restype = ctypes.c_int
        L.ssd_kernel_name.restype = ctypes.c_char_p
        L.ssd_kernel_name.argtypes = [ctypes.c_int]
        L.ssd_profile.restype = ctypes.c_int
        L.ssd_profile.argtypes = [ctypes.c_int]
        L.ssd_profile_read.restype = ctypes.c_int
        L.ssd_profile_read.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_longlong),
                                       ctypes.c_int]
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def make_shape(x, Bm, chunk, seg=0, flags=0):
    """Shape descriptor from the tensors themselves (x [B,L,H,P], Bm [B,L,G,N])."""
    B, L, H, P = x.shape
    G, N = Bm.shape[2], Bm.shape[3]
    if x.dtype == torch.bfloat16:
        dt = SSD_DTYPE_BF16
    elif x.dtype == torch.float32:
        dt = SSD_DTYPE_F32
    else:
        raise TypeError("x must be float32 or bfloat16")
    return SSDShape(B, L, H, P, N, G, int(chunk), int(seg), dt, int(flags), 0, 0, 0)


def workspace_bytes(shape, op):
    return int(lib().ssd_workspace_bytes(ctypes.byref(shape), int(op)))


def boundary_bytes(shape):
    return int(lib().ssd_boundary_bytes(ctypes.byref(shape)))


def alloc_workspace(shape, op, device):
    n = workspace_bytes(shape, op)
    if n == 0:
        raise SSDError(SSD_EINVAL, "ssd_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def poll_status(ws):
    return int(lib().ssd_poll_status(_ptr(ws)))


def selftest_wait_timeout(ws, limit_cycles, stream=None):
    """Makes one bounded device-side wait run out (a barrier nothing arrives on); see include/ssd.h."""
    st = torch.cuda.current_stream() if stream is None else stream
    rc = lib().ssd_selftest_wait_timeout(_ptr(ws), ws.numel() * ws.element_size(), int(limit_cycles),
                                         ctypes.c_void_p(st.cuda_stream))
    if rc:
        raise SSDError(rc, "ssd_selftest_wait_timeout")


def launch_count():
    """Kernels launched by the library in this process so far."""
    return int(lib().ssd_launch_count())


def profile(enable):
    lib().ssd_profile(1 if enable else 0)


def profile_read():
    """{kernel kind name: (total ms, launches)} since profiling was enabled; clears the record."""
    n = lib().ssd_kernel_kinds()
    ms = (ctypes.c_double * n)()
    cnt = (ctypes.c_longlong * n)()
    rc = lib().ssd_profile_read(ms, cnt, n)
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_profile_read")
    return {lib().ssd_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n)}


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check_inputs(x, dt, A, Bm, Cm, D):
    for name, t in (("x", x), ("dt", dt), ("A", A), ("Bm", Bm), ("Cm", Cm), ("D", D)):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("%s must be a contiguous CUDA tensor" % name)
    if dt.dtype != torch.float32 or A.dtype != torch.float32 or D.dtype != torch.float32:
        raise TypeError("dt, A, D must be float32")
    if Bm.dtype != x.dtype or Cm.dtype != x.dtype:
        raise TypeError("Bm, Cm must have the dtype of x")


def ssd_fwd(x, dt, A, Bm, Cm, D, h0=None, *, chunk, seg=0, flags=0, y=None, h_final=None,
            ws=None, stream=None):
    """y, h_final = SSD forward (Eq. 1).  `seg` only sizes the scratch."""
    _check_inputs(x, dt, A, Bm, Cm, D)
    shape = make_shape(x, Bm, chunk, seg, flags)
    B, L, H, P = x.shape
    N = Bm.shape[3]
    y = torch.empty_like(x) if y is None else y
    h_final = torch.empty(B, H, P, N, dtype=torch.float32, device=x.device) if h_final is None else h_final
    ws = alloc_workspace(shape, SSD_OP_FWD, x.device) if ws is None else ws
    rc = lib().ssd_fwd(ctypes.byref(shape), _ptr(x), _ptr(dt), _ptr(A), _ptr(Bm), _ptr(Cm), _ptr(D),
                       _ptr(h0), _ptr(y), _ptr(h_final), _ptr(ws), ws.numel(), _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_fwd")
    return y, h_final


def ssd_fwd_static_ws(x, dt, A, Bm, Cm, D, h0=None, *, chunk, seg=0, flags=0, y, h_final, stream=None):
    """ssd_fwd for callers that cannot allocate: the scratch is a fixed SSD_STATIC_WS_BYTES array
    built into the library (shared by all calls on the device: do not overlap two of them), and
    this wrapper allocates nothing either, so `y` and `h_final` must be passed in.  Raises
    SSDError(SSD_ETOOLARGE) when the shape needs more scratch than that; a smaller `seg` needs less."""
    _check_inputs(x, dt, A, Bm, Cm, D)
    shape = make_shape(x, Bm, chunk, seg, flags)
    rc = lib().ssd_fwd_static_ws(ctypes.byref(shape), _ptr(x), _ptr(dt), _ptr(A), _ptr(Bm), _ptr(Cm),
                                 _ptr(D), _ptr(h0), _ptr(y), _ptr(h_final), _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_fwd_static_ws")
    return y, h_final


def ssd_fwd_segmented(x, dt, A, Bm, Cm, D, h0=None, *, chunk, seg, flags=0, y=None, h_final=None,
                      boundary=None, ws=None, stream=None):
    """y, h_final, boundary = forward that also stores the state entering every segment
    (Algorithm 1, sequence axis)."""
    _check_inputs(x, dt, A, Bm, Cm, D)
    shape = make_shape(x, Bm, chunk, seg, flags)
    B, L, H, P = x.shape
    N = Bm.shape[3]
    y = torch.empty_like(x) if y is None else y
    h_final = torch.empty(B, H, P, N, dtype=torch.float32, device=x.device) if h_final is None else h_final
    if boundary is None:
        nb = boundary_bytes(shape)
        if nb == 0:
            raise SSDError(SSD_EINVAL, "ssd_boundary_bytes")
        boundary = torch.empty(B, nb // (4 * B * H * P * N), H, P, N, dtype=torch.float32, device=x.device)
    ws = alloc_workspace(shape, SSD_OP_FWD_SEG, x.device) if ws is None else ws
    rc = lib().ssd_fwd_segmented(ctypes.byref(shape), _ptr(x), _ptr(dt), _ptr(A), _ptr(Bm), _ptr(Cm),
                                 _ptr(D), _ptr(h0), _ptr(y), _ptr(h_final), _ptr(boundary), _ptr(ws),
                                 ws.numel(), _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_fwd_segmented")
    return y, h_final, boundary


def ssd_bwd_segmented(x, dt, A, Bm, Cm, D, boundary, dy, dh_final=None, *, chunk, seg, flags=0,
                      out=None, want_dh0=True, ws=None, stream=None):
    """Gradients of Loss = <y,dy> + <h_final,dh_final> by Algorithm 2 along the sequence axis.
    Returns dict(dx, ddt, dA, dB, dC, dD, dh0)."""
    _check_inputs(x, dt, A, Bm, Cm, D)
    shape = make_shape(x, Bm, chunk, seg, flags)
    B, L, H, P = x.shape
    N = Bm.shape[3]
    dev = x.device
    if out is None:
        out = dict(dx=torch.empty_like(x), ddt=torch.empty_like(dt),
                   dA=torch.empty(H, dtype=torch.float32, device=dev),
                   dB=torch.empty_like(Bm), dC=torch.empty_like(Cm),
                   dD=torch.empty(H, dtype=torch.float32, device=dev),
                   dh0=torch.empty(B, H, P, N, dtype=torch.float32, device=dev) if want_dh0 else None)
    ws = alloc_workspace(shape, SSD_OP_BWD_SEG, dev) if ws is None else ws
    rc = lib().ssd_bwd_segmented(ctypes.byref(shape), _ptr(x), _ptr(dt), _ptr(A), _ptr(Bm), _ptr(Cm),
                                 _ptr(D), _ptr(boundary), _ptr(dy), _ptr(dh_final), _ptr(out["dx"]),
                                 _ptr(out["ddt"]), _ptr(out["dA"]), _ptr(out["dB"]), _ptr(out["dC"]),
                                 _ptr(out["dD"]), _ptr(out.get("dh0")), _ptr(ws), ws.numel(),
                                 _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_bwd_segmented")
    return out


def ssd_decode_step(x, dt, A, Bm, Cm, D, h, y=None, stream=None):
    """One token of Eq. 1: h (fp32 [B,H,P,N]) is advanced in place, y [B,1,H,P] is returned.
    x [B,1,H,P], dt [B,1,H], Bm/Cm [B,1,G,N] may be one-token slices of longer tensors."""
    if not (x.is_cuda and h.is_cuda):
        raise ValueError("device tensors required")
    B, L, H, P = x.shape
    G, N = Bm.shape[2], Bm.shape[3]
    if L != 1 or dt.shape != (B, 1, H) or Cm.shape != Bm.shape or Bm.shape[:2] != (B, 1):
        raise ValueError("ssd_decode_step takes one token: x [B,1,H,P], dt [B,1,H], Bm/Cm [B,1,G,N]")
    if h.shape != (B, H, P, N) or h.dtype != torch.float32 or not h.is_contiguous():
        raise ValueError("h must be a contiguous float32 [B,H,P,N] tensor")
    if x.dtype not in (torch.bfloat16, torch.float32) or Bm.dtype != x.dtype or Cm.dtype != x.dtype:
        raise TypeError("x, Bm, Cm must share dtype float32 or bfloat16")
    # one-token slices of longer tensors are made dense here (a few KB); the C call also takes batch strides
    x, dt, Bm, Cm = x.contiguous(), dt.contiguous(), Bm.contiguous(), Cm.contiguous()
    y = torch.empty(B, 1, H, P, dtype=x.dtype, device=x.device) if y is None else y
    if not y.is_contiguous() or y.shape != x.shape or y.dtype != x.dtype:
        raise ValueError("y must be a dense tensor like x")
    code = SSD_DTYPE_BF16 if x.dtype == torch.bfloat16 else SSD_DTYPE_F32
    shape = SSDShape(B, 1, H, P, N, G, 0, 0, code, 0, 0, 0, 0)
    rc = lib().ssd_decode_step(ctypes.byref(shape), _ptr(x), _ptr(dt), _ptr(A), _ptr(Bm), _ptr(Cm), _ptr(D),
                               _ptr(h), _ptr(y), _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_decode_step")
    return y


def _conv_args(u):
    B, L, C = u.shape
    if u.dtype == torch.bfloat16:
        code = SSD_DTYPE_BF16
    elif u.dtype == torch.float32:
        code = SSD_DTYPE_F32
    else:
        raise TypeError("u must be float32 or bfloat16")
    if not u.is_cuda or u.stride(2) != 1 or u.stride(1) != C:
        raise ValueError("u must be a CUDA tensor [B, L, C] with contiguous rows")
    return B, L, C, code, (u.stride(0) if B > 1 else 0)


def ssd_conv_fwd(u, w, bias, state_in=None, *, out=None, state_out=None, stream=None):
    """out, state_out = SiLU(depthwise causal conv4(u)); state_in / state_out [B,3,C] carry the three inputs across
    a segment cut."""
    B, L, C, code, bs = _conv_args(u)
    out = torch.empty_like(u) if out is None else out
    state_out = torch.empty(B, 3, C, dtype=u.dtype, device=u.device) if state_out is None else state_out
    rc = lib().ssd_conv_fwd(B, L, C, code, _ptr(u), bs, _ptr(w), _ptr(bias), _ptr(state_in), _ptr(out), _ptr(state_out),
                            _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_conv_fwd")
    return out, state_out


def ssd_conv_bwd(u, w, bias, state_in, dout, dtail=None, *, du=None, dstate=None, dw=None, dbias=None, accumulate=False,
                 ws=None, stream=None):
    """du, dstate, dw, dbias of one segment (Algorithm 2's order: the segment to the right first; its dstate is this
    call's dtail)."""
    B, L, C, code, bs = _conv_args(u)
    dev = u.device
    du = torch.empty_like(u) if du is None else du
    dstate = torch.empty(B, 3, C, dtype=torch.float32, device=dev) if dstate is None else dstate
    dw = torch.zeros(C, 4, dtype=torch.float32, device=dev) if dw is None else dw
    dbias = torch.zeros(C, dtype=torch.float32, device=dev) if dbias is None else dbias
    nws = int(lib().ssd_conv_workspace_bytes(B, L, C))
    ws = torch.empty(nws, dtype=torch.uint8, device=dev) if ws is None else ws
    rc = lib().ssd_conv_bwd(B, L, C, code, _ptr(u), bs, _ptr(w), _ptr(bias), _ptr(state_in), _ptr(dout), _ptr(dtail),
                            _ptr(du), _ptr(dstate), _ptr(dw), _ptr(dbias), 1 if accumulate else 0, _ptr(ws), ws.numel(),
                            _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_conv_bwd")
    return du, dstate, dw, dbias


def _norm_args(y):
    if y.dtype == torch.bfloat16:
        code = SSD_DTYPE_BF16
    elif y.dtype == torch.float32:
        code = SSD_DTYPE_F32
    else:
        raise TypeError("y must be float32 or bfloat16")
    if not y.is_cuda or not y.is_contiguous():
        raise ValueError("y must be a contiguous CUDA tensor [..., D]")
    D = y.shape[-1]
    return y.numel() // D, D, code


def ssd_gated_norm_fwd(y, z, gamma, *, group=None, eps=1e-5, out=None, stream=None):
    """out = RMSNorm(y * silu(z)) * gamma over groups of `group` channels (default: the whole last dimension)."""
    rows, D, code = _norm_args(y)
    out = torch.empty_like(y) if out is None else out
    rc = lib().ssd_gated_norm_fwd(rows, D, D if group is None else int(group), code, _ptr(y), _ptr(z), _ptr(gamma), float(eps),
                                  _ptr(out), _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_gated_norm_fwd")
    return out


def ssd_gated_norm_bwd(y, z, gamma, dout, *, group=None, eps=1e-5, dy=None, dz=None, dgamma=None, accumulate=False, ws=None,
                       stream=None):
    rows, D, code = _norm_args(y)
    dy = torch.empty_like(y) if dy is None else dy
    dz = torch.empty_like(y) if dz is None else dz
    dgamma = torch.zeros(D, dtype=torch.float32, device=y.device) if dgamma is None else dgamma
    nws = int(lib().ssd_gated_norm_workspace_bytes(rows, D))
    ws = torch.empty(nws, dtype=torch.uint8, device=y.device) if ws is None else ws
    rc = lib().ssd_gated_norm_bwd(rows, D, D if group is None else int(group), code, _ptr(y), _ptr(z), _ptr(gamma), float(eps),
                                  _ptr(dout), _ptr(dy), _ptr(dz), _ptr(dgamma), 1 if accumulate else 0, _ptr(ws), ws.numel(),
                                  _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_gated_norm_bwd")
    return dy, dz, dgamma


def _glue_shape(t):
    B, L, H, P = t.shape
    if t.dtype == torch.bfloat16:
        dt = SSD_DTYPE_BF16
    elif t.dtype == torch.float32:
        dt = SSD_DTYPE_F32
    else:
        raise TypeError("tensor must be float32 or bfloat16")
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("tensor must be a contiguous CUDA tensor")
    return SSDShape(B, L, H, P, 1, 1, 64, 0, dt, 0, 0, 0, 0)


def ssd_glue_fwd(x, y, W, x_next, stream=None):
    """x_next = W (y + x) per (batch, step, head): the hand-over between two stacked layers."""
    rc = lib().ssd_glue_fwd(ctypes.byref(_glue_shape(x)), _ptr(x), _ptr(y), _ptr(W), _ptr(x_next), _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_glue_fwd")
    return x_next


def ssd_glue_bwd(g_next, W, dz, stream=None):
    """dz = W^T g_next: the gradient of the layer's output (its dy) and of the skip branch."""
    rc = lib().ssd_glue_bwd(ctypes.byref(_glue_shape(g_next)), _ptr(g_next), _ptr(W), _ptr(dz), _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_glue_bwd")
    return dz


def ssd_glue_residual(dx, dz, stream=None):
    """dx += dz (the skip branch of the layer's input gradient)."""
    rc = lib().ssd_glue_residual(ctypes.byref(_glue_shape(dx)), _ptr(dx), _ptr(dz), _stream(stream))
    if rc != SSD_OK:
        raise SSDError(rc, "ssd_glue_residual")
    return dx
