/*
 * libssd — the Mamba-2 SSD selective-scan layer, forward and backward, under the sequence-axis
 * half of Multi-Axis Gradient Checkpointing (MA-GC), for NVIDIA B200 (sm_100a).
 *
 * The layer is the recurrence of Eq. 1 of the paper in the form Mamba-2 uses it (one scalar decay
 * per head, the input scaled by the step size, a skip term):
 *
 *     h_t = exp(dt_t * A_h) * h_{t-1} + dt_t * x_t B_t^T        h_t in R^{P x N}
 *     y_t = C_t h_t + D_h * x_t
 *
 * per batch b and head h; head h uses the B/C vectors of group g = h / (H/G).
 *
 * Conventions common to every call
 *  - All tensor pointers are DEVICE pointers owned by the caller.  The library allocates no device
 *    memory, frees nothing and never synchronises; work is enqueued on `stream` (a cudaStream_t passed
 *    as void*, NULL = the legacy default stream) or ordered after and before it (see SSD_FLAG_SERIAL):
 *    everything a call enqueued is complete once `stream` has reached the point of the call's return.  `shape` is a HOST pointer, read before return.
 *  - Row-major, innermost dimension contiguous:
 *      x, y, dy, dx        [B, L, H, P]   I/O dtype (fp32 or bf16), batch stride x_bstride
 *      dt, ddt             [B, L, H]      fp32, batch stride dt_bstride
 *      Bm, Cm, dB, dC      [B, L, G, N]   I/O dtype, batch stride bc_bstride
 *      A, D, dA, dD        [H]            fp32
 *      h0, h_final, dh_final, dh0  [B, H, P, N]  fp32, dense
 *      boundary            [B, nseg, H, P, N]    fp32, dense, nseg = ceil(L / seg);
 *                          boundary[:,k] is the state ENTERING segment k (boundary[:,0] = h0).
 *    Batch strides are in elements; 0 means dense.  They let a caller pass an L-slice of a longer
 *    tensor.  Outputs use the same strides as the matching inputs (y, dx like x; ddt like dt;
 *    dB, dC like Bm).
 *  - Every pointer must be 16-byte aligned and every row (H*P, G*N elements) a multiple of 16 bytes.
 *  - `ws` is caller-provided scratch of at least ssd_workspace_bytes(shape, op) bytes, 256-byte
 *    aligned.  Its first word is a status word the kernels set when a bounded device-side wait
 *    gives up (see ssd_poll_status).  Calls sharing a workspace must not overlap on the GPU.
 *  - Return value: SSD_OK (0) or a negative SSD_E* code.  On error nothing has been enqueued,
 *    except SSD_ECUDA, which reports a failed launch part-way (ssd_last_cuda_error() gives the
 *    CUDA code).
 *  - Deterministic: the same inputs give the same bits run to run, and the gradients of
 *    ssd_bwd_segmented do not depend on `seg` (seg == L is the unsegmented backward).
 *  - Gradient outputs are overwritten, not accumulated into (dA, dD: unless SSD_FLAG_ACCUM_PARAM_GRADS).
 */
#ifndef SSD_H_
#define SSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SSD_VERSION 100

enum { SSD_DTYPE_F32 = 0, SSD_DTYPE_BF16 = 1 };

/* shape.flags */
enum {
    SSD_FLAG_FORCE_SIMT = 1,       /* bf16 I/O: use the CUDA-core kernels instead of the tensor-core ones */
    SSD_FLAG_ACCUM_PARAM_GRADS = 2,/* ssd_bwd_segmented: dA and dD are added to, not overwritten (a driver that
                                      back-propagates one grid cell at a time sums them over the cells) */
    SSD_FLAG_SKIP_GRAD = 16,       /* ssd_bwd_segmented: dx += dy, the gradient that a skip connection around the layer
                                      (next input = f(y + x)) sends straight to x; folded into the dx kernel's output
                                      (one rounding), instead of a separate read-add-write pass over dx */
    SSD_FLAG_SPLIT_BC = 8,         /* ssd_bwd_segmented, tensor-core path: dB and dC by two kernels that each mask the
                                      score tiles themselves, instead of the one that masks them once for both (a
                                      cross-check; the same values up to the order of the fp32 head sums) */
    SSD_FLAG_SERIAL = 4            /* ssd_fwd / ssd_fwd_segmented / ssd_bwd_segmented: launch every kernel on `stream`
                                      itself, in order.  By default the tensor-core path, when there is more than one
                                      segment, runs a segment's state chain (chunk sums, state passes) one segment ahead
                                      of the large kernels, and the backward's dB/dC kernel and finishing kernels beside
                                      dx, on library-owned helper streams forked off `stream` and joined back into it
                                      before the call's last kernel; results are the same bits.  ssd_fwd_static_ws
                                      always runs in order on `stream` */
};

/* `op` of ssd_workspace_bytes */
enum { SSD_OP_FWD = 0, SSD_OP_FWD_SEG = 1, SSD_OP_BWD_SEG = 2 };

enum {
    SSD_OK = 0,
    SSD_EINVAL = -1,       /* null pointer, non-positive size, H % G, L % chunk, seg % chunk      */
    SSD_EUNSUPPORTED = -2, /* P != 64, N not in {64,128}, chunk not in {64,128,256}, bad dtype    */
    SSD_EALIGN = -3,       /* pointer or stride not 16-byte aligned                               */
    SSD_EWORKSPACE = -4,   /* ws too small or misaligned                                          */
    SSD_EDEVICE = -5,      /* current device is not compute capability 10.x                       */
    SSD_ECUDA = -6,        /* a CUDA call failed; see ssd_last_cuda_error()                       */
    SSD_ETIMEOUT = -7,     /* a bounded device-side wait expired (reported by ssd_poll_status)    */
    SSD_ETOOLARGE = -8     /* ssd_fwd_static_ws: the shape needs more scratch than the built-in buffer */
};

/*
 * Problem description.  `chunk` is the block length of the chunked scan (the paper keeps the
 * sequence-axis checkpoint interval a multiple of 256 for it, Section 4.1 "Memory-Efficient Setup");
 * `seg` is that checkpoint interval s of Algorithms 1 and 2, in tokens, a multiple of `chunk`.
 * The last segment may be shorter (L % seg != 0 is allowed); L % chunk must be 0.
 */
typedef struct ssd_shape {
    int32_t B, L, H, P, N, G;
    int32_t chunk;
    int32_t seg;   /* 0 means L (one segment) */
    int32_t dtype; /* SSD_DTYPE_* : type of x, Bm, Cm, y, dy, dx, dB, dC */
    int32_t flags; /* SSD_FLAG_* */
    int64_t x_bstride, dt_bstride, bc_bstride; /* elements; 0 => dense */
} ssd_shape_t;

/* Bytes of scratch `ws` that `op` needs for this shape (0 on an invalid shape).  Grows with
 * seg/chunk (the per-segment chunk states: the "grid cell" term of Eq. 4), not with L, apart from
 * 8 bytes per (batch, head, chunk) of dA/dD partial sums in the backward.  With four segments or more
 * the tensor-core path keeps second copies of what neighbouring segments' kernels touch at the same
 * time, unless shape->flags has SSD_FLAG_SERIAL: size the buffer with the flags the call will use.
 * Whether the tensor-core path is taken depends on the CUDA driver being present (it resolves the
 * tensor-map encoder at run time), so the answer is the one for the machine the query runs on. */
size_t ssd_workspace_bytes(const ssd_shape_t *shape, int op);

/* Bytes of the `boundary` buffer: B * ceil(L/seg) * H * P * N * 4 (the S_ckpt of Algorithm 1). */
size_t ssd_boundary_bytes(const ssd_shape_t *shape);

/*
 * Forward of Eq. 1 over the whole sequence.  h0 == NULL means a zero initial state; h_final may be
 * NULL.  The sequence is processed `seg` tokens at a time (scratch is sized by seg), which does not
 * change any output bit.
 */
int ssd_fwd(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
            const void *Bm, const void *Cm, const float *D, const float *h0,
            void *y, float *h_final, void *ws, size_t ws_bytes, void *stream);

/*
 * ssd_fwd for callers that cannot provide scratch memory.  (The paper has no counterpart; this is
 * a packaging variant of ssd_fwd.)
 *
 * Who needs it: code that runs where device allocation is off limits -- inside a region that must
 * not call cudaMalloc (a latency-critical serving loop, a plug-in whose host owns all memory, a
 * process that has already handed the whole device to another allocator) -- and so has no way to
 * obtain the `ws` buffer that ssd_fwd asks for.  Here the scratch is a fixed array of
 * SSD_STATIC_WS_BYTES bytes that lives inside the library's device image: every GPU that loads the
 * library holds those bytes until the process exits, whether or not this call is ever used.
 * The call itself performs no allocation of any kind; inputs and outputs are still the caller's.
 *
 * Same arguments and results as ssd_fwd (bit-identical outputs), minus ws / ws_bytes.
 *  - Every kernel runs in order on `stream`, so the scratch is laid out as for SSD_FLAG_SERIAL (no
 *    second copies).  Returns SSD_ETOOLARGE, with nothing enqueued, when that layout --
 *    ssd_workspace_bytes(shape with SSD_FLAG_SERIAL set, SSD_OP_FWD) -- exceeds SSD_STATIC_WS_BYTES:
 *    shrink `seg` (scratch grows with seg/chunk, not with L) or use ssd_fwd with your own buffer.
 *  - The first call on each device looks up the device address of the built-in array (with that
 *    device current).  Make that first call outside any CUDA stream capture.
 *  - All calls on one device share the one array, and it keeps whatever the previous call left
 *    in it; the call re-initialises the parts that must start from zero.  Two calls that overlap
 *    on the same GPU (different streams, or different host threads) race on it: serialise them.
 */
#define SSD_STATIC_WS_BYTES (8u * 1024u * 1024u)
int ssd_fwd_static_ws(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
                      const void *Bm, const void *Cm, const float *D, const float *h0,
                      void *y, float *h_final, void *stream);

/*
 * Forward with sequence-axis checkpoints (Algorithm 1, one layer): as ssd_fwd, and in addition
 * stores the state entering each segment of `seg` tokens into `boundary` (required, written in
 * full, boundary[:,0] = h0 or zeros).
 */
int ssd_fwd_segmented(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
                      const void *Bm, const void *Cm, const float *D, const float *h0,
                      void *y, float *h_final, float *boundary,
                      void *ws, size_t ws_bytes, void *stream);

/*
 * Backward with grid-cell restoration along the sequence axis (Algorithm 2, one layer):
 * walks the segments right to left; for each, recomputes the chunk states from boundary[:,k]
 * (Recompute_Forward), back-propagates through the segment (Backward) and hands the state
 * gradient to the segment on its left.  For Loss = <y, dy> + <h_final, dh_final> it writes
 * dx, ddt, dA, dB, dC, dD and (if non-NULL) dh0.  dh_final == NULL means zero (the nabla_state
 * input of Algorithm 2).  `boundary` must come from ssd_fwd_segmented with the same shape.
 */
int ssd_bwd_segmented(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
                      const void *Bm, const void *Cm, const float *D, const float *boundary,
                      const void *dy, const float *dh_final,
                      void *dx, float *ddt, float *dA, void *dB, void *dC, float *dD,
                      float *dh0, void *ws, size_t ws_bytes, void *stream);

/*
 * Layer-axis glue for a stack of SSD layers (Algorithms 1 and 2 keep only each layer's input along the
 * layer axis; the benchmark's stacked configuration feeds layer j+1 with x_{j+1} = W (y_j + x_j), W a fixed
 * P x P row-major fp32 matrix applied per (batch, step, head)).  Tensors are [B, L, H, P] in the I/O dtype
 * with batch stride x_bstride; only B, L, H, P, dtype and x_bstride of `shape` are read (P must be 64).
 *   ssd_glue_fwd      : x_next = W (y + x)
 *   ssd_glue_bwd      : dz = W^T g_next     (dz is the dy of the layer's SSD backward)
 *   ssd_glue_residual : dx += dz            (the skip branch; call after ssd_bwd_segmented wrote dx -- or pass
 *                                            SSD_FLAG_SKIP_GRAD to ssd_bwd_segmented, which then adds dy itself)
 * Device pointers, enqueued on `stream`, no scratch.  Returns SSD_OK or SSD_EINVAL / SSD_EUNSUPPORTED /
 * SSD_EALIGN / SSD_ECUDA.
 */
int ssd_glue_fwd(const ssd_shape_t *shape, const void *x, const void *y, const float *W, void *x_next, void *stream);
int ssd_glue_bwd(const ssd_shape_t *shape, const void *g_next, const float *W, void *dz, void *stream);
int ssd_glue_residual(const ssd_shape_t *shape, void *dx, const void *dz, void *stream);

/*
 * One token of Eq. 1 for forward-only streaming (autoregressive decoding, or the tail of a sequence
 * that is not a multiple of `chunk`): memory does not grow with the sequence, the state is all that
 * is carried.  `shape->L` must be 1; B, H, P, N, G, dtype and the batch strides are read, `chunk`,
 * `seg` and `flags` are ignored.
 *   x, y  [B, 1, H, P] I/O dtype;  dt [B, 1, H] fp32;  Bm, Cm [B, 1, G, N] I/O dtype;  A, D [H] fp32;
 *   h     [B, H, P, N] fp32, dense: the state BEFORE the token on entry, AFTER it on return (in place).
 * ssd_fwd over a prefix followed by ssd_decode_step per token continues the same recurrence: feed
 * ssd_fwd's h_final as `h`.  Any P; N in {64,128}.  Device pointers, enqueued on `stream`, no scratch.
 * Returns SSD_OK or SSD_EINVAL / SSD_EUNSUPPORTED / SSD_EALIGN / SSD_ECUDA.
 */
int ssd_decode_step(const ssd_shape_t *shape, const void *x, const float *dt, const float *A,
                    const void *Bm, const void *Cm, const float *D, float *h, void *y, void *stream);

/*
 * Depthwise causal convolution of width 4 followed by SiLU, the stage in front of the SSD layer in a Mamba-2
 * block, over C channels (x, B and C together: d_inner + 2 G N), with the sequence-axis checkpoint of its own
 * state: the last three inputs per channel (Appendix C counts them into the sequence checkpoint constant).
 *     pre[t,c] = bias[c] + sum_{k<4} w[c,k] u[t-3+k, c] ,   out = pre * sigmoid(pre)
 *   u, out, dout, du   [B, L, C]  I/O dtype, batch stride u_bstride elements (0 = dense); C % 8 == 0, L >= 3
 *   w [C,4], bias [C]  fp32
 *   state_in, state_out [B,3,C]   I/O dtype, dense: the three inputs in front of the segment (NULL = zeros) and
 *                                 the last three of it (NULL = not wanted); forward a segment at a time by
 *                                 feeding each call's state_out to the next call's state_in
 * ssd_conv_bwd: for Loss = <out, dout> + (what later segments contribute), walking the segments right to left:
 *   dtail  [B,3,C] fp32 or NULL: gradient that the segment to the right sends to this segment's last three
 *                                inputs (that call's `dstate`); NULL for the last segment
 *   dstate [B,3,C] fp32 or NULL: out: gradient reaching the three inputs in front of this segment
 *   du: written; dw [C,4], dbias [C]: written, or added to when `accumulate` != 0 (sum over segments)
 *   ws: ssd_conv_workspace_bytes(B, L, C) bytes of scratch, 256-byte aligned (per-tile partials of dw, dbias,
 *       added in a fixed order: deterministic)
 * Device pointers, enqueued on `stream`.  Returns SSD_OK or SSD_EINVAL / SSD_EUNSUPPORTED / SSD_EALIGN /
 * SSD_EWORKSPACE / SSD_EDEVICE / SSD_ECUDA.
 */
size_t ssd_conv_workspace_bytes(int B, int L, int C);
int ssd_conv_fwd(int B, int L, int C, int dtype, const void *u, long long u_bstride, const float *w, const float *bias,
                 const void *state_in, void *out, void *state_out, void *stream);
int ssd_conv_bwd(int B, int L, int C, int dtype, const void *u, long long u_bstride, const float *w, const float *bias,
                 const void *state_in, const void *dout, const float *dtail, void *du, float *dstate, float *dw,
                 float *dbias, int accumulate, void *ws, size_t ws_bytes, void *stream);

/*
 * Gated RMS normalisation, the stage behind the SSD layer in a Mamba-2 block:
 *     v = y * silu(z) ,   out = v * rsqrt(mean(v^2) + eps) * gamma
 * with the mean over groups of `group` adjacent channels (D % group == 0, group % 4 == 0, group <= 8192; group = D
 * normalises the whole row).  Token-local: a segment is a range of rows and nothing is carried across a cut.
 *   y, z, out, dout, dy, dz  [rows, D] dense, I/O dtype (rows = B * L of the segment);  gamma, dgamma [D] fp32
 * ssd_gated_norm_bwd writes dy, dz and dgamma (added to when `accumulate` != 0: sum over segments); `ws` holds
 * ssd_gated_norm_workspace_bytes(rows, D) bytes of per-tile partial sums of dgamma, 256-byte aligned, added in a fixed
 * order (deterministic).  Device pointers, enqueued on `stream`.  Returns SSD_OK or SSD_EINVAL / SSD_EUNSUPPORTED /
 * SSD_EALIGN / SSD_EWORKSPACE / SSD_EDEVICE / SSD_ECUDA.
 */
size_t ssd_gated_norm_workspace_bytes(long long rows, int D);
int ssd_gated_norm_fwd(long long rows, int D, int group, int dtype, const void *y, const void *z, const float *gamma, float eps,
                       void *out, void *stream);
int ssd_gated_norm_bwd(long long rows, int D, int group, int dtype, const void *y, const void *z, const float *gamma, float eps,
                       const void *dout, void *dy, void *dz, float *dgamma, int accumulate, void *ws, size_t ws_bytes,
                       void *stream);

/*
 * Self-test of the failure path of the bounded device-side waits (no counterpart in the paper).  Every wait of
 * the kernels (on a TMA copy, on another warp) has a time limit; when one runs out the kernel sets the status word
 * at the start of `ws` and runs to its normal end, and ssd_poll_status reports SSD_ETIMEOUT.  This call exercises
 * exactly that on a barrier that nothing ever arrives on: one warp waits `limit_cycles` clock cycles (a few
 * thousand is enough), gives up and returns.  Nothing else is in flight, so the context stays fully usable.
 * `ws`: device memory, 256-byte aligned, at least 512 bytes (the status word, and at ws + 256 the cycles waited).
 * After synchronising `stream`, ssd_poll_status(ws) must return SSD_ETIMEOUT.
 */
int ssd_selftest_wait_timeout(void *ws, size_t ws_bytes, long long limit_cycles, void *stream);

/*
 * Reads the status word at the start of `ws` (device memory) with a blocking copy: call it after
 * synchronising the stream.  Returns SSD_OK, SSD_ETIMEOUT if some kernel abandoned a bounded wait
 * (its outputs are then undefined), or SSD_ECUDA if the copy failed.
 */
int ssd_poll_status(void *ws);

/* Text for an SSD_* code (static storage). */
const char *ssd_strerror(int code);

/* SSD_VERSION the library was built from. */
int ssd_version(void);

/* The cudaError_t of the most recent failed CUDA call made by this library on this thread. */
int ssd_last_cuda_error(void);

/*
 * Instrumentation (not part of the method; the paper has no counterpart).
 * ssd_launch_count: kernels this library has launched in this process so far.
 * ssd_kernel_kinds / ssd_kernel_name: number of distinct kernel kinds and their names.
 * ssd_profile(1) makes later calls bracket every kernel launch with a pair of CUDA events on the
 * caller's stream (events are created on demand: the one place the library creates CUDA objects);
 * ssd_profile(0) stops it.  ssd_profile_read waits for the recorded events, writes the summed
 * milliseconds and the launch count per kernel kind into ms[n] / launches[n] (HOST arrays,
 * n >= ssd_kernel_kinds()) and clears the record.  Not thread-safe; meant for benchmarks.
 */
long long ssd_launch_count(void);
int ssd_kernel_kinds(void);
const char *ssd_kernel_name(int kind);
int ssd_profile(int enable);
int ssd_profile_read(double *ms, long long *launches, int n);

#ifdef __cplusplus
}
#endif
#endif /* SSD_H_ */
