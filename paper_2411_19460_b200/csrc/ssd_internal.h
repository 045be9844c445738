// Internal declarations shared by the host driver and the kernel files of libssd.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ssd.h"

namespace ssd {

// Everything one segment's kernels need.  Passed by value to every kernel.
// Programmatic dependent launch: a kernel launched through launch_pdl() may be scheduled while its predecessor
// in the stream is still running (its CTAs take the SMs the predecessor's last wave leaves idle, and set up
// their barriers / tensor memory there); pdl_wait() returns once the predecessor has completed and its writes
// are visible, and must precede the kernel's first global-memory access.  pdl_launch_dependents() lets the
// successor be scheduled from this point on.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

struct SegParams {
    int B, L, H, P, N, G, Q;
    int hpg;       // heads per group
    int t0;        // first token of the segment
    int nc;        // chunks in this segment
    int c0;        // global index of the segment's first chunk
    int ncs;       // chunk capacity of the workspace (chunks of a full segment)
    int nct;       // chunks in the whole sequence (L / Q)
    int nsl;       // head slices per group in the dB/dC partial buffers
    int bc_fused;  // 1: the fused dB/dC kernel wrote them: two slots per slice (see ssd_tc_bcf.cu), second parts of rho/psi
    int ndd;          // partial sums of dD per (head, chunk) that the kernels of this path write (<= 16)
    int nsplit_scan;  // head ranges per group in the tensor-core scan kernels (no effect on results)
    float dx_skip;    // 1 when dx also takes dy (a skip connection around the layer), else 0
    int64_t x_bs, dt_bs, bc_bs;  // batch strides, elements

    // caller tensors
    const void *x, *Bm, *Cm, *dy;
    const float *dt, *A, *D;
    void *y, *dx, *dB, *dC;
    float *ddt;

    // workspace regions (all fp32 unless noted)
    unsigned int *status;  // [0] = error flag of bounded waits
    float *cs;             // [B,H,ncs,Q]   inclusive cumsum of dt*A inside each chunk
    float *dtT;            // [B,H,ncs,Q]   dt transposed to head-major
    float *Hst;            // [B,ncs+1,H,P,N] slot c = state entering chunk c; slot nc = leaving the segment
    float *Gst;            // [B,ncs+1,H,P,N] slot c+1 = dLoss/d(state leaving chunk c)
    __nv_bfloat16 *Hbf;    // [B,ncs+1,H,P,N] bf16 copy of Hst (tensor-core path)
    __nv_bfloat16 *Gbf;    // [B,ncs+1,H,P,N] bf16 copy of Gst (tensor-core path)
    float *hcarry;         // [B,H,P,N]     state handed from segment to segment (forward)
    float *gcarry;         // [B,H,P,N]     state gradient handed right-to-left (backward)
    float *ghdot;          // [B,H,ncs,16]  partial sums of exp(cs_last) <Gout_c, H_in,c>
    float *ddt_dir;        // [B,H,ncs,Q]   direct part of ddt
    float *rho;            // [B,H,ncs,Q]   C_t . dC_t of this head (CUDA-core path: all of it; tensor-core
                           //               path: its intra-chunk part)
    float *rhob, *psib;    // [B,H,ncs,Q]   fused dB/dC kernel: second parts of rho / psi (else NULL)
    float *rho2;           // [B,H,ncs,Q]   tensor-core path: C_t . (inter-chunk part of this head's dC_t); else NULL
    float *psi;            // [B,H,ncs,Q]   B_t . (intra-chunk part of this head's dB_t)
    float *psi2;           // [B,H,ncs,Q]   B_t . (inter-chunk part of this head's dB_t)
    float *pB, *pC;        // [B,seg,G,nsl,N] per-head-slice partial dB / dC
    float *dAp;            // [B,H,nct]     per-chunk partial of dA
    float *dDp;            // [B,H,nct,16]  partials of dD, the first ndd of each group of 16 in use
};

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- kernel launchers (each returns the cudaError_t of its launch) ----
// ssd_simt.cu : CUDA-core kernels, any I/O dtype
cudaError_t launch_chunk_cumsum(const SegParams &p, cudaStream_t st);
cudaError_t launch_chunk_state_simt(const SegParams &p, int dtype, int mode, cudaStream_t st);
// init: state entering the segment (NULL = zeros), batch stride init_bs elements;
// boundary_out (nullable): where to store that state, batch stride bnd_bs; final_out nullable.
cudaError_t launch_state_pass_fwd(const SegParams &p, const float *init, long long init_bs,
                                  float *boundary_out, long long bnd_bs, float *final_out,
                                  bool want_bf16, cudaStream_t st);
cudaError_t launch_state_pass_bwd(const SegParams &p, const float *init, float *left_out,
                                  bool want_bf16, cudaStream_t st);
cudaError_t launch_masked_product_simt(const SegParams &p, int dtype, int mode, cudaStream_t st);
cudaError_t launch_bwd_finish(const SegParams &p, cudaStream_t st);
cudaError_t launch_reduce_dbdc(const SegParams &p, int dtype, cudaStream_t st);
cudaError_t launch_final_dAdD(const SegParams &p, float *dA, float *dD, bool accumulate, cudaStream_t st);
// ssd_glue.cu : layer-axis glue of a layer stack
cudaError_t launch_glue(int dtype, bool transpose, const void *a, const void *b, const float *W, void *out,
                        long long rows_per_batch, long long bstride, int B, cudaStream_t st);
cudaError_t launch_residual(int dtype, void *dst, const void *src, long long n_per_batch, long long bstride, int B,
                            cudaStream_t st);

// ssd_conv.cu : depthwise causal convolution (width 4) + SiLU in front of the SSD layer, with its 3-token state
int conv_tiles(int L);
cudaError_t launch_conv_fwd(int dtype, const void *u, long long u_bs, const float *w, const float *bias,
                            const void *state_in, void *out, void *state_out, int B, int L, int C, cudaStream_t st);
cudaError_t launch_conv_bwd(int dtype, const void *u, long long u_bs, const float *w, const float *bias,
                            const void *state_in, const void *dout, const float *dtail, void *du, float *dstate,
                            float *dw, float *dbias, int accumulate, float *part, int B, int L, int C, cudaStream_t st);
// ssd_norm.cu : gated RMS normalisation behind the SSD layer
long long gated_norm_tiles(long long rows);
int gated_norm_max_group();
cudaError_t launch_gated_norm_fwd(int dtype, const void *y, const void *z, const float *gamma, float eps, void *out,
                                  long long rows, int D, int group, cudaStream_t st);
cudaError_t launch_gated_norm_bwd(int dtype, const void *y, const void *z, const float *gamma, float eps, const void *dout,
                                  void *dy, void *dz, float *dgamma, int accumulate, float *part, long long rows, int D,
                                  int group, cudaStream_t st);
// ssd_decode.cu : one token of the recurrence, state updated in place
cudaError_t launch_decode_step(int dtype, int N, const void *x, const float *dt, const float *A, const void *Bm,
                               const void *Cm, const float *D, float *h, void *y, int B, int H, int P, int G,
                               long long x_bs, long long dt_bs, long long bc_bs, cudaStream_t st);

// ssd_tc.cu : tensor-core (tcgen05 / TMEM / TMA) kernels, bf16 I/O
struct TcMaps {
    CUtensorMap x, dy, Bm, Cm;  // [B][L][H*64] / [B][L][G*128], box 64 x 128 rows
    CUtensorMap y, dx;          // outputs, same geometry as x; box 64 columns x 32 rows (TMA stores)
    CUtensorMap Hbf, Gbf;       // bf16 chunk states as [rows][128], box 64 x 64 rows
};
bool tc_supported(int dtype, int flags, int P, int N, int Q, int hpg);
bool tc_make_maps(const SegParams &p, TcMaps &m);
cudaError_t launch_chunk_state_tc(const SegParams &p, const TcMaps &m, int mode, cudaStream_t st);
// ssd_tc_scan.cu : y (SC_FWD) or dx, ddt_direct, dD partials (SC_DX)
cudaError_t launch_scan_tc(const SegParams &p, const TcMaps &m, int mode, cudaStream_t st);
enum { SC_FWD = 0, SC_DX = 1 };
// ssd_tc_bc.cu : per-slice partial dC, rho (GB_DC) or partial dB, psi, psi2 (GB_DB)
cudaError_t launch_grad_bc_tc(const SegParams &p, const TcMaps &m, int mode, cudaStream_t st);
enum { GB_DC = 0, GB_DB = 1 };
// ssd_tc_bcf.cu : dB and dC from one masked tile (partial slices, rho, psi and their second parts)
cudaError_t launch_grad_bc_fused(const SegParams &p, const TcMaps &m, cudaStream_t st);

enum { STATE_MODE_FWD = 0, STATE_MODE_DSTATE = 1 };
// kernel kinds, for the launch counter and the optional per-kind timing
enum {
    KIND_CUMSUM = 0, KIND_CHUNK_STATE, KIND_STATE_PASS_FWD, KIND_SCAN_FWD, KIND_DSTATE,
    KIND_STATE_PASS_BWD, KIND_BWD_DX, KIND_BWD_DC, KIND_BWD_DB, KIND_BWD_FINISH, KIND_REDUCE_DBDC,
    KIND_FINAL, KIND_GLUE, KIND_DECODE, KIND_BWD_DBDC, KIND_CONV, KIND_NORM, KIND_COUNT
};
enum { MP_FWD = 0, MP_BWD_DX = 1, MP_DC = 2, MP_DB = 3 };

}  // namespace ssd
