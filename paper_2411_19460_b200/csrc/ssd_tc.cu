// Tensor-core kernels of libssd for bf16 I/O on sm_100a: tcgen05.mma with fp32 accumulators in
// TMEM, operands staged in shared memory by TMA (128-byte swizzle), epilogues through tcgen05.ld.
// Shapes served: P = 64, N = 128, chunk Q = 256, an even number of heads per group.
//
// Notation per (batch b, head h), chunk of Q steps: a_t = dt_t*A_h, cs_t = inclusive cumsum of a
// inside the chunk, H_in = state entering the chunk, Gout = dLoss/d(state leaving the chunk); all
// of it is Eq. 1 of the paper regrouped by chunks.
#include <cstring>

#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

using namespace sm100;

// ------------------------------------------------------------------ host: tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 tensor [dim2][dim1][dim0] (dim0 contiguous), box {box_cols, box_rows, 1}; 128-byte swizzle for
// 64-element (128-byte) box rows, none for narrower ones.
static bool make_map3(CUtensorMap *m, const void *ptr, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                      uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box_rows, uint32_t box_cols = 64) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {dim0, dim1, dim2};
    cuuint64_t strides[2] = {stride1_elems * 2, stride2_elems * 2};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, box_cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tc_supported(int dtype, int flags, int P, int N, int Q, int hpg) {
    return dtype == SSD_DTYPE_BF16 && !(flags & SSD_FLAG_FORCE_SIMT) && P == 64 && N == 128 && Q == 256 &&
           (hpg % 2) == 0 && encode_fn() != nullptr;
}

// Builds the tensor maps of one API call.  x/dy/Bm/Cm may be null when the call does not use them.
bool tc_make_maps(const SegParams &p, TcMaps &m) {
    memset(&m, 0, sizeof(m));
    const uint64_t HP = (uint64_t)p.H * 64, GN = (uint64_t)p.G * 128;
    bool ok = true;
    if (p.x) ok = ok && make_map3(&m.x, p.x, HP, p.L, p.B, HP, p.x_bs, 128);
    if (p.dy) ok = ok && make_map3(&m.dy, p.dy, HP, p.L, p.B, HP, p.x_bs, 128);
    if (p.y) ok = ok && make_map3(&m.y, p.y, HP, p.L, p.B, HP, p.x_bs, 32);
    if (p.dx) ok = ok && make_map3(&m.dx, p.dx, HP, p.L, p.B, HP, p.x_bs, 32);
    if (p.Bm) ok = ok && make_map3(&m.Bm, p.Bm, GN, p.L, p.B, GN, p.bc_bs, 128);
    if (p.Cm) ok = ok && make_map3(&m.Cm, p.Cm, GN, p.L, p.B, GN, p.bc_bs, 128);
    // bf16 state copies viewed as [B*(ncs+1)*H*64 rows][128]
    const uint64_t srows = (uint64_t)p.B * (p.ncs + 1) * p.H * 64;
    if (p.Hbf) ok = ok && make_map3(&m.Hbf, p.Hbf, 128, srows, 1, 128, srows * 128, 64);
    if (p.Gbf) ok = ok && make_map3(&m.Gbf, p.Gbf, 128, srows, 1, 128, srows * 128, 64);
    return ok;
}

// ------------------------------------------------------------------ chunk sums / state-gradient sums on tensor cores
// One CTA per (chunk, head pair, batch): D[128 = (head-in-pair, p)][N] = sum_s Xw[s][(h2,p)] * V[s][n]
//   mode FWD   : X = x,  V = Bm, w_s = exp(cs_last - cs_s) dt_s  -> Hst slot c+1   (S_c)
//   mode DSTATE: X = dy, V = Cm, w_t = exp(cs_t)                 -> Gst slot c     (E_c)
// Both operands are MN-major straight from the row-major tensors (rows = time = the contraction
// index).  The per-row weight is multiplied into the X tile in shared memory (it is uniform along
// a row, so the swizzle does not matter).  The kernel is bound by its loads, so a CTA keeps only
// ONE 64 KB stage (half a chunk) and two to three CTAs share an SM: one CTA's load overlaps the
// others' scaling, MMAs and epilogue.
//
// Mode FWD also computes the chunk cumsum of dt*A for its two heads and leaves cs / dtT for the
// later kernels of the segment.  Mode DSTATE also produces, per head, rho2_t = e^{cs_t} dy_t . (H_in C_t): the inter-chunk part of
// C_t . dC_t that the decay gradient needs.  The C tile is already in shared memory (as rows of
// time it is a K-major A operand), so it is one more product C (128 x N) * H_in^T (N x P) per head
// and half into spare TMEM columns, and a row dot with the already scaled dy tile.
constexpr int CS_THREADS = 256;
constexpr int CS_OUT_STAGE = 128 * 528;   // result tile staged as 128 rows of 512 B, 16 B of padding each
constexpr int CS_STAGE = 65536;   // X head0 16K | X head1 16K | V n0-63 16K | V n64-127 16K   (128 time rows)

__global__ void __launch_bounds__(CS_THREADS, 3)
k_chunk_state_tc(SegParams p, int mode, const __grid_constant__ CUtensorMap tmX,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmH) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar_ld, bar_mma, bar_h;
    __shared__ uint32_t tmem_base, abort_flag;
    __shared__ float wsm[2][256];

    pdl_launch_dependents();
    pdl_wait();       // the first loads are issued right below, by the thread that also sets up the barriers
    const int c = blockIdx.x, hp = blockIdx.y, b = blockIdx.z;
    const int h0 = hp * 2, g = h0 / p.hpg;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int qrow = (warp & 3) * 32 + (tid & 31);   // row of the accumulator this thread can read (TMEM lane)
    const int chalf = warp >> 2;                      // which half of the work of that row it takes
    const int tok0 = p.t0 + c * 256;
    const bool dstate = (mode == STATE_MODE_DSTATE);

    auto issue_stage = [&](int half) {
        mbar_arrive_expect_tx(&bar_ld, CS_STAGE);
        tma_load_3d(smem, &tmX, &bar_ld, h0 * 64, tok0 + half * 128, b);
        tma_load_3d(smem + 16384, &tmX, &bar_ld, h0 * 64 + 64, tok0 + half * 128, b);
        tma_load_3d(smem + 32768, &tmV, &bar_ld, g * 128, tok0 + half * 128, b);
        tma_load_3d(smem + 49152, &tmV, &bar_ld, g * 128 + 64, tok0 + half * 128, b);
    };

    if (tid == 0) {
        mbar_init(&bar_ld, 1);
        mbar_init(&bar_mma, 1);
        mbar_init(&bar_h, 1);
        abort_flag = 0;
        fence_barrier_init();
        issue_stage(0);
        if (dstate) {
            mbar_arrive_expect_tx(&bar_h, 32768);
            for (int hh = 0; hh < 2; ++hh) {
                const int row = ((b * (p.ncs + 1) + c) * p.H + h0 + hh) * 64;   // state entering chunk c
                tma_load_3d(smem + CS_STAGE + hh * 16384, &tmH, &bar_h, 0, row, 0);
                tma_load_3d(smem + CS_STAGE + hh * 16384 + 8192, &tmH, &bar_h, 64, row, 0);
            }
        }
    }
    const uint32_t ncol_tmem = dstate ? 256u : 128u;   // E or S: 128 columns; Yoff of two heads: 128 more
    if (warp == 0) tmem_alloc(&tmem_base, ncol_tmem);
    if (!dstate) {
        // the chunk cumsum, fused in: the chunk's cumulative sums of dt*A for the two heads (warp hh scans head hh: a
        // lane owns 8 consecutive steps, lane totals meet in a warp-shuffle scan), kept for every later
        // kernel of the segment in cs / dtT, and turned into the per-row weights right here.
        if (warp < 2) {
            const int hh = warp, lane = tid & 31, h = h0 + hh;
            const float Ah = __ldg(p.A + h);
            const float *dtp = p.dt + (size_t)b * p.dt_bs + (size_t)(tok0 + lane * 8) * p.H + h;
            float d[8], a[8], run = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) d[j] = __ldg(dtp + (size_t)j * p.H);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                run += d[j] * Ah;
                a[j] = run;
            }
            float incl = run;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const float v = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += v;
            }
            float excl = __shfl_up_sync(0xffffffffu, incl, 1);
            if (lane == 0) excl = 0.f;
            const float last = __shfl_sync(0xffffffffu, incl, 31);
            float *cso = p.cs + ((((size_t)b * p.H + h) * p.ncs + c) << 8) + lane * 8;
            float *dto = p.dtT + ((((size_t)b * p.H + h) * p.ncs + c) << 8) + lane * 8;
            float cv[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                cv[j] = a[j] + excl;
                wsm[hh][lane * 8 + j] = __expf(fminf(last - cv[j], 0.f)) * d[j];
            }
            *reinterpret_cast<float4 *>(cso) = make_float4(cv[0], cv[1], cv[2], cv[3]);
            *reinterpret_cast<float4 *>(cso + 4) = make_float4(cv[4], cv[5], cv[6], cv[7]);
            *reinterpret_cast<float4 *>(dto) = make_float4(d[0], d[1], d[2], d[3]);
            *reinterpret_cast<float4 *>(dto + 4) = make_float4(d[4], d[5], d[6], d[7]);
        }
    } else {
        // per-row weights of both heads from the cumulative sums the forward-mode launch left
        for (int i = tid; i < 512; i += CS_THREADS) {
            const int hh = i >> 8, t = i & 255;
            const float *csb = p.cs + ((((size_t)b * p.H + h0 + hh) * p.ncs + c) << 8);
            wsm[hh][t] = __expf(csb[t]);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base;
    const uint32_t idesc = umma_idesc_bf16(128, 128, true, true);
    // operand descriptors as (low word, high word); the issue loops below add compile-time constants
    // (16-byte units) to the low word only
    const uint64_t dXa = umma_desc_sw128(smem_u32(smem), 16384, 1024), dVb = umma_desc_sw128(smem_u32(smem + 32768), 16384, 1024);
    const uint64_t dCk = umma_desc_sw128(smem_u32(smem + 32768), 16, 1024), dHk = umma_desc_sw128(smem_u32(smem + CS_STAGE), 16, 1024);
    const uint32_t loXa = (uint32_t)dXa, hiXa = (uint32_t)(dXa >> 32), loVb = (uint32_t)dVb, hiVb = (uint32_t)(dVb >> 32);
    const uint32_t loCk = (uint32_t)dCk, hiCk = (uint32_t)(dCk >> 32), loHk = (uint32_t)dHk, hiHk = (uint32_t)(dHk >> 32);

    for (int half = 0; half < 2; ++half) {
        mbar_wait(&bar_ld, half, &abort_flag, p.status);
        // scale the X pair: 2 heads x 128 rows x 8 chunks of 16 B
        for (int q = tid; q < 2048; q += CS_THREADS) {
            const int hh = q >> 10, row = (q >> 3) & 127;
            const float w = wsm[hh][half * 128 + row];
            uint4 *ptr = reinterpret_cast<uint4 *>(smem + (size_t)q * 16);
            uint4 v = *ptr;
            __nv_bfloat162 *e = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float2 f = __bfloat1622float2(e[k]);
                e[k] = __floats2bfloat162_rn(f.x * w, f.y * w);
            }
            *ptr = v;
        }
        fence_proxy_async_smem();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after_sync();
            if (half == 0) umma_bf16_fixed<false>(tm, dXa, dVb, idesc);
            else umma_bf16_fixed<true>(tm, dXa, dVb, idesc);
#pragma unroll
            for (int ks = 1; ks < 8; ++ks)
                umma_bf16_fixed<true>(tm, umma_desc_words(loXa + ks * 128, hiXa), umma_desc_words(loVb + ks * 128, hiVb), idesc);
            if (dstate) {
                // Yoff[t, p] = sum_n C[t, n] H_in[p, n] for the 128 time rows of this half, per head
                if (half == 0) {
                    mbar_wait(&bar_h, 0, &abort_flag, p.status);
                    tc_fence_after_sync();
                }
                const uint32_t idy = umma_idesc_bf16(128, 64, false, false);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint64_t ad = umma_desc_words(loCk + (kk >> 2) * 1024 + (kk & 3) * 2, hiCk);
                        const uint64_t bd = umma_desc_words(loHk + hh * 1024 + (kk >> 2) * 512 + (kk & 3) * 2, hiHk);
                        if (kk == 0) umma_bf16_fixed<false>(tm + 128 + hh * 64, ad, bd, idy);
                        else umma_bf16_fixed<true>(tm + 128 + hh * 64, ad, bd, idy);
                    }
                }
            }
            umma_commit(&bar_mma);
        }
        mbar_wait(&bar_mma, half, &abort_flag, p.status);
        tc_fence_after_sync();
        if (dstate) {
            // rho2_t = (e^{cs_t} dy_t) . Yoff_t with the scaled dy row read back from shared memory
            {
                const int hh = chalf;
                float y0[32], y1[32];
                const uint32_t ta = tm + ((uint32_t)((warp & 3) * 32) << 16) + 128 + hh * 64;
                tmem_ld32_nowait(ta, y0);
                tmem_ld32_nowait(ta + 32, y1);
                tmem_ld_wait32(y0);
                tmem_ld_wait32(y1);
                const unsigned char *row = smem + hh * 16384 + qrow * 128;
                float acc = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint4 v = *reinterpret_cast<const uint4 *>(row + ((j ^ (qrow & 7)) << 4));
                    const __nv_bfloat162 *e = reinterpret_cast<const __nv_bfloat162 *>(&v);
                    const float *yy = (j < 4) ? (y0 + j * 8) : (y1 + (j - 4) * 8);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float2 f = __bfloat1622float2(e[k]);
                        acc = fmaf(f.x, yy[2 * k], acc);
                        acc = fmaf(f.y, yy[2 * k + 1], acc);
                    }
                }
                p.rho2[((((size_t)b * p.H + h0 + hh) * p.ncs + c) << 8) + half * 128 + qrow] = acc;
            }
        }
        tc_fence_before_sync();
        fence_proxy_async_smem();              // order this thread's accesses to the stage before the next TMA write
        __syncthreads();                       // the stage (and the Yoff columns) may be overwritten now
        if (half == 0 && tid == 0) issue_stage(1);
    }

    // The CTA's 128 x 128 fp32 result (two heads x 64 rows) is one contiguous 64 KB block of the state
    // buffer.  Row-per-thread global stores would touch 32 different lines per instruction, so the tile is
    // staged in the (now dead) stage, rows padded to 528 bytes (conflict-free row-per-thread writes), and
    // every row leaves as one 512-byte bulk copy.
    {
        float *stg = reinterpret_cast<float *>(smem);
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 32) {
            float v[32];
            tmem_ld32(tm + ((uint32_t)((warp & 3) * 32) << 16) + chalf * 64 + c0, v);
#pragma unroll
            for (int i = 0; i < 32; i += 4)
                *reinterpret_cast<float4 *>(stg + qrow * 132 + chalf * 64 + c0 + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
        }
        fence_proxy_async_smem();
        __syncthreads();
        if (tid < 128) {
            const int slot = dstate ? c : c + 1;
            float *base = dstate ? p.Gst : p.Hst;
            float *out = base + ((((size_t)b * (p.ncs + 1) + slot) * p.H + h0) * 64 + tid) * 128;
            bulk_store(out, stg + tid * 132, 512);
            tma_store_commit();
            tma_store_wait_read();
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tm, ncol_tmem);
}

cudaError_t launch_chunk_state_tc(const SegParams &p, const TcMaps &m, int mode, cudaStream_t st) {
    // forward mode: the stage, reused (and slightly outgrown) by the padded result tile
    const int smem = (mode == STATE_MODE_DSTATE ? CS_STAGE + 32768 : CS_OUT_STAGE) + 1024;
    cudaError_t e = cudaFuncSetAttribute(k_chunk_state_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         CS_STAGE + 32768 + 1024);
    if (e != cudaSuccess) return e;
    dim3 grid(p.nc, p.H / 2, p.B);
    if (mode == STATE_MODE_FWD) return launch_pdl(k_chunk_state_tc, grid, dim3(CS_THREADS), (size_t)smem, st, p, mode, m.x, m.Bm, m.Hbf);
    return launch_pdl(k_chunk_state_tc, grid, dim3(CS_THREADS), (size_t)smem, st, p, mode, m.dy, m.Cm, m.Hbf);
}

}  // namespace ssd
