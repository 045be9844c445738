// Tensor-core kernel for the two masked products whose score matrix is per head and whose result
// is summed over the heads of a group (bf16 I/O, P = 64, N = 128, Q = 256):
//
//   GB_DC (a11): dC_t = sum_h [ sum_{s<=t} W_h[t,s] B_s + e^{cs_t} dy_t^T H_in ]          rows t
//   GB_DB (a11): dB_s = sum_h [ sum_{t>=s} W_h[t,s] C_t + dt_s e^{cs_last-cs_s} x_s^T Gout ]  rows s
//   with W_h[t,s] = (dy_t . x_s) e^{cs_t-cs_s} dt_s   (s <= t)
//
// and the per-head scalars the decay gradient needs (a12):
//   rho_t  = C_t . (this head's dC_t)                         (GB_DC)
//   psi_s  = B_s . (intra-chunk part of this head's dB_s)     (GB_DB)
//   psi2_s = B_s . (inter-chunk part of this head's dB_s)     (GB_DB)
// (Eq. 1 of the paper regrouped by chunks; cs = inclusive cumsum of dt*A inside the chunk.)
//
// One CTA owns (chunk, 128-row block, group, a range of the group's heads) and keeps the group's
// value rows (B or C) in shared memory for all of them.  Per head: score pieces S = Rows * Cols^T
// (128 x 64, K = P) go to a four-slot TMEM ring; eight mask warps turn each piece into the bf16
// masked tile W (same mask factorisation and the same rounding in both modes, so that rho and psi
// are built from identical W and their difference cancels cleanly); acc1 = W * V and
// acc2 = Rows * State accumulate in TMEM; the epilogue reads them once per head, takes the dot
// products with the thread's own C/B row, and adds the head into register accumulators.  The sum
// over the CTA's heads is written as one fp32 partial slice; a later kernel adds the slices.
#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

using namespace sm100;

namespace {

constexpr int GB_THREADS = 320;           // warp 0 producer, warp 1 MMA, warps 2..9 mask + epilogue
constexpr uint32_t GB_OFF_V = 0;          // 64 KB  [n-half][ncols rows][128 B], kept for all heads
constexpr uint32_t GB_OFF_AB = 65536;     // 2 x 48 KB  per head: rows operand 16 KB | cols operand 32 KB
constexpr uint32_t GB_OFF_ST = 163840;    // 16 KB  bf16 chunk state [n-half][64 p rows][128 B]
constexpr uint32_t GB_OFF_M = 180224;     // 2 x 16 KB  masked pieces
constexpr uint32_t GB_OFF_VEC = 212992;   // per-head vectors, double buffered
constexpr uint32_t GB_VEC_FLOATS = 256 * 3 + 64;
constexpr uint32_t GB_OFF_PART = GB_OFF_VEC + 2 * GB_VEC_FLOATS * 4;   // 2 x 3 x 128 floats
constexpr uint32_t GB_SMEM = GB_OFF_PART + 2 * 3 * 128 * 4 + 1024;

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void bar_mask_warps() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ float2 unpack2(uint32_t w) {
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w));
}

}  // namespace

template <int MODE>
__global__ void __launch_bounds__(GB_THREADS, 1)
k_grad_bc_tc(SegParams p, const __grid_constant__ CUtensorMap tmRow,   // DC: dy ; DB: x
             const __grid_constant__ CUtensorMap tmCol,                // DC: x  ; DB: dy
             const __grid_constant__ CUtensorMap tmV,                  // DC: Bm ; DB: Cm
             const __grid_constant__ CUtensorMap tmSt) {               // DC: Hbf; DB: Gbf
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar_v, abfull[2], abempty[2], stfull, stempty, sfull[4], sempty[4], mfull[2],
        mempty[2], accfull, accempty;
    __shared__ uint32_t tmem_base, abort_flag;

    constexpr bool DC = (MODE == GB_DC);
    const int nc = p.nc, nsl = p.nsl;
    const int rb = DC ? 1 - (int)(blockIdx.x / nc) : (int)(blockIdx.x / nc);   // long CTAs first
    const int c = blockIdx.x % nc, b = blockIdx.z;
    const int g = blockIdx.y / nsl, sl = blockIdx.y % nsl;
    const int hps = (p.hpg + nsl - 1) / nsl;
    const int h_begin = g * p.hpg + sl * hps;
    const int h_end = min(g * p.hpg + p.hpg, h_begin + hps);
    const int nheads = max(h_end - h_begin, 0);
    const int colbase = DC ? 0 : rb * 128;
    const int ncols = DC ? (rb + 1) * 128 : 256 - rb * 128;
    const int npieces = ncols >> 6;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tok0 = p.t0 + c * 256;
    const int slot = DC ? c : c + 1;

    if (tid == 0) {
        mbar_init(&bar_v, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&abfull[i], 1);
            mbar_init(&abempty[i], 1);
            mbar_init(&mfull[i], 256);
            mbar_init(&mempty[i], 1);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(&sfull[i], 1);
            mbar_init(&sempty[i], 256);
        }
        mbar_init(&stfull, 1);
        mbar_init(&stempty, 1);
        mbar_init(&accfull, 1);
        mbar_init(&accempty, 256);
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc(&tmem_base, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base;
    // TMEM columns: S ring [0,256) in four 64-column slots ; acc1 [256,384) ; acc2 [384,512)
    volatile uint32_t *abortp = &abort_flag;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0 && nheads > 0) {
            mbar_arrive_expect_tx(&bar_v, (uint32_t)ncols * 256u);
            for (int nh = 0; nh < 2; ++nh)
                for (int r0 = 0; r0 < ncols; r0 += 128)
                    tma_load_3d(smem + GB_OFF_V + nh * ncols * 128 + r0 * 128, &tmV, &bar_v, g * 128 + nh * 64,
                                tok0 + colbase + r0, b);
            const int strow = (b * (p.ncs + 1) + slot) * p.H;
            for (int hi = 0; hi < nheads; ++hi) {
                const int buf = hi & 1, h = h_begin + hi;
                if (hi >= 2) mbar_wait(&abempty[buf], ((hi >> 1) - 1) & 1, abortp, p.status);
                unsigned char *ab = smem + GB_OFF_AB + buf * 49152;
                mbar_arrive_expect_tx(&abfull[buf], 16384u + (uint32_t)ncols * 128u);
                tma_load_3d(ab, &tmRow, &abfull[buf], h * 64, tok0 + rb * 128, b);
                for (int r0 = 0; r0 < ncols; r0 += 128)
                    tma_load_3d(ab + 16384 + r0 * 128, &tmCol, &abfull[buf], h * 64, tok0 + colbase + r0, b);
                if (hi >= 1) mbar_wait(&stempty, (hi - 1) & 1, abortp, p.status);
                mbar_arrive_expect_tx(&stfull, 16384);
                tma_load_3d(smem + GB_OFF_ST, &tmSt, &stfull, 0, (strow + h) * 64, 0);
                tma_load_3d(smem + GB_OFF_ST + 8192, &tmSt, &stfull, 64, (strow + h) * 64, 0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && nheads > 0) {
            const uint32_t sV = smem_u32(smem + GB_OFF_V), sAB = smem_u32(smem + GB_OFF_AB);
            const uint32_t sSt = smem_u32(smem + GB_OFF_ST), sM = smem_u32(smem + GB_OFF_M);
            const uint32_t idS = umma_idesc_bf16(128, 64, false, false);    // rows (K-major) x cols (K-major)
            const uint32_t id2 = umma_idesc_bf16(128, 128, false, true);    // W piece (K-major) x V (MN-major)
            const uint32_t id3 = umma_idesc_bf16(128, 128, false, true);    // rows (K-major) x state (MN-major)
            const uint32_t acc1 = tm + 256, acc2 = tm + 384;
            uint32_t mcount[2] = {0, 0};

            auto issue_scores = [&](int hi, int jj) {
                const int buf = hi & 1;
                if (jj == 0) {
                    mbar_wait(&abfull[buf], (hi >> 1) & 1, abortp, p.status);
                    tc_fence_after_sync();
                }
                if (hi >= 1) {
                    mbar_wait(&sempty[jj], (hi - 1) & 1, abortp, p.status);
                    tc_fence_after_sync();
                }
                const uint32_t a = sAB + buf * 49152, bc = a + 16384 + jj * 8192;
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_bf16(tm + jj * 64, umma_desc_sw128(a + k * 32, 16, 1024),
                              umma_desc_sw128(bc + k * 32, 16, 1024), idS, k ? 1u : 0u);
                umma_commit(&sfull[jj]);
            };

            for (int jj = 0; jj < npieces; ++jj) issue_scores(0, jj);
            mbar_wait(&bar_v, 0, abortp, p.status);
            for (int hi = 0; hi < nheads; ++hi) {
                const int buf = hi & 1;
                if (hi >= 1) mbar_wait(&accempty, (hi - 1) & 1, abortp, p.status);
                mbar_wait(&stfull, hi & 1, abortp, p.status);
                tc_fence_after_sync();
                {
                    const uint32_t a = sAB + buf * 49152;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16(acc2, umma_desc_sw128(a + k * 32, 16, 1024),
                                  umma_desc_sw128(sSt + k * 2048, 8192, 1024), id3, k ? 1u : 0u);
                    umma_commit(&stempty);
                }
                for (int jj = 0; jj < npieces; ++jj) {
                    const int ms = jj & 1;
                    mbar_wait(&mfull[ms], mcount[ms] & 1, abortp, p.status);
                    ++mcount[ms];
                    tc_fence_after_sync();
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16(acc1, umma_desc_sw128(sM + ms * 16384 + k * 32, 16, 1024),
                                  umma_desc_sw128(sV + (jj * 64 + k * 16) * 128, (uint32_t)ncols * 128u, 1024), id2,
                                  (jj | k) ? 1u : 0u);
                    umma_commit(&mempty[ms]);
                    if (jj == npieces - 1) {
                        umma_commit(&accfull);
                        umma_commit(&abempty[buf]);
                    }
                    if (hi + 1 < nheads) issue_scores(hi + 1, jj);
                }
            }
        }
    } else if (nheads > 0) {
        // ------------------------------------------------------------ mask + epilogue warps
        const int q = warp & 3;                    // TMEM lane quarter this warp may access
        const int half = (warp - 2) >> 2;          // which 32 columns of a piece / 64 columns of acc
        const int mt = (warp - 2) * 32 + lane;     // 0..255 among the mask threads
        const int rl = q * 32 + lane;              // row inside the 128-row block
        const int r = rb * 128 + rl;               // row inside the chunk
        const int isub = r >> 5;
        const uint32_t tlane = (uint32_t)(q * 32) << 16;
        float *vec = reinterpret_cast<float *>(smem + GB_OFF_VEC);
        float *part = reinterpret_cast<float *>(smem + GB_OFF_PART);
        uint32_t wcount = 0;                       // pieces this thread has written to each M slot so far

        // this thread's 64 values of its own C (DC) or B (DB) row, packed bf16
        uint32_t Rp[32];
        {
            const __nv_bfloat16 *src = (const __nv_bfloat16 *)(DC ? p.Cm : p.Bm) + (size_t)b * p.bc_bs +
                                       (size_t)(tok0 + r) * p.G * 128 + (size_t)g * 128 + half * 64;
            const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint4 v = __ldg(s4 + k);
                Rp[4 * k] = v.x; Rp[4 * k + 1] = v.y; Rp[4 * k + 2] = v.z; Rp[4 * k + 3] = v.w;
            }
        }
        float sums[64];
#pragma unroll
        for (int k = 0; k < 64; ++k) sums[k] = 0.f;

        for (int hi = 0; hi < nheads; ++hi) {
            const int h = h_begin + hi;
            float *cs2 = vec + (hi & 1) * GB_VEC_FLOATS, *cf = cs2 + 256, *dtv = cs2 + 512, *blk = cs2 + 768;
            {
                const size_t vo = (((size_t)b * p.H + h) * p.ncs + c) << 8;
                cs2[mt] = p.cs[vo + mt] * kLog2e;
                dtv[mt] = p.dtT[vo + mt];
            }
            bar_mask_warps();
            // cf: DC  e^{cs[t|31] - cs[t]} dt_t  (column factor) ; DB  e^{cs[t] - cs[t&~31]} (column factor)
            cf[mt] = DC ? ex2f(cs2[mt | 31] - cs2[mt]) * dtv[mt] : ex2f(cs2[mt] - cs2[mt & ~31]);
            if (mt < 64) {
                const int i = mt >> 3, j = mt & 7;   // blk[i][j] = e^{cs[32 i] - cs[32 j + 31]}, j < i
                blk[mt] = (j < i) ? ex2f(cs2[32 * i] - cs2[32 * j + 31]) : 0.f;
            }
            bar_mask_warps();
            const float csr = cs2[r];
            const float dtr = dtv[r];
            // row factor: DC  e^{cs_r - cs[r&~31]} ; DB  e^{cs[r|31] - cs_r} dt_r
            const float rowf = DC ? ex2f(csr - cs2[r & ~31]) : ex2f(cs2[r | 31] - csr) * dtr;
            const float offs = DC ? ex2f(csr) : ex2f(cs2[255] - csr) * dtr;

            // ---- masked pieces: this thread does the 32 columns `half` of every piece
            for (int jj = 0; jj < npieces; ++jj) {
                const int ms = jj & 1;
                const int cb = colbase + jj * 64 + half * 32;
                const int jsub = cb >> 5;
                const bool zero = DC ? (jsub > isub) : (jsub < isub);
                float v[32];
                mbar_wait(&sfull[jj], hi & 1, abortp, p.status);
                tc_fence_after_sync();
                if (!zero) tmem_ld32(tm + tlane + jj * 64 + half * 32, v);
                tc_fence_before_sync();
                mbar_arrive(&sempty[jj]);
                uint32_t pk[16];
                if (zero) {
#pragma unroll
                    for (int k = 0; k < 16; ++k) pk[k] = 0u;
                } else {
                    if (jsub != isub) {
                        if (DC) {
                            const float f = rowf * blk[isub * 8 + jsub];
#pragma unroll
                            for (int k = 0; k < 32; k += 4) {
                                const float4 cv = *reinterpret_cast<const float4 *>(cf + cb + k);
                                v[k] *= cv.x * f;
                                v[k + 1] *= cv.y * f;
                                v[k + 2] *= cv.z * f;
                                v[k + 3] *= cv.w * f;
                            }
                        } else {
                            const float bl = blk[jsub * 8 + isub];
#pragma unroll
                            for (int k = 0; k < 32; k += 4) {
                                const float4 cv = *reinterpret_cast<const float4 *>(cf + cb + k);
                                v[k] *= rowf * (cv.x * bl);
                                v[k + 1] *= rowf * (cv.y * bl);
                                v[k + 2] *= rowf * (cv.z * bl);
                                v[k + 3] *= rowf * (cv.w * bl);
                            }
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < 32; k += 4) {
                            const float4 cc = *reinterpret_cast<const float4 *>(cs2 + cb + k);
                            const float ccv[4] = {cc.x, cc.y, cc.z, cc.w};
                            float dv[4] = {dtr, dtr, dtr, dtr};
                            if (DC) {
                                const float4 d4 = *reinterpret_cast<const float4 *>(dtv + cb + k);
                                dv[0] = d4.x; dv[1] = d4.y; dv[2] = d4.z; dv[3] = d4.w;
                            }
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int col = cb + k + e;
                                const bool on = DC ? (col <= r) : (col >= r);
                                const float ex = (DC ? ex2f(csr - ccv[e]) : ex2f(ccv[e] - csr)) * dv[e];
                                v[k + e] = on ? v[k + e] * ex : 0.f;
                            }
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 16; ++k) pk[k] = pack2(v[2 * k], v[2 * k + 1]);
                }
                // the slot is free once the MMAs of the piece that last used it are done
                const uint32_t nth = wcount >> (ms * 16) & 0xffffu;
                if (nth >= 1) mbar_wait(&mempty[ms], (nth - 1) & 1, abortp, p.status);
                wcount += 1u << (ms * 16);
                unsigned char *mrow = smem + GB_OFF_M + ms * 16384 + rl * 128;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const int chunk16 = half * 4 + ch;
                    *reinterpret_cast<uint4 *>(mrow + ((chunk16 ^ (rl & 7)) << 4)) =
                        make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
                }
                fence_proxy_async_smem();
                mbar_arrive(&mfull[ms]);
            }

            // ---- epilogue of this head: columns [64 half, 64 half + 64) of both accumulators
            mbar_wait(&accfull, hi & 1, abortp, p.status);
            tc_fence_after_sync();
            float d1 = 0.f, d2 = 0.f;
#pragma unroll
            for (int b16 = 0; b16 < 4; ++b16) {
                float a1[16], a2[16];
                tmem_ld16(tm + tlane + 256 + half * 64 + b16 * 16, a1);
                tmem_ld16(tm + tlane + 384 + half * 64 + b16 * 16, a2);
#pragma unroll
                for (int k = 0; k < 16; k += 2) {
                    const float2 rv = unpack2(Rp[b16 * 8 + (k >> 1)]);
                    const float t0 = offs * a2[k], t1 = offs * a2[k + 1];
                    d1 = fmaf(rv.x, a1[k], d1);
                    d1 = fmaf(rv.y, a1[k + 1], d1);
                    d2 = fmaf(rv.x, t0, d2);
                    d2 = fmaf(rv.y, t1, d2);
                    sums[b16 * 16 + k] += a1[k] + t0;
                    sums[b16 * 16 + k + 1] += a1[k + 1] + t1;
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&accempty);
            float *pp = part + (hi & 1) * 384;
            if (half == 1) {
                pp[rl] = d1;
                pp[128 + rl] = d2;
            }
            bar_mask_warps();
            if (half == 0) {
                const size_t vo = ((((size_t)b * p.H + h) * p.ncs + c) << 8) + r;
                const float e1 = d1 + pp[rl], e2 = d2 + pp[128 + rl];
                // the inter-chunk parts (rho2, psi2) come from the dstate and dx kernels
                if (DC) p.rho[vo] = e1;
                else p.psi[vo] = e1;
                (void)e2;
            }
        }

        // ---- partial slice of the group sum: [B, seg, G, nsl, N] fp32
        {
            const size_t segcap = (size_t)p.ncs * 256;
            const size_t tl = (size_t)c * 256 + r;
            float *dst = (DC ? p.pC : p.pB) + ((((size_t)b * segcap + tl) * p.G + g) * nsl + sl) * 128 + half * 64;
#pragma unroll
            for (int k = 0; k < 64; k += 4)
                *reinterpret_cast<float4 *>(dst + k) = make_float4(sums[k], sums[k + 1], sums[k + 2], sums[k + 3]);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tm, 512);
    }
}

cudaError_t launch_grad_bc_tc(const SegParams &p, const TcMaps &m, int mode, cudaStream_t st) {
    dim3 grid(p.nc * 2, p.nsl * p.G, p.B);
    cudaError_t e;
    if (mode == GB_DC) {
        e = cudaFuncSetAttribute(k_grad_bc_tc<GB_DC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GB_SMEM);
        if (e != cudaSuccess) return e;
        k_grad_bc_tc<GB_DC><<<grid, GB_THREADS, GB_SMEM, st>>>(p, m.dy, m.x, m.Bm, m.Hbf);
    } else {
        e = cudaFuncSetAttribute(k_grad_bc_tc<GB_DB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GB_SMEM);
        if (e != cudaSuccess) return e;
        k_grad_bc_tc<GB_DB><<<grid, GB_THREADS, GB_SMEM, st>>>(p, m.x, m.dy, m.Cm, m.Gbf);
    }
    return cudaGetLastError();
}

}  // namespace ssd
