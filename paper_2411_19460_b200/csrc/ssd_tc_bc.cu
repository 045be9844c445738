// Tensor-core kernel for the two masked products whose score matrix is per head and whose result
// is summed over the heads of a group (bf16 I/O, P = 64, N = 128, Q = 256):
//
//   GB_DC: dC_t = sum_h [ sum_{s<=t} W_h[t,s] B_s + e^{cs_t} dy_t^T H_in ]              rows t
//   GB_DB: dB_s = sum_h [ sum_{t>=s} W_h[t,s] C_t + dt_s e^{cs_last-cs_s} x_s^T Gout ]  rows s
//   with W_h[t,s] = (dy_t . x_s) e^{cs_t-cs_s} dt_s   (s <= t)
//
// and the per-head scalars the decay gradient needs:
//   rho_t = sum_s W_h[t,s] (C_t.B_s)  = C_t . (intra-chunk part of this head's dC_t)     (GB_DC)
//   psi_s = sum_t W_h[t,s] (C_t.B_s)  = B_s . (intra-chunk part of this head's dB_s)     (GB_DB)
// (Eq. 1 of the paper regrouped by chunks; cs = inclusive cumsum of dt*A inside the chunk.)
//
// One CTA owns (chunk, 128-row block, group, a range of the group's heads).  Once per CTA the tile
// CB = C B^T (or its transpose) goes to TMEM and the group's value rows (B or C) to shared memory.
// Per head:
//   MMA warp   : score units S = Rows * Cols^T (K = P, 128 columns) into a TMEM buffer;
//                acc += W * V per finished unit; acc += (scaled Rows) * State.
//   vector warp : the head's cumulative sums, step sizes and mask factors, one head ahead
//   16 mask warps: S -> W (decay mask, same factorisation and same bf16 rounding in both modes, so
//                that rho and psi are built from identical W and rho - psi cancels cleanly), stored
//                to shared memory as the A operand; the row sums of W o CB give rho / psi; then the
//                head's row operand scaled by e^{cs_t} (or dt_s e^{cs_last-cs_s}) as one more
//                64-wide K piece, which folds the inter-chunk term into the same accumulator.
// The accumulator stays in TMEM across all heads of the CTA: the head sum costs nothing, and there
// is no per-head epilogue.  It is written once, as an fp32 partial slice; a later kernel adds the
// slices of a group in a fixed order.
#include <type_traits>

#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

using namespace sm100;

namespace {

constexpr int GB_THREADS = 608;           // warp 0 producer, warp 1 MMA, warps 2..17 mask, warp 18 vectors
constexpr uint32_t GB_OFF_V = 0;          // 64 KB  [n-half][ncols rows][128 B], kept for all heads
constexpr uint32_t GB_OFF_R = 65536;      // 2 x 16 KB  the head's row operand (dy or x rows of the block)
constexpr uint32_t GB_OFF_C = 98304;      // 32 KB  the head's column operand (x or dy rows of the column range)
constexpr uint32_t GB_OFF_ST = 131072;    // 16 KB  bf16 chunk state [n-half][64 p rows][128 B]
constexpr uint32_t GB_OFF_M = 147456;     // 2 x 32 KB  masked units (two 16 KB pieces each); first use: C/B rows for CB
constexpr uint32_t GB_OFF_VEC = 212992;   // per-head vectors, double buffered
constexpr uint32_t GB_VEC_FLOATS = 256 * 3 + 64;
constexpr uint32_t GB_OFF_PART = GB_OFF_VEC + 2 * GB_VEC_FLOATS * 4;   // 2 x 3 x 128 floats
constexpr uint32_t GB_SMEM = GB_OFF_PART + 2 * 384 * 4 + 1024;

constexpr uint32_t TM_CB = 0, TM_S = 256, TM_ACC = 384;

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
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
             const __grid_constant__ CUtensorMap tmG,                  // DC: Cm ; DB: Bm  (rows of the CB tile)
             const __grid_constant__ CUtensorMap tmSt) {               // DC: Hbf; DB: Gbf
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar_ld, bar_cb, rfull[2], rempty[2], cfull[2], cempty[2], stfull, stempty, sfull, sempty,
        mfull[2], mempty[2], accfull, vfull[2], vempty[2];
    __shared__ uint32_t tmem_base, abort_flag;

    constexpr bool DC = (MODE == GB_DC);
    // 1-D grid; the first half are the long CTAs (the row block with the larger column range), so the
    // tail of the launch is filled with short ones
    const int nc = p.nc, nsl = p.nsl, ny = nsl * p.G;
    const int half_grid = (int)(gridDim.x >> 1), jid = (int)blockIdx.x % half_grid;
    const bool is_long = (int)blockIdx.x < half_grid;
    const int rb = DC ? (is_long ? 1 : 0) : (is_long ? 0 : 1);
    const int c = jid % nc, yid = (jid / nc) % ny, b = jid / (nc * ny);
    const int g = yid / nsl, sl = yid % nsl;
    const int hps = (p.hpg + nsl - 1) / nsl;
    const int h_begin = g * p.hpg + sl * hps;
    const int h_end = min(g * p.hpg + p.hpg, h_begin + hps);
    const int nheads = max(h_end - h_begin, 0);
    const int colbase = DC ? 0 : rb * 128;
    const int ncols = DC ? (rb + 1) * 128 : 256 - rb * 128;
    const int nunits = ncols >> 7;            // units of two 64-column pieces
    const int ncb = (ncols == 128) ? 2 : 1;   // column-operand buffers that fit in 32 KB
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tok0 = p.t0 + c * 256;
    const int slot = DC ? c : c + 1;

    if (tid == 0) {
        mbar_init(&bar_ld, 1);
        mbar_init(&bar_cb, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&rfull[i], 1);
            mbar_init(&rempty[i], 1 + 512);   // inter-chunk MMAs (one commit) + the mask threads that scaled it
            mbar_init(&cfull[i], 1);
            mbar_init(&cempty[i], 1);
            mbar_init(&mfull[i], 512);
            mbar_init(&vfull[i], 32);
            mbar_init(&vempty[i], 512);
            mbar_init(&mempty[i], 1);
        }
        mbar_init(&stfull, 1);
        mbar_init(&stempty, 1);
        mbar_init(&sfull, 1);
        mbar_init(&sempty, 512);
        mbar_init(&accfull, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc(&tmem_base, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();
    pdl_wait();       // barriers and tensor memory are set up; everything below reads what earlier kernels wrote
    const uint32_t tm = tmem_base;
    volatile uint32_t *abortp = &abort_flag;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0 && nheads > 0) {
            mbar_arrive_expect_tx(&bar_ld, 32768u + (uint32_t)ncols * 256u);
            tma_load_3d(smem + GB_OFF_M, &tmG, &bar_ld, g * 128, tok0 + rb * 128, b);
            tma_load_3d(smem + GB_OFF_M + 16384, &tmG, &bar_ld, g * 128 + 64, tok0 + rb * 128, b);
            for (int nh = 0; nh < 2; ++nh)
                for (int r0 = 0; r0 < ncols; r0 += 128)
                    tma_load_3d(smem + GB_OFF_V + nh * ncols * 128 + r0 * 128, &tmV, &bar_ld, g * 128 + nh * 64,
                                tok0 + colbase + r0, b);
            const int strow = (b * (p.ncs + 1) + slot) * p.H;
            for (int hi = 0; hi < nheads; ++hi) {
                const int h = h_begin + hi, rbuf = hi & 1, cbuf = hi % ncb, cuse = hi / ncb;
                if (hi >= 2) mbar_wait(&rempty[rbuf], ((hi >> 1) - 1) & 1, abortp, p.status);
                mbar_arrive_expect_tx(&rfull[rbuf], 16384);
                tma_load_3d(smem + GB_OFF_R + rbuf * 16384, &tmRow, &rfull[rbuf], h * 64, tok0 + rb * 128, b);
                if (cuse >= 1) mbar_wait(&cempty[cbuf], (cuse - 1) & 1, abortp, p.status);
                mbar_arrive_expect_tx(&cfull[cbuf], (uint32_t)ncols * 128u);
                for (int r0 = 0; r0 < ncols; r0 += 128)
                    tma_load_3d(smem + GB_OFF_C + cbuf * 16384 + r0 * 128, &tmCol, &cfull[cbuf], h * 64,
                                tok0 + colbase + r0, b);
                if (hi >= 1) mbar_wait(&stempty, (hi - 1) & 1, abortp, p.status);
                mbar_arrive_expect_tx(&stfull, 16384);
                tma_load_3d(smem + GB_OFF_ST, &tmSt, &stfull, 0, (strow + h) * 64, 0);
                tma_load_3d(smem + GB_OFF_ST + 8192, &tmSt, &stfull, 64, (strow + h) * 64, 0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && nheads > 0) {
            const uint32_t sV = smem_u32(smem + GB_OFF_V), sR = smem_u32(smem + GB_OFF_R);
            const uint32_t sC = smem_u32(smem + GB_OFF_C), sSt = smem_u32(smem + GB_OFF_ST);
            const uint32_t sM = smem_u32(smem + GB_OFF_M);
            const uint32_t idCB = umma_idesc_bf16(128, (uint32_t)ncols, false, false);
            const uint32_t idS = umma_idesc_bf16(128, 128, false, false);   // rows (K-major) x 128 cols (K-major)
            const uint32_t idW = umma_idesc_bf16(128, 128, false, true);    // W / scaled rows (K-major) x V / state (MN-major)
            // CB tile, once
            mbar_wait(&bar_ld, 0, abortp, p.status);
            tc_fence_after_sync();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                umma_bf16(tm + TM_CB, umma_desc_sw128(sM + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024),
                          umma_desc_sw128(sV + (kk >> 2) * (ncols * 128) + (kk & 3) * 32, 16, 1024), idCB, kk ? 1u : 0u);
            umma_commit(&bar_cb);

            // Descriptors as (low word, high word): inside the unrolled loops every operand address is the low
            // word plus a compile-time constant (16-byte units), so an MMA costs the issuing thread an add or two.
            const uint64_t dR = umma_desc_sw128(sR, 16, 1024), dC = umma_desc_sw128(sC, 16, 1024);
            const uint64_t dMm = umma_desc_sw128(sM, 16, 1024), dSt = umma_desc_sw128(sSt, 8192, 1024);
            const uint64_t dV = umma_desc_sw128(sV, (uint32_t)ncols * 128u, 1024);
            const uint32_t loR = (uint32_t)dR, hiR = (uint32_t)(dR >> 32), loC = (uint32_t)dC, hiC = (uint32_t)(dC >> 32);
            const uint32_t loM = (uint32_t)dMm, hiM = (uint32_t)(dMm >> 32), loSt = (uint32_t)dSt, hiSt = (uint32_t)(dSt >> 32);
            const uint32_t loV = (uint32_t)dV, hiV = (uint32_t)(dV >> 32);

            auto run = [&](auto nu_c) {
                constexpr int NU = decltype(nu_c)::value;      // score units per head: 1 or 2
                constexpr int NCB = (NU == 1) ? 2 : 1;         // column-operand buffers
                // scores of unit u of head hi into the S buffer (128 columns = one N = 128 product, K = P)
                auto issue_scores = [&](int hi, int u, uint32_t lo_r, uint32_t lo_c) {
                    if (u == 0) {
                        const int rbuf = hi & 1, cbuf = (NCB == 2) ? (hi & 1) : 0, cuse = (NCB == 2) ? (hi >> 1) : hi;
                        mbar_wait(&rfull[rbuf], (hi >> 1) & 1, abortp, p.status);
                        mbar_wait(&cfull[cbuf], cuse & 1, abortp, p.status);
                        tc_fence_after_sync();
                    }
                    umma_bf16_fixed<false>(tm + TM_S, umma_desc_words(lo_r, hiR), umma_desc_words(lo_c, hiC), idS);
#pragma unroll
                    for (int k = 1; k < 4; ++k)
                        umma_bf16_fixed<true>(tm + TM_S, umma_desc_words(lo_r + k * 2, hiR), umma_desc_words(lo_c + k * 2, hiC), idS);
                    umma_commit(&sfull);
                };
                uint32_t sidx = 0;   // index of the score unit the mask warps are working on
                uint32_t job = 0;    // M buffers consumed so far
                issue_scores(0, 0, loR, loC);
                if (NU == 1) umma_commit(&cempty[0]);
                for (int hi = 0; hi < nheads; ++hi) {
                    const int rbuf = hi & 1, cbuf = (NCB == 2) ? (hi & 1) : 0;
                    const uint32_t lo_r = loR + rbuf * 1024, lo_c = loC + cbuf * 1024;
                    const int nrbuf = (hi + 1) & 1, ncbuf = (NCB == 2) ? ((hi + 1) & 1) : 0;
#pragma unroll
                    for (int u = 0; u < NU; ++u) {
                        // next score unit as soon as the mask warps have copied the current one out of TMEM
                        const bool last_u = (u == NU - 1);
                        if (!last_u || hi + 1 < nheads) {
                            mbar_wait(&sempty, sidx & 1, abortp, p.status);
                            tc_fence_after_sync();
                            if (!last_u) {
                                issue_scores(hi, u + 1, lo_r, lo_c + (u + 1) * 1024);
                                if (u + 1 == NU - 1) umma_commit(&cempty[cbuf]);
                            } else {
                                issue_scores(hi + 1, 0, loR + nrbuf * 1024, loC + ncbuf * 1024);
                                if (NU == 1) umma_commit(&cempty[ncbuf]);
                            }
                        }
                        ++sidx;
                        const uint32_t mb = job & 1;
                        mbar_wait(&mfull[mb], (job >> 1) & 1, abortp, p.status);
                        tc_fence_after_sync();
                        const uint32_t lo_m = loM + mb * 2048, lo_v = loV + u * 1024;   // 32 KB buffers; 128 rows of V
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const uint64_t ad = umma_desc_words(lo_m + (k >> 2) * 1024 + (k & 3) * 2, hiM);
                            const uint64_t bd = umma_desc_words(lo_v + k * 128, hiV);
                            if (u == 0 && k == 0) {
                                if (hi == 0) umma_bf16_fixed<false>(tm + TM_ACC, ad, bd, idW);
                                else umma_bf16_fixed<true>(tm + TM_ACC, ad, bd, idW);
                            } else {
                                umma_bf16_fixed<true>(tm + TM_ACC, ad, bd, idW);
                            }
                        }
                        umma_commit(&mempty[mb]);
                        ++job;
                    }
                    {   // inter-chunk piece: (scaled rows) [128 x 64] x state [64 x 128]
                        const uint32_t mb = job & 1;
                        mbar_wait(&stfull, hi & 1, abortp, p.status);
                        mbar_wait(&mfull[mb], (job >> 1) & 1, abortp, p.status);
                        tc_fence_after_sync();
                        const uint32_t lo_m = loM + mb * 2048;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_bf16_fixed<true>(tm + TM_ACC, umma_desc_words(lo_m + k * 2, hiM),
                                                  umma_desc_words(loSt + k * 128, hiSt), idW);
                        umma_commit(&mempty[mb]);
                        umma_commit(&stempty);
                        umma_commit(&rempty[hi & 1]);
                        ++job;
                    }
                }
                umma_commit(&accfull);
            };
            if (nunits == 2) run(std::integral_constant<int, 2>{});
            else run(std::integral_constant<int, 1>{});
        }
    } else if (warp == 18) {
        // ------------------------------------------------------------ vector warp
        // Per head: the 256 cumulative sums (log2 units) and step sizes of the chunk, the column factor
        // of the mask factorisation and the 8 x 8 table of sub-tile-to-sub-tile decays, written to a
        // double-buffered area one head ahead of the mask warps.  Each lane owns 8 consecutive steps.
        if (nheads > 0) {
            float *vec = reinterpret_cast<float *>(smem + GB_OFF_VEC);
            for (int hi = 0; hi < nheads; ++hi) {
                const int buf = hi & 1, h = h_begin + hi;
                const size_t vo = ((((size_t)b * p.H + h) * p.ncs + c) << 8) + lane * 8;
                const float4 c0 = __ldg(reinterpret_cast<const float4 *>(p.cs + vo));
                const float4 c1 = __ldg(reinterpret_cast<const float4 *>(p.cs + vo + 4));
                const float4 d0 = __ldg(reinterpret_cast<const float4 *>(p.dtT + vo));
                const float4 d1 = __ldg(reinterpret_cast<const float4 *>(p.dtT + vo + 4));
                if (hi >= 2) mbar_wait(&vempty[buf], ((hi >> 1) - 1) & 1, abortp, p.status);
                float *cs2 = vec + buf * GB_VEC_FLOATS, *cf = cs2 + 256, *dtv = cs2 + 512, *blk = cs2 + 768;
                const float cv[8] = {c0.x * kLog2e, c0.y * kLog2e, c0.z * kLog2e, c0.w * kLog2e,
                                     c1.x * kLog2e, c1.y * kLog2e, c1.z * kLog2e, c1.w * kLog2e};
                const float dv[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
                *reinterpret_cast<float4 *>(cs2 + lane * 8) = make_float4(cv[0], cv[1], cv[2], cv[3]);
                *reinterpret_cast<float4 *>(cs2 + lane * 8 + 4) = make_float4(cv[4], cv[5], cv[6], cv[7]);
                *reinterpret_cast<float4 *>(dtv + lane * 8) = d0;
                *reinterpret_cast<float4 *>(dtv + lane * 8 + 4) = d1;
                __syncwarp();
                // cf: DC  e^{cs[t|31] - cs[t]} dt_t ; DB  e^{cs[t] - cs[t&~31]}
                const float ref = DC ? cs2[(lane * 8) | 31] : cs2[(lane * 8) & ~31];
                float o[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) o[k] = DC ? ex2f(ref - cv[k]) * dv[k] : ex2f(cv[k] - ref);
                *reinterpret_cast<float4 *>(cf + lane * 8) = make_float4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<float4 *>(cf + lane * 8 + 4) = make_float4(o[4], o[5], o[6], o[7]);
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    const int idx = lane + 32 * w, i = idx >> 3, j = idx & 7;   // blk[i][j] = e^{cs[32 i] - cs[32 j + 31]}, j < i
                    blk[idx] = (j < i) ? ex2f(cs2[32 * i] - cs2[32 * j + 31]) : 0.f;
                }
                mbar_arrive(&vfull[buf]);
            }
        }
    } else if (nheads > 0) {
        // ------------------------------------------------------------ mask warps
        // Four warps per TMEM lane quarter: warp (q, quar) owns rows 32 q .. 32 q + 31 of the block and
        // the 16-column slice `quar` of every 64-column piece (columns 32 quar .. of the accumulator).
        const int q = warp & 3;
        const int quar = (warp - 2) >> 2;
        const int rl = q * 32 + lane;              // row inside the 128-row block
        const int r = rb * 128 + rl;               // row inside the chunk
        const int isub = r >> 5;
        const uint32_t tlane = (uint32_t)(q * 32) << 16;
        float *vec = reinterpret_cast<float *>(smem + GB_OFF_VEC);
        float *part = reinterpret_cast<float *>(smem + GB_OFF_PART);   // [head parity][3][128]
        uint32_t job = 0, sidx = 0;

        for (int hi = 0; hi < nheads; ++hi) {
            float *cs2 = vec + (hi & 1) * GB_VEC_FLOATS, *cf = cs2 + 256, *dtv = cs2 + 512, *blk = cs2 + 768;
            mbar_wait(&vfull[hi & 1], (hi >> 1) & 1, abortp, p.status);
            const float csr = cs2[r];
            const float dtr = dtv[r];
            // row factor: DC  e^{cs_r - cs[r&~31]} ; DB  e^{cs[r|31] - cs_r} dt_r
            const float rowf = DC ? ex2f(csr - cs2[r & ~31]) : ex2f(cs2[r | 31] - csr) * dtr;
            const float offs = DC ? ex2f(csr) : ex2f(cs2[255] - csr) * dtr;
            float2 dacc = make_float2(0.f, 0.f);
            if (hi == 0) {
                mbar_wait(&bar_cb, 0, abortp, p.status);
                tc_fence_after_sync();
            }

            for (int u = 0; u < nunits; ++u) {
                // ---- copy this thread's two 16-column score slices of the unit out of TMEM
                float v[2][16];
                bool z[2];
                mbar_wait(&sfull, sidx & 1, abortp, p.status);
                tc_fence_after_sync();
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    const int jsub = (colbase + u * 128 + w * 64 + quar * 16) >> 5;
                    z[w] = DC ? (jsub > isub) : (jsub < isub);
                    if (!z[w]) tmem_ld16_nowait(tm + tlane + TM_S + w * 64 + quar * 16, v[w]);
                }
#pragma unroll
                for (int w = 0; w < 2; ++w)
                    if (!z[w]) tmem_ld_wait16(v[w]);
                tc_fence_before_sync();
                mbar_arrive(&sempty);
                ++sidx;
                const uint32_t mb = job & 1;
                if (job >= 2) mbar_wait(&mempty[mb], ((job >> 1) - 1) & 1, abortp, p.status);
                ++job;
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    const int cb = colbase + u * 128 + w * 64 + quar * 16;   // first column of the slice (in chunk)
                    const int jsub = cb >> 5;
                    unsigned char *mrow = smem + GB_OFF_M + mb * 32768 + w * 16384 + rl * 128;
                    uint32_t pk[8];
                    if (z[w]) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) pk[k] = 0u;
                    } else {
                        float *vv = v[w];
                        float cbv[16];
                        tmem_ld16_nowait(tm + tlane + TM_CB + u * 128 + w * 64 + quar * 16, cbv);
                        if (jsub != isub) {
                            // (packed fp32 pairs; DC: cf (rowf blk) ; DB: rowf (cf blk) -- the same two factors
                            //  (dn dt) and (up blk) multiplied in the same order in both modes)
                            const float s1 = DC ? rowf * blk[isub * 8 + jsub] : blk[jsub * 8 + isub];
                            const float2 s1v = make_float2(s1, s1), rfv = make_float2(rowf, rowf);
#pragma unroll
                            for (int k = 0; k < 16; k += 4) {
                                const float4 cv = *reinterpret_cast<const float4 *>(cf + cb + k);
                                float2 m0 = __fmul2_rn(make_float2(cv.x, cv.y), s1v);
                                float2 m1 = __fmul2_rn(make_float2(cv.z, cv.w), s1v);
                                if (!DC) {
                                    m0 = __fmul2_rn(rfv, m0);
                                    m1 = __fmul2_rn(rfv, m1);
                                }
                                const float2 w0 = __fmul2_rn(make_float2(vv[k], vv[k + 1]), m0);
                                const float2 w1 = __fmul2_rn(make_float2(vv[k + 2], vv[k + 3]), m1);
                                vv[k] = w0.x; vv[k + 1] = w0.y; vv[k + 2] = w1.x; vv[k + 3] = w1.y;
                            }
                        } else {
#pragma unroll
                            for (int k = 0; k < 16; k += 4) {
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
                                    vv[k + e] = on ? vv[k + e] * ex : 0.f;
                                }
                            }
                        }
#pragma unroll
                        for (int k = 0; k < 8; ++k) pk[k] = pack2(vv[2 * k], vv[2 * k + 1]);
                        // row sum of W o CB, in fp32 from the unrounded W: both modes form bit-identical
                        // W and CB elements, so rho and psi are row and column sums of one matrix
                        tmem_ld_wait16(cbv);
#pragma unroll
                        for (int k = 0; k < 16; k += 2)
                            dacc = __ffma2_rn(make_float2(vv[k], vv[k + 1]), make_float2(cbv[k], cbv[k + 1]), dacc);
                    }
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        const int chunk16 = quar * 2 + ch;
                        *reinterpret_cast<uint4 *>(mrow + ((chunk16 ^ (rl & 7)) << 4)) =
                            make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
                    }
                }
                tc_fence_before_sync();
                fence_proxy_async_smem();
                mbar_arrive(&mfull[mb]);
            }
            mbar_arrive(&vempty[hi & 1]);

            // ---- inter-chunk piece: this thread's 16 values of its row of the head's row operand, scaled
            {
                const int rbuf = hi & 1;
                mbar_wait(&rfull[rbuf], (hi >> 1) & 1, abortp, p.status);
                const unsigned char *rrow = smem + GB_OFF_R + rbuf * 16384 + rl * 128;
                uint4 o[2];
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const uint4 qv = *reinterpret_cast<const uint4 *>(rrow + (((quar * 2 + k) ^ (rl & 7)) << 4));
                    const uint32_t *qw = reinterpret_cast<const uint32_t *>(&qv);
                    uint32_t *ow = reinterpret_cast<uint32_t *>(&o[k]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = unpack2(qw[e]);
                        ow[e] = pack2(f.x * offs, f.y * offs);
                    }
                }
                mbar_arrive(&rempty[rbuf]);
                const uint32_t mb = job & 1;
                if (job >= 2) mbar_wait(&mempty[mb], ((job >> 1) - 1) & 1, abortp, p.status);
                ++job;
                unsigned char *mrow = smem + GB_OFF_M + mb * 32768 + rl * 128;
#pragma unroll
                for (int k = 0; k < 2; ++k)
                    *reinterpret_cast<uint4 *>(mrow + (((quar * 2 + k) ^ (rl & 7)) << 4)) = o[k];
                fence_proxy_async_smem();
                mbar_arrive(&mfull[mb]);
            }

            // ---- rho / psi of this head: the four column slices of a row meet through shared memory
            {
                const float dsum = dacc.x + dacc.y;
                float *pp = part + (hi & 1) * 384;
                if (quar > 0) pp[(quar - 1) * 128 + rl] = dsum;
                asm volatile("bar.sync %0, 128;" ::"r"(2 + q) : "memory");
                if (quar == 0) {
                    const size_t vo = ((((size_t)b * p.H + h_begin + hi) * p.ncs + c) << 8) + r;
                    const float e = ((dsum + pp[rl]) + pp[128 + rl]) + pp[256 + rl];
                    if (DC) p.rho[vo] = e;
                    else p.psi[vo] = e;
                }
            }
        }

        // ---- the CTA's partial slice of the group sum: [B, seg, G, nsl, N] fp32
        mbar_wait(&accfull, 0, abortp, p.status);
        tc_fence_after_sync();
        {
            const size_t segcap = (size_t)p.ncs * 256;
            const size_t tl = (size_t)c * 256 + r;
            float *dst = (DC ? p.pC : p.pB) + ((((size_t)b * segcap + tl) * p.G + g) * nsl + sl) * 128 + quar * 32;
            float a[32];
            tmem_ld32(tm + tlane + TM_ACC + quar * 32, a);
#pragma unroll
            for (int k = 0; k < 32; k += 4)
                *reinterpret_cast<float4 *>(dst + k) = make_float4(a[k], a[k + 1], a[k + 2], a[k + 3]);
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
    dim3 grid(p.nc * 2 * p.nsl * p.G * p.B);
    cudaError_t e;
    if (mode == GB_DC) {
        e = cudaFuncSetAttribute(k_grad_bc_tc<GB_DC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GB_SMEM);
        if (e != cudaSuccess) return e;
        return launch_pdl(k_grad_bc_tc<GB_DC>, grid, dim3(GB_THREADS), (size_t)GB_SMEM, st, p, m.dy, m.x, m.Bm, m.Cm, m.Hbf);
    } else {
        e = cudaFuncSetAttribute(k_grad_bc_tc<GB_DB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GB_SMEM);
        if (e != cudaSuccess) return e;
        return launch_pdl(k_grad_bc_tc<GB_DB>, grid, dim3(GB_THREADS), (size_t)GB_SMEM, st, p, m.x, m.dy, m.Cm, m.Bm, m.Gbf);
    }
    return cudaGetLastError();
}

}  // namespace ssd
