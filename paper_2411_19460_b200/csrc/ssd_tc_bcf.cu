// Tensor-core kernel for dB and dC together (bf16 I/O, P = 64, N = 128, Q = 256).  Both are products of
// the same masked, per-head score tile
//     W_h[t,s] = (dy_t . x_s) e^{cs_t-cs_s} dt_s   (s <= t),
//   dC_t = sum_h [ sum_s W_h[t,s] B_s + e^{cs_t} dy_t^T H_in ]               (W as the K-major A operand)
//   dB_s = sum_h [ sum_t W_h[t,s] C_t + dt_s e^{cs_last-cs_s} x_s^T Gout ]   (W as the MN-major A operand)
// so a CTA masks one 128 x 128 tile of W per head and feeds it to both products.  Per head it also forms
// the scalars of the decay gradient, rho_t = sum_s W[t,s] (C_t.B_s) and psi_s = sum_t W[t,s] (C_t.B_s):
// row and column sums of one fp32 matrix.  (Eq. 1 of the paper regrouped by chunks; cs = inclusive cumsum
// of dt*A inside the chunk.)
//
// One CTA owns (chunk, tile, group, a range of the group's heads); the three causal tiles of a 256-step
// chunk are (t-block, s-block) = (1,0) full, (0,0) and (1,1) diagonal.  TMEM holds CB = C B^T of the tile
// (128 columns), the score buffer (128), and the two accumulators (128 each), which stay there across all
// heads of the CTA and leave once, as fp32 partial slices that a later kernel adds in a fixed order.
// Shared memory holds the C rows of the t-block and the B rows of the s-block for the whole CTA (operands
// of CB, and the MN-major B operands of the two products), and per head the dy / x rows (double buffered),
// one buffer for the scaled rows of an inter-chunk term, and the two bf16 chunk states (double buffered: the
// second copies live where the head sum of W goes at the very end, which is free until then, so a state's
// load has a whole head of time to land).
// The inter-chunk terms are spread over the tiles: (0,0) adds dC's for t-block 0, (1,0) dB's for s-block 0,
// (1,1) dC's for t-block 1 and then dB's for s-block 1.
//   warp 0 producer (TMA) | warp 1 MMA issuer | warps 2..17 mask warps | warp 18 per-head vectors
#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

using namespace sm100;

namespace {

constexpr int GF_THREADS = 608;
constexpr uint32_t GF_OFF_CT = 0;          // 32 KB  C rows of the t-block  [n-half][128 rows][128 B]
constexpr uint32_t GF_OFF_BT = 32768;      // 32 KB  B rows of the s-block
constexpr uint32_t GF_OFF_R = 65536;       // 2 x (dy rows of the t-block 16 KB | x rows of the s-block 16 KB)
constexpr uint32_t GF_OFF_W = 131072;      // 32 KB  head sum of the masked tiles [s-half][128 t rows][128 B]; until then: states of odd heads
constexpr uint32_t GF_OFF_SC = 163840;     // 16 KB  scaled rows of an inter-chunk term
constexpr uint32_t GF_OFF_ST = 180224;     // 2 x 16 KB  bf16 chunk states (entering: H, gradient leaving: G) of even heads
constexpr uint32_t GF_OFF_VEC = 212992;    // per-head vectors, double buffered
constexpr uint32_t GF_VEC_FLOATS = 256 * 3 + 64;
constexpr uint32_t GF_OFF_PART = GF_OFF_VEC + 2 * GF_VEC_FLOATS * 4;   // [head parity][rho: 4 slices x 128 rows | psi: 4 quarters x 128 cols]
constexpr uint32_t GF_SMEM = GF_OFF_PART + 2 * 1024 * 4 + 1024;

constexpr uint32_t TF_CB = 0, TF_S = 128, TF_ACCC = 256, TF_ACCB = 384;

constexpr float kLog2eF = 1.4426950408889634f;

__device__ __forceinline__ float ex2g(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2g(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ float2 unpack2g(uint32_t w) {
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w));
}

}  // namespace

__global__ void __launch_bounds__(GF_THREADS, 1)
k_grad_bc_fused(SegParams p, const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmDy,
                const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmC,
                const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmG) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar_ld, bar_cb, rfull[2], rempty[2], sfull, sempty, wfull, scfull, scempty, hfull[2], hempty[2],
        gfull[2], gempty[2], stdone, accfull, vfull[2], vempty[2], pfull[2], pempty[2];
    __shared__ uint32_t tmem_base, abort_flag;

    // 1-D grid: all full tiles first (they have the most mask work), then the two diagonal kinds
    const int nc = p.nc, nsl = p.nsl, ny = nsl * p.G;
    const int third = (int)(gridDim.x / 3), jid = (int)blockIdx.x % third;
    const int kind = (int)blockIdx.x / third;           // 0: tile (1,0)  1: tile (0,0)  2: tile (1,1)
    const int tb = (kind == 1) ? 0 : 1, sb = (kind == 2) ? 1 : 0;
    const bool diag = (tb == sb);
    const bool doC = (kind != 0);                       // adds dC's inter-chunk term of its t-block
    const bool doB = (kind != 1);                       // adds dB's inter-chunk term of its s-block
    const int c = jid % nc, yid = (jid / nc) % ny, b = jid / (nc * ny);
    const int g = yid / nsl, sl = yid % nsl;
    const int hps = (p.hpg + nsl - 1) / nsl;
    const int h_begin = g * p.hpg + sl * hps;
    const int h_end = min(g * p.hpg + p.hpg, h_begin + hps);
    const int nheads = max(h_end - h_begin, 0);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tok0 = p.t0 + c * 256;

    if (tid == 0) {
        mbar_init(&bar_ld, 1);
        mbar_init(&bar_cb, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&rfull[i], 1);
            mbar_init(&rempty[i], 1 + 16);    // the head's MMAs (one commit) + the mask warps that scaled its rows
            mbar_init(&vfull[i], 1);
            mbar_init(&vempty[i], 16);
            mbar_init(&pfull[i], 16);         // the mask warps' partial sums of rho / psi of a head
            mbar_init(&pempty[i], 1);
            mbar_init(&hfull[i], 1);
            mbar_init(&hempty[i], 1);
            mbar_init(&gfull[i], 1);
            mbar_init(&gempty[i], 1);
        }
        mbar_init(&sfull, 1);
        mbar_init(&sempty, 16);
        mbar_init(&wfull, 16);
        mbar_init(&scfull, 16);
        mbar_init(&scempty, 1);
        mbar_init(&stdone, 1);
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
            mbar_arrive_expect_tx(&bar_ld, 65536u);
            for (int nh = 0; nh < 2; ++nh) {
                tma_load_3d(smem + GF_OFF_CT + nh * 16384, &tmC, &bar_ld, g * 128 + nh * 64, tok0 + tb * 128, b);
                tma_load_3d(smem + GF_OFF_BT + nh * 16384, &tmB, &bar_ld, g * 128 + nh * 64, tok0 + sb * 128, b);
            }
            const int rowH = (b * (p.ncs + 1) + c) * p.H, rowG = (b * (p.ncs + 1) + c + 1) * p.H;
            for (int hi = 0; hi < nheads; ++hi) {
                const int h = h_begin + hi, rbuf = hi & 1;
                if (hi >= 2) mbar_wait(&rempty[rbuf], ((hi >> 1) - 1) & 1, abortp, p.status);
                mbar_arrive_expect_tx(&rfull[rbuf], 32768);
                tma_load_3d(smem + GF_OFF_R + rbuf * 32768, &tmDy, &rfull[rbuf], h * 64, tok0 + tb * 128, b);
                tma_load_3d(smem + GF_OFF_R + rbuf * 32768 + 16384, &tmX, &rfull[rbuf], h * 64, tok0 + sb * 128, b);
                unsigned char *stb = smem + (rbuf ? GF_OFF_W : GF_OFF_ST);   // states of odd heads: the spare buffer
                if (doC) {
                    if (hi >= 2) mbar_wait(&hempty[rbuf], ((hi >> 1) - 1) & 1, abortp, p.status);
                    mbar_arrive_expect_tx(&hfull[rbuf], 16384);
                    tma_load_3d(stb, &tmH, &hfull[rbuf], 0, (rowH + h) * 64, 0);
                    tma_load_3d(stb + 8192, &tmH, &hfull[rbuf], 64, (rowH + h) * 64, 0);
                }
                if (doB) {
                    if (hi >= 2) mbar_wait(&gempty[rbuf], ((hi >> 1) - 1) & 1, abortp, p.status);
                    mbar_arrive_expect_tx(&gfull[rbuf], 16384);
                    tma_load_3d(stb + 16384, &tmG, &gfull[rbuf], 0, (rowG + h) * 64, 0);
                    tma_load_3d(stb + 16384 + 8192, &tmG, &gfull[rbuf], 64, (rowG + h) * 64, 0);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && nheads > 0) {
            const uint32_t idKK = umma_idesc_bf16(128, 128, false, false);   // CB and the scores: both operands K-major
            const uint32_t idKM = umma_idesc_bf16(128, 128, false, true);    // W (K-major) x B rows (MN-major); scaled rows x state
            const uint32_t idMM = umma_idesc_bf16(128, 128, true, true);     // W^T (MN-major) x C rows (MN-major)
            // descriptors as (low word, high word): every offset below is a compile-time constant in 16-byte units
            const uint64_t dCk = umma_desc_sw128(smem_u32(smem + GF_OFF_CT), 16, 1024), dBk = umma_desc_sw128(smem_u32(smem + GF_OFF_BT), 16, 1024);
            const uint64_t dCm = umma_desc_sw128(smem_u32(smem + GF_OFF_CT), 16384, 1024), dBm = umma_desc_sw128(smem_u32(smem + GF_OFF_BT), 16384, 1024);
            const uint64_t dRk = umma_desc_sw128(smem_u32(smem + GF_OFF_R), 16, 1024);
            const uint64_t dWk = umma_desc_sw128(smem_u32(smem + GF_OFF_W), 16, 1024), dWm = umma_desc_sw128(smem_u32(smem + GF_OFF_W), 16384, 1024);
            const uint64_t dSk = umma_desc_sw128(smem_u32(smem + GF_OFF_SC), 16, 1024);
            const uint64_t dSt = umma_desc_sw128(smem_u32(smem + GF_OFF_ST), 8192, 1024);
            const uint64_t dSt1 = umma_desc_sw128(smem_u32(smem + GF_OFF_W), 8192, 1024);    // states of odd heads
            const uint32_t loCk = (uint32_t)dCk, hiK = (uint32_t)(dCk >> 32), loBk = (uint32_t)dBk;
            const uint32_t loCm = (uint32_t)dCm, hiM = (uint32_t)(dCm >> 32), loBm = (uint32_t)dBm;
            const uint32_t loRk = (uint32_t)dRk, loWk = (uint32_t)dWk, loWm = (uint32_t)dWm, loSk = (uint32_t)dSk;
            const uint32_t loSt0 = (uint32_t)dSt, loSt1 = (uint32_t)dSt1, hiSt = (uint32_t)(dSt >> 32);

            // CB tile, once
            mbar_wait(&bar_ld, 0, abortp, p.status);
            tc_fence_after_sync();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t o = (kk >> 2) * 1024 + (kk & 3) * 2;
                if (kk == 0) umma_bf16_fixed<false>(tm + TF_CB, umma_desc_words(loCk + o, hiK), umma_desc_words(loBk + o, hiK), idKK);
                else umma_bf16_fixed<true>(tm + TF_CB, umma_desc_words(loCk + o, hiK), umma_desc_words(loBk + o, hiK), idKK);
            }
            umma_commit(&bar_cb);

            // scores of head hi: dy rows (t-block) x x rows (s-block)^T, K = P
            auto issue_scores = [&](int hi) {
                const int rbuf = hi & 1;
                mbar_wait(&rfull[rbuf], (hi >> 1) & 1, abortp, p.status);
                tc_fence_after_sync();
                const uint32_t lo_a = loRk + rbuf * 2048, lo_b = lo_a + 1024;
                umma_bf16_fixed<false>(tm + TF_S, umma_desc_words(lo_a, hiK), umma_desc_words(lo_b, hiK), idKK);
#pragma unroll
                for (int k = 1; k < 4; ++k)
                    umma_bf16_fixed<true>(tm + TF_S, umma_desc_words(lo_a + k * 2, hiK), umma_desc_words(lo_b + k * 2, hiK), idKK);
                umma_commit(&sfull);
            };

            issue_scores(0);
            uint32_t scuse = 0;   // uses of the scaled-rows buffer so far
            for (int hi = 0; hi < nheads; ++hi) {
                // inter-chunk terms: scaled rows (K = p) times a chunk state.  A tile's first one is published by the
                // mask warps before they mask the head, so it is issued first: the scaled-rows buffer is free again
                // by the time tile (1,1) wants it for its second one.
                const uint32_t loSt = (hi & 1) ? loSt1 : loSt0;
                auto inter_dC = [&]() {   // dC += (e^{cs_t} dy_t) H_in
                    mbar_wait(&hfull[hi & 1], (hi >> 1) & 1, abortp, p.status);
                    mbar_wait(&scfull, scuse & 1, abortp, p.status);
                    ++scuse;
                    tc_fence_after_sync();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t ad = umma_desc_words(loSk + k * 2, hiK), bd = umma_desc_words(loSt + k * 128, hiSt);
                        if (k == 0 && hi == 0) umma_bf16_fixed<false>(tm + TF_ACCC, ad, bd, idKM);
                        else umma_bf16_fixed<true>(tm + TF_ACCC, ad, bd, idKM);
                    }
                    umma_commit(&scempty);
                    umma_commit(&hempty[hi & 1]);
                };
                auto inter_dB = [&](bool first_into_acc) {   // dB += (dt_s e^{cs_last-cs_s} x_s) Gout
                    mbar_wait(&gfull[hi & 1], (hi >> 1) & 1, abortp, p.status);
                    mbar_wait(&scfull, scuse & 1, abortp, p.status);
                    ++scuse;
                    tc_fence_after_sync();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t ad = umma_desc_words(loSk + k * 2, hiK), bd = umma_desc_words(loSt + 1024 + k * 128, hiSt);
                        if (k == 0 && first_into_acc) umma_bf16_fixed<false>(tm + TF_ACCB, ad, bd, idKM);
                        else umma_bf16_fixed<true>(tm + TF_ACCB, ad, bd, idKM);
                    }
                    umma_commit(&scempty);
                    umma_commit(&gempty[hi & 1]);
                };
                if (doC) inter_dC();
                else inter_dB(hi == 0);
                // next head's scores as soon as the mask warps are done with this head's (they read them last)
                if (hi + 1 < nheads) {
                    mbar_wait(&sempty, hi & 1, abortp, p.status);
                    tc_fence_after_sync();
                    issue_scores(hi + 1);
                }
                if (doC && doB) inter_dB(hi == 0);
                umma_commit(&rempty[hi & 1]);
            }
            umma_commit(&stdone);     // every product that read a chunk state is done: the spare buffer may take the head sum
            // the head sum of the masked tiles (made in fp32 by the mask warps, rounded once): both products
            mbar_wait(&wfull, 0, abortp, p.status);
            tc_fence_after_sync();
#pragma unroll
            for (int k = 0; k < 8; ++k) {   // dC += Wsum B : K = s
                const uint64_t ad = umma_desc_words(loWk + (k >> 2) * 1024 + (k & 3) * 2, hiK);
                const uint64_t bd = umma_desc_words(loBm + k * 128, hiM);
                if (k == 0 && !doC) umma_bf16_fixed<false>(tm + TF_ACCC, ad, bd, idKM);
                else umma_bf16_fixed<true>(tm + TF_ACCC, ad, bd, idKM);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {   // dB += Wsum^T C : K = t
                const uint64_t ad = umma_desc_words(loWm + k * 128, hiM);
                const uint64_t bd = umma_desc_words(loCm + k * 128, hiM);
                if (k == 0 && !doB) umma_bf16_fixed<false>(tm + TF_ACCB, ad, bd, idMM);
                else umma_bf16_fixed<true>(tm + TF_ACCB, ad, bd, idMM);
            }
            umma_commit(&accfull);
        }
    } else if (warp == 18) {
        // ------------------------------------------------------------ vector warp
        // Per head: the 256 cumulative sums (log2 units) and step sizes of the chunk, the column factor
        // e^{cs[s|31] - cs[s]} dt_s of the mask factorisation and the 8 x 8 table of sub-tile-to-sub-tile
        // decays, written to a double-buffered area one head ahead of the mask warps.
        if (nheads > 0) {
            float *vec = reinterpret_cast<float *>(smem + GF_OFF_VEC);
            // rho / psi of a finished head: the mask warps' partial sums added in a fixed order.  Rows of t-block 1
            // (columns of s-block 0) are covered by two tiles: the second part goes to rhob (psib), and the tile
            // that has no partner writes a zero there.
            auto finish_head = [&](int hj) {
                const int par = hj & 1;
                const float *pr = reinterpret_cast<const float *>(smem + GF_OFF_PART) + par * 1024;
                mbar_wait(&pfull[par], (hj >> 1) & 1, abortp, p.status);
                const size_t vb = (((size_t)b * p.H + h_begin + hj) * p.ncs + c) << 8;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int i = k * 32 + lane;
                    const float er = ((pr[i] + pr[128 + i]) + pr[256 + i]) + pr[384 + i];
                    const float ep = ((pr[512 + i] + pr[640 + i]) + pr[768 + i]) + pr[896 + i];
                    const size_t ro = vb + tb * 128 + i, so = vb + sb * 128 + i;
                    if (kind == 2) p.rhob[ro] = er;
                    else p.rho[ro] = er;
                    if (kind == 1) p.rhob[ro] = 0.f;
                    if (kind == 0) p.psib[so] = ep;
                    else p.psi[so] = ep;
                    if (kind == 2) p.psib[so] = 0.f;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&pempty[par]);
            };
            for (int hi = 0; hi < nheads; ++hi) {
                const int buf = hi & 1, h = h_begin + hi;
                const size_t vo = ((((size_t)b * p.H + h) * p.ncs + c) << 8) + lane * 8;
                const float4 c0 = __ldg(reinterpret_cast<const float4 *>(p.cs + vo));
                const float4 c1 = __ldg(reinterpret_cast<const float4 *>(p.cs + vo + 4));
                const float4 d0 = __ldg(reinterpret_cast<const float4 *>(p.dtT + vo));
                const float4 d1 = __ldg(reinterpret_cast<const float4 *>(p.dtT + vo + 4));
                if (hi >= 2) mbar_wait(&vempty[buf], ((hi >> 1) - 1) & 1, abortp, p.status);
                float *cs2 = vec + buf * GF_VEC_FLOATS, *cf = cs2 + 256, *dtv = cs2 + 512, *blk = cs2 + 768;
                const float cv[8] = {c0.x * kLog2eF, c0.y * kLog2eF, c0.z * kLog2eF, c0.w * kLog2eF,
                                     c1.x * kLog2eF, c1.y * kLog2eF, c1.z * kLog2eF, c1.w * kLog2eF};
                const float dv[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
                *reinterpret_cast<float4 *>(cs2 + lane * 8) = make_float4(cv[0], cv[1], cv[2], cv[3]);
                *reinterpret_cast<float4 *>(cs2 + lane * 8 + 4) = make_float4(cv[4], cv[5], cv[6], cv[7]);
                *reinterpret_cast<float4 *>(dtv + lane * 8) = d0;
                *reinterpret_cast<float4 *>(dtv + lane * 8 + 4) = d1;
                __syncwarp();
                const float ref = cs2[(lane * 8) | 31];
                float o[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) o[k] = ex2g(ref - cv[k]) * dv[k];
                *reinterpret_cast<float4 *>(cf + lane * 8) = make_float4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<float4 *>(cf + lane * 8 + 4) = make_float4(o[4], o[5], o[6], o[7]);
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    const int idx = lane + 32 * w, i = idx >> 3, j = idx & 7;   // blk[i][j] = e^{cs[32 i] - cs[32 j + 31]}, j < i
                    blk[idx] = (j < i) ? ex2g(cs2[32 * i] - cs2[32 * j + 31]) : 0.f;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&vfull[buf]);
                if (hi >= 1) finish_head(hi - 1);
            }
            finish_head(nheads - 1);
        }
    } else if (nheads > 0) {
        // ------------------------------------------------------------ mask warps
        // Four warps per TMEM lane quarter: warp (q, quar) owns rows 32 q .. 32 q + 31 of the t-block and the
        // 16-column slice `quar` of both 64-column halves of the tile.
        const int q = warp & 3;
        const int quar = (warp - 2) >> 2;
        const int rl = q * 32 + lane;              // row inside the 128-row block (t for W and dC, s for dB)
        const int r = tb * 128 + rl;               // t inside the chunk
        const int rs = sb * 128 + rl;              // s inside the chunk, for the rows this thread scales for dB
        const int isub = r >> 5;
        const uint32_t tlane = (uint32_t)(q * 32) << 16;
        float *vec = reinterpret_cast<float *>(smem + GF_OFF_VEC);
        uint32_t scuse = 0;
        float wsum[32];                             // this thread's row of sum_h W_h: columns w * 16 + j of its two slices
#pragma unroll
        for (int k = 0; k < 32; ++k) wsum[k] = 0.f;

        for (int hi = 0; hi < nheads; ++hi) {
            float *cs2 = vec + (hi & 1) * GF_VEC_FLOATS, *cf = cs2 + 256, *dtv = cs2 + 512, *blk = cs2 + 768;
            mbar_wait(&vfull[hi & 1], (hi >> 1) & 1, abortp, p.status);
            const float csr = cs2[r];
            const float rowf = ex2g(csr - cs2[r & ~31]);                 // e^{cs_t - cs[first row of t's sub-tile]}
            const float offsC = ex2g(csr);                                // dC's inter-chunk row scale
            const float offsB = dtv[rs] * ex2g(cs2[255] - cs2[rs]);       // dB's inter-chunk row scale
            if (hi == 0) {
                mbar_wait(&bar_cb, 0, abortp, p.status);
                tc_fence_after_sync();
            }

            // ---- inter-chunk terms: the head's rows scaled per row, as one more K = P operand (dy rows of the
            // t-block by e^{cs_t} for dC, x rows of the s-block by dt_s e^{cs_last-cs_s} for dB).  A tile's first one
            // is published before the masking below, so that its MMAs run while W is being made.
            auto scale_rows = [&](int which) {
                const unsigned char *rrow = smem + GF_OFF_R + (hi & 1) * 32768 + which * 16384 + rl * 128;
                unsigned char *srow = smem + GF_OFF_SC + rl * 128;
                const float sc = which == 0 ? offsC : offsB;
                uint4 o[2];
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const uint4 qv = *reinterpret_cast<const uint4 *>(rrow + (((quar * 2 + k) ^ (rl & 7)) << 4));
                    const uint32_t *qw = reinterpret_cast<const uint32_t *>(&qv);
                    uint32_t *ow = reinterpret_cast<uint32_t *>(&o[k]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = unpack2g(qw[e]);
                        ow[e] = pack2g(f.x * sc, f.y * sc);
                    }
                }
                if (scuse >= 1) mbar_wait(&scempty, (scuse - 1) & 1, abortp, p.status);
                ++scuse;
#pragma unroll
                for (int k = 0; k < 2; ++k)
                    *reinterpret_cast<uint4 *>(srow + (((quar * 2 + k) ^ (rl & 7)) << 4)) = o[k];
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&scfull);
            };
            mbar_wait(&rfull[hi & 1], (hi >> 1) & 1, abortp, p.status);
            scale_rows(doC ? 0 : 1);

            // ---- W = score o mask (fp32) for this thread's two 16-column slices, one after the other: added to
            // the head sum; Z = W o CB gives the row sum (rho) and, through a transposing butterfly over the
            // warp's 32 rows, the column sums (psi).  The score buffer is released after the second slice.
            float2 dacc = make_float2(0.f, 0.f);
            float csum = 0.f;                                // lanes 0..15: column j of slice 0, lanes 16..31: of slice 1
            mbar_wait(&sfull, hi & 1, abortp, p.status);
            tc_fence_after_sync();
#pragma unroll
            for (int w = 0; w < 2; ++w) {
                const int cb = sb * 128 + w * 64 + quar * 16;   // first column of the slice (s in chunk)
                const int jsub = cb >> 5;
                if (diag && (jsub > isub)) continue;            // above the diagonal: W = 0 (uniform over the warp)
                float vv[16], cbv[16];
                tmem_ld16_nowait(tm + tlane + TF_S + w * 64 + quar * 16, vv);
                tmem_ld16_nowait(tm + tlane + TF_CB + w * 64 + quar * 16, cbv);
                tmem_ld_wait16(vv);
                if (jsub != isub) {
                    const float s1 = rowf * blk[isub * 8 + jsub];
                    const float2 s1v = make_float2(s1, s1);
#pragma unroll
                    for (int k = 0; k < 16; k += 4) {
                        const float4 cv = *reinterpret_cast<const float4 *>(cf + cb + k);
                        const float2 w0 = __fmul2_rn(make_float2(vv[k], vv[k + 1]), __fmul2_rn(make_float2(cv.x, cv.y), s1v));
                        const float2 w1 = __fmul2_rn(make_float2(vv[k + 2], vv[k + 3]), __fmul2_rn(make_float2(cv.z, cv.w), s1v));
                        vv[k] = w0.x; vv[k + 1] = w0.y; vv[k + 2] = w1.x; vv[k + 3] = w1.y;
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 16; k += 4) {
                        const float4 cc = *reinterpret_cast<const float4 *>(cs2 + cb + k);
                        const float4 d4 = *reinterpret_cast<const float4 *>(dtv + cb + k);
                        const float ccv[4] = {cc.x, cc.y, cc.z, cc.w};
                        const float dv[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const bool on = (cb + k + e) <= r;
                            const float ex = ex2g(csr - ccv[e]) * dv[e];
                            vv[k + e] = on ? vv[k + e] * ex : 0.f;
                        }
                    }
                }
                tmem_ld_wait16(cbv);
#pragma unroll
                for (int k = 0; k < 16; k += 2) {
                    const float2 wv = make_float2(vv[k], vv[k + 1]);
                    const float2 a = __fadd2_rn(make_float2(wsum[w * 16 + k], wsum[w * 16 + k + 1]), wv);
                    wsum[w * 16 + k] = a.x;
                    wsum[w * 16 + k + 1] = a.y;
                    const float2 zz = __fmul2_rn(wv, make_float2(cbv[k], cbv[k + 1]));
                    vv[k] = zz.x;
                    vv[k + 1] = zz.y;
                    dacc = __fadd2_rn(dacc, zz);
                }
                // column sums of Z over the warp's rows: 16 values -> lane l ends with column l & 15
#pragma unroll
                for (int o = 8, cnt = 16; o >= 1; o >>= 1, cnt >>= 1) {
                    const bool up = (lane & o) != 0;
#pragma unroll
                    for (int i = 0; i < cnt / 2; ++i) {
                        const float send = up ? vv[i] : vv[i + cnt / 2];
                        const float keep = up ? vv[i + cnt / 2] : vv[i];
                        vv[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                    }
                }
                const float tot = vv[0] + __shfl_xor_sync(0xffffffffu, vv[0], 16);
                if ((lane >> 4) == w) csum = tot;
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&sempty);
                mbar_arrive(&vempty[hi & 1]);
            }
            if (doC && doB) scale_rows(1);     // tile (1,1): its second inter-chunk term
            __syncwarp();
            if (lane == 0) mbar_arrive(&rempty[hi & 1]);     // this warp has read the head's rows

            // ---- rho_t / psi_s: every warp leaves its partial sums (over its 16-column slice / its 32 rows) in
            // shared memory; the vector warp adds them in a fixed order and writes them out, so no mask warp waits
            // for another one here
            {
                const int par = hi & 1;
                float *pr = reinterpret_cast<float *>(smem + GF_OFF_PART) + par * 1024;
                if (hi >= 2) mbar_wait(&pempty[par], ((hi >> 1) - 1) & 1, abortp, p.status);
                pr[quar * 128 + rl] = dacc.x + dacc.y;
                const int lc = (lane >> 4) * 64 + quar * 16 + (lane & 15);     // column of the tile this lane holds
                pr[512 + q * 128 + lc] = csum;
                __syncwarp();
                if (lane == 0) mbar_arrive(&pfull[par]);
            }
        }

        // ---- the head sum of W, rounded once to bf16: [s-half w][row][128 B], this thread's 16 columns of a
        // half = chunks quar * 2, quar * 2 + 1.  The buffer held chunk states until the last head's products ended.
        mbar_wait(&stdone, 0, abortp, p.status);
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            unsigned char *mrow = smem + GF_OFF_W + w * 16384 + rl * 128;
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
                const float *a = wsum + w * 16 + ch * 8;
                *reinterpret_cast<uint4 *>(mrow + (((quar * 2 + ch) ^ (rl & 7)) << 4)) =
                    make_uint4(pack2g(a[0], a[1]), pack2g(a[2], a[3]), pack2g(a[4], a[5]), pack2g(a[6], a[7]));
            }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&wfull);

        // ---- the CTA's partial slices of the group sums: [B, seg, G, 2 nsl, N] fp32.  Every row of an accumulator is
        // 512 contiguous bytes of its slice.  Row-per-thread global stores would touch 32 different lines per
        // instruction, so the two accumulators are staged in shared memory (every operand buffer is dead once the last
        // products are done), rows padded to 528 bytes (conflict-free row-per-thread writes), and each row leaves as
        // one bulk copy.
        mbar_wait(&accfull, 0, abortp, p.status);
        tc_fence_after_sync();
        {
            float *stgC = reinterpret_cast<float *>(smem), *stgB = reinterpret_cast<float *>(smem + 128 * 528);
            float a[32];
            tmem_ld32(tm + tlane + TF_ACCC + quar * 32, a);
#pragma unroll
            for (int k = 0; k < 32; k += 4)
                *reinterpret_cast<float4 *>(stgC + rl * 132 + quar * 32 + k) = make_float4(a[k], a[k + 1], a[k + 2], a[k + 3]);
            tmem_ld32(tm + tlane + TF_ACCB + quar * 32, a);
#pragma unroll
            for (int k = 0; k < 32; k += 4)
                *reinterpret_cast<float4 *>(stgB + rl * 132 + quar * 32 + k) = make_float4(a[k], a[k + 1], a[k + 2], a[k + 3]);
            fence_proxy_async_smem();
            asm volatile("bar.sync 1, 512;" ::: "memory");        // the sixteen mask warps
            const int m = tid - 64;                               // 0..511 over the mask warps
            if (m < 256) {
                const size_t segcap = (size_t)p.ncs * 256;
                const int nsl2 = 2 * nsl, row = m & 127;
                if (m < 128) {
                    // dC rows t: tiles (1,0) and (0,0) fill the even slot of their rows, (1,1) the odd slot of t-block 1
                    const size_t tl = (size_t)c * 256 + tb * 128 + row;
                    const int slot = sl * 2 + (kind == 2 ? 1 : 0);
                    bulk_store(p.pC + ((((size_t)b * segcap + tl) * p.G + g) * nsl2 + slot) * 128, stgC + row * 132, 512);
                } else {
                    // dB rows s: tiles (0,0) and (1,1) fill the even slot of their rows, (1,0) the odd slot of s-block 0
                    const size_t tl = (size_t)c * 256 + sb * 128 + row;
                    const int slot = sl * 2 + (kind == 0 ? 1 : 0);
                    bulk_store(p.pB + ((((size_t)b * segcap + tl) * p.G + g) * nsl2 + slot) * 128, stgB + row * 132, 512);
                }
                tma_store_commit();
                tma_store_wait_all();
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tm, 512);
    }
}

cudaError_t launch_grad_bc_fused(const SegParams &p, const TcMaps &m, cudaStream_t st) {
    dim3 grid(3 * p.nc * p.nsl * p.G * p.B);
    cudaError_t e = cudaFuncSetAttribute(k_grad_bc_fused, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GF_SMEM);
    if (e != cudaSuccess) return e;
    return launch_pdl(k_grad_bc_fused, grid, dim3(GF_THREADS), (size_t)GF_SMEM, st, p, m.x, m.dy, m.Bm, m.Cm, m.Hbf, m.Gbf);
}

}  // namespace ssd
