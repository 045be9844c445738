// Tensor-core kernel for the two masked products whose score matrix is shared by the heads of a
// group (bf16 I/O, P = 64, N = 128, Q = 256):
//
//   SC_FWD: y_t  = sum_{s<=t} (C_t.B_s) e^{cs_t-cs_s} dt_s x_s + e^{cs_t} C_t H_in + D x_t
//   SC_DX : u_s  = sum_{t>=s} (B_s.C_t) e^{cs_t-cs_s} dy_t      + e^{cs_last-cs_s} B_s Gout
//                   dx_s = D dy_s + dt_s u_s ;  ddt_direct_s = x_s . u_s ;  dD partial = sum dy.x ;
//                   psi2_s = dt_s e^{cs_last-cs_s} x_s . (Gout B_s)   (inter-chunk part of B_s . dB_s)
//
// (Eq. 1 of the paper regrouped by chunks; cs = inclusive cumsum of dt*A inside the chunk.)
//
// One CTA owns (chunk, 128-row block, group, a range of the group's heads).  The score tile
// S = Rows * Cols^T (128 x up to 256, K = N) is computed ONCE with tcgen05.mma into TMEM and stays
// there in fp32 for every head of the range.  Per head the CTA runs five roles that meet only
// through mbarriers:
//   producer warp   : TMA loads of the head's value rows (x or dy; three stages, so a load is issued
//                     two heads before it is needed: a 32 KB tile takes about 3000 cycles to land)
//                     and of its bf16 chunk state (two buffers)
//   MMA warp        : acc2 = Rows * State^T (K = N); acc1 += M_piece * V per 64-column piece
//   vector warp     : the head's cumulative sums, step sizes and mask factors, one head ahead
//   8 mask warps    : read S from TMEM, apply the decay mask, round to bf16 and store the piece of M
//                     to a two-slot ring in shared memory (A operand of the next MMAs)
//   4 epilogue warps: the previous head's accumulators (double-buffered in TMEM) -> y or dx; x and dy
//                     come from the value tile already in shared memory, the output overwrites it in
//                     place and leaves by one TMA store per warp, which then releases the stage.
// The decay mask is factored per 32 x 32 sub-tile: strictly off-diagonal sub-tiles use
//   e^{cs_t-cs_s} = e^{cs_t-cs_i0} * e^{cs_i0-cs_j1} * e^{cs_j1-cs_s}      (i0 = first row of the row
// sub-tile, j1 = last column of the column sub-tile), three factors that are each <= 1 because cs
// is non-increasing, so only O(Q) exponentials are needed per head instead of O(Q^2); diagonal
// sub-tiles are exponentiated element by element.
#include <type_traits>

#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

using namespace sm100;

namespace {

// warp 0 producer, 1 MMA, 2..17 mask, 18 vectors, 19.. epilogue: one warp per TMEM lane quarter for y, two for dx,
// whose epilogue (three row sums besides the output) set the pace of the kernel with one
__host__ __device__ constexpr int sc_epilogue_warps(int mode) { return mode == SC_FWD ? 4 : 8; }
__host__ __device__ constexpr int sc_threads(int mode) { return (19 + sc_epilogue_warps(mode)) * 32; }
constexpr uint32_t OFF_ROWS = 0;          // 32 KB  [n-half][128 rows][128 B]
constexpr uint32_t OFF_X = 32768;         // 3 x 32 KB value stages; first the score-columns operand (<= 64 KB)
constexpr uint32_t OFF_M = 131072;        // 2 x 16 KB ring of masked pieces
constexpr uint32_t OFF_ST = 163840;       // 2 x 16 KB  bf16 chunk state [n-half][64 rows][128 B]
constexpr uint32_t OFF_XR = 196608;       // 16 KB  SC_DX: the head's x rows of this row block
constexpr uint32_t OFF_VEC = 212992;      // per-head vectors, double buffered
constexpr uint32_t VEC_FLOATS = 256 * 3 + 64;
constexpr uint32_t SC_SMEM = OFF_VEC + 2 * VEC_FLOATS * 4 + 1024;
constexpr int PF_AHEAD = 3;               // L2 prefetch distance of the producer, in heads

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
__device__ __forceinline__ void unpack8(const uint4 &q, float *f) {
    const __nv_bfloat162 *e = reinterpret_cast<const __nv_bfloat162 *>(&q);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float2 t = __bfloat1622float2(e[k]);
        f[2 * k] = t.x;
        f[2 * k + 1] = t.y;
    }
}

__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

}  // namespace

template <int MODE>
__global__ void __launch_bounds__(sc_threads(MODE), 1)
k_scan_tc(SegParams p, int nsplit, const __grid_constant__ CUtensorMap tmRow,
          const __grid_constant__ CUtensorMap tmCol, const __grid_constant__ CUtensorMap tmV,
          const __grid_constant__ CUtensorMap tmSt, const __grid_constant__ CUtensorMap tmOut,
          const __grid_constant__ CUtensorMap tmXr) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar_ab, bar_s, xfull[3], xempty[3], hfull[2], hempty[2], xrfull, xrempty, mfull[2], mempty[2],
        accfull[2], accempty[2], vfull[2], vempty[2];
    __shared__ uint32_t tmem_base, abort_flag;
    __shared__ float epx[2][128][2], epd[2][4];    // SC_DX: row sums handed from one epilogue warp of a pair to the other

    constexpr bool FWD = (MODE == SC_FWD);
    constexpr int EPW = sc_epilogue_warps(MODE), NPP = 16 / EPW;   // epilogue warps; 16-column passes per warp
    // 1-D grid; the first half are the long CTAs (the row block with the larger column range), so the
    // tail of the launch is filled with short ones
    const int nc = p.nc, ny = nsplit * p.G;
    const int half_grid = (int)(gridDim.x >> 1), jid = (int)blockIdx.x % half_grid;
    const bool is_long = (int)blockIdx.x < half_grid;
    const int rb = FWD ? (is_long ? 1 : 0) : (is_long ? 0 : 1);
    const int c = jid % nc, yid = (jid / nc) % ny, b = jid / (nc * ny);
    const int g = yid / nsplit, sp = yid % nsplit;
    const int hps = (p.hpg + nsplit - 1) / nsplit;
    const int h_begin = g * p.hpg + sp * hps;
    const int h_end = min(g * p.hpg + p.hpg, h_begin + hps);
    if (h_begin >= h_end) return;
    const int nheads = h_end - h_begin;
    const int colbase = FWD ? 0 : rb * 128;
    const int ncols = FWD ? (rb + 1) * 128 : 256 - rb * 128;
    const int npieces = ncols >> 6;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tok0 = p.t0 + c * 256;
    const int slot = FWD ? c : c + 1;

    if (tid == 0) {
        mbar_init(&bar_ab, 1);
        mbar_init(&bar_s, 1);
        for (int i = 0; i < 3; ++i) {
            mbar_init(&xfull[i], 1);
            mbar_init(&xempty[i], 1 + 4);     // the MMAs (one commit) and the four output stores staged in it
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&hfull[i], 1);
            mbar_init(&hempty[i], 1);
            mbar_init(&mfull[i], 8);           // one arrival per warp (lane 0, after __syncwarp()) of the slot's eight
            mbar_init(&mempty[i], 1);
            mbar_init(&accfull[i], 1);
            mbar_init(&accempty[i], EPW);
            mbar_init(&vfull[i], 1);
            mbar_init(&vempty[i], 16 + EPW);
        }
        mbar_init(&xrfull, 1);
        mbar_init(&xrempty, EPW);
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
    // TMEM columns: S [0,256) ; acc1[b] at 256 + 128 b ; acc2[b] at 320 + 128 b
    volatile uint32_t *abortp = &abort_flag;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            mbar_arrive_expect_tx(&bar_ab, 32768u + (uint32_t)ncols * 256u);
            tma_load_3d(smem + OFF_ROWS, &tmRow, &bar_ab, g * 128, tok0 + rb * 128, b);
            tma_load_3d(smem + OFF_ROWS + 16384, &tmRow, &bar_ab, g * 128 + 64, tok0 + rb * 128, b);
            for (int nh = 0; nh < 2; ++nh)
                for (int r0 = 0; r0 < ncols; r0 += 128)
                    tma_load_3d(smem + OFF_X + nh * ncols * 128 + r0 * 128, &tmCol, &bar_ab, g * 128 + nh * 64,
                                tok0 + colbase + r0, b);
            const int strow = (b * (p.ncs + 1) + slot) * p.H;
            for (int hi = 0; hi < nheads; ++hi) {
                const int buf = hi & 1, xs = hi % 3, xuse = hi / 3, h = h_begin + hi;
                if (hi >= 2) mbar_wait(&hempty[buf], ((hi >> 1) - 1) & 1, abortp, p.status);
                mbar_arrive_expect_tx(&hfull[buf], 16384);
                tma_load_3d(smem + OFF_ST + buf * 16384, &tmSt, &hfull[buf], 0, (strow + h) * 64, 0);
                tma_load_3d(smem + OFF_ST + buf * 16384 + 8192, &tmSt, &hfull[buf], 64, (strow + h) * 64, 0);
                if (hi == 0) mbar_wait(&bar_s, 0, abortp, p.status);   // score MMAs done: the column operand is dead
                if (xuse >= 1) mbar_wait(&xempty[xs], (xuse - 1) & 1, abortp, p.status);
                mbar_arrive_expect_tx(&xfull[xs], (uint32_t)ncols * 128u);
                for (int r0 = 0; r0 < ncols; r0 += 128)
                    tma_load_3d(smem + OFF_X + xs * 32768 + r0 * 128, &tmV, &xfull[xs], h * 64, tok0 + colbase + r0, b);
                if (!FWD) {
                    if (hi >= 1) mbar_wait(&xrempty, (hi - 1) & 1, abortp, p.status);
                    mbar_arrive_expect_tx(&xrfull, 16384);
                    tma_load_3d(smem + OFF_XR, &tmXr, &xrfull, h * 64, tok0 + rb * 128, b);
                }
                // A value stage is held until the head's output has left it, so its next load can be issued only
                // about one head before it is needed.  Ask for the tiles of the head three ahead (and the state two
                // ahead) in L2 now; the later loads then take an L2 hit's time.
                if (hi + PF_AHEAD < nheads) {
                    const int hp = h + PF_AHEAD;
                    for (int r0 = 0; r0 < ncols; r0 += 128) tma_prefetch_3d(&tmV, hp * 64, tok0 + colbase + r0, b);
                    if (!FWD) tma_prefetch_3d(&tmXr, hp * 64, tok0 + rb * 128, b);
                }
                if (hi + PF_AHEAD - 1 < nheads) {
                    tma_prefetch_3d(&tmSt, 0, (strow + h + PF_AHEAD - 1) * 64, 0);
                    tma_prefetch_3d(&tmSt, 64, (strow + h + PF_AHEAD - 1) * 64, 0);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t sRows = smem_u32(smem + OFF_ROWS), sX = smem_u32(smem + OFF_X);
            const uint32_t sM = smem_u32(smem + OFF_M), sSt = smem_u32(smem + OFF_ST);
            const uint32_t idS = umma_idesc_bf16(128, (uint32_t)ncols, false, false);
            const uint32_t id3 = umma_idesc_bf16(128, 64, false, false);
            const uint32_t id2 = umma_idesc_bf16(128, 64, false, true);
            mbar_wait(&bar_ab, 0, abortp, p.status);
            tc_fence_after_sync();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint64_t ad = umma_desc_sw128(sRows + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024);
                const uint64_t bd = umma_desc_sw128(sX + (kk >> 2) * (ncols * 128) + (kk & 3) * 32, 16, 1024);
                umma_bf16(tm, ad, bd, idS, kk ? 1u : 0u);
            }
            umma_commit(&bar_s);
            // Descriptors of the loop-invariant operands as (low word, high word); every offset below is a
            // compile-time constant in 16-byte units once the loops are unrolled.
            const uint64_t dRows = umma_desc_sw128(sRows, 16, 1024), dSt = umma_desc_sw128(sSt, 16, 1024);
            const uint64_t dM = umma_desc_sw128(sM, 16, 1024), dX = umma_desc_sw128(sX, 8192, 1024);
            const uint32_t loR = (uint32_t)dRows, hiR = (uint32_t)(dRows >> 32), loS = (uint32_t)dSt, hiS = (uint32_t)(dSt >> 32);
            const uint32_t loM = (uint32_t)dM, hiM = (uint32_t)(dM >> 32), loX = (uint32_t)dX, hiX = (uint32_t)(dX >> 32);
            auto run = [&](auto np_c) {
                constexpr int NP = decltype(np_c)::value;     // pieces per head: 2 or 4, so piece jj uses ring slot jj & 1
                int xs = 0, xuse = 0;
                for (int hi = 0; hi < nheads; ++hi) {
                    const int buf = hi & 1;
                    const uint32_t acc1 = tm + 256 + buf * 128, acc2 = acc1 + 64;
                    const uint32_t loSb = loS + buf * 1024, loXh = loX + xs * 2048;
                    const uint32_t par = (uint32_t)(hi >> 1) & 1u;
                    if (hi >= 2) mbar_wait(&accempty[buf], par ^ 1u, abortp, p.status);
                    mbar_wait(&hfull[buf], par, abortp, p.status);
                    tc_fence_after_sync();
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t oa = (kk >> 2) * 1024 + (kk & 3) * 2, ob = (kk >> 2) * 512 + (kk & 3) * 2;
                        if (kk == 0) umma_bf16_fixed<false>(acc2, umma_desc_words(loR + oa, hiR), umma_desc_words(loSb + ob, hiS), id3);
                        else umma_bf16_fixed<true>(acc2, umma_desc_words(loR + oa, hiR), umma_desc_words(loSb + ob, hiS), id3);
                    }
                    umma_commit(&hempty[buf]);
                    mbar_wait(&xfull[xs], (uint32_t)xuse & 1u, abortp, p.status);
                    const uint32_t pbase = (uint32_t)(hi * (NP / 2)) & 1u;      // parity of ring use (hi NP + jj) >> 1
#pragma unroll
                    for (int jj = 0; jj < NP; ++jj) {
                        const int ms = jj & 1;
                        mbar_wait(&mfull[ms], pbase ^ (uint32_t)((jj >> 1) & 1), abortp, p.status);
                        tc_fence_after_sync();
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const uint64_t ad = umma_desc_words(loM + ms * 1024 + k * 2, hiM);
                            const uint64_t bd = umma_desc_words(loXh + jj * 512 + k * 128, hiX);
                            if (jj == 0 && k == 0) umma_bf16_fixed<false>(acc1, ad, bd, id2);
                            else umma_bf16_fixed<true>(acc1, ad, bd, id2);
                        }
                        umma_commit(&mempty[ms]);
                    }
                    umma_commit(&accfull[buf]);
                    umma_commit(&xempty[xs]);
                    if (++xs == 3) { xs = 0; ++xuse; }
                }
            };
            if (npieces == 4) run(std::integral_constant<int, 4>{});
            else run(std::integral_constant<int, 2>{});
        }
    } else if (warp == 18) {
        // ------------------------------------------------------------ vector warp
        // Per head: the 256 cumulative sums (log2 units) and step sizes of the chunk, the column factor
        // of the mask factorisation and the 8 x 8 table of sub-tile-to-sub-tile decays, written to a
        // double-buffered area one head ahead of their readers.  Each lane owns 8 consecutive steps.
        float *vec = reinterpret_cast<float *>(smem + OFF_VEC);
        for (int hi = 0; hi < nheads; ++hi) {
            const int buf = hi & 1, h = h_begin + hi;
            const size_t vo = ((((size_t)b * p.H + h) * p.ncs + c) << 8) + lane * 8;
            const float4 c0 = __ldg(reinterpret_cast<const float4 *>(p.cs + vo));
            const float4 c1 = __ldg(reinterpret_cast<const float4 *>(p.cs + vo + 4));
            const float4 d0 = __ldg(reinterpret_cast<const float4 *>(p.dtT + vo));
            const float4 d1 = __ldg(reinterpret_cast<const float4 *>(p.dtT + vo + 4));
            if (hi >= 2) mbar_wait(&vempty[buf], ((hi >> 1) - 1) & 1, abortp, p.status);
            float *cs2 = vec + buf * VEC_FLOATS, *cf = cs2 + 256, *dtv = cs2 + 512, *blk = cs2 + 768;
            const float cv[8] = {c0.x * kLog2e, c0.y * kLog2e, c0.z * kLog2e, c0.w * kLog2e,
                                 c1.x * kLog2e, c1.y * kLog2e, c1.z * kLog2e, c1.w * kLog2e};
            const float dv[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
            *reinterpret_cast<float4 *>(cs2 + lane * 8) = make_float4(cv[0], cv[1], cv[2], cv[3]);
            *reinterpret_cast<float4 *>(cs2 + lane * 8 + 4) = make_float4(cv[4], cv[5], cv[6], cv[7]);
            *reinterpret_cast<float4 *>(dtv + lane * 8) = d0;
            *reinterpret_cast<float4 *>(dtv + lane * 8 + 4) = d1;
            __syncwarp();
            const float ref = FWD ? cs2[(lane * 8) | 31] : cs2[(lane * 8) & ~31];
            float o[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) o[k] = FWD ? ex2f(ref - cv[k]) * dv[k] : ex2f(cv[k] - ref);
            *reinterpret_cast<float4 *>(cf + lane * 8) = make_float4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<float4 *>(cf + lane * 8 + 4) = make_float4(o[4], o[5], o[6], o[7]);
#pragma unroll
            for (int w = 0; w < 2; ++w) {
                const int idx = lane + 32 * w, i = idx >> 3, j = idx & 7;   // blk[i][j] = e^{cs[32 i] - cs[32 j + 31]}, j < i
                blk[idx] = (j < i) ? ex2f(cs2[32 * i] - cs2[32 * j + 31]) : 0.f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&vfull[buf]);
        }
    } else if (warp >= 2 && warp < 18) {
        // ------------------------------------------------------------ mask warps
        // Two warps per TMEM lane quarter: warp (q, half) owns rows 32 q .. 32 q + 31 of the block.
        const int q = warp & 3;
        const int half = (warp - 2) >> 3;          // which pieces (and ring slot) this warp's group takes
        const int sub = ((warp - 2) >> 2) & 1;     // which 32-column sub-tile of those pieces
        const int rl = q * 32 + lane;              // row inside the 128-row block
        const int r = rb * 128 + rl;               // row inside the chunk
        const int isub = r >> 5;
        const uint32_t tlane = (uint32_t)(q * 32) << 16;
        float *vec = reinterpret_cast<float *>(smem + OFF_VEC);

        // Four warps per lane quarter in two groups that alternate pieces: group `half` masks pieces half,
        // half + 2, ... (one 32-column sub-tile per warp) and always fills ring slot `half`, so the per-piece
        // hand-over costs (slot wait, stores, proxy fence, arrival) of one group overlap the other's arithmetic.
        uint32_t muse = 0;   // how often this warp has filled its ring slot
        for (int hi = 0; hi < nheads; ++hi) {
            float *cs2 = vec + (hi & 1) * VEC_FLOATS, *cf = cs2 + 256, *dtv = cs2 + 512, *blk = cs2 + 768;
            mbar_wait(&vfull[hi & 1], (hi >> 1) & 1, abortp, p.status);
            const float csr = cs2[r];
            const float rowf = FWD ? ex2f(csr - cs2[r & ~31]) : ex2f(cs2[r | 31] - csr);
            if (hi == 0) {
                mbar_wait(&bar_s, 0, abortp, p.status);
                tc_fence_after_sync();
            }
            for (int jj = half; jj < npieces; jj += 2) {
                uint32_t pks[16];
                {
                    const int cb = colbase + jj * 64 + sub * 32;    // first column of the sub-tile (in chunk)
                    const int jsub = cb >> 5;
                    const bool zero = FWD ? (jsub > isub) : (jsub < isub);
                    if (zero) {
#pragma unroll
                        for (int k = 0; k < 16; ++k) pks[k] = 0u;
                    } else {
                        float v[32];
                        tmem_ld32(tm + tlane + jj * 64 + sub * 32, v);
                        if (jsub != isub) {
                            const float f = rowf * (FWD ? blk[isub * 8 + jsub] : blk[jsub * 8 + isub]);
                            const float2 f2 = make_float2(f, f);
#pragma unroll
                            for (int k = 0; k < 32; k += 4) {
                                const float4 cv = *reinterpret_cast<const float4 *>(cf + cb + k);
                                const float2 w0 = __fmul2_rn(make_float2(v[k], v[k + 1]), __fmul2_rn(make_float2(cv.x, cv.y), f2));
                                const float2 w1 = __fmul2_rn(make_float2(v[k + 2], v[k + 3]), __fmul2_rn(make_float2(cv.z, cv.w), f2));
                                pks[k >> 1] = pack2(w0.x, w0.y);
                                pks[(k >> 1) + 1] = pack2(w1.x, w1.y);
                            }
                        } else {
#pragma unroll
                            for (int k = 0; k < 32; k += 4) {
                                const float4 cc = *reinterpret_cast<const float4 *>(cs2 + cb + k);
                                const float ccv[4] = {cc.x, cc.y, cc.z, cc.w};
                                float dv[4] = {1.f, 1.f, 1.f, 1.f};
                                if (FWD) {
                                    const float4 d4 = *reinterpret_cast<const float4 *>(dtv + cb + k);
                                    dv[0] = d4.x; dv[1] = d4.y; dv[2] = d4.z; dv[3] = d4.w;
                                }
                                float w[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int col = cb + k + e;
                                    const bool on = FWD ? (col <= r) : (col >= r);
                                    const float ex = FWD ? ex2f(csr - ccv[e]) * dv[e] : ex2f(ccv[e] - csr);
                                    w[e] = on ? v[k + e] * ex : 0.f;
                                }
                                pks[k >> 1] = pack2(w[0], w[1]);
                                pks[(k >> 1) + 1] = pack2(w[2], w[3]);
                            }
                        }
                    }
                }
                // the ring slot is free once the MMAs of the piece that last used it are done
                if (muse >= 1) mbar_wait(&mempty[half], (muse - 1) & 1, abortp, p.status);
                ++muse;
                unsigned char *mrow = smem + OFF_M + half * 16384 + rl * 128;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch)
                    *reinterpret_cast<uint4 *>(mrow + (((sub * 4 + ch) ^ (rl & 7)) << 4)) =
                        make_uint4(pks[4 * ch], pks[4 * ch + 1], pks[4 * ch + 2], pks[4 * ch + 3]);
                tc_fence_before_sync();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&mfull[half]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&vempty[hi & 1]);
        }
    } else if (warp >= 19) {
        // ------------------------------------------------------------ epilogue warps (one or two per TMEM lane quarter)
        // x (and dy) come from the tiles TMA already brought to shared memory; the output overwrites the
        // rows just read, in place (the MMAs of the head are done with the stage), and leaves by one TMA
        // store per lane quarter (32 rows x 64 columns), after which the stage is released.  With two warps per
        // quarter each takes 32 of the 64 output columns.
        const int q = warp & 3;
        const int ech = (warp - 19) >> 2;          // which 32 output columns
        const int rl = q * 32 + lane;              // row inside the 128-row block
        const int r = rb * 128 + rl;               // row inside the chunk
        const uint32_t tlane = (uint32_t)(q * 32) << 16;
        const float *vec = reinterpret_cast<const float *>(smem + OFF_VEC);
        for (int hi = 0; hi < nheads; ++hi) {
            const int buf = hi & 1, xs = hi % 3, xuse = hi / 3, h = h_begin + hi;
            const float *cs2 = vec + buf * VEC_FLOATS, *dtv = cs2 + 512;
            mbar_wait(&vfull[buf], (hi >> 1) & 1, abortp, p.status);
            const float csr = cs2[r];
            const float offs = FWD ? ex2f(csr) : ex2f(cs2[255] - csr);
            const float dtr = dtv[r];
            __syncwarp();
            if (lane == 0) mbar_arrive(&vempty[buf]);
            const float Dh = __ldg(p.D + h);
            const float Dx = Dh + (FWD ? 0.f : p.dx_skip);       // dx: D dy, plus dy itself under a skip connection
            mbar_wait(&xfull[xs], xuse & 1, abortp, p.status);
            if (!FWD) mbar_wait(&xrfull, hi & 1, abortp, p.status);
            unsigned char *blockbase = smem + OFF_X + xs * 32768 + ((FWD ? rb * 128 : 0) + q * 32) * 128;
            unsigned char *vrow = blockbase + lane * 128;                 // x row (SC_FWD) / dy row (SC_DX), then output
            const unsigned char *xrow = smem + OFF_XR + rl * 128;         // SC_DX: x row
            mbar_wait(&accfull[buf], (hi >> 1) & 1, abortp, p.status);
            tc_fence_after_sync();
            float dd = 0.f, dd2 = 0.f, dsum = 0.f;
#pragma unroll
            for (int pp = 0; pp < NPP; ++pp) {
                const int pass = ech * NPP + pp;
                float a1[16], a2[16];
                tmem_ld16_nowait(tm + tlane + 256 + buf * 128 + pass * 16, a1);
                tmem_ld16_nowait(tm + tlane + 320 + buf * 128 + pass * 16, a2);
                tmem_ld_wait16(a1);
                tmem_ld_wait16(a2);
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    const uint32_t off = (uint32_t)((2 * pass + c2) ^ (rl & 7)) << 4;
                    float vv[8], xv[8];
                    unpack8(*reinterpret_cast<const uint4 *>(vrow + off), vv);
                    if (!FWD) unpack8(*reinterpret_cast<const uint4 *>(xrow + off), xv);
                    uint4 o;
                    uint32_t *ow = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
                    for (int e = 0; e < 8; e += 2) {
                        const int i = c2 * 8 + e;
                        const float u0 = fmaf(offs, a2[i], a1[i]);
                        const float u1 = fmaf(offs, a2[i + 1], a1[i + 1]);
                        if (FWD) {
                            ow[e >> 1] = pack2(fmaf(Dh, vv[e], u0), fmaf(Dh, vv[e + 1], u1));
                        } else {
                            dd = fmaf(xv[e], u0, dd);
                            dd = fmaf(xv[e + 1], u1, dd);
                            dd2 = fmaf(xv[e], a2[i], dd2);
                            dd2 = fmaf(xv[e + 1], a2[i + 1], dd2);
                            dsum = fmaf(vv[e], xv[e], dsum);
                            dsum = fmaf(vv[e + 1], xv[e + 1], dsum);
                            ow[e >> 1] = pack2(fmaf(Dx, vv[e], dtr * u0), fmaf(Dx, vv[e + 1], dtr * u1));
                        }
                    }
                    *reinterpret_cast<uint4 *>(vrow + off) = o;
                }
            }
            if (!FWD) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, off);
                if (EPW == 8 && ech == 1) {      // the upper columns' sums go to the other warp of the quarter (buffers alternate by head)
                    epx[buf][rl][0] = dd;
                    epx[buf][rl][1] = dd2;
                    if (lane == 0) epd[buf][q] = dsum;
                }
            }
            tc_fence_before_sync();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&accempty[buf]);
                if (!FWD) mbar_arrive(&xrempty);
            }
            if (EPW == 8) named_bar_sync(1 + q, 64);          // both halves of the quarter's 32 x 64 block are in place
            if (ech == 0) {
                if (lane == 0) {
                    tma_store_3d(&tmOut, blockbase, h * 64, tok0 + rb * 128 + q * 32, b);
                    tma_store_commit();
                    tma_store_wait_read();              // the store has read the block: the stage may be refilled
                    mbar_arrive(&xempty[xs]);
                }
                if (!FWD) {
                    if (EPW == 8) {
                        dd += epx[buf][rl][0];
                        dd2 += epx[buf][rl][1];
                        dsum += epd[buf][q];
                    }
                    const size_t vo = ((((size_t)b * p.H + h) * p.ncs + c) << 8) + r;
                    p.ddt_dir[vo] = dd;
                    // psi2_s = B_s . (inter-chunk part of this head's dB_s) = dt_s e^{cs_last-cs_s} x_s . (Gout B_s)
                    p.psi2[vo] = dtr * offs * dd2;
                    // dy.x of this quarter's 32 rows: one of 8 partials per (head, chunk), summed later in a fixed order
                    if (lane == 0) p.dDp[((((size_t)b * p.H + h) * p.nct + p.c0 + c) << 4) + rb * 4 + q] = dsum;
                }
            }
        }
        if (lane == 0) tma_store_wait_all();
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tm, 512);
    }
}

cudaError_t launch_scan_tc(const SegParams &p, const TcMaps &m, int mode, cudaStream_t st) {
    const int nsplit = p.nsplit_scan;
    dim3 grid(p.nc * 2 * nsplit * p.G * p.B);
    cudaError_t e;
    if (mode == SC_FWD) {
        e = cudaFuncSetAttribute(k_scan_tc<SC_FWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SC_SMEM);
        if (e != cudaSuccess) return e;
        return launch_pdl(k_scan_tc<SC_FWD>, grid, dim3(sc_threads(SC_FWD)), (size_t)SC_SMEM, st, p, nsplit, m.Cm, m.Bm, m.x, m.Hbf, m.y, m.x);
    } else {
        e = cudaFuncSetAttribute(k_scan_tc<SC_DX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SC_SMEM);
        if (e != cudaSuccess) return e;
        return launch_pdl(k_scan_tc<SC_DX>, grid, dim3(sc_threads(SC_DX)), (size_t)SC_SMEM, st, p, nsplit, m.Bm, m.Cm, m.dy, m.Gbf, m.dx, m.x);
    }
    return cudaGetLastError();
}

}  // namespace ssd
