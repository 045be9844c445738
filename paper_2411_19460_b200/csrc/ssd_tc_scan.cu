// Tensor-core kernel for the two masked products whose score matrix is shared by the heads of a
// group (bf16 I/O, P = 64, N = 128, Q = 256):
//
//   SC_FWD (a5+a6): y_t  = sum_{s<=t} (C_t.B_s) e^{cs_t-cs_s} dt_s x_s + e^{cs_t} C_t H_in + D x_t
//   SC_DX  (a10)  : u_s  = sum_{t>=s} (B_s.C_t) e^{cs_t-cs_s} dy_t      + e^{cs_last-cs_s} B_s Gout
//                   dx_s = D dy_s + dt_s u_s ;  ddt_direct_s = x_s . u_s ;  dD partial = sum dy.x
//
// (Eq. 1 of the paper regrouped by chunks; cs = inclusive cumsum of dt*A inside the chunk.)
//
// One CTA owns (chunk, 128-row block, group, a range of the group's heads).  The score tile
// S = Rows * Cols^T (128 x up to 256, K = N) is computed ONCE with tcgen05.mma into TMEM and stays
// there in fp32 for every head of the range.  Per head the CTA then runs a three-role pipeline:
//   producer warp : TMA loads of the head's value rows (x or dy) and its bf16 chunk state
//   MMA warp      : acc2 = Rows * State^T (K = N), acc1 = sum over 64-column pieces of M_piece * V
//   4 mask warps  : read S from TMEM, apply the decay mask, round to bf16 and store the piece to
//                   shared memory (A operand of the next MMA); then the epilogue of the previous
//                   head from the double-buffered accumulators.
// The decay mask is factored per 32 x 32 sub-tile: strictly off-diagonal sub-tiles use
//   e^{cs_t-cs_s} = e^{cs_t-cs_i0} * e^{cs_i0-cs_j1} * e^{cs_j1-cs_s}      (i0 = first row of the row
// sub-tile, j1 = last column of the column sub-tile), three factors that are each <= 1 because cs
// is non-increasing, so only O(Q) exponentials are needed per head instead of O(Q^2); diagonal
// sub-tiles are exponentiated element by element.
#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

using namespace sm100;

namespace {

constexpr int SC_THREADS = 192;
constexpr uint32_t OFF_ROWS = 0;          // 32 KB  [n-half][128 rows][128 B]
constexpr uint32_t OFF_BX = 32768;        // 64 KB  score columns operand, then two value buffers
constexpr uint32_t OFF_M = 98304;         // 64 KB  four 16 KB pieces of the masked tile
constexpr uint32_t OFF_ST = 163840;       // 32 KB  two state buffers [n-half][64 rows][128 B]
constexpr uint32_t OFF_VEC = 196608;      // per-head vectors, double buffered
constexpr uint32_t VEC_FLOATS = 256 * 3 + 64;
constexpr uint32_t SC_SMEM = OFF_VEC + 2 * VEC_FLOATS * 4 + 1024;

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void bar_mask_warps() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
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

}  // namespace

template <int MODE>
__global__ void __launch_bounds__(SC_THREADS, 1)
k_scan_tc(SegParams p, int nsplit, const __grid_constant__ CUtensorMap tmRow,
          const __grid_constant__ CUtensorMap tmCol, const __grid_constant__ CUtensorMap tmV,
          const __grid_constant__ CUtensorMap tmSt) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar_ab, bar_s, xfull[2], hfull[2], xhempty[2], mfull[4], mempty[4], accfull[2],
        accempty[2];
    __shared__ uint32_t tmem_base, abort_flag;
    __shared__ float dred[4];

    constexpr bool FWD = (MODE == SC_FWD);
    const int nc = p.nc;
    const int rb = FWD ? 1 - (int)(blockIdx.x / nc) : (int)(blockIdx.x / nc);  // long CTAs first
    const int c = blockIdx.x % nc, b = blockIdx.z;
    const int g = blockIdx.y / nsplit, sp = blockIdx.y % nsplit;
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
        for (int i = 0; i < 2; ++i) {
            mbar_init(&xfull[i], 1);
            mbar_init(&hfull[i], 1);
            mbar_init(&xhempty[i], 1);
            mbar_init(&accfull[i], 1);
            mbar_init(&accempty[i], 128);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(&mfull[i], 128);
            mbar_init(&mempty[i], 1);
        }
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc(&tmem_base, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
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
                    tma_load_3d(smem + OFF_BX + nh * ncols * 128 + r0 * 128, &tmCol, &bar_ab, g * 128 + nh * 64,
                                tok0 + colbase + r0, b);
            const int strow = (b * (p.ncs + 1) + slot) * p.H;
            for (int hi = 0; hi < nheads && hi < 2; ++hi) {
                mbar_arrive_expect_tx(&hfull[hi], 16384);
                tma_load_3d(smem + OFF_ST + hi * 16384, &tmSt, &hfull[hi], 0, (strow + h_begin + hi) * 64, 0);
                tma_load_3d(smem + OFF_ST + hi * 16384 + 8192, &tmSt, &hfull[hi], 64, (strow + h_begin + hi) * 64, 0);
            }
            mbar_wait(&bar_s, 0, abortp, p.status);   // score MMAs done: the column operand is dead
            for (int hi = 0; hi < nheads; ++hi) {
                const int buf = hi & 1, h = h_begin + hi;
                if (hi >= 2) {
                    mbar_wait(&xhempty[buf], ((hi >> 1) - 1) & 1, abortp, p.status);
                    mbar_arrive_expect_tx(&hfull[buf], 16384);
                    tma_load_3d(smem + OFF_ST + buf * 16384, &tmSt, &hfull[buf], 0, (strow + h) * 64, 0);
                    tma_load_3d(smem + OFF_ST + buf * 16384 + 8192, &tmSt, &hfull[buf], 64, (strow + h) * 64, 0);
                }
                mbar_arrive_expect_tx(&xfull[buf], (uint32_t)ncols * 128u);
                for (int r0 = 0; r0 < ncols; r0 += 128)
                    tma_load_3d(smem + OFF_BX + buf * 32768 + r0 * 128, &tmV, &xfull[buf], h * 64,
                                tok0 + colbase + r0, b);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t sRows = smem_u32(smem + OFF_ROWS), sBX = smem_u32(smem + OFF_BX);
            const uint32_t sM = smem_u32(smem + OFF_M), sSt = smem_u32(smem + OFF_ST);
            const uint32_t idS = umma_idesc_bf16(128, (uint32_t)ncols, false, false);
            const uint32_t id3 = umma_idesc_bf16(128, 64, false, false);
            const uint32_t id2 = umma_idesc_bf16(128, 64, false, true);
            mbar_wait(&bar_ab, 0, abortp, p.status);
            tc_fence_after_sync();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint64_t ad = umma_desc_sw128(sRows + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024);
                const uint64_t bd = umma_desc_sw128(sBX + (kk >> 2) * (ncols * 128) + (kk & 3) * 32, 16, 1024);
                umma_bf16(tm, ad, bd, idS, kk ? 1u : 0u);
            }
            umma_commit(&bar_s);
            for (int hi = 0; hi < nheads; ++hi) {
                const int buf = hi & 1;
                const uint32_t acc1 = tm + 256 + buf * 128, acc2 = acc1 + 64;
                if (hi >= 2) mbar_wait(&accempty[buf], ((hi >> 1) - 1) & 1, abortp, p.status);
                mbar_wait(&hfull[buf], (hi >> 1) & 1, abortp, p.status);
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t ad = umma_desc_sw128(sRows + (kk >> 2) * 16384 + (kk & 3) * 32, 16, 1024);
                    const uint64_t bd = umma_desc_sw128(sSt + buf * 16384 + (kk >> 2) * 8192 + (kk & 3) * 32, 16, 1024);
                    umma_bf16(acc2, ad, bd, id3, kk ? 1u : 0u);
                }
                mbar_wait(&xfull[buf], (hi >> 1) & 1, abortp, p.status);
                for (int jj = 0; jj < npieces; ++jj) {
                    mbar_wait(&mfull[jj], hi & 1, abortp, p.status);
                    tc_fence_after_sync();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t ad = umma_desc_sw128(sM + jj * 16384 + k * 32, 16, 1024);
                        const uint64_t bd = umma_desc_sw128(sBX + buf * 32768 + (jj * 64 + k * 16) * 128, 8192, 1024);
                        umma_bf16(acc1, ad, bd, id2, (jj | k) ? 1u : 0u);
                    }
                    umma_commit(&mempty[jj]);
                }
                umma_commit(&accfull[buf]);
                umma_commit(&xhempty[buf]);
            }
        }
    } else {
        // ------------------------------------------------------------ mask + epilogue warps
        const int q = warp & 3;                    // TMEM lane quarter this warp may access
        const int mt = (warp - 2) * 32 + lane;     // 0..127 among the mask threads
        const int rl = q * 32 + lane;              // row inside the 128-row block
        const int r = rb * 128 + rl;               // row inside the chunk
        const int isub = r >> 5;
        const uint32_t tlane = (uint32_t)(q * 32) << 16;
        float *vec = reinterpret_cast<float *>(smem + OFF_VEC);
        const size_t HP = (size_t)p.H * 64;
        float offs_prev = 0.f, dt_prev = 0.f;

        auto epilogue = [&](int hi, float offs, float dtr) {
            const int buf = hi & 1, h = h_begin + hi;
            mbar_wait(&accfull[buf], (hi >> 1) & 1, abortp, p.status);
            tc_fence_after_sync();
            const float Dh = __ldg(p.D + h);
            const size_t rowoff = (size_t)b * p.x_bs + (size_t)(tok0 + r) * HP + (size_t)h * 64;
            const uint4 *xr = reinterpret_cast<const uint4 *>((const __nv_bfloat16 *)p.x + rowoff);
            float dd = 0.f, dsum = 0.f;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float a1[32], a2[32];
                tmem_ld32(tm + tlane + 256 + buf * 128 + half * 32, a1);
                tmem_ld32(tm + tlane + 320 + buf * 128 + half * 32, a2);
                if (FWD) {
                    uint4 *yr = reinterpret_cast<uint4 *>((__nv_bfloat16 *)p.y + rowoff);
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8) {
                        float xv[8];
                        unpack8(__ldg(xr + half * 4 + k8), xv);
                        uint4 o;
                        uint32_t *ow = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
                        for (int e = 0; e < 8; e += 2) {
                            const int i = k8 * 8 + e;
                            const float v0 = fmaf(Dh, xv[e], fmaf(offs, a2[i], a1[i]));
                            const float v1 = fmaf(Dh, xv[e + 1], fmaf(offs, a2[i + 1], a1[i + 1]));
                            ow[e >> 1] = pack2(v0, v1);
                        }
                        yr[half * 4 + k8] = o;
                    }
                } else {
                    const uint4 *dyr = reinterpret_cast<const uint4 *>((const __nv_bfloat16 *)p.dy + rowoff);
                    uint4 *dxr = reinterpret_cast<uint4 *>((__nv_bfloat16 *)p.dx + rowoff);
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8) {
                        float xv[8], dyv[8];
                        unpack8(__ldg(xr + half * 4 + k8), xv);
                        unpack8(__ldg(dyr + half * 4 + k8), dyv);
                        uint4 o;
                        uint32_t *ow = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
                        for (int e = 0; e < 8; e += 2) {
                            const int i = k8 * 8 + e;
                            const float u0 = fmaf(offs, a2[i], a1[i]);
                            const float u1 = fmaf(offs, a2[i + 1], a1[i + 1]);
                            dd = fmaf(xv[e], u0, dd);
                            dd = fmaf(xv[e + 1], u1, dd);
                            dsum = fmaf(dyv[e], xv[e], dsum);
                            dsum = fmaf(dyv[e + 1], xv[e + 1], dsum);
                            ow[e >> 1] = pack2(fmaf(Dh, dyv[e], dtr * u0), fmaf(Dh, dyv[e + 1], dtr * u1));
                        }
                        dxr[half * 4 + k8] = o;
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&accempty[buf]);
            if (!FWD) {
                p.ddt_dir[((((size_t)b * p.H + h) * p.ncs + c) << 8) + r] = dd;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, off);
                if (lane == 0) dred[warp - 2] = dsum;
                bar_mask_warps();
                if (mt == 0) {
                    const float s = ((dred[0] + dred[1]) + dred[2]) + dred[3];
                    float *dst = p.dDp + (((((size_t)b * p.H + h) * p.nct + p.c0 + c) << 2) + rb * 2);
                    dst[0] = s;
                    dst[1] = 0.f;
                }
                bar_mask_warps();
            }
        };

        for (int hi = 0; hi < nheads; ++hi) {
            const int h = h_begin + hi;
            float *cs2 = vec + (hi & 1) * VEC_FLOATS, *cf = cs2 + 256, *dtv = cs2 + 512, *blk = cs2 + 768;
            // ---- per-head vectors
            {
                const size_t vo = (((size_t)b * p.H + h) * p.ncs + c) << 8;
                cs2[mt] = p.cs[vo + mt] * kLog2e;
                cs2[mt + 128] = p.cs[vo + mt + 128] * kLog2e;
                dtv[mt] = p.dtT[vo + mt];
                dtv[mt + 128] = p.dtT[vo + mt + 128];
            }
            bar_mask_warps();
#pragma unroll
            for (int w = 0; w < 2; ++w) {
                const int t = mt + w * 128;
                cf[t] = FWD ? ex2f(cs2[t | 31] - cs2[t]) * dtv[t] : ex2f(cs2[t] - cs2[t & ~31]);
            }
            if (mt < 64) {
                const int i = mt >> 3, j = mt & 7;   // blk[i][j] = e^{cs[32 i] - cs[32 j + 31]}, j < i
                blk[mt] = (j < i) ? ex2f(cs2[32 * i] - cs2[32 * j + 31]) : 0.f;
            }
            bar_mask_warps();
            const float csr = cs2[r];
            const float rowf = FWD ? ex2f(csr - cs2[r & ~31]) : ex2f(cs2[r | 31] - csr);
            const float offs = FWD ? ex2f(csr) : ex2f(cs2[255] - csr);
            const float dtr = dtv[r];

            if (hi == 0) {
                mbar_wait(&bar_s, 0, abortp, p.status);
                tc_fence_after_sync();
            }
            // ---- masked pieces
            for (int jj = 0; jj < npieces; ++jj) {
                if (hi >= 1) mbar_wait(&mempty[jj], (hi - 1) & 1, abortp, p.status);
                unsigned char *mrow = smem + OFF_M + jj * 16384 + rl * 128;
#pragma unroll
                for (int sub = 0; sub < 2; ++sub) {
                    const int cb = colbase + jj * 64 + sub * 32;   // first column of the sub-tile (in chunk)
                    const int jsub = cb >> 5;
                    uint32_t pk[16];
                    const bool zero = FWD ? (jsub > isub) : (jsub < isub);
                    if (zero) {
#pragma unroll
                        for (int k = 0; k < 16; ++k) pk[k] = 0u;
                    } else {
                        float v[32];
                        tmem_ld32(tm + tlane + jj * 64 + sub * 32, v);
                        if (jsub != isub) {
                            const float f = rowf * (FWD ? blk[isub * 8 + jsub] : blk[jsub * 8 + isub]);
#pragma unroll
                            for (int k = 0; k < 32; k += 4) {
                                const float4 cv = *reinterpret_cast<const float4 *>(cf + cb + k);
                                v[k] *= cv.x * f;
                                v[k + 1] *= cv.y * f;
                                v[k + 2] *= cv.z * f;
                                v[k + 3] *= cv.w * f;
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
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const int col = cb + k + e;
                                    const bool on = FWD ? (col <= r) : (col >= r);
                                    const float ex = FWD ? ex2f(csr - ccv[e]) * dv[e] : ex2f(ccv[e] - csr);
                                    v[k + e] = on ? v[k + e] * ex : 0.f;
                                }
                            }
                        }
#pragma unroll
                        for (int k = 0; k < 16; ++k) pk[k] = pack2(v[2 * k], v[2 * k + 1]);
                    }
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        const int chunk16 = sub * 4 + ch;
                        *reinterpret_cast<uint4 *>(mrow + ((chunk16 ^ (rl & 7)) << 4)) =
                            make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
                    }
                }
                tc_fence_before_sync();
                fence_proxy_async_smem();
                mbar_arrive(&mfull[jj]);
            }
            if (hi >= 1) epilogue(hi - 1, offs_prev, dt_prev);
            offs_prev = offs;
            dt_prev = dtr;
        }
        epilogue(nheads - 1, offs_prev, dt_prev);
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
    dim3 grid(p.nc * 2, nsplit * p.G, p.B);
    cudaError_t e;
    if (mode == SC_FWD) {
        e = cudaFuncSetAttribute(k_scan_tc<SC_FWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SC_SMEM);
        if (e != cudaSuccess) return e;
        k_scan_tc<SC_FWD><<<grid, SC_THREADS, SC_SMEM, st>>>(p, nsplit, m.Cm, m.Bm, m.x, m.Hbf);
    } else {
        e = cudaFuncSetAttribute(k_scan_tc<SC_DX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SC_SMEM);
        if (e != cudaSuccess) return e;
        k_scan_tc<SC_DX><<<grid, SC_THREADS, SC_SMEM, st>>>(p, nsplit, m.Bm, m.Cm, m.dy, m.Gbf);
    }
    return cudaGetLastError();
}

}  // namespace ssd
