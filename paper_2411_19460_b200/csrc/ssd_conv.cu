// Depthwise causal convolution (width 4) with SiLU: the stage in front of the SSD layer in a Mamba-2 block,
// over the channels (x, B, C) = d_inner + 2 G N.  Its only state across a sequence cut is the last three
// inputs per channel, which is why Appendix C of the paper counts (d_conv - 1)(d_inner + 2 G N) elements of
// "convolution state" into the sequence-axis checkpoint: forward hands the last three tokens of a segment to
// the next one; backward walks the segments right to left and hands the gradient that reaches the three
// tokens in front of a segment to the segment on its left.
//     pre[t,c] = bias[c] + sum_{k<4} w[c,k] u[t-3+k, c]        out = pre * sigmoid(pre)
// Bandwidth-shaped kernels over 512 adjacent channels per CTA, a thread owning 4 of them with a sliding window in
// registers; rows reach shared memory by bulk async copies, one per token row (the channels of a row are contiguous:
// up to 1 KB), so that many kilobytes per SM are in flight without holding registers, and results go straight to
// global memory (8 or 16 bytes per thread, coalesced over the channels).  Forward: one 32-token tile per CTA, staged
// whole (plus the three-token halo).  Backward: a range of tokens per CTA streamed through a ring of 8-token stages.
// Weight and bias gradients: one partial per backward CTA, then a fixed-order sum (no atomics).
#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

using namespace sm100;

namespace {

constexpr int CV_THREADS = 128;   // x 4 channels = 512 channels per CTA
constexpr int CV_CH = 4;          // channels per thread: one 8-byte bf16 vector (16 bytes in fp32)
constexpr int CV_TILE_F = 32;     // tokens per CTA, forward

// 1 / (1 + e^-x) from one ex2.approx and one rcp.approx (relative error of the order of 1e-7; the kernels are bound
// by instruction issue, not by memory, and an IEEE division alone would cost as much as the rest of an element)
__device__ __forceinline__ float sigmoid_fast(float x) {
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * -1.4426950408889634f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.f + e));
    return r;
}

template <typename T> __device__ __forceinline__ void ld4(const T *p, float *f);
template <> __device__ __forceinline__ void ld4<float>(const float *p, float *f) {
    const float4 a = *reinterpret_cast<const float4 *>(p);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
}
template <> __device__ __forceinline__ void ld4<__nv_bfloat16>(const __nv_bfloat16 *p, float *f) {
    const uint2 v = *reinterpret_cast<const uint2 *>(p);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v.y));
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}
template <typename T> __device__ __forceinline__ void st4(T *p, const float *f);
template <> __device__ __forceinline__ void st4<float>(float *p, const float *f) {
    *reinterpret_cast<float4 *>(p) = make_float4(f[0], f[1], f[2], f[3]);
}
template <> __device__ __forceinline__ void st4<__nv_bfloat16>(__nv_bfloat16 *p, const float *f) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(f[0], f[1]), hi = __floats2bfloat162_rn(f[2], f[3]);
    uint2 v;
    v.x = *reinterpret_cast<unsigned int *>(&lo);
    v.y = *reinterpret_cast<unsigned int *>(&hi);
    *reinterpret_cast<uint2 *>(p) = v;
}

// The same four channels as two pairs, for the packed two-lane fp32 instructions of the backward kernel.
template <typename T> __device__ __forceinline__ void ld2x2(const T *p, float2 &a, float2 &b);
template <> __device__ __forceinline__ void ld2x2<float>(const float *p, float2 &a, float2 &b) {
    const float4 v = *reinterpret_cast<const float4 *>(p);
    a = make_float2(v.x, v.y);
    b = make_float2(v.z, v.w);
}
template <> __device__ __forceinline__ void ld2x2<__nv_bfloat16>(const __nv_bfloat16 *p, float2 &a, float2 &b) {
    const uint2 v = *reinterpret_cast<const uint2 *>(p);
    a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v.x));
    b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v.y));
}
__device__ __forceinline__ float2 sigmoid_fast2(float2 x) {
    const float2 t = __fmul2_rn(x, make_float2(-1.4426950408889634f, -1.4426950408889634f));
    float2 e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"(t.x));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"(t.y));
    const float2 d = __fadd2_rn(e, make_float2(1.f, 1.f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r.x) : "f"(d.x));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r.y) : "f"(d.y));
    return r;
}

// Stage rows [t_first, t_last) of a [L, C] tensor (channels cbase .. cbase + nch) into shared memory, row r of the
// stage = token t_first + r, 512 channels of room per row.  Tokens in front of the segment come from the carried
// state (3 rows) or are zero-filled; called by one thread, completion on `bar`.
template <typename T>
__device__ __forceinline__ void stage_rows(T *stage, const T *src, const T *state, long long t_first, long long t_last, int C,
                                           int cbase, int nch, uint64_t *bar) {
    const uint32_t row_bytes = (uint32_t)nch * sizeof(T);
    uint32_t total = 0;
    for (long long t = t_first; t < t_last; ++t)
        if (t >= 0 || state) total += row_bytes;
    if (total) mbar_arrive_expect_tx(bar, total);
    else mbar_arrive(bar);
    for (long long t = t_first; t < t_last; ++t) {
        T *dst = stage + (size_t)(t - t_first) * 512;
        if (t >= 0) bulk_load(dst, src + (size_t)t * C + cbase, row_bytes, bar);
        else if (state) bulk_load(dst, state + (size_t)(3 + t) * C + cbase, row_bytes, bar);
    }
}

template <typename T>
__global__ void __launch_bounds__(CV_THREADS) k_conv_fwd(const T *u, long long u_bs, const float *w, const float *bias,
                                                         const T *state_in, T *out, T *state_out, int L, int C) {
    extern __shared__ __align__(128) unsigned char cv_smem[];
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    __shared__ unsigned int status_dummy;
    T *su = reinterpret_cast<T *>(cv_smem);                       // [CV_TILE_F + 3][512]
    pdl_launch_dependents();
    pdl_wait();       // the previous kernel of the stream (a neighbouring segment's) has finished
    const int cbase = blockIdx.x * 512, nch = min(512, C - cbase);
    const int c0 = cbase + threadIdx.x * CV_CH;
    const int b = blockIdx.z;
    const long long t_begin = (long long)blockIdx.y * CV_TILE_F, t_end = min(t_begin + (long long)CV_TILE_F, (long long)L);
    const T *ub = u + (size_t)b * u_bs;
    const T *sb = state_in ? state_in + (size_t)b * 3 * C : nullptr;
    T *ob = out + (size_t)b * u_bs;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        status_dummy = 0;
        fence_barrier_init();
    }
    // rows in front of the segment without a carried state: zeros (plain stores, before the barrier below)
    if (!sb && t_begin < 3)
        for (int i = threadIdx.x; i < (int)(3 - t_begin) * 512; i += CV_THREADS) su[i] = (T)0.f;
    __syncthreads();
    if (threadIdx.x == 0) stage_rows(su, ub, sb, t_begin - 3, t_end, C, cbase, nch, &bar);
    const bool active = c0 < C;
    float wk[CV_CH][4], bs[CV_CH];
    if (active) {
#pragma unroll
        for (int i = 0; i < CV_CH; ++i) {
            const float4 wv = *reinterpret_cast<const float4 *>(w + (size_t)(c0 + i) * 4);
            wk[i][0] = wv.x; wk[i][1] = wv.y; wk[i][2] = wv.z; wk[i][3] = wv.w;
            bs[i] = bias[c0 + i];
        }
    }
    mbar_wait(&bar, 0, &abort_flag, &status_dummy);
    if (!active) return;
    const T *sp = su + threadIdx.x * CV_CH;
    float x0[CV_CH], x1[CV_CH], x2[CV_CH], x3[CV_CH];   // u[t-3], u[t-2], u[t-1], u[t]
    ld4(sp, x0);
    ld4(sp + 512, x1);
    ld4(sp + 1024, x2);
    const int nt = (int)(t_end - t_begin);
#pragma unroll 4
    for (int j = 0; j < nt; ++j) {
        ld4(sp + (size_t)(j + 3) * 512, x3);
        float o[CV_CH];
#pragma unroll
        for (int i = 0; i < CV_CH; ++i) {
            const float pre = fmaf(wk[i][3], x3[i], fmaf(wk[i][2], x2[i], fmaf(wk[i][1], x1[i], fmaf(wk[i][0], x0[i], bs[i]))));
            o[i] = pre * sigmoid_fast(pre);
            x0[i] = x1[i]; x1[i] = x2[i]; x2[i] = x3[i];
        }
        st4(ob + (size_t)(t_begin + j) * C + c0, o);
    }
    // the last three inputs of the segment are the state of the next one
    if (state_out && t_end == L) {
        T *so = state_out + (size_t)b * 3 * C;
        st4(so + c0, x0);
        st4(so + (size_t)C + c0, x1);
        st4(so + (size_t)2 * C + c0, x2);
    }
}

// Backward over a range of consecutive tokens.  dpre[t] = dout[t] * silu'(pre[t]);  du[t] = sum_k w[k] dpre[t+3-k].
// A CTA owns 512 channels and walks its range front to back with the last three inputs and the last four dpre in
// registers, so nothing is staged or formed twice inside the range; only at its end does it form dpre of the three
// tokens behind it (for its own last du's; past the end of the segment they are not formed: their effect arrives
// as `dtail`).  The rows of u and dout stream through a ring of 8-token stages filled by a producer warp with one
// bulk copy per row, so the loads of later stages are in flight while a stage is being consumed.
// dw, dbias: one partial per range, the range's own tokens.
constexpr int CV_STG_TOK = 8;
constexpr int CV_STAGES = 3;
constexpr int CV_BWD_THREADS = CV_THREADS + 32;   // four compute warps and the producer warp

template <typename T>
__global__ void __launch_bounds__(CV_BWD_THREADS, 4)
k_conv_bwd(const T *u, long long u_bs, const float *w, const float *bias, const T *state_in, const T *dout,
           const float *dtail, T *du, float *dstate, float *part, int L, int C, int RL) {
    extern __shared__ __align__(128) unsigned char cv_smem[];
    __shared__ uint64_t full[CV_STAGES], empty[CV_STAGES];
    __shared__ uint32_t abort_flag;
    __shared__ unsigned int status_dummy;
    T *ring = reinterpret_cast<T *>(cv_smem);                     // [stage][u rows | dout rows][512]
    pdl_launch_dependents();
    pdl_wait();
    const int cbase = blockIdx.x * 512, nch = min(512, C - cbase);
    const int b = blockIdx.z;
    const long long r_begin = (long long)blockIdx.y * RL, r_end = min(r_begin + (long long)RL, (long long)L);
    const int ntok = (int)(r_end - r_begin), nst = (ntok + CV_STG_TOK - 1) / CV_STG_TOK;
    const T *ub = u + (size_t)b * u_bs, *gb = dout + (size_t)b * u_bs;
    const T *sb = state_in ? state_in + (size_t)b * 3 * C : nullptr;
    T *dub = du + (size_t)b * u_bs;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < CV_STAGES; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], CV_THREADS / 32);    // one arrival per compute warp
        }
        abort_flag = 0;
        status_dummy = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == CV_THREADS / 32) {
        // ---- producer
        if (lane == 0) {
            const uint32_t row_bytes = (uint32_t)nch * sizeof(T);
            for (int i = 0; i < nst; ++i) {
                const int slot = i % CV_STAGES;
                if (i >= CV_STAGES) mbar_wait(&empty[slot], ((i / CV_STAGES) - 1) & 1, &abort_flag, &status_dummy);
                const long long t0 = r_begin + (long long)i * CV_STG_TOK;
                const int n = (int)min((long long)CV_STG_TOK, r_end - t0);
                mbar_arrive_expect_tx(&full[slot], 2u * (uint32_t)n * row_bytes);
                T *su = ring + (size_t)slot * (2 * CV_STG_TOK * 512), *sg = su + CV_STG_TOK * 512;
                for (int j = 0; j < n; ++j) {
                    bulk_load(su + (size_t)j * 512, ub + (size_t)(t0 + j) * C + cbase, row_bytes, &full[slot]);
                    bulk_load(sg + (size_t)j * 512, gb + (size_t)(t0 + j) * C + cbase, row_bytes, &full[slot]);
                }
            }
        }
        return;
    }
    const int c0 = cbase + threadIdx.x * CV_CH;
    const bool active = c0 < C;      // inactive threads (past the last channel) still take part in the hand-overs
    // two channel pairs per thread: every quantity below is a float2 over (c, c + 1), so that the multiply-adds
    // issue as packed two-lane instructions
    constexpr int NP = CV_CH / 2;
    const float2 zero2 = make_float2(0.f, 0.f), one2 = make_float2(1.f, 1.f), mone2 = make_float2(-1.f, -1.f);
    float2 wk[NP][4], bs[NP];
    float2 x0[NP], x1[NP], x2[NP], x3[NP];
    float2 d0[NP], d1[NP], d2[NP], d3[NP];     // dpre[t], dpre[t+1], dpre[t+2], dpre[t+3] while emitting du[t]
    float2 aw[NP][4], ab[NP];
    const bool head_range = (dstate != nullptr) && blockIdx.y == 0;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        aw[i][0] = aw[i][1] = aw[i][2] = aw[i][3] = zero2;
        ab[i] = zero2;
        d0[i] = d1[i] = d2[i] = d3[i] = zero2;
        x0[i] = x1[i] = x2[i] = x3[i] = zero2;
        wk[i][0] = wk[i][1] = wk[i][2] = wk[i][3] = bs[i] = zero2;
    }
    // the input at token t of the segment; in front of it the carried state, or zeros
    auto ld_u = [&](long long t, float2 *v) {
        if (t >= 0) ld2x2(ub + (size_t)t * C + c0, v[0], v[1]);
        else if (sb) ld2x2(sb + (size_t)(3 + t) * C + c0, v[0], v[1]);
        else v[0] = v[1] = zero2;
    };
    if (active) {
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            const float4 wa = *reinterpret_cast<const float4 *>(w + (size_t)(c0 + 2 * i) * 4);
            const float4 wb = *reinterpret_cast<const float4 *>(w + (size_t)(c0 + 2 * i + 1) * 4);
            wk[i][0] = make_float2(wa.x, wb.x); wk[i][1] = make_float2(wa.y, wb.y);
            wk[i][2] = make_float2(wa.z, wb.z); wk[i][3] = make_float2(wa.w, wb.w);
            bs[i] = make_float2(bias[c0 + 2 * i], bias[c0 + 2 * i + 1]);
        }
        ld_u(r_begin - 3, x0);
        ld_u(r_begin - 2, x1);
        ld_u(r_begin - 1, x2);
    }
    // dpre of token s from its input x3 (the window x0..x2 holds the three before it) and g = dout[s]; own tokens
    // also feed the weight and bias gradients.  Then the windows move on and du[s - 3] is complete.
    auto token = [&](long long s, const float2 *g, bool own, bool formed) {
        float2 dp[NP];
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            if (formed) {
                const float2 pre = __ffma2_rn(wk[i][3], x3[i], __ffma2_rn(wk[i][2], x2[i], __ffma2_rn(wk[i][1], x1[i], __ffma2_rn(wk[i][0], x0[i], bs[i]))));
                const float2 sgm = sigmoid_fast2(pre);
                // dpre = dout * silu'(pre),  silu'(z) = s (1 + z (1 - s))
                dp[i] = __fmul2_rn(__fmul2_rn(g[i], sgm), __ffma2_rn(pre, __ffma2_rn(sgm, mone2, one2), one2));
                if (own) {
                    aw[i][0] = __ffma2_rn(dp[i], x0[i], aw[i][0]);
                    aw[i][1] = __ffma2_rn(dp[i], x1[i], aw[i][1]);
                    aw[i][2] = __ffma2_rn(dp[i], x2[i], aw[i][2]);
                    aw[i][3] = __ffma2_rn(dp[i], x3[i], aw[i][3]);
                    ab[i] = __fadd2_rn(ab[i], dp[i]);
                }
                x0[i] = x1[i]; x1[i] = x2[i]; x2[i] = x3[i];
            } else {
                dp[i] = zero2;
            }
            d0[i] = d1[i]; d1[i] = d2[i]; d2[i] = d3[i]; d3[i] = dp[i];
        }
        if (head_range && s == 2) {
            // What the first three dpre rows of the segment (now d1, d2, d3) send to the three tokens in front of it:
            // token -3 feeds pre[0] through w[0]; token -2: pre[0] w[1], pre[1] w[0]; token -1: pre[0] w[2], pre[1] w[1],
            // pre[2] w[0].
            float *ds = dstate + (size_t)b * 3 * C + c0;
            float e[CV_CH];
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const float2 v = __fmul2_rn(wk[i][0], d1[i]);
                e[2 * i] = v.x; e[2 * i + 1] = v.y;
            }
            st4(ds, e);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const float2 v = __ffma2_rn(wk[i][0], d2[i], __fmul2_rn(wk[i][1], d1[i]));
                e[2 * i] = v.x; e[2 * i + 1] = v.y;
            }
            st4(ds + (size_t)C, e);
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const float2 v = __ffma2_rn(wk[i][0], d3[i], __ffma2_rn(wk[i][1], d2[i], __fmul2_rn(wk[i][2], d1[i])));
                e[2 * i] = v.x; e[2 * i + 1] = v.y;
            }
            st4(ds + (size_t)2 * C, e);
        }
        const long long t = s - 3;
        if (t >= r_begin) {
            float o[CV_CH];
#pragma unroll
            for (int i = 0; i < NP; ++i) {
                const float2 v = __ffma2_rn(wk[i][3], d0[i], __ffma2_rn(wk[i][2], d1[i], __ffma2_rn(wk[i][1], d2[i], __fmul2_rn(wk[i][0], d3[i]))));
                o[2 * i] = v.x;
                o[2 * i + 1] = v.y;
            }
            if (dtail && t >= (long long)L - 3) {
                float e[CV_CH];
                ld4(dtail + ((size_t)b * 3 + (size_t)(t - ((long long)L - 3))) * C + c0, e);
#pragma unroll
                for (int i = 0; i < CV_CH; ++i) o[i] += e[i];
            }
            st4(dub + (size_t)t * C + c0, o);
        }
    };
    for (int i = 0; i < nst; ++i) {
        const int slot = i % CV_STAGES;
        mbar_wait(&full[slot], (i / CV_STAGES) & 1, &abort_flag, &status_dummy);
        if (active) {
            const T *spu = ring + (size_t)slot * (2 * CV_STG_TOK * 512) + threadIdx.x * CV_CH, *spg = spu + CV_STG_TOK * 512;
            const long long t0 = r_begin + (long long)i * CV_STG_TOK;
            const int n = (int)min((long long)CV_STG_TOK, r_end - t0);
#pragma unroll 4
            for (int j = 0; j < n; ++j) {
                float2 g[NP];
                ld2x2(spu + (size_t)j * 512, x3[0], x3[1]);
                ld2x2(spg + (size_t)j * 512, g[0], g[1]);
                token(t0 + j, g, true, true);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[slot]);      // this warp has read the stage
    }
    if (!active) return;
    // the three tokens behind the range complete its last du's (plain loads: 16 bytes per thread and token)
    for (int k = 0; k < 3; ++k) {
        const long long s = r_end + k;
        float2 g[NP] = {zero2, zero2};
        const bool formed = s < (long long)L;
        if (formed) {
            ld2x2(ub + (size_t)s * C + c0, x3[0], x3[1]);
            ld2x2(gb + (size_t)s * C + c0, g[0], g[1]);
        }
        token(s, g, false, formed);
    }
    // partial weight / bias gradients of this range: part[b][range][5][C]
    {
        float *pp = part + (((size_t)b * gridDim.y + blockIdx.y) * 5) * C + c0;
        float col[CV_CH];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
#pragma unroll
            for (int i = 0; i < NP; ++i) { col[2 * i] = aw[i][k].x; col[2 * i + 1] = aw[i][k].y; }
            st4(pp + (size_t)k * C, col);
        }
#pragma unroll
        for (int i = 0; i < NP; ++i) { col[2 * i] = ab[i].x; col[2 * i + 1] = ab[i].y; }
        st4(pp + (size_t)4 * C, col);
    }
}

// dw[c][k], dbias[c] from the tile partials, in fp64 and in a fixed order: a CTA owns 32 adjacent channels of one of the
// five rows (four taps, bias); its eight warps take the tiles round-robin (coalesced 128-byte reads, several in flight),
// then the eight partial sums are added in warp order.
__global__ void __launch_bounds__(256) k_conv_reduce(const float *part, float *dw, float *dbias, int C, int ntiles, int B,
                                                     int accumulate) {
    __shared__ double red[8][32];
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    const int nblk = (C + 31) / 32;
    const int k = blockIdx.x / nblk, c = (blockIdx.x % nblk) * 32 + lane;
    double s = 0.0;
    if (c < C) {
        const long long total = (long long)B * ntiles;
#pragma unroll 4
        for (long long t = wp; t < total; t += 8) s += (double)part[((size_t)t * 5 + k) * C + c];
    }
    red[wp][lane] = s;
    __syncthreads();
    if (wp == 0 && c < C) {
        double tot = 0.0;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += red[i][lane];
        if (k < 4) {
            float *d = dw + (size_t)c * 4 + k;
            *d = accumulate ? *d + (float)tot : (float)tot;
        } else {
            dbias[c] = accumulate ? dbias[c] + (float)tot : (float)tot;
        }
    }
}

template <typename T>
cudaError_t conv_fwd_t(const T *u, long long u_bs, const float *w, const float *bias, const T *state_in, T *out, T *state_out,
                       int B, int L, int C, cudaStream_t st) {
    const int smem = (CV_TILE_F + 3) * 512 * (int)sizeof(T);
    cudaError_t e = cudaFuncSetAttribute(k_conv_fwd<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    dim3 grid((C + 511) / 512, (L + CV_TILE_F - 1) / CV_TILE_F, B);
    return launch_pdl(k_conv_fwd<T>, grid, dim3(CV_THREADS), (size_t)smem, st, u, u_bs, w, bias, state_in, out, state_out, L, C);
}

// Tokens per CTA of the backward: about four CTAs per SM over the whole launch, whole stages, and never
// more ranges than conv_tiles() promises scratch for.
static int conv_range_len(int B, int L, int C) {
    const int nblk = (C + 511) / 512;
    int want = (4 * 148) / (nblk * B);
    if (want < 1) want = 1;
    int rl = ((L + want - 1) / want + CV_STG_TOK - 1) / CV_STG_TOK * CV_STG_TOK;
    if (rl < 32) rl = 32;
    return rl;
}

template <typename T>
cudaError_t conv_bwd_t(const T *u, long long u_bs, const float *w, const float *bias, const T *state_in, const T *dout,
                       const float *dtail, T *du, float *dstate, float *part, int B, int L, int C, int RL, cudaStream_t st) {
    const int smem = CV_STAGES * 2 * CV_STG_TOK * 512 * (int)sizeof(T);
    cudaError_t e = cudaFuncSetAttribute(k_conv_bwd<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    dim3 grid((C + 511) / 512, (L + RL - 1) / RL, B);
    return launch_pdl(k_conv_bwd<T>, grid, dim3(CV_BWD_THREADS), (size_t)smem, st, u, u_bs, w, bias, state_in, dout, dtail, du, dstate,
                      part, L, C, RL);
}

}  // namespace

int conv_tiles(int L) { return (L + 31) / 32; }

cudaError_t launch_conv_fwd(int dtype, const void *u, long long u_bs, const float *w, const float *bias,
                            const void *state_in, void *out, void *state_out, int B, int L, int C, cudaStream_t st) {
    if (dtype == SSD_DTYPE_F32)
        return conv_fwd_t<float>((const float *)u, u_bs, w, bias, (const float *)state_in, (float *)out, (float *)state_out, B,
                                 L, C, st);
    return conv_fwd_t<__nv_bfloat16>((const __nv_bfloat16 *)u, u_bs, w, bias, (const __nv_bfloat16 *)state_in,
                                     (__nv_bfloat16 *)out, (__nv_bfloat16 *)state_out, B, L, C, st);
}

cudaError_t launch_conv_bwd(int dtype, const void *u, long long u_bs, const float *w, const float *bias,
                            const void *state_in, const void *dout, const float *dtail, void *du, float *dstate,
                            float *dw, float *dbias, int accumulate, float *part, int B, int L, int C, cudaStream_t st) {
    const int RL = conv_range_len(B, L, C);
    cudaError_t e;
    if (dtype == SSD_DTYPE_F32)
        e = conv_bwd_t<float>((const float *)u, u_bs, w, bias, (const float *)state_in, (const float *)dout, dtail, (float *)du,
                              dstate, part, B, L, C, RL, st);
    else
        e = conv_bwd_t<__nv_bfloat16>((const __nv_bfloat16 *)u, u_bs, w, bias, (const __nv_bfloat16 *)state_in,
                                      (const __nv_bfloat16 *)dout, dtail, (__nv_bfloat16 *)du, dstate, part, B, L, C, RL, st);
    if (e != cudaSuccess) return e;
    return launch_pdl(k_conv_reduce, dim3(5 * ((C + 31) / 32)), dim3(256), (size_t)0, st, (const float *)part, dw, dbias, C,
                      (L + RL - 1) / RL, B, accumulate);
}

}  // namespace ssd
