// Gated RMS normalisation behind the SSD layer in a Mamba-2 block: v = y * silu(z), out = v * rsqrt(mean(v^2) + eps) * gamma,
// the mean taken over groups of `group` adjacent channels (the whole d_inner, or d_inner / G).  Token-local: no state
// crosses a sequence cut, so a segment is just a range of rows.  One CTA owns one group index and a tile of rows; a row of
// a group is held in registers (up to 8 four-channel vectors per thread, 256 threads: groups of up to 8192 channels), so
// every tensor is read once; the sums over a row meet through warp shuffles and shared memory in a fixed order; the
// gradient of gamma is accumulated per CTA over its rows and added over the tiles by a second kernel (no atomics).
#include "ssd_internal.h"
#include "ssd_sm100.cuh"

namespace ssd {

using namespace sm100;

namespace {

constexpr int GN_THREADS = 256;
constexpr int GN_MAXV = 8;        // four-channel vectors per thread, at most (the kernels are instantiated for 1, 2, 4, 5 and 8)
constexpr int GN_ROWS = 16;       // rows per CTA
constexpr int GN_STAGES = 3;      // rows in flight per CTA in the staged kernels

template <typename T> __device__ __forceinline__ void gld4(const T *p, float *f);
template <> __device__ __forceinline__ void gld4<float>(const float *p, float *f) {
    const float4 a = *reinterpret_cast<const float4 *>(p);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
}
template <> __device__ __forceinline__ void gld4<__nv_bfloat16>(const __nv_bfloat16 *p, float *f) {
    const uint2 v = *reinterpret_cast<const uint2 *>(p);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v.y));
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}
template <typename T> __device__ __forceinline__ void gst4(T *p, const float *f);
template <> __device__ __forceinline__ void gst4<float>(float *p, const float *f) {
    *reinterpret_cast<float4 *>(p) = make_float4(f[0], f[1], f[2], f[3]);
}
template <> __device__ __forceinline__ void gst4<__nv_bfloat16>(__nv_bfloat16 *p, const float *f) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(f[0], f[1]), hi = __floats2bfloat162_rn(f[2], f[3]);
    uint2 v;
    v.x = *reinterpret_cast<unsigned int *>(&lo);
    v.y = *reinterpret_cast<unsigned int *>(&hi);
    *reinterpret_cast<uint2 *>(p) = v;
}
__device__ __forceinline__ float sigmoid_gn(float x) {
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * -1.4426950408889634f));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.f + e));
    return r;
}
// sum over the CTA in a fixed order: lanes by shuffle tree, then the eight warps in order
__device__ __forceinline__ float block_sum(float v, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                       // red may still be read from the previous call
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < GN_THREADS / 32; ++w) s += red[w];
    return s;
}

template <typename T, int NV>
__global__ void __launch_bounds__(GN_THREADS) k_gated_norm_fwd(const T *y, const T *z, const float *gamma, float eps, T *out,
                                                               long long rows, int D, int group) {
    __shared__ float red[GN_THREADS / 32];
    const int gi = blockIdx.y, nv = group / 4;
    const long long r0 = (long long)blockIdx.x * GN_ROWS, r1 = min(r0 + (long long)GN_ROWS, rows);
    float gm[NV][4];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int i = threadIdx.x + k * GN_THREADS;
        if (i < nv) gld4(gamma + (size_t)gi * group + (size_t)i * 4, gm[k]);
    }
    for (long long r = r0; r < r1; ++r) {
        const size_t base = (size_t)r * D + (size_t)gi * group;
        float v[NV][4];
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int i = threadIdx.x + k * GN_THREADS;
            if (i < nv) {
                float a[4], b[4];
                gld4(y + base + (size_t)i * 4, a);
                gld4(z + base + (size_t)i * 4, b);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    v[k][e] = a[e] * b[e] * sigmoid_gn(b[e]);
                    ss = fmaf(v[k][e], v[k][e], ss);
                }
            }
        }
        const float n = rsqrtf(block_sum(ss, red) / (float)group + eps);
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int i = threadIdx.x + k * GN_THREADS;
            if (i < nv) {
                float o[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) o[e] = v[k][e] * n * gm[k][e];
                gst4(out + base + (size_t)i * 4, o);
            }
        }
    }
}

template <typename T, int NV>
__global__ void __launch_bounds__(GN_THREADS, NV <= 5 ? 2 : 1) k_gated_norm_bwd(const T *y, const T *z, const float *gamma, float eps,
                                                               const T *dout, T *dy, T *dz, float *part, long long rows, int D,
                                                               int group) {
    __shared__ float red[GN_THREADS / 32];
    const int gi = blockIdx.y, nv = group / 4;
    const long long r0 = (long long)blockIdx.x * GN_ROWS, r1 = min(r0 + (long long)GN_ROWS, rows);
    float gm[NV][4], dg[NV][4];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int i = threadIdx.x + k * GN_THREADS;
        if (i < nv) gld4(gamma + (size_t)gi * group + (size_t)i * 4, gm[k]);
#pragma unroll
        for (int e = 0; e < 4; ++e) dg[k][e] = 0.f;
    }
    for (long long r = r0; r < r1; ++r) {
        const size_t base = (size_t)r * D + (size_t)gi * group;
        float v[NV][4], zz[NV][4], yy[NV][4], g[NV][4];
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int i = threadIdx.x + k * GN_THREADS;
            if (i < nv) {
                gld4(y + base + (size_t)i * 4, yy[k]);
                gld4(z + base + (size_t)i * 4, zz[k]);
                gld4(dout + base + (size_t)i * 4, g[k]);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    v[k][e] = yy[k][e] * zz[k][e] * sigmoid_gn(zz[k][e]);
                    ss = fmaf(v[k][e], v[k][e], ss);
                }
            }
        }
        const float n = rsqrtf(block_sum(ss, red) / (float)group + eps);
        // xh = v n ;  dvh = dout gamma ;  c = mean(dvh xh) ;  dv = n (dvh - xh c)
        float dot = 0.f;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int i = threadIdx.x + k * GN_THREADS;
            if (i < nv) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float xh = v[k][e] * n;
                    dg[k][e] = fmaf(g[k][e], xh, dg[k][e]);
                    dot = fmaf(g[k][e] * gm[k][e], xh, dot);
                }
            }
        }
        const float cmean = block_sum(dot, red) / (float)group;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int i = threadIdx.x + k * GN_THREADS;
            if (i < nv) {
                float oy[4], oz[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float xh = v[k][e] * n;
                    const float dv = n * fmaf(-xh, cmean, g[k][e] * gm[k][e]);
                    const float sg = sigmoid_gn(zz[k][e]);
                    oy[e] = dv * zz[k][e] * sg;                                         // d silu(z) y / dy
                    oz[e] = dv * yy[k][e] * sg * fmaf(zz[k][e], 1.f - sg, 1.f);          // y silu'(z)
                }
                gst4(dy + base + (size_t)i * 4, oy);
                gst4(dz + base + (size_t)i * 4, oz);
            }
        }
    }
    // this CTA's part of dgamma: part[tile][D]
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int i = threadIdx.x + k * GN_THREADS;
        if (i < nv) gst4(part + (size_t)blockIdx.x * D + (size_t)gi * group + (size_t)i * 4, dg[k]);
    }
}

// ---- staged variants: the rows of a CTA's tile stream through a ring of GN_STAGES shared-memory buffers filled by
// bulk async copies (one per tensor and row: the channels of a group are contiguous), so that several rows per CTA
// are in flight without holding them in registers; the arithmetic then reads a row from shared memory as often as
// it needs to.  Used when the ring fits (bf16 rows of the model sizes do); otherwise the kernels above.
template <typename T, int NV, bool BWD>
__global__ void __launch_bounds__(GN_THREADS, 2) k_gated_norm_staged(const T *y, const T *z, const float *gamma, float eps,
                                                                     const T *dout, T *out_or_dy, T *dz, float *part,
                                                                     long long rows, int D, int group) {
    extern __shared__ __align__(128) unsigned char gn_smem[];
    __shared__ float red[GN_THREADS / 32];
    __shared__ uint64_t full[GN_STAGES];
    __shared__ uint32_t abort_flag;
    __shared__ unsigned int status_dummy;
    constexpr int NT = BWD ? 3 : 2;                       // tensors staged per row
    const int gi = blockIdx.y, nv = group / 4;
    const long long r0 = (long long)blockIdx.x * GN_ROWS;
    const int nrows = (int)min((long long)GN_ROWS, rows - r0);
    const uint32_t row_bytes = (uint32_t)group * sizeof(T);
    T *ring = reinterpret_cast<T *>(gn_smem);             // [GN_STAGES][NT][group]
    auto issue = [&](int j) {                             // thread 0: row r0 + j into stage j % GN_STAGES
        const int st = j % GN_STAGES;
        const size_t base = (size_t)(r0 + j) * D + (size_t)gi * group;
        T *dst = ring + (size_t)st * NT * group;
        mbar_arrive_expect_tx(&full[st], NT * row_bytes);
        bulk_load(dst, y + base, row_bytes, &full[st]);
        bulk_load(dst + group, z + base, row_bytes, &full[st]);
        if (BWD) bulk_load(dst + 2 * (size_t)group, dout + base, row_bytes, &full[st]);
    };
    if (threadIdx.x == 0) {
        for (int i = 0; i < GN_STAGES; ++i) mbar_init(&full[i], 1);
        abort_flag = 0;
        status_dummy = 0;
        fence_barrier_init();
        for (int j = 0; j < GN_STAGES - 1 && j < nrows; ++j) issue(j);
    }
    float gm[NV][4], dg[NV][4];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
        const int i = threadIdx.x + k * GN_THREADS;
        if (i < nv) gld4(gamma + (size_t)gi * group + (size_t)i * 4, gm[k]);
#pragma unroll
        for (int e = 0; e < 4; ++e) dg[k][e] = 0.f;
    }
    __syncthreads();
    for (int j = 0; j < nrows; ++j) {
        // the stage that row j + GN_STAGES - 1 goes to was read in iteration j - 1, which ended with a CTA barrier
        if (threadIdx.x == 0 && j + GN_STAGES - 1 < nrows) issue(j + GN_STAGES - 1);
        const int st = j % GN_STAGES;
        mbar_wait(&full[st], (uint32_t)(j / GN_STAGES) & 1u, &abort_flag, &status_dummy);
        const T *sy = ring + (size_t)st * NT * group, *sz = sy + group, *sg = sy + 2 * (size_t)group;
        const size_t base = (size_t)(r0 + j) * D + (size_t)gi * group;
        float v[NV][4];
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int i = threadIdx.x + k * GN_THREADS;
            if (i < nv) {
                float a[4], b[4];
                gld4(sy + (size_t)i * 4, a);
                gld4(sz + (size_t)i * 4, b);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    v[k][e] = a[e] * b[e] * sigmoid_gn(b[e]);
                    ss = fmaf(v[k][e], v[k][e], ss);
                }
            }
        }
        const float n = rsqrtf(block_sum(ss, red) / (float)group + eps);
        if (!BWD) {
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int i = threadIdx.x + k * GN_THREADS;
                if (i < nv) {
                    float o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) o[e] = v[k][e] * n * gm[k][e];
                    gst4(out_or_dy + base + (size_t)i * 4, o);
                }
            }
        } else {
            // xh = v n ;  dvh = dout gamma ;  c = mean(dvh xh) ;  dv = n (dvh - xh c)
            float dot = 0.f;
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int i = threadIdx.x + k * GN_THREADS;
                if (i < nv) {
                    float g[4];
                    gld4(sg + (size_t)i * 4, g);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float xh = v[k][e] * n;
                        dg[k][e] = fmaf(g[e], xh, dg[k][e]);
                        dot = fmaf(g[e] * gm[k][e], xh, dot);
                    }
                }
            }
            const float cmean = block_sum(dot, red) / (float)group;
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int i = threadIdx.x + k * GN_THREADS;
                if (i < nv) {
                    float a[4], b[4], g[4], oy[4], oz[4];
                    gld4(sy + (size_t)i * 4, a);
                    gld4(sz + (size_t)i * 4, b);
                    gld4(sg + (size_t)i * 4, g);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float xh = v[k][e] * n;
                        const float dv = n * fmaf(-xh, cmean, g[e] * gm[k][e]);
                        const float sgm = sigmoid_gn(b[e]);
                        oy[e] = dv * b[e] * sgm;
                        oz[e] = dv * a[e] * sgm * fmaf(b[e], 1.f - sgm, 1.f);
                    }
                    gst4(out_or_dy + base + (size_t)i * 4, oy);
                    gst4(dz + base + (size_t)i * 4, oz);
                }
            }
        }
        __syncthreads();                                  // every thread is done with stage `st`
    }
    if (BWD) {
#pragma unroll
        for (int k = 0; k < NV; ++k) {
            const int i = threadIdx.x + k * GN_THREADS;
            if (i < nv) gst4(part + (size_t)blockIdx.x * D + (size_t)gi * group + (size_t)i * 4, dg[k]);
        }
    }
}

// dgamma from the tile partials, in fp64 and in a fixed order: a CTA owns 32 adjacent channels; its eight warps take the
// tiles round-robin (coalesced reads, several in flight), then the eight partial sums are added in warp order.
__global__ void __launch_bounds__(256) k_gated_norm_reduce(const float *part, float *dgamma, int D, int ntiles, int accumulate) {
    __shared__ double red[8][32];
    const int lane = threadIdx.x & 31, wp = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + lane;
    double s = 0.0;
    if (c < D) {
#pragma unroll 4
        for (int t = wp; t < ntiles; t += 8) s += (double)part[(size_t)t * D + c];
    }
    red[wp][lane] = s;
    __syncthreads();
    if (wp == 0 && c < D) {
        double tot = 0.0;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += red[i][lane];
        dgamma[c] = accumulate ? dgamma[c] + (float)tot : (float)tot;
    }
}

}  // namespace

long long gated_norm_tiles(long long rows) { return (rows + GN_ROWS - 1) / GN_ROWS; }
int gated_norm_max_group() { return GN_MAXV * GN_THREADS * 4; }

template <typename T>
static cudaError_t norm_fwd_t(const T *y, const T *z, const float *gamma, float eps, T *out, long long rows, int D, int group,
                              cudaStream_t st) {
    dim3 grid((unsigned)gated_norm_tiles(rows), D / group);
    const int need = (group / 4 + GN_THREADS - 1) / GN_THREADS;
    const size_t ring = (size_t)GN_STAGES * 2 * group * sizeof(T);
    if (ring <= 100 * 1024 && need <= 5 && ((size_t)group * sizeof(T)) % 16 == 0) {
#define GN_SCASE(NV)                                                                                                   \
    do {                                                                                                               \
        cudaError_t e = cudaFuncSetAttribute(k_gated_norm_staged<T, NV, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring); \
        if (e != cudaSuccess) return e;                                                                                \
        k_gated_norm_staged<T, NV, false><<<grid, GN_THREADS, ring, st>>>(y, z, gamma, eps, (const T *)nullptr, out, (T *)nullptr, \
                                                                          (float *)nullptr, rows, D, group);            \
    } while (0)
        if (need <= 1) GN_SCASE(1); else if (need <= 2) GN_SCASE(2); else if (need <= 4) GN_SCASE(4); else GN_SCASE(5);
#undef GN_SCASE
        return cudaGetLastError();
    }
#define GN_CASE(NV) k_gated_norm_fwd<T, NV><<<grid, GN_THREADS, 0, st>>>(y, z, gamma, eps, out, rows, D, group)
    if (need <= 1) GN_CASE(1); else if (need <= 2) GN_CASE(2); else if (need <= 4) GN_CASE(4); else if (need <= 5) GN_CASE(5); else GN_CASE(8);
#undef GN_CASE
    return cudaGetLastError();
}
template <typename T>
static cudaError_t norm_bwd_t(const T *y, const T *z, const float *gamma, float eps, const T *dout, T *dy, T *dz, float *part,
                              long long rows, int D, int group, cudaStream_t st) {
    dim3 grid((unsigned)gated_norm_tiles(rows), D / group);
    const int need = (group / 4 + GN_THREADS - 1) / GN_THREADS;
    const size_t ring = (size_t)GN_STAGES * 3 * group * sizeof(T);
    if (ring <= 100 * 1024 && need <= 5 && ((size_t)group * sizeof(T)) % 16 == 0) {
#define GN_SCASE(NV)                                                                                                   \
    do {                                                                                                               \
        cudaError_t e = cudaFuncSetAttribute(k_gated_norm_staged<T, NV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring); \
        if (e != cudaSuccess) return e;                                                                                \
        k_gated_norm_staged<T, NV, true><<<grid, GN_THREADS, ring, st>>>(y, z, gamma, eps, dout, dy, dz, part, rows, D, group); \
    } while (0)
        if (need <= 1) GN_SCASE(1); else if (need <= 2) GN_SCASE(2); else if (need <= 4) GN_SCASE(4); else GN_SCASE(5);
#undef GN_SCASE
        return cudaGetLastError();
    }
#define GN_CASE(NV) k_gated_norm_bwd<T, NV><<<grid, GN_THREADS, 0, st>>>(y, z, gamma, eps, dout, dy, dz, part, rows, D, group)
    if (need <= 1) GN_CASE(1); else if (need <= 2) GN_CASE(2); else if (need <= 4) GN_CASE(4); else if (need <= 5) GN_CASE(5); else GN_CASE(8);
#undef GN_CASE
    return cudaGetLastError();
}

cudaError_t launch_gated_norm_fwd(int dtype, const void *y, const void *z, const float *gamma, float eps, void *out,
                                  long long rows, int D, int group, cudaStream_t st) {
    if (dtype == SSD_DTYPE_F32) return norm_fwd_t<float>((const float *)y, (const float *)z, gamma, eps, (float *)out, rows, D, group, st);
    return norm_fwd_t<__nv_bfloat16>((const __nv_bfloat16 *)y, (const __nv_bfloat16 *)z, gamma, eps, (__nv_bfloat16 *)out, rows, D,
                                     group, st);
}

cudaError_t launch_gated_norm_bwd(int dtype, const void *y, const void *z, const float *gamma, float eps, const void *dout,
                                  void *dy, void *dz, float *dgamma, int accumulate, float *part, long long rows, int D,
                                  int group, cudaStream_t st) {
    cudaError_t e;
    if (dtype == SSD_DTYPE_F32)
        e = norm_bwd_t<float>((const float *)y, (const float *)z, gamma, eps, (const float *)dout, (float *)dy, (float *)dz, part,
                              rows, D, group, st);
    else
        e = norm_bwd_t<__nv_bfloat16>((const __nv_bfloat16 *)y, (const __nv_bfloat16 *)z, gamma, eps, (const __nv_bfloat16 *)dout,
                                      (__nv_bfloat16 *)dy, (__nv_bfloat16 *)dz, part, rows, D, group, st);
    if (e != cudaSuccess) return e;
    k_gated_norm_reduce<<<(D + 31) / 32, 256, 0, st>>>(part, dgamma, D, (int)gated_norm_tiles(rows), accumulate);
    return cudaGetLastError();
}

}  // namespace ssd
