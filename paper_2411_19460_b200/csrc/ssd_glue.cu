// Layer-axis glue for a stack of SSD layers under Multi-Axis Gradient Checkpointing (Algorithms 1
// and 2 of the paper keep only each layer's INPUT along the layer axis): layer j maps x_j to
// y_j = SSD_j(x_j) and hands x_{j+1} = W (y_j + x_j) to the next layer, W a fixed P x P mixing matrix
// applied per (batch, step, head).  Backward: dz = W^T g_{j+1}; dy_j = dz; dx_j = (SSD backward) + dz.
// Bandwidth-shaped kernels; bf16 or fp32 I/O.  fp32: CUDA cores, fp32 arithmetic.  bf16: the 64 x 64 product runs on
// the tensor cores through warp-level mma (W rounded to bf16 once per CTA, fp32 accumulation): at 4096 multiply-adds
// per 128-byte row the CUDA-core version was five times over its memory time.
#include <mma.h>

#include "ssd_internal.h"

namespace ssd {

namespace {

template <typename T> __device__ __forceinline__ void load_row64(const T *src, float *z);
template <> __device__ __forceinline__ void load_row64<float>(const float *src, float *z) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(src) + k);
        z[4 * k] = v.x; z[4 * k + 1] = v.y; z[4 * k + 2] = v.z; z[4 * k + 3] = v.w;
    }
}
template <> __device__ __forceinline__ void load_row64<__nv_bfloat16>(const __nv_bfloat16 *src, float *z) {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(src) + k);
        const __nv_bfloat162 *e = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(e[i]);
            z[8 * k + 2 * i] = f.x;
            z[8 * k + 2 * i + 1] = f.y;
        }
    }
}
template <typename T> __device__ __forceinline__ void store4(T *dst, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float *dst, float a, float b, float c, float d) {
    *reinterpret_cast<float4 *>(dst) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16 *dst, float a, float b, float c, float d) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 pk;
    pk.x = *reinterpret_cast<unsigned int *>(&lo);
    pk.y = *reinterpret_cast<unsigned int *>(&hi);
    *reinterpret_cast<uint2 *>(dst) = pk;
}

// out[row, i] = sum_j M[i][j] (a[row, j] + b[row, j])   with M = W (TRANSPOSE = false) or W^T (true);
// b may be null.  One thread per 64-vector; M is staged in shared memory as Mt[j][i] so that four
// consecutive outputs come from one broadcast 16-byte read.
template <typename T, bool TRANSPOSE>
__global__ void __launch_bounds__(128) k_glue(const T *a, const T *b, const float *W, T *out, long long rows_per_batch,
                                              long long bstride, int B) {
    __shared__ float Mt[64][64];
    for (int idx = threadIdx.x; idx < 4096; idx += 128) {
        const int r = idx >> 6, cidx = idx & 63;            // W[r][cidx]
        if (TRANSPOSE) Mt[r][cidx] = W[idx];                // M = W^T: M[i][j] = W[j][i] -> Mt[j][i] = W[j][i]
        else Mt[cidx][r] = W[idx];                          // M = W  : Mt[j][i] = W[i][j]
    }
    __syncthreads();
    const long long total = rows_per_batch * B;
    for (long long row = (long long)blockIdx.x * 128 + threadIdx.x; row < total; row += (long long)gridDim.x * 128) {
        const long long bb = row / rows_per_batch, rr = row % rows_per_batch;
        const size_t off = (size_t)bb * bstride + (size_t)rr * 64;
        float z[64];
        load_row64(a + off, z);
        if (b) {
            float zb[64];
            load_row64(b + off, zb);
#pragma unroll
            for (int j = 0; j < 64; ++j) z[j] += zb[j];
        }
#pragma unroll 2
        for (int i0 = 0; i0 < 64; i0 += 4) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                const float4 m = *reinterpret_cast<const float4 *>(&Mt[j][i0]);
                acc.x = fmaf(m.x, z[j], acc.x);
                acc.y = fmaf(m.y, z[j], acc.y);
                acc.z = fmaf(m.z, z[j], acc.z);
                acc.w = fmaf(m.w, z[j], acc.w);
            }
            store4(out + off + i0, acc.x, acc.y, acc.z, acc.w);
        }
    }
}

// The same product for bf16 rows on the tensor cores.  A warp owns 16 consecutive rows (one contiguous 2 KB block of
// the row-major [rows][64] tensor): it fetches them with 16-byte loads that cover whole 512-byte spans per instruction,
// forms Z = a (+ b) in bf16 and parks it in a padded shared-memory tile, multiplies it by the bf16 copy of W with
// 4 x 4 warp-level mma steps (fp32 accumulation), and sends the 16 result rows out the same way, through a padded
// fp32 staging tile.  Row strides of 72 elements keep the fragment accesses off one bank.
constexpr int GL_LD = 72;
template <bool TRANSPOSE>
__global__ void __launch_bounds__(128) k_glue_bf16_mma(const __nv_bfloat16 *a, const __nv_bfloat16 *b, const float *W,
                                                       __nv_bfloat16 *out, long long rows_per_batch, long long bstride, int B) {
    using namespace nvcuda;
    __shared__ __align__(32) __nv_bfloat16 Wb[64 * GL_LD];
    __shared__ __align__(32) __nv_bfloat16 zs[4][16 * GL_LD];
    __shared__ __align__(32) float stage[4][16 * GL_LD];
    for (int idx = threadIdx.x; idx < 4096; idx += 128) Wb[(idx >> 6) * GL_LD + (idx & 63)] = __float2bfloat16_rn(W[idx]);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long ntiles = rows_per_batch * B / 16;
    auto tile_offset = [&](long long t) {
        const long long row0 = t * 16, bb = row0 / rows_per_batch, rr = row0 % rows_per_batch;
        return (size_t)bb * bstride + (size_t)rr * 64;
    };
    // 16-byte chunk c of a tile's block (128 of them): row c / 8, columns (c % 8) * 8 ..; the next tile's rows are
    // requested as soon as the current ones have been parked in shared memory
    uint4 va[4], vb[4];
    auto fetch = [&](size_t off) {
#pragma unroll
        for (int q = 0; q < 4; ++q) va[q] = __ldg(reinterpret_cast<const uint4 *>(a + off) + q * 32 + lane);
        if (b) {
#pragma unroll
            for (int q = 0; q < 4; ++q) vb[q] = __ldg(reinterpret_cast<const uint4 *>(b + off) + q * 32 + lane);
        }
    };
    const long long t_first = (long long)blockIdx.x * 4 + warp, t_step = (long long)gridDim.x * 4;
    if (t_first < ntiles) fetch(tile_offset(t_first));
    for (long long t = t_first; t < ntiles; t += t_step) {
        const size_t off = tile_offset(t);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint4 z = va[q];
            if (b) {
                __nv_bfloat162 *zp = reinterpret_cast<__nv_bfloat162 *>(&z);
                const __nv_bfloat162 *bp = reinterpret_cast<const __nv_bfloat162 *>(&vb[q]);
#pragma unroll
                for (int i = 0; i < 4; ++i) zp[i] = __hadd2(zp[i], bp[i]);
            }
            const int c = q * 32 + lane;
            *reinterpret_cast<uint4 *>(&zs[warp][(c >> 3) * GL_LD + (c & 7) * 8]) = z;
        }
        if (t + t_step < ntiles) fetch(tile_offset(t + t_step));
        __syncwarp();
        wmma::fragment<wmma::matrix_a, 16, 16, 16, __nv_bfloat16, wmma::row_major> za[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) wmma::load_matrix_sync(za[k], zs[warp] + k * 16, GL_LD);
        // out[row, i] = sum_j M[i][j] z[j]: the B operand is element (k = j, n = i) = M[i][j].  M = W: W[n][k], i.e. W
        // read column-major; M = W^T: W[k][n], row-major.
#pragma unroll
        for (int n = 0; n < 4; ++n) {
            wmma::fragment<wmma::accumulator, 16, 16, 16, float> acc;
            wmma::fill_fragment(acc, 0.f);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (TRANSPOSE) {
                    wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::row_major> mb;
                    wmma::load_matrix_sync(mb, Wb + (k * 16) * GL_LD + n * 16, GL_LD);
                    wmma::mma_sync(acc, za[k], mb, acc);
                } else {
                    wmma::fragment<wmma::matrix_b, 16, 16, 16, __nv_bfloat16, wmma::col_major> mb;
                    wmma::load_matrix_sync(mb, Wb + (n * 16) * GL_LD + k * 16, GL_LD);
                    wmma::mma_sync(acc, za[k], mb, acc);
                }
            }
            wmma::store_matrix_sync(stage[warp] + n * 16, acc, GL_LD, wmma::mem_row_major);
        }
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int c = q * 32 + lane;
            const float *src = stage[warp] + (c >> 3) * GL_LD + (c & 7) * 8;
            const float4 v0 = *reinterpret_cast<const float4 *>(src), v1 = *reinterpret_cast<const float4 *>(src + 4);
            __nv_bfloat162 p0 = __floats2bfloat162_rn(v0.x, v0.y), p1 = __floats2bfloat162_rn(v0.z, v0.w);
            __nv_bfloat162 p2 = __floats2bfloat162_rn(v1.x, v1.y), p3 = __floats2bfloat162_rn(v1.z, v1.w);
            uint4 pk;
            pk.x = *reinterpret_cast<unsigned int *>(&p0);
            pk.y = *reinterpret_cast<unsigned int *>(&p1);
            pk.z = *reinterpret_cast<unsigned int *>(&p2);
            pk.w = *reinterpret_cast<unsigned int *>(&p3);
            *(reinterpret_cast<uint4 *>(out + off) + c) = pk;
        }
        __syncwarp();      // both tiles are reused by the warp's next 16 rows
    }
}

// dst += src, elementwise over [B][rows_per_batch * 64]
template <typename T>
__global__ void __launch_bounds__(256) k_residual(T *dst, const T *src, long long n_per_batch, long long bstride, int B) {
    const long long total = n_per_batch * B / 4;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
        const long long e = i * 4, bb = e / n_per_batch, rr = e % n_per_batch;
        const size_t off = (size_t)bb * bstride + (size_t)rr;
        float d[4], s[4];
        if (sizeof(T) == 4) {
            const float4 dv = *reinterpret_cast<const float4 *>(dst + off), sv = *reinterpret_cast<const float4 *>(src + off);
            d[0] = dv.x; d[1] = dv.y; d[2] = dv.z; d[3] = dv.w;
            s[0] = sv.x; s[1] = sv.y; s[2] = sv.z; s[3] = sv.w;
        } else {
            const uint2 dv = *reinterpret_cast<const uint2 *>(dst + off), sv = *reinterpret_cast<const uint2 *>(src + off);
            const float2 d0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&dv.x));
            const float2 d1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&dv.y));
            const float2 s0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&sv.x));
            const float2 s1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&sv.y));
            d[0] = d0.x; d[1] = d0.y; d[2] = d1.x; d[3] = d1.y;
            s[0] = s0.x; s[1] = s0.y; s[2] = s1.x; s[3] = s1.y;
        }
        store4(dst + off, d[0] + s[0], d[1] + s[1], d[2] + s[2], d[3] + s[3]);
    }
}

}  // namespace

cudaError_t launch_glue(int dtype, bool transpose, const void *a, const void *b, const float *W, void *out,
                        long long rows_per_batch, long long bstride, int B, cudaStream_t st) {
    const long long total = rows_per_batch * B;
    const unsigned blocks = (unsigned)((total + 127) / 128 < 148 * 16 ? (total + 127) / 128 : 148 * 16);
    if (dtype == SSD_DTYPE_F32) {
        if (transpose) k_glue<float, true><<<blocks, 128, 0, st>>>((const float *)a, (const float *)b, W, (float *)out, rows_per_batch, bstride, B);
        else k_glue<float, false><<<blocks, 128, 0, st>>>((const float *)a, (const float *)b, W, (float *)out, rows_per_batch, bstride, B);
    } else if (rows_per_batch % 16 == 0) {
        const long long tiles = total / 16;
        const unsigned mblocks = (unsigned)((tiles + 3) / 4 < 148 * 6 ? (tiles + 3) / 4 : 148 * 6);   // six 37 KB CTAs fit an SM: one wave
        if (transpose) k_glue_bf16_mma<true><<<mblocks, 128, 0, st>>>((const __nv_bfloat16 *)a, (const __nv_bfloat16 *)b, W, (__nv_bfloat16 *)out, rows_per_batch, bstride, B);
        else k_glue_bf16_mma<false><<<mblocks, 128, 0, st>>>((const __nv_bfloat16 *)a, (const __nv_bfloat16 *)b, W, (__nv_bfloat16 *)out, rows_per_batch, bstride, B);
    } else {
        if (transpose) k_glue<__nv_bfloat16, true><<<blocks, 128, 0, st>>>((const __nv_bfloat16 *)a, (const __nv_bfloat16 *)b, W, (__nv_bfloat16 *)out, rows_per_batch, bstride, B);
        else k_glue<__nv_bfloat16, false><<<blocks, 128, 0, st>>>((const __nv_bfloat16 *)a, (const __nv_bfloat16 *)b, W, (__nv_bfloat16 *)out, rows_per_batch, bstride, B);
    }
    return cudaGetLastError();
}

cudaError_t launch_residual(int dtype, void *dst, const void *src, long long n_per_batch, long long bstride, int B,
                            cudaStream_t st) {
    const long long total = n_per_batch * B / 4;
    const unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 32 ? (total + 255) / 256 : 148 * 32);
    if (dtype == SSD_DTYPE_F32) k_residual<float><<<blocks, 256, 0, st>>>((float *)dst, (const float *)src, n_per_batch, bstride, B);
    else k_residual<__nv_bfloat16><<<blocks, 256, 0, st>>>((__nv_bfloat16 *)dst, (const __nv_bfloat16 *)src, n_per_batch, bstride, B);
    return cudaGetLastError();
}

}  // namespace ssd
