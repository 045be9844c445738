// One step of the recurrence of Eq. 1 for autoregressive decoding / forward-only streaming: the state
// is the only thing carried between tokens, so memory does not grow with the sequence.
//     h <- exp(dt A_h) h + dt x B^T ,   y = C h + D_h x          per (batch, head)
// Bandwidth-shaped: the fp32 state is read and written once; one warp owns one row h[b,h,p,:] (N values,
// 16-byte accesses, consecutive warps on consecutive rows), and reduces y[b,h,p] with shuffles.
#include "ssd_internal.h"

namespace ssd {

namespace {

template <typename T> __device__ __forceinline__ float ldf(const T *p);
template <> __device__ __forceinline__ float ldf<float>(const float *p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T *p, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// rows = B*H*P; N = 32 * NV * 4 is not required: each lane owns N/32 consecutive values (NV = N/32 in {2,4}).
template <typename T, int NV>
__global__ void __launch_bounds__(256) k_decode_step(const T *x, const float *dt, const float *A, const T *Bm,
                                                     const T *Cm, const float *D, float *h, T *y, int B, int H,
                                                     int P, int G, long long x_bs, long long dt_bs, long long bc_bs) {
    constexpr int N = 32 * NV;
    const int lane = threadIdx.x & 31;
    const long long rows = (long long)B * H * P;
    const int hpg = H / G;
    for (long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5); row < rows; row += (long long)gridDim.x * 8) {
        const int p = (int)(row % P);
        const int hh = (int)((row / P) % H);
        const int b = (int)(row / ((long long)P * H));
        const float dtv = __ldg(dt + (size_t)b * dt_bs + hh);
        const float decay = expf(dtv * __ldg(A + hh));
        const float xv = ldf(x + (size_t)b * x_bs + (size_t)hh * P + p);
        const float dx = dtv * xv;
        const T *Bp = Bm + (size_t)b * bc_bs + (size_t)(hh / hpg) * N + lane * NV;
        const T *Cp = Cm + (size_t)b * bc_bs + (size_t)(hh / hpg) * N + lane * NV;
        float *hp = h + (size_t)row * N + lane * NV;
        float hv[NV];
        if (NV == 4) {
            const float4 v = *reinterpret_cast<const float4 *>(hp);
            hv[0] = v.x; hv[1] = v.y; hv[NV - 2] = v.z; hv[NV - 1] = v.w;
        } else {
            const float2 v = *reinterpret_cast<const float2 *>(hp);
            hv[0] = v.x; hv[1] = v.y;
        }
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            hv[i] = fmaf(hv[i], decay, dx * ldf(Bp + i));
            acc = fmaf(ldf(Cp + i), hv[i], acc);
        }
        if (NV == 4) *reinterpret_cast<float4 *>(hp) = make_float4(hv[0], hv[1], hv[NV - 2], hv[NV - 1]);
        else *reinterpret_cast<float2 *>(hp) = make_float2(hv[0], hv[1]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) stf(y + (size_t)b * x_bs + (size_t)hh * P + p, fmaf(__ldg(D + hh), xv, acc));
    }
}

}  // namespace

cudaError_t launch_decode_step(int dtype, int N, const void *x, const float *dt, const float *A, const void *Bm,
                               const void *Cm, const float *D, float *h, void *y, int B, int H, int P, int G,
                               long long x_bs, long long dt_bs, long long bc_bs, cudaStream_t st) {
    const long long rows = (long long)B * H * P;
    const unsigned blocks = (unsigned)((rows + 7) / 8 < 148 * 64 ? (rows + 7) / 8 : 148 * 64);
#define SSD_DECODE_CASE(T, NV)                                                                                  \
    k_decode_step<T, NV><<<blocks, 256, 0, st>>>((const T *)x, dt, A, (const T *)Bm, (const T *)Cm, D, h, (T *)y, \
                                                 B, H, P, G, x_bs, dt_bs, bc_bs)
    if (dtype == SSD_DTYPE_F32) {
        if (N == 128) SSD_DECODE_CASE(float, 4); else SSD_DECODE_CASE(float, 2);
    } else {
        if (N == 128) SSD_DECODE_CASE(__nv_bfloat16, 4); else SSD_DECODE_CASE(__nv_bfloat16, 2);
    }
#undef SSD_DECODE_CASE
    return cudaGetLastError();
}

}  // namespace ssd
