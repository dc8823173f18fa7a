// Debug reference kernels: one thread per output element, no tiling, no tensor cores.
// They exist so that the tensor-core path can be cross-checked on the GPU at sizes the CPU
// oracle cannot reach; asx_run selects them only with ASX_IMPL_NAIVE and never falls back to
// them.  They compute the same definition (Section 3.2): kept rows get act(conv + bias),
// dropped rows get zeros (Algorithm 2, post-processing).
#include <cuda_bf16.h>
#include "asx_internal.h"

namespace asx {

namespace {

// Element types: bf16 (the default storage) or fp32 (ASX_F32; products of the fp32 values as they
// are, not of their TF32 parts).
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ void from_f32(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
__device__ __forceinline__ void from_f32(float* p, float v) { *p = v; }

template <typename T>
__global__ void naive_zero_dropped(ConvGeom g, T* __restrict__ y,
                                   const uint8_t* __restrict__ mask)
{
    const long long total = (long long)g.M * g.C_out;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int row = (int)(i / g.C_out);
        const int p = (g.rows == g.P) ? row % g.P : row;
        if (mask[p] == 0) from_f32(y + i, 0.f);
    }
}

template <typename T>
__global__ void naive_kept_rows(ConvGeom g, const T* __restrict__ x,
                                const T* __restrict__ w, const float* __restrict__ bias,
                                T* __restrict__ y, const int32_t* __restrict__ kept,
                                const int32_t* __restrict__ count, int relu)
{
    const int cnt = *count;
    const long long Mk = (g.rows == g.P) ? (long long)g.Nb * cnt : cnt;
    const long long total = Mk * g.C_out;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int rk = (int)(i / g.C_out);
        const int co = (int)(i - (long long)rk * g.C_out);
        int row;
        if (g.rows == g.P) {
            const int n = rk / cnt;
            row = n * g.P + kept[rk - n * cnt];
        } else {
            row = kept[rk];
        }
        const int n = row / g.P, p = row - n * g.P;
        const int oy = p / g.Wo, ox = p - oy * g.Wo;
        float acc = 0.f;
        for (int ky = 0; ky < g.kh; ++ky) {
            const int iy = oy * g.stride - g.pad + ky;
            if (iy < 0 || iy >= g.H) continue;
            for (int kx = 0; kx < g.kw; ++kx) {
                const int ix = ox * g.stride - g.pad + kx;
                if (ix < 0 || ix >= g.W) continue;
                const T* xp = x + (((long long)n * g.H + iy) * g.W + ix) * g.C_in;
                const T* wp = w + (((long long)co * g.kh + ky) * g.kw + kx) * g.C_in;
                for (int ci = 0; ci < g.C_in; ++ci)
                    acc = fmaf(to_f32(xp[ci]), to_f32(wp[ci]), acc);
            }
        }
        float v = acc + (bias ? bias[co] : 0.f);
        if (relu == 1) v = fmaxf(v, 0.f);
        if (relu == 2) v = v / (1.f + expf(-v));     // SiLU
        from_f32(y + (long long)row * g.C_out + co, v);
    }
}

}  // namespace

cudaError_t launch_naive(const ConvGeom& g, const void* x, const void* w, const float* bias, void* y,
                         const uint8_t* mask, const int32_t* kept, const int32_t* count, int relu, int f32,
                         cudaStream_t st)
{
    const long long total = (long long)g.M * g.C_out;
    int blocks = (int)((total + 255) / 256 < 148 * 32 ? (total + 255) / 256 : 148 * 32);
    if (blocks < 1) blocks = 1;
    if (f32) {
        naive_zero_dropped<float><<<blocks, 256, 0, st>>>(g, static_cast<float*>(y), mask);
        naive_kept_rows<float><<<blocks, 256, 0, st>>>(g, static_cast<const float*>(x), static_cast<const float*>(w), bias,
                                                       static_cast<float*>(y), kept, count, relu);
        return cudaGetLastError();
    }
    naive_zero_dropped<<<blocks, 256, 0, st>>>(g, static_cast<__nv_bfloat16*>(y), mask);
    naive_kept_rows<<<blocks, 256, 0, st>>>(g, static_cast<const __nv_bfloat16*>(x),
                                            static_cast<const __nv_bfloat16*>(w), bias,
                                            static_cast<__nv_bfloat16*>(y), kept, count, relu);
    return cudaGetLastError();
}

}  // namespace asx
