// Plain convolution on CUDA cores with the same fused epilogue as the tensor-core path
// (folded-BN bias, residual operand, ReLU).  Validation only: one thread per four output
// channels of one output pixel, fp32 accumulation, no tensor cores.  T = float gives the
// fp32 validation path; T = bf16 reads and writes the tensor-core path's storage.
#include "fp_internal.h"

namespace fp {

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T>
__global__ void conv_simt_kernel(ConvArgs a) {
    const T* __restrict__ x = (const T*)a.x;
    const T* __restrict__ w = (const T*)a.w;
    const T* __restrict__ res = (const T*)a.res;
    T* __restrict__ y = (T*)a.y;
    const int kq = a.K_pad / 4;
    const size_t total = (size_t)a.N * a.P * a.Q * kq;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int k4 = (int)(i % kq) * 4;
        size_t t = i / kq;
        const int q = (int)(t % a.Q); t /= a.Q;
        const int p = (int)(t % a.P);
        const size_t n = t / a.P;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int r = 0; r < a.R; ++r) {
            const int ih = p * a.stride + r - a.pad;
            if (ih < 0 || ih >= a.H) continue;
            for (int s = 0; s < a.S; ++s) {
                const int iw = q * a.stride + s - a.pad;
                if (iw < 0 || iw >= a.W) continue;
                const T* xp = x + ((n * a.H + ih) * a.W + iw) * a.C_pad;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const T* wp = w + (((size_t)(k4 + j) * a.R + r) * a.S + s) * a.C_pad;
                    float sum = acc[j];
                    for (int c = 0; c < a.C_pad; ++c) sum = fmaf(to_f<T>(xp[c]), to_f<T>(wp[c]), sum);
                    acc[j] = sum;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = k4 + j;
            float v = acc[j] + a.bias[k];
            if (a.res_mode == 1) {
                v += to_f<T>(res[((n * a.P + p) * a.Q + q) * a.K_pad + k]);
            } else if (a.res_mode == 2) {
                const int c = k - a.res_pad_lo;
                if (c >= 0 && c < a.res_C)
                    v += to_f<T>(res[((n * a.res_H + p * a.res_stride) * a.res_W + q * a.res_stride) * a.res_C_pad + c]);
            }
            y[((n * a.P + p) * a.Q + q) * a.K_pad + k] = from_f<T>(a.relu ? fmaxf(v, 0.0f) : v);
        }
    }
}

void launch_conv_simt(const ConvArgs& a, int is_bf16, cudaStream_t st) {
    const size_t total = (size_t)a.N * a.P * a.Q * (a.K_pad / 4);
    size_t blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (blocks < 1) blocks = 1;
    if (is_bf16) conv_simt_kernel<__nv_bfloat16><<<(int)blocks, 256, 0, st>>>(a);
    else conv_simt_kernel<float><<<(int)blocks, 256, 0, st>>>(a);
}

}  // namespace fp
