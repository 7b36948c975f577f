// Plain convolution on CUDA cores with the same fused epilogue as the tensor-core path
// (folded-BN bias, residual operand, ReLU) on the planar-8 layout.  Validation only: one
// thread per output vector (8 filters of one output position, border positions included and
// written as zeros), fp32 accumulation, no tensor cores.  T = float is the fp32 validation
// path; T = bf16 reads and writes the tensor-core path's storage.
#include "fp_internal.h"

namespace fp {

namespace {

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
    const int Wp = a.W + 2, P2i = (a.H + 2) * Wp, Qp = a.Q + 2, P2o = (a.P + 2) * Qp;
    const size_t plane_i = (size_t)a.N * P2i, plane_o = (size_t)a.N * P2o;
    const int kchunks = a.K_pad / 8, cchunks = a.C_pad / 8;
    const size_t total = plane_o * kchunks;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int jo = (int)(i / plane_o);
        const size_t f = i - (size_t)jo * plane_o;
        const size_t n = f / P2o;
        const int rem = (int)(f - n * P2o);
        const int p = rem / Qp - 1, q = rem % Qp - 1;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
        const bool inside = p >= 0 && p < a.P && q >= 0 && q < a.Q;
        if (inside) {
            for (int r = 0; r < a.R; ++r) {
                const int ih = p * a.stride + r - a.pad;
                if (ih < 0 || ih >= a.H) continue;
                for (int s = 0; s < a.S; ++s) {
                    const int iw = q * a.stride + s - a.pad;
                    if (iw < 0 || iw >= a.W) continue;
                    const int tap = r * a.S + s;
                    for (int jc = 0; jc < cchunks; ++jc) {
                        const T* xp = x + ((size_t)jc * plane_i + n * P2i + (size_t)(ih + 1) * Wp + (iw + 1)) * 8;
                        const T* wp = w + (((size_t)tap * cchunks + jc) * a.K_pad + (size_t)jo * 8) * 8;
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            float sum = acc[e];
#pragma unroll
                            for (int c = 0; c < 8; ++c) sum = fmaf(to_f<T>(xp[c]), to_f<T>(wp[e * 8 + c]), sum);
                            acc[e] = sum;
                        }
                    }
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int k = jo * 8 + e;
                float v = acc[e] + a.bias[k];
                if (a.res_mode == 1) {
                    v += to_f<T>(res[i * 8 + e]);
                } else if (a.res_mode == 2) {
                    const int c = k - a.res_pad_lo;
                    if (c >= 0 && c < a.res_C) {
                        const int rWp = a.res_W + 2, rP2 = (a.res_H + 2) * rWp;
                        const size_t rv = (size_t)(c / 8) * a.N * rP2 + n * rP2 + (size_t)(p * a.res_stride + 1) * rWp +
                                          (q * a.res_stride + 1);
                        v += to_f<T>(res[rv * 8 + (c & 7)]);
                    }
                }
                acc[e] = a.relu ? fmaxf(v, 0.0f) : v;
            }
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) y[i * 8 + e] = from_f<T>(acc[e]);
    }
}

}  // namespace

void launch_conv_simt(const ConvArgs& a, int is_bf16, cudaStream_t st) {
    const size_t total = (size_t)a.N * (a.P + 2) * (a.Q + 2) * (a.K_pad / 8);
    size_t blocks = (total + 255) / 256;
    const size_t cap = (size_t)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (is_bf16) conv_simt_kernel<__nv_bfloat16><<<(int)blocks, 256, 0, st>>>(a);
    else conv_simt_kernel<float><<<(int)blocks, 256, 0, st>>>(a);
}

}  // namespace fp
