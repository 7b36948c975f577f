// Memory-bound operators of the fused graph: boundary layout conversion, max pooling,
// the global-average-pool + FC head, and a debug dump.  Activations are NHWC with the
// channel count padded to a multiple of 16; padded channels always hold zeros.
#include "fp_internal.h"

namespace fp {

__device__ __forceinline__ float ld_act(const void* p, size_t i, int is_bf16) {
    return is_bf16 ? __bfloat162float(((const __nv_bfloat16*)p)[i]) : ((const float*)p)[i];
}

// NCHW (fp32 or bf16) -> NHWC (bf16 or fp32), channels zero-padded to C_pad.
// One thread per output pixel writes its C_pad channels with 16-byte stores; reads are
// coalesced across pixels for every channel plane.
template <typename OutT, int CP>
__global__ void input_to_nhwc_kernel(const void* __restrict__ in, int in_is_bf16, OutT* __restrict__ out, int N, int C,
                                     int HW) {
    const size_t total = (size_t)N * HW;
    for (size_t pix = blockIdx.x * (size_t)blockDim.x + threadIdx.x; pix < total;
         pix += (size_t)gridDim.x * blockDim.x) {
        const size_t n = pix / HW, hw = pix - n * HW;
        __align__(16) OutT v[CP];
#pragma unroll
        for (int c = 0; c < CP; ++c) {
            float f = 0.0f;
            if (c < C) f = ld_act(in, (n * C + c) * HW + hw, in_is_bf16);
            if constexpr (sizeof(OutT) == 2) v[c] = __float2bfloat16_rn(f); else v[c] = f;
        }
        uint4* dst = reinterpret_cast<uint4*>(out + pix * CP);
        const uint4* src = reinterpret_cast<const uint4*>(v);
#pragma unroll
        for (int i = 0; i < (int)(CP * sizeof(OutT) / 16); ++i) dst[i] = src[i];
    }
}

__global__ void input_to_nhwc_generic_kernel(const void* __restrict__ in, int in_is_bf16, void* __restrict__ out,
                                             int out_is_bf16, int N, int C, int HW, int C_pad) {
    const size_t total = (size_t)N * HW * C_pad;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % C_pad);
        const size_t pix = i / C_pad;
        const size_t n = pix / HW, hw = pix - n * HW;
        const float f = c < C ? ld_act(in, (n * C + c) * HW + hw, in_is_bf16) : 0.0f;
        if (out_is_bf16) ((__nv_bfloat16*)out)[i] = __float2bfloat16_rn(f); else ((float*)out)[i] = f;
    }
}

// Max pooling over NHWC, 8 channels (16 bytes of bf16) or 4 channels (16 bytes of fp32) per thread.
template <bool BF16>
__global__ void maxpool_kernel(const void* __restrict__ x, void* __restrict__ y, int N, int H, int W, int C_pad, int P,
                               int Q, int R, int stride, int pad) {
    constexpr int V = BF16 ? 8 : 4;
    const int cv = C_pad / V;
    const size_t total = (size_t)N * P * Q * cv;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % cv);
        size_t t = i / cv;
        const int q = (int)(t % Q); t /= Q;
        const int p = (int)(t % P);
        const size_t n = t / P;
        float m[V];
#pragma unroll
        for (int j = 0; j < V; ++j) m[j] = -INFINITY;
        for (int r = 0; r < R; ++r) {
            const int ih = p * stride + r - pad;
            if (ih < 0 || ih >= H) continue;
            for (int s = 0; s < R; ++s) {
                const int iw = q * stride + s - pad;
                if (iw < 0 || iw >= W) continue;
                const size_t off = ((n * H + ih) * W + iw) * C_pad + (size_t)c * V;
                const uint4 raw = *reinterpret_cast<const uint4*>(
                    BF16 ? (const void*)((const __nv_bfloat16*)x + off) : (const void*)((const float*)x + off));
                if constexpr (BF16) {
                    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 f = __bfloat1622float2(h2[j]);
                        m[2 * j] = fmaxf(m[2 * j], f.x);
                        m[2 * j + 1] = fmaxf(m[2 * j + 1], f.y);
                    }
                } else {
                    const float* f = reinterpret_cast<const float*>(&raw);
#pragma unroll
                    for (int j = 0; j < 4; ++j) m[j] = fmaxf(m[j], f[j]);
                }
            }
        }
        const size_t o = ((n * P + p) * Q + q) * C_pad + (size_t)c * V;
        if constexpr (BF16) {
            uint4 outv;
            __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&outv);
#pragma unroll
            for (int j = 0; j < 4; ++j) h2[j] = __floats2bfloat162_rn(m[2 * j], m[2 * j + 1]);
            *reinterpret_cast<uint4*>((__nv_bfloat16*)y + o) = outv;
        } else {
            *reinterpret_cast<float4*>((float*)y + o) = make_float4(m[0], m[1], m[2], m[3]);
        }
    }
}

// Head: spatial sum per channel (fp32), then logits[k] = sum_c s[c] * Wfc[k][c] + b[k] with the
// 1/(H*W) of the average already folded into Wfc.  One block per image; the channel sums live in
// shared memory; one warp per class row with a shuffle reduction.
__global__ void head_kernel(const void* __restrict__ x, int is_bf16, int HW, int C_pad, const float* __restrict__ fcw,
                            const float* __restrict__ fcb, int n_classes, float* __restrict__ logits) {
    extern __shared__ float sums[];
    const size_t n = blockIdx.x;
    for (int c = threadIdx.x; c < C_pad; c += blockDim.x) {
        float s = 0.0f;
        for (int i = 0; i < HW; ++i) s += ld_act(x, (n * HW + i) * C_pad + c, is_bf16);
        sums[c] = s;
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    for (int k = warp; k < n_classes; k += nwarps) {
        const float* wr = fcw + (size_t)k * C_pad;
        float s = 0.0f;
        for (int c = lane; c < C_pad; c += 32) s = fmaf(sums[c], wr[c], s);
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
        if (lane == 0) logits[n * n_classes + k] = s + fcb[k];
    }
}

__global__ void nhwc_to_nchw_f32_kernel(const void* __restrict__ x, int is_bf16, float* __restrict__ out, int N, int HW,
                                        int C_pad, const int32_t* __restrict__ chan_dst, int C_out) {
    const size_t total = (size_t)N * HW * C_pad;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % C_pad);
        const size_t pix = i / C_pad;
        const size_t n = pix / HW, hw = pix - n * HW;
        const int cd = chan_dst[c];
        if (cd >= 0) out[(n * C_out + cd) * HW + hw] = ld_act(x, i, is_bf16);
    }
}

static inline int grid_for(size_t n, int threads) {
    size_t b = (n + threads - 1) / threads;
    const size_t cap = 148 * 16;
    if (b < 1) b = 1;
    return (int)(b > cap ? cap : b);
}

void launch_input_to_nhwc(const void* in, int in_is_bf16, void* out, int out_is_bf16, int N, int C, int H, int W,
                          int C_pad, cudaStream_t st) {
    const int HW = H * W;
    const size_t pix = (size_t)N * HW;
    if (C_pad == 16 && out_is_bf16) {
        input_to_nhwc_kernel<__nv_bfloat16, 16><<<grid_for(pix, 256), 256, 0, st>>>(in, in_is_bf16, (__nv_bfloat16*)out, N, C, HW);
    } else if (C_pad == 16) {
        input_to_nhwc_kernel<float, 16><<<grid_for(pix, 256), 256, 0, st>>>(in, in_is_bf16, (float*)out, N, C, HW);
    } else {
        input_to_nhwc_generic_kernel<<<grid_for(pix * C_pad, 256), 256, 0, st>>>(in, in_is_bf16, out, out_is_bf16, N, C, HW, C_pad);
    }
}

void launch_maxpool(const void* x, void* y, int is_bf16, int N, int H, int W, int C_pad, int P, int Q, int R,
                    int stride, int pad, cudaStream_t st) {
    const size_t n = (size_t)N * P * Q * (C_pad / (is_bf16 ? 8 : 4));
    if (is_bf16) maxpool_kernel<true><<<grid_for(n, 256), 256, 0, st>>>(x, y, N, H, W, C_pad, P, Q, R, stride, pad);
    else maxpool_kernel<false><<<grid_for(n, 256), 256, 0, st>>>(x, y, N, H, W, C_pad, P, Q, R, stride, pad);
}

void launch_head(const void* x, int is_bf16, int N, int HW, int C_pad, const float* fcw, const float* fcb,
                 int n_classes, float* logits, cudaStream_t st) {
    head_kernel<<<N, 256, (size_t)C_pad * sizeof(float), st>>>(x, is_bf16, HW, C_pad, fcw, fcb, n_classes, logits);
}

void launch_nhwc_to_nchw_f32(const void* x, int is_bf16, float* out, int N, int H, int W, int C_pad,
                             const int32_t* chan_dst, int C_out, cudaStream_t st) {
    const size_t n = (size_t)N * H * W * C_pad;
    nhwc_to_nchw_f32_kernel<<<grid_for(n, 256), 256, 0, st>>>(x, is_bf16, out, N, H * W, C_pad, chan_dst, C_out);
}

}  // namespace fp
