// Internal declarations shared by the host graph builder and the kernel launchers.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

namespace fp {

// ---------------------------------------------------------------------------------------
// Convolution launch description (one fused operator: conv + bias + residual + ReLU)
// ---------------------------------------------------------------------------------------
struct ConvArgs {
    const void* x;        // NHWC activations [N][H][W][C_pad]   (bf16 or fp32)
    void* y;              // NHWC output      [N][P][Q][K_pad]
    const void* res;      // residual operand or nullptr
    const void* w;        // packed filters   [K_pad][R][S][C_pad]
    const float* bias;    // [K_pad]
    int N, H, W, C_pad, P, Q, K_pad, R, S, stride, pad;
    int relu;
    int res_mode;         // 0 none, 1 same shape as y, 2 subsample + zero-channel pad
    int res_H, res_W, res_C_pad, res_C, res_pad_lo, res_stride;
};

// Filter preparation --------------------------------------------------------------------
// W'[k0+k][c0+c][r+r0][s+s0] = omega_k * W[k][c][r][s] inside a (K_dst, C_dst, R_dst, S_dst) bank.
void launch_fold_weights(const float* w, const float* bn, int K, int C, int R, int S, float eps,
                         float* dst, int C_dst, int R_dst, int S_dst, int k0, int c0, int r0, int s0,
                         cudaStream_t st);
// b[k0+k] = lambda_k (accumulate = 0) or b[k0+k] + lambda_k (accumulate = 1)
void launch_fold_bias(const float* bn, int K, float eps, float* dst_b, int k0, int accumulate, cudaStream_t st);
// unit centre taps: dst[k0+k][c0 + k - shift][R/2][S/2] = 1 for 0 <= k-shift < C_id
void launch_identity_filters(float* dst, int C_dst, int R, int S, int k0, int c0, int K_id, int C_id, int shift,
                             cudaStream_t st);
void launch_count_nonfinite(const float* p, size_t n, int* d_count, cudaStream_t st);
void launch_score_filters(const float* w, int K, int per_filter, int norm, double* scores, cudaStream_t st);
void launch_rank_mask(const double* scores, int K, int q, int32_t* rank, uint8_t* mask, cudaStream_t st);
// packed[kr][rs][cp] = w[row_src[kr]][chan_src[cp]][rs] (zero where an index is -1); bf16 and/or fp32 copies
void launch_repack(const float* w, int C, int RS, const int32_t* row_src, int K_pad, const int32_t* chan_src,
                   int C_pad, float scale, __nv_bfloat16* out_bf16, float* out_f32, cudaStream_t st);
void launch_pack_bias(const float* b, const int32_t* row_src, int K_pad, float* out, cudaStream_t st);

// Memory-bound operators ------------------------------------------------------------------
void launch_input_to_nhwc(const void* in, int in_is_bf16, void* out, int out_is_bf16, int N, int C, int H, int W,
                          int C_pad, cudaStream_t st);
void launch_maxpool(const void* x, void* y, int is_bf16, int N, int H, int W, int C_pad, int P, int Q, int R,
                    int stride, int pad, cudaStream_t st);
void launch_head(const void* x, int is_bf16, int N, int HW, int C_pad, const float* fcw, const float* fcb,
                 int n_classes, float* logits, cudaStream_t st);
void launch_nhwc_to_nchw_f32(const void* x, int is_bf16, float* out, int N, int H, int W, int C_pad,
                             const int32_t* chan_dst, int C_out, cudaStream_t st);

// Convolutions ------------------------------------------------------------------------------
// CUDA-core validation kernels: fp32 activations/filters, or bf16 activations/filters with
// fp32 accumulation (same storage as the tensor-core path, used to localise differences).
void launch_conv_simt(const ConvArgs& a, int is_bf16, cudaStream_t st);

// Tensor-core path: per-layer plan (tile shape, TMA descriptors) built once per fp_prune.
struct ConvPlanTC {
    CUtensorMap tm_x;     // activations, 4-D {C, W, H, N}
    CUtensorMap tm_w;     // filters, 3-D {C, R*S, K}
    int valid;
    int tile_w, tile_h, tile_n;   // output pixels per CTA tile = tile_w * tile_h * tile_n = 128
    int tiles_w, tiles_h, tiles_n;
    int kc;               // channels per K block (16, 32 or 64)
    int c_blocks;         // K blocks per filter tap
    int n_tile;           // filters per CTA tile (multiple of 16, <= 256)
    int n_tiles;
    int stages;
    int tmem_cols;
    int swizzle_bytes;    // 32, 64 or 128
    unsigned smem_bytes;
    int grid;
};
// Returns 0 on success, otherwise writes a message.
int plan_conv_tc(const ConvArgs& a, ConvPlanTC* plan, char* err, size_t err_len);
void launch_conv_tc(const ConvPlanTC& plan, const ConvArgs& a, int* d_status, cudaStream_t st);

}  // namespace fp
