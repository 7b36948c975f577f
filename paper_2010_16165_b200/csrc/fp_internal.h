// Internal declarations shared by the host graph builder and the kernel launchers.
//
// Activation layout ("planar-8 with border"): channels are grouped in chunks of 8 (one 16-byte
// vector of bf16, or 32 bytes of fp32); every image carries a one-pixel border of zeros.
// For a batch of N images of H x W pixels and C_pad channels the vector of chunk j, image n,
// pixel (h, w) sits at vector index
//       j * (N * P2)  +  n * P2  +  (h + 1) * (W + 2)  +  (w + 1),      P2 = (H + 2) * (W + 2).
// So each chunk is one contiguous plane over the whole batch; a run of consecutive "flat
// positions" f = n*P2 + (h+1)*(W+2) + (w+1) is contiguous in memory for every chunk, and the
// 3x3 neighbourhood of position f is f + dr*(W+2) + ds.  Every kernel that writes a tensor
// writes all of its positions, zeros on the border, so the border never has to be cleared.
// Buffers carry `kGuardVectors` vectors of slack before and after the data, because tiles of
// flat positions read a halo that may start before the first plane or end after the last.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

namespace fp {

// Streaming multiprocessors of the current device (asked once per device; 148 on a B200).  Grids are sized from it.
inline int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { cudaGetLastError(); n = 148; }
        cached[dev] = n;
    }
    return cached[dev];
}

constexpr int kGuardVectors = 1024;   // >= 128 + (W + 3) + 8 for every supported width (W <= 512)
constexpr int kMaxWidth = 512;

// ---------------------------------------------------------------------------------------
// Convolution launch description (one fused operator: conv + bias + residual + ReLU)
// ---------------------------------------------------------------------------------------
struct ConvArgs {
    const void* x;        // input activations, planar-8 with border (vector 0 of plane 0)
    void* y;              // output activations, same layout, P x Q pixels, K_pad channels
    const void* res;      // residual operand or nullptr
    const void* w;        // packed filters [R*S][C_pad/8][K_pad][8]
    const float* bias;    // [K_pad]
    int N, H, W, C_pad, P, Q, K_pad, R, S, stride, pad;   // pad: rows; columns are padded by pad when S == R, by (S-1)/2 otherwise
    int relu;
    int res_mode;         // 0 none, 1 same shape as y, 2 subsample + zero-channel pad
    int res_H, res_W, res_C_pad, res_C, res_pad_lo, res_stride;
    // Scattered output (tensor-core path): the K_pad packed filter rows hold only the kept filters of a convolution
    // whose output tensor keeps its full width out_C_pad (a residual stream that other layers write too); output
    // channel c takes accumulator column out_map[c], or only the shortcut when out_map[c] < 0.  Filter tile t
    // (rows t*n_tile ..) owns the output chunks tile_chunk0[t] .. tile_chunk0[t+1]-1 and holds exactly their filters.
    int scatter, out_C_pad;
    const int32_t* out_map;        // [out_C_pad], device
    const int32_t* tile_chunk0;    // [n_tiles + 1], device
    int n_tile_forced;             // > 0: filters per CTA tile fixed by the caller (scatter), else chosen by the plan
    // Parity-split tensors (tensor-core path).  A tensor that only stride-2 convolutions read is stored as four
    // half-resolution tensors, one per (row parity, column parity) of its pixels, in the order 00, 10, 11, 01, laid out
    // as 4 N images of (H/2) x (W/2) pixels: image pp * N + n holds the pixels (2i + a, 2j + b) of image n.
    int y_split;                   // write the output that way (the kernel's own grid stays P x Q)
    int x_plane_mult;              // 0/1: x is a plain tensor; 4: x is a split tensor and this 1x1 layer reads its images
                                   //      0 .. N-1 only (parity 00 = the pixels a 1x1 / stride-2 convolution reads)
    // A second input tensor along the reduction (tensor-core path, 1x1 / stride-1 layers): channel chunks >= x2_chunk0 of
    // the C_pad channels come from x2 (chunk - x2_chunk0 of it), a tensor on the same position grid - the input of a
    // projection shortcut, whose filters are then stacked behind this layer's along the channels (Sec. IV-B: one
    // convolution [W2' || S_w] instead of two and an add).  x2_plane_mult 4: x2 is parity-split and its images 0..N-1
    // (parity 00) are the ones read, as for a 1x1 / stride-2 convolution.
    const void* x2;
    int x2_chunk0;                 // 0: no second input stacked along the channels
    int x2_plane_mult;
    // The same for a 3x3 / stride-1 layer with streamed filters: the projection enters as extra K groups that have a
    // centre tap only - x2_C_pad channels of x2, filters w2 = [chunk][K_pad][8] (the projection's own packed bank).
    const void* w2;
    int x2_C_pad;                  // 0: none
    int x_s2d;                     // x is a split tensor and this is the 3x3 / stride 2 / pad 1 convolution over the tensor
                                   // it was split from: H, W, P, Q are the half resolution, stride is given as 1; the nine
                                   // taps read the parity images at offsets -1 / 0 rows and columns
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
// Algorithm 1's loop body over ALL filter banks of a model in three launches.  One SoftBank per convolution;
// filter_bank[g] names the bank of global filter g (filters of all banks numbered consecutively, bank by bank).
struct SoftBank {
    float* w;             // K x per fp32, updated and zeroized in place
    long long dw_off;     // element offset of the bank's addends in the update array
    int K, per, q;        // filters, weights per filter, filters to zeroize
    int k_off;            // global number of the bank's first filter
};
// w += dw (one fp32 addition per weight; dw may be nullptr) and the filter scores of the updated weights, in the
// fixed summation order of launch_score_filters
void launch_soft_update_score(const SoftBank* banks, const int32_t* filter_bank, int total_filters, const float* dw,
                              int norm, double* scores, cudaStream_t st);
// per bank: rank by (score, index) ascending, mask the first q (one block per bank)
void launch_soft_rank(const SoftBank* banks, int n_banks, int max_K, const double* scores, int32_t* rank, uint8_t* mask,
                      cudaStream_t st);
// masked filters become zero
void launch_soft_zeroize(const SoftBank* banks, const int32_t* filter_bank, int total_filters, const uint8_t* mask,
                         cudaStream_t st);
// Convolution filters: packed[rs][cp/8][kr][cp%8] = w[row_src[kr]][chan_src[cp]][rs] (zero where an index is -1)
void launch_repack_conv(const float* w, int C, int RS, const int32_t* row_src, int K_pad, const int32_t* chan_src,
                        int C_pad, __nv_bfloat16* out_bf16, float* out_f32, cudaStream_t st);
// Streamed filter bank: from packed[rs][cp/8][K_pad][8] to blocks in the order the tensor-core kernel streams them,
// blocked[filter tile t][K group g][rs][chunk in group][row in tile][8] (groups of `cg` chunks, the last one shorter;
// tiles of `n_tile` rows, rows past K_pad zero): n_tiles * RS * (C_pad/8) * n_tile * 8 elements
void launch_reblock_bank(const __nv_bfloat16* packed, int RS, int cchunks, int K_pad, int n_tile, int n_tiles, int cg,
                         __nv_bfloat16* blocked, cudaStream_t st);
// FC matrix: packed[k][cp] = w[k][chan_src[cp]] * scale
void launch_repack_fc(const float* w, int C, int K, const int32_t* chan_src, int C_pad, float scale, float* out,
                      cudaStream_t st);
// 7x7 first convolution as a 3x1 convolution over the packed network input (80 channels)
void launch_repack_stem(const float* w, int C, const int32_t* row_src, int K_pad, __nv_bfloat16* out, cudaStream_t st);
void launch_add_bias(const float* a, const float* b, int n, float* out, cudaStream_t st);          // out = a + b (fp32)
void launch_pack_bias(const float* b, const int32_t* row_src, int K_pad, float* out, cudaStream_t st);
// 3x3 filters of one layer of a fused run: blob[r][cp/8][48*(kr/16) + 16*s + kr%16][cp%8], the three
// horizontal taps stacked along the filter (N) axis of the MMA (see chain_tc.cu)
void launch_repack_chain(const float* w, int C, const int32_t* row_src, int K_pad, const int32_t* chan_src, int C_pad,
                         __nv_bfloat16* out, cudaStream_t st);

// Memory-bound operators ------------------------------------------------------------------
// Both convert images n0 .. n0 + n_count - 1 of a batch of N images (`in` and `out` are the whole batch's buffers).
void launch_input_to_planar(const void* in, int in_is_bf16, void* out, int out_is_bf16, int N, int C, int H, int W,
                            int C_pad, int n0, int n_count, cudaStream_t st);
void launch_input_to_stem_planar(const void* in, int in_is_bf16, void* out, int N, int C, int H, int W, int n0, int n_count,
                                 cudaStream_t st);
void launch_maxpool(const void* x, void* y, int is_bf16, int N, int H, int W, int C_pad, int P, int Q, int R,
                    int stride, int pad, cudaStream_t st);
void launch_head(const void* x, int is_bf16, int N, int H, int W, int C_pad, const float* fcw, const float* fcb,
                 int n_classes, float* logits, float* pool_scratch, cudaStream_t st);
void launch_planar_to_nchw_f32(const void* x, int is_bf16, float* out, int N, int H, int W, int C_pad, int C_out,
                               int split, cudaStream_t st);

// Convolutions ------------------------------------------------------------------------------
// CUDA-core validation kernels: fp32 activations/filters, or bf16 activations/filters with
// fp32 accumulation (same storage as the tensor-core path, used to localise differences).
void launch_conv_simt(const ConvArgs& a, int is_bf16, cudaStream_t st);

// Tensor-core path: per-layer plan built once per fp_prune.
struct ConvPlanTC {
    int valid;
    int flat;             // 1: stride-1 "same" convolution, activation tiles fetched as contiguous runs
                          //    of flat positions (bulk copies); 0: gathered by loader threads
    int b_resident;       // flat only: the whole filter bank stays in shared memory
    int blocked_bank;     // 1: 1x1 layer with unified stages, bank stored block by block; 2: gathered layer with several
                          // filter tiles, bank stored tile by tile (launch_reblock_bank either way)
    int cg;               // channel chunks (of 8) per K block
    int groups;           // K blocks per filter tap = ceil((C_pad/8) / cg)
    int halo;             // flat: vectors fetched before and after the 128 positions of a tile
    int rows_a;           // flat: vectors per chunk per tile (128 + 2*halo, rounded up to 8)
    int a_stages, b_stages;
    int tpk;              // gather: filter taps per K block (several when the channel count is small)
    int n_tile, n_tiles;  // filters per CTA tile (multiple of 16, <= 256)
    int epi_warps;        // 4, or 8 for wide filter tiles
    int tps;              // streamed filters: 128-position tiles per pipeline step
    int tmem_cols;
    unsigned smem_bytes;
    int ctas_per_sm;
};
// Filters per CTA tile the plan would choose for K_pad filter rows of this geometry (used to lay out scattered banks).
void conv_tc_filter_tile(const ConvArgs& a, int K_pad, int* n_tile, int* n_tiles);
// Returns 0 on success, otherwise writes a message.
int plan_conv_tc(const ConvArgs& a, ConvPlanTC* plan, char* err, size_t err_len);
// skip_round / wait_cycles: diagnostic launch (see fp_debug_expire_wait): the activation producer of a stride-1 layer leaves
// out one round of copies and every wait gives up after wait_cycles SM clock cycles; -1 / 0 for a normal launch
void launch_conv_tc(const ConvPlanTC& plan, const ConvArgs& a, int* d_status, cudaStream_t st, int skip_round = -1,
                    long long wait_cycles = 0);

// First convolution (7x7 / stride 2 / pad 3, at most 3 input channels, ReLU) and the 3x3 / stride 2 / pad 1 max pooling
// behind it as one kernel that reads the NCHW bf16 network input and writes the pooled tensor.
struct StemPoolArgs {
    const void* x;        // network input, N x C x H x W, NCHW, bf16
    void* y;              // pooled tensor, planar-8 with border, (H/4) x (W/4) pixels, K_pad channels, N images
    const void* w;        // filters [16 taps (ta, tb)][2 chunks of 8][K_pad rows][8] bf16 over the parity channels (launch_repack_stem_direct)
    const float* bias;    // [K_pad]
    int N, C, H, W, K_pad;
    int n0, n_count;      // the images this launch handles (the tensor's plane pitch is that of all N)
};
struct StemPoolPlan { int valid, tiles, tmem_cols; unsigned smem_bytes; };
bool stem_pool_supported(int C, int H, int W, int K_pad);
int plan_stem_pool(const StemPoolArgs& a, StemPoolPlan* plan, char* err, size_t err_len);
void launch_stem_pool(const StemPoolPlan& plan, const StemPoolArgs& a, int* d_status, cudaStream_t st);
// its filters: out[k / 8][kr][k % 8] = w[row_src[kr]][c][r][s] with k = (r * C + c) * 7 + s (zero rows / zero k padding)
void launch_repack_stem_direct(const float* w, int C, const int32_t* row_src, int K_pad, __nv_bfloat16* out, cudaStream_t st);

// A run of stride-1 3x3 convolutions executed by one kernel with the activations in shared memory.
constexpr int kChainMaxLayers = 40;
struct ChainLayer {
    int cchunks;          // input channels / 8
    int K_pad;            // output channels, multiple of 16, <= 80
    int relu;
    int res;              // 1: add the tensor two layers back (the one this layer overwrites in place)
    int blob_off;         // byte offset of the layer's filter blob (filters, then K_pad fp32 biases) in `w`
    int blob_bytes;
};
struct ChainArgs {
    const void* x;        // input of the first layer (global): planar-8 with border, or, with in_mode 1 / 2, the
                          // network input itself: N x in_C x H x W, NCHW, fp32 / bf16 (rounded to bf16 on load)
    void* y;              // output of the last layer, same layout
    const void* res;      // shortcut operand of the FIRST layer (global) or nullptr
    const void* w;        // filter blobs of all layers
    int N, H, W, n_layers;
    int in_mode, in_C;
    int res_mode;         // first layer: 0 none, 1 same shape as its output, 2 subsample + zero-channel pad
    int res_H, res_W, res_C_pad, res_C, res_pad_lo, res_stride;
    ChainLayer layers[kChainMaxLayers];
};
struct ChainPlan {
    int valid;
    int G;                // images per group (per CTA at a time)
    int tiles;            // 128-position tiles per group
    int plane_rows;       // vectors per channel chunk of an activation buffer
    int buf_bytes, wbuf_bytes, acc_cols, tmem_cols;
    int stages;           // accumulator stages in tensor memory (ring)
    int issuers;          // MMA-issuing warps (each owns stages/issuers accumulator stages)
    int split;            // epilogue groups per tile (1, 2, 4): each takes every split-th channel chunk
    unsigned smem_bytes;
};
int chain_layer_blob_bytes(int cchunks, int K_pad);
bool chain_layer_supported(int H, int W, int K_pad, int C_pad);
int plan_chain_tc(const ChainArgs& a, ChainPlan* plan, char* err, size_t err_len);
void launch_chain_tc(const ChainPlan& plan, const ChainArgs& a, int* d_status, cudaStream_t st);

}  // namespace fp
