// Filter preparation kernels: BN folding (Eq. 3-5 merged into the convolution), identity
// filters of the auxiliary convolutions (Sec. IV-B.1), filter scoring (Eq. 6), ranking and
// masking (Algorithm 1), and repacking of the surviving filters into K,R,S,C order.
#include "fp_internal.h"

namespace fp {

// omega_k with one rounded fp32 operation per step: t = var + eps; r = sqrt(t); omega = gamma / r.
__device__ __forceinline__ float bn_omega(const float* bn, int K, int k, float eps) {
    const float t = __fadd_rn(bn[3 * K + k], eps);
    const float r = __fsqrt_rn(t);
    return __fdiv_rn(bn[k], r);
}

__global__ void fold_weights_kernel(const float* __restrict__ w, const float* __restrict__ bn, int K, int C, int R,
                                    int S, float eps, float* __restrict__ dst, int C_dst, int R_dst, int S_dst,
                                    int k0, int c0, int r0, int s0) {
    const int per = C * R * S;
    const size_t total = (size_t)K * per;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int k = (int)(i / per);
        int rem = (int)(i - (size_t)k * per);
        const int c = rem / (R * S);
        rem -= c * R * S;
        const int r = rem / S, s = rem - r * S;
        const float omega = bn_omega(bn, K, k, eps);
        dst[(((size_t)(k0 + k) * C_dst + (c0 + c)) * R_dst + (r + r0)) * S_dst + (s + s0)] = __fmul_rn(omega, w[i]);
    }
}

// lambda = beta - omega * mean, the product and the difference rounded separately.
__global__ void fold_bias_kernel(const float* __restrict__ bn, int K, float eps, float* __restrict__ dst, int k0,
                                 int accumulate) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    const float omega = bn_omega(bn, K, k, eps);
    const float m = __fmul_rn(omega, bn[2 * K + k]);
    const float lam = __fsub_rn(bn[K + k], m);
    dst[k0 + k] = accumulate ? __fadd_rn(dst[k0 + k], lam) : lam;
}

__global__ void identity_filters_kernel(float* dst, int C_dst, int R, int S, int k0, int c0, int K_id, int C_id,
                                        int shift) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K_id) return;
    const int c = k - shift;
    if (c < 0 || c >= C_id) return;
    dst[(((size_t)(k0 + k) * C_dst + (c0 + c)) * R + R / 2) * S + S / 2] = 1.0f;
}

__global__ void count_nonfinite_kernel(const float* __restrict__ p, size_t n, int* count) {
    int bad = 0;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        bad += !isfinite(p[i]);
    if (bad) atomicAdd(count, bad);
}

// One warp per filter.  Lane l accumulates elements l, l+32, ... in increasing order in fp64
// (each |w| or w*w is exact in fp64), then the 32 partial sums are combined pairwise with
// partners at distance 16, 8, 4, 2, 1.  The order is part of the definition of the score, so
// that the resulting double - and therefore the ranking - does not depend on the launch shape.
__global__ void score_filters_kernel(const float* __restrict__ w, int K, int per, int norm, double* __restrict__ scores) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= K) return;
    const float* f = w + (size_t)warp * per;
    double s = 0.0;
    for (int t = lane; t < per; t += 32) {
        const double v = (double)f[t];
        s = __dadd_rn(s, norm ? __dmul_rn(v, v) : fabs(v));
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) s = __dadd_rn(s, __shfl_xor_sync(0xffffffffu, s, d));
    if (lane == 0) scores[warp] = s;
}

// rank[k] = number of filters ordered before k in ascending (score, index) order; the first q are masked.
__global__ void rank_mask_kernel(const double* __restrict__ scores, int K, int q, int32_t* __restrict__ rank,
                                 uint8_t* __restrict__ mask) {
    extern __shared__ double sh[];
    for (int i = threadIdx.x; i < K; i += blockDim.x) sh[i] = scores[i];
    __syncthreads();
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const double sk = sh[k];
        int before = 0;
        for (int j = 0; j < K; ++j) {
            const double sj = sh[j];
            before += (sj < sk) || (sj == sk && j < k);
        }
        rank[k] = before;
        mask[k] = before >= q ? 1 : 0;
    }
}

// Algorithm 1's loop body over all banks.  One warp per filter: lane l updates and accumulates elements l, l+32, ...
// in increasing order, then the 32 partial sums are combined pairwise at distances 16, 8, 4, 2, 1 - the order
// that defines a score (see score_filters_kernel).
__global__ void soft_update_score_kernel(const SoftBank* __restrict__ banks, const int32_t* __restrict__ filter_bank,
                                         int total_filters, const float* __restrict__ dw, int norm,
                                         double* __restrict__ scores) {
    const int g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (g >= total_filters) return;
    const SoftBank b = banks[filter_bank[g]];
    const int k = g - b.k_off;
    float* f = b.w + (size_t)k * b.per;
    const float* d = dw ? dw + b.dw_off + (size_t)k * b.per : nullptr;
    double s = 0.0;
    for (int t = lane; t < b.per; t += 32) {
        float v = f[t];
        if (d) { v = __fadd_rn(v, d[t]); f[t] = v; }
        const double x = (double)v;
        s = __dadd_rn(s, norm ? __dmul_rn(x, x) : fabs(x));
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s = __dadd_rn(s, __shfl_xor_sync(0xffffffffu, s, o));
    if (lane == 0) scores[g] = s;
}

__global__ void soft_rank_kernel(const SoftBank* __restrict__ banks, const double* __restrict__ scores,
                                 int32_t* __restrict__ rank, uint8_t* __restrict__ mask) {
    extern __shared__ double sh[];
    const SoftBank b = banks[blockIdx.x];
    for (int i = threadIdx.x; i < b.K; i += blockDim.x) sh[i] = scores[b.k_off + i];
    __syncthreads();
    for (int k = threadIdx.x; k < b.K; k += blockDim.x) {
        const double sk = sh[k];
        int before = 0;
        for (int j = 0; j < b.K; ++j) {
            const double sj = sh[j];
            before += (sj < sk) || (sj == sk && j < k);
        }
        rank[b.k_off + k] = before;
        mask[b.k_off + k] = before >= b.q ? 1 : 0;
    }
}

__global__ void soft_zeroize_kernel(const SoftBank* __restrict__ banks, const int32_t* __restrict__ filter_bank,
                                    int total_filters, const uint8_t* __restrict__ mask) {
    const int g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (g >= total_filters || mask[g]) return;
    const SoftBank b = banks[filter_bank[g]];
    float* f = b.w + (size_t)(g - b.k_off) * b.per;
    for (int t = lane; t < b.per; t += 32) f[t] = 0.0f;
}

// Filters of one convolution in the order the MMA wants them: tap-major, then chunks of 8 input
// channels, then the filter, then the channel within the chunk.  For a fixed tap and chunk the
// K_pad x 8 block is a stack of 16-byte rows - the canonical K-major operand layout without swizzle.
__global__ void repack_conv_kernel(const float* __restrict__ w, int C, int RS, const int32_t* __restrict__ row_src,
                                   int K_pad, const int32_t* __restrict__ chan_src, int C_pad,
                                   __nv_bfloat16* __restrict__ out_bf16, float* __restrict__ out_f32) {
    const size_t total = (size_t)RS * C_pad * K_pad;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int e = (int)(i % 8);
        size_t t = i / 8;
        const int kr = (int)(t % K_pad); t /= K_pad;
        const int chunk = (int)(t % (C_pad / 8));
        const int rs = (int)(t / (C_pad / 8));
        const int cp = chunk * 8 + e;
        const int ks = row_src[kr], cs = chan_src[cp];
        float v = 0.0f;
        if (ks >= 0 && cs >= 0) v = w[((size_t)ks * C + cs) * RS + rs];
        if (out_bf16) out_bf16[i] = __float2bfloat16_rn(v);
        if (out_f32) out_f32[i] = v;
    }
}

// Filters of a 3x3 convolution for a fused run of layers: for tap row r and channel chunk the operand is
// a stack of 3*K_pad 16-byte rows; filter kr at horizontal tap s is row 48*(kr/16) + 16*s + kr%16.
__global__ void repack_chain_kernel(const float* __restrict__ w, int C, const int32_t* __restrict__ row_src, int K_pad,
                                    const int32_t* __restrict__ chan_src, int C_pad, __nv_bfloat16* __restrict__ out) {
    const size_t total = (size_t)9 * C_pad * K_pad;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int e = (int)(i % 8);
        size_t t = i / 8;
        const int n = (int)(t % (3 * K_pad)); t /= 3 * K_pad;
        const int chunk = (int)(t % (C_pad / 8));
        const int r = (int)(t / (C_pad / 8));
        const int kr = (n / 48) * 16 + n % 16, sx = (n % 48) / 16;
        const int ks = row_src[kr], cs = chan_src[chunk * 8 + e];
        float v = 0.0f;
        if (ks >= 0 && cs >= 0) v = w[((size_t)ks * C + cs) * 9 + r * 3 + sx];
        out[i] = __float2bfloat16_rn(v);
    }
}

// Filters of a 7x7 first convolution in the order the packed network input wants them (see
// input_to_stem_planar_kernel): a 3x1 convolution over 80 packed channels.  Tap dr (0..2 = offsets
// -1,0,+1), chunk 0-2 (group E) take filter row r = 2*dr + 1, chunks 3-5 (O') take r = 2*dr at dr = 0, 1,
// chunks 6-8 (O) take r = 2*dr + 2 at dr = 1, 2; packed channel j = s*C + c within a group; everything else
// zero.  (Input row 2p+1 is held twice, as O of packed row p and as O' of row p+1; it is taken from row p,
// because below the last image row there is only the zero border.)
__global__ void repack_stem_kernel(const float* __restrict__ w, int C, const int32_t* __restrict__ row_src, int K_pad,
                                   __nv_bfloat16* __restrict__ out) {
    const size_t total = (size_t)3 * 10 * K_pad * 8;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int e = (int)(i % 8);
        size_t t = i / 8;
        const int kr = (int)(t % K_pad); t /= K_pad;
        const int chunk = (int)(t % 10);
        const int dr = (int)(t / 10);
        float v = 0.0f;
        const int ks = row_src[kr];
        if (ks >= 0 && chunk < 9) {
            const int group = chunk / 3;
            const int j = (chunk % 3) * 8 + e;
            const int sx = j / C, c = j - sx * C;
            int r = -1;
            if (group == 0) r = 2 * dr + 1;
            else if (group == 1) { if (dr < 2) r = 2 * dr; }
            else if (dr >= 1) r = 2 * dr + 2;
            if (r >= 0 && sx < 7) v = w[(((size_t)ks * C + c) * 7 + r) * 7 + sx];
        }
        out[i] = __float2bfloat16_rn(v);
    }
}

// Filters of the first convolution for the kernel that fuses it with the pooling: the 7x7 / stride-2 window over C
// channels as a 4x4 window over the 4 C parity channels of the half-resolution input - tap (ta, tb), channel
// (2a + b) C + c takes w[k][c][2 ta + a - 1][2 tb + b - 1] (zero where an index is -1) - as [tap][chunk of 8][filter][8].
__global__ void repack_stem_direct_kernel(const float* __restrict__ w, int C, const int32_t* __restrict__ row_src, int K_pad,
                                          __nv_bfloat16* __restrict__ out) {
    const int total = 16 * 2 * K_pad * 8;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int e = i % 8, kr = (i / 8) % K_pad, chunk = (i / (8 * K_pad)) % 2, tap = i / (16 * K_pad);
        const int ch = chunk * 8 + e, ta = tap >> 2, tb = tap & 3;
        float v = 0.0f;
        const int ks = row_src[kr];
        if (ks >= 0 && ch < 4 * C) {
            const int par = ch / C, c = ch - par * C;
            const int r = 2 * ta + (par >> 1) - 1, s = 2 * tb + (par & 1) - 1;
            if (r >= 0 && s >= 0) v = w[(((size_t)ks * C + c) * 7 + r) * 7 + s];
        }
        out[i] = __float2bfloat16_rn(v);
    }
}

__global__ void reblock_bank_kernel(const uint4* __restrict__ packed, int RS, int cchunks, int K_pad, int n_tile, int n_tiles,
                                    int cg, uint4* __restrict__ blocked) {
    const size_t total = (size_t)n_tiles * RS * cchunks * n_tile;          // 16-byte rows
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        // i = ((t * cchunks*RS ... decoded block by block: tile t, then group g (cgg chunks), tap, chunk, row
        const size_t per_tile = (size_t)RS * cchunks * n_tile;
        const int t = (int)(i / per_tile);
        size_t r = i - (size_t)t * per_tile;
        const size_t full_group = (size_t)RS * cg * n_tile;
        const int g = (int)(r / full_group);
        r -= (size_t)g * full_group;
        int cgg = cchunks - g * cg;
        if (cgg > cg) cgg = cg;
        const int tap = (int)(r / ((size_t)cgg * n_tile));
        r -= (size_t)tap * cgg * n_tile;
        const int c = (int)(r / n_tile), row = (int)(r - (size_t)c * n_tile);
        const int k = t * n_tile + row;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (k < K_pad) v = packed[((size_t)tap * cchunks + (g * cg + c)) * K_pad + k];
        blocked[i] = v;
    }
}

__global__ void repack_fc_kernel(const float* __restrict__ w, int C, int K, const int32_t* __restrict__ chan_src,
                                 int C_pad, float scale, float* __restrict__ out) {
    const size_t total = (size_t)K * C_pad;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int cp = (int)(i % C_pad);
        const int k = (int)(i / C_pad);
        const int cs = chan_src[cp];
        out[i] = cs >= 0 ? w[(size_t)k * C + cs] * scale : 0.0f;
    }
}

__global__ void pack_bias_kernel(const float* __restrict__ b, const int32_t* __restrict__ row_src, int K_pad,
                                 float* __restrict__ out) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K_pad) return;
    out[k] = row_src[k] >= 0 ? b[row_src[k]] : 0.0f;
}

static inline int blocks_for(size_t n, int threads) {
    const int cap = fp::sm_count() * 8;
    size_t b = (n + threads - 1) / threads;
    if (b < 1) b = 1;
    return (int)(b > (size_t)cap ? cap : b);
}

void launch_fold_weights(const float* w, const float* bn, int K, int C, int R, int S, float eps, float* dst,
                         int C_dst, int R_dst, int S_dst, int k0, int c0, int r0, int s0, cudaStream_t st) {
    const size_t n = (size_t)K * C * R * S;
    fold_weights_kernel<<<blocks_for(n, 256), 256, 0, st>>>(w, bn, K, C, R, S, eps, dst, C_dst, R_dst, S_dst, k0, c0, r0, s0);
}

void launch_fold_bias(const float* bn, int K, float eps, float* dst_b, int k0, int accumulate, cudaStream_t st) {
    fold_bias_kernel<<<(K + 127) / 128, 128, 0, st>>>(bn, K, eps, dst_b, k0, accumulate);
}

void launch_identity_filters(float* dst, int C_dst, int R, int S, int k0, int c0, int K_id, int C_id, int shift,
                             cudaStream_t st) {
    identity_filters_kernel<<<(K_id + 127) / 128, 128, 0, st>>>(dst, C_dst, R, S, k0, c0, K_id, C_id, shift);
}

void launch_count_nonfinite(const float* p, size_t n, int* d_count, cudaStream_t st) {
    if (n == 0) return;
    count_nonfinite_kernel<<<blocks_for(n, 256), 256, 0, st>>>(p, n, d_count);
}

void launch_score_filters(const float* w, int K, int per_filter, int norm, double* scores, cudaStream_t st) {
    const int warps_per_block = 8;
    score_filters_kernel<<<(K + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, st>>>(w, K, per_filter, norm, scores);
}

void launch_rank_mask(const double* scores, int K, int q, int32_t* rank, uint8_t* mask, cudaStream_t st) {
    rank_mask_kernel<<<1, 256, (size_t)K * sizeof(double), st>>>(scores, K, q, rank, mask);
}

void launch_soft_update_score(const SoftBank* banks, const int32_t* filter_bank, int total_filters, const float* dw,
                              int norm, double* scores, cudaStream_t st) {
    const int warps_per_block = 8;
    soft_update_score_kernel<<<(total_filters + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, st>>>(
        banks, filter_bank, total_filters, dw, norm, scores);
}
void launch_soft_rank(const SoftBank* banks, int n_banks, int max_K, const double* scores, int32_t* rank, uint8_t* mask,
                      cudaStream_t st) {
    soft_rank_kernel<<<n_banks, 256, (size_t)max_K * sizeof(double), st>>>(banks, scores, rank, mask);
}
void launch_soft_zeroize(const SoftBank* banks, const int32_t* filter_bank, int total_filters, const uint8_t* mask,
                         cudaStream_t st) {
    const int warps_per_block = 8;
    soft_zeroize_kernel<<<(total_filters + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, st>>>(
        banks, filter_bank, total_filters, mask);
}

void launch_repack_conv(const float* w, int C, int RS, const int32_t* row_src, int K_pad, const int32_t* chan_src,
                        int C_pad, __nv_bfloat16* out_bf16, float* out_f32, cudaStream_t st) {
    const size_t n = (size_t)K_pad * RS * C_pad;
    repack_conv_kernel<<<blocks_for(n, 256), 256, 0, st>>>(w, C, RS, row_src, K_pad, chan_src, C_pad, out_bf16, out_f32);
}

void launch_repack_chain(const float* w, int C, const int32_t* row_src, int K_pad, const int32_t* chan_src, int C_pad,
                         __nv_bfloat16* out, cudaStream_t st) {
    repack_chain_kernel<<<blocks_for((size_t)9 * C_pad * K_pad, 256), 256, 0, st>>>(w, C, row_src, K_pad, chan_src, C_pad, out);
}

void launch_repack_stem(const float* w, int C, const int32_t* row_src, int K_pad, __nv_bfloat16* out, cudaStream_t st) {
    repack_stem_kernel<<<blocks_for((size_t)240 * K_pad, 256), 256, 0, st>>>(w, C, row_src, K_pad, out);
}

void launch_repack_stem_direct(const float* w, int C, const int32_t* row_src, int K_pad, __nv_bfloat16* out, cudaStream_t st) {
    repack_stem_direct_kernel<<<blocks_for((size_t)256 * K_pad, 256), 256, 0, st>>>(w, C, row_src, K_pad, out);
}

void launch_reblock_bank(const __nv_bfloat16* packed, int RS, int cchunks, int K_pad, int n_tile, int n_tiles, int cg,
                         __nv_bfloat16* blocked, cudaStream_t st) {
    const size_t n = (size_t)n_tiles * RS * cchunks * n_tile;
    reblock_bank_kernel<<<blocks_for(n, 256), 256, 0, st>>>((const uint4*)packed, RS, cchunks, K_pad, n_tile, n_tiles, cg, (uint4*)blocked);
}

void launch_repack_fc(const float* w, int C, int K, const int32_t* chan_src, int C_pad, float scale, float* out,
                      cudaStream_t st) {
    repack_fc_kernel<<<blocks_for((size_t)K * C_pad, 256), 256, 0, st>>>(w, C, K, chan_src, C_pad, scale, out);
}

__global__ void add_bias_kernel(const float* __restrict__ a, const float* __restrict__ b, int n, float* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = a[i] + b[i];
}

void launch_add_bias(const float* a, const float* b, int n, float* out, cudaStream_t st) {
    add_bias_kernel<<<(n + 127) / 128, 128, 0, st>>>(a, b, n, out);
}

void launch_pack_bias(const float* b, const int32_t* row_src, int K_pad, float* out, cudaStream_t st) {
    pack_bias_kernel<<<(K_pad + 127) / 128, 128, 0, st>>>(b, row_src, K_pad, out);
}

}  // namespace fp
