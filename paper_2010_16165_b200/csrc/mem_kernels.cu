// Memory-bound operators of the fused graph in the planar-8 layout with a zero border (see
// fp_internal.h): boundary layout conversion, max pooling, the global-average-pool + FC head,
// and a debug dump.  One thread handles one vector (8 channels of one pixel), so a warp touches
// 32 consecutive vectors of a chunk plane: 512 contiguous bytes of bf16.
#include "fp_internal.h"

namespace fp {

namespace {

struct __align__(16) Vec8h { __nv_bfloat162 v[4]; };
struct __align__(32) Vec8f { float v[8]; };

template <bool BF16>
__device__ __forceinline__ void load_vec8(const void* base, size_t vec, float (&f)[8]) {
    if constexpr (BF16) {
        const Vec8h r = reinterpret_cast<const Vec8h*>(base)[vec];
#pragma unroll
        for (int i = 0; i < 4; ++i) { const float2 g = __bfloat1622float2(r.v[i]); f[2 * i] = g.x; f[2 * i + 1] = g.y; }
    } else {
        const Vec8f r = reinterpret_cast<const Vec8f*>(base)[vec];
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = r.v[i];
    }
}

template <bool BF16>
__device__ __forceinline__ void store_vec8(void* base, size_t vec, const float (&f)[8]) {
    if constexpr (BF16) {
        Vec8h r;
#pragma unroll
        for (int i = 0; i < 4; ++i) r.v[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        reinterpret_cast<Vec8h*>(base)[vec] = r;
    } else {
        Vec8f r;
#pragma unroll
        for (int i = 0; i < 8; ++i) r.v[i] = f[i];
        reinterpret_cast<Vec8f*>(base)[vec] = r;
    }
}

// NCHW (fp32 or bf16) -> planar-8 with border.  Thread = (chunk, flat position); reads of one
// channel plane are coalesced along w, writes are contiguous vectors.
// Images n0 .. n0 + n_count - 1 of a batch of N (the others are left alone: a caller that receives its input in
// pieces converts each piece as it arrives).
template <bool OUT_BF16>
__global__ void input_to_planar_kernel(const void* __restrict__ in, int in_is_bf16, void* __restrict__ out, int N, int C,
                                       int H, int W, int chunks, int n0, int n_count) {
    const int Wp = W + 2, P2 = (H + 2) * Wp;
    const size_t plane = (size_t)N * P2;
    const size_t part = (size_t)n_count * P2;
    const size_t total = part * chunks;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int j = (int)(i / part);
        const size_t f = i - (size_t)j * part;
        const size_t n = n0 + f / P2;
        const int rem = (int)(f % P2);
        const int h = rem / Wp - 1, w = rem % Wp - 1;
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = 0.0f;
        if (h >= 0 && h < H && w >= 0 && w < W) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int c = j * 8 + e;
                if (c < C) {
                    const size_t src = ((n * C + c) * H + h) * W + w;
                    v[e] = in_is_bf16 ? __bfloat162float(((const __nv_bfloat16*)in)[src]) : ((const float*)in)[src];
                }
            }
        }
        store_vec8<OUT_BF16>(out, (size_t)j * plane + n * P2 + rem, v);
    }
}

// Network input for a 7x7 / stride-2 / pad-3 first convolution with at most 3 input channels, packed so
// that the convolution becomes a stride-1 3x1 convolution at the output resolution (P = H/2, Q = W/2):
// the 7 horizontal taps and the input channels become 24 packed channels j = s*C + c, and the input
// rows are split by parity into three 24-channel groups
//     E (chunks 0-2):  E [p][q][j] = x[c][2p    ][2q + s - 3]
//     O'(chunks 3-5):  O'[p][q][j] = x[c][2p - 1][2q + s - 3]      (odd rows, shifted down by one)
//     O (chunks 6-8):  O [p][q][j] = x[c][2p + 1][2q + s - 3]
// (chunk 9 is zero padding to an even chunk count).  Output row p needs input rows 2p-3 .. 2p+3, which
// are O'(p-1), E(p-1), O'(p), E(p), O(p), E(p+1), O(p+1): vertical offsets -1, 0, +1 only.
// One block per (image, output row incl. the two border rows): the three input rows the output row needs are
// staged in shared memory (coalesced reads, each input element read once per block), then every thread builds
// packed vectors from them.  32-bit index arithmetic only.
__global__ void input_to_stem_planar_kernel(const void* __restrict__ in, int in_is_bf16, __nv_bfloat16* __restrict__ out,
                                            int N, int C, int H, int W, int n0) {
    extern __shared__ float rows[];                  // [3 rows: 2p-1, 2p, 2p+1][C][W + 6], zero where outside the image
    __shared__ int tap_off[24];                      // packed channel j = s*C + c -> c*(W+6) + s, or -1 (padding)
    const int P = H / 2, Q = W / 2, Qp = Q + 2, P2 = (P + 2) * Qp;
    const int n = n0 + blockIdx.x / (P + 2), pp = blockIdx.x % (P + 2);
    const int p = pp - 1;
    const size_t plane = (size_t)N * P2;
    uint4* outv = reinterpret_cast<uint4*>(out) + (size_t)n * P2 + (size_t)pp * Qp;
    if (p < 0 || p >= P) {                           // border row: zeros in every chunk
        for (int i = threadIdx.x; i < 10 * Qp; i += blockDim.x) {
            const int j8 = i / Qp, qq = i - j8 * Qp;
            outv[(size_t)j8 * plane + qq] = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    const int Ws = W + 6;
    if (threadIdx.x < 24) {
        const int sx = threadIdx.x / C, c = threadIdx.x - sx * C;
        tap_off[threadIdx.x] = sx < 7 ? c * Ws + sx : -1;
    }
    for (int i = threadIdx.x; i < 3 * C * Ws; i += blockDim.x) {
        const int rc = i / Ws, col = i - rc * Ws;
        const int r = rc / C, c = rc - r * C;
        const int ih = 2 * p - 1 + r, iw = col - 3;
        float v = 0.0f;
        if (ih >= 0 && ih < H && iw >= 0 && iw < W) {
            const size_t src = (((size_t)n * C + c) * H + ih) * W + iw;
            v = in_is_bf16 ? __bfloat162float(((const __nv_bfloat16*)in)[src]) : ((const float*)in)[src];
        }
        rows[i] = v;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 10 * Qp; i += blockDim.x) {
        const int j8 = i / Qp, qq = i - j8 * Qp;
        const int q = qq - 1;
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = 0.0f;
        if (j8 < 9 && q >= 0 && q < Q) {
            const int group = j8 / 3;                // 0 = E (row 2p), 1 = O' (row 2p-1), 2 = O (row 2p+1)
            const int r = group == 0 ? 1 : group == 1 ? 0 : 2;
            const float* base = rows + r * C * Ws + 2 * q;          // input column 2q + s - 3 sits at 2q + s
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int off = tap_off[(j8 - group * 3) * 8 + e];
                if (off >= 0) v[e] = base[off];
            }
        }
        Vec8h o;
#pragma unroll
        for (int e = 0; e < 4; ++e) o.v[e] = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
        reinterpret_cast<Vec8h*>(outv)[(size_t)j8 * plane + qq] = o;
    }
}

// The same packing for exactly three input channels (RGB): with C fixed, tap s and channel c of packed channel j
// are compile-time constants, so a vector is eight shared-memory loads at immediate offsets (no table, no
// divisions), and the rows are staged row by row.  One thread per output column.
__global__ void input_to_stem_planar_rgb_kernel(const void* __restrict__ in, int in_is_bf16, __nv_bfloat16* __restrict__ out,
                                                int N, int H, int W, int n0) {
    constexpr int C = 3;
    extern __shared__ float rows[];                  // [3 rows: 2p-1, 2p, 2p+1][C][W + 6], zero where outside the image
    const int P = H / 2, Q = W / 2, Qp = Q + 2, P2 = (P + 2) * Qp;
    const int n = n0 + blockIdx.x / (P + 2), pp = blockIdx.x % (P + 2);
    const int p = pp - 1;
    const size_t plane = (size_t)N * P2;
    Vec8h* outv = reinterpret_cast<Vec8h*>(out) + (size_t)n * P2 + (size_t)pp * Qp;
    Vec8h zero;
#pragma unroll
    for (int e = 0; e < 4; ++e) zero.v[e] = __floats2bfloat162_rn(0.0f, 0.0f);
    if (p < 0 || p >= P) {                           // border row: zeros in every chunk
        for (int j8 = 0; j8 < 10; ++j8)
            for (int qq = threadIdx.x; qq < Qp; qq += blockDim.x) outv[(size_t)j8 * plane + qq] = zero;
        return;
    }
    const int Ws = W + 6;
    for (int rc = 0; rc < 3 * C; ++rc) {
        const int r = rc / C, c = rc - r * C;
        const int ih = 2 * p - 1 + r;
        const bool row_in = ih >= 0 && ih < H;
        const size_t src = (((size_t)n * C + c) * H + (row_in ? ih : 0)) * W;
        for (int col = threadIdx.x; col < Ws; col += blockDim.x) {
            const int iw = col - 3;
            float v = 0.0f;
            if (row_in && iw >= 0 && iw < W)
                v = in_is_bf16 ? __bfloat162float(((const __nv_bfloat16*)in)[src + iw]) : ((const float*)in)[src + iw];
            rows[rc * Ws + col] = v;
        }
    }
    __syncthreads();
    for (int qq = threadIdx.x; qq < Qp; qq += blockDim.x) {
        const int q = qq - 1;
        const bool inside = q >= 0 && q < Q;
#pragma unroll
        for (int group = 0; group < 3; ++group) {    // 0 = E (row 2p), 1 = O' (row 2p-1), 2 = O (row 2p+1)
            const int r = group == 0 ? 1 : group == 1 ? 0 : 2;
            const float* base = rows + r * C * Ws + (inside ? 2 * q : 0);    // input column 2q + s - 3 sits at 2q + s
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                float v[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int j = k * 8 + e, sx = j / C, c = j - sx * C;     // constants after unrolling
                    v[e] = (sx < 7 && inside) ? base[c * Ws + sx] : 0.0f;
                }
                Vec8h o;
#pragma unroll
                for (int e = 0; e < 4; ++e) o.v[e] = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
                outv[(size_t)(group * 3 + k) * plane + qq] = o;
            }
        }
        outv[(size_t)9 * plane + qq] = zero;
    }
}

// Max pooling; padded positions never win.  Output border positions are written as zeros.
// blockIdx.x = (chunk, image, output row incl. borders), threads run along the row: no divisions per element,
// 32-bit arithmetic, and a warp reads runs of neighbouring vectors.
template <bool BF16>
__global__ void maxpool_kernel(const void* __restrict__ x, void* __restrict__ y, int N, int H, int W, int chunks, int P,
                               int Q, int R, int stride, int pad) {
    const int Wp = W + 2, P2i = (H + 2) * Wp, Qp = Q + 2, P2o = (P + 2) * Qp;
    const int rows_per_image = P + 2;
    const int row = blockIdx.x * blockDim.y + threadIdx.y;
    if (row >= chunks * N * rows_per_image) return;
    const int jn = row / rows_per_image, pp = row - jn * rows_per_image;     // jn = chunk * N + image
    const int p = pp - 1;
    const size_t in_base = (size_t)jn * P2i, out_base = (size_t)jn * P2o + (size_t)pp * Qp;
    for (int qq = threadIdx.x; qq < Qp; qq += blockDim.x) {
        const int q = qq - 1;
        float m[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) m[e] = 0.0f;
        if (p >= 0 && p < P && q >= 0 && q < Q) {
#pragma unroll
            for (int e = 0; e < 8; ++e) m[e] = -INFINITY;
            for (int r = 0; r < R; ++r) {
                const int ih = p * stride + r - pad;
                if (ih < 0 || ih >= H) continue;
                for (int sx = 0; sx < R; ++sx) {
                    const int iw = q * stride + sx - pad;
                    if (iw < 0 || iw >= W) continue;
                    float v[8];
                    load_vec8<BF16>(x, in_base + (size_t)((ih + 1) * Wp + (iw + 1)), v);
#pragma unroll
                    for (int e = 0; e < 8; ++e) m[e] = fmaxf(m[e], v[e]);
                }
            }
        }
        store_vec8<BF16>(y, out_base + qq, m);
    }
}

// 3x3 / stride-2 / pad-1 max pooling of bf16 activations, the ImageNet stem's pooling.  The generic kernel above
// issues nine 16-byte loads per output whose addresses are 32 bytes apart between neighbouring threads (eight
// cache lines per warp-wide load), and the L1 pipeline, not DRAM, bounds it.  Here a warp that owns 32 neighbouring
// outputs reads the 64 input columns under them with two fully coalesced loads per input row (lane l holds
// columns 2*q0 + l and 2*q0 + 32 + l; lane 0 also fetches column 2*q0 - 1), takes the maximum down the three rows
// first, then across each window of three columns with warp shuffles.  The maximum of bf16 values is one of them,
// so packed bf16 compares give the same result as fp32 ones.  Same block shape as the generic kernel.
__device__ __forceinline__ Vec8h vmax(const Vec8h& a, const Vec8h& b) {
    Vec8h r;
#pragma unroll
    for (int i = 0; i < 4; ++i) r.v[i] = __hmax2(a.v[i], b.v[i]);
    return r;
}
__device__ __forceinline__ Vec8h vshfl(const Vec8h& a, int src_lane) {
    Vec8h r;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t w = __shfl_sync(0xffffffffu, *reinterpret_cast<const uint32_t*>(&a.v[i]), src_lane);
        r.v[i] = *reinterpret_cast<const __nv_bfloat162*>(&w);
    }
    return r;
}
__global__ void maxpool3s2_bf16_kernel(const Vec8h* __restrict__ x, Vec8h* __restrict__ y, int N, int H, int W, int chunks,
                                       int P, int Q) {
    const int Wp = W + 2, P2i = (H + 2) * Wp, Qp = Q + 2, P2o = (P + 2) * Qp;
    const int rows_per_image = P + 2;
    const int row = blockIdx.x * blockDim.y + threadIdx.y;
    if (row >= chunks * N * rows_per_image) return;                           // the same for a whole warp
    const int jn = row / rows_per_image, pp = row - jn * rows_per_image;     // jn = chunk * N + image
    const int p = pp - 1;
    const size_t in_base = (size_t)jn * P2i, out_base = (size_t)jn * P2o + (size_t)pp * Qp;
    const int lane = threadIdx.x & 31;
    Vec8h ninf, zero;
#pragma unroll
    for (int i = 0; i < 4; ++i) { ninf.v[i] = __floats2bfloat162_rn(-INFINITY, -INFINITY); zero.v[i] = __floats2bfloat162_rn(0.0f, 0.0f); }
    for (int qq0 = threadIdx.x - lane; qq0 < Qp; qq0 += blockDim.x) {         // warp-uniform: all 32 lanes take part
        const int qq = qq0 + lane, q = qq - 1;
        if (p < 0 || p >= P) {                                                // border row: zeros
            if (qq < Qp) y[out_base + qq] = zero;
            continue;
        }
        const int c0 = 2 * (qq0 - 1);                  // input column under the warp's first output
        const int ca = c0 + lane, cb = c0 + 32 + lane, ce = c0 - 1;
        Vec8h A = ninf, B = ninf, E = ninf;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int ih = 2 * p - 1 + r;
            if (ih < 0 || ih >= H) continue;
            const Vec8h* src = x + in_base + (size_t)(ih + 1) * Wp + 1;
            if (ca >= 0 && ca < W) A = vmax(A, src[ca]);
            if (cb >= 0 && cb < W) B = vmax(B, src[cb]);
            if (lane == 0 && ce >= 0 && ce < W) E = vmax(E, src[ce]);
        }
        // windows centred on the even lanes: W_A[l] = max(A[l-1], A[l], A[l+1]) with A[-1] = E; W_B alike with B[-1] = A[31]
        Vec8h upA = vshfl(A, (lane + 31) & 31), dnA = vshfl(A, (lane + 1) & 31);
        Vec8h upB = vshfl(B, (lane + 31) & 31), dnB = vshfl(B, (lane + 1) & 31);
        const Vec8h a31 = upA;                          // on lane 0 the rotation delivered A[31]
        if (lane == 0) { upA = E; upB = a31; }
        const Vec8h WA = vmax(vmax(upA, A), dnA), WB = vmax(vmax(upB, B), dnB);
        // output j of the warp sits over columns 2j-1 .. 2j+1: window 2j of A (j < 16) or 2j-32 of B
        const Vec8h fa = vshfl(WA, (2 * lane) & 31), fb = vshfl(WB, (2 * lane) & 31);
        if (qq < Qp) y[out_base + qq] = (q >= 0 && q < Q) ? (lane < 16 ? fa : fb) : zero;
    }
}

// Head, step 1: spatial sum per channel in fp32.  One warp per (image, chunk of 8 channels): lanes
// stride over the interior positions with 16-byte loads, shuffle-reduce, and write 8 sums.
template <bool BF16>
__global__ void pool_sum_kernel(const void* __restrict__ x, int N, int H, int W, int chunks, float* __restrict__ sums) {
    const int Wp = W + 2, P2 = (H + 2) * Wp, HW = H * W;
    const size_t plane = (size_t)N * P2;
    const int lane = threadIdx.x & 31;
    const size_t warp = (blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5;
    if (warp >= (size_t)N * chunks) return;
    const int j = (int)(warp % chunks);
    const size_t n = warp / chunks;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
    for (int i = lane; i < HW; i += 32) {
        const int h = i / W, w = i - h * W;
        float v[8];
        load_vec8<BF16>(x, (size_t)j * plane + n * P2 + (size_t)(h + 1) * Wp + (w + 1), v);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += v[e];
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], d);
    }
    if (lane == 0) {
#pragma unroll
        for (int e = 0; e < 8; ++e) sums[n * (size_t)chunks * 8 + j * 8 + e] = acc[e];
    }
}

// Head, step 2: logits[n][k] = sum_c sums[n][c] * Wfc[k][c] + b[k]; the 1/(H*W) of the average is
// already folded into Wfc.  A block handles IMG images x 32 classes, the channels in slabs of 512: the slab of
// channel sums of its images sits in shared memory and every FC row it reads serves all of them (16 images per
// block instead of 4 was measured and is slower at batch 64-256: fewer blocks, and L2 is not the bound).
// A warp owns the classes k0 + warp + 8*t and walks their FC rows together: four independent row loads per
// step.  Each (image, class) sum has a fixed order: lanes stride over the channels, then a butterfly over the lanes.
constexpr int kFcClasses = 32, kFcSlab = 512;
template <int IMG>
__global__ void fc_kernel(const float* __restrict__ sums, int N, int C_pad, const float* __restrict__ fcw,
                          const float* __restrict__ fcb, int n_classes, float* __restrict__ logits) {
    extern __shared__ float sh[];          // IMG * kFcSlab
    const int n0 = blockIdx.x * IMG, k0 = blockIdx.y * kFcClasses;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kWarps = 8, kPerWarp = kFcClasses / kWarps;       // launched with 256 threads
    const float* wr[kPerWarp];
    float acc[kPerWarp][IMG];
#pragma unroll
    for (int t = 0; t < kPerWarp; ++t) {
        const int k = k0 + warp + kWarps * t;
        wr[t] = fcw + (size_t)(k < n_classes ? k : 0) * C_pad;
#pragma unroll
        for (int i = 0; i < IMG; ++i) acc[t][i] = 0.0f;
    }
    for (int c0 = 0; c0 < C_pad; c0 += kFcSlab) {
        const int cw = C_pad - c0 < kFcSlab ? C_pad - c0 : kFcSlab;
        __syncthreads();                   // the previous slab has been consumed
        for (int img = warp; img < IMG; img += kWarps)
            for (int cc = lane; cc < cw; cc += 32)
                sh[img * kFcSlab + cc] = (n0 + img < N) ? sums[(size_t)(n0 + img) * C_pad + c0 + cc] : 0.0f;
        __syncthreads();
#pragma unroll 4
        for (int c = lane; c < cw; c += 32) {      // unrolled: 16 row loads in flight per lane
            float wv[kPerWarp];
#pragma unroll
            for (int t = 0; t < kPerWarp; ++t) wv[t] = wr[t][c0 + c];
#pragma unroll
            for (int i = 0; i < IMG; ++i) {
                const float sv = sh[i * kFcSlab + c];
#pragma unroll
                for (int t = 0; t < kPerWarp; ++t) acc[t][i] = fmaf(sv, wv[t], acc[t][i]);
            }
        }
    }
#pragma unroll
    for (int t = 0; t < kPerWarp; ++t) {
        const int k = k0 + warp + kWarps * t;
#pragma unroll
        for (int i = 0; i < IMG; ++i) {
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) acc[t][i] += __shfl_xor_sync(0xffffffffu, acc[t][i], d);
        }
        if (lane == 0 && k < n_classes) {
            const float b = fcb ? fcb[k] : 0.0f;
#pragma unroll
            for (int i = 0; i < IMG; ++i)
                if (n0 + i < N) logits[(size_t)(n0 + i) * n_classes + k] = acc[t][i] + b;
        }
    }
}

template <bool BF16>
__global__ void planar_to_nchw_f32_kernel(const void* __restrict__ x, float* __restrict__ out, int N, int H, int W,
                                          int chunks, int C_out, int split) {
    // a parity-split tensor (see ConvArgs) is 4 N images of half the size
    const int Wp = split ? W / 2 + 2 : W + 2, P2 = split ? (H / 2 + 2) * Wp : (H + 2) * Wp;
    const size_t plane = (size_t)N * P2 * (split ? 4 : 1);
    const size_t total = (size_t)N * chunks * H * W;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int w = (int)(i % W);
        size_t t = i / W;
        const int h = (int)(t % H); t /= H;
        const int j = (int)(t % chunks);
        const size_t n = t / chunks;
        float v[8];
        size_t pos = n * P2 + (size_t)(h + 1) * Wp + (w + 1);
        if (split) {
            const int pp = (h & 1) ? ((w & 1) ? 2 : 1) : ((w & 1) ? 3 : 0);
            pos = ((size_t)pp * N + n) * P2 + (size_t)((h >> 1) + 1) * Wp + ((w >> 1) + 1);
        }
        load_vec8<BF16>(x, (size_t)j * plane + pos, v);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int c = j * 8 + e;
            if (c < C_out) out[((n * C_out + c) * H + h) * W + w] = v[e];
        }
    }
}

inline int grid_for(size_t n, int threads) {
    size_t b = (n + threads - 1) / threads;
    const size_t cap = (size_t)sm_count() * 16;
    if (b < 1) b = 1;
    return (int)(b > cap ? cap : b);
}

}  // namespace

void launch_input_to_planar(const void* in, int in_is_bf16, void* out, int out_is_bf16, int N, int C, int H, int W,
                            int C_pad, int n0, int n_count, cudaStream_t st) {
    const size_t n = (size_t)n_count * (H + 2) * (W + 2) * (C_pad / 8);
    if (out_is_bf16) input_to_planar_kernel<true><<<grid_for(n, 256), 256, 0, st>>>(in, in_is_bf16, out, N, C, H, W, C_pad / 8, n0, n_count);
    else input_to_planar_kernel<false><<<grid_for(n, 256), 256, 0, st>>>(in, in_is_bf16, out, N, C, H, W, C_pad / 8, n0, n_count);
}

void launch_input_to_stem_planar(const void* in, int in_is_bf16, void* out, int N, int C, int H, int W, int n0, int n_count,
                                 cudaStream_t st) {
    const size_t smem = (size_t)3 * C * (W + 6) * sizeof(float);      // <= 36 KB for the supported widths
    if (C == 3) input_to_stem_planar_rgb_kernel<<<n_count * (H / 2 + 2), 128, smem, st>>>(in, in_is_bf16, (__nv_bfloat16*)out, N, H, W, n0);
    else input_to_stem_planar_kernel<<<n_count * (H / 2 + 2), 256, smem, st>>>(in, in_is_bf16, (__nv_bfloat16*)out, N, C, H, W, n0);
}

void launch_maxpool(const void* x, void* y, int is_bf16, int N, int H, int W, int C_pad, int P, int Q, int R,
                    int stride, int pad, cudaStream_t st) {
    // the chunk planes are contiguous over the batch: (chunk, image) pairs are numbered jn = chunk * N + image
    const int tx = Q + 2 <= 32 ? 32 : Q + 2 <= 64 ? 64 : 128, ty = 256 / tx;
    const int rows = (C_pad / 8) * N * (P + 2);
    const dim3 block(tx, ty), grid((rows + ty - 1) / ty);
    if (is_bf16 && R == 3 && stride == 2 && pad == 1)
        maxpool3s2_bf16_kernel<<<grid, block, 0, st>>>((const Vec8h*)x, (Vec8h*)y, N, H, W, C_pad / 8, P, Q);
    else if (is_bf16) maxpool_kernel<true><<<grid, block, 0, st>>>(x, y, N, H, W, C_pad / 8, P, Q, R, stride, pad);
    else maxpool_kernel<false><<<grid, block, 0, st>>>(x, y, N, H, W, C_pad / 8, P, Q, R, stride, pad);
}

void launch_head(const void* x, int is_bf16, int N, int H, int W, int C_pad, const float* fcw, const float* fcb,
                 int n_classes, float* logits, float* pool_scratch, cudaStream_t st) {
    const size_t warps = (size_t)N * (C_pad / 8);
    const int blocks = (int)((warps * 32 + 255) / 256);
    if (is_bf16) pool_sum_kernel<true><<<blocks, 256, 0, st>>>(x, N, H, W, C_pad / 8, pool_scratch);
    else pool_sum_kernel<false><<<blocks, 256, 0, st>>>(x, N, H, W, C_pad / 8, pool_scratch);
    const int classes = (n_classes + kFcClasses - 1) / kFcClasses;
    // Every block re-reads the FC rows of its classes: with many channels and images that traffic (through L2) is what
    // bounds the kernel, so wide heads take 16 images per block (ResNet-50 at batch 128: 2048 channels, 8 MB of FC
    // weights read 8 times instead of 32); narrow ones keep 4, where more blocks matter more.
    if (C_pad >= 1024 && N >= 64)
        fc_kernel<16><<<dim3((N + 15) / 16, classes), 256, 16 * kFcSlab * sizeof(float), st>>>(pool_scratch, N, C_pad, fcw, fcb, n_classes, logits);
    else
        fc_kernel<4><<<dim3((N + 3) / 4, classes), 256, 4 * kFcSlab * sizeof(float), st>>>(pool_scratch, N, C_pad, fcw, fcb, n_classes, logits);
}

void launch_planar_to_nchw_f32(const void* x, int is_bf16, float* out, int N, int H, int W, int C_pad, int C_out,
                               int split, cudaStream_t st) {
    const size_t n = (size_t)N * (C_pad / 8) * H * W;
    if (is_bf16) planar_to_nchw_f32_kernel<true><<<grid_for(n, 256), 256, 0, st>>>(x, out, N, H, W, C_pad / 8, C_out, split);
    else planar_to_nchw_f32_kernel<false><<<grid_for(n, 256), 256, 0, st>>>(x, out, N, H, W, C_pad / 8, C_out, split);
}

}  // namespace fp
