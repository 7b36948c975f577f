// First convolution + max pooling of an ImageNet-shaped network in one kernel for sm_100a:
//     NCHW bf16 input  ->  7x7 / stride 2 / pad 3 convolution (folded-BN bias, ReLU)  ->  3x3 / stride 2 / pad 1
//     max pooling  ->  planar-8 bf16 tensor with a zero border (fp_internal.h).
// The convolution's output, four times the size of the pooled tensor, never leaves the SM.
//
//   Unit of work   one image and two pooled rows: their 3x3 windows cover five convolution rows, which need fifteen
//                  input rows.  Persistent CTAs walk the units.
//   Input          each (channel, row) is one contiguous run of the NCHW input: fifteen rows per channel are fetched
//                  with bulk copies into shared memory (16 bytes of zeros on either side of a row are the horizontal
//                  padding, rows outside the image are cleared by the threads); the next unit's rows are requested
//                  while this unit is computed.
//   GEMM           The 7x7 / stride-2 window over C channels is a 4x4 / stride-1 window over the 4 C channels of the
//                  input's four pixel parities at half resolution (input row 2i + a, column 2j + b -> channel
//                  (2a + b) C + c of half-resolution pixel (i, j); filter tap r = 2 ta + a - 1, s = 2 tb + b - 1, the taps
//                  with r or s = -1 being zero).  The compute warps rewrite a unit's staged rows once into that form
//                  - planar, 16 channels in two chunks of 8, eight half-resolution rows of W/2 + 3 pixels - and the
//                  convolution is then sixteen taps of one K = 16 step each over FLAT positions of that grid, the operand
//                  of tap (ta, tb) being the same rows ta * pitch + tb further on: no per-position gathering.  M = the
//                  unit's 5 x pitch positions in tiles of 128 (the three pad columns per row are computed and dropped),
//                  N = K_pad filters.  One thread issues the tcgen05 MMAs of a unit while the compute warps pool the
//                  previous unit and rewrite the next one's rows (two parity buffers); the accumulators of the unit's
//                  tiles stay in tensor memory until the epilogue has read them.
//   Epilogue       tcgen05.ld -> bias -> ReLU -> bf16 into a shared-memory copy of the five convolution rows (zeros for
//                  rows outside the image: after the ReLU a zero never wins a window it should not), then the 3x3
//                  maxima, written with 16-byte stores, 512 contiguous bytes per warp; the units at an image's
//                  first and last rows also write the output tensor's zero border rows.
//   Waits          bounded, as in the other tensor-core kernels: a wait that runs out raises the status word, every
//                  thread leaves the loop at the next block-wide vote, tensor memory is released.
#include "fp_internal.h"
#include "tc_common.cuh"

#include <cstdio>
#include <cstring>

namespace fp {

using namespace tc;

namespace {

constexpr int kBuildWarps = 8;             // compute warps; one more warp fetches the input, another issues the MMAs
constexpr int kThreads = 32 * (kBuildWarps + 2);
constexpr int kTaps = 16;                  // 4 x 4 taps over the parity channels, one K = 16 step each
constexpr int kRowsIn = 15, kConvRows = 5, kHalfRows = 8;
constexpr int kMaxTiles = 8;

struct SpParams {
    StemPoolArgs a;
    int Hc, Wc, Hp, Wp;            // convolution and pooled sizes
    int pitch;                     // elements per staged input row: W + 16
    int in_bytes;                  // one input buffer: C * 15 * pitch * 2
    int pitch_x;                   // half-resolution pixels per row of the parity form: Wc + 3 (columns -2 .. Wc)
    int x_rows;                    // 16-byte rows per chunk of a parity buffer (8 * pitch_x, plus what the last tile's taps reach)
    int b_bytes;                   // filters: 16 taps * 2 chunks * K_pad * 16
    int conv_pos;                  // 5 * Wc
    int tiles;                     // ceil(5 * pitch_x / 128)
    int units_per_image, n_units;  // Hp / 2 (rounded up); images x that
    int tmem_cols;
    FastDiv div_px, div_upi;
    int* status;
};

struct SpCtrl {
    uint64_t in_full[2];
    uint64_t in_empty[2];
    uint64_t b_full;
    uint64_t x_full[2];
    uint64_t tmem_free;
    uint64_t mma_done[kMaxTiles];
    uint32_t tmem_base;
    int abort_flag;
};

// The staged rows of a unit (C channels x 15 input rows, 8 zero elements on either side of a row) rewritten as the
// parity form: half-resolution row h (0..7) holds input rows 2h - 1 (parity 0; none for h = 0: zeros, its taps are zero)
// and 2h (parity 1) of the staged window, pixel jx (0 .. pitch_x - 1) the input columns 2 (jx - 2) and 2 (jx - 2) + 1 -
// one aligned 32-bit load per (row parity, channel) gives both column parities.  Channel (2a + b) C + c.
template <int C>
__device__ __forceinline__ void parity_rows(const unsigned short* in_buf, int pitch, uint4* x_buf, int x_rows, int pitch_x,
                                            FastDiv div_px, int tid) {
    const int total = kHalfRows * pitch_x;
    for (int i = tid; i < total; i += 32 * kBuildWarps) {
        const int h = (int)fdiv((uint32_t)i, div_px), jx = i - h * pitch_x;
        uint32_t hv[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) hv[e] = 0u;
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            const int r = 2 * h - 1 + a;
#pragma unroll
            for (int c = 0; c < C; ++c) {
                uint32_t pair = 0u;
                if (r >= 0) pair = *reinterpret_cast<const uint32_t*>(in_buf + (c * kRowsIn + r) * pitch + 4 + 2 * jx);
                hv[(2 * a) * C + c] = pair & 0xffffu;
                hv[(2 * a + 1) * C + c] = pair >> 16;
            }
        }
        x_buf[i] = make_uint4(hv[0] | (hv[1] << 16), hv[2] | (hv[3] << 16), hv[4] | (hv[5] << 16), hv[6] | (hv[7] << 16));
        x_buf[x_rows + i] = make_uint4(hv[8] | (hv[9] << 16), hv[10] | (hv[11] << 16), hv[12] | (hv[13] << 16), hv[14] | (hv[15] << 16));
    }
}

// barrier 1: the compute warps only (the input producer runs on its own)
__device__ __forceinline__ void bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(32 * kBuildWarps) : "memory"); }
__device__ __forceinline__ bool bar_or(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)pred), "n"(32 * kBuildWarps) : "memory");
    return r != 0;
}

__global__ void __launch_bounds__(kThreads) stem_pool_kernel(const SpParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    SpCtrl* ctrl = reinterpret_cast<SpCtrl*>(smem_raw);
    const uint32_t base = smem_u32(smem_raw);
    const uint32_t ctrl_bytes = (uint32_t)((sizeof(SpCtrl) + 127) & ~127u);
    float* bias_s = reinterpret_cast<float*>(smem_raw + ctrl_bytes);                         // K_pad floats
    const uint32_t b_addr = (base + ctrl_bytes + (uint32_t)p.a.K_pad * 4u + 1023u) & ~1023u;
    const uint32_t x_addr = b_addr + (uint32_t)((p.b_bytes + 127) & ~127);
    const uint32_t x_bytes = 2u * (uint32_t)p.x_rows * 16u;                                  // one parity buffer: two chunks
    const uint32_t in_addr = x_addr + 2u * x_bytes;
    const uint32_t conv_addr = in_addr + 2u * (uint32_t)p.in_bytes;
    uint8_t* in_ptr = smem_raw + (in_addr - base);
    uint8_t* conv_ptr = smem_raw + (conv_addr - base);
    uint8_t* x_ptr = smem_raw + (x_addr - base);
    volatile int* abort_flag = &ctrl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t in_full0 = base + (uint32_t)offsetof(SpCtrl, in_full);
    const uint32_t in_empty0 = base + (uint32_t)offsetof(SpCtrl, in_empty);
    const uint32_t b_full = base + (uint32_t)offsetof(SpCtrl, b_full);
    const uint32_t x_full0 = base + (uint32_t)offsetof(SpCtrl, x_full);
    const uint32_t tmem_free = base + (uint32_t)offsetof(SpCtrl, tmem_free);
    const uint32_t mma_done0 = base + (uint32_t)offsetof(SpCtrl, mma_done);
    const int C = p.a.C, K_pad = p.a.K_pad, chunks_out = K_pad >> 3;

    if (threadIdx.x == 0) {
        mbar_init(in_full0, 1); mbar_init(in_full0 + 8, 1);
        mbar_init(in_empty0, 32 * kBuildWarps); mbar_init(in_empty0 + 8, 32 * kBuildWarps);
        mbar_init(b_full, 1);
        mbar_init(x_full0, 32 * kBuildWarps); mbar_init(x_full0 + 8, 32 * kBuildWarps);
        mbar_init(tmem_free, 32 * kBuildWarps);
        for (int t = 0; t < kMaxTiles; ++t) mbar_init(mma_done0 + 8 * t, 1);
        ctrl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = threadIdx.x; i < K_pad; i += kThreads) bias_s[i] = p.a.bias[i];
    // the 16 bytes on either side of every staged row stay zero for the whole kernel: copies never touch them
    for (int i = threadIdx.x; i < 2 * C * kRowsIn; i += kThreads) {
        uint4* row = reinterpret_cast<uint4*>(in_ptr + (size_t)i * p.pitch * 2);
        row[0] = make_uint4(0, 0, 0, 0);
        row[(p.pitch * 2) / 16 - 1] = make_uint4(0, 0, 0, 0);
    }
    // the parity buffers' rows behind the eight half-resolution rows are read by the last tile's taps (for positions that
    // are dropped) and never written: zeros, so that no NaN pattern reaches an accumulator
    for (int i = threadIdx.x; i < (int)(2u * x_bytes / 16u); i += kThreads) reinterpret_cast<uint4*>(x_ptr)[i] = make_uint4(0, 0, 0, 0);
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + (uint32_t)offsetof(SpCtrl, tmem_base)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_base);

    // filters: resident for the whole kernel (the filters are not written by the previous kernel in the stream)
    if (threadIdx.x == 0) {
        mbar_expect_tx(b_full, (uint32_t)p.b_bytes);
        for (int off = 0; off < p.b_bytes; off += 16384) {
            const int n = p.b_bytes - off < 16384 ? p.b_bytes - off : 16384;
            bulk_copy(b_addr + off, reinterpret_cast<const uint8_t*>(p.a.w) + off, (uint32_t)n, b_full);
        }
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const uint8_t* xin = reinterpret_cast<const uint8_t*>(p.a.x);
    uint4* yout = reinterpret_cast<uint4*>(p.a.y);
    const int Wq = p.Wp + 2, P2o = (p.Hp + 2) * Wq;
    const long long plane_out = (long long)p.a.N * P2o;

    bool ok = true;

    if (warp == kBuildWarps) {
        // ------------------------------ input producer ------------------------------
        // Per unit: the fifteen input rows of every channel, one bulk copy per (channel, row) inside the image; rows
        // outside the image are cleared first (the arrival below publishes those stores to the waiting threads).
        uint32_t phase[2] = {0, 0};
        int it = 0;
        for (int u = blockIdx.x; u < p.n_units && ok; u += gridDim.x, ++it) {
            const int buf = it & 1;
            bool w = true;
            if (lane == 0) w = mbar_wait(in_empty0 + 8 * buf, phase[buf] ^ 1, abort_flag);
            phase[buf] ^= 1;
            w = __shfl_sync(0xffffffffu, w, 0);
            if (!w) { ok = false; break; }
            const int img = (int)fdiv((uint32_t)u, p.div_upi);
            const int pr = u - img * p.units_per_image;
            const int n = p.a.n0 + img;
            const int row0 = 8 * pr - 5;
            const int lo = row0 < 0 ? -row0 : 0, hi = row0 + kRowsIn > p.a.H ? p.a.H - row0 : kRowsIn;     // staged rows lo .. hi-1 exist
            const int per = hi - lo;
            if (per < kRowsIn) {
                const int vec_per_row = (p.pitch * 2) / 16;
                for (int i = lane; i < C * kRowsIn * vec_per_row; i += 32) {
                    const int r = (i / vec_per_row) % kRowsIn;
                    if (r < lo || r >= hi) reinterpret_cast<uint4*>(in_ptr + (size_t)buf * p.in_bytes)[i] = make_uint4(0, 0, 0, 0);
                }
            }
            __syncwarp();
            const uint32_t bar = in_full0 + 8 * buf;
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)(C * per * p.a.W * 2));
            __syncwarp();
            for (int i = lane; i < C * per; i += 32) {
                const int c = i / per, r = lo + (i - c * per);
                bulk_copy(in_addr + buf * p.in_bytes + (uint32_t)(((c * kRowsIn + r) * p.pitch + 8) * 2),
                          xin + (((long long)n * C + c) * p.a.H + (row0 + r)) * p.a.W * 2, (uint32_t)(p.a.W * 2), bar);
            }
        }
        if (!ok && lane == 0) { atomicExch(&ctrl->abort_flag, 1); atomicExch(p.status, 6); }
    } else if (warp == kBuildWarps + 1) {
        // ------------------------------ MMA issuer ------------------------------
        // One thread: waits until the compute threads have rewritten a unit's rows and have read the previous unit's
        // accumulators, then issues the unit's MMAs - per tile of 128 flat positions sixteen taps of one K = 16 step,
        // the operand of tap (ta, tb) starting ta * pitch + tb rows further on - and commits every tile to a barrier of
        // its own, so that the epilogue starts on the first tile while the others are computed.
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(K_pad >> 3) << 17) | ((128u >> 4) << 24);
            ok = mbar_wait(b_full, 0, abort_flag);
            int it = 0;
            for (int u = blockIdx.x; u < p.n_units && ok; u += gridDim.x, ++it) {
                const int xb = it & 1;
                if (!mbar_wait(x_full0 + 8 * xb, (uint32_t)((it >> 1) & 1), abort_flag)) { ok = false; break; }
                if (it > 0 && !mbar_wait(tmem_free, (uint32_t)((it - 1) & 1), abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_unit = ((x_addr + xb * x_bytes) >> 4) | ((uint32_t)p.x_rows << 16);
                const uint32_t b_lo0 = (b_addr >> 4) | ((uint32_t)K_pad << 16);
                for (int t = 0; t < p.tiles; ++t) {
                    const uint32_t d = tmem_base + (uint32_t)(t * K_pad);
                    uint32_t a_row = a_unit + (uint32_t)(t * 128);
                    uint32_t b_lo = b_lo0;
#pragma unroll
                    for (int ta = 0; ta < 4; ++ta) {
#pragma unroll
                        for (int tb = 0; tb < 4; ++tb) {
                            umma_bf16_lo(d, a_row + (uint32_t)tb, b_lo, idesc, (ta | tb) ? 1u : 0u);
                            b_lo += 2u * (uint32_t)K_pad;
                        }
                        a_row += (uint32_t)p.pitch_x;
                    }
                    umma_commit(mma_done0 + 8 * t);
                }
            }
            if (!ok) { atomicExch(&ctrl->abort_flag, 1); atomicExch(p.status, 6); }
        }
    } else {
    // ------------------------------ the eight compute warps ------------------------------
    {   // (every thread waits for the filters - cheap - so that the vote below is uniform)
        const bool w = mbar_wait(b_full, 0, abort_flag);
        ok = !bar_or(!w);
    }
    uint32_t in_phase[2] = {0, 0};
    // rewrites the staged rows of the CTA's unit number `it` into parity buffer it & 1 and hands both on
    auto rewrite = [&](int it) -> bool {
        const int buf = it & 1;
        const bool w = mbar_wait(in_full0 + 8 * buf, in_phase[buf], abort_flag);
        in_phase[buf] ^= 1;
        if (bar_or(!w)) return false;
        const unsigned short* in_buf = reinterpret_cast<const unsigned short*>(in_ptr + (size_t)buf * p.in_bytes);
        uint4* x_buf = reinterpret_cast<uint4*>(x_ptr + (size_t)buf * x_bytes);
        if (C == 3) parity_rows<3>(in_buf, p.pitch, x_buf, p.x_rows, p.pitch_x, p.div_px, threadIdx.x);
        else if (C == 2) parity_rows<2>(in_buf, p.pitch, x_buf, p.x_rows, p.pitch_x, p.div_px, threadIdx.x);
        else parity_rows<1>(in_buf, p.pitch, x_buf, p.x_rows, p.pitch_x, p.div_px, threadIdx.x);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> MMA reads
        mbar_arrive(x_full0 + 8 * buf);
        mbar_arrive(in_empty0 + 8 * buf);                              // the staged rows are free for the unit after the next
        return true;
    };
    int it = 0;
    if (blockIdx.x < p.n_units) ok = ok && rewrite(0);
    for (int u = blockIdx.x; u < p.n_units && ok; u += gridDim.x, ++it) {
        const int img = (int)fdiv((uint32_t)u, p.div_upi);
        const int pr = u - img * p.units_per_image;
        const int n = p.a.n0 + img;
        // the next unit's rows first: its MMAs then run while this unit is pooled
        if (u + (int)gridDim.x < p.n_units && !rewrite(it + 1)) { ok = false; break; }

        // ---- epilogue 1: accumulators -> bias, ReLU, bf16 -> the unit's convolution rows in shared memory ----
        {
            const int quarter = warp & 3, half = warp >> 2;      // TMEM lanes 32 * quarter ..; the 16-column groups alternate between the two halves
            bool w = true;
            for (int t = 0; t < p.tiles; ++t) {
                if (w) w = __all_sync(0xffffffffu, mbar_wait(mma_done0 + 8 * t, (uint32_t)(it & 1), abort_flag));
                if (!w) continue;                                // (warp-uniform) the vote below takes everybody out together
                tc_fence_after();
                const int m = t * 128 + quarter * 32 + lane;
                const int j = (int)fdiv((uint32_t)m, p.div_px), q = m - j * p.pitch_x;
                const bool pos = j < kConvRows && q < p.Wc;      // the pad columns and the rows behind the fifth are dropped
                const int hc = 4 * pr - 1 + j;
                const bool live = pos && hc >= 0 && hc < p.Hc;
                uint32_t v[3][16];                               // this warp's column groups of the tile (K_pad <= 96): one wait for all
                __syncwarp();
#pragma unroll
                for (int g = 0; g < 3; ++g) {
                    const int c0 = 16 * half + 32 * g;
                    if (c0 < K_pad) tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(t * K_pad + c0), v[g]);
                }
                tmem_ld_wait();
                if (pos) {
                    const int idx = j * p.Wc + q;
#pragma unroll
                    for (int g = 0; g < 3; ++g) {
                        const int c0 = 16 * half + 32 * g;
                        if (c0 < K_pad) {
                            uint4 o[2];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const float f0 = live ? __uint_as_float(v[g][2 * i]) + bias_s[c0 + 2 * i] : 0.0f;
                                const float f1 = live ? __uint_as_float(v[g][2 * i + 1]) + bias_s[c0 + 2 * i + 1] : 0.0f;
                                reinterpret_cast<uint32_t*>(o)[i] = pack_bf16x2_relu(f0, f1);
                            }
                            uint4* dst = reinterpret_cast<uint4*>(conv_ptr) + (size_t)(c0 >> 3) * p.conv_pos + idx;
                            dst[0] = o[0];
                            dst[p.conv_pos] = o[1];
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(tmem_free);                              // the accumulators may be overwritten by the next unit's MMAs
            if (bar_or(!w)) { ok = false; break; }               // (also: the convolution rows are complete)
        }

        // ---- epilogue 2: 3x3 / 2 maxima of the two pooled rows, border columns included; border rows at the image's ends ----
        {
            // A lane takes one convolution column: the maxima down rows 0-2 and 2-4 (five 16-byte loads, conflict-free),
            // then across the three columns of a window with shuffles; the even lanes hold the pooled columns.
            const uint4* cv = reinterpret_cast<const uint4*>(conv_ptr);
            const int rows_here = (2 * pr + 1 < p.Hp) ? 2 : 1;
            for (int ch = warp; ch < chunks_out; ch += kBuildWarps) {
                const uint4* cplane = cv + (size_t)ch * p.conv_pos;
                uint4* ybase = yout + (long long)ch * plane_out + (long long)n * P2o + (long long)(2 * pr + 1) * Wq;
                // 30 new columns per turn: lane l holds column w_start - 1 + l, windows are centred on the even columns
                for (int w_start = 0; w_start < p.Wc; w_start += 30) {
                    const int wc = w_start - 1 + lane;
                    const bool in = wc >= 0 && wc < p.Wc;
                    __nv_bfloat162 top[4], bot[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) top[e] = bot[e] = __floats2bfloat162_rn(0.0f, 0.0f);
                    if (in) {
                        uint4 r[5];
#pragma unroll
                        for (int j = 0; j < 5; ++j) r[j] = cplane[j * p.Wc + wc];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const __nv_bfloat162 mid = reinterpret_cast<const __nv_bfloat162*>(&r[2])[e];
                            top[e] = __hmax2(__hmax2(reinterpret_cast<const __nv_bfloat162*>(&r[0])[e], reinterpret_cast<const __nv_bfloat162*>(&r[1])[e]), mid);
                            bot[e] = __hmax2(__hmax2(reinterpret_cast<const __nv_bfloat162*>(&r[3])[e], reinterpret_cast<const __nv_bfloat162*>(&r[4])[e]), mid);
                        }
                    }
                    // columns outside the image hold zeros, below every post-ReLU value
                    uint32_t tv[4], bv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint32_t t0 = *reinterpret_cast<uint32_t*>(&top[e]), b0 = *reinterpret_cast<uint32_t*>(&bot[e]);
                        uint32_t tl = __shfl_up_sync(0xffffffffu, t0, 1), tr = __shfl_down_sync(0xffffffffu, t0, 1);
                        uint32_t bl = __shfl_up_sync(0xffffffffu, b0, 1), br = __shfl_down_sync(0xffffffffu, b0, 1);
                        __nv_bfloat162 tm = __hmax2(top[e], __hmax2(*reinterpret_cast<__nv_bfloat162*>(&tl), *reinterpret_cast<__nv_bfloat162*>(&tr)));
                        __nv_bfloat162 bm = __hmax2(bot[e], __hmax2(*reinterpret_cast<__nv_bfloat162*>(&bl), *reinterpret_cast<__nv_bfloat162*>(&br)));
                        tv[e] = *reinterpret_cast<uint32_t*>(&tm);
                        bv[e] = *reinterpret_cast<uint32_t*>(&bm);
                    }
                    // lanes 1 .. 30 hold complete windows; the even columns among them are pooled columns q = wc / 2
                    if (lane >= 1 && lane <= 30 && in && (wc & 1) == 0) {
                        const int q = wc >> 1;
                        ybase[q + 1] = make_uint4(tv[0], tv[1], tv[2], tv[3]);
                        if (rows_here == 2) ybase[Wq + q + 1] = make_uint4(bv[0], bv[1], bv[2], bv[3]);
                    }
                }
                // border columns of the two rows, border rows at the image's ends
                if (lane < 2) {
                    const int qq = lane == 0 ? 0 : Wq - 1;
                    ybase[qq] = make_uint4(0, 0, 0, 0);
                    if (rows_here == 2) ybase[Wq + qq] = make_uint4(0, 0, 0, 0);
                }
                if (pr == 0 || pr == p.units_per_image - 1) {
                    uint4* ytop = yout + (long long)ch * plane_out + (long long)n * P2o;
                    for (int qq = lane; qq < Wq; qq += 32) {
                        if (pr == 0) ytop[qq] = make_uint4(0, 0, 0, 0);
                        if (pr == p.units_per_image - 1) ytop[(long long)(p.Hp + 1) * Wq + qq] = make_uint4(0, 0, 0, 0);
                    }
                }
            }
        }
        bar_sync();               // the convolution rows are free again
    }
    if (!ok && threadIdx.x == 0) { atomicExch(&ctrl->abort_flag, 1); atomicExch(p.status, 6); }
    }


    // ---- teardown ----
    if (!ok) {
        // give copies that are still in flight time to land before shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

constexpr unsigned kSmemMax = 232448u - 1024u;

int pow2_at_least(int v) { int p = 32; while (p < v) p <<= 1; return p; }

}  // namespace

// shared memory of the kernel for one shape, and its tile count / parity-buffer rows
static unsigned stem_pool_smem(int C, int W, int K_pad, int* tiles_out, int* x_rows_out) {
    const int Wc = W / 2, pitch_x = Wc + 3;
    const int tiles = (kConvRows * pitch_x + 127) / 128;
    const int x_rows = (tiles * 128 + 3 * pitch_x + 3 + 7) & ~7;
    if (tiles_out) *tiles_out = tiles;
    if (x_rows_out) *x_rows_out = x_rows;
    const unsigned ctrl = (unsigned)((sizeof(SpCtrl) + 127) & ~127u);
    return ctrl + (unsigned)K_pad * 4u + 1024u + (unsigned)((kTaps * 2 * K_pad * 16 + 127) & ~127) + 2u * (unsigned)(2 * x_rows * 16) +
           2u * (unsigned)(C * kRowsIn * (W + 16) * 2) + (unsigned)((K_pad / 8) * kConvRows * Wc * 16);
}

bool stem_pool_supported(int C, int H, int W, int K_pad) {
    if (C < 1 || C > 3 || H % 4 || W % 8 || H < 8 || W < 8 || K_pad % 16 || K_pad < 16 || K_pad > 96) return false;
    int tiles = 0, x_rows = 0;
    const unsigned smem = stem_pool_smem(C, W, K_pad, &tiles, &x_rows);
    if (tiles > kMaxTiles || tiles * K_pad > 512) return false;
    return smem <= kSmemMax;
}

int plan_stem_pool(const StemPoolArgs& a, StemPoolPlan* plan, char* err, size_t err_len) {
    memset(plan, 0, sizeof(*plan));
    if (!stem_pool_supported(a.C, a.H, a.W, a.K_pad)) { snprintf(err, err_len, "first convolution + pooling: shape not supported"); return 1; }
    int x_rows = 0;
    plan->smem_bytes = stem_pool_smem(a.C, a.W, a.K_pad, &plan->tiles, &x_rows);
    plan->tmem_cols = pow2_at_least(plan->tiles * a.K_pad);
    if (cudaFuncSetAttribute(stem_pool_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax) != cudaSuccess) {
        snprintf(err, err_len, "cannot raise the dynamic shared memory limit");
        cudaGetLastError();
        return 1;
    }
    plan->valid = 1;
    return 0;
}

void launch_stem_pool(const StemPoolPlan& plan, const StemPoolArgs& a, int* d_status, cudaStream_t st) {
    SpParams p;
    memset(&p, 0, sizeof(p));
    p.a = a;
    p.Hc = a.H / 2; p.Wc = a.W / 2; p.Hp = p.Hc / 2; p.Wp = p.Wc / 2;
    p.pitch = a.W + 16;
    p.in_bytes = a.C * kRowsIn * p.pitch * 2;
    p.pitch_x = p.Wc + 3;
    stem_pool_smem(a.C, a.W, a.K_pad, nullptr, &p.x_rows);
    p.b_bytes = kTaps * 2 * a.K_pad * 16;
    p.conv_pos = kConvRows * p.Wc;
    p.tiles = plan.tiles;
    p.units_per_image = (p.Hp + 1) / 2;
    p.n_units = a.n_count * p.units_per_image;
    p.tmem_cols = plan.tmem_cols;
    p.div_px = make_fastdiv((uint32_t)p.pitch_x);
    p.div_upi = make_fastdiv((uint32_t)p.units_per_image);
    p.status = d_status;
    int grid = sm_count();
    if (grid > p.n_units) grid = p.n_units;
    if (grid < 1) grid = 1;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)kThreads);
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    void* args[1] = {(void*)&p};
    cudaLaunchKernelExC(&cfg, (const void*)stem_pool_kernel, args);
}

}  // namespace fp
