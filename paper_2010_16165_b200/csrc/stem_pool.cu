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
//   GEMM           M = the unit's 5 x (W/2) convolution positions in tiles of 128, N = K_pad filters, K = 49 C taps
//                  padded to 160.  All threads build a tile's A operand (K-major, 16-byte rows: 8 consecutive k of one
//                  position) from the staged rows through a table of offsets, two A buffers, one thread issues the
//                  tcgen05 MMAs; the five accumulators stay in tensor memory until the unit's last MMA.
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
constexpr int kKChunks = 20;               // K = 160 >= 49 * 3
constexpr int kRowsIn = 15, kConvRows = 5;

struct SpParams {
    StemPoolArgs a;
    int Hc, Wc, Hp, Wp;            // convolution and pooled sizes
    int pitch;                     // elements per staged input row: W + 16
    int in_bytes;                  // one input buffer: C * 15 * pitch * 2
    int a_bytes;                   // one A tile: 20 * 128 * 16
    int b_bytes;                   // filters: 20 * K_pad * 16
    int conv_pos;                  // 5 * Wc
    int tiles;                     // ceil(conv_pos / 128)
    int units_per_image, n_units;  // Hp / 2 (rounded up); images x that
    int tmem_cols;
    FastDiv div_wc, div_upi, div_wp2;
    int* status;
};

struct SpCtrl {
    uint64_t in_full[2];
    uint64_t in_empty[2];
    uint64_t b_full;
    uint64_t mma_done[2];
    uint64_t a_full[2];
    uint32_t tmem_base;
    int abort_flag;
    int koff[kKChunks * 8];        // k -> element offset of tap (r, s, c) from a position's window origin
};

// A position's 147 taps for three input channels, k = (r * 3 + c) * 7 + s, as the K-major operand rows of one half
// (k in [80 HALF, 80 HALF + 80)) of its 160 k.  The window of a (row, channel) starts at an odd element (column 2w - 3
// behind 8 elements of padding), so its element 0 is a 16-bit load and (1,2), (3,4), (5,6) are aligned 32-bit loads: 84
// shared-memory loads per position instead of 147 - the builder is bound by the load/store unit's issue rate.
// Everything is unrolled: which loads a half needs and where their halves go are compile-time facts.
template <int HALF>
__device__ __forceinline__ void build_rgb(const unsigned short* origin, int pitch, uint4* a_dst) {
    uint32_t wd[40];
#pragma unroll
    for (int i = 0; i < 40; ++i) wd[i] = 0u;
#pragma unroll
    for (int rc = 0; rc < 21; ++rc) {
        const int k0 = rc * 7;                               // k of this window's element 0
        if (k0 + 6 < 80 * HALF || k0 >= 80 * HALF + 80) continue;
        const int r = rc / 3, c = rc - 3 * r;
        const unsigned short* wdw = origin + (c * kRowsIn + r) * pitch;
        uint32_t e[7];
        const bool need0 = k0 >= 80 * HALF && k0 < 80 * HALF + 80;
        if (need0) e[0] = wdw[0];
#pragma unroll
        for (int pr = 0; pr < 3; ++pr) {
            const int ka = k0 + 1 + 2 * pr, kb = ka + 1;
            const bool na = ka >= 80 * HALF && ka < 80 * HALF + 80, nb = kb >= 80 * HALF && kb < 80 * HALF + 80;
            if (na || nb) {
                const uint32_t pair = *reinterpret_cast<const uint32_t*>(wdw + 1 + 2 * pr);
                e[1 + 2 * pr] = pair & 0xffffu;
                e[2 + 2 * pr] = pair >> 16;
            }
        }
#pragma unroll
        for (int sx = 0; sx < 7; ++sx) {
            const int k = k0 + sx;
            if (k >= 80 * HALF && k < 80 * HALF + 80) {
                const int kk = k - 80 * HALF;
                wd[kk >> 1] |= (kk & 1) ? (e[sx] << 16) : e[sx];
            }
        }
    }
#pragma unroll
    for (int cc = 0; cc < 10; ++cc)
        a_dst[(10 * HALF + cc) * 128] = make_uint4(wd[4 * cc], wd[4 * cc + 1], wd[4 * cc + 2], wd[4 * cc + 3]);
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
    const uint32_t a_addr = b_addr + (uint32_t)((p.b_bytes + 127) & ~127);
    const uint32_t in_addr = a_addr + 2u * (uint32_t)p.a_bytes;
    const uint32_t conv_addr = in_addr + 2u * (uint32_t)p.in_bytes;
    uint8_t* in_ptr = smem_raw + (in_addr - base);
    uint8_t* conv_ptr = smem_raw + (conv_addr - base);
    volatile int* abort_flag = &ctrl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t in_full0 = base + (uint32_t)offsetof(SpCtrl, in_full);
    const uint32_t b_full = base + (uint32_t)offsetof(SpCtrl, b_full);
    const uint32_t mma_done0 = base + (uint32_t)offsetof(SpCtrl, mma_done);
    const int C = p.a.C, K_pad = p.a.K_pad, chunks_out = K_pad >> 3;

    if (threadIdx.x == 0) {
        mbar_init(in_full0, 1); mbar_init(in_full0 + 8, 1);
        mbar_init(base + (uint32_t)offsetof(SpCtrl, in_empty), 1); mbar_init(base + (uint32_t)offsetof(SpCtrl, in_empty) + 8, 1);
        mbar_init(b_full, 1);
        mbar_init(mma_done0, 1); mbar_init(mma_done0 + 8, 1);
        mbar_init(base + (uint32_t)offsetof(SpCtrl, a_full), 32 * kBuildWarps); mbar_init(base + (uint32_t)offsetof(SpCtrl, a_full) + 8, 32 * kBuildWarps);
        ctrl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int k = threadIdx.x; k < kKChunks * 8; k += kThreads) {
        int off = 0;
        if (k < 49 * C) {
            const int rc = k / 7, s = k - rc * 7, r = rc / C, c = rc - r * C;
            off = (c * kRowsIn + r) * p.pitch + s;
        }
        ctrl->koff[k] = off;
    }
    for (int i = threadIdx.x; i < K_pad; i += kThreads) bias_s[i] = p.a.bias[i];
    // the 16 bytes on either side of every staged row stay zero for the whole kernel: copies never touch them
    for (int i = threadIdx.x; i < 2 * C * kRowsIn; i += kThreads) {
        uint4* row = reinterpret_cast<uint4*>(in_ptr + (size_t)i * p.pitch * 2);
        row[0] = make_uint4(0, 0, 0, 0);
        row[(p.pitch * 2) / 16 - 1] = make_uint4(0, 0, 0, 0);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + (uint32_t)offsetof(SpCtrl, tmem_base)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
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

    const uint32_t in_empty0 = base + (uint32_t)offsetof(SpCtrl, in_empty);
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
        // One thread: waits until every compute thread has stored its part of a tile's operand, issues the tile's MMAs and
        // commits them to the barrier that frees the operand buffer (and, behind a unit's last tile, tells the compute
        // warps that the accumulators are complete).  A thread of its own, so that the compute warps go on building.
        if (lane == 0) {
            const uint32_t a_full0 = base + (uint32_t)offsetof(SpCtrl, a_full);
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(K_pad >> 3) << 17) | ((128u >> 4) << 24);
            uint32_t full_phase[2] = {0, 0};
            ok = mbar_wait(b_full, 0, abort_flag);
            int it = 0;
            for (int u = blockIdx.x; u < p.n_units && ok; u += gridDim.x, ++it) {
                for (int t = 0; t < p.tiles; ++t) {
                    const int ab = t & 1;
                    if (!mbar_wait(a_full0 + 8 * ab, full_phase[ab], abort_flag)) { ok = false; break; }
                    full_phase[ab] ^= 1;
                    tc_fence_after();
                    uint32_t a_lo = ((a_addr + ab * p.a_bytes) >> 4) | (128u << 16);
                    uint32_t b_lo = (b_addr >> 4) | ((uint32_t)K_pad << 16);
                    const uint32_t d = tmem_base + (uint32_t)(t * K_pad);
#pragma unroll
                    for (int ks = 0; ks < kKChunks / 2; ++ks) {
                        umma_bf16_lo(d, a_lo, b_lo, idesc, ks ? 1u : 0u);
                        a_lo += 256u;
                        b_lo += 2u * (uint32_t)K_pad;
                    }
                    umma_commit(mma_done0 + 8 * ab);
                    // the last tile has been built: the staged input rows are free for the unit after the next
                    if (t == p.tiles - 1) mbar_arrive(in_empty0 + 8 * (it & 1));
                }
            }
            if (!ok) { atomicExch(&ctrl->abort_flag, 1); atomicExch(p.status, 6); }
        }
    } else {
    // ------------------------------ the eight compute warps ------------------------------
    {   // filters have to be in before the first MMA; every thread waits (cheap) so that the vote below is uniform
        const bool w = mbar_wait(b_full, 0, abort_flag);
        ok = !bar_or(!w);
    }
    uint32_t in_phase[2] = {0, 0}, mma_phase[2] = {0, 0};
    int it = 0;
    for (int u = blockIdx.x; u < p.n_units && ok; u += gridDim.x, ++it) {
        const int buf = it & 1;
        const int img = (int)fdiv((uint32_t)u, p.div_upi);
        const int pr = u - img * p.units_per_image;
        const int n = p.a.n0 + img;
        {
            const bool w = mbar_wait(in_full0 + 8 * buf, in_phase[buf], abort_flag);
            in_phase[buf] ^= 1;
            if (bar_or(!w)) { ok = false; break; }
        }
        const uint32_t in_buf = in_addr + buf * p.in_bytes;

        // ---- convolution: build A tile by tile, MMAs behind ----
        for (int t = 0; t < p.tiles; ++t) {
            const int ab = t & 1;
            bool w = true;
            if (t >= 2) { w = mbar_wait(mma_done0 + 8 * ab, mma_phase[ab], abort_flag); mma_phase[ab] ^= 1; }
            const int m = t * 128 + (threadIdx.x & 127);
            if (w && m < p.conv_pos) {
                const int j = (int)fdiv((uint32_t)m, p.div_wc), wc = m - j * p.Wc;
                const unsigned short* origin = reinterpret_cast<const unsigned short*>(smem_raw + (in_buf - base)) +
                                               ((2 * j) * p.pitch + 8 + 2 * wc - 3);
                const int c0 = (threadIdx.x >> 7) * (kKChunks / 2);
                uint4* a_dst = reinterpret_cast<uint4*>(smem_raw + (a_addr - base) + ab * p.a_bytes) + (threadIdx.x & 127);
                if (C == 3) {
                    if (threadIdx.x < 128) build_rgb<0>(origin, p.pitch, a_dst);
                    else build_rgb<1>(origin, p.pitch, a_dst);
                } else {
                    // all loads first, then all stores: the stores could alias the loads for all the compiler knows, and
                    // interleaved they would leave one 16-byte group's loads in flight at a time
                    uint4 v[kKChunks / 2];
#pragma unroll
                    for (int cc = 0; cc < kKChunks / 2; ++cc) {
                        const int ch = c0 + cc;
                        const int4 o0 = *reinterpret_cast<const int4*>(&ctrl->koff[ch * 8]);
                        const int4 o1 = *reinterpret_cast<const int4*>(&ctrl->koff[ch * 8 + 4]);
                        v[cc].x = (uint32_t)origin[o0.x] | ((uint32_t)origin[o0.y] << 16);
                        v[cc].y = (uint32_t)origin[o0.z] | ((uint32_t)origin[o0.w] << 16);
                        v[cc].z = (uint32_t)origin[o1.x] | ((uint32_t)origin[o1.y] << 16);
                        v[cc].w = (uint32_t)origin[o1.z] | ((uint32_t)origin[o1.w] << 16);
                    }
#pragma unroll
                    for (int cc = 0; cc < kKChunks / 2; ++cc) a_dst[(c0 + cc) * 128] = v[cc];
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> MMA reads
            if (!w) { atomicExch(&ctrl->abort_flag, 1); ok = false; break; }     // the vote after the last tile takes everybody out together
            mbar_arrive(base + (uint32_t)offsetof(SpCtrl, a_full) + 8 * ab);
        }
        {   // the last two tiles' commits (a unit of one tile has only one)
            bool w = ok;
            for (int t = p.tiles >= 2 ? p.tiles - 2 : 0; t < p.tiles && w; ++t) {
                const int ab = t & 1;
                w = mbar_wait(mma_done0 + 8 * ab, mma_phase[ab], abort_flag);
                mma_phase[ab] ^= 1;
            }
            if (bar_or(!w)) { ok = false; break; }
            tc_fence_after();
        }

        // ---- epilogue 1: accumulators -> bias, ReLU, bf16 -> the unit's convolution rows in shared memory ----
        {
            const int quarter = warp & 3, half = warp >> 2;      // TMEM lanes 32 * quarter ..; the 16-column groups alternate between the two halves
            for (int t = 0; t < p.tiles; ++t) {
                const int m = t * 128 + quarter * 32 + lane;
                const int j = (int)fdiv((uint32_t)(m < p.conv_pos ? m : 0), p.div_wc);
                const int hc = 4 * pr - 1 + j;
                const bool live = m < p.conv_pos && hc >= 0 && hc < p.Hc;
                uint32_t v[3][16];                               // this warp's column groups of the tile (K_pad <= 96): one wait for all
                __syncwarp();
#pragma unroll
                for (int g = 0; g < 3; ++g) {
                    const int c0 = 16 * half + 32 * g;
                    if (c0 < K_pad) tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(t * K_pad + c0), v[g]);
                }
                tmem_ld_wait();
                if (m < p.conv_pos) {
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
                            uint4* dst = reinterpret_cast<uint4*>(conv_ptr) + (size_t)(c0 >> 3) * p.conv_pos + m;
                            dst[0] = o[0];
                            dst[p.conv_pos] = o[1];
                        }
                    }
                }
            }
            tc_fence_before();
        }
        bar_sync();

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

bool stem_pool_supported(int C, int H, int W, int K_pad) {
    if (C < 1 || C > 3 || H % 4 || W % 8 || H < 8 || W < 8 || K_pad % 16 || K_pad < 16) return false;
    const int Wc = W / 2, tiles = (kConvRows * Wc + 127) / 128;
    if (tiles * K_pad > 512) return false;
    const unsigned smem = 1024u + 512u + (unsigned)K_pad * 4u + 1024u + (unsigned)(kKChunks * K_pad * 16 + 128) +
                          2u * (unsigned)(kKChunks * 128 * 16) + 2u * (unsigned)(C * kRowsIn * (W + 16) * 2) +
                          (unsigned)((K_pad / 8) * kConvRows * Wc * 16);
    return smem <= kSmemMax;
}

int plan_stem_pool(const StemPoolArgs& a, StemPoolPlan* plan, char* err, size_t err_len) {
    memset(plan, 0, sizeof(*plan));
    if (!stem_pool_supported(a.C, a.H, a.W, a.K_pad)) { snprintf(err, err_len, "first convolution + pooling: shape not supported"); return 1; }
    const int Wc = a.W / 2;
    plan->tiles = (kConvRows * Wc + 127) / 128;
    plan->tmem_cols = pow2_at_least(plan->tiles * a.K_pad);
    const unsigned ctrl = (unsigned)((sizeof(SpCtrl) + 127) & ~127u);
    plan->smem_bytes = ctrl + (unsigned)a.K_pad * 4u + 1024u + (unsigned)((kKChunks * a.K_pad * 16 + 127) & ~127) +
                       2u * (unsigned)(kKChunks * 128 * 16) + 2u * (unsigned)(a.C * kRowsIn * (a.W + 16) * 2) +
                       (unsigned)((a.K_pad / 8) * kConvRows * Wc * 16);
    if (plan->smem_bytes > kSmemMax) { snprintf(err, err_len, "first convolution + pooling does not fit shared memory"); return 1; }
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
    p.a_bytes = kKChunks * 128 * 16;
    p.b_bytes = kKChunks * a.K_pad * 16;
    p.conv_pos = kConvRows * p.Wc;
    p.tiles = plan.tiles;
    p.units_per_image = (p.Hp + 1) / 2;
    p.n_units = a.n_count * p.units_per_image;
    p.tmem_cols = plan.tmem_cols;
    p.div_wc = make_fastdiv((uint32_t)p.Wc);
    p.div_upi = make_fastdiv((uint32_t)p.units_per_image);
    p.div_wp2 = make_fastdiv((uint32_t)(p.Wp + 2));
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
