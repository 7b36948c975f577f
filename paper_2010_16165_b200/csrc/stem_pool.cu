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

constexpr int kThreads = 256;
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
    uint64_t b_full;
    uint64_t mma_done[2];
    uint32_t tmem_base;
    int abort_flag;
    int koff[kKChunks * 8];        // k -> element offset of tap (r, s, c) from a position's window origin
};

__device__ __forceinline__ uint32_t ld_shared_u16(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
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
        mbar_init(b_full, 1);
        mbar_init(mma_done0, 1); mbar_init(mma_done0 + 8, 1);
        ctrl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int k = threadIdx.x; k < kKChunks * 8; k += kThreads) {
        int off = 0;
        if (k < 49 * C) {
            const int r = k / (7 * C), rem = k - r * 7 * C, s = rem / C, c = rem - s * C;
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

    // requests the fifteen input rows of every channel for unit `u` into buffer `buf` (warp 0, one copy per lane and turn),
    // rows inside the image only
    auto request = [&](int u, int buf) {
        const int img = (int)fdiv((uint32_t)u, p.div_upi);
        const int pr = u - img * p.units_per_image;
        const int n = p.a.n0 + img;
        const int row0 = 8 * pr - 5;
        const int lo = row0 < 0 ? -row0 : 0, hi = row0 + kRowsIn > p.a.H ? p.a.H - row0 : kRowsIn;     // staged rows lo .. hi-1 exist
        const int per = hi - lo;
        const uint32_t bar = in_full0 + 8 * buf;
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)(C * per * p.a.W * 2));
        __syncwarp();
        for (int i = lane; i < C * per; i += 32) {
            const int c = i / per, r = lo + (i - c * per);
            bulk_copy(in_addr + buf * p.in_bytes + (uint32_t)(((c * kRowsIn + r) * p.pitch + 8) * 2),
                      xin + (((long long)n * C + c) * p.a.H + (row0 + r)) * p.a.W * 2, (uint32_t)(p.a.W * 2), bar);
        }
    };
    // staged rows of unit `u` that lie outside the image: cleared by all threads (no copy writes them)
    auto clear_outside = [&](int u, int buf) {
        const int img = (int)fdiv((uint32_t)u, p.div_upi);
        const int pr = u - img * p.units_per_image;
        const int row0 = 8 * pr - 5;
        if (row0 >= 0 && row0 + kRowsIn <= p.a.H) return;
        const int vec_per_row = (p.pitch * 2) / 16;
        for (int i = threadIdx.x; i < C * kRowsIn * vec_per_row; i += kThreads) {
            const int cr = i / vec_per_row, r = cr % kRowsIn;
            if (row0 + r < 0 || row0 + r >= p.a.H)
                reinterpret_cast<uint4*>(in_ptr + (size_t)buf * p.in_bytes)[i] = make_uint4(0, 0, 0, 0);
        }
    };

    bool ok = true;
    const int first = blockIdx.x;
    if (first < p.n_units) {
        clear_outside(first, 0);
        if (warp == 0) request(first, 0);
    }
    {   // filters have to be in before the first MMA; every thread waits (cheap) so that the vote below is uniform
        const bool w = mbar_wait(b_full, 0, abort_flag);
        ok = !__syncthreads_or(!w);
    }
    uint32_t in_phase[2] = {0, 0}, mma_phase[2] = {0, 0};
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(K_pad >> 3) << 17) | ((128u >> 4) << 24);
    int it = 0;
    for (int u = first; u < p.n_units && ok; u += gridDim.x, ++it) {
        const int buf = it & 1;
        const int img = (int)fdiv((uint32_t)u, p.div_upi);
        const int pr = u - img * p.units_per_image;
        const int n = p.a.n0 + img;
        // the other input buffer was last read while the previous unit's tiles were built: free since the barrier
        // that ended that unit
        const int un = u + gridDim.x;
        if (un < p.n_units) {
            clear_outside(un, buf ^ 1);
            if (warp == 0) request(un, buf ^ 1);
        }
        {
            const bool w = mbar_wait(in_full0 + 8 * buf, in_phase[buf], abort_flag);
            in_phase[buf] ^= 1;
            if (__syncthreads_or(!w)) { ok = false; break; }      // also makes the cleared rows visible to everybody
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
                const uint32_t origin = in_buf + (uint32_t)(((2 * j) * p.pitch + 8 + 2 * wc - 3) * 2);
                const int c0 = (threadIdx.x >> 7) * (kKChunks / 2);
                for (int ch = c0; ch < c0 + kKChunks / 2; ++ch) {
                    const int4 o0 = *reinterpret_cast<const int4*>(&ctrl->koff[ch * 8]);
                    const int4 o1 = *reinterpret_cast<const int4*>(&ctrl->koff[ch * 8 + 4]);
                    uint4 v;
                    v.x = ld_shared_u16(origin + 2 * o0.x) | (ld_shared_u16(origin + 2 * o0.y) << 16);
                    v.y = ld_shared_u16(origin + 2 * o0.z) | (ld_shared_u16(origin + 2 * o0.w) << 16);
                    v.z = ld_shared_u16(origin + 2 * o1.x) | (ld_shared_u16(origin + 2 * o1.y) << 16);
                    v.w = ld_shared_u16(origin + 2 * o1.z) | (ld_shared_u16(origin + 2 * o1.w) << 16);
                    *reinterpret_cast<uint4*>(smem_raw + (a_addr - base) + ab * p.a_bytes + (ch * 128 + (threadIdx.x & 127)) * 16) = v;
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> MMA reads
            if (__syncthreads_or(!w)) { ok = false; break; }
            if (threadIdx.x == 0) {
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
            }
        }
        if (!ok) break;
        {   // the last two tiles' commits (a unit of one tile has only one)
            bool w = true;
            for (int t = p.tiles >= 2 ? p.tiles - 2 : 0; t < p.tiles; ++t) {
                const int ab = t & 1;
                w = w && mbar_wait(mma_done0 + 8 * ab, mma_phase[ab], abort_flag);
                mma_phase[ab] ^= 1;
            }
            if (__syncthreads_or(!w)) { ok = false; break; }
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
                for (int c0 = 16 * half; c0 < K_pad; c0 += 32) {
                    uint32_t v[16];
                    __syncwarp();
                    tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(t * K_pad + c0), v);
                    tmem_ld_wait();
                    if (m < p.conv_pos) {
                        uint4 o[2];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float f0 = live ? __uint_as_float(v[2 * i]) + bias_s[c0 + 2 * i] : 0.0f;
                            const float f1 = live ? __uint_as_float(v[2 * i + 1]) + bias_s[c0 + 2 * i + 1] : 0.0f;
                            reinterpret_cast<uint32_t*>(o)[i] = pack_bf16x2_relu(f0, f1);
                        }
                        uint4* dst = reinterpret_cast<uint4*>(conv_ptr) + (size_t)(c0 >> 3) * p.conv_pos + m;
                        dst[0] = o[0];
                        dst[p.conv_pos] = o[1];
                    }
                }
            }
            tc_fence_before();
        }
        __syncthreads();

        // ---- epilogue 2: 3x3 / 2 maxima of the two pooled rows, border columns included; border rows at the image's ends ----
        {
            const uint4* cv = reinterpret_cast<const uint4*>(conv_ptr);
            const int rows_here = (2 * pr + 1 < p.Hp) ? 2 : 1;
            const int items = chunks_out * rows_here * Wq;
            for (int i = threadIdx.x; i < items; i += kThreads) {
                const int ch = (int)fdiv((uint32_t)i, p.div_wp2) / rows_here;      // i = (ch * rows_here + pl) * Wq + qq
                const int rest = i - ch * rows_here * Wq;
                const int pl = rest >= Wq ? 1 : 0, qq = rest - pl * Wq;
                const int q = qq - 1;
                uint4 best = make_uint4(0, 0, 0, 0);
                if (q >= 0 && q < p.Wp) {
                    __nv_bfloat162 mx[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) mx[e] = __floats2bfloat162_rn(0.0f, 0.0f);
#pragma unroll
                    for (int dr = 0; dr < 3; ++dr) {
                        const int j = 2 * pl + dr;                              // convolution row within the unit
#pragma unroll
                        for (int ds = 0; ds < 3; ++ds) {
                            const int wc = 2 * q - 1 + ds;
                            if (wc >= 0 && wc < p.Wc) {
                                const uint4 raw = cv[(size_t)ch * p.conv_pos + j * p.Wc + wc];
                                const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                                for (int e = 0; e < 4; ++e) mx[e] = __hmax2(mx[e], h2[e]);
                            }
                        }
                    }
                    best = *reinterpret_cast<uint4*>(mx);
                }
                const int pp = 2 * pr + pl;
                yout[(long long)ch * plane_out + (long long)n * P2o + (long long)(pp + 1) * Wq + qq] = best;
            }
            if (pr == 0 || pr == p.units_per_image - 1) {
                const int brow = pr == 0 ? 0 : p.Hp + 1;
                for (int i = threadIdx.x; i < chunks_out * Wq; i += kThreads) {
                    const int ch = i / Wq, qq = i - ch * Wq;
                    yout[(long long)ch * plane_out + (long long)n * P2o + (long long)brow * Wq + qq] = make_uint4(0, 0, 0, 0);
                    if (p.units_per_image == 1)
                        yout[(long long)ch * plane_out + (long long)n * P2o + (long long)(p.Hp + 1) * Wq + qq] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        __syncthreads();          // the convolution rows and this unit's input buffer are free again
    }
    if (!ok && threadIdx.x == 0) { atomicExch(&ctrl->abort_flag, 1); atomicExch(p.status, 6); }

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
