// Implicit-GEMM convolution for sm_100a: TMA-staged activation and filter tiles, tcgen05 BF16
// MMA with FP32 accumulators in tensor memory, fused epilogue (folded-BN bias + shortcut +
// ReLU, BF16 store).
//
//   GEMM view     M = N*P*Q output pixels, N = K_pad filters, K = R*S*C_pad.
//   CTA tile      128 output pixels (a tile_w x tile_h x tile_n box of the NHWC output) x n_tile filters.
//   K blocks      one filter tap (r,s) x kc channels (kc = 16/32/64 -> 32/64/128-byte swizzled rows).
//                 The activation block of a tap is one 4-D TMA box of the NHWC input shifted by the
//                 tap offset; out-of-range coordinates are zero-filled by the TMA unit, which is the
//                 convolution's zero padding.  Strided convolutions use the tensor map's element strides.
//   Warp roles    warp 0: TMA producer (one lane).  warp 1: tensor-memory allocation + MMA issue (one lane).
//                 warps 2-5: epilogue, one thread per accumulator row (TMEM lane).
//   Pipelines     `stages` shared-memory stages (full/empty mbarriers) between producer and MMA;
//                 two accumulator stages in tensor memory (tmem_full/tmem_empty) between MMA and
//                 epilogue, so the epilogue of tile i overlaps the MMAs of tile i+1.  Persistent CTAs.
//   Waits         every mbarrier wait is bounded; when one runs out the CTA raises a status word in
//                 global memory, all roles leave their loops, tensor memory is released and the
//                 kernel returns (results are then invalid and the host reports FP_ERR_TIMEOUT).
#include "fp_internal.h"

#include <cstdio>
#include <cstring>

namespace fp {

namespace {

constexpr int kThreads = 192;
constexpr int kMaxStages = 8;
constexpr uint32_t kWaitLimit = 1u << 24;          // polls per wait, and
constexpr long long kWaitCycles = 2000000000LL;    // SM clock cycles per wait (about a second)

struct TcParams {
    ConvArgs a;
    int tile_w, tile_h, tile_n, tiles_w, tiles_h, tiles_n;
    int kc, c_blocks, n_tile, n_tiles, stages;
    int a_bytes, b_bytes;       // bytes per stage
    int sbo;                    // byte distance between 8-row groups in a staged tile
    int layout_type;            // shared-memory descriptor swizzle code
    int tmem_cols;
    int total_tiles;
    int* status;
};

// ---- PTX wrappers -------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the time limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 32) __nanosleep(32);
        if ((i & 127) == 127) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitCycles) return false;
        }
    }
    return false;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor for a K-major operand tile whose rows are one swizzle span
// wide: start address, leading offset 16 B, stride offset = 8 rows, descriptor version 1.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, int sbo, int layout_type) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)(layout_type & 7) << 61;
    return d;
}

// Shared-memory control block at the start of dynamic shared memory.
struct Ctrl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(kThreads)
conv_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem_raw);
    const uint32_t ctrl_addr = smem_u32(smem_raw);
    const uint32_t tiles_base = (ctrl_addr + (uint32_t)sizeof(Ctrl) + 1023u) & ~1023u;
    volatile int* abort_flag = &ctrl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = ctrl_addr + (uint32_t)offsetof(Ctrl, full);
    const uint32_t empty0 = ctrl_addr + (uint32_t)offsetof(Ctrl, empty);
    const uint32_t tfull0 = ctrl_addr + (uint32_t)offsetof(Ctrl, tmem_full);
    const uint32_t tempty0 = ctrl_addr + (uint32_t)offsetof(Ctrl, tmem_empty);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(tfull0 + 8 * s, 1); mbar_init(tempty0 + 8 * s, 128); }
        ctrl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(ctrl_addr + (uint32_t)offsetof(Ctrl, tmem_base)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_base);

    const int taps = p.a.R * p.a.S;
    const int kblocks = taps * p.c_blocks;
    const int stage_bytes = p.a_bytes + p.b_bytes;

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
                int t = tile;
                const int nt = t % p.n_tiles; t /= p.n_tiles;
                const int tw = t % p.tiles_w; t /= p.tiles_w;
                const int th = t % p.tiles_h; t /= p.tiles_h;
                const int tn = t;
                const int x0 = tw * p.tile_w * p.a.stride - p.a.pad;
                const int y0 = th * p.tile_h * p.a.stride - p.a.pad;
                const int n0 = tn * p.tile_n;
                for (int tap = 0; tap < taps && ok; ++tap) {
                    const int r = tap / p.a.S, s = tap - r * p.a.S;
                    for (int cb = 0; cb < p.c_blocks; ++cb) {
                        if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                        const uint32_t fb = full0 + 8 * stage;
                        const uint32_t sa = tiles_base + stage * stage_bytes;
                        mbar_expect_tx(fb, (uint32_t)stage_bytes);
                        tma_load_4d(sa, &tm_x, fb, cb * p.kc, x0 + s, y0 + r, n0);
                        tma_load_3d(sa + p.a_bytes, &tm_w, fb, cb * p.kc, tap, nt * p.n_tile);
                        if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                    }
                }
            }
            if (!ok) { atomicExch((int*)&ctrl->abort_flag, 1); atomicExch(p.status, 1); }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer --------------------------------
        if (lane == 0) {
            // instruction descriptor: D = f32, A = B = bf16, both K-major, N = n_tile, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_tile >> 3) << 17) | ((128u >> 4) << 24);
            uint32_t stage = 0, phase = 0;
            uint32_t acc_phase[2] = {0, 0};
            int local = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++local) {
                const int acc = local & 1;
                if (!mbar_wait(tempty0 + 8 * acc, acc_phase[acc] ^ 1, abort_flag)) { ok = false; break; }
                acc_phase[acc] ^= 1;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * p.n_tile);
                uint32_t accumulate = 0;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const int cb = kb % p.c_blocks;
                    int ksteps = (p.a.C_pad - cb * p.kc);
                    ksteps = (ksteps < p.kc ? ksteps : p.kc) >> 4;
                    const uint32_t sa = tiles_base + stage * stage_bytes;
                    const uint32_t sb = sa + p.a_bytes;
                    for (int ks = 0; ks < ksteps; ++ks) {
                        const uint64_t da = make_smem_desc(sa + ks * 32, p.sbo, p.layout_type);
                        const uint64_t db = make_smem_desc(sb + ks * 32, p.sbo, p.layout_type);
                        umma_bf16(d_tmem, da, db, idesc, accumulate);
                        accumulate = 1;
                    }
                    umma_commit(empty0 + 8 * stage);     // releases the stage once these MMAs have read it
                    if (++stage == (uint32_t)p.stages) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit(tfull0 + 8 * acc);   // accumulator complete
            }
            if (!ok) { atomicExch((int*)&ctrl->abort_flag, 1); atomicExch(p.status, 2); }
        }
    } else {
        // ------------------------------ epilogue ----------------------------------
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31 belong to this warp
        const int row = quarter * 32 + lane;          // accumulator row = pixel within the tile
        const int w_l = row % p.tile_w;
        const int h_l = (row / p.tile_w) % p.tile_h;
        const int n_l = row / (p.tile_w * p.tile_h);
        uint32_t acc_phase[2] = {0, 0};
        int local = 0;
        bool ok = true;
        const __nv_bfloat16* __restrict__ res = (const __nv_bfloat16*)p.a.res;
        __nv_bfloat16* __restrict__ y = (__nv_bfloat16*)p.a.y;
        for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x, ++local) {
            int t = tile;
            const int nt = t % p.n_tiles; t /= p.n_tiles;
            const int tw = t % p.tiles_w; t /= p.tiles_w;
            const int th = t % p.tiles_h; t /= p.tiles_h;
            const int tn = t;
            const int q = tw * p.tile_w + w_l, pp = th * p.tile_h + h_l, n = tn * p.tile_n + n_l;
            const bool valid = q < p.a.Q && pp < p.a.P && n < p.a.N;
            const int acc = local & 1;
            ok = mbar_wait(tfull0 + 8 * acc, acc_phase[acc], abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            acc_phase[acc] ^= 1;
            tc_fence_after();
            const int k_base = nt * p.n_tile;
            int cols = p.a.K_pad - k_base;
            if (cols > p.n_tile) cols = p.n_tile;
            const size_t out_off = (((size_t)n * p.a.P + pp) * p.a.Q + q) * p.a.K_pad + k_base;
            size_t res_off = 0;
            if (p.a.res_mode == 2)
                res_off = (((size_t)n * p.a.res_H + (size_t)pp * p.a.res_stride) * p.a.res_W + (size_t)q * p.a.res_stride) * p.a.res_C_pad;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * p.n_tile);
            for (int c0 = 0; c0 < cols; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(taddr + c0, v);
                tmem_ld_wait();
                if (valid) {
                    float f[16];
                    const float4* b4 = reinterpret_cast<const float4*>(p.a.bias + k_base + c0);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float4 b = __ldg(b4 + i);
                        f[4 * i + 0] = __uint_as_float(v[4 * i + 0]) + b.x;
                        f[4 * i + 1] = __uint_as_float(v[4 * i + 1]) + b.y;
                        f[4 * i + 2] = __uint_as_float(v[4 * i + 2]) + b.z;
                        f[4 * i + 3] = __uint_as_float(v[4 * i + 3]) + b.w;
                    }
                    if (p.a.res_mode == 1) {
                        const uint4* rp = reinterpret_cast<const uint4*>(res + out_off + c0);
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            const uint4 raw = __ldg(rp + hh);
                            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 g = __bfloat1622float2(h2[i]);
                                f[8 * hh + 2 * i] += g.x;
                                f[8 * hh + 2 * i + 1] += g.y;
                            }
                        }
                    } else if (p.a.res_mode == 2) {
                        // shortcut by subsampling: output channel k takes input channel k - pad_lo
                        const int cs = k_base + c0 - p.a.res_pad_lo;
                        if (cs >= 0 && cs + 16 <= p.a.res_C && (cs & 7) == 0) {
                            const uint4* rp = reinterpret_cast<const uint4*>(res + res_off + cs);
#pragma unroll
                            for (int hh = 0; hh < 2; ++hh) {
                                const uint4 raw = __ldg(rp + hh);
                                const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const float2 g = __bfloat1622float2(h2[i]);
                                    f[8 * hh + 2 * i] += g.x;
                                    f[8 * hh + 2 * i + 1] += g.y;
                                }
                            }
                        } else if (cs + 16 > 0 && cs < p.a.res_C) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const int c = cs + i;
                                if (c >= 0 && c < p.a.res_C) f[i] += __bfloat162float(res[res_off + c]);
                            }
                        }
                    }
                    if (p.a.relu) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) f[i] = fmaxf(f[i], 0.0f);
                    }
                    uint4 o[2];
                    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(o);
#pragma unroll
                    for (int i = 0; i < 8; ++i) o2[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
                    uint4* yp = reinterpret_cast<uint4*>(y + out_off + c0);
                    yp[0] = o[0];
                    yp[1] = o[1];
                }
            }
            tc_fence_before();
            mbar_arrive(tempty0 + 8 * acc);
        }
        if (!ok && lane == 0) { atomicExch((int*)&ctrl->abort_flag, 1); atomicExch(p.status, 3); }
    }

    // ---- teardown: everyone arrives here, also after a wait that ran out ----
    if (*abort_flag) {
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

int pow2_at_least(int v) { int p = 1; while (p < v) p <<= 1; return p; }

}  // namespace

int plan_conv_tc(const ConvArgs& a, ConvPlanTC* plan, char* err, size_t err_len) {
    memset(plan, 0, sizeof(*plan));
    EncodeTiledFn encode = get_encode();
    if (!encode) { snprintf(err, err_len, "cuTensorMapEncodeTiled is not available"); return 1; }
    if (a.C_pad % 16 || a.K_pad % 16) { snprintf(err, err_len, "channel counts must be padded to 16"); return 1; }
    if (a.stride < 1 || a.stride > 8) { snprintf(err, err_len, "stride %d not supported", a.stride); return 1; }

    // --- pixel tile: tile_w x tile_h x tile_n = 128 ---
    int tw = pow2_at_least(a.Q < 128 ? a.Q : 128);
    if (tw < 8) tw = 8;
    while (tw * a.stride > 256) tw >>= 1;
    int th = pow2_at_least(a.P < 128 / tw ? a.P : 128 / tw);
    if (th > 128 / tw) th = 128 / tw;
    while (th * a.stride > 256) th >>= 1;
    int tn = 128 / (tw * th);
    plan->tile_w = tw; plan->tile_h = th; plan->tile_n = tn;
    plan->tiles_w = (a.Q + tw - 1) / tw;
    plan->tiles_h = (a.P + th - 1) / th;
    plan->tiles_n = (a.N + tn - 1) / tn;

    // --- K blocking ---
    plan->kc = a.C_pad >= 64 ? 64 : a.C_pad >= 32 ? 32 : 16;
    if (a.C_pad == 48) plan->kc = 16;           // three exact 16-channel blocks instead of 64 with padding
    plan->c_blocks = (a.C_pad + plan->kc - 1) / plan->kc;
    plan->swizzle_bytes = plan->kc * 2;

    // --- filter tile ---
    int n_tiles = (a.K_pad + 255) / 256;
    int n_tile = ((a.K_pad + n_tiles - 1) / n_tiles + 15) / 16 * 16;
    const long m_tiles = (long)plan->tiles_w * plan->tiles_h * plan->tiles_n;
    while (m_tiles * n_tiles < 148 && n_tile > 64) {      // few pixel tiles: split filters further to fill the SMs
        n_tiles *= 2;
        n_tile = ((a.K_pad + n_tiles - 1) / n_tiles + 15) / 16 * 16;
    }
    n_tiles = (a.K_pad + n_tile - 1) / n_tile;
    plan->n_tile = n_tile; plan->n_tiles = n_tiles;
    plan->tmem_cols = pow2_at_least(2 * n_tile < 32 ? 32 : 2 * n_tile);

    // --- shared memory ---
    const int a_bytes = 128 * plan->kc * 2;
    const int b_bytes = n_tile * plan->kc * 2;
    int stages = (200 * 1024) / (a_bytes + b_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) { snprintf(err, err_len, "tile does not fit shared memory"); return 1; }
    plan->stages = stages;
    unsigned smem = (unsigned)(sizeof(Ctrl) + 1024 + (size_t)stages * (a_bytes + b_bytes));
    // co-resident CTAs must not ask for more than the 512 tensor-memory columns of an SM
    const int tmem_ctas = 512 / plan->tmem_cols;
    const unsigned min_smem = 232448u / (unsigned)(tmem_ctas + 1) + 1u;
    if (smem < min_smem && tmem_ctas < 16) smem = min_smem;
    plan->smem_bytes = smem;
    int ctas_per_sm = (int)(232448u / (smem + 1024u));
    if (ctas_per_sm > tmem_ctas) ctas_per_sm = tmem_ctas;
    if (ctas_per_sm > 4) ctas_per_sm = 4;
    if (ctas_per_sm < 1) ctas_per_sm = 1;
    plan->grid = 148 * ctas_per_sm;

    // --- tensor maps ---
    const CUtensorMapSwizzle sw = plan->swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : plan->swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    {
        cuuint64_t dims[4] = {(cuuint64_t)a.C_pad, (cuuint64_t)a.W, (cuuint64_t)a.H, (cuuint64_t)a.N};
        cuuint64_t strides[3] = {(cuuint64_t)a.C_pad * 2, (cuuint64_t)a.W * a.C_pad * 2, (cuuint64_t)a.H * a.W * a.C_pad * 2};
        cuuint32_t box[4] = {(cuuint32_t)plan->kc, (cuuint32_t)(tw * a.stride), (cuuint32_t)(th * a.stride), (cuuint32_t)tn};
        cuuint32_t estr[4] = {1, (cuuint32_t)a.stride, (cuuint32_t)a.stride, 1};
        CUresult r = encode(&plan->tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(a.x), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { snprintf(err, err_len, "activation tensor map rejected (CUresult %d)", (int)r); return 1; }
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)a.C_pad, (cuuint64_t)(a.R * a.S), (cuuint64_t)a.K_pad};
        cuuint64_t strides[2] = {(cuuint64_t)a.C_pad * 2, (cuuint64_t)a.R * a.S * a.C_pad * 2};
        cuuint32_t box[3] = {(cuuint32_t)plan->kc, 1, (cuuint32_t)n_tile};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = encode(&plan->tm_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(a.w), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { snprintf(err, err_len, "filter tensor map rejected (CUresult %d)", (int)r); return 1; }
    }
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 232448 - 1024) != cudaSuccess) {
            snprintf(err, err_len, "cannot raise the dynamic shared memory limit");
            cudaGetLastError();
            return 1;
        }
        attr_set = true;
    }
    plan->valid = 1;
    return 0;
}

void launch_conv_tc(const ConvPlanTC& plan, const ConvArgs& a, int* d_status, cudaStream_t st) {
    TcParams p;
    p.a = a;
    p.tile_w = plan.tile_w; p.tile_h = plan.tile_h; p.tile_n = plan.tile_n;
    p.tiles_w = plan.tiles_w; p.tiles_h = plan.tiles_h;
    p.tiles_n = (a.N + plan.tile_n - 1) / plan.tile_n;
    p.kc = plan.kc; p.c_blocks = plan.c_blocks; p.n_tile = plan.n_tile; p.n_tiles = plan.n_tiles; p.stages = plan.stages;
    p.a_bytes = 128 * plan.kc * 2;
    p.b_bytes = plan.n_tile * plan.kc * 2;
    p.sbo = 8 * plan.kc * 2;
    p.layout_type = plan.swizzle_bytes == 128 ? 2 : plan.swizzle_bytes == 64 ? 4 : 6;
    p.tmem_cols = plan.tmem_cols;
    p.total_tiles = p.tiles_w * p.tiles_h * p.tiles_n * p.n_tiles;
    p.status = d_status;
    int grid = plan.grid < p.total_tiles ? plan.grid : p.total_tiles;
    if (grid < 1) grid = 1;
    conv_tc_kernel<<<grid, kThreads, plan.smem_bytes, st>>>(plan.tm_x, plan.tm_w, p);
}

}  // namespace fp
