// Implicit-GEMM convolution for sm_100a: tcgen05 BF16 MMA with FP32 accumulators in tensor
// memory, operands staged in shared memory by the bulk-copy (TMA) engine, fused epilogue
// (folded-BN bias + shortcut + ReLU, BF16 store).  Activations use the planar-8 layout with a
// zero border described in fp_internal.h.
//
//   GEMM view     M = flat output positions (border positions included: they are computed and then
//                 overwritten with zeros), N = K_pad filters, K = R*S*C_pad.
//   CTA tile      128 consecutive flat positions x n_tile filters; persistent CTAs walk the tiles.
//   Operands      K-major, no swizzle: an operand block is a stack of 16-byte rows (8 channels of
//                 one position / one filter); the two 8-channel halves of a K=16 MMA step live in
//                 two such stacks ("planes"), `LBO` apart.
//   FLAT modes    stride-1 "same" convolutions (3x3 pad 1, 3x1 pad 1x0, 1x1 pad 0).  Because every chunk plane
//                 is contiguous over flat positions, the activations a tile needs - its 128
//                 positions plus a halo of (W+3) before and after (3x3) - are ONE contiguous run per
//                 chunk, fetched with one bulk copy.  The operand of filter tap (r,s) is the same
//                 shared-memory block read from a start address shifted by (r-1)*(W+2)+(s-1) rows,
//                 so each activation is fetched once per tile, not once per tap.  The zero border
//                 in memory is the convolution's padding.  Filters either stay resident in shared
//                 memory for the whole kernel (small banks), are streamed per (filter row, K block) into a ring of
//                 their own, or share a stage with the activations of their K block (1x1 layers, and the strided
//                 3x3 layers below: one ring, several producer warps).
//   Parity-split  a 3x3 / stride-2 / pad-1 convolution over a tensor stored as four half-resolution parity images
//   inputs        (ConvArgs in fp_internal.h) is a FLAT convolution too: four contiguous runs per chunk, tap (r,s)
//                 reading the run of parity ((r+1)&1, (s+1)&1) at an offset of -1 or 0 rows and columns; a 1x1 /
//                 stride-2 convolution reads the parity-00 images alone.  The epilogue can write a tensor in that form.
//   GATHER mode   any other geometry (strided layers over plain tensors, 7x7, ...): 128 loader threads fetch the vectors of
//                 their output position for each (tap, K block) with 16-byte loads, zero where the
//                 window leaves the image.
//   Warp roles    warp 0: bulk-copy producer (one lane per chunk copy).  warp 1: tensor-memory allocation, lane 0 issues
//                 the MMAs.  Then 4 or 8 epilogue warps, one thread per accumulator row (8: each takes half of the
//                 columns).  Behind them: the filter producer and up to three more MMA-issuing warps (one per position
//                 tile of a step) when filters are streamed; three more producer and three more issuing warps with
//                 unified stages; the four loader warps in GATHER mode.
//   Pipelines     full/empty mbarrier rings for the shared-memory stages; two accumulator stages in
//                 tensor memory so the epilogue of one tile overlaps the MMAs of the next.
//   Waits         every mbarrier wait is bounded; when one runs out the CTA raises a status word in
//                 global memory, all roles leave their loops, tensor memory is released and the
//                 kernel returns (results are then invalid and the host reports FP_ERR_TIMEOUT).
#include "fp_internal.h"
#include "tc_common.cuh"

#include <cstdio>
#include <cstring>

namespace fp {

namespace {

using namespace tc;

constexpr int kMaxStages = 8;

// FLAT_STREAM: activations per K group and filters per (K group, tap) in two rings (convolutions with several taps);
// FLAT_UNIFIED: one ring whose stages hold a K group's activations and filters together (1x1 convolutions).
enum { MODE_FLAT_RESIDENT = 0, MODE_FLAT_STREAM = 1, MODE_GATHER = 2, MODE_FLAT_UNIFIED = 3 };

struct TcParams {
    ConvArgs a;
    FastDiv div_ntiles, div_p2out, div_qp;
    int Wp_in, P2_in, Qp, P2_out;
    long long plane_in, plane_out;      // vectors per chunk plane (N * P2)
    long long m_total;                  // flat output positions
    int taps, cchunks, cg, groups, halo, rows_a, a_stages, b_stages;
    int n_tile, n_tiles, tmem_cols, total_tiles;
    int tpk, kblocks;                   // gather: taps per K block, K blocks per tile
    int tps;                            // streamed filters: 128-position tiles per pipeline step (share each filter block)
    int n_producers;                    // streamed filters: producer warps in use (divides a_stages)
    int a_stage_bytes, b_stage_bytes, b_bank_bytes;
    long long bank_tile_bytes;          // streamed filters: bytes of one filter tile's part of the bank (all taps, all chunks)
    int lut_bytes;                      // gather: table of plane offsets, 8 entries of 8 bytes per K block
    int scatter_bytes;                  // scattered output: channel -> accumulator column map and the tiles' chunk ranges
    long long plane_in2;                // vectors per channel chunk of the second input tensor (ConvArgs::x2)
    int cchunks2, groups2;              // streamed 3x3 layer: chunks / extra K groups of the second input (centre tap only)
    int a_par;                          // activation runs per channel chunk in a stage: 1, or 4 parity images (x_s2d)
    long long par_stride;               // x_s2d: vectors between the parity images of one chunk (N * P2)
    int tap_off[9];                     // x_s2d: start row of each tap's operand within a chunk's part of the stage
    int y_split, y_P2h, y_Wh2;          // split output: half-resolution grid
    long long plane_y;                  // vectors per chunk plane of the output tensor
    long long wait_cycles;              // limit of every barrier wait in SM clock cycles (0: about a second)
    int skip_round;                     // diagnostic: the activation producer leaves out this round's copies (-1: none)
    int* status;
};

// Issues the MMAs of one K block of a FLAT-mode tile: R*R filter taps x KSTEPS K=16 steps, fully
// unrolled so that the single issuing thread spends a handful of instructions per MMA.  Operand
// descriptors differ only in their low words: one address unit is one 16-byte row, so a tap's
// activation operand is `a_lo + r*Wp + s` and a K step advances both operands by two planes.
template <int R, int S, int KSTEPS>
__device__ __forceinline__ void issue_flat_resident(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t Wp,
                                                    uint32_t a_ks, uint32_t b_ks, uint32_t b_tap, uint32_t idesc,
                                                    uint32_t accumulate) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int sx = 0; sx < S; ++sx) {
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                umma_bf16_lo(d_tmem, a_lo + (uint32_t)r * Wp + (uint32_t)sx + (uint32_t)ks * a_ks,
                             b_lo + (uint32_t)(r * S + sx) * b_tap + (uint32_t)ks * b_ks, idesc,
                             (r | sx | ks) ? 1u : accumulate);
            }
        }
    }
}

template <int R, int S>
__device__ __forceinline__ void issue_flat_resident_k(int ksteps, uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo,
                                                      uint32_t Wp, uint32_t a_ks, uint32_t b_ks, uint32_t b_tap,
                                                      uint32_t idesc, uint32_t accumulate) {
    switch (ksteps) {
        case 1: issue_flat_resident<R, S, 1>(d_tmem, a_lo, b_lo, Wp, a_ks, b_ks, b_tap, idesc, accumulate); break;
        case 2: issue_flat_resident<R, S, 2>(d_tmem, a_lo, b_lo, Wp, a_ks, b_ks, b_tap, idesc, accumulate); break;
        case 3: issue_flat_resident<R, S, 3>(d_tmem, a_lo, b_lo, Wp, a_ks, b_ks, b_tap, idesc, accumulate); break;
        default: issue_flat_resident<R, S, 4>(d_tmem, a_lo, b_lo, Wp, a_ks, b_ks, b_tap, idesc, accumulate); break;
    }
}

// The K=16 steps of one (tap, K group) block for one accumulator, unrolled.
template <int KSTEPS>
__device__ __forceinline__ void issue_ksteps_n(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_ks, uint32_t b_ks,
                                               uint32_t idesc, uint32_t accumulate) {
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks)
        umma_bf16_lo(d_tmem, a_lo + (uint32_t)ks * a_ks, b_lo + (uint32_t)ks * b_ks, idesc, ks ? 1u : accumulate);
}
__device__ __forceinline__ void issue_ksteps(int ksteps, uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_ks,
                                             uint32_t b_ks, uint32_t idesc, uint32_t accumulate) {
    // (a plain counted loop: a switch over unrolled bodies measured the same)
#pragma unroll 1
    for (int ks = 0; ks < ksteps; ++ks) {
        umma_bf16_lo(d_tmem, a_lo, b_lo, idesc, ks ? 1u : accumulate);
        a_lo += a_ks;
        b_lo += b_ks;
    }
}

// The nine taps of a 3x3 / stride-2 window over parity images for one K group, fully unrolled: every tap's operand
// starts at its own row of the stage (tap_off), its filters follow the previous tap's.  (As a loop over rows and columns
// that looked its offset up by a computed index, each tap cost the issuing thread about 350 cycles - ResNet-50's
// three strided 3x3 layers at batch 128: 51 / 48 / 47 us so, 33 / 28 / 27 us unrolled.)
template <int KSTEPS>
__device__ __forceinline__ void issue_taps9(uint32_t d_tmem, uint32_t a_row0, const int (&tap_off)[9], uint32_t b_lo, uint32_t b_tap,
                                            uint32_t a_ks, uint32_t b_ks, uint32_t idesc, uint32_t accumulate) {
#pragma unroll
    for (int t = 0; t < 9; ++t)
        issue_ksteps_n<KSTEPS>(d_tmem, a_row0 + (uint32_t)tap_off[t], b_lo + (uint32_t)t * b_tap, a_ks, b_ks, idesc, t ? 1u : accumulate);
}

// Shared-memory control block at the start of dynamic shared memory.
struct Ctrl {
    uint64_t a_full[kMaxStages];
    uint64_t a_empty[kMaxStages];
    uint64_t b_full[kMaxStages];
    uint64_t b_empty[kMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    int pad_[2];          // keeps sizeof(Ctrl) a multiple of 16: the bias table follows
};
static_assert(sizeof(Ctrl) % 16 == 0, "bias table must stay 16-byte aligned");

__device__ __forceinline__ void raise(Ctrl* ctrl, int* status, int code) {
    atomicExch(&ctrl->abort_flag, 1);
    atomicExch(status, code);
}

// Threads: warp 0 producer, warp 1 MMA, EPI epilogue warps (4, or 8 for wide filter tiles: two warps per
// TMEM lane quarter, each taking half of the columns), then either 4 loader warps (GATHER) or 4 filter-producer
// warps and 3 more MMA warps (FLAT_STREAM).  One thread gets through a (wait, expect, copy) round of the bulk-copy
// engine in about 500 cycles whatever the copy's size (measured: 4 KB to 32 KB copies all take 530 cycles per round
// per thread, and the rate scales with the number of threads up to about 100 B/cycle per SM), so the filter blocks
// of a streamed bank, 12-18 KB each, are issued round-robin by four warps.  A single thread cannot issue MMAs as fast as the tensor pipe
// retires them (measured: 75-110 cycles per issued MMA against 56-64 of execution at N = 96-128), so in
// FLAT_STREAM, where one CTA owns the SM, each 128-position tile of a step has an issuing warp of its own.
constexpr int kProducers = 4;          // unified stages: warp 0 and three more warps issue the stages' copies in turn
__host__ __device__ constexpr int extra_threads(int mode) {
    return mode == MODE_FLAT_RESIDENT ? 0 : mode == MODE_FLAT_UNIFIED ? 32 * ((kProducers - 1) + 3) : 128;
}

template <int MODE, int EPI>
__global__ void __launch_bounds__(64 + 32 * EPI + extra_threads(MODE))
conv_tc_kernel(const TcParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem_raw);
    const uint32_t ctrl_addr = smem_u32(smem_raw);
    float* bias_s = reinterpret_cast<float*>(smem_raw + sizeof(Ctrl));            // K_pad floats
    int2* lut = reinterpret_cast<int2*>(smem_raw + sizeof(Ctrl) + (size_t)p.a.K_pad * 4u);   // gather mode only
    int* smap = reinterpret_cast<int*>(smem_raw + sizeof(Ctrl) + (size_t)p.a.K_pad * 4u + (size_t)p.lut_bytes);   // scattered output only
    int* schunk0 = smap + p.a.out_C_pad;
    float* sstrip = reinterpret_cast<float*>(schunk0 + ((p.n_tiles + 1 + 3) & ~3));          // EPI warps x 32 rows x 33 words
    const uint32_t b_base = (ctrl_addr + (uint32_t)sizeof(Ctrl) + (uint32_t)p.a.K_pad * 4u + (uint32_t)p.lut_bytes +
                             (uint32_t)p.scatter_bytes + 1023u) & ~1023u;
    const uint32_t b_region = MODE == MODE_FLAT_RESIDENT ? (uint32_t)p.b_bank_bytes
                              : MODE == MODE_FLAT_STREAM ? (uint32_t)(p.b_stages * p.b_stage_bytes) : 0u;
    const uint32_t a_base = b_base + ((b_region + 127u) & ~127u);
    volatile int* abort_flag = &ctrl->abort_flag;
    const long long wait_limit = p.wait_cycles > 0 ? p.wait_cycles : kWaitCycles;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t a_full0 = ctrl_addr + (uint32_t)offsetof(Ctrl, a_full);
    const uint32_t a_empty0 = ctrl_addr + (uint32_t)offsetof(Ctrl, a_empty);
    const uint32_t b_full0 = ctrl_addr + (uint32_t)offsetof(Ctrl, b_full);
    const uint32_t b_empty0 = ctrl_addr + (uint32_t)offsetof(Ctrl, b_empty);
    const uint32_t tfull0 = ctrl_addr + (uint32_t)offsetof(Ctrl, tmem_full);
    const uint32_t tempty0 = ctrl_addr + (uint32_t)offsetof(Ctrl, tmem_empty);

    // MMA-issuing warps: warp 1, plus (streamed filters) the last three warps, one per tile of a step
    const uint32_t n_issuers = (MODE == MODE_FLAT_STREAM || MODE == MODE_FLAT_UNIFIED) ? (uint32_t)p.tps : 1u;
    const int issuer = warp == 1 ? 0
                       : (MODE == MODE_FLAT_STREAM && warp >= 3 + EPI) ? warp - (2 + EPI)
                       : (MODE == MODE_FLAT_UNIFIED && warp >= 1 + EPI + kProducers) ? warp - (EPI + kProducers) : -1;
    // unified stages: producer warps (warp 0, then the first kProducers - 1 of the extra warps)
    const int prod = MODE != MODE_FLAT_UNIFIED ? -1 : warp == 0 ? 0 : (warp >= 2 + EPI && warp < 1 + EPI + kProducers) ? warp - (1 + EPI) : -1;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(a_full0 + 8 * s, MODE == MODE_GATHER ? 129 : 1);   // gather: 128 loaders + the filter producer
            mbar_init(a_empty0 + 8 * s, n_issuers);
            mbar_init(b_full0 + 8 * s, 1);
            mbar_init(b_empty0 + 8 * s, n_issuers);
        }
        for (int s = 0; s < 2; ++s) { mbar_init(tfull0 + 8 * s, n_issuers); mbar_init(tempty0 + 8 * s, 32 * EPI); }
        ctrl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = threadIdx.x; i < p.a.K_pad; i += blockDim.x) bias_s[i] = p.a.bias[i];   // filters' data: safe before the dependency wait
    if (p.a.scatter) {
        for (int i = threadIdx.x; i < p.a.out_C_pad; i += blockDim.x) smap[i] = p.a.out_map[i];
        for (int i = threadIdx.x; i <= p.n_tiles; i += blockDim.x) schunk0[i] = p.a.tile_chunk0[i];
    }
    if (MODE == MODE_GATHER) {
        // Plane i of K block kb holds channel chunk c of tap (r, s): its offset from the tile's first tap, in
        // 16-byte vectors, and r, s, "in use" and the block's plane count, are the same for every tile.
        for (int e = threadIdx.x; e < p.kblocks * 8; e += blockDim.x) {
            const int kb = e >> 3, i = e & 7;
            int tap0, g, ntap, cgg;
            if (p.groups > 1) { tap0 = kb / p.groups; g = kb - tap0 * p.groups; ntap = 1; cgg = p.cchunks - g * p.cg; if (cgg > p.cg) cgg = p.cg; }
            else { tap0 = kb * p.tpk; g = 0; ntap = p.taps - tap0 < p.tpk ? p.taps - tap0 : p.tpk; cgg = p.cchunks; }
            const int planes = ntap * cgg;
            const int tt = i / cgg, c = i - tt * cgg;
            const int tap = tap0 + tt, r = tap / p.a.S, sx = tap - r * p.a.S;
            lut[e] = i < planes ? make_int2((g * p.cg + c) * (int)p.plane_in + r * p.Wp_in + sx, r | (sx << 8) | (1 << 16) | (planes << 24))
                                : make_int2(0, planes << 24);
        }
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

    const uint4* __restrict__ xv = reinterpret_cast<const uint4*>(p.a.x);
    const uint4* __restrict__ wv = reinterpret_cast<const uint4*>(p.a.w);
    // channel chunk -> its plane: the chunks behind x2_chunk0 are the second input tensor's
    const uint4* __restrict__ x2v = reinterpret_cast<const uint4*>(p.a.x2);
    const int chunk2 = p.a.x2_chunk0 > 0 ? p.a.x2_chunk0 : 0x7fffffff;
    auto chunk_plane = [&](int chunk) -> const uint4* {
        return chunk < chunk2 ? xv + (long long)chunk * p.plane_in : x2v + (long long)(chunk - chunk2) * p.plane_in2;
    };

    // Programmatic dependent launch: everything above, and the filter-bank copy below, touches
    // nothing the previous kernel in the stream writes, so it may overlap that kernel's tail.  The
    // next kernel is allowed to start its own prologue now; activations (and every global write) wait
    // until the previous kernel has completed and its writes are visible.
    if (MODE == MODE_FLAT_RESIDENT && threadIdx.x == 0) {
        mbar_expect_tx(b_full0, (uint32_t)p.b_bank_bytes);
        for (int off = 0; off < p.b_bank_bytes; off += 32768) {
            const int n = p.b_bank_bytes - off < 32768 ? p.b_bank_bytes - off : 32768;
            bulk_copy(b_base + off, reinterpret_cast<const uint8_t*>(p.a.w) + (long long)(blockIdx.x % p.n_tiles) * p.b_bank_bytes + off,
                      (uint32_t)n, b_full0);
        }
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (MODE == MODE_FLAT_UNIFIED && prod >= 0) {
        // ------------------------------ producers, unified stages ------------------------------
        // One stage per (step of tps position tiles, K group): the group's activation rows for all tiles of the step
        // (one copy per channel chunk) and the group's filters for all taps (one copy: the bank is stored block by
        // block in this order).  The stages are issued in turn by n_producers warps; that number divides the number of
        // stages, so a stage is always refilled by the same warp: a warp that ran ahead onto a stage another warp still
        // has to fill could not tell "two phases behind" from "ready" by the barrier's parity.
        bool ok = true;
        uint32_t stage = 0, phase = 0;
        int turn = 0;
        const uint32_t stage_bytes = (uint32_t)(p.a_stage_bytes + p.b_stage_bytes);
        for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
            const int mt = (int)fdiv((uint32_t)tile, p.div_ntiles);
            const int nt = tile - mt * p.n_tiles;
            const long long f0 = (long long)mt * p.tps * 128;
            for (int g = 0; g < p.groups; ++g) {
                if (turn == prod) {
                    const bool w = __all_sync(0xffffffffu, mbar_wait(a_empty0 + 8 * stage, phase ^ 1, abort_flag, wait_limit));
                    if (!w) { ok = false; break; }
                    int cgg = p.cchunks - g * p.cg;
                    if (cgg > p.cg) cgg = p.cg;
                    const uint32_t fb = a_full0 + 8 * stage;
                    const uint32_t dst = a_base + stage * stage_bytes;
                    const uint32_t b_bytes = (uint32_t)(p.taps * cgg * p.n_tile * 16);
                    const int na = p.a_par * cgg;          // activation runs: one per chunk, or per chunk and parity image (<= 16)
                    if (lane == 0) mbar_expect_tx(fb, (uint32_t)(na * p.rows_a * 16) + b_bytes);
                    __syncwarp();
                    if (lane < na) {
                        const int c = p.a_par == 1 ? lane : lane >> 2, pp = p.a_par == 1 ? 0 : lane & 3;
                        bulk_copy(dst + lane * p.rows_a * 16,
                                  chunk_plane(g * p.cg + c) + (long long)pp * p.par_stride + f0 - p.halo,
                                  (uint32_t)(p.rows_a * 16), fb);
                    } else if (lane >= 16) {
                        // the group's filter block is one contiguous run of the bank: pieces of 16 KB, one per lane
                        const uint32_t off = (uint32_t)(lane - 16) * 16384u;
                        if (off < b_bytes)
                            bulk_copy(dst + (uint32_t)p.a_stage_bytes + off,
                                      reinterpret_cast<const uint8_t*>(p.a.w) + (long long)nt * p.bank_tile_bytes +
                                          (long long)p.taps * (g * p.cg) * p.n_tile * 16 + off,
                                      b_bytes - off < 16384u ? b_bytes - off : 16384u, fb);
                    }
                }
                if (++turn == p.n_producers) turn = 0;
                if (++stage == (uint32_t)p.a_stages) { stage = 0; phase ^= 1; }
            }
        }
        if (!ok && lane == 0) raise(ctrl, p.status, 1);
    } else if (warp == 0) {
        // ------------------------------ bulk-copy producer ------------------------------
        if (MODE != MODE_GATHER) {
            // One lane per channel chunk issues that chunk's copy, so the copies of a K block are issued
            // side by side instead of one after the other.  (All lanes test the stage's barrier: one lane testing and a
            // shuffle of the result was measured slower - 41.0 -> 37.7 us on ResNet-50's 1024 -> 308 layer at batch 128.)
            bool ok = true;
            uint32_t stage = 0, phase = 0;
            int round = 0;
            for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
                const long long f0 = (long long)fdiv((uint32_t)tile, p.div_ntiles) * p.tps * 128;
                for (int g = 0; g < p.groups + p.groups2; ++g) {
                    const bool w = __all_sync(0xffffffffu, mbar_wait(a_empty0 + 8 * stage, phase ^ 1, abort_flag, wait_limit));
                    if (!w) { ok = false; break; }
                    int cgg = p.cchunks - g * p.cg;
                    if (cgg > p.cg) cgg = p.cg;
                    const uint32_t fb = a_full0 + 8 * stage;
                    const uint32_t dst = a_base + stage * p.a_stage_bytes;
                    if (g >= p.groups) {
                        // the K groups of the second input tensor (a projection shortcut's input on this layer's grid)
                        const int g2 = g - p.groups;
                        cgg = p.cchunks2 - g2 * p.cg;
                        if (cgg > p.cg) cgg = p.cg;
                        if (lane == 0) mbar_expect_tx(fb, (uint32_t)(cgg * p.rows_a * 16));
                        __syncwarp();
                        if (lane < cgg)
                            bulk_copy(dst + lane * p.rows_a * 16, x2v + (long long)(g2 * p.cg + lane) * p.plane_in2 + f0 - p.halo,
                                      (uint32_t)(p.rows_a * 16), fb);
                        ++round;
                    } else
                    if (round++ != p.skip_round) {       // (a diagnostic launch leaves one round out: its stage never fills)
                        if (lane == 0) mbar_expect_tx(fb, (uint32_t)(p.a_par * cgg * p.rows_a * 16));
                        __syncwarp();
                        // one run per channel chunk - or, over a parity-split tensor, one per chunk and parity image
                        for (int i = lane; i < p.a_par * cgg; i += 32) {
                            const int c = p.a_par == 1 ? i : i >> 2, pp = p.a_par == 1 ? 0 : i & 3;
                            bulk_copy(dst + i * p.rows_a * 16,
                                      chunk_plane(g * p.cg + c) + (long long)pp * p.par_stride + f0 - p.halo,
                                      (uint32_t)(p.rows_a * 16), fb);
                        }
                    }
                    if (++stage == (uint32_t)p.a_stages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok && lane == 0) raise(ctrl, p.status, 1);
        } else {
            // GATHER: filters of each K block into the stage the loader threads fill, one lane per plane
            bool ok = true;
            uint32_t stage = 0, phase = 0;
            for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
                const int nt = tile - (int)fdiv((uint32_t)tile, p.div_ntiles) * p.n_tiles;
                int nrows = p.a.K_pad - nt * p.n_tile;
                if (nrows > p.n_tile) nrows = p.n_tile;
                for (int kb = 0; kb < p.kblocks; ++kb) {
                    // a K block is either one tap x one channel group, or (few channels) several whole taps
                    int tap0, g, ntap, cgg;
                    if (p.groups > 1) { tap0 = kb / p.groups; g = kb - tap0 * p.groups; ntap = 1; cgg = p.cchunks - g * p.cg; if (cgg > p.cg) cgg = p.cg; }
                    else { tap0 = kb * p.tpk; g = 0; ntap = p.taps - tap0 < p.tpk ? p.taps - tap0 : p.tpk; cgg = p.cchunks; }
                    const bool w = __all_sync(0xffffffffu, mbar_wait(a_empty0 + 8 * stage, phase ^ 1, abort_flag, wait_limit));
                    if (!w) { ok = false; break; }
                    const uint32_t fb = a_full0 + 8 * stage;
                    const uint32_t dst = a_base + stage * (p.a_stage_bytes + p.b_stage_bytes) + p.a_stage_bytes;
                    // the K block's planes are consecutive (tap, chunk) planes of the bank, which is stored filter tile by
                    // filter tile ([tile][plane][row]; with one tile that is the packed layout itself): one copy
                    if (lane == 0) {
                        const uint32_t bytes = (uint32_t)(ntap * cgg * p.n_tile * 16);
                        mbar_expect_tx(fb, bytes);
                        bulk_copy(dst, reinterpret_cast<const uint8_t*>(p.a.w) + (long long)nt * p.bank_tile_bytes +
                                           (long long)(tap0 * p.cchunks + g * p.cg) * p.n_tile * 16, bytes, fb);
                    }
                    if (++stage == (uint32_t)p.a_stages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok && lane == 0) raise(ctrl, p.status, 1);
        }
    } else if (issuer >= 0) {
        // ------------------------------ MMA issuer --------------------------------
        if (lane == 0 && issuer < (int)n_issuers) {
            // instruction descriptor: D = f32, A = B = bf16, both K-major, N = n_tile, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_tile >> 3) << 17) | ((128u >> 4) << 24);
            uint32_t a_stage = 0, a_phase = 0, b_stage = 0, b_phase = 0;
            uint32_t acc_phase0 = 0, acc_phase1 = 0;
            int local = 0;
            bool ok = true;
            if (MODE == MODE_FLAT_RESIDENT) ok = mbar_wait(b_full0, 0, abort_flag, wait_limit);
            for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++local) {
                const int acc = local & 1;
                const uint32_t ph = acc ? acc_phase1 : acc_phase0;
                if (!mbar_wait(tempty0 + 8 * acc, ph ^ 1, abort_flag, wait_limit)) { ok = false; break; }
                if (acc) acc_phase1 ^= 1; else acc_phase0 ^= 1;
                tc_fence_after();
                const int nt = tile - (int)fdiv((uint32_t)tile, p.div_ntiles) * p.n_tiles;
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * p.tps * p.n_tile);
                uint32_t accumulate = 0;
                if (MODE == MODE_FLAT_UNIFIED) {
                    // one wait and one commit per stage; each tile of the step has its own issuing warp and accumulator
                    const uint32_t stage_bytes = (uint32_t)(p.a_stage_bytes + p.b_stage_bytes);
                    const uint32_t a_ks = 2u * (uint32_t)(p.a_par * p.rows_a), b_ks = 2u * (uint32_t)p.n_tile;
                    const uint32_t d_acc = d_tmem + (uint32_t)(issuer * p.n_tile);
                    for (int g = 0; g < p.groups && ok; ++g) {
                        if (!mbar_wait(a_full0 + 8 * a_stage, a_phase, abort_flag, wait_limit)) { ok = false; break; }
                        tc_fence_after();
                        int cgg = p.cchunks - g * p.cg;
                        if (cgg > p.cg) cgg = p.cg;
                        const int ksteps = cgg >> 1;
                        const uint32_t sa = a_base + a_stage * stage_bytes;
                        uint32_t a_row = ((sa >> 4) + (uint32_t)(issuer * 128)) | ((uint32_t)(p.a_par * p.rows_a) << 16);
                        const uint32_t a_row0 = a_row;
                        uint32_t b_lo = ((sa + (uint32_t)p.a_stage_bytes) >> 4) | ((uint32_t)p.n_tile << 16);
                        const uint32_t b_tap = (uint32_t)(cgg * p.n_tile);
                        if (p.a.x_s2d) {
                            if (ksteps == 1) issue_taps9<1>(d_acc, a_row0, p.tap_off, b_lo, b_tap, a_ks, b_ks, idesc, accumulate);
                            else issue_taps9<2>(d_acc, a_row0, p.tap_off, b_lo, b_tap, a_ks, b_ks, idesc, accumulate);
                            accumulate = 1;
                        } else
                        for (int r = 0; r < p.a.R; ++r) {
                            for (int sx = 0; sx < p.a.S; ++sx) {
                                issue_ksteps(ksteps, d_acc, a_row + (uint32_t)sx, b_lo, a_ks, b_ks, idesc, accumulate);
                                accumulate = 1;
                                b_lo += b_tap;
                            }
                            a_row += (uint32_t)p.Wp_in;
                        }
                        umma_commit(a_empty0 + 8 * a_stage);     // releases the stage once these MMAs have read it
                        if (++a_stage == (uint32_t)p.a_stages) { a_stage = 0; a_phase ^= 1; }
                    }
                } else if (MODE != MODE_GATHER) {
                    // Descriptors differ only in their 16-byte start-address field, so the inner loops
                    // just add row counts to the low word (rows are 16 bytes: one row = one address unit).
                    for (int g = 0; g < p.groups && ok; ++g) {
                        if (!mbar_wait(a_full0 + 8 * a_stage, a_phase, abort_flag, wait_limit)) { ok = false; break; }
                        tc_fence_after();
                        int cgg = p.cchunks - g * p.cg;
                        if (cgg > p.cg) cgg = p.cg;
                        const int ksteps = cgg >> 1;
                        uint32_t a_row = ((a_base + a_stage * p.a_stage_bytes) >> 4) | ((uint32_t)(p.a_par * p.rows_a) << 16);
                        uint32_t b_tap = 0;
                        if (MODE == MODE_FLAT_RESIDENT)
                            b_tap = ((b_base >> 4) + (uint32_t)(g * p.cg * p.n_tile)) | ((uint32_t)p.n_tile << 16);   // this CTA's filter tile only
                        const uint32_t a_ks = 2u * (uint32_t)(p.a_par * p.rows_a);
                        const uint32_t b_ks = 2u * (uint32_t)p.n_tile;
                        const uint32_t b_tap_step = (uint32_t)(p.cchunks * p.n_tile);
                        if (MODE == MODE_FLAT_RESIDENT && p.a.x_s2d) {
                            // nine taps over the four parity images: each tap's operand starts at its own row of the stage
                            // (unrolled: an index into the parameters that is not a constant costs some 300 cycles per use)
#pragma unroll
                            for (int tap = 0; tap < 9; ++tap)
                                issue_ksteps(ksteps, d_tmem, a_row + (uint32_t)p.tap_off[tap], b_tap + (uint32_t)tap * b_tap_step, a_ks, b_ks,
                                             idesc, tap ? 1u : accumulate);
                            accumulate = 1;
                        } else if (MODE == MODE_FLAT_RESIDENT) {
                            if (p.a.R == 3 && p.a.S == 3)
                                issue_flat_resident_k<3, 3>(ksteps, d_tmem, a_row, b_tap, (uint32_t)p.Wp_in, a_ks, b_ks, b_tap_step, idesc, accumulate);
                            else if (p.a.R == 3)
                                issue_flat_resident_k<3, 1>(ksteps, d_tmem, a_row, b_tap, (uint32_t)p.Wp_in, a_ks, b_ks, b_tap_step, idesc, accumulate);
                            else
                                issue_flat_resident_k<1, 1>(ksteps, d_tmem, a_row, b_tap, (uint32_t)p.Wp_in, a_ks, b_ks, b_tap_step, idesc, accumulate);
                            accumulate = 1;
                        } else {
                        for (int r = 0; r < p.a.R && ok; ++r) {
                            // streamed filters: one block per (K group, filter row).  Every 128-position tile of the step
                            // uses it: its own accumulator and issuing warp, its activation rows 128 further on
                            if (!mbar_wait(b_full0 + 8 * b_stage, b_phase, abort_flag, wait_limit)) { ok = false; break; }
                            tc_fence_after();
                            uint32_t b_lo = ((b_base + b_stage * p.b_stage_bytes) >> 4) | ((uint32_t)p.n_tile << 16);
                            for (int sx = 0; sx < p.a.S; ++sx) {
                                issue_ksteps(ksteps, d_tmem + (uint32_t)(issuer * p.n_tile), a_row + (uint32_t)sx + (uint32_t)(issuer * 128),
                                             b_lo, a_ks, b_ks, idesc, accumulate);
                                accumulate = 1;
                                b_lo += (uint32_t)(cgg * p.n_tile);
                            }
                            umma_commit(b_empty0 + 8 * b_stage);
                            if (++b_stage == (uint32_t)p.b_stages) { b_stage = 0; b_phase ^= 1; }
                            a_row += (uint32_t)p.Wp_in;
                        }
                        }
                        if (!ok) break;
                        umma_commit(a_empty0 + 8 * a_stage);     // releases the stage once these MMAs have read it
                        if (++a_stage == (uint32_t)p.a_stages) { a_stage = 0; a_phase ^= 1; }
                    }
                    // streamed 3x3 layer with a projection shortcut taken in: the K groups of the second input, centre tap only
                    for (int g2 = 0; MODE == MODE_FLAT_STREAM && g2 < p.groups2 && ok; ++g2) {
                        if (!mbar_wait(a_full0 + 8 * a_stage, a_phase, abort_flag, wait_limit)) { ok = false; break; }
                        if (!mbar_wait(b_full0 + 8 * b_stage, b_phase, abort_flag, wait_limit)) { ok = false; break; }
                        tc_fence_after();
                        int cgg = p.cchunks2 - g2 * p.cg;
                        if (cgg > p.cg) cgg = p.cg;
                        const uint32_t a_row = (((a_base + a_stage * p.a_stage_bytes) >> 4) + (uint32_t)p.halo + (uint32_t)(issuer * 128)) |
                                               ((uint32_t)p.rows_a << 16);
                        const uint32_t b_lo = ((b_base + b_stage * p.b_stage_bytes) >> 4) | ((uint32_t)p.n_tile << 16);
                        issue_ksteps(cgg >> 1, d_tmem + (uint32_t)(issuer * p.n_tile), a_row, b_lo, 2u * (uint32_t)p.rows_a,
                                     2u * (uint32_t)p.n_tile, idesc, accumulate);
                        accumulate = 1;
                        umma_commit(b_empty0 + 8 * b_stage);
                        if (++b_stage == (uint32_t)p.b_stages) { b_stage = 0; b_phase ^= 1; }
                        umma_commit(a_empty0 + 8 * a_stage);
                        if (++a_stage == (uint32_t)p.a_stages) { a_stage = 0; a_phase ^= 1; }
                    }
                } else {
                    const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
                    for (int kb = 0; kb < p.kblocks; ++kb) {
                        if (!mbar_wait(a_full0 + 8 * a_stage, a_phase, abort_flag, wait_limit)) { ok = false; break; }
                        tc_fence_after();
                        int planes;
                        if (p.groups > 1) { const int g = kb % p.groups; planes = p.cchunks - g * p.cg; if (planes > p.cg) planes = p.cg; }
                        else { const int tap0 = kb * p.tpk; planes = (p.taps - tap0 < p.tpk ? p.taps - tap0 : p.tpk) * p.cchunks; }
                        const uint32_t sa = a_base + a_stage * stage_bytes;
                        const uint32_t sb = sa + p.a_stage_bytes;
                        uint32_t a_lo = (sa >> 4) | (128u << 16);
                        uint32_t b_lo = (sb >> 4) | ((uint32_t)p.n_tile << 16);
                        for (int ks = 0; ks < planes / 2; ++ks) {
                            umma_bf16_lo(d_tmem, a_lo, b_lo, idesc, accumulate);
                            accumulate = 1;
                            a_lo += 256u;
                            b_lo += 2u * (uint32_t)p.n_tile;
                        }
                        umma_commit(a_empty0 + 8 * a_stage);
                        if (++a_stage == (uint32_t)p.a_stages) { a_stage = 0; a_phase ^= 1; }
                    }
                }
                if (ok) umma_commit(tfull0 + 8 * acc);   // accumulator complete
            }
            if (!ok) raise(ctrl, p.status, 2);
        }
    } else if (warp < 2 + EPI) {
        // ------------------------------ epilogue ----------------------------------
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31 belong to this warp
        const int half = (warp - 2) >> 2;             // with 8 epilogue warps: which half of the columns
        const int row = quarter * 32 + lane;          // accumulator row = position within the tile
        uint32_t acc_phase0 = 0, acc_phase1 = 0;
        int local = 0;
        bool ok = true;
        const uint4* __restrict__ res = reinterpret_cast<const uint4*>(p.a.res);
        const __nv_bfloat16* __restrict__ res_s = reinterpret_cast<const __nv_bfloat16*>(p.a.res);
        uint4* __restrict__ y = reinterpret_cast<uint4*>(p.a.y);
        for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x, ++local) {
            const int mt = (int)fdiv((uint32_t)tile, p.div_ntiles);
            const int nt = tile - mt * p.n_tiles;
            const int acc = local & 1;
            const uint32_t ph = acc ? acc_phase1 : acc_phase0;
            for (int t = 0; t < p.tps; ++t) {
            const long long f = ((long long)mt * p.tps + t) * 128 + row;
            const bool exists = f < p.m_total;
            const int n = (int)fdiv((uint32_t)f, p.div_p2out);
            const int rem = (int)f - n * p.P2_out;
            const int hp = (int)fdiv((uint32_t)rem, p.div_qp), wq = rem - hp * p.Qp;
            const bool interior = exists && hp >= 1 && hp <= p.a.P && wq >= 1 && wq <= p.a.Q;
            const int k_base = nt * p.n_tile;
            int cols = p.a.K_pad - k_base;
            if (cols > p.n_tile) cols = p.n_tile;
            const long long vec0 = (long long)(k_base >> 3) * p.plane_out + f;     // shortcut operand: vector of columns 0..7
            // where the output goes: the same position - or, for a parity-split output tensor, pixel (h, w) of image n as
            // pixel (h >> 1, w >> 1) of image pp * N + n, pp numbering the parities (h & 1, w & 1) as 00, 10, 11, 01 (the
            // border positions go along: row -1 becomes row -1 of the odd-row images, and so on)
            long long fy = f;
            if (p.y_split) {
                const int h = hp - 1, w = wq - 1;
                const int pp = (h & 1) ? ((w & 1) ? 2 : 1) : ((w & 1) ? 3 : 0);
                fy = ((long long)pp * p.a.N + n) * p.y_P2h + ((h >> 1) + 1) * p.y_Wh2 + ((w >> 1) + 1);
            }
            const long long yvec0 = (long long)(k_base >> 3) * p.plane_y + fy;
            int c_begin = 0, c_end = cols;
            if (EPI == 8) {
                const int first = ((cols >> 4) + 1) / 2 * 16;                      // columns of the first half
                if (half) c_begin = first; else c_end = first;
            }
            // the same-shape residual of this warp's first 64 columns is requested before the accumulator
            // is waited for; later columns are requested four 16-column chunks ahead
            uint4 rq[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) rq[i] = make_uint4(0, 0, 0, 0);
            const bool res1 = interior && p.a.res_mode == 1;
            if (res1 && !p.a.scatter) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (c_begin + i * 8 < c_end) rq[i] = __ldg(res + vec0 + (long long)((c_begin >> 3) + i) * p.plane_out);
            }
            if (t == 0) {
                ok = mbar_wait(tfull0 + 8 * acc, ph, abort_flag, wait_limit);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (acc) acc_phase1 ^= 1; else acc_phase0 ^= 1;
                tc_fence_after();
            }
            long long res_vec = 0;
            if (p.a.res_mode == 2) {
                const int rWp = p.a.res_W + 2, rP2 = (p.a.res_H + 2) * rWp;
                res_vec = (long long)n * rP2 + (long long)((hp - 1) * p.a.res_stride + 1) * rWp + ((wq - 1) * p.a.res_stride + 1);
            }
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((acc * p.tps + t) * p.n_tile);
            if (p.a.scatter) {
                // Scattered output: this filter tile owns the output chunks [q_begin, q_end) of the full-width tensor, and its
                // accumulator columns are the kept filters of those chunks in channel order.  Columns are read 16 at a
                // time and parked in a per-warp strip of shared memory (a ring of 32 columns per row, row pitch 33 words:
                // conflict-free); a chunk of 8 output channels then picks its kept channels' columns from there by index -
                // the same index in every lane - and takes the shortcut alone for the others.
                int q_begin = schunk0[nt], q_end = schunk0[nt + 1];
                if (EPI == 8) {
                    const int mid = q_begin + (q_end - q_begin + 1) / 2;
                    if (half) q_begin = mid; else q_end = mid;
                }
                float* strip = sstrip + ((warp - 2) * 32 + lane) * 33;
                const long long rplane = (long long)p.a.N * (p.a.res_H + 2) * (p.a.res_W + 2);
                uint4 rnext = make_uint4(0, 0, 0, 0);
                if (res1 && q_begin < q_end) rnext = __ldg(res + (long long)q_begin * p.plane_out + f);
                int loaded = -1;                 // accumulator columns [.., loaded) of this tile are in the strip
                for (int q = q_begin; q < q_end; ++q) {
                    const uint4 rcur = rnext;
                    if (res1 && q + 1 < q_end) rnext = __ldg(res + (long long)(q + 1) * p.plane_out + f);
                    const int4 m0 = *reinterpret_cast<const int4*>(smap + 8 * q);
                    const int4 m1 = *reinterpret_cast<const int4*>(smap + 8 * q + 4);
                    const int col[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
                    int first = -1, last = -1;   // accumulator columns (within the tile) this chunk needs: consecutive ones
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (col[e] >= 0) { last = col[e] - k_base; if (first < 0) first = last; }
                    if (loaded < 0 && first >= 0) loaded = first & ~15;                            // first group this warp needs
                    while (last >= loaded && loaded >= 0) {
                        uint32_t v[16];
                        __syncwarp();
                        tmem_ld16(taddr + (uint32_t)loaded, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i) strip[(loaded & 16) + i] = __uint_as_float(v[i]);
                        loaded += 16;
                    }
                    if (!exists) continue;
                    uint4 o = make_uint4(0, 0, 0, 0);
                    if (interior) {
                        float fv[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) fv[e] = col[e] >= 0 ? strip[(col[e] - k_base) & 31] + bias_s[col[e]] : 0.0f;
                        if (p.a.res_mode == 1) {
                            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&rcur);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 g = __bfloat1622float2(h2[i]);
                                fv[2 * i] += g.x;
                                fv[2 * i + 1] += g.y;
                            }
                        } else if (p.a.res_mode == 2) {
                            const int cs = 8 * q - p.a.res_pad_lo;
                            if (cs >= 0 && cs + 8 <= p.a.res_C_pad && (cs & 7) == 0) {
                                const uint4 raw = __ldg(res + (long long)(cs >> 3) * rplane + res_vec);
                                const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const float2 g = __bfloat1622float2(h2[i]);
                                    fv[2 * i] += g.x;
                                    fv[2 * i + 1] += g.y;
                                }
                            } else if (cs + 8 > 0 && cs < p.a.res_C) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const int c = cs + i;
                                    if (c >= 0 && c < p.a.res_C)
                                        fv[i] += __bfloat162float(res_s[((long long)(c >> 3) * rplane + res_vec) * 8 + (c & 7)]);
                                }
                            }
                        }
                        if (p.a.relu) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) fv[i] = fmaxf(fv[i], 0.0f);
                        }
                        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
                        for (int i = 0; i < 4; ++i) o2[i] = __floats2bfloat162_rn(fv[2 * i], fv[2 * i + 1]);
                    }
                    y[(long long)q * p.plane_y + fy] = o;
                }
            } else if (p.a.res_mode != 2) {
                // Dense output, no shortcut or a same-shape one: the shortcut's vectors are requested 64 columns ahead into
                // four register pairs used in turn (no copies), the ReLU is folded into the bf16 conversion.  (32 columns
                // per tensor-memory load were faster on the layers this loop bounds, but the registers cost the layers with
                // resident filters their second CTA per SM: 47 -> 57 us on ResNet-50's 256 -> 77 layer.)  Layers with a short reduction are bound by this loop's instruction count (ResNet-50's
                // 154 -> 1024 layers: 290 instructions per 16 columns and lane before, 11 % tensor-pipe activity).
                auto process16 = [&](int c0, const uint4& r0, const uint4& r1) {
                    uint32_t v[16];
                    __syncwarp();
                    tmem_ld16(taddr + c0, v);
                    tmem_ld_wait();
                    if (!exists) return;
                    uint4* yp = y + yvec0 + (long long)(c0 >> 3) * p.plane_y;
                    const float4* b4 = reinterpret_cast<const float4*>(bias_s + k_base + c0);
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        const uint4& rr = ch == 0 ? r0 : r1;
                        const float4 ba = b4[2 * ch], bb = b4[2 * ch + 1];
                        float f0 = __uint_as_float(v[8 * ch + 0]) + ba.x, f1 = __uint_as_float(v[8 * ch + 1]) + ba.y;
                        float f2 = __uint_as_float(v[8 * ch + 2]) + ba.z, f3 = __uint_as_float(v[8 * ch + 3]) + ba.w;
                        float f4 = __uint_as_float(v[8 * ch + 4]) + bb.x, f5 = __uint_as_float(v[8 * ch + 5]) + bb.y;
                        float f6 = __uint_as_float(v[8 * ch + 6]) + bb.z, f7 = __uint_as_float(v[8 * ch + 7]) + bb.w;
                        if (p.a.res_mode == 1) {
                            // a bf16 is the upper half of the float with the same value
                            f0 += __uint_as_float(rr.x << 16); f1 += __uint_as_float(rr.x & 0xffff0000u);
                            f2 += __uint_as_float(rr.y << 16); f3 += __uint_as_float(rr.y & 0xffff0000u);
                            f4 += __uint_as_float(rr.z << 16); f5 += __uint_as_float(rr.z & 0xffff0000u);
                            f6 += __uint_as_float(rr.w << 16); f7 += __uint_as_float(rr.w & 0xffff0000u);
                        }
                        uint4 o;
                        if (p.a.relu) {
                            o.x = pack_bf16x2_relu(f0, f1); o.y = pack_bf16x2_relu(f2, f3);
                            o.z = pack_bf16x2_relu(f4, f5); o.w = pack_bf16x2_relu(f6, f7);
                        } else {
                            o.x = pack_bf16x2(f0, f1); o.y = pack_bf16x2(f2, f3);
                            o.z = pack_bf16x2(f4, f5); o.w = pack_bf16x2(f6, f7);
                        }
                        if (!interior) o = make_uint4(0, 0, 0, 0);
                        yp[(long long)ch * p.plane_y] = o;
                    }
                };
                auto refill = [&](int c0, uint4& r0, uint4& r1) {     // shortcut vectors of columns c0 .. c0+15
                    if (!res1 || c0 >= c_end) return;
                    const uint4* rp = res + vec0 + (long long)(c0 >> 3) * p.plane_out;
                    r0 = __ldg(rp);
                    r1 = __ldg(rp + p.plane_out);
                };
                for (int c0 = c_begin; c0 < c_end; c0 += 64) {
                    process16(c0, rq[0], rq[1]);
                    refill(c0 + 64, rq[0], rq[1]);
                    if (c0 + 16 < c_end) { process16(c0 + 16, rq[2], rq[3]); refill(c0 + 80, rq[2], rq[3]); }
                    if (c0 + 32 < c_end) { process16(c0 + 32, rq[4], rq[5]); refill(c0 + 96, rq[4], rq[5]); }
                    if (c0 + 48 < c_end) { process16(c0 + 48, rq[6], rq[7]); refill(c0 + 112, rq[6], rq[7]); }
                }
            } else
            for (int c0 = c_begin; c0 < c_end; c0 += 16) {
                uint32_t v[16];
                __syncwarp();
                tmem_ld16(taddr + c0, v);
                tmem_ld_wait();
                if (exists) {
                const long long out_vec = yvec0 + (long long)(c0 >> 3) * p.plane_y;
                uint4 o[2];
                o[0] = make_uint4(0, 0, 0, 0);
                o[1] = o[0];
                if (interior) {
                    float fv[16];
                    const float4* b4 = reinterpret_cast<const float4*>(bias_s + k_base + c0);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float4 b = b4[i];
                        fv[4 * i + 0] = __uint_as_float(v[4 * i + 0]) + b.x;
                        fv[4 * i + 1] = __uint_as_float(v[4 * i + 1]) + b.y;
                        fv[4 * i + 2] = __uint_as_float(v[4 * i + 2]) + b.z;
                        fv[4 * i + 3] = __uint_as_float(v[4 * i + 3]) + b.w;
                    }
                    if (p.a.res_mode == 1) {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&rq[hh]);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 g = __bfloat1622float2(h2[i]);
                                fv[8 * hh + 2 * i] += g.x;
                                fv[8 * hh + 2 * i + 1] += g.y;
                            }
                        }
                    } else if (p.a.res_mode == 2) {
                        // shortcut by subsampling: output channel k takes input channel k - pad_lo
                        const long long rplane = (long long)p.a.N * (p.a.res_H + 2) * (p.a.res_W + 2);
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            const int cs = k_base + c0 + 8 * hh - p.a.res_pad_lo;
                            if (cs >= 0 && cs + 8 <= p.a.res_C_pad && (cs & 7) == 0) {
                                const uint4 raw = __ldg(res + (long long)(cs >> 3) * rplane + res_vec);
                                const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const float2 g = __bfloat1622float2(h2[i]);
                                    fv[8 * hh + 2 * i] += g.x;
                                    fv[8 * hh + 2 * i + 1] += g.y;
                                }
                            } else if (cs + 8 > 0 && cs < p.a.res_C) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const int c = cs + i;
                                    if (c >= 0 && c < p.a.res_C)
                                        fv[8 * hh + i] += __bfloat162float(res_s[((long long)(c >> 3) * rplane + res_vec) * 8 + (c & 7)]);
                                }
                            }
                        }
                    }
                    if (p.a.relu) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) fv[i] = fmaxf(fv[i], 0.0f);
                    }
                    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(o);
#pragma unroll
                    for (int i = 0; i < 8; ++i) o2[i] = __floats2bfloat162_rn(fv[2 * i], fv[2 * i + 1]);
                }
                y[out_vec] = o[0];
                y[out_vec + p.plane_y] = o[1];
                }
                // rotate the residual queue and refill its tail
#pragma unroll
                for (int i = 0; i < 6; ++i) rq[i] = rq[i + 2];
                if (res1 && c0 + 64 < c_end) {   // (dense output only: this loop is not entered when the output is scattered)
                    const long long vn = vec0 + (long long)((c0 + 64) >> 3) * p.plane_out;
                    rq[6] = __ldg(res + vn);
                    rq[7] = __ldg(res + vn + p.plane_out);
                }
            }
            }   // tiles of the step
            if (!ok) break;
            tc_fence_before();
            mbar_arrive(tempty0 + 8 * acc);
        }
        if (!ok && lane == 0) raise(ctrl, p.status, 3);
    } else if (MODE == MODE_FLAT_STREAM) {
        // ------------------------------ filter producer (streamed filters) --------------
        if (warp == 2 + EPI) {
            // One filter block per (K group, filter row): [tap of the row][chunk][filter].  When a tile takes all filters
            // a tap's chunks are one contiguous run of the packed bank: one copy per tap; otherwise one copy per
            // (tap, chunk), spread over the lanes.
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            const bool whole = p.n_tiles == 1;
            for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
                const int nt = tile - (int)fdiv((uint32_t)tile, p.div_ntiles) * p.n_tiles;
                int nrows = p.a.K_pad - nt * p.n_tile;
                if (nrows > p.n_tile) nrows = p.n_tile;
                for (int g = 0; g < p.groups && ok; ++g) {
                    int cgg = p.cchunks - g * p.cg;
                    if (cgg > p.cg) cgg = p.cg;
                    for (int r = 0; r < p.a.R; ++r) {
                        const bool w = __all_sync(0xffffffffu, mbar_wait(b_empty0 + 8 * stage, phase ^ 1, abort_flag, wait_limit));
                        if (!w) { ok = false; break; }
                        const uint32_t fb = b_full0 + 8 * stage;
                        const uint32_t dst = b_base + stage * p.b_stage_bytes;
                        if (lane == 0) mbar_expect_tx(fb, (uint32_t)(p.a.S * cgg * nrows * 16));
                        __syncwarp();
                        const uint4* src = wv + ((long long)(r * p.a.S) * p.cchunks + g * p.cg) * p.a.K_pad + nt * p.n_tile;
                        if (whole) {
                            if (lane < p.a.S)
                                bulk_copy(dst + lane * cgg * p.n_tile * 16, src + (long long)lane * p.cchunks * p.a.K_pad, (uint32_t)(cgg * nrows * 16), fb);
                        } else {
                            for (int i = lane; i < p.a.S * cgg; i += 32) {
                                const int sx = i / cgg, c = i - sx * cgg;
                                bulk_copy(dst + i * p.n_tile * 16, src + ((long long)sx * p.cchunks + c) * p.a.K_pad, (uint32_t)(nrows * 16), fb);
                            }
                        }
                        if (++stage == (uint32_t)p.b_stages) { stage = 0; phase ^= 1; }
                    }
                }
                // the second input's K groups: one block each, the centre tap's filters from the projection's own bank
                for (int g2 = 0; g2 < p.groups2 && ok; ++g2) {
                    int cgg = p.cchunks2 - g2 * p.cg;
                    if (cgg > p.cg) cgg = p.cg;
                    const bool w = __all_sync(0xffffffffu, mbar_wait(b_empty0 + 8 * stage, phase ^ 1, abort_flag, wait_limit));
                    if (!w) { ok = false; break; }
                    const uint32_t fb = b_full0 + 8 * stage;
                    const uint32_t dst = b_base + stage * p.b_stage_bytes;
                    if (lane == 0) mbar_expect_tx(fb, (uint32_t)(cgg * nrows * 16));
                    __syncwarp();
                    const uint4* src = reinterpret_cast<const uint4*>(p.a.w2) + (long long)(g2 * p.cg) * p.a.K_pad + nt * p.n_tile;
                    if (whole) {
                        if (lane == 0) bulk_copy(dst, src, (uint32_t)(cgg * nrows * 16), fb);
                    } else if (lane < cgg) {
                        bulk_copy(dst + lane * p.n_tile * 16, src + (long long)lane * p.a.K_pad, (uint32_t)(nrows * 16), fb);
                    }
                    if (++stage == (uint32_t)p.b_stages) { stage = 0; phase ^= 1; }
                }
            }
            if (!ok && lane == 0) raise(ctrl, p.status, 4);
        }
    } else if (MODE == MODE_GATHER) {
        // ------------------------------ loader threads (gathered activations) -----------
        const int m = threadIdx.x - 32 * (2 + EPI);  // 0..127: row of the tile this thread fills
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
        for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x) {
            const long long f = (long long)fdiv((uint32_t)tile, p.div_ntiles) * 128 + m;
            const int n = (int)fdiv((uint32_t)f, p.div_p2out);
            const int rem = (int)f - n * p.P2_out;
            const int hp = (int)fdiv((uint32_t)rem, p.div_qp), wq = rem - hp * p.Qp;
            const bool interior = f < p.m_total && hp >= 1 && hp <= p.a.P && wq >= 1 && wq <= p.a.Q;
            const int ih0 = (hp - 1) * p.a.stride - p.a.pad, iw0 = (wq - 1) * p.a.stride - p.a.pad;
            const long long base = (long long)n * p.P2_in + (long long)(ih0 + 1) * p.Wp_in + (iw0 + 1);
            uint32_t rmask = 0, smask = 0;       // filter rows / columns that fall inside the image
            if (interior) {
                for (int r = 0; r < p.a.R; ++r) rmask |= (uint32_t)(ih0 + r >= 0 && ih0 + r < p.a.H) << r;
                for (int sx = 0; sx < p.a.S; ++sx) smask |= (uint32_t)(iw0 + sx >= 0 && iw0 + sx < p.a.W) << sx;
            }
            for (int kb = 0; kb < p.kblocks && ok; ++kb) {
                // the eight loads have separate destinations, so all of them are in flight together
                uint4 v[8];
                const int2* L = lut + kb * 8;
                const int planes = L[0].y >> 24;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int2 e = L[i];
                    const bool valid = ((e.y >> 16) & (rmask >> (e.y & 0xff)) & (smask >> ((e.y >> 8) & 0xff)) & 1) != 0;
                    v[i] = make_uint4(0, 0, 0, 0);
                    if (valid) v[i] = __ldg(xv + base + e.x);
                }
                if (!mbar_wait(a_empty0 + 8 * stage, phase ^ 1, abort_flag, wait_limit)) { ok = false; break; }
                uint8_t* dst = smem_raw + (a_base - ctrl_addr) + stage * stage_bytes + m * 16;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (i < planes) *reinterpret_cast<uint4*>(dst + i * 128 * 16) = v[i];
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> MMA reads
                mbar_arrive(a_full0 + 8 * stage);
                if (++stage == (uint32_t)p.a_stages) { stage = 0; phase ^= 1; }
            }
        }
        if (!ok) raise(ctrl, p.status, 5);
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

int pow2_at_least(int v) { int p = 1; while (p < v) p <<= 1; return p; }
int round_up_i(int v, int m) { return (v + m - 1) / m * m; }

const void* kernel_for(int mode, int epi) {
    if (mode == MODE_FLAT_RESIDENT) return epi == 8 ? (const void*)conv_tc_kernel<MODE_FLAT_RESIDENT, 8> : (const void*)conv_tc_kernel<MODE_FLAT_RESIDENT, 4>;
    if (mode == MODE_FLAT_STREAM) return epi == 8 ? (const void*)conv_tc_kernel<MODE_FLAT_STREAM, 8> : (const void*)conv_tc_kernel<MODE_FLAT_STREAM, 4>;
    if (mode == MODE_FLAT_UNIFIED) return epi == 8 ? (const void*)conv_tc_kernel<MODE_FLAT_UNIFIED, 8> : (const void*)conv_tc_kernel<MODE_FLAT_UNIFIED, 4>;
    return epi == 8 ? (const void*)conv_tc_kernel<MODE_GATHER, 8> : (const void*)conv_tc_kernel<MODE_GATHER, 4>;
}

constexpr unsigned kSmemMax = 232448u - 1024u;     // opt-in dynamic shared memory per CTA
constexpr unsigned kSmemPerSm = 233472u;           // 228 KB per SM

// Filters per CTA tile.  At most 128: two CTAs then share an SM's 512 tensor-memory columns, which doubles the
// epilogue warps and the loads in flight; a 128-wide MMA already runs at the full tensor rate.
void choose_filter_tile(const ConvArgs& a, int K_pad, int* n_tile_out, int* n_tiles_out) {
    const int sms = sm_count();
    const int taps = a.R * a.S;
    const bool flat = a.stride == 1 && a.P == a.H && a.Q == a.W &&
                      ((a.R == 1 && a.S == 1 && a.pad == 0) || (a.R == 3 && (a.S == 3 || a.S == 1) && a.pad == 1));
    const long long m_total = (long long)a.N * (a.P + 2) * (a.Q + 2);
    const long long m_tiles = (m_total + 127) / 128;
    int n_tiles = (K_pad + 127) / 128;
    int n_tile = round_up_i((K_pad + n_tiles - 1) / n_tiles, 16);
    const long long bank = (long long)taps * a.C_pad * K_pad * 2;
    if (!(flat && bank <= 100 * 1024)) {
        // Few position tiles: split the filters over more CTAs, but only while that doubles the SMs in use.  An MMA
        // costs about the same for 64 filters as for 128, so a split that merely puts two half-width CTAs on an SM
        // doubles the work (measured, ResNet-18 batch 64: 512->359 filters at 7x7, 72 us split in six, 39 us in three).
        while (m_tiles * n_tiles * 2 <= sms && n_tile > 64) {
            n_tiles *= 2;
            n_tile = round_up_i((K_pad + n_tiles - 1) / n_tiles, 16);
        }
        // A 1x1 layer with a long reduction and 129-192 filters is bound by the MMA count: one tile of all filters (one
        // position tile per step: tensor memory) instead of two of half the width, an MMA costing the pipe about the
        // same for 80 filters as for 160 (measured, ResNet-50 batch 128: 1024 -> 160 at 14x14 30.6 -> 28.5 us,
        // 512 -> 160 at 28x28 45.1 -> 42.1 us; with 320 filters two tiles of 160 lose against three of 112).
        if (taps == 1 && flat && K_pad > 128 && K_pad <= 192 && m_tiles >= sms) { n_tiles = 1; n_tile = K_pad; }
    }
    *n_tile_out = n_tile;
    *n_tiles_out = (K_pad + n_tile - 1) / n_tile;
}

}  // namespace

void conv_tc_filter_tile(const ConvArgs& a, int K_pad, int* n_tile, int* n_tiles) { choose_filter_tile(a, K_pad, n_tile, n_tiles); }

int plan_conv_tc(const ConvArgs& a, ConvPlanTC* plan, char* err, size_t err_len) {
    memset(plan, 0, sizeof(*plan));
    const int sms = sm_count();
    if (a.C_pad % 16 || a.K_pad % 16) { snprintf(err, err_len, "channel counts must be padded to 16"); return 1; }
    if (a.W > kMaxWidth || a.Q > kMaxWidth) { snprintf(err, err_len, "images wider than %d are not supported", kMaxWidth); return 1; }
    const int cchunks = a.C_pad / 8;
    const int taps = a.R * a.S;
    const int a_par = a.x_s2d ? 4 : 1;       // activation runs per chunk in a stage (parity images)
    plan->flat = (a.stride == 1 && a.P == a.H && a.Q == a.W &&
                  ((a.R == 1 && a.S == 1 && a.pad == 0) || (a.R == 3 && (a.S == 3 || a.S == 1) && a.pad == 1))) ? 1 : 0;
    plan->cg = cchunks < 8 ? cchunks : 8;
    plan->groups = (cchunks + plan->cg - 1) / plan->cg;
    const long long m_total = (long long)a.N * (a.P + 2) * (a.Q + 2);
    const long long m_tiles = (m_total + 127) / 128;
    if (m_total + 128 >= (1ll << 31)) { snprintf(err, err_len, "more than 2^31 output positions"); return 1; }

    // --- filter tile ---
    int n_tile, n_tiles;
    if (a.n_tile_forced > 0) { n_tile = a.n_tile_forced; n_tiles = (a.K_pad + n_tile - 1) / n_tile; }
    else choose_filter_tile(a, a.K_pad, &n_tile, &n_tiles);
    // Resident filters: a CTA keeps ITS filter tile's part of the bank (the grid is a multiple of the number of filter
    // tiles, so a CTA's tiles all have the same one), all taps and channels of it, in shared memory for the whole
    // kernel.  (With the whole bank as the unit, the layers that write ResNet-50's residual stream at 14x14 and 7x7 -
    // 160 -> 1024 and 320 -> 2048 filters, 327 KB and 1.3 MB - streamed their filters with one CTA on an SM; their
    // time goes to the epilogue, which a second CTA's warps double.)
    // Measured at batch 128 (single layers, cold L2): 80 -> 512 at 28x28 59.4 -> 51.6 us (20 KB instead of the whole 82 KB:
    // more activation stages), 160 -> 1024 at 14x14 45.3 -> 39.6 us; but 320 -> 2048 at 7x7 38.9 -> 47.6 us and the
    // 256 -> 512 projection 55.1 -> 59.1 us, whose 64-80 KB tile parts leave two stages of four channel chunks: a layer
    // whose whole bank does not fit takes the resident form only with a part of at most 48 KB.
    const long long bank = (long long)taps * a.C_pad * n_tile * 2;
    const long long whole_bank = (long long)taps * a.C_pad * a.K_pad * 2;
    bool bank_fits = plan->flat && bank <= 100 * 1024 && (whole_bank <= 100 * 1024 || bank <= 48 * 1024);
    plan->n_tile = n_tile; plan->n_tiles = n_tiles;

    unsigned smem = (unsigned)sizeof(Ctrl) + (unsigned)a.K_pad * 4u + 1024u;
    unsigned scatter_smem = 0;
    if (a.scatter) scatter_smem = (unsigned)round_up_i((a.out_C_pad + n_tiles + 1) * 4, 16) + 8u * 32u * 33u * 4u;
    smem += scatter_smem;
    int want_ctas = 1;
    if (plan->flat) {
        plan->halo = ((a.R - 1) / 2) * (a.W + 2) + (a.S - 1) / 2;      // rows above + columns to the left
        plan->tps = 1;
        // A 128-position tile is fetched with `halo` rows on either side.  On wide images (the 112-wide stem: 114
        // rows each side of 128) that is most of the traffic into shared memory, so such a layer takes the
        // streamed form, whose steps of several tiles share one halo, even though its filters would fit
        // (measured on the ResNet-18 stem at batch 64: 89 us resident, 61 us streamed).
        const bool wide_halo = 2 * plan->halo > 128;
        // rows of one activation run: the step's positions with the halo before and after them (the taps of a strided
        // window over parity images only reach back)
        auto run_rows = [&](int tps) { return round_up_i(tps * 128 + (a_par > 1 ? 1 : 2) * plan->halo, 8); };
        bool stream = !bank_fits || wide_halo;
        const bool unified = stream && (taps == 1 || a_par > 1);
        if (unified) {
            // 1x1 convolutions with a streamed bank, and 3x3 / stride-2 convolutions over parity images (whose activation
            // part of a stage is four times a stride-1 layer's, so that the nine taps' filters beside it are in
            // proportion).  A stage holds one K group of channel chunks: its activation
            // rows for the `tps` position tiles of a step and its filters - one wait and one commit per stage for the
            // issuing threads, one expected-bytes arrival for the producer.  The K group is the largest that still
            // leaves three stages (two in flight while one is read: at 60-100 B/cycle and a latency of one or two
            // thousand cycles about 100 KB have to be in flight), since every stage costs its producer and the
            // issuing threads a fixed 300-500 cycles.  (Measured on ResNet-50, batch 128: the 1024 -> 154 layers
            // 30.9 -> 23.3 us, 512 -> 154 54 -> 40 us.  With several taps a stage would have to hold all taps' filters,
            // which leaves room for two or three K-chunk pairs only: such layers were up to 1.7x slower this way and
            // keep the two-ring form below.)
            const unsigned avail = kSmemMax - smem;
            int best_tps = 0, best_cg = 0, best_stages = 0;
            for (int tps = 4; tps >= 1 && !best_tps; tps >>= 1) {
                if (2 * tps * n_tile > 512 || tps * 128 + plan->halo + 8 > kGuardVectors) continue;
                if (tps > 1 && ((m_tiles + tps - 1) / tps) * n_tiles < sms / 2) continue;
                const int rows = run_rows(tps);
                // (parity images: four runs per chunk, at most 16 runs per stage)
                for (int cg = a_par > 1 ? (cchunks < 4 ? cchunks : 4) : (cchunks < 16 ? cchunks : 16) & ~1; cg >= 2; cg -= 2) {
                    const unsigned st = (unsigned)(a_par * cg * rows * 16 + taps * cg * n_tile * 16);
                    int stages = (int)(avail / st);
                    if (stages > kMaxStages) stages = kMaxStages;
                    if (stages == 7) stages = 6;          // the producer warps (2, 3 or 4 of them) must divide the stages
                    if (stages == 5) stages = 4;
                    const int groups = (cchunks + cg - 1) / cg;
                    if (stages >= (groups >= 3 ? 3 : 2)) { best_tps = tps; best_cg = cg; best_stages = stages; break; }
                }
            }
            if (!best_tps) { snprintf(err, err_len, "tile does not fit shared memory"); return 1; }
            plan->tps = best_tps; plan->cg = best_cg; plan->a_stages = best_stages;
            plan->groups = (cchunks + best_cg - 1) / best_cg;
            plan->rows_a = run_rows(plan->tps);
            plan->b_resident = 0;
            plan->b_stages = 0;
            plan->blocked_bank = 1;
            bank_fits = false;
            smem += (unsigned)plan->a_stages * (unsigned)(a_par * plan->cg * plan->rows_a * 16 + taps * plan->cg * n_tile * 16);
        } else {
        if (stream) {
            // Streamed filters: a filter block holds one filter row (S taps) of a K group.  Every block costs the issuing
            // thread a barrier test, a fence and a commit (some 300 cycles) on top of its MMAs, and a block per tap left a
            // third of the main loop to that.  Several 128-position tiles per step share every block: layers with few
            // positions and many filters re-stream the bank once per position tile and are bound by L2 bandwidth, so
            // sharing pays even when it leaves only half of the SMs with a CTA (measured on ResNet-18 at batch 64:
            // 368->512 filters at 7x7, 55 us with 164 single-tile CTAs, 32 us with 84 two-tile CTAs).  The search prefers
            // three blocks in flight over two, then more tiles per step, then longer K groups.
            bool found = false;
            for (int want_b = 3; want_b >= 2 && !found; --want_b)
                for (int tps = 4; tps >= 1 && !found; tps >>= 1) {
                    if (2 * tps * n_tile > 512 || tps * 128 + plan->halo + 8 > kGuardVectors) continue;
                    if (tps > 1 && ((m_tiles + tps - 1) / tps) * n_tiles < sms * 2 / 5) continue;
                    const int cg_hi = bank_fits ? plan->cg : (cchunks < 12 ? cchunks : 12), cg_lo = bank_fits ? plan->cg : (cchunks < 4 ? cchunks : 4);
                    for (int cg = cg_hi; cg >= cg_lo && !found; cg -= 2) {
                        const unsigned b_try = (unsigned)(a.S * cg * n_tile * 16), a_try = (unsigned)(cg * run_rows(tps) * 16);
                        if (smem + (unsigned)want_b * b_try + 2u * a_try > kSmemMax) continue;
                        found = true;
                        plan->tps = tps; plan->cg = cg; plan->groups = (cchunks + cg - 1) / cg;
                    }
                }
            if (!found && !bank_fits) { snprintf(err, err_len, "tile does not fit shared memory"); return 1; }
        }
        if (bank_fits && wide_halo && plan->tps >= 2) bank_fits = false;
        else if (bank_fits) plan->tps = 1;
        plan->rows_a = run_rows(plan->tps);
        unsigned a_stage = (unsigned)(a_par * plan->cg * plan->rows_a * 16);
        if (bank_fits) {
            plan->b_resident = 1;
            plan->b_stages = 1;
            if (n_tiles > 1) plan->blocked_bank = 2;        // [filter tile][(tap, chunk) plane][row]: a tile's part is one run
            const unsigned fixed = smem + (unsigned)round_up_i((int)bank, 128);
            auto fit = [&](int cg, int* stages) {
                const unsigned st = (unsigned)(a_par * cg * plan->rows_a * 16);
                *stages = 4;
                while (*stages > 2 && fixed + *stages * st > 110 * 1024) --*stages;
                return fixed + *stages * st;
            };
            unsigned total = fit(plan->cg, &plan->a_stages);
            // One thread issues a CTA's MMAs, about 100 cycles apiece, and that bounds a layer of few filters; a
            // second CTA on the SM doubles the rate.  Where only the activation stages keep a second CTA out,
            // they are halved to four channel chunks (measured, 64 -> 48 filters at 56x56, batch 64: 27 -> 20 us).
            if (plan->cg == 8 && total + 1024u > kSmemPerSm / 2) {
                int st4;
                const unsigned t4 = fit(4, &st4);
                if (t4 + 1024u <= kSmemPerSm / 2) {
                    plan->cg = 4;
                    plan->groups = (cchunks + 3) / 4;
                    plan->a_stages = st4;
                    total = t4;
                }
            }
            // A 1x1 layer with a long reduction whose bank leaves the two-CTA form three stages of four chunks is bound by
            // the bytes it has in flight (512 -> 80 at 28x28: 2 x 24 KB per SM, 46.6 us): one CTA with up to eight stages of
            // eight chunks is taken where that at least doubles them (40.3 us; layers that already have four 16 KB stages
            // per CTA lose their second CTA for nothing: 256 -> 48 at 56x56 54.8 -> 62.8 us).
            if (taps == 1 && a_par == 1 && cchunks >= 16) {
                const unsigned st8 = (unsigned)(8 * plan->rows_a * 16);
                int stages = fixed + st8 < kSmemMax ? (int)((kSmemMax - fixed) / st8) : 0;
                if (stages > kMaxStages) stages = kMaxStages;
                const bool two_ctas = total + 1024u <= kSmemPerSm / 2;
                const unsigned now = (two_ctas ? 2u : 1u) * (unsigned)plan->a_stages * (unsigned)(plan->cg * plan->rows_a * 16);
                if (stages >= 4 && (unsigned)stages * st8 >= 2u * now) {
                    plan->cg = 8; plan->groups = (cchunks + 7) / 8;
                    plan->a_stages = stages;
                    total = fixed + (unsigned)stages * st8;
                }
            }
            while (total > kSmemMax && plan->cg > 2) {          // parity images: stages four times the size
                plan->cg -= 2;
                plan->groups = (cchunks + plan->cg - 1) / plan->cg;
                total = fit(plan->cg, &plan->a_stages);
            }
            smem = total;
        } else {
            a_stage = (unsigned)(a_par * plan->cg * plan->rows_a * 16);
            plan->b_resident = 0;
            plan->b_stages = 4;
            const unsigned b_stage = (unsigned)(a.S * plan->cg * n_tile * 16);
            plan->a_stages = plan->tps > 1 ? 2 : 3;
            while (plan->a_stages > 2 && smem + plan->b_stages * b_stage + plan->a_stages * a_stage > kSmemMax) --plan->a_stages;
            while (plan->b_stages > 2 && smem + plan->b_stages * b_stage + plan->a_stages * a_stage > kSmemMax) --plan->b_stages;
            smem += (unsigned)round_up_i((int)(plan->b_stages * b_stage), 128) + plan->a_stages * a_stage;
        }
        }
        want_ctas = 4;
    } else {
        plan->tpk = plan->groups > 1 ? 1 : 8 / cchunks;
        if (plan->tpk > taps) plan->tpk = taps;
        if (plan->tpk < 1) plan->tpk = 1;
        const int planes = plan->groups > 1 ? plan->cg : plan->tpk * cchunks;
        const unsigned stage = (unsigned)(planes * 128 * 16 + planes * n_tile * 16);
        if ((long long)a.N * (a.H + 2) * (a.W + 2) * cchunks >= (1ll << 31)) { snprintf(err, err_len, "input of more than 2^31 vectors"); return 1; }
        const int kblocks = plan->groups > 1 ? taps * plan->groups : (taps + plan->tpk - 1) / plan->tpk;
        smem += (unsigned)kblocks * 64u;                 // the plane-offset table
        // The loader threads wait out one load latency per K block, so co-resident CTAs are what hides it:
        // small stages leave shared memory for up to four CTAs with two or three stages each (the register
        // count below decides how many really fit), large ones get two CTAs with up to six stages.
        plan->a_stages = 3;
        want_ctas = 4;
        while (plan->a_stages > 2 && smem + plan->a_stages * stage > 56 * 1024) --plan->a_stages;
        if (smem + plan->a_stages * stage > 56 * 1024) {
            plan->a_stages = 6;
            want_ctas = 2;
            while (plan->a_stages > 2 && smem + plan->a_stages * stage > kSmemPerSm / 2 - 1024u) --plan->a_stages;   // two CTAs must fit
        }
        plan->b_stages = plan->a_stages;
        if (n_tiles > 1) plan->blocked_bank = 2;        // [filter tile][plane][row]: a K block's filters are one run
        smem += plan->a_stages * stage;
    }
    if (plan->tps < 1) plan->tps = 1;
    plan->tmem_cols = pow2_at_least(2 * plan->tps * n_tile < 32 ? 32 : 2 * plan->tps * n_tile);
    const int tmem_ctas = 512 / plan->tmem_cols;
    if (smem > kSmemMax) { snprintf(err, err_len, "tile does not fit shared memory (%u bytes)", smem); return 1; }
    // co-resident CTAs must not ask for more than the 512 tensor-memory columns of an SM
    const unsigned min_smem = kSmemPerSm / (unsigned)(tmem_ctas + 1) + 1u;
    if (tmem_ctas < 16 && smem < min_smem) smem = min_smem;
    plan->smem_bytes = smem;
    int ctas = (int)(kSmemPerSm / (smem + 1024u));
    if (ctas > tmem_ctas) ctas = tmem_ctas;
    if (ctas > want_ctas) ctas = want_ctas;
    if (ctas < 1) ctas = 1;
    // Wide filter tiles get eight epilogue warps, except in gather mode when there are more tiles than SMs: the
    // eight-warp form needs too many registers for a second CTA on the SM, and a second CTA is what hides the
    // loaders' latency there (measured on ResNet-50, batch 128: every strided layer about 30 % faster with four).
    const int epi = (n_tile >= 64 && (plan->flat || m_tiles * n_tiles <= sms)) ? 8 : 4;
    plan->epi_warps = epi;
    const int mode = !plan->flat ? MODE_GATHER : bank_fits ? MODE_FLAT_RESIDENT : plan->blocked_bank == 1 ? MODE_FLAT_UNIFIED : MODE_FLAT_STREAM;
    const void* fn = kernel_for(mode, epi);
    // a per-device attribute: set it for the device this plan is made on (cheap, so not cached)
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax) != cudaSuccess) {
        snprintf(err, err_len, "cannot raise the dynamic shared memory limit");
        cudaGetLastError();
        return 1;
    }
    cudaFuncAttributes fa;
    cudaError_t oe = cudaFuncGetAttributes(&fa, fn);
    if (oe != cudaSuccess) { snprintf(err, err_len, "cudaFuncGetAttributes: %s", cudaGetErrorString(oe)); cudaGetLastError(); return 1; }
    const int threads = 64 + 32 * epi + extra_threads(mode);
    const int regs_per_warp = round_up_i(fa.numRegs * 32, 256);
    int occ = 65536 / (regs_per_warp * (threads / 32));
    if (occ > 2048 / threads) occ = 2048 / threads;
    if (occ < 1) occ = 1;
    if (ctas > occ) ctas = occ;
    plan->ctas_per_sm = ctas;
    plan->valid = 1;
    return 0;
}

void launch_conv_tc(const ConvPlanTC& plan, const ConvArgs& a, int* d_status, cudaStream_t st, int skip_round, long long wait_cycles) {
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.a = a;
    p.Wp_in = a.W + 2; p.P2_in = (a.H + 2) * (a.W + 2);
    p.Qp = a.Q + 2; p.P2_out = (a.P + 2) * (a.Q + 2);
    p.plane_in = (long long)a.N * p.P2_in * (a.x_plane_mult > 1 || a.x_s2d ? 4 : 1);
    p.plane_in2 = (long long)a.N * p.P2_in * (a.x2_plane_mult > 1 ? 4 : 1);
    p.cchunks2 = a.x2_C_pad / 8;
    p.groups2 = a.x2_C_pad > 0 ? (p.cchunks2 + plan.cg - 1) / plan.cg : 0;
    p.plane_out = (long long)a.N * p.P2_out;
    p.m_total = p.plane_out;
    p.plane_y = p.plane_out;
    if (a.y_split) {
        p.y_split = 1; p.y_Wh2 = a.Q / 2 + 2; p.y_P2h = (a.P / 2 + 2) * p.y_Wh2;
        p.plane_y = 4ll * a.N * p.y_P2h;
    }
    p.a_par = a.x_s2d ? 4 : 1;
    p.par_stride = (long long)a.N * p.P2_in;
    for (int t = 0; t < 9; ++t) {
        // tap (r, s) of the 3x3 / stride-2 window reads input row 2p + r - 1: odd rows one row up for r = 0, even rows
        // for r = 1, odd rows for r = 2; columns likewise.  Parity images in the order 00, 10, 11, 01.
        const int r = t / 3, sx = t % 3;
        const int pa = r == 1 ? 0 : 1, pb = sx == 1 ? 0 : 1;
        const int pp = pa ? (pb ? 2 : 1) : (pb ? 3 : 0);
        p.tap_off[t] = pp * plan.rows_a + plan.halo + (r == 0 ? -(a.W + 2) : 0) + (sx == 0 ? -1 : 0);
    }
    p.taps = a.R * a.S; p.cchunks = a.C_pad / 8; p.cg = plan.cg; p.groups = plan.groups;
    p.halo = plan.halo; p.rows_a = plan.rows_a; p.a_stages = plan.a_stages; p.b_stages = plan.b_stages;
    p.n_tile = plan.n_tile; p.n_tiles = plan.n_tiles; p.tmem_cols = plan.tmem_cols;
    const long long m_tiles = (p.m_total + 127) / 128;
    p.tps = plan.tps > 0 ? plan.tps : 1;
    p.n_producers = plan.a_stages % 4 == 0 ? 4 : plan.a_stages % 3 == 0 ? 3 : plan.a_stages % 2 == 0 ? 2 : 1;
    p.total_tiles = (int)(((m_tiles + p.tps - 1) / p.tps) * plan.n_tiles);
    const int gplanes = plan.groups > 1 ? plan.cg : plan.tpk * p.cchunks;      // gather: planes per stage
    p.a_stage_bytes = plan.flat ? plan.cg * p.a_par * plan.rows_a * 16 : gplanes * 128 * 16;
    p.b_stage_bytes = plan.blocked_bank == 1 ? p.taps * plan.cg * plan.n_tile * 16 : plan.flat ? a.S * plan.cg * plan.n_tile * 16 : gplanes * plan.n_tile * 16;
    p.bank_tile_bytes = (long long)p.taps * p.cchunks * plan.n_tile * 16;
    p.tpk = plan.tpk > 0 ? plan.tpk : 1;
    p.kblocks = plan.groups > 1 ? p.taps * plan.groups : (p.taps + p.tpk - 1) / p.tpk;
    p.b_bank_bytes = p.taps * a.C_pad * plan.n_tile * 2;        // resident filters: one filter tile's part
    p.lut_bytes = plan.flat ? 0 : p.kblocks * 64;
    p.scatter_bytes = a.scatter ? round_up_i((a.out_C_pad + plan.n_tiles + 1) * 4, 16) + 8 * 32 * 33 * 4 : 0;
    p.status = d_status;
    p.skip_round = skip_round; p.wait_cycles = wait_cycles;
    p.div_ntiles = make_fastdiv((uint32_t)plan.n_tiles);
    p.div_p2out = make_fastdiv((uint32_t)p.P2_out);
    p.div_qp = make_fastdiv((uint32_t)p.Qp);
    int grid = sm_count() * plan.ctas_per_sm;
    if (grid > p.total_tiles) grid = p.total_tiles;
    if (plan.b_resident && plan.n_tiles > 1 && grid > plan.n_tiles) grid -= grid % plan.n_tiles;   // a CTA's tiles share a filter tile
    if (grid < 1) grid = 1;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    const int mode = !plan.flat ? MODE_GATHER : plan.b_resident ? MODE_FLAT_RESIDENT : plan.blocked_bank == 1 ? MODE_FLAT_UNIFIED : MODE_FLAT_STREAM;
    cfg.blockDim = dim3((unsigned)(64 + 32 * plan.epi_warps + extra_threads(mode)));
    cfg.dynamicSmemBytes = plan.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    void* args[1] = {(void*)&p};
    cudaLaunchKernelExC(&cfg, kernel_for(mode, plan.epi_warps), args);
}

}  // namespace fp
