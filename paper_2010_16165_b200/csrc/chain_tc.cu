// A run of consecutive stride-1 3x3 convolutions (the convolutions of a stage of basic residual
// blocks) as ONE kernel: every CTA carries a group of G whole images through all layers of the run,
// with the activations in shared memory from the first layer's input to the last layer's output.
// Only the run's input, the first layer's shortcut operand and the run's output touch global memory;
// the filters of each layer are streamed into a double buffer while the previous layer computes.
//
//   Activation layout in shared memory: planar-8 (one 16-byte vector = 8 channels of one position),
//   row pitch W with NO column border, one zero row above every image and one below the last:
//       position f = img*(H+1)*W + hrow*W + w,   hrow = 0 is the zero row, hrow = h + 1 a pixel row.
//   W divides 32, so a warp of the epilogue always covers whole image rows.
//
//   GEMM view of one layer: M = positions (tiles of 128), K = input channels, and the three
//   HORIZONTAL filter taps are stacked along N:   D[p, (s,k)] = sum_{r,c} x[p + (r-1)*W, c] * W'[k,c,r,s]
//   (column of (s,k) = 48*(k/16) + 16*s + k%16: the 48 values one thread needs for 16 channels are adjacent).
//   The vertical taps are three accumulating MMAs whose A operand is the same shared-memory plane
//   read from a start address shifted by (r-1)*W rows (the zero rows are the vertical padding).  The
//   horizontal taps are recombined in the epilogue with two warp shuffles,
//       y[p, k] = D[p-1, (0,k)] + D[p, (1,k)] + D[p+1, (2,k)],
//   where the neighbour terms are dropped in the first / last column of an image row (that is the
//   horizontal padding).  For the narrow layers this path is built for (16..64 channels) one MMA of
//   N = 3*K_pad replaces three of N = K_pad, and the tensor pipe's time per MMA hardly depends on N there.
//
//   Warp roles: warp 0 streams filter blobs (bulk copies), warp 1 owns tensor memory and lane 0
//   issues the MMAs, warps 2-17 are the epilogue: four groups of four warps (one warp per quarter of
//   the 128 accumulator rows).  A group takes every (4/split)-th tile and every split-th channel chunk
//   of it (split = 1, 2 or 4: runs with few tiles per layer spread each tile over more warps).  The
//   same warps load the run's input and store its output.
//   Pipelining: the accumulators form a ring of up to 8 stages in tensor memory, so the MMAs of later
//   tiles run while earlier tiles are in their epilogue (an MMA group completes about a thousand cycles
//   after it is issued).  Layers overlap too: tile t of a layer needs only tiles t-1, t, t+1 of the
//   previous layer (the vertical halo is W <= 32 positions), tracked with one mbarrier per tile, so
//   the next layer's first tiles are issued while the current layer's last tiles are in flight.
//   Every wait is bounded and raises a status word.
#include "fp_internal.h"
#include "tc_common.cuh"

#include <cstdio>
#include <cstring>

namespace fp {

namespace {

using namespace tc;

struct ChainParams {
    ChainArgs a;
    int G, tiles, plane_rows, buf_bytes, wbuf_bytes, tmem_cols, acc_cols, n_groups, stages, split, issuers, ring;
    int img_pos, w_shift, P2, Wp;
    FastDiv div_rows;
    long long plane_in, plane_out, plane_res;
    int rP2, rWp;
    int* status;
};

constexpr int kMaxStages = 8;
constexpr int kMaxTiles = 64;        // per group; a unit takes at most 32 of them (one bit each in a mask)

struct ChainCtrl {
    uint64_t w_full[2], w_empty[2], tmem_full[kMaxStages], tmem_empty[kMaxStages], tile_done[2][kMaxTiles], group_sync;
    uint32_t tmem_base;
    int abort_flag;
    int pad_[4];
};
static_assert(sizeof(ChainCtrl) % 16 == 0, "buffers behind the control block must stay 16-byte aligned");

constexpr int kEpiThreads = 512;
constexpr int kLoadBatch = 2;                      // tiles whose global loads a thread keeps in flight together
constexpr int kIssuers = 4;                        // MMA-issuing warps: warp 1 and the last three
constexpr int kThreads = 64 + kEpiThreads + 32 * (kIssuers - 1);

__device__ __forceinline__ void raise_chain(ChainCtrl* ctrl, int* status, int code) {
    atomicExch(&ctrl->abort_flag, 1);
    atomicExch(status, code);
}

// 8 channels of one position of the first layer's shortcut operand (read from global memory)
__device__ __forceinline__ uint4 load_residual_vec(const ChainParams& p, int chunk, int n, int hrow, int wcol) {
    const uint4* __restrict__ res = reinterpret_cast<const uint4*>(p.a.res);
    if (p.a.res_mode == 1) {
        if (chunk * 8 >= p.a.res_C_pad) return make_uint4(0, 0, 0, 0);
        return __ldg(res + (long long)chunk * p.plane_res + (long long)n * p.rP2 + (long long)hrow * p.rWp + (wcol + 1));
    }
    // subsampled input, channel k of the output takes channel k - pad_lo of the operand
    const long long pos = (long long)n * p.rP2 + (long long)((hrow - 1) * p.a.res_stride + 1) * p.rWp + (wcol * p.a.res_stride + 1);
    const int cs = chunk * 8 - p.a.res_pad_lo;
    if (cs >= 0 && cs + 8 <= p.a.res_C_pad && (cs & 7) == 0) return __ldg(res + (long long)(cs >> 3) * p.plane_res + pos);
    uint4 out = make_uint4(0, 0, 0, 0);
    if (cs + 8 > 0 && cs < p.a.res_C) {
        const __nv_bfloat16* __restrict__ rs = reinterpret_cast<const __nv_bfloat16*>(p.a.res);
        __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(&out);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int c = cs + i;
            if (c >= 0 && c < p.a.res_C) o[i] = rs[((long long)(c >> 3) * p.plane_res + pos) * 8 + (c & 7)];
        }
    }
    return out;
}

// The MMAs of one tile: three vertical taps x KSTEPS K=16 steps, unrolled with every operand address a
// register + constant, because the issuing thread's own instruction latency is what limits narrow layers.
template <int KSTEPS>
__device__ __forceinline__ void issue_tile(bool leader, uint32_t d_tmem, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t b0,
                                           uint32_t b1, uint32_t b2, uint32_t a_ks, uint32_t b_ks, uint32_t idesc) {
    if (leader) {
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) umma_bf16_lo(d_tmem, a0 + ks * a_ks, b0 + ks * b_ks, idesc, ks ? 1u : 0u);
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) umma_bf16_lo(d_tmem, a1 + ks * a_ks, b1 + ks * b_ks, idesc, 1u);
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) umma_bf16_lo(d_tmem, a2 + ks * a_ks, b2 + ks * b_ks, idesc, 1u);
    }
}

__global__ void __launch_bounds__(kThreads, 1) chain_tc_kernel(const __grid_constant__ ChainParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    ChainCtrl* ctrl = reinterpret_cast<ChainCtrl*>(smem_raw);
    const uint32_t ctrl_addr = smem_u32(smem_raw);
    const uint32_t wbuf0 = (ctrl_addr + (uint32_t)sizeof(ChainCtrl) + 127u) & ~127u;
    const uint32_t act0 = wbuf0 + 2u * (uint32_t)p.wbuf_bytes;
    uint8_t* const wbuf_ptr = smem_raw + (wbuf0 - ctrl_addr);
    uint8_t* const act_ptr = smem_raw + (act0 - ctrl_addr);
    volatile int* abort_flag = &ctrl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t w_full0 = ctrl_addr + (uint32_t)offsetof(ChainCtrl, w_full);
    const uint32_t w_empty0 = ctrl_addr + (uint32_t)offsetof(ChainCtrl, w_empty);
    const uint32_t tfull0 = ctrl_addr + (uint32_t)offsetof(ChainCtrl, tmem_full);
    const uint32_t tempty0 = ctrl_addr + (uint32_t)offsetof(ChainCtrl, tmem_empty);
    const uint32_t tdone0 = ctrl_addr + (uint32_t)offsetof(ChainCtrl, tile_done);
    const uint32_t group_sync = ctrl_addr + (uint32_t)offsetof(ChainCtrl, group_sync);
    const int split = p.split, units = 4 / p.split;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(w_full0 + 8 * s, 1);
            mbar_init(w_empty0 + 8 * s, p.issuers + kEpiThreads / 32);    // the MMA issuers + every epilogue warp (bias reads)
        }
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(tfull0 + 8 * s, 1);
            mbar_init(tempty0 + 8 * s, 128 * split);               // every thread that reads the stage
        }
        for (int t = 0; t < p.tiles; ++t) {
            mbar_init(tdone0 + 8 * t, 128 * split);
            mbar_init(tdone0 + 8 * (kMaxTiles + t), 128 * split);
        }
        mbar_init(group_sync, kEpiThreads);
        ctrl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // the layer table in shared memory: an index into the kernel's parameters that is not a compile-time constant costs
    // some 300 cycles per use, and every layer of the run starts with one
    __shared__ ChainLayer s_layers[kChainMaxLayers];
    for (int i = threadIdx.x; i < p.a.n_layers * (int)(sizeof(ChainLayer) / 4); i += blockDim.x)
        reinterpret_cast<int*>(s_layers)[i] = reinterpret_cast<const int*>(p.a.layers)[i];
    // The W guard rows before and after each chunk plane are only read for rows whose results are discarded,
    // but they must hold finite values (the epilogue masks neighbour terms by multiplying with 0): zero them once.
    {
        const int planes = 2 * (p.buf_bytes / (p.plane_rows * 16));
        const int guard = p.a.W;
        for (int i = threadIdx.x; i < planes * 2 * guard; i += blockDim.x) {
            const int pl = i / (2 * guard), r = i - pl * 2 * guard;
            const int row = r < guard ? r : p.plane_rows - 2 * guard + r;
            *reinterpret_cast<uint4*>(act_ptr + ((size_t)pl * p.plane_rows + row) * 16) = make_uint4(0, 0, 0, 0);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(ctrl_addr + (uint32_t)offsetof(ChainCtrl, tmem_base)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_base);

    // Programmatic dependent launch: the next kernel may begin its prologue now.  The filter producer
    // reads only filters (never written by a forward) and starts at once; every other role waits until
    // the previous kernel has completed before it touches activations.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp != 0) asm volatile("griddepcontrol.wait;" ::: "memory");

    const int L = p.a.n_layers;
    const uint32_t plane_bytes = (uint32_t)p.plane_rows * 16u;

    if (warp == 0) {
        // ------------------------------ filter producer ------------------------------
        bool ok = true;
        uint32_t it = 0;
        for (int g = blockIdx.x; g < p.n_groups && ok; g += gridDim.x) {
            for (int l = 0; l < L; ++l, ++it) {
                const uint32_t wb = it & 1, wph = (it >> 1) & 1;
                bool w = true;
                if (lane == 0) w = mbar_wait(w_empty0 + 8 * wb, wph ^ 1, abort_flag);
                w = __shfl_sync(0xffffffffu, w, 0);
                if (!w) { ok = false; break; }
                const int bytes = s_layers[l].blob_bytes;
                const uint32_t fb = w_full0 + 8 * wb;
                if (lane == 0) mbar_expect_tx(fb, (uint32_t)bytes);
                __syncwarp();
                const uint8_t* src = reinterpret_cast<const uint8_t*>(p.a.w) + s_layers[l].blob_off;
                for (int off = lane * 4096; off < bytes; off += 32 * 4096) {
                    const int n = bytes - off < 4096 ? bytes - off : 4096;
                    bulk_copy(wbuf0 + wb * p.wbuf_bytes + off, src + off, (uint32_t)n, fb);
                }
            }
        }
        if (!ok && lane == 0) raise_chain(ctrl, p.status, 11);
    } else if (warp == 1 || warp >= 2 + kEpiThreads / 32) {
        // ------------------------------ MMA issuers -----------------------------------
        // A single thread issues the handful of MMAs of a narrow tile more slowly than the tensor pipe
        // executes them (a bounded mbarrier test alone costs about a hundred cycles), so up to four warps take
        // the tiles round robin; each tile's accumulation chain stays within one thread.  Every issuer owns
        // the accumulator stages iss, iss + issuers, ...: all uses of a stage are then in one thread's program
        // order, which the parity waits on the stage's barriers rely on.
        const int iss = warp == 1 ? 0 : warp - (1 + kEpiThreads / 32);
        // The whole warp runs the loop in step (one lane issues): operand descriptors are then warp-uniform values.
        // (Every lane tests the barriers: one lane testing and a shuffle of the result measured 10-20 % slower per step.)
        if (iss < p.issuers) {
            const bool leader = lane == 0;
            bool ok = true;
            uint32_t it = 0, ring_pos = 0, ring_phase = 0;     // position in this issuer's ring of accumulator stages
            for (int g = blockIdx.x; g < p.n_groups && ok; g += gridDim.x) {
                for (int l = 0; l < L && ok; ++l, ++it) {
                    const ChainLayer& ly = s_layers[l];
                    const uint32_t wb = it & 1, wph = (it >> 1) & 1;
                    // Tile t's input is complete when its barrier has completed `it` + 1 times (once per group load
                    // and per layer).  Completions alternate between two barriers per tile, so that a parity test
                    // cannot mistake "two completions ahead" for "not yet": a tile is never two layers ahead of a
                    // neighbour that still waits for it.
                    const uint32_t td = tdone0 + 8u * (uint32_t)kMaxTiles * (it & 1), tdp = (it >> 1) & 1;
                    if (!mbar_wait(w_full0 + 8 * wb, wph, abort_flag)) { ok = false; break; }
                    const uint32_t N = 3u * (uint32_t)ly.K_pad;
                    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((N >> 3) << 17) | ((128u >> 4) << 24);
                    const int ksteps = ly.cchunks >> 1;
                    const uint32_t src = act0 + (uint32_t)(l & 1) * (uint32_t)p.buf_bytes;
                    // low descriptor words: start address / 16 | (bytes between the two K halves / 16) << 16
                    const uint32_t a_r0 = (src >> 4) | ((uint32_t)p.plane_rows << 16);     // tap row r = 0 starts W rows before the tile
                    const uint32_t a_r1 = a_r0 + (uint32_t)p.a.W, a_r2 = a_r1 + (uint32_t)p.a.W;
                    const uint32_t b_r0 = ((wbuf0 + wb * (uint32_t)p.wbuf_bytes) >> 4) | (N << 16);
                    const uint32_t b_r1 = b_r0 + (uint32_t)ly.cchunks * N, b_r2 = b_r1 + (uint32_t)ly.cchunks * N;
                    const uint32_t a_ks = 2u * (uint32_t)p.plane_rows, b_ks = 2u * N;
                    for (int t = iss; t < p.tiles; t += p.issuers) {
                        const uint32_t stage = (uint32_t)iss + (uint32_t)p.issuers * ring_pos, sph = ring_phase;
                        if (++ring_pos == (uint32_t)p.ring) { ring_pos = 0; ring_phase ^= 1; }
                        if (!mbar_wait(tempty0 + 8 * stage, sph ^ 1, abort_flag)) { ok = false; break; }
                        // the tile reads positions t*128 - W .. t*128 + 127 + W of the previous layer's output
                        if (t > 0 && !mbar_wait(td + 8 * (t - 1), tdp, abort_flag)) { ok = false; break; }
                        if (!mbar_wait(td + 8 * t, tdp, abort_flag)) { ok = false; break; }
                        if (t + 1 < p.tiles && !mbar_wait(td + 8 * (t + 1), tdp, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t d_tmem = tmem_base + stage * (uint32_t)p.acc_cols;
                        const uint32_t to = (uint32_t)(t * 128);
                        switch (ksteps) {
                            case 1: issue_tile<1>(leader, d_tmem, a_r0 + to, a_r1 + to, a_r2 + to, b_r0, b_r1, b_r2, a_ks, b_ks, idesc); break;
                            case 2: issue_tile<2>(leader, d_tmem, a_r0 + to, a_r1 + to, a_r2 + to, b_r0, b_r1, b_r2, a_ks, b_ks, idesc); break;
                            case 3: issue_tile<3>(leader, d_tmem, a_r0 + to, a_r1 + to, a_r2 + to, b_r0, b_r1, b_r2, a_ks, b_ks, idesc); break;
                            case 4: issue_tile<4>(leader, d_tmem, a_r0 + to, a_r1 + to, a_r2 + to, b_r0, b_r1, b_r2, a_ks, b_ks, idesc); break;
                            default: {
                                uint32_t accumulate = 0;
                                for (int r = 0; r < 3; ++r) {
                                    uint32_t a_lo = (r == 0 ? a_r0 : r == 1 ? a_r1 : a_r2) + to, b_lo = r == 0 ? b_r0 : r == 1 ? b_r1 : b_r2;
                                    for (int ks = 0; ks < ksteps; ++ks) {
                                        if (leader) umma_bf16_lo(d_tmem, a_lo, b_lo, idesc, accumulate);
                                        accumulate = 1;
                                        a_lo += a_ks; b_lo += b_ks;
                                    }
                                }
                            }
                        }
                        if (leader) umma_commit(tfull0 + 8 * stage);
                    }
                    if (ok && leader) umma_commit(w_empty0 + 8 * wb);     // the filter buffer is free once this warp's MMAs have read it
                }
            }
            if (!ok && leader) raise_chain(ctrl, p.status, 12);
        }
    } else {
        // ------------------------------ load / epilogue / store ------------------------
        const int etid = threadIdx.x - 64;
        const int grp = (warp - 2) >> 2;
        const int unit = grp / split;                 // takes tiles unit, unit + units, ... (the tiles of MMA issuer `unit`)
        const int part = grp - unit * split;          // takes 16-channel groups part, part + split, ...
        const int quarter = warp & 3;                 // TMEM lanes 32*quarter .. +31
        const int W = p.a.W, H = p.a.H;
        const int wcol = lane & (W - 1);              // W divides 32: the column of this thread's positions never changes
        const float m_left = wcol > 0 ? 1.0f : 0.0f, m_right = wcol < W - 1 ? 1.0f : 0.0f;
        const int tiles = p.tiles;
        const uint32_t ring = (uint32_t)p.ring, acc_cols = (uint32_t)p.acc_cols;
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int f_first = unit * 128 + quarter * 32 + lane;       // this thread's position in its first tile
        const size_t tile_step_bytes = (size_t)units * 128 * 16;
        const uint4* __restrict__ xv = reinterpret_cast<const uint4*>(p.a.x);
        uint4* __restrict__ yv = reinterpret_cast<uint4*>(p.a.y);
        bool ok = true;
        uint32_t it = 0, gs_it = 0, ring_pos = 0, ring_phase = 0;
        uint32_t pixel_mask = 0;       // bit i: this thread's position in the unit's i-th tile is a pixel of an image of the batch
        for (int g = blockIdx.x; g < p.n_groups && ok; g += gridDim.x) {
            if (gs_it) {
                // every MMA and every epilogue of the previous group has finished before its buffers are overwritten
                mbar_arrive(group_sync);
                if (!mbar_wait(group_sync, (gs_it - 1) & 1, abort_flag)) { ok = false; break; }
            }
            ++gs_it;
            // ---- load the group's images (and the first layer's shortcut operand); each thread loads the
            //      positions and 16-channel groups it will later own in the epilogues.  kLoadBatch tiles at a time,
            //      all global loads of a batch issued before the first shared-memory store (latencies overlap).
            //      The input is either a planar-8 tensor or the network input itself (NCHW, fp32 or bf16). ----
            {
                const int in_groups = p.a.layers[0].cchunks >> 1;
                const int out_groups = p.a.layers[0].K_pad >> 4;
                uint8_t* b0 = act_ptr + (size_t)W * 16;
                uint8_t* b1 = b0 + p.buf_bytes;
                pixel_mask = 0;
                int slot = 0;
                for (int tb = unit; tb < tiles; tb += kLoadBatch * units, slot += kLoadBatch) {
                    int fq[kLoadBatch], nq[kLoadBatch], hq[kLoadBatch];
                    bool pq[kLoadBatch];
#pragma unroll
                    for (int q = 0; q < kLoadBatch; ++q) {
                        const int t = tb + q * units;
                        const int f = t * 128 + quarter * 32 + lane;
                        const int row = f >> p.w_shift;
                        const int img = (int)fdiv((uint32_t)row, p.div_rows);
                        const int hrow = row - img * (H + 1);
                        const int n = g * p.G + img;
                        const bool pixel = t < tiles && hrow >= 1 && img < p.G && n < p.a.N;
                        fq[q] = f; nq[q] = n; hq[q] = hrow; pq[q] = pixel;
                        if (t < tiles) pixel_mask |= (pixel ? 1u : 0u) << (slot + q);
                    }
                    for (int cq = part; cq < in_groups; cq += split) {
                        uint4 v[kLoadBatch][2];
#pragma unroll
                        for (int q = 0; q < kLoadBatch; ++q) {
                            v[q][0] = make_uint4(0, 0, 0, 0);
                            v[q][1] = v[q][0];
                            if (!pq[q]) continue;
                            if (p.a.in_mode == 0) {
                                const long long gpos = (long long)nq[q] * p.P2 + (long long)hq[q] * p.Wp + (wcol + 1);
                                v[q][0] = __ldg(xv + (long long)(2 * cq) * p.plane_in + gpos);
                                v[q][1] = __ldg(xv + (long long)(2 * cq + 1) * p.plane_in + gpos);
                            } else {
                                // channels 16*cq .. 16*cq+15 of pixel (h, w) of image n, rounded to bf16
                                const long long e0 = ((long long)nq[q] * p.a.in_C * H + (hq[q] - 1)) * W + wcol;
                                __nv_bfloat16 tmp[16];
#pragma unroll
                                for (int i = 0; i < 16; ++i) {
                                    const int ch = 16 * cq + i;
                                    float val = 0.0f;
                                    if (ch < p.a.in_C) {
                                        const long long e = e0 + (long long)ch * H * W;
                                        val = p.a.in_mode == 1 ? __ldg(reinterpret_cast<const float*>(p.a.x) + e)
                                                               : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.a.x)[e]);
                                    }
                                    tmp[i] = __float2bfloat16_rn(val);
                                }
                                v[q][0] = *reinterpret_cast<const uint4*>(tmp);
                                v[q][1] = *reinterpret_cast<const uint4*>(tmp + 8);
                            }
                        }
#pragma unroll
                        for (int q = 0; q < kLoadBatch; ++q) {
                            if (tb + q * units < tiles) {
                                uint8_t* d = b0 + (size_t)(2 * cq) * plane_bytes + (size_t)fq[q] * 16;
                                *reinterpret_cast<uint4*>(d) = v[q][0];
                                *reinterpret_cast<uint4*>(d + plane_bytes) = v[q][1];
                            }
                        }
                    }
                    if (p.a.res_mode) {
                        for (int cq = part; cq < out_groups; cq += split) {
                            uint4 v[kLoadBatch][2];
#pragma unroll
                            for (int q = 0; q < kLoadBatch; ++q) {
                                v[q][0] = make_uint4(0, 0, 0, 0);
                                v[q][1] = v[q][0];
                                if (pq[q]) {
                                    v[q][0] = load_residual_vec(p, 2 * cq, nq[q], hq[q], wcol);
                                    v[q][1] = load_residual_vec(p, 2 * cq + 1, nq[q], hq[q], wcol);
                                }
                            }
#pragma unroll
                            for (int q = 0; q < kLoadBatch; ++q) {
                                if (tb + q * units < tiles) {
                                    uint8_t* d = b1 + (size_t)(2 * cq) * plane_bytes + (size_t)fq[q] * 16;
                                    *reinterpret_cast<uint4*>(d) = v[q][0];
                                    *reinterpret_cast<uint4*>(d + plane_bytes) = v[q][1];
                                }
                            }
                        }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic stores -> MMA operand reads
                for (int t = unit; t < tiles; t += units) mbar_arrive(tdone0 + 8 * ((it & 1) * kMaxTiles + t));
            }
            // ---- layers ----
            for (int l = 0; l < L && ok; ++l, ++it) {
                const ChainLayer& ly = s_layers[l];
                const uint32_t wb = it & 1, wph = (it >> 1) & 1;
                const bool last = l == L - 1;
                if (!mbar_wait(w_full0 + 8 * wb, wph, abort_flag)) { ok = false; break; }     // the bias is in the blob
                const int K_pad = ly.K_pad, kgroups = K_pad >> 4;
                const bool res = ly.res != 0, relu = ly.relu != 0;
                const float4* bias4 = reinterpret_cast<const float4*>(wbuf_ptr + (size_t)wb * p.wbuf_bytes +
                                                                      (size_t)(3 * ly.cchunks * 3 * K_pad) * 16);
                // this thread's vector in chunk plane 0 of the destination buffer, for its first tile
                uint8_t* dst = act_ptr + (size_t)((l + 1) & 1) * p.buf_bytes + (size_t)(W + f_first) * 16;
                const uint32_t td_next = tdone0 + 8u * (uint32_t)kMaxTiles * ((it + 1) & 1);
                uint32_t pm = pixel_mask;
                for (int t = unit; t < tiles; t += units, pm >>= 1, dst += tile_step_bytes) {
                    const bool pixel = pm & 1u;
                    // the accumulator stage: this unit's tiles are the tiles of issuer `unit`, in the same order
                    const uint32_t stage = (uint32_t)unit + (uint32_t)units * ring_pos, sph = ring_phase;
                    if (++ring_pos == ring) { ring_pos = 0; ring_phase ^= 1; }
                    bool w = mbar_wait(tfull0 + 8 * stage, sph, abort_flag);
                    w = __all_sync(0xffffffffu, w);
                    if (!w) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t taddr = tmem_lane + stage * acc_cols;
                    for (int kq = part; kq < kgroups; kq += split) {
                        uint32_t vlc[32], vr[16];
                        tmem_ld32(taddr + (uint32_t)(kq * 48), vlc);
                        tmem_ld16(taddr + (uint32_t)(kq * 48 + 32), vr);
                        uint4* slot0 = reinterpret_cast<uint4*>(dst + (size_t)(2 * kq) * plane_bytes);
                        uint4* slot1 = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(slot0) + plane_bytes);
                        uint4 rv[2];
                        rv[0] = make_uint4(0, 0, 0, 0);
                        rv[1] = rv[0];
                        if (res) { rv[0] = *slot0; rv[1] = *slot1; }
                        float bb[16];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float4 b = bias4[kq * 4 + i];
                            bb[4 * i] = b.x; bb[4 * i + 1] = b.y; bb[4 * i + 2] = b.z; bb[4 * i + 3] = b.w;
                        }
                        tmem_ld_wait();
                        // of the 48 columns: [0,16) tap s = 0, wanted by the position on the right; [16,32) the centre
                        // tap; [32,48) tap s = 2, wanted by the position on the left.  The masks drop the neighbour's
                        // term in the first / last column of an image row (all values involved are finite).
                        float o[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const float lf = __shfl_up_sync(0xffffffffu, __uint_as_float(vlc[i]), 1);
                            const float rt = __shfl_down_sync(0xffffffffu, __uint_as_float(vr[i]), 1);
                            o[i] = fmaf(rt, m_right, fmaf(lf, m_left, __uint_as_float(vlc[16 + i]) + bb[i]));
                        }
                        if (res) {
                            const uint32_t* rw = reinterpret_cast<const uint32_t*>(rv);
#pragma unroll
                            for (int i = 0; i < 8; ++i) {                // bf16 pair -> two floats
                                o[2 * i] += __uint_as_float(rw[i] << 16);
                                o[2 * i + 1] += __uint_as_float(rw[i] & 0xffff0000u);
                            }
                        }
                        uint4 ov[2];
                        ov[0] = make_uint4(0, 0, 0, 0);
                        ov[1] = ov[0];
                        if (pixel) {
                            uint32_t* ow = reinterpret_cast<uint32_t*>(ov);
                            if (relu) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) ow[i] = pack_bf16x2_relu(o[2 * i], o[2 * i + 1]);
                            } else {
#pragma unroll
                                for (int i = 0; i < 8; ++i) ow[i] = pack_bf16x2(o[2 * i], o[2 * i + 1]);
                            }
                        }
                        if (!last) { *slot0 = ov[0]; *slot1 = ov[1]; }
                        else if (pixel) {
                            const int f = t * 128 + quarter * 32 + lane;
                            const int row = f >> p.w_shift;
                            const int img = (int)fdiv((uint32_t)row, p.div_rows);
                            const int hrow = row - img * (H + 1);
                            const long long gpos = (long long)(g * p.G + img) * p.P2 + (long long)hrow * p.Wp + (wcol + 1);
                            yv[(long long)(2 * kq) * p.plane_out + gpos] = ov[0];
                            yv[(long long)(2 * kq + 1) * p.plane_out + gpos] = ov[1];
                        }
                    }
                    tc_fence_before();
                    mbar_arrive(tempty0 + 8 * stage);
                    if (!last) {
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        mbar_arrive(td_next + 8 * t);
                    }
                }
                if (!ok) break;
                __syncwarp();
                if (lane == 0) mbar_arrive(w_empty0 + 8 * wb);       // this warp no longer reads the layer's bias
            }
            if (!ok) break;
            // ---- zero border of the group's output images in global memory ----
            {
                const int out_chunks = s_layers[L - 1].K_pad >> 3;
                const int border = 2 * p.Wp + 2 * H;
                const int total = p.G * border * out_chunks;
                for (int i = etid; i < total; i += kEpiThreads) {
                    const int c = i / (p.G * border);
                    const int r2 = i - c * (p.G * border);
                    const int img = r2 / border, b = r2 - img * border;
                    const int n = g * p.G + img;
                    if (n >= p.a.N) continue;
                    int row, col;
                    if (b < p.Wp) { row = 0; col = b; }
                    else if (b < 2 * p.Wp) { row = H + 1; col = b - p.Wp; }
                    else { const int s2 = b - 2 * p.Wp; row = 1 + (s2 >> 1); col = (s2 & 1) ? W + 1 : 0; }
                    yv[(long long)c * p.plane_out + (long long)n * p.P2 + (long long)row * p.Wp + col] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        if (!ok && lane == 0) raise_chain(ctrl, p.status, 13);
    }

    // ---- teardown: everyone arrives here, also after a wait that ran out ----
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(1000);     // let copies in flight land before shared memory is released
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
constexpr unsigned kSmemMin = 120u * 1024u;        // more than half an SM: one CTA per SM, so tensor memory is never contended

int round_up_i(int v, int m) { return (v + m - 1) / m * m; }

}  // namespace

int chain_layer_blob_bytes(int cchunks, int K_pad) { return 3 * cchunks * 3 * K_pad * 16 + K_pad * 4; }

bool chain_layer_supported(int H, int W, int K_pad, int C_pad) {
    if (!(W == 8 || W == 16 || W == 32)) return false;
    if (H < 1 || H > 64) return false;
    if (K_pad % 16 || C_pad % 16 || K_pad > 80 || C_pad > 128) return false;
    return true;
}

int plan_chain_tc(const ChainArgs& a, ChainPlan* plan, char* err, size_t err_len) {
    memset(plan, 0, sizeof(*plan));
    if (a.n_layers < 1 || a.n_layers > kChainMaxLayers) { snprintf(err, err_len, "bad layer count"); return 1; }
    int max_chunks = 0, max_blob = 0, max_N = 0;
    for (int l = 0; l < a.n_layers; ++l) {
        const ChainLayer& ly = a.layers[l];
        if (!chain_layer_supported(a.H, a.W, ly.K_pad, ly.cchunks * 8)) { snprintf(err, err_len, "layer %d not supported", l); return 1; }
        max_chunks = ly.cchunks > max_chunks ? ly.cchunks : max_chunks;
        max_chunks = (ly.K_pad >> 3) > max_chunks ? (ly.K_pad >> 3) : max_chunks;
        max_blob = ly.blob_bytes > max_blob ? ly.blob_bytes : max_blob;
        max_N = 3 * ly.K_pad > max_N ? 3 * ly.K_pad : max_N;
    }
    const int wbuf = round_up_i(max_blob, 128);
    const int img_pos = (a.H + 1) * a.W;
    int best_G = 0; double best_cost = 0;
    for (int G = 1; G <= 64 && G <= a.N; ++G) {
        const int tiles = (G * img_pos + a.W + 127) / 128;
        const int rows = 2 * a.W + tiles * 128;
        if (rows > 16383 || tiles > kMaxTiles) break;
        const unsigned smem = (unsigned)sizeof(ChainCtrl) + 128u + 2u * wbuf + 2u * (unsigned)max_chunks * rows * 16u;
        if (smem > kSmemMax) break;
        const int groups = (a.N + G - 1) / G;
        const int sms = sm_count();
        const int rounds = (groups + sms - 1) / sms;
        const double cost = rounds * (tiles + 1.5);
        if (best_G == 0 || cost <= best_cost) { best_G = G; best_cost = cost; }
    }
    if (best_G == 0) { snprintf(err, err_len, "one image does not fit shared memory"); return 1; }
    plan->G = best_G;
    plan->tiles = (best_G * img_pos + a.W + 127) / 128;
    plan->plane_rows = 2 * a.W + plan->tiles * 128;
    plan->buf_bytes = max_chunks * plan->plane_rows * 16;
    plan->wbuf_bytes = wbuf;
    plan->acc_cols = max_N;
    plan->tmem_cols = 512;                              // one CTA per SM: all of tensor memory is the accumulator ring
    plan->stages = 512 / max_N < kMaxStages ? 512 / max_N : kMaxStages;
    plan->split = plan->tiles <= 4 ? 4 : plan->tiles <= 8 ? 2 : 1;
    // One MMA issuer per epilogue unit (4 / split of them): the tiles of an issuer, i.e. all uses of its
    // accumulator stages, then go to one unit in the issuer's own order.  Not more units than stages or tiles.
    while (4 / plan->split > plan->stages || 4 / plan->split > plan->tiles) plan->split *= 2;
    plan->issuers = 4 / plan->split;
    unsigned smem = (unsigned)sizeof(ChainCtrl) + 128u + 2u * wbuf + 2u * (unsigned)plan->buf_bytes;
    if (smem < kSmemMin) smem = kSmemMin;
    plan->smem_bytes = smem;
    // a per-device attribute: set it for the device this plan is made on (cheap, so not cached)
    if (cudaFuncSetAttribute(chain_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax) != cudaSuccess) {
        snprintf(err, err_len, "cannot raise the dynamic shared memory limit");
        cudaGetLastError();
        return 1;
    }
    plan->valid = 1;
    return 0;
}

void launch_chain_tc(const ChainPlan& plan, const ChainArgs& a, int* d_status, cudaStream_t st) {
    ChainParams p;
    memset(&p, 0, sizeof(p));
    p.a = a;
    // the group size was planned for the largest batch; a smaller batch just has fewer groups
    p.G = plan.G; p.tiles = plan.tiles; p.plane_rows = plan.plane_rows; p.buf_bytes = plan.buf_bytes;
    p.wbuf_bytes = plan.wbuf_bytes; p.tmem_cols = plan.tmem_cols; p.acc_cols = plan.acc_cols;
    p.stages = plan.stages; p.split = plan.split; p.issuers = plan.issuers;
    p.ring = plan.stages / plan.issuers;
    p.n_groups = (a.N + plan.G - 1) / plan.G;
    p.img_pos = (a.H + 1) * a.W;
    p.w_shift = a.W == 8 ? 3 : a.W == 16 ? 4 : 5;
    p.Wp = a.W + 2; p.P2 = (a.H + 2) * (a.W + 2);
    p.div_rows = make_fastdiv((uint32_t)(a.H + 1));
    p.plane_in = (long long)a.N * p.P2;
    p.plane_out = p.plane_in;
    p.rWp = a.res_W + 2; p.rP2 = (a.res_H + 2) * (a.res_W + 2);
    p.plane_res = (long long)a.N * p.rP2;
    p.status = d_status;
    const int sms = sm_count();
    int grid = p.n_groups < sms ? p.n_groups : sms;
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
    cudaLaunchKernelExC(&cfg, (const void*)chain_tc_kernel, args);
}

}  // namespace fp
