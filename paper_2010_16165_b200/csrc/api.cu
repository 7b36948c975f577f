// C-ABI entry points and the host-side fused-graph builder.
//
// fp_fuse walks the node list, recognises conv-BN-(ReLU) chains and residual blocks, and
// emits a list of fused operators: convolutions whose epilogue carries the folded BN shift,
// the shortcut operand and the ReLU, max pools, and one head (average pool + FC).  Where a
// block is flagged aggressive the paper's rewriting (Sec. IV-B) is applied instead: identity
// filters are stacked under conv1 along K, the shortcut's filters beside conv2 along C, and
// no residual operand remains.  fp_prune selects masks on the device and re-derives every
// packed filter bank, activation shape and launch plan from them.
#include "../../include/fupruner.h"
#include "fp_internal.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <string>
#include <vector>

namespace {

thread_local std::string g_err;

fp_status fail(fp_status st, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    g_err = buf;
    return st;
}

#define CK(call)                                                                                        \
    do {                                                                                                \
        cudaError_t e_ = (call);                                                                        \
        if (e_ != cudaSuccess)                                                                          \
            return fail(e_ == cudaErrorMemoryAllocation ? FP_ERR_NOMEM : FP_ERR_CUDA, "%s: %s (%s:%d)", \
                        #call, cudaGetErrorString(e_), __FILE__, __LINE__);                             \
    } while (0)

#define TRY(expr)                          \
    do {                                   \
        fp_status s_ = (expr);             \
        if (s_ != FP_OK) return s_;        \
    } while (0)

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

struct Tensor {
    int C_full = 0;            // channels before pruning
    int C = 0;                 // channels stored (kept)
    int C_pad = 0;             // storage width, multiple of 16
    int H = 0, W = 0;
    std::vector<int> keep;     // stored channel j holds original channel keep[j]
    void* d = nullptr;
    size_t bytes = 0;
    int producer = -1;         // index into ops, -1 = network input
    int split = 0;             // stored parity-split (fp::ConvArgs): only stride-2 convolutions read it
};

struct FConv {
    int conv_index = -1;       // number among the description's FP_CONV nodes
    int src = -1, out = -1;    // tensor ids
    int K = 0, C = 0, R = 0, S = 0, stride = 1, pad = 0;   // fused, unpruned geometry
    int n_orig = 0;            // filter count of the original operator (Algorithm 1's m)
    int role = 0;              // 0 plain, 1 aggressive conv1 (identity filters stacked), 2 aggressive conv2
    int relu = 0;
    int res_mode = 0, res_tid = -1, res_pad_lo = 0, res_stride = 1;
    float* d_w32 = nullptr;    // fused fp32 filters, K x C x R x S
    float* d_b32 = nullptr;    // fused bias, K
    std::vector<uint8_t> mask;
    std::vector<int32_t> rank;
    // derived by replan()
    int compact = 0;           // 1: pruned filters are physically removed from the output tensor
    int scatter = 0;           // 1: only kept filters are computed, scattered into a full-width output (residual stream)
    int n_tile_forced = 0;     // scatter: filters per CTA tile the packed bank was laid out for
    int32_t* d_out_map = nullptr;   // scatter: output channel -> packed filter row (-1 = no filter kept)
    int32_t* d_chunk0 = nullptr;    // scatter: first output chunk of every filter tile, and the end
    int n_mult = 1;            // 4: a 1x1 layer over a parity-split tensor runs on its 4 N half-size images
    int proj = -1;             // >= 0: the projection shortcut (index into convs) that this layer computes itself
    int proj_kind = 0;         // 1: filters stacked along the channels (1x1 layer); 2: extra centre-tap K groups (streamed 3x3 layer)
    int absorbed = 0;          // 1: this projection runs inside the layer that adds its result; its operator launches nothing
    void* d_wp_plain = nullptr;     // the packed bank before any re-blocking ([tap][chunk][K_pad][8])
    int K_kept = 0, K_rows = 0, K_pad = 0, C_kept = 0, C_pad = 0;
    void* d_wp = nullptr;      // packed filters in the compute type, K_pad x R x S x C_pad
    float* d_bp = nullptr;
    int32_t* d_row = nullptr;  // packed filter row -> fused filter (-1 = zero row)
    int32_t* d_chan = nullptr; // packed input channel -> fused input channel (-1 = zero channel)
    fp::ConvArgs args;
    fp::ConvPlanTC tc;
};

struct Pool { int src, out, R, stride, pad; };

// Consecutive stride-1 3x3 convolutions that one kernel runs with the activations in shared memory.
struct Chain {
    int first_op = -1, last_op = -1;
    std::vector<int> convs;    // indices into the handle's convs, in execution order
    fp::ChainArgs args;
    fp::ChainPlan plan;
    uint8_t* d_blob = nullptr;
};

struct Op { int kind; int idx; };
constexpr int kHostPieces = 8;     // fp_forward_host copies the input in up to this many pieces   // kind: 0 conv, 1 pool, 2 head, 3 input conversion

struct GraphKey {
    int batch; int first; const void* in; const void* out; cudaStream_t st;      // first: first operator of the captured range
    bool operator<(const GraphKey& o) const {
        if (batch != o.batch) return batch < o.batch;
        if (first != o.first) return first < o.first;
        if (in != o.in) return in < o.in;
        if (out != o.out) return out < o.out;
        return st < o.st;
    }
};

}  // namespace

struct fp_handle_s {
    std::vector<fp_node> nodes;
    int in_C = 0, in_H = 0, in_W = 0, in_dtype = 0, compute = 0, use_graph = 0, keep_outputs = 0;
    float eps = 1e-5f;
    int max_batch = 0;
    int n_desc_convs = 0;
    std::vector<int> conv_to_fused;        // description conv number -> index into convs, -1 absorbed
    std::vector<FConv> convs;
    std::vector<Pool> pools;
    std::vector<Tensor> tensors;           // tensor 0 = network input (after layout conversion)
    std::vector<Op> ops;
    std::vector<Chain> chains;             // re-derived by fp_prune
    std::vector<int> op_chain;             // operator -> chain number, -1 = launched on its own
    int input_fused = 0;                   // 1: the first fused run reads the network input directly (no layout conversion launch)
    // head
    int head_src = -1, n_classes = 0, fc_C = 0;
    const float* d_fcw = nullptr;          // classes x fc_C (copy of the description's FC weights)
    const float* d_fcb = nullptr;
    float* d_fcw_packed = nullptr;         // classes x C_pad, scaled by 1/(H*W)
    float* d_pool = nullptr;               // max_batch x C_pad channel sums (between the two head kernels)
    // buffers
    std::vector<void*> act_buffers;        // activation storage (re-planned by fp_prune)
    std::vector<void*> pack_buffers;       // packed filters / biases / index arrays
    std::vector<void*> fixed_buffers;      // fused fp32 filters etc. (live until fp_destroy)
    void* d_in_stage = nullptr;            // device staging for fp_forward_host
    float* d_logits_stage = nullptr;
    void* (*alloc)(size_t, void*) = nullptr;      // the caller's device allocator (fp_fuse_with_allocator), or cudaMalloc / cudaFree
    void (*dealloc)(void*, void*) = nullptr;
    void* alloc_user = nullptr;
    int* d_status = nullptr;
    cudaStream_t copy_stream = nullptr;    // fp_forward_host: input pieces are copied here while earlier pieces are converted
    int stage_used = 0;                    // the staging buffer has been read by a kernel queued behind copy_events[kHostPieces]
    cudaEvent_t copy_events[kHostPieces + 1] = {};
    double* d_scores = nullptr; int32_t* d_rank = nullptr; uint8_t* d_mask = nullptr;
    std::map<GraphKey, cudaGraphExec_t> graphs;
    const void* last_input = nullptr; int last_batch = 0;
    int soft_epochs = 0;                   // passes of fp_soft_prune_epoch since fp_fuse
    // dynamic pruning over all banks at once: bank table, filter -> bank map, scores / ranks / masks of all filters
    fp::SoftBank* d_soft_banks = nullptr; int32_t* d_soft_map = nullptr;
    double* d_soft_scores = nullptr; int32_t* d_soft_rank = nullptr; uint8_t* d_soft_mask = nullptr;
    int soft_total = 0;
    int stem_packed = 0;                   // network input stored in the packed form of a 7x7/2 first convolution
    int stem_fused = 0;                    // operators 0-2 (input conversion, 7x7/2 convolution, 3x3/2 max pooling) run as one kernel
    fp::StemPoolArgs stem_args;
    fp::StemPoolPlan stem_plan;
    int scatter_policy = 0;                // fp_model_desc::scatter
    int planned = 0;                       // 1: buffers, packed banks and launch plans match the masks (set by replan)
    int act_is_bf16() const { return compute != FP_COMPUTE_FP32; }
    size_t act_elem() const { return act_is_bf16() ? 2 : 4; }
    size_t in_elem() const { return in_dtype == FP_DTYPE_BF16 ? 2 : 4; }
};

namespace {

void drop_graphs(fp_handle h) {
    for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second);
    h->graphs.clear();
}

// Device memory comes from the caller's allocator where fp_fuse_with_allocator was given one, else from cudaMalloc.
void dev_free(fp_handle h, void* p) {
    if (!p) return;
    if (h->dealloc) h->dealloc(p, h->alloc_user);
    else cudaFree(p);
}

void free_list(fp_handle h, std::vector<void*>& v) {
    for (void* p : v) dev_free(h, p);
    v.clear();
}

fp_status dev_alloc_raw(fp_handle h, void** out, size_t bytes) {
    void* p = nullptr;
    if (bytes == 0) bytes = 16;
    if (h->alloc) {
        p = h->alloc(bytes, h->alloc_user);
        if (!p) return fail(FP_ERR_NOMEM, "the caller's allocator returned NULL for %zu bytes", bytes);
        if ((uintptr_t)p % 256) {
            h->dealloc(p, h->alloc_user);
            return fail(FP_ERR_ARG, "the caller's allocator returned memory that is not 256-byte aligned");
        }
    } else {
        cudaError_t e = cudaMalloc(&p, bytes);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(FP_ERR_NOMEM, "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(e));
        }
    }
    *out = p;
    return FP_OK;
}

fp_status dev_alloc(fp_handle h, std::vector<void*>& owner, void** out, size_t bytes) {
    void* p = nullptr;
    TRY(dev_alloc_raw(h, &p, bytes));
    owner.push_back(p);
    *out = p;
    return FP_OK;
}

// ---------------------------------------------------------------------------------------
// description -> fused operators
// ---------------------------------------------------------------------------------------

struct Builder {
    fp_handle h;
    const float* d_weights; const float* d_bn;   // the handle's own copies
    size_t n_weights, n_bn;
    std::vector<std::vector<int>> cons;
    std::vector<int> node_tensor;     // node id -> tensor id (or -1)
    std::vector<int> conv_number;     // node id -> description conv number
    cudaStream_t st = 0;

    int tensor_of(int node) const { return node < 0 ? 0 : node_tensor[node]; }

    fp_status check_conv_node(int id) {
        const fp_node& n = h->nodes[id];
        if (n.K <= 0 || n.C <= 0 || n.R <= 0 || n.S <= 0 || n.stride <= 0 || n.pad < 0)
            return fail(FP_ERR_DESC, "node %d: bad convolution geometry", id);
        if (n.w_off < 0 || (size_t)n.w_off + (size_t)n.K * n.C * n.R * n.S > n_weights)
            return fail(FP_ERR_DESC, "node %d: weights outside the weight array", id);
        if (cons[id].size() != 1 || h->nodes[cons[id][0]].op != FP_BN)
            return fail(FP_ERR_DESC, "node %d: a convolution must feed exactly one batch norm", id);
        const fp_node& b = h->nodes[cons[id][0]];
        if (b.K != n.K)
            return fail(FP_ERR_SHAPE, "node %d: batch norm has %d channels, convolution %d", cons[id][0], b.K, n.K);
        if (b.bn_off < 0 || (size_t)b.bn_off + 4 * (size_t)b.K > n_bn)
            return fail(FP_ERR_DESC, "node %d: BN parameters outside the BN array", cons[id][0]);
        return FP_OK;
    }

    // New fused conv from description node `conv_id`: a zeroed (K+extra_K) x (C+extra_C) bank with the
    // node's BN-folded filters in rows [0,K), columns [0,C) and the folded shift in bias [0,K).
    fp_status emit_conv(int conv_id, int src_tid, int relu, int extra_C, int* out_index) {
        TRY(check_conv_node(conv_id));
        const fp_node& n = h->nodes[conv_id];
        const Tensor src = h->tensors[src_tid];
        if (src.C_full != n.C + extra_C)
            return fail(FP_ERR_SHAPE, "node %d: convolution expects %d input channels, producer has %d", conv_id,
                        n.C + extra_C, src.C_full);
        if (src.H + 2 * n.pad < n.R || src.W + 2 * n.pad < n.S)
            return fail(FP_ERR_SHAPE, "node %d: window larger than the padded input", conv_id);
        FConv f;
        f.conv_index = conv_number[conv_id];
        f.src = src_tid;
        f.K = n.K; f.C = n.C + extra_C; f.R = n.R; f.S = n.S; f.stride = n.stride; f.pad = n.pad;
        f.n_orig = n.K; f.relu = relu;
        const size_t cnt = (size_t)f.K * f.C * f.R * f.S;
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&f.d_w32, cnt * sizeof(float)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&f.d_b32, (size_t)f.K * sizeof(float)));
        CK(cudaMemsetAsync(f.d_w32, 0, cnt * sizeof(float), st));
        CK(cudaMemsetAsync(f.d_b32, 0, (size_t)f.K * sizeof(float), st));
        const fp_node& b = h->nodes[cons[conv_id][0]];
        fp::launch_fold_weights(d_weights + n.w_off, d_bn + b.bn_off, n.K, n.C, n.R, n.S, h->eps, f.d_w32, f.C, f.R,
                                f.S, 0, 0, 0, 0, st);
        fp::launch_fold_bias(d_bn + b.bn_off, n.K, h->eps, f.d_b32, 0, 0, st);
        Tensor t;
        t.C_full = f.K;
        t.H = (src.H + 2 * f.pad - f.R) / f.stride + 1;
        t.W = (src.W + 2 * f.pad - f.S) / f.stride + 1;
        t.producer = (int)h->ops.size();
        h->tensors.push_back(t);
        f.out = (int)h->tensors.size() - 1;
        h->convs.push_back(f);
        h->conv_to_fused[f.conv_index] = (int)h->convs.size() - 1;
        h->ops.push_back({0, (int)h->convs.size() - 1});
        *out_index = (int)h->convs.size() - 1;
        return FP_OK;
    }

    // K_id identity filters (the auxiliary convolution xconv-C) under the filters of fused convolution `fi`:
    // its output becomes [conv(x) ; x].  The operator is then a fused one: n = K + K_id filters, m = K originally.
    fp_status stack_identity_filters(int fi, int K_id) {
        const FConv f0 = h->convs[fi];
        const int K1 = f0.K, C = f0.C, RS = f0.R * f0.S;
        float *nw, *nb;
        const size_t cnt = (size_t)(K1 + K_id) * C * RS;
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&nw, cnt * sizeof(float)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&nb, (size_t)(K1 + K_id) * sizeof(float)));
        CK(cudaMemsetAsync(nw, 0, cnt * sizeof(float), st));
        CK(cudaMemsetAsync(nb, 0, (size_t)(K1 + K_id) * sizeof(float), st));
        CK(cudaMemcpyAsync(nw, f0.d_w32, (size_t)K1 * C * RS * sizeof(float), cudaMemcpyDeviceToDevice, st));
        CK(cudaMemcpyAsync(nb, f0.d_b32, (size_t)K1 * sizeof(float), cudaMemcpyDeviceToDevice, st));
        fp::launch_identity_filters(nw, C, f0.R, f0.S, K1, 0, K_id, C, 0, st);
        FConv& f = h->convs[fi];
        f.d_w32 = nw; f.d_b32 = nb; f.K = K1 + K_id; f.role = 1;
        h->tensors[f.out].C_full = K1 + K_id;
        return FP_OK;
    }

    bool is_relu_output(int tid) const {
        const int px = h->tensors[tid].producer;
        if (px < 0) return false;
        if (h->ops[px].kind == 0) return h->convs[h->ops[px].idx].relu != 0;
        if (h->ops[px].kind == 1) return is_relu_output(h->pools[h->ops[px].idx].src);   // max of non-negatives
        return false;
    }

    // Aggressive fusion of a three-convolution (bottleneck) block, which the paper does not describe (it stops at
    // two-convolution blocks): the block input is carried through all three convolutions.  conv1'' = [W1' ; I]
    // (1x1), conv2'' = diag(W2', I at the centre tap) - the pass-through is subsampled with conv2's stride -,
    // conv3'' = [W3' | S] with S the identity or the projection's folded 1x1 filters; no add remains.
    fp_status fuse_bottleneck(int id, int relu_id, int conv3_id, int fbi, int x_tid, int h_tid, int mode, int proj_id) {
        const fp_node& c3 = h->nodes[conv3_id];
        const FConv fb0 = h->convs[fbi];                                   // the 3x3 convolution
        const int pa = h->tensors[fb0.src].producer;
        if (pa < 0 || h->ops[pa].kind != 0)
            return fail(FP_ERR_UNSUPPORTED, "node %d: aggressive fusion needs a 1x1 - 3x3 - 1x1 block", id);
        const int fai = h->ops[pa].idx;
        const FConv fa0 = h->convs[fai];                                   // the first 1x1 convolution
        if (fa0.src != x_tid || !fa0.relu || !fb0.relu || fa0.res_mode || fb0.res_mode || fa0.role || fb0.role ||
            fa0.R != 1 || fa0.S != 1 || fa0.stride != 1 || fa0.pad != 0 || fb0.R != 3 || fb0.S != 3 || fb0.pad != 1 ||
            c3.stride != 1 || c3.pad != 0 || mode == 1)
            return fail(FP_ERR_UNSUPPORTED, "node %d: aggressive fusion needs a 1x1 - 3x3 - 1x1 block with an identity or projection shortcut", id);
        if (!is_relu_output(x_tid))
            return fail(FP_ERR_UNSUPPORTED, "node %d: aggressive fusion needs a block input that is a ReLU output", id);
        const int C = fa0.C, Kw = fa0.K;
        if (fb0.K != Kw || fb0.C != Kw || c3.C != Kw) return fail(FP_ERR_SHAPE, "node %d: bottleneck widths differ", id);
        {   // conv1'': C identity filters under the 1x1 convolution
            float *nw, *nb;
            TRY(dev_alloc(h, h->fixed_buffers, (void**)&nw, (size_t)(Kw + C) * C * sizeof(float)));
            TRY(dev_alloc(h, h->fixed_buffers, (void**)&nb, (size_t)(Kw + C) * sizeof(float)));
            CK(cudaMemsetAsync(nw, 0, (size_t)(Kw + C) * C * sizeof(float), st));
            CK(cudaMemsetAsync(nb, 0, (size_t)(Kw + C) * sizeof(float), st));
            CK(cudaMemcpyAsync(nw, fa0.d_w32, (size_t)Kw * C * sizeof(float), cudaMemcpyDeviceToDevice, st));
            CK(cudaMemcpyAsync(nb, fa0.d_b32, (size_t)Kw * sizeof(float), cudaMemcpyDeviceToDevice, st));
            fp::launch_identity_filters(nw, C, 1, 1, Kw, 0, C, C, 0, st);
            FConv& fa = h->convs[fai];
            fa.d_w32 = nw; fa.d_b32 = nb; fa.K = Kw + C; fa.role = 1;
            h->tensors[fa.out].C_full = Kw + C;
        }
        {   // conv2'': block diagonal, the pass-through on the centre tap
            const int n = Kw + C;
            float *nw, *nb;
            TRY(dev_alloc(h, h->fixed_buffers, (void**)&nw, (size_t)n * n * 9 * sizeof(float)));
            TRY(dev_alloc(h, h->fixed_buffers, (void**)&nb, (size_t)n * sizeof(float)));
            CK(cudaMemsetAsync(nw, 0, (size_t)n * n * 9 * sizeof(float), st));
            CK(cudaMemsetAsync(nb, 0, (size_t)n * sizeof(float), st));
            CK(cudaMemcpy2DAsync(nw, (size_t)n * 9 * sizeof(float), fb0.d_w32, (size_t)Kw * 9 * sizeof(float),
                                 (size_t)Kw * 9 * sizeof(float), Kw, cudaMemcpyDeviceToDevice, st));
            CK(cudaMemcpyAsync(nb, fb0.d_b32, (size_t)Kw * sizeof(float), cudaMemcpyDeviceToDevice, st));
            fp::launch_identity_filters(nw, n, 3, 3, Kw, Kw, C, C, 0, st);
            FConv& fb = h->convs[fbi];
            fb.d_w32 = nw; fb.d_b32 = nb; fb.K = n; fb.C = n; fb.role = 1;
            h->tensors[fb.out].C_full = n;
        }
        int ci;
        TRY(emit_conv(conv3_id, h_tid, 1, C, &ci));            // K3 x (Kw + C), conv3 folded into columns [0,Kw)
        FConv& f = h->convs[ci];
        f.role = 2;
        if (mode == 0) {
            if (f.K != C) return fail(FP_ERR_SHAPE, "node %d: identity shortcut needs as many filters as block inputs", id);
            fp::launch_identity_filters(f.d_w32, f.C, 1, 1, 0, Kw, f.K, C, 0, st);
        } else {
            TRY(check_conv_node(proj_id));
            const fp_node& pr = h->nodes[proj_id];
            if (pr.R != 1 || pr.S != 1 || pr.pad != 0 || pr.stride != fb0.stride || pr.C != C || pr.K != f.K)
                return fail(FP_ERR_UNSUPPORTED, "node %d: projection shortcut must be 1x1 with the 3x3 convolution's stride", id);
            const fp_node& pb = h->nodes[cons[proj_id][0]];
            fp::launch_fold_weights(d_weights + pr.w_off, d_bn + pb.bn_off, pr.K, pr.C, 1, 1, h->eps, f.d_w32, f.C, 1, 1,
                                    0, Kw, 0, 0, st);
            fp::launch_fold_bias(d_bn + pb.bn_off, pr.K, h->eps, f.d_b32, 0, 1, st);
            h->conv_to_fused[conv_number[proj_id]] = -1;
        }
        node_tensor[relu_id] = h->convs[ci].out;
        return FP_OK;
    }

    fp_status handle_add(int id) {
        const fp_node& n = h->nodes[id];
        if (cons[id].size() != 1 || h->nodes[cons[id][0]].op != FP_RELU)
            return fail(FP_ERR_DESC, "node %d: an add must feed exactly one ReLU", id);
        const int relu_id = cons[id][0];
        if (n.in0 < 0 || h->nodes[n.in0].op != FP_BN || h->nodes[n.in0].in0 < 0 ||
            h->nodes[h->nodes[n.in0].in0].op != FP_CONV)
            return fail(FP_ERR_DESC, "node %d: first add operand must be the batch norm of a convolution", id);
        const int conv2_id = h->nodes[n.in0].in0;
        const fp_node& c2 = h->nodes[conv2_id];
        int mode;   // 0 identity tensor, 1 subsample + zero-channel pad, 2 projection
        int x_node, proj_id = -1;
        const fp_node* sc = n.in1 >= 0 ? &h->nodes[n.in1] : nullptr;
        if (n.in1 < 0 || node_tensor[n.in1] >= 0) { mode = 0; x_node = n.in1; }
        else if (sc->op == FP_SHORTCUT_A) { mode = 1; x_node = sc->in0; }
        else if (sc->op == FP_BN && sc->in0 >= 0 && h->nodes[sc->in0].op == FP_CONV) {
            mode = 2; proj_id = sc->in0; x_node = h->nodes[proj_id].in0;
        } else return fail(FP_ERR_DESC, "node %d: unsupported shortcut operand", id);
        const int x_tid = tensor_of(x_node);
        const int h_tid = tensor_of(c2.in0);
        if (x_tid < 0 || h_tid < 0) return fail(FP_ERR_DESC, "node %d: operands are not materialised tensors", id);
        int ci;
        if (!n.aggressive) {
            int res_mode = 1, res_tid = x_tid, pad_lo = 0, rstride = 1;
            if (mode == 1) { res_mode = 2; pad_lo = sc->pad_lo; rstride = sc->stride; }
            if (mode == 2) {
                int pi;
                TRY(emit_conv(proj_id, x_tid, 0, 0, &pi));
                res_tid = h->convs[pi].out;
            }
            TRY(emit_conv(conv2_id, h_tid, 1, 0, &ci));
            FConv& f = h->convs[ci];
            const Tensor& o = h->tensors[f.out];
            const Tensor& r = h->tensors[res_tid];
            if (res_mode == 1) {
                if (r.C_full != f.K || r.H != o.H || r.W != o.W)
                    return fail(FP_ERR_SHAPE, "node %d: add operands differ in shape", id);
            } else {
                if (rstride <= 0 || (r.H + rstride - 1) / rstride != o.H || (r.W + rstride - 1) / rstride != o.W ||
                    pad_lo < 0 || pad_lo + r.C_full > f.K || sc->K != f.K || sc->C != r.C_full)
                    return fail(FP_ERR_SHAPE, "node %d: shortcut does not match the main branch", id);
            }
            f.res_mode = res_mode; f.res_tid = res_tid; f.res_pad_lo = pad_lo; f.res_stride = rstride;
        } else {
            // ---- aggressive fusion (Sec. IV-B): conv1'' = [W1' ; I], conv2'' = [W2' | S_w], no add ----
            const int p1 = h->tensors[h_tid].producer;
            if (p1 < 0 || h->ops[p1].kind != 0)
                return fail(FP_ERR_UNSUPPORTED, "node %d: aggressive fusion needs a two-convolution block", id);
            const int f1i = h->ops[p1].idx;
            const FConv f1c = h->convs[f1i];
            if (c2.R == 1 && c2.S == 1) {
                TRY(fuse_bottleneck(id, relu_id, conv2_id, f1i, x_tid, h_tid, mode, proj_id));
                return FP_OK;
            }
            if (f1c.src != x_tid || !f1c.relu || f1c.res_mode != 0 || f1c.role != 0 || f1c.R != 3 || f1c.S != 3 ||
                f1c.pad != 1 || c2.R != 3 || c2.S != 3 || c2.stride != 1 || c2.pad != 1)
                return fail(FP_ERR_UNSUPPORTED, "node %d: aggressive fusion supports 3x3 two-convolution blocks only", id);
            // the pass-through channels go through conv1's ReLU: the block input must be non-negative
            if (!is_relu_output(x_tid))
                return fail(FP_ERR_UNSUPPORTED, "node %d: aggressive fusion needs a block input that is a ReLU output", id);
            if (mode == 1 && sc->stride != f1c.stride)
                return fail(FP_ERR_SHAPE, "node %d: shortcut stride differs from conv1", id);
            if (mode == 2) {
                TRY(check_conv_node(proj_id));
                const fp_node& pr = h->nodes[proj_id];
                if (pr.R != 1 || pr.S != 1 || pr.pad != 0 || pr.stride != f1c.stride || pr.C != f1c.C)
                    return fail(FP_ERR_UNSUPPORTED, "node %d: projection shortcut must be 1x1 with conv1's stride", id);
            }
            const int C = f1c.C, K1 = f1c.K;
            {   // widen conv1: C extra identity filters (the auxiliary convolution), zero shift for them
                float *nw, *nb;
                const size_t cnt = (size_t)(K1 + C) * C * 9;
                TRY(dev_alloc(h, h->fixed_buffers, (void**)&nw, cnt * sizeof(float)));
                TRY(dev_alloc(h, h->fixed_buffers, (void**)&nb, (size_t)(K1 + C) * sizeof(float)));
                CK(cudaMemsetAsync(nw, 0, cnt * sizeof(float), st));
                CK(cudaMemsetAsync(nb, 0, (size_t)(K1 + C) * sizeof(float), st));
                CK(cudaMemcpyAsync(nw, f1c.d_w32, (size_t)K1 * C * 9 * sizeof(float), cudaMemcpyDeviceToDevice, st));
                CK(cudaMemcpyAsync(nb, f1c.d_b32, (size_t)K1 * sizeof(float), cudaMemcpyDeviceToDevice, st));
                fp::launch_identity_filters(nw, C, 3, 3, K1, 0, C, C, 0, st);
                FConv& f1 = h->convs[f1i];
                f1.d_w32 = nw; f1.d_b32 = nb; f1.K = K1 + C; f1.role = 1;
                h->tensors[f1.out].C_full = K1 + C;
            }
            TRY(emit_conv(conv2_id, h_tid, 1, C, &ci));     // K2 x (K1 + C), conv2 folded into columns [0,K1)
            FConv& f = h->convs[ci];
            f.role = 2;
            if (mode == 0) {
                if (f.K != C) return fail(FP_ERR_SHAPE, "node %d: identity shortcut needs K2 == C", id);
                fp::launch_identity_filters(f.d_w32, f.C, 3, 3, 0, K1, f.K, C, 0, st);
            } else if (mode == 1) {
                if (sc->pad_lo < 0 || sc->pad_lo + C > f.K || sc->K != f.K || sc->C != C)
                    return fail(FP_ERR_SHAPE, "node %d: shortcut does not match the main branch", id);
                fp::launch_identity_filters(f.d_w32, f.C, 3, 3, 0, K1, f.K, C, sc->pad_lo, st);
            } else {
                const fp_node& pr = h->nodes[proj_id];
                if (pr.K != f.K) return fail(FP_ERR_SHAPE, "node %d: projection has %d filters, conv2 %d", id, pr.K, f.K);
                const fp_node& pb = h->nodes[cons[proj_id][0]];
                // the 1x1 projection padded with zeros to 3x3 (centre tap), folded with its own BN
                fp::launch_fold_weights(d_weights + pr.w_off, d_bn + pb.bn_off, pr.K, pr.C, 1, 1, h->eps, f.d_w32, f.C, 3, 3,
                                        0, K1, 1, 1, st);
                fp::launch_fold_bias(d_bn + pb.bn_off, pr.K, h->eps, f.d_b32, 0, 1, st);
                h->conv_to_fused[conv_number[proj_id]] = -1;
            }
            const Tensor& o = h->tensors[f.out];
            const Tensor& xin = h->tensors[x_tid];
            if ((xin.H + f1c.stride - 1) / f1c.stride != o.H || (xin.W + f1c.stride - 1) / f1c.stride != o.W)
                return fail(FP_ERR_SHAPE, "node %d: shortcut spatial size mismatch", id);
        }
        node_tensor[relu_id] = h->convs[ci].out;
        return FP_OK;
    }

    fp_status run() {
        const int nn = (int)h->nodes.size();
        cons.assign(nn, {});
        node_tensor.assign(nn, -1);
        conv_number.assign(nn, -1);
        int nc = 0;
        for (int i = 0; i < nn; ++i) {
            const fp_node& n = h->nodes[i];
            if (n.op < FP_CONV || n.op > FP_CONCAT) return fail(FP_ERR_DESC, "node %d: unknown op %d", i, n.op);
            if (n.in0 < -1 || n.in0 >= i) return fail(FP_ERR_DESC, "node %d: in0 must name an earlier node", i);
            const bool two = n.op == FP_ADD || n.op == FP_CONCAT;
            if (two && (n.in1 < -1 || n.in1 >= i)) return fail(FP_ERR_DESC, "node %d: in1 must name an earlier node", i);
            if (n.in0 >= 0) cons[n.in0].push_back(i);
            if (two && n.in1 >= 0) cons[n.in1].push_back(i);
            if (n.op == FP_CONV) conv_number[i] = nc++;
        }
        h->n_desc_convs = nc;
        h->conv_to_fused.assign(nc, -1);
        Tensor in;
        in.C_full = h->in_C; in.H = h->in_H; in.W = h->in_W; in.producer = -1;
        h->tensors.push_back(in);
        h->ops.push_back({3, 0});
        for (int i = 0; i < nn; ++i) {
            const fp_node& n = h->nodes[i];
            switch (n.op) {
                case FP_CONV: {
                    TRY(check_conv_node(i));
                    const int bn_id = cons[i][0];
                    const std::vector<int>& nxt = cons[bn_id];
                    if (nxt.size() == 1 && h->nodes[nxt[0]].op == FP_ADD) break;   // emitted with its add
                    const int src = tensor_of(n.in0);
                    if (src < 0) return fail(FP_ERR_DESC, "node %d: input is not a materialised tensor", i);
                    int ci;
                    // The concatenation structure (Sec. IV-B.1): y = concat(conv(x), x) becomes one convolution with
                    // the identity filters of xconv-C stacked under its own: y = new_conv(x, [W' ; I]).
                    const bool has_relu = nxt.size() == 1 && h->nodes[nxt[0]].op == FP_RELU;
                    const int last = has_relu ? nxt[0] : bn_id;
                    if (cons[last].size() == 1 && h->nodes[cons[last][0]].op == FP_CONCAT &&
                        h->nodes[cons[last][0]].in0 == last && h->nodes[cons[last][0]].in1 == n.in0) {
                        const int cat = cons[last][0];
                        if (n.stride != 1 || n.R != n.S || n.R % 2 == 0 || n.pad != n.R / 2)
                            return fail(FP_ERR_UNSUPPORTED, "node %d: the concatenation structure needs a stride-1 'same' convolution", i);
                        if (has_relu && !is_relu_output(src))
                            return fail(FP_ERR_UNSUPPORTED, "node %d: fusing concat(relu(conv(x)), x) needs x to be a ReLU output", i);
                        if (h->nodes[cat].K != n.K + n.C) return fail(FP_ERR_SHAPE, "node %d: concatenation has %d channels, operands %d", cat, h->nodes[cat].K, n.K + n.C);
                        TRY(emit_conv(i, src, has_relu ? 1 : 0, 0, &ci));
                        TRY(stack_identity_filters(ci, n.C));
                        node_tensor[cat] = h->convs[ci].out;
                        break;
                    }
                    if (has_relu) {
                        TRY(emit_conv(i, src, 1, 0, &ci));
                        node_tensor[nxt[0]] = h->convs[ci].out;
                    } else {
                        TRY(emit_conv(i, src, 0, 0, &ci));
                        node_tensor[bn_id] = h->convs[ci].out;
                    }
                    break;
                }
                case FP_ADD: TRY(handle_add(i)); break;
                case FP_MAXPOOL: {
                    const int src = tensor_of(n.in0);
                    if (src < 0) return fail(FP_ERR_DESC, "node %d: input is not a materialised tensor", i);
                    const Tensor s = h->tensors[src];
                    if (n.R <= 0 || n.stride <= 0 || n.pad < 0 || n.pad >= n.R || s.H + 2 * n.pad < n.R || s.W + 2 * n.pad < n.R)
                        return fail(FP_ERR_DESC, "node %d: bad pooling geometry", i);
                    Tensor t;
                    t.C_full = s.C_full;
                    t.H = (s.H + 2 * n.pad - n.R) / n.stride + 1;
                    t.W = (s.W + 2 * n.pad - n.R) / n.stride + 1;
                    t.producer = (int)h->ops.size();
                    h->tensors.push_back(t);
                    h->pools.push_back({src, (int)h->tensors.size() - 1, n.R, n.stride, n.pad});
                    h->ops.push_back({1, (int)h->pools.size() - 1});
                    node_tensor[i] = (int)h->tensors.size() - 1;
                    break;
                }
                case FP_GAVGPOOL: {
                    const int src = tensor_of(n.in0);
                    if (src < 0) return fail(FP_ERR_DESC, "node %d: input is not a materialised tensor", i);
                    if (cons[i].size() != 1 || h->nodes[cons[i][0]].op != FP_FC)
                        return fail(FP_ERR_DESC, "node %d: global average pool must feed the FC layer", i);
                    const fp_node& f = h->nodes[cons[i][0]];
                    if (f.C != h->tensors[src].C_full || f.K <= 0)
                        return fail(FP_ERR_SHAPE, "node %d: FC expects %d inputs, producer has %d", cons[i][0], f.C, h->tensors[src].C_full);
                    if (f.w_off < 0 || (size_t)f.w_off + (size_t)f.K * f.C > n_weights ||
                        (f.b_off >= 0 && (size_t)f.b_off + f.K > n_weights))
                        return fail(FP_ERR_DESC, "node %d: FC weights outside the weight array", cons[i][0]);
                    if (h->head_src >= 0) return fail(FP_ERR_DESC, "node %d: more than one head", i);
                    h->head_src = src; h->n_classes = f.K; h->fc_C = f.C;
                    h->d_fcw = d_weights + f.w_off;
                    h->d_fcb = f.b_off >= 0 ? d_weights + f.b_off : nullptr;
                    h->ops.push_back({2, 0});
                    break;
                }
                default: break;   // BN, ReLU, shortcut, FC are consumed by the patterns above
            }
        }
        if (h->head_src < 0) return fail(FP_ERR_DESC, "description has no global-average-pool + FC head");
        for (const Tensor& t : h->tensors)
            if (t.W > fp::kMaxWidth) return fail(FP_ERR_UNSUPPORTED, "images wider than %d pixels are not supported", fp::kMaxWidth);
        if (h->ops.back().kind != 2) return fail(FP_ERR_DESC, "the head must be the last operator");
        return FP_OK;
    }
};

// ---------------------------------------------------------------------------------------
// masks -> shapes, packed filters, activation memory, launch plans
// ---------------------------------------------------------------------------------------

struct Use { int op; int how; };   // how: 0 main input, 1 residual operand

std::vector<std::vector<Use>> tensor_uses(fp_handle h) {
    std::vector<std::vector<Use>> u(h->tensors.size());
    for (int i = 0; i < (int)h->ops.size(); ++i) {
        const Op& op = h->ops[i];
        if (op.kind == 0) {
            const FConv& f = h->convs[op.idx];
            u[f.src].push_back({i, 0});
            if (f.res_mode) u[f.res_tid].push_back({i, 1});
        } else if (op.kind == 1) {
            u[h->pools[op.idx].src].push_back({i, 0});
        } else if (op.kind == 2) {
            u[h->head_src].push_back({i, 0});
        }
    }
    return u;
}

// Channels of a tensor can be physically dropped iff every reader is a convolution's main input
// (or a pool whose own result is compactable).  Residual streams keep their full width.
bool compactable(fp_handle h, const std::vector<std::vector<Use>>& uses, int tid) {
    if (uses[tid].empty()) return false;
    for (const Use& u : uses[tid]) {
        if (u.how == 1) return false;
        const Op& op = h->ops[u.op];
        if (op.kind == 0) continue;
        if (op.kind == 1) { if (!compactable(h, uses, h->pools[op.idx].out)) return false; continue; }
        return false;
    }
    return true;
}

fp_status upload_i32(fp_handle h, const std::vector<int32_t>& v, int32_t** out) {
    TRY(dev_alloc(h, h->pack_buffers, (void**)out, v.size() * sizeof(int32_t)));
    CK(cudaMemcpy(*out, v.data(), v.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    return FP_OK;
}

bool chain_candidate(fp_handle h, const FConv& f) {
    if (h->compute != FP_COMPUTE_BF16_TC || h->keep_outputs || f.scatter) return false;
    if (f.R != 3 || f.S != 3 || f.stride != 1 || f.pad != 1) return false;
    if ((h->stem_packed || h->stem_fused) && f.src == 0) return false;
    if (h->tensors[f.src].split || h->tensors[f.out].split) return false;
    const Tensor& s = h->tensors[f.src];
    return fp::chain_layer_supported(s.H, s.W, f.K_pad, f.C_pad);
}

// Finds runs of consecutive operators that are stride-1 3x3 convolutions where each reads the previous
// one's output, a shortcut operand (other than the first layer's) is the tensor two layers back, and no
// tensor inside the run is read from outside it; packs their filters for the fused kernel.
fp_status find_chains(fp_handle h, const std::vector<std::vector<Use>>& uses) {
    h->chains.clear();
    h->op_chain.assign(h->ops.size(), -1);
    const int n_ops = (int)h->ops.size();
    int i = 0;
    while (i < n_ops) {
        if (h->ops[i].kind != 0 || !chain_candidate(h, h->convs[h->ops[i].idx])) { ++i; continue; }
        // longest candidate run starting at operator i
        int len = 1;
        while (i + len < n_ops && len < fp::kChainMaxLayers && h->ops[i + len].kind == 0) {
            const FConv& f = h->convs[h->ops[i + len].idx];
            const FConv& prev = h->convs[h->ops[i + len - 1].idx];
            if (!chain_candidate(h, f) || f.src != prev.out) break;
            if (f.res_mode != 0 && !(f.res_mode == 1 && f.res_tid == prev.src)) break;
            ++len;
        }
        // shorten until every tensor inside the run is read only inside it, and the run fits the kernel
        fp::ChainArgs a;
        fp::ChainPlan plan;
        for (; len >= 2; --len) {
            bool ok = true;
            for (int j = 0; j + 1 < len && ok; ++j) {
                const int tid = h->convs[h->ops[i + j].idx].out;
                for (const Use& u : uses[tid]) {
                    const bool main_next = u.how == 0 && u.op == i + j + 1;
                    const bool res_after = u.how == 1 && u.op == i + j + 2 && j + 2 < len;
                    if (!main_next && !res_after) { ok = false; break; }
                }
            }
            if (!ok) continue;
            memset(&a, 0, sizeof(a));
            const FConv& f0 = h->convs[h->ops[i].idx];
            const Tensor& s0 = h->tensors[f0.src];
            a.N = h->max_batch; a.H = s0.H; a.W = s0.W; a.n_layers = len;
            a.res_mode = f0.res_mode;
            if (f0.res_mode) {
                const Tensor& r = h->tensors[f0.res_tid];
                a.res_H = r.H; a.res_W = r.W; a.res_C_pad = r.C_pad; a.res_C = r.C;
                a.res_pad_lo = f0.res_pad_lo; a.res_stride = f0.res_stride;
            }
            int off = 0;
            for (int j = 0; j < len; ++j) {
                const FConv& f = h->convs[h->ops[i + j].idx];
                fp::ChainLayer& ly = a.layers[j];
                ly.cchunks = f.C_pad / 8; ly.K_pad = f.K_pad; ly.relu = f.relu;
                ly.res = j == 0 ? (f.res_mode != 0) : (f.res_mode == 1);
                ly.blob_off = off;
                ly.blob_bytes = fp::chain_layer_blob_bytes(ly.cchunks, ly.K_pad);
                off += (ly.blob_bytes + 127) / 128 * 128;
            }
            char msg[256];
            if (fp::plan_chain_tc(a, &plan, msg, sizeof(msg)) != 0) continue;
            Chain ch;
            ch.first_op = i; ch.last_op = i + len - 1; ch.args = a; ch.plan = plan;
            for (int j = 0; j < len; ++j) ch.convs.push_back(h->ops[i + j].idx);
            TRY(dev_alloc(h, h->pack_buffers, (void**)&ch.d_blob, (size_t)off));
            for (int j = 0; j < len; ++j) {
                const FConv& f = h->convs[ch.convs[j]];
                const fp::ChainLayer& ly = a.layers[j];
                fp::launch_repack_chain(f.d_w32, f.C, f.d_row, f.K_pad, f.d_chan, f.C_pad,
                                        (__nv_bfloat16*)(ch.d_blob + ly.blob_off), 0);
                fp::launch_pack_bias(f.d_b32, f.d_row, f.K_pad,
                                     (float*)(ch.d_blob + ly.blob_off + (size_t)9 * f.C_pad * f.K_pad * 2), 0);
            }
            CK(cudaGetLastError());
            for (int j = 0; j < len; ++j) h->op_chain[i + j] = (int)h->chains.size();
            h->chains.push_back(ch);
            break;
        }
        i += len >= 2 ? len : 1;
    }
    // A run whose first layer is the only reader of the network input converts the layout while it loads.
    h->input_fused = 0;
    for (Chain& ch : h->chains) {
        const FConv& f0 = h->convs[ch.convs.front()];
        if (f0.src == 0 && uses[0].size() == 1 && !h->stem_packed) {
            ch.args.in_mode = h->in_dtype == FP_DTYPE_BF16 ? 2 : 1;
            ch.args.in_C = h->in_C;
            h->input_fused = 1;
        }
    }
    return FP_OK;
}

// How a convolution reads a parity-split input tensor: 0 it cannot, 'A' 3x3 / stride 2 / pad 1 (nine taps over the four
// parity images), 'B' 1x1 / stride 2 (the parity-00 image), 'C' 1x1 / stride 1 without shortcut (position by position:
// its output is then split the same way).
char split_reader(const FConv& f) {
    if (f.R == 3 && f.S == 3 && f.stride == 2 && f.pad == 1) return 'A';
    if (f.R == 1 && f.S == 1 && f.stride == 2 && f.pad == 0) return 'B';
    if (f.R == 1 && f.S == 1 && f.stride == 1 && f.pad == 0 && f.res_mode == 0) return 'C';
    return 0;
}

// Which tensors are stored parity-split (tensor-core path): tensors written by a convolution of their own kernel, with
// even height and width, that only stride-2 convolutions read - directly, or through 1x1 layers whose output is split
// in turn (the first 1x1 of a strided bottleneck block).  A stride-2 convolution over such a tensor is a stride-1
// convolution over contiguous runs (bulk copies) instead of a gather.
void decide_splits(fp_handle h, const std::vector<std::vector<Use>>& uses) {
    const int nt = (int)h->tensors.size();
    for (Tensor& t : h->tensors) t.split = 0;
    if (h->compute != FP_COMPUTE_BF16_TC) return;
    std::vector<int> cand(nt, 0);
    for (int t = 1; t < nt; ++t) {
        const Tensor& T = h->tensors[t];
        if (T.producer < 0 || h->ops[T.producer].kind != 0 || T.H % 2 || T.W % 2 || T.H < 2 || T.W < 2 || uses[t].empty()) continue;
        const FConv& pf = h->convs[h->ops[T.producer].idx];
        if (pf.src == 0 && (pf.R == 7 || h->stem_packed)) continue;                    // the first convolution has forms of its own
        cand[t] = 1;
    }
    for (bool changed = true; changed;) {
        changed = false;
        for (int t = 1; t < nt; ++t) {
            if (!cand[t]) continue;
            bool ok = true;
            for (const Use& u : uses[t]) {
                if (u.how != 0 || h->ops[u.op].kind != 0) { ok = false; break; }
                const FConv& f = h->convs[h->ops[u.op].idx];
                const char kind = split_reader(f);
                if (!kind || (kind == 'C' && !cand[f.out])) { ok = false; break; }
            }
            if (!ok) { cand[t] = 0; changed = true; }
        }
    }
    for (int t = 1; t < nt; ++t) h->tensors[t].split = cand[t];
}

// Geometry of the launch of fused convolution f (no pointers, no channel counts of the output).
void conv_geometry(fp_handle h, const FConv& f, fp::ConvArgs* a) {
    const Tensor& src = h->tensors[f.src];
    const Tensor& out = h->tensors[f.out];
    a->N = h->max_batch; a->H = src.H; a->W = src.W; a->C_pad = src.C_pad; a->P = out.H; a->Q = out.W;
    a->R = f.R; a->S = f.S; a->stride = f.stride; a->pad = f.pad; a->relu = f.relu;
    a->y_split = 0; a->x_plane_mult = 0; a->x_s2d = 0;
    if (h->stem_packed && f.src == 0) {      // 3x1 stride-1 convolution over the packed input, at the output resolution
        a->H = out.H; a->W = out.W; a->C_pad = 80; a->R = 3; a->S = 1; a->stride = 1; a->pad = 1;
    }
    if (src.split) {
        const char kind = split_reader(f);
        a->H = src.H / 2; a->W = src.W / 2; a->stride = 1;
        if (kind == 'A') { a->x_s2d = 1; }
        else if (kind == 'B') { a->x_plane_mult = 4; }
        else { a->N = 4 * h->max_batch; a->P = out.H / 2; a->Q = out.W / 2; }        // 'C': 4 N half-size images in, the same out
        if (kind != 'C' && out.split) a->y_split = 1;
    } else if (out.split) {
        a->y_split = 1;
    }
}

// Rebuilds everything that depends on the masks.  The old buffers are released first, so while this runs - and
// after it failed half-way (out of memory, a layer left without filters) - the handle has no plan: `planned` stays
// 0 and every call that would launch kernels refuses until a later fp_prune succeeds.
fp_status replan(fp_handle h) {
    h->planned = 0;
    drop_graphs(h);
    CK(cudaDeviceSynchronize());
    free_list(h, h->act_buffers);
    free_list(h, h->pack_buffers);
    const auto uses = tensor_uses(h);
    const int bf16 = h->act_is_bf16();
    cudaStream_t st = 0;

    // --- shapes in execution order ---
    {
        Tensor& t = h->tensors[0];
        t.C = t.C_full; t.C_pad = round_up(t.C, 16);
        t.keep.resize(t.C);
        for (int c = 0; c < t.C; ++c) t.keep[c] = c;
    }
    // A 7x7 / stride-2 / pad-3 first convolution on <= 3 channels runs as a 3x1 convolution over a packed
    // copy of the input (tensor-core path only; the validation paths keep the plain form).
    h->stem_packed = 0;
    for (const FConv& f : h->convs)
        if (f.src == 0 && h->compute == FP_COMPUTE_BF16_TC && uses[0].size() == 1 && f.R == 7 && f.S == 7 &&
            f.stride == 2 && f.pad == 3 && f.C <= 3 && h->in_H % 2 == 0 && h->in_W % 2 == 0)
            h->stem_packed = 1;
    decide_splits(h, uses);
    for (FConv& f : h->convs) {
        f.n_mult = (h->tensors[f.src].split && split_reader(f) == 'C') ? 4 : 1;
        f.proj = -1; f.proj_kind = 0; f.absorbed = 0;
    }
    // ... and, where a 3x3 / stride-2 max pooling is the only reader of that convolution and the input is bf16, input
    // conversion, convolution and pooling run as one kernel (decided below, once the filter count is known).
    h->stem_fused = 0;
    bool stem_candidate = false;
    if (h->stem_packed && !h->keep_outputs && h->in_dtype == FP_DTYPE_BF16 && h->ops.size() >= 3 && h->ops[1].kind == 0 &&
        h->ops[2].kind == 1) {
        const FConv& f = h->convs[h->ops[1].idx];
        const Pool& pl = h->pools[h->ops[2].idx];
        stem_candidate = f.src == 0 && f.relu && f.res_mode == 0 && pl.src == f.out && uses[f.out].size() == 1 &&
                         pl.R == 3 && pl.stride == 2 && pl.pad == 1 && h->in_H % 4 == 0 && h->in_W % 8 == 0;
    }
    for (const Op& op : h->ops) {
        if (op.kind == 0) {
            FConv& f = h->convs[op.idx];
            const Tensor& src = h->tensors[f.src];
            Tensor& out = h->tensors[f.out];
            std::vector<int> kept;
            for (int k = 0; k < f.K; ++k) if (f.mask[k]) kept.push_back(k);
            if (kept.empty()) return fail(FP_ERR_EMPTY_LAYER, "convolution %d keeps no filter", f.conv_index);
            f.K_kept = (int)kept.size();
            f.compact = (f.res_mode == 0 && compactable(h, uses, f.out)) ? 1 : 0;
            f.C_kept = src.C; f.C_pad = src.C_pad;
            // A convolution that writes a residual stream (its output is added to, or read as, a shortcut) cannot drop
            // output channels: other layers write them too.  On the tensor-core path it still computes only its kept
            // filters and scatters them into the full-width tensor in the epilogue; layers that can join a fused run of
            // layers, and the validation paths, keep pruned filters as zero rows instead.
            f.scatter = 0; f.n_tile_forced = 0; f.d_out_map = nullptr; f.d_chunk0 = nullptr;
            if (!f.compact && h->compute == FP_COMPUTE_BF16_TC && round_up(f.K_kept, 16) < round_up(f.K, 16)) {
                const bool runs_fused = !h->keep_outputs && f.R == 3 && f.S == 3 && f.stride == 1 && f.pad == 1 &&
                                        !(h->stem_packed && f.src == 0) &&
                                        fp::chain_layer_supported(src.H, src.W, round_up(f.K, 16), src.C_pad);
                // It has to pay: an MMA over n filters costs the tensor pipe about max(n/2, 32 + n/4) cycles (the second
                // term is the operand fetch), so 64 -> 48 or 128 -> 96 columns save a tenth while the scattering epilogue
                // costs more than that on layers with a short reduction; it is used where the tensor-pipe cost of the
                // kept filters is at most 0.8 of the full width's and the reduction is at least 1024 long.
                fp::ConvArgs ga;
                memset(&ga, 0, sizeof(ga));
                conv_geometry(h, f, &ga);
                auto pipe_cost = [&](int K_pad) {
                    int nt = 0, nts = 0;
                    fp::conv_tc_filter_tile(ga, K_pad, &nt, &nts);
                    return nts * std::max(nt / 2, 32 + nt / 4);
                };
                // And the layer has to fill the GPU more than twice over: with fewer tiles than that, fewer columns only
                // mean fewer busy SMs, not a shorter kernel (measured, ResNet-18 at batch 64, 512 -> 359 filters at 7x7:
                // 41 position tiles; 28 us with zero rows on 84 CTAs, 41 us scattered on 63).
                int nt_s = 0, nts_s = 0;
                fp::conv_tc_filter_tile(ga, round_up(f.K_kept, 16), &nt_s, &nts_s);
                const long long m_tiles = ((long long)ga.N * (ga.P + 2) * (ga.Q + 2) + 127) / 128;
                const bool pays = 5 * pipe_cost(round_up(f.K_kept, 16)) <= 4 * pipe_cost(round_up(f.K, 16)) &&
                                  ga.R * ga.S * ga.C_pad >= 1024 && m_tiles * nts_s >= 2 * fp::sm_count();
                if (!runs_fused && h->scatter_policy >= 0 && (pays || h->scatter_policy > 0)) f.scatter = 1;
            }
            std::vector<int32_t> row_src, chan_src(f.C_pad, -1);
            if (f.scatter) {
                // Filter tiles must own whole output chunks (8 channels = one 16-byte vector per position): fill each tile
                // with consecutive chunks while their kept filters fit, and pad its rows with zero filters.
                fp::ConvArgs ga;
                memset(&ga, 0, sizeof(ga));
                conv_geometry(h, f, &ga);
                const int out_C_pad = round_up(f.K, 16), n_chunks = out_C_pad / 8;
                int n_tile = 0, n_tiles = 0;
                fp::conv_tc_filter_tile(ga, round_up(f.K_kept, 16), &n_tile, &n_tiles);
                std::vector<int> cnt(n_chunks, 0);
                for (int k : kept) ++cnt[k / 8];
                std::vector<int32_t> chunk0;
                for (;;) {
                    chunk0.assign(1, 0);
                    int cur = 0;
                    for (int q = 0; q < n_chunks; ++q) {
                        if (cur + cnt[q] > n_tile) { chunk0.push_back(q); cur = 0; }
                        cur += cnt[q];
                    }
                    chunk0.push_back(n_chunks);
                    if ((int)chunk0.size() - 1 <= n_tiles || n_tile >= 128) break;
                    n_tile += 16;            // chunk-aligned tiles wasted too many rows: widen the tile and try again
                }
                n_tiles = (int)chunk0.size() - 1;
                std::vector<int32_t> out_map(out_C_pad, -1);
                row_src.assign((size_t)n_tiles * n_tile, -1);
                for (int t = 0; t < n_tiles; ++t) {
                    int r = t * n_tile;
                    for (int c = chunk0[t] * 8; c < chunk0[t + 1] * 8 && c < f.K; ++c)
                        if (f.mask[c]) { row_src[r] = c; out_map[c] = r; ++r; }
                }
                f.K_rows = f.K; f.K_pad = n_tiles * n_tile; f.n_tile_forced = n_tile;
                out.keep.resize(f.K);
                for (int k = 0; k < f.K; ++k) out.keep[k] = k;
                TRY(upload_i32(h, out_map, &f.d_out_map));
                TRY(upload_i32(h, chunk0, &f.d_chunk0));
                out.C = f.K; out.C_pad = out_C_pad;
            } else {
                if (f.compact) {
                    f.K_rows = f.K_kept;
                    out.keep = kept;
                    for (int k : kept) row_src.push_back(k);
                } else {
                    f.K_rows = f.K;
                    out.keep.resize(f.K);
                    for (int k = 0; k < f.K; ++k) { out.keep[k] = k; row_src.push_back(f.mask[k] ? k : -1); }
                }
                f.K_pad = round_up(f.K_rows, 16);
                row_src.resize(f.K_pad, -1);
                out.C = f.K_rows; out.C_pad = f.K_pad;
            }
            for (int c = 0; c < src.C; ++c) chan_src[c] = src.keep[c];
            if (f.src == 0 && stem_candidate && !f.scatter && fp::stem_pool_supported(f.C, h->in_H, h->in_W, f.K_pad)) {
                h->stem_fused = 1;
                h->stem_packed = 0;
                int32_t* d_row;
                TRY(upload_i32(h, row_src, &d_row));
                f.d_row = d_row; f.d_chan = nullptr;
                TRY(dev_alloc(h, h->pack_buffers, &f.d_wp, (size_t)256 * f.K_pad * 2));
                TRY(dev_alloc(h, h->pack_buffers, (void**)&f.d_bp, (size_t)f.K_pad * sizeof(float)));
                fp::launch_repack_stem_direct(f.d_w32, f.C, d_row, f.K_pad, (__nv_bfloat16*)f.d_wp, st);
                fp::launch_pack_bias(f.d_b32, d_row, f.K_pad, f.d_bp, st);
                f.tc.valid = 0;
                continue;
            }
            // launch plan of the tensor-core kernel (geometry only; the pointers follow once memory is planned)
            f.tc.valid = 0;
            // A 1x1 layer that adds a projection shortcut (a 1x1 convolution, stride 1 or 2, no ReLU, read by nobody else)
            // takes the projection in: its filters are stacked behind this layer's along the channels and its input
            // tensor becomes a second input of this layer (Sec. IV-B's [W2' || S_w] for this one kind of block) - the
            // projection's output is neither written nor read back.  A stride-2 projection must read a parity-split
            // tensor (its pixels are then the parity-00 images, on this layer's position grid).  Not with keep_outputs
            // (every operator's output is wanted then) and not where either layer scatters its output.
            int pj = -1;
            if (h->compute == FP_COMPUTE_BF16_TC && !h->keep_outputs && f.res_mode == 1 && f.R == 1 && f.S == 1 && f.stride == 1 &&
                f.pad == 0 && !f.scatter && !src.split && !out.split && uses[f.res_tid].size() == 1) {
                const Tensor& rt = h->tensors[f.res_tid];
                if (rt.producer >= 0 && h->ops[rt.producer].kind == 0) {
                    const int cand = h->ops[rt.producer].idx;
                    const FConv& q = h->convs[cand];
                    const Tensor& X = h->tensors[q.src];
                    if (q.R == 1 && q.S == 1 && q.pad == 0 && q.res_mode == 0 && !q.relu && !q.scatter && !q.compact && q.K == f.K &&
                        q.K_pad == f.K_pad && q.n_mult == 1 && q.tc.valid && q.d_wp_plain && !(h->stem_packed && q.src == 0) &&
                        ((q.stride == 1 && !X.split) || (q.stride == 2 && X.split)))
                        pj = cand;
                }
            }
            const int C_pad_total = f.C_pad + (pj >= 0 ? h->convs[pj].C_pad : 0);
            if (h->compute == FP_COMPUTE_BF16_TC) {
                fp::ConvArgs ga;
                memset(&ga, 0, sizeof(ga));
                conv_geometry(h, f, &ga);
                ga.C_pad = (h->stem_packed && f.src == 0) ? 80 : C_pad_total;
                ga.K_pad = f.K_pad;
                ga.scatter = f.scatter; ga.out_C_pad = out.C_pad; ga.n_tile_forced = f.n_tile_forced;
                char msg[256];
                if (fp::plan_conv_tc(ga, &f.tc, msg, sizeof(msg)) != 0)
                    return fail(FP_ERR_UNSUPPORTED, "convolution %d: %s", f.conv_index, msg);
            }
            // pack filters and bias
            int32_t *d_row, *d_chan;
            TRY(upload_i32(h, row_src, &d_row));
            TRY(upload_i32(h, chan_src, &d_chan));
            f.d_row = d_row; f.d_chan = d_chan;
            const bool packed_stem = h->stem_packed && f.src == 0;
            const size_t cnt = packed_stem ? (size_t)f.K_pad * 3 * 80 : (size_t)f.K_pad * f.R * f.S * f.C_pad;
            TRY(dev_alloc(h, h->pack_buffers, &f.d_wp, cnt * h->act_elem()));
            TRY(dev_alloc(h, h->pack_buffers, (void**)&f.d_bp, (size_t)f.K_pad * sizeof(float)));
            if (packed_stem) fp::launch_repack_stem(f.d_w32, f.C, d_row, f.K_pad, (__nv_bfloat16*)f.d_wp, st);
            else fp::launch_repack_conv(f.d_w32, f.C, f.R * f.S, d_row, f.K_pad, d_chan, f.C_pad,
                                   bf16 ? (__nv_bfloat16*)f.d_wp : nullptr, bf16 ? nullptr : (float*)f.d_wp, st);
            fp::launch_pack_bias(f.d_b32, d_row, f.K_pad, f.d_bp, st);
            f.d_wp_plain = f.d_wp;
            if (pj >= 0) {
                // [chunk][K_pad][8]: this layer's chunks, then the projection's; the biases add up
                FConv& q = h->convs[pj];
                const size_t b1 = (size_t)f.C_pad * f.K_pad * h->act_elem(), b2 = (size_t)q.C_pad * f.K_pad * h->act_elem();
                void* cat; float* bsum;
                TRY(dev_alloc(h, h->pack_buffers, &cat, b1 + b2));
                TRY(dev_alloc(h, h->pack_buffers, (void**)&bsum, (size_t)f.K_pad * sizeof(float)));
                CK(cudaMemcpyAsync(cat, f.d_wp, b1, cudaMemcpyDeviceToDevice, st));
                CK(cudaMemcpyAsync((uint8_t*)cat + b1, q.d_wp_plain, b2, cudaMemcpyDeviceToDevice, st));
                fp::launch_add_bias(f.d_bp, q.d_bp, f.K_pad, bsum, st);
                f.d_wp = cat; f.d_bp = bsum;
                f.proj = pj; f.proj_kind = 1; q.absorbed = 1;
            }
            // The same for a 3x3 / stride-1 layer with streamed filters (the second layer of a basic block that changes the
            // resolution): the projection becomes extra K groups with a centre tap only, read from its own packed bank.
            if (pj < 0 && h->compute == FP_COMPUTE_BF16_TC && !h->keep_outputs && f.res_mode == 1 && f.R == 3 && f.S == 3 &&
                f.stride == 1 && f.pad == 1 && !f.scatter && !src.split && !out.split && uses[f.res_tid].size() == 1 && f.tc.valid &&
                f.tc.flat && !f.tc.b_resident && f.tc.blocked_bank == 0 && !(h->stem_packed && f.src == 0)) {
                const Tensor& rt = h->tensors[f.res_tid];
                if (rt.producer >= 0 && h->ops[rt.producer].kind == 0) {
                    const int cand = h->ops[rt.producer].idx;
                    FConv& q = h->convs[cand];
                    const Tensor& X = h->tensors[q.src];
                    if (q.R == 1 && q.S == 1 && q.pad == 0 && q.res_mode == 0 && !q.relu && !q.scatter && !q.compact && q.K == f.K &&
                        q.K_pad == f.K_pad && q.n_mult == 1 && q.tc.valid && q.d_wp_plain && !(h->stem_packed && q.src == 0) &&
                        ((q.stride == 1 && !X.split) || (q.stride == 2 && X.split))) {
                        float* bsum;
                        TRY(dev_alloc(h, h->pack_buffers, (void**)&bsum, (size_t)f.K_pad * sizeof(float)));
                        fp::launch_add_bias(f.d_bp, q.d_bp, f.K_pad, bsum, st);
                        f.d_bp = bsum;
                        f.proj = cand; f.proj_kind = 2; q.absorbed = 1;
                    }
                }
            }
            if (f.tc.valid && f.tc.blocked_bank) {
                // the streamed form of the kernel reads its bank block by block: one copy per pipeline stage
                const int taps = packed_stem ? 3 : f.R * f.S, cchunks = (packed_stem ? 80 : C_pad_total) / 8;
                void* blocked;
                TRY(dev_alloc(h, h->pack_buffers, &blocked, (size_t)f.tc.n_tiles * taps * cchunks * f.tc.n_tile * 16));
                if (f.tc.blocked_bank == 1)          // 1x1 layer, unified stages: [tile][K group][tap][chunk][row]
                    fp::launch_reblock_bank((const __nv_bfloat16*)f.d_wp, taps, cchunks, f.K_pad, f.tc.n_tile, f.tc.n_tiles, f.tc.cg,
                                            (__nv_bfloat16*)blocked, st);
                else                                 // gathered layer with several filter tiles: [tile][(tap, chunk) plane][row]
                    fp::launch_reblock_bank((const __nv_bfloat16*)f.d_wp, 1, taps * cchunks, f.K_pad, f.tc.n_tile, f.tc.n_tiles,
                                            taps * cchunks, (__nv_bfloat16*)blocked, st);
                f.d_wp = blocked;
            }
        } else if (op.kind == 1) {
            const Pool& p = h->pools[op.idx];
            const Tensor& src = h->tensors[p.src];
            Tensor& out = h->tensors[p.out];
            out.C = src.C; out.C_pad = src.C_pad; out.keep = src.keep;
        } else if (op.kind == 2) {
            const Tensor& src = h->tensors[h->head_src];
            std::vector<int32_t> chan_src(src.C_pad, -1);
            for (int c = 0; c < src.C; ++c) chan_src[c] = src.keep[c];
            int32_t* d_chan;
            TRY(upload_i32(h, chan_src, &d_chan));
            TRY(dev_alloc(h, h->pack_buffers, (void**)&h->d_fcw_packed, (size_t)h->n_classes * src.C_pad * sizeof(float)));
            TRY(dev_alloc(h, h->pack_buffers, (void**)&h->d_pool, (size_t)h->max_batch * src.C_pad * sizeof(float)));
            // the average's 1/(H*W) is folded into the FC weights
            fp::launch_repack_fc(h->d_fcw, h->fc_C, h->n_classes, d_chan, src.C_pad, 1.0f / (float)(src.H * src.W),
                                 h->d_fcw_packed, st);
        }
    }
    CK(cudaGetLastError());
    TRY(find_chains(h, uses));

    // --- activation memory: buffers are reused once their last reader has run ---
    {
        const int nt = (int)h->tensors.size();
        std::vector<int> last_use(nt, -1);
        for (int t = 0; t < nt; ++t)
            for (const Use& u : uses[t]) last_use[t] = std::max(last_use[t], u.op);
        for (int i = 0; i < (int)h->ops.size(); ++i)           // a layer that took a projection in also reads the projection's input
            if (h->ops[i].kind == 0 && h->convs[h->ops[i].idx].proj >= 0) {
                const int x = h->convs[h->convs[h->ops[i].idx].proj].src;
                last_use[x] = std::max(last_use[x], i);
            }
        struct Buf { void* p; size_t bytes; int free_after; };
        std::vector<Buf> bufs;
        for (int i = 0; i < (int)h->ops.size(); ++i) {
            const Op& op = h->ops[i];
            int tid = -1;
            if (op.kind == 0 && h->op_chain[i] >= 0) {
                // a fused run is one kernel: only its last tensor exists in memory, and it must not share
                // a buffer with the run's inputs, which other CTAs still read while the first ones finish
                const Chain& ch = h->chains[h->op_chain[i]];
                if (i != ch.last_op) h->tensors[h->convs[op.idx].out].d = nullptr;
                if (i != ch.first_op) continue;
                tid = h->convs[ch.convs.back()].out;
            }
            else if (op.kind == 0) tid = h->convs[op.idx].out;
            else if (op.kind == 1) tid = h->pools[op.idx].out;
            else if (op.kind == 3) tid = 0;
            if (h->stem_fused && (i == 0 || i == 1)) {          // neither the converted input nor the first convolution's output exists
                h->tensors[tid].d = nullptr;
                continue;
            }
            if (op.kind == 0 && h->convs[op.idx].absorbed) {    // a projection computed inside the layer that adds it
                h->tensors[tid].d = nullptr;
                continue;
            }
            if (tid < 0) continue;
            Tensor& t = h->tensors[tid];
            // planar-8 with border, plus guard vectors before and after (halo reads of the first/last tiles)
            const size_t vec_bytes = 8 * h->act_elem();
            t.bytes = ((size_t)(t.C_pad / 8) * h->max_batch * (t.H + 2) * (t.W + 2) + 2 * (size_t)fp::kGuardVectors) * vec_bytes;
            if (t.split)
                t.bytes = ((size_t)(t.C_pad / 8) * 4 * h->max_batch * (t.H / 2 + 2) * (t.W / 2 + 2) + 2 * (size_t)fp::kGuardVectors) * vec_bytes;
            if (tid == 0 && h->stem_packed)
                t.bytes = ((size_t)10 * h->max_batch * (t.H / 2 + 2) * (t.W / 2 + 2) + 2 * (size_t)fp::kGuardVectors) * vec_bytes;
            int best = -1;
            if (!h->keep_outputs)
                for (int b = 0; b < (int)bufs.size(); ++b)
                    if (bufs[b].free_after < i && bufs[b].bytes >= t.bytes && (best < 0 || bufs[b].bytes < bufs[best].bytes)) best = b;
            if (best < 0) {
                void* p;
                TRY(dev_alloc(h, h->act_buffers, &p, t.bytes));
                CK(cudaMemsetAsync(p, 0, t.bytes, st));
                bufs.push_back({p, t.bytes, 0});
                best = (int)bufs.size() - 1;
            }
            t.d = (uint8_t*)bufs[best].p + (size_t)fp::kGuardVectors * vec_bytes;
            bufs[best].free_after = std::max(last_use[tid], i);
        }
    }

    // --- launch arguments and tensor-core plans ---
    for (FConv& f : h->convs) {
        const Tensor& src = h->tensors[f.src];
        const Tensor& out = h->tensors[f.out];
        fp::ConvArgs& a = f.args;
        memset(&a, 0, sizeof(a));
        a.x = src.d; a.y = out.d; a.w = f.d_wp; a.bias = f.d_bp;
        conv_geometry(h, f, &a);
        a.C_pad = (h->stem_packed && f.src == 0) ? 80 : f.C_pad;
        a.K_pad = f.K_pad;
        a.scatter = f.scatter; a.out_C_pad = out.C_pad; a.out_map = f.d_out_map; a.tile_chunk0 = f.d_chunk0;
        a.n_tile_forced = f.n_tile_forced;
        a.res_mode = f.res_mode;
        if (f.proj >= 0) {
            const FConv& q = h->convs[f.proj];
            const Tensor& X = h->tensors[q.src];
            a.x2 = X.d; a.x2_plane_mult = X.split ? 4 : 1;
            if (f.proj_kind == 1) { a.C_pad = f.C_pad + q.C_pad; a.x2_chunk0 = f.C_pad / 8; }
            else { a.w2 = q.d_wp_plain; a.x2_C_pad = q.C_pad; }
            a.res_mode = 0;
        } else if (f.res_mode) {
            const Tensor& r = h->tensors[f.res_tid];
            a.res = r.d; a.res_H = r.H; a.res_W = r.W; a.res_C_pad = r.C_pad; a.res_C = r.C;
            a.res_pad_lo = f.res_pad_lo; a.res_stride = f.res_stride;
        }
    }
    for (Chain& ch : h->chains) {
        const FConv& f0 = h->convs[ch.convs.front()];
        const FConv& fl = h->convs[ch.convs.back()];
        ch.args.x = f0.args.x; ch.args.res = f0.args.res; ch.args.y = fl.args.y; ch.args.w = ch.d_blob;
    }
    if (h->stem_fused) {
        const FConv& f = h->convs[h->ops[1].idx];
        fp::StemPoolArgs& a = h->stem_args;
        memset(&a, 0, sizeof(a));
        a.y = h->tensors[h->pools[h->ops[2].idx].out].d; a.w = f.d_wp; a.bias = f.d_bp;
        a.N = h->max_batch; a.C = f.C; a.H = h->in_H; a.W = h->in_W; a.K_pad = f.K_pad; a.n0 = 0; a.n_count = h->max_batch;
        char msg[256];
        if (fp::plan_stem_pool(a, &h->stem_plan, msg, sizeof(msg)) != 0) return fail(FP_ERR_UNSUPPORTED, "%s", msg);
    }
    CK(cudaDeviceSynchronize());
    h->planned = 1;
    return FP_OK;
}

fp_status need_plan(fp_handle h, const char* who) {
    if (h->planned) return FP_OK;
    return fail(FP_ERR_ARG, "%s: the last fp_prune / fp_soft_prune_finish failed and left the handle without a plan; "
                            "call fp_prune again", who);
}

// ---------------------------------------------------------------------------------------
// execution
// ---------------------------------------------------------------------------------------

// n0, n_count: the images an input conversion handles (the other operators always run the whole batch)
void launch_op(fp_handle h, int op_index, const void* d_input, int batch, float* d_logits, cudaStream_t st, int n0 = 0,
               int n_count = -1) {
    if (n_count < 0) n_count = batch;
    const Op& op = h->ops[op_index];
    const int bf16 = h->act_is_bf16();
    if (op.kind == 3 && (h->input_fused || h->stem_fused)) return;        // the first kernel reads the network input itself
    if (h->stem_fused && op_index == 2) return;         // pooled inside the first convolution's kernel
    if (h->stem_fused && op_index == 1) {
        fp::StemPoolArgs a = h->stem_args;
        a.x = d_input; a.N = batch; a.n0 = n0; a.n_count = n_count;
        fp::launch_stem_pool(h->stem_plan, a, h->d_status, st);
        return;
    }
    if (op.kind == 0 && h->convs[op.idx].absorbed) return;        // runs inside the layer that adds its result
    if (op.kind == 0 && h->op_chain[op_index] >= 0) {
        const Chain& ch = h->chains[h->op_chain[op_index]];
        if (op_index != ch.first_op) return;       // the run's first operator launches all of it
        fp::ChainArgs a = ch.args;
        a.N = batch;
        if (a.in_mode) a.x = d_input;
        fp::launch_chain_tc(ch.plan, a, h->d_status, st);
        return;
    }
    if (op.kind == 3) {
        const Tensor& t = h->tensors[0];
        if (h->stem_packed) fp::launch_input_to_stem_planar(d_input, h->in_dtype == FP_DTYPE_BF16, t.d, batch, t.C, t.H, t.W, n0, n_count, st);
        else fp::launch_input_to_planar(d_input, h->in_dtype == FP_DTYPE_BF16, t.d, bf16, batch, t.C, t.H, t.W, t.C_pad, n0, n_count, st);
    } else if (op.kind == 0) {
        FConv& f = h->convs[op.idx];
        fp::ConvArgs a = f.args;
        a.N = batch * f.n_mult;
        if (h->compute == FP_COMPUTE_BF16_TC) fp::launch_conv_tc(f.tc, a, h->d_status, st);
        else fp::launch_conv_simt(a, bf16, st);
    } else if (op.kind == 1) {
        const Pool& p = h->pools[op.idx];
        const Tensor& s = h->tensors[p.src];
        const Tensor& o = h->tensors[p.out];
        fp::launch_maxpool(s.d, o.d, bf16, batch, s.H, s.W, s.C_pad, o.H, o.W, p.R, p.stride, p.pad, st);
    } else {
        const Tensor& s = h->tensors[h->head_src];
        fp::launch_head(s.d, bf16, batch, s.H, s.W, s.C_pad, h->d_fcw_packed, h->d_fcb, h->n_classes, d_logits, h->d_pool, st);
    }
}

void launch_all(fp_handle h, const void* d_input, int batch, float* d_logits, cudaStream_t st, int first = 0) {
    for (int i = first; i < (int)h->ops.size(); ++i) launch_op(h, i, d_input, batch, d_logits, st);
}

fp_status all_ones_masks(fp_handle h) {
    for (FConv& f : h->convs) {
        f.mask.assign(f.K, 1);
        f.rank.assign(f.K, 0);
        for (int k = 0; k < f.K; ++k) f.rank[k] = k;
    }
    return FP_OK;
}

}  // namespace

// =========================================================================================
// C ABI
// =========================================================================================

extern "C" const char* fp_last_error(void) { return g_err.c_str(); }

namespace fp_detail {
fp_status set_error(fp_status st, const char* msg) { return fail(st, "%s", msg); }
}

extern "C" fp_status fp_destroy(fp_handle h) {
    if (!h) return FP_OK;
    cudaDeviceSynchronize();
    drop_graphs(h);
    if (h->copy_stream) {
        cudaStreamDestroy(h->copy_stream);
        for (cudaEvent_t e : h->copy_events) if (e) cudaEventDestroy(e);
    }
    free_list(h, h->act_buffers);
    free_list(h, h->pack_buffers);
    free_list(h, h->fixed_buffers);
    delete h;
    return FP_OK;
}

extern "C" fp_status fp_fuse(const fp_model_desc* desc, const float* d_weights, size_t n_weights, const float* d_bn,
                             size_t n_bn, int32_t max_batch, fp_handle* out) {
    return fp_fuse_with_allocator(desc, d_weights, n_weights, d_bn, n_bn, max_batch, nullptr, nullptr, nullptr, out);
}

extern "C" fp_status fp_fuse_with_allocator(const fp_model_desc* desc, const float* d_weights, size_t n_weights,
                                            const float* d_bn, size_t n_bn, int32_t max_batch,
                                            void* (*alloc)(size_t, void*), void (*dealloc)(void*, void*), void* user,
                                            fp_handle* out) {
    if (!desc || !out || !d_weights || !desc->nodes) return fail(FP_ERR_ARG, "fp_fuse: NULL argument");
    if ((alloc == nullptr) != (dealloc == nullptr)) return fail(FP_ERR_ARG, "fp_fuse: alloc and dealloc must be given together");
    if (!d_bn && n_bn) return fail(FP_ERR_ARG, "fp_fuse: NULL BN array");
    if (desc->n_nodes <= 0 || max_batch <= 0) return fail(FP_ERR_ARG, "fp_fuse: n_nodes and max_batch must be positive");
    if (desc->in_C <= 0 || desc->in_H <= 0 || desc->in_W <= 0) return fail(FP_ERR_ARG, "fp_fuse: bad input shape");
    if (desc->in_dtype != FP_DTYPE_F32 && desc->in_dtype != FP_DTYPE_BF16) return fail(FP_ERR_ARG, "fp_fuse: bad in_dtype");
    if (desc->compute < 0 || desc->compute > 2) return fail(FP_ERR_ARG, "fp_fuse: bad compute mode");
    if (desc->scatter < -1 || desc->scatter > 1) return fail(FP_ERR_ARG, "fp_fuse: bad scatter policy");
    if (!(desc->bn_eps > 0.0f) || !std::isfinite(desc->bn_eps)) return fail(FP_ERR_ARG, "fp_fuse: bn_eps must be positive");
    int dev = 0;
    cudaDeviceProp prop;
    CK(cudaGetDevice(&dev));
    CK(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10) return fail(FP_ERR_UNSUPPORTED, "fp_fuse: needs a compute-capability 10.x GPU (found %d.%d)", prop.major, prop.minor);

    fp_handle h = new fp_handle_s();
    h->alloc = alloc; h->dealloc = dealloc; h->alloc_user = user;
    h->nodes.assign(desc->nodes, desc->nodes + desc->n_nodes);
    h->in_C = desc->in_C; h->in_H = desc->in_H; h->in_W = desc->in_W;
    h->in_dtype = desc->in_dtype; h->compute = desc->compute; h->use_graph = desc->use_graph;
    h->keep_outputs = desc->keep_outputs;
    h->scatter_policy = desc->scatter;
    h->eps = desc->bn_eps; h->max_batch = max_batch;
    fp_status s = FP_OK;
    auto body = [&]() -> fp_status {
        // own copies of the parameters, checked for NaN/Inf on the device
        float *wcopy, *bcopy;
        int* d_bad;
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&wcopy, n_weights * sizeof(float)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&bcopy, n_bn * sizeof(float)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&d_bad, sizeof(int)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_status, sizeof(int)));
        CK(cudaMemcpy(wcopy, d_weights, n_weights * sizeof(float), cudaMemcpyDeviceToDevice));
        if (n_bn) CK(cudaMemcpy(bcopy, d_bn, n_bn * sizeof(float), cudaMemcpyDeviceToDevice));
        CK(cudaMemset(d_bad, 0, sizeof(int)));
        CK(cudaMemset(h->d_status, 0, sizeof(int)));
        fp::launch_count_nonfinite(wcopy, n_weights, d_bad, 0);
        fp::launch_count_nonfinite(bcopy, n_bn, d_bad, 0);
        int bad = 0;
        CK(cudaMemcpy(&bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost));
        if (bad) return fail(FP_ERR_NONFINITE, "fp_fuse: %d non-finite values in the weights or BN statistics", bad);
        Builder b;
        b.h = h; b.d_weights = wcopy; b.d_bn = bcopy; b.n_weights = n_weights; b.n_bn = n_bn;
        TRY(b.run());
        CK(cudaGetLastError());
        int max_K = 1;
        for (const FConv& f : h->convs) max_K = std::max(max_K, f.K);
        if ((size_t)max_K * sizeof(double) > 48 * 1024) return fail(FP_ERR_UNSUPPORTED, "fp_fuse: more than 6144 filters in one convolution");
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_scores, (size_t)max_K * sizeof(double)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_rank, (size_t)max_K * sizeof(int32_t)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_mask, (size_t)max_K));
        TRY(dev_alloc(h, h->fixed_buffers, &h->d_in_stage, (size_t)max_batch * h->in_C * h->in_H * h->in_W * h->in_elem()));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_logits_stage, (size_t)max_batch * h->n_classes * sizeof(float)));
        all_ones_masks(h);
        TRY(replan(h));
        return FP_OK;
    };
    s = body();
    if (s != FP_OK) {
        std::string keep = g_err;
        fp_destroy(h);
        g_err = keep;
        return s;
    }
    *out = h;
    return FP_OK;
}

static fp_status score_conv(fp_handle h, const FConv& f, int norm) {
    fp::launch_score_filters(f.d_w32, f.K, f.C * f.R * f.S, norm, h->d_scores, 0);
    CK(cudaGetLastError());
    return FP_OK;
}

extern "C" fp_status fp_score(fp_handle h, int32_t conv_index, int32_t norm, double* h_scores) {
    if (!h || !h_scores) return fail(FP_ERR_ARG, "fp_score: NULL argument");
    if (norm != FP_NORM_L1 && norm != FP_NORM_L2) return fail(FP_ERR_ARG, "fp_score: bad norm");
    if (conv_index < 0 || conv_index >= h->n_desc_convs || h->conv_to_fused[conv_index] < 0)
        return fail(FP_ERR_ARG, "fp_score: convolution %d does not exist in the fused graph", conv_index);
    const FConv& f = h->convs[h->conv_to_fused[conv_index]];
    TRY(score_conv(h, f, norm));
    CK(cudaMemcpy(h_scores, h->d_scores, (size_t)f.K * sizeof(double), cudaMemcpyDeviceToHost));
    return FP_OK;
}

extern "C" fp_status fp_prune(fp_handle h, int32_t norm, const double* h_ratios, const uint8_t* const* h_masks) {
    if (!h) return fail(FP_ERR_ARG, "fp_prune: NULL handle");
    if (norm != FP_NORM_L1 && norm != FP_NORM_L2) return fail(FP_ERR_ARG, "fp_prune: bad norm");
    // select every mask first (all scores are taken on the unpruned fused weights), then apply
    std::vector<std::vector<uint8_t>> masks(h->convs.size());
    std::vector<std::vector<int32_t>> ranks(h->convs.size());
    for (size_t i = 0; i < h->convs.size(); ++i) {
        const FConv& f = h->convs[i];
        masks[i].resize(f.K);
        ranks[i].resize(f.K);
        TRY(score_conv(h, f, norm));
        const uint8_t* given = h_masks ? h_masks[f.conv_index] : nullptr;
        int q;
        if (f.role != 0) q = f.K - f.n_orig;               // fused operator: back to its original filter count
        else {
            const double r = h_ratios ? h_ratios[f.conv_index] : 0.0;
            if (!(r >= 0.0) || r > 1.0) return fail(FP_ERR_ARG, "fp_prune: ratio of convolution %d outside [0,1]", f.conv_index);
            q = (int)std::floor(r * (double)f.K + 1e-9);
        }
        fp::launch_rank_mask(h->d_scores, f.K, q, h->d_rank, h->d_mask, 0);
        CK(cudaGetLastError());
        CK(cudaMemcpy(ranks[i].data(), h->d_rank, (size_t)f.K * sizeof(int32_t), cudaMemcpyDeviceToHost));
        if (given) {
            for (int k = 0; k < f.K; ++k) {
                if (given[k] > 1) return fail(FP_ERR_ARG, "fp_prune: mask of convolution %d has a value other than 0/1", f.conv_index);
                masks[i][k] = given[k];
            }
        } else {
            CK(cudaMemcpy(masks[i].data(), h->d_mask, (size_t)f.K, cudaMemcpyDeviceToHost));
        }
        int kept = 0;
        for (int k = 0; k < f.K; ++k) kept += masks[i][k];
        if (kept == 0) return fail(FP_ERR_EMPTY_LAYER, "fp_prune: convolution %d would keep no filter", f.conv_index);
    }
    for (size_t i = 0; i < h->convs.size(); ++i) { h->convs[i].mask = masks[i]; h->convs[i].rank = ranks[i]; }
    return replan(h);
}

// One pass of Algorithm 1's loop body: update, score, select, zeroize in place.  The running graph is untouched.
extern "C" fp_status fp_soft_prune_epoch(fp_handle h, int32_t norm, const double* h_ratios, const float* d_updates) {
    if (!h) return fail(FP_ERR_ARG, "fp_soft_prune_epoch: NULL handle");
    if (norm != FP_NORM_L1 && norm != FP_NORM_L2) return fail(FP_ERR_ARG, "fp_soft_prune_epoch: bad norm");
    // validate everything before the banks are touched
    std::vector<int> q(h->convs.size(), 0);
    for (size_t i = 0; i < h->convs.size(); ++i) {
        const FConv& f = h->convs[i];
        if (f.role != 0) q[i] = f.K - f.n_orig;
        else {
            const double r = h_ratios ? h_ratios[f.conv_index] : 0.0;
            if (!(r >= 0.0) || r > 1.0) return fail(FP_ERR_ARG, "fp_soft_prune_epoch: ratio of convolution %d outside [0,1]", f.conv_index);
            q[i] = (int)std::floor(r * (double)f.K + 1e-9);
        }
        if (q[i] >= f.K) return fail(FP_ERR_EMPTY_LAYER, "fp_soft_prune_epoch: convolution %d would keep no filter", f.conv_index);
    }
    // bank table in description order (the order of the update array), filters numbered bank by bank
    std::vector<fp::SoftBank> banks;
    std::vector<int32_t> map;
    std::vector<size_t> fused_of;
    long long off = 0;
    int k_off = 0, max_K = 1;
    for (int ci = 0; ci < h->n_desc_convs; ++ci) {
        if (h->conv_to_fused[ci] < 0) continue;
        const size_t i = (size_t)h->conv_to_fused[ci];
        const FConv& f = h->convs[i];
        fp::SoftBank b;
        b.w = f.d_w32; b.dw_off = off; b.K = f.K; b.per = f.C * f.R * f.S; b.q = q[i]; b.k_off = k_off;
        for (int k = 0; k < f.K; ++k) map.push_back((int32_t)banks.size());
        banks.push_back(b);
        fused_of.push_back(i);
        off += (long long)f.K * b.per;
        k_off += f.K;
        max_K = std::max(max_K, f.K);
    }
    if (!h->d_soft_banks) {
        h->soft_total = k_off;
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_soft_banks, banks.size() * sizeof(fp::SoftBank)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_soft_map, map.size() * sizeof(int32_t)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_soft_scores, (size_t)k_off * sizeof(double)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_soft_rank, (size_t)k_off * sizeof(int32_t)));
        TRY(dev_alloc(h, h->fixed_buffers, (void**)&h->d_soft_mask, (size_t)k_off));
        CK(cudaMemcpy(h->d_soft_map, map.data(), map.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    }
    CK(cudaMemcpy(h->d_soft_banks, banks.data(), banks.size() * sizeof(fp::SoftBank), cudaMemcpyHostToDevice));
    fp::launch_soft_update_score(h->d_soft_banks, h->d_soft_map, k_off, d_updates, norm, h->d_soft_scores, 0);
    fp::launch_soft_rank(h->d_soft_banks, (int)banks.size(), max_K, h->d_soft_scores, h->d_soft_rank, h->d_soft_mask, 0);
    fp::launch_soft_zeroize(h->d_soft_banks, h->d_soft_map, k_off, h->d_soft_mask, 0);
    CK(cudaGetLastError());
    std::vector<int32_t> all_rank(k_off);
    std::vector<uint8_t> all_mask(k_off);
    CK(cudaMemcpy(all_rank.data(), h->d_soft_rank, (size_t)k_off * sizeof(int32_t), cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(all_mask.data(), h->d_soft_mask, (size_t)k_off, cudaMemcpyDeviceToHost));
    for (size_t bi = 0; bi < banks.size(); ++bi) {
        FConv& f = h->convs[fused_of[bi]];
        f.rank.assign(all_rank.begin() + banks[bi].k_off, all_rank.begin() + banks[bi].k_off + f.K);
        f.mask.assign(all_mask.begin() + banks[bi].k_off, all_mask.begin() + banks[bi].k_off + f.K);
    }
    ++h->soft_epochs;
    return FP_OK;
}

extern "C" fp_status fp_soft_prune_finish(fp_handle h) {
    if (!h) return fail(FP_ERR_ARG, "fp_soft_prune_finish: NULL handle");
    if (h->soft_epochs == 0) return fail(FP_ERR_ARG, "fp_soft_prune_finish: no fp_soft_prune_epoch has run");
    return replan(h);
}

// Operators first .. last of the forward on `st`, as a replayed CUDA graph where the handle asks for one.
static fp_status forward_from(fp_handle h, const void* d_input, int32_t batch, float* d_logits, cudaStream_t st, int first) {
    const bool graphable = h->use_graph && st != 0 && st != cudaStreamLegacy && st != cudaStreamPerThread;
    if (!graphable) {
        launch_all(h, d_input, batch, d_logits, st, first);
        CK(cudaGetLastError());
        return FP_OK;
    }
    GraphKey key{batch, first, d_input, d_logits, st};
    auto it = h->graphs.find(key);
    if (it == h->graphs.end()) {
        cudaStreamCaptureStatus cs;
        CK(cudaStreamIsCapturing(st, &cs));
        if (cs != cudaStreamCaptureStatusNone) {   // already inside someone else's capture: just record the launches
            launch_all(h, d_input, batch, d_logits, st, first);
            CK(cudaGetLastError());
            return FP_OK;
        }
        cudaGraph_t g;
        CK(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
        launch_all(h, d_input, batch, d_logits, st, first);
        cudaError_t e = cudaStreamEndCapture(st, &g);
        if (e != cudaSuccess) return fail(FP_ERR_CUDA, "graph capture failed: %s", cudaGetErrorString(e));
        cudaGraphExec_t ge;
        e = cudaGraphInstantiate(&ge, g, 0);
        cudaGraphDestroy(g);
        if (e != cudaSuccess) return fail(FP_ERR_CUDA, "graph instantiate failed: %s", cudaGetErrorString(e));
        if (h->graphs.size() >= 16) drop_graphs(h);
        it = h->graphs.emplace(key, ge).first;
    }
    CK(cudaGraphLaunch(it->second, st));
    return FP_OK;
}

extern "C" fp_status fp_forward(fp_handle h, const void* d_input, int32_t batch, float* d_logits, void* stream) {
    if (!h || !d_input || !d_logits) return fail(FP_ERR_ARG, "fp_forward: NULL argument");
    if (batch <= 0) return fail(FP_ERR_ARG, "fp_forward: batch must be positive");
    if (batch > h->max_batch) return fail(FP_ERR_BOUNDS, "fp_forward: batch %d exceeds max_batch %d", batch, h->max_batch);
    TRY(need_plan(h, "fp_forward"));
    h->last_input = d_input; h->last_batch = batch;
    return forward_from(h, d_input, batch, d_logits, (cudaStream_t)stream, 0);
}

extern "C" fp_status fp_debug_expire_wait(fp_handle h, void* stream) {
    if (!h) return fail(FP_ERR_ARG, "fp_debug_expire_wait: NULL handle");
    TRY(need_plan(h, "fp_debug_expire_wait"));
    for (int i = 0; i < (int)h->ops.size(); ++i) {
        const Op& op = h->ops[i];
        if (op.kind != 0 || h->op_chain[i] >= 0 || (h->stem_fused && i == 1)) continue;
        const FConv& f = h->convs[op.idx];
        if (!f.tc.valid || !f.tc.flat || f.tc.blocked_bank || h->tensors[f.src].split || h->tensors[f.out].split || f.proj >= 0 || f.absorbed) continue;
        // the first round of the activation producer is left out, so the MMA-issuing thread's wait for that stage runs
        // out after a millisecond (two million cycles), raises the status word and takes every role of the CTA with it
        fp::launch_conv_tc(f.tc, f.args, h->d_status, (cudaStream_t)stream, 0, 2000000LL);
        CK(cudaGetLastError());
        return FP_OK;
    }
    return fail(FP_ERR_UNSUPPORTED, "fp_debug_expire_wait: the graph has no stride-1 convolution that runs on its own");
}

extern "C" fp_status fp_forward_host(fp_handle h, const void* h_input, int32_t batch, float* h_logits, void* stream) {
    TRY(fp_forward_host_async(h, h_input, batch, h_logits, stream));
    CK(cudaStreamSynchronize((cudaStream_t)stream));
    return FP_OK;
}

extern "C" fp_status fp_forward_host_async(fp_handle h, const void* h_input, int32_t batch, float* h_logits, void* stream) {
    if (!h || !h_input || !h_logits) return fail(FP_ERR_ARG, "fp_forward_host: NULL argument");
    if (batch <= 0) return fail(FP_ERR_ARG, "fp_forward_host: batch must be positive");
    if (batch > h->max_batch) return fail(FP_ERR_BOUNDS, "fp_forward_host: batch %d exceeds max_batch %d", batch, h->max_batch);
    TRY(need_plan(h, "fp_forward_host"));
    cudaStream_t st = (cudaStream_t)stream;
    const size_t image_bytes = (size_t)h->in_C * h->in_H * h->in_W * h->in_elem();
    h->last_input = h->d_in_stage; h->last_batch = batch;
    // Where the forward starts with a layout conversion of its own, the input crosses the bus in pieces on a second
    // stream and every piece is converted as soon as it has arrived, so only the last piece's copy is exposed; the
    // rest of the network then runs once on the whole batch.  (Where the first fused run of layers reads the network
    // input itself, the input is small: one copy, then the forward.)
    // (pieces of at least 8 MB: a copy has a fixed cost of some tens of microseconds, measured 1.14 ms end to end with
    // eight 2.4 MB pieces against 0.95 ms with one copy on ResNet-18 at batch 64)
    const size_t total_bytes = (size_t)batch * image_bytes;
    const bool own_input_op = h->ops[0].kind == 3 && !h->input_fused;
    const int pieces = (own_input_op && batch >= 2) ? std::max(1, std::min(std::min(kHostPieces, batch), (int)(total_bytes >> 23))) : 1;
    const int piece_op = h->stem_fused ? 1 : 0, tail_op = h->stem_fused ? 3 : 1;     // the kernel that takes the input in; what follows it
    if (own_input_op) {
        if (!h->copy_stream) {
            CK(cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
            for (int i = 0; i <= kHostPieces; ++i) CK(cudaEventCreateWithFlags(&h->copy_events[i], cudaEventDisableTiming));
        }
        // Only that first kernel reads the staging buffer: the copies wait for the previous call's first kernel(s) - the
        // event recorded behind them below - and not for the rest of its forward, so that a caller who queues call after
        // call (fp_forward_host_async) has the next input cross the bus while the network still runs on this one.
        if (h->stage_used) CK(cudaStreamWaitEvent(h->copy_stream, h->copy_events[kHostPieces], 0));
        for (int c = 0; c < pieces; ++c) {
            const int n0 = (int)((long long)batch * c / pieces), n1 = (int)((long long)batch * (c + 1) / pieces);
            CK(cudaMemcpyAsync((uint8_t*)h->d_in_stage + (size_t)n0 * image_bytes, (const uint8_t*)h_input + (size_t)n0 * image_bytes,
                               (size_t)(n1 - n0) * image_bytes, cudaMemcpyHostToDevice, h->copy_stream));
            CK(cudaEventRecord(h->copy_events[c], h->copy_stream));
            CK(cudaStreamWaitEvent(st, h->copy_events[c], 0));
            launch_op(h, piece_op, h->d_in_stage, batch, h->d_logits_stage, st, n0, n1 - n0);
        }
        CK(cudaGetLastError());
        CK(cudaEventRecord(h->copy_events[kHostPieces], st));         // the staging buffer is free again
        h->stage_used = 1;
        TRY(forward_from(h, h->d_in_stage, batch, h->d_logits_stage, st, tail_op));
    } else {
        CK(cudaMemcpyAsync(h->d_in_stage, h_input, (size_t)batch * image_bytes, cudaMemcpyHostToDevice, st));
        TRY(forward_from(h, h->d_in_stage, batch, h->d_logits_stage, st, 0));
    }
    CK(cudaMemcpyAsync(h_logits, h->d_logits_stage, (size_t)batch * h->n_classes * sizeof(float), cudaMemcpyDeviceToHost, st));
    return FP_OK;
}

static void fill_op_info(fp_handle h, int i, fp_op_info* o) {
    memset(o, 0, sizeof(*o));
    const Op& op = h->ops[i];
    const double e = (double)h->act_elem();
    o->kind = op.kind; o->conv_index = -1;
    o->chain = h->op_chain[i];
    if (op.kind == 0) {
        const FConv& f = h->convs[op.idx];
        const Tensor& s = h->tensors[f.src];
        const Tensor& t = h->tensors[f.out];
        o->conv_index = f.conv_index;
        o->K = f.K_kept; o->C = f.C_kept; o->R = f.R; o->S = f.S; o->stride = f.stride; o->pad = f.pad;
        o->K_pad = f.K_pad; o->C_pad = f.C_pad; o->H = s.H; o->W = s.W; o->P = t.H; o->Q = t.W;
        o->res_mode = f.res_mode; o->relu = f.relu;
        o->flops_per_image = 2.0 * t.H * t.W * (double)f.K_kept * f.C_kept * f.R * f.S;
        double b = (double)s.H * s.W * s.C * e + (double)t.H * t.W * t.C * e;
        if (f.res_mode == 1 && f.proj < 0) b += (double)t.H * t.W * t.C * e;
        if (f.res_mode == 2) b += (double)t.H * t.W * h->tensors[f.res_tid].C * e;
        o->bytes_per_image = b;
        o->bytes_fixed = (double)f.K_kept * f.C_kept * f.R * f.S * e + 4.0 * f.K_kept;
        if (f.proj >= 0) {
            // the projection shortcut computed inside this layer: its input at this layer's resolution, its filters, its flops
            const FConv& q = h->convs[f.proj];
            o->bytes_per_image += (double)t.H * t.W * q.C_kept * e;
            o->bytes_fixed += (double)q.K_kept * q.C_kept * e + 4.0 * q.K_kept;
            o->flops_per_image += 2.0 * t.H * t.W * (double)q.K_kept * q.C_kept;
        }
        if (f.absorbed) { o->flops_per_image = 0.0; o->bytes_per_image = 0.0; o->bytes_fixed = 0.0; }
    } else if (op.kind == 1) {
        const Pool& p = h->pools[op.idx];
        const Tensor& s = h->tensors[p.src];
        const Tensor& t = h->tensors[p.out];
        o->K = o->C = s.C; o->K_pad = o->C_pad = s.C_pad; o->R = o->S = p.R; o->stride = p.stride; o->pad = p.pad;
        o->H = s.H; o->W = s.W; o->P = t.H; o->Q = t.W;
        o->bytes_per_image = ((double)s.H * s.W + (double)t.H * t.W) * s.C * e;
    } else if (op.kind == 2) {
        const Tensor& s = h->tensors[h->head_src];
        o->K = h->n_classes; o->C = s.C; o->K_pad = h->n_classes; o->C_pad = s.C_pad; o->H = s.H; o->W = s.W; o->P = o->Q = 1;
        o->R = o->S = 1; o->stride = 1;
        o->flops_per_image = 2.0 * h->n_classes * s.C + (double)s.H * s.W * s.C;
        o->bytes_per_image = (double)s.H * s.W * s.C * e + 4.0 * h->n_classes;
        o->bytes_fixed = 4.0 * h->n_classes * (s.C + 1);
    } else {
        const Tensor& t = h->tensors[0];
        o->K = o->C = t.C; o->K_pad = o->C_pad = t.C_pad; o->H = o->P = t.H; o->W = o->Q = t.W; o->R = o->S = 1; o->stride = 1;
        o->bytes_per_image = (double)t.H * t.W * t.C * ((double)h->in_elem() + e);
    }
}

extern "C" fp_status fp_query(fp_handle h, int32_t what, int32_t index, void* h_out, size_t bytes) {
    if (!h || !h_out) return fail(FP_ERR_ARG, "fp_query: NULL argument");
    auto need = [&](size_t n) -> fp_status {
        return bytes >= n ? FP_OK : fail(FP_ERR_ARG, "fp_query: output buffer too small (%zu < %zu)", bytes, n);
    };
    auto conv_of = [&](const FConv** f) -> fp_status {
        if (index < 0 || index >= h->n_desc_convs) return fail(FP_ERR_ARG, "fp_query: convolution %d out of range", index);
        *f = h->conv_to_fused[index] >= 0 ? &h->convs[h->conv_to_fused[index]] : nullptr;
        return FP_OK;
    };
    const FConv* f = nullptr;
    switch (what) {
        case FP_Q_N_CONVS: TRY(need(4)); *(int32_t*)h_out = h->n_desc_convs; return FP_OK;
        case FP_Q_N_CLASSES: TRY(need(4)); *(int32_t*)h_out = h->n_classes; return FP_OK;
        case FP_Q_N_OPS: TRY(need(4)); *(int32_t*)h_out = (int32_t)h->ops.size(); return FP_OK;
        case FP_Q_N_LAUNCHES: {
            TRY(need(4));
            int n = (int)h->ops.size() + 1;                                  // the head is two kernels
            for (const Chain& ch : h->chains) n -= (int)ch.convs.size() - 1; // a fused run is one
            n -= h->input_fused;
            n -= 2 * h->stem_fused;                                          // conversion, convolution and pooling are one
            for (const FConv& c : h->convs) n -= c.absorbed;                 // a projection inside the layer that adds it
            *(int32_t*)h_out = n;
            return FP_OK;
        }
        case FP_Q_CONV_K_FUSED: TRY(need(4)); TRY(conv_of(&f)); *(int32_t*)h_out = f ? f->K : 0; return FP_OK;
        case FP_Q_CONV_K_KEPT: TRY(need(4)); TRY(conv_of(&f)); *(int32_t*)h_out = f ? f->K_kept : 0; return FP_OK;
        case FP_Q_CONV_C_KEPT: TRY(need(4)); TRY(conv_of(&f)); *(int32_t*)h_out = f ? f->C_kept : 0; return FP_OK;
        case FP_Q_CONV_BANK_ELEMS: TRY(need(8)); TRY(conv_of(&f)); *(int64_t*)h_out = f ? (int64_t)f->K * f->C * f->R * f->S : 0; return FP_OK;
        case FP_Q_MASK:
            TRY(conv_of(&f));
            if (!f) return fail(FP_ERR_ARG, "fp_query: convolution %d was absorbed by fusion", index);
            TRY(need(f->K)); memcpy(h_out, f->mask.data(), f->K); return FP_OK;
        case FP_Q_RANK:
            TRY(conv_of(&f));
            if (!f) return fail(FP_ERR_ARG, "fp_query: convolution %d was absorbed by fusion", index);
            TRY(need((size_t)f->K * 4)); memcpy(h_out, f->rank.data(), (size_t)f->K * 4); return FP_OK;
        case FP_Q_FLOPS: {
            TRY(need(8));
            double s = 0;
            for (int i = 0; i < (int)h->ops.size(); ++i) { fp_op_info o; fill_op_info(h, i, &o); s += o.flops_per_image; }
            *(double*)h_out = s; return FP_OK;
        }
        case FP_Q_BYTES: {
            TRY(need(16));
            double a = 0, b = 0;
            for (int i = 0; i < (int)h->ops.size(); ++i) { fp_op_info o; fill_op_info(h, i, &o); a += o.bytes_per_image; b += o.bytes_fixed; }
            ((double*)h_out)[0] = a; ((double*)h_out)[1] = b; return FP_OK;
        }
        case FP_Q_OP_INFO:
            if (index < 0 || index >= (int)h->ops.size()) return fail(FP_ERR_ARG, "fp_query: operator %d out of range", index);
            TRY(need(sizeof(fp_op_info)));
            fill_op_info(h, index, (fp_op_info*)h_out);
            return FP_OK;
        case FP_Q_OP_OUTPUT: {
            if (index < 0 || index >= (int)h->ops.size() || h->ops[index].kind == 2)
                return fail(FP_ERR_ARG, "fp_query: operator %d has no activation output", index);
            if (h->last_batch <= 0) return fail(FP_ERR_ARG, "fp_query: no forward has run yet");
            TRY(need_plan(h, "fp_query"));
            if (h->ops[index].kind == 3 && h->stem_packed) return fail(FP_ERR_UNSUPPORTED, "fp_query: the network input is stored in packed form");
            if (h->ops[index].kind == 3 && (h->input_fused || h->stem_fused)) return fail(FP_ERR_UNSUPPORTED, "fp_query: the network input is converted inside the first fused run "
                                                                        "and never stored (set keep_outputs to run every layer on its own)");
            const Op& op = h->ops[index];
            const int tid = op.kind == 0 ? h->convs[op.idx].out : op.kind == 1 ? h->pools[op.idx].out : 0;
            const Tensor& t = h->tensors[tid];
            if (!t.d) return fail(FP_ERR_UNSUPPORTED, "fp_query: operator %d runs inside another kernel (a fused run of layers, or the layer "
                                  "that adds this projection shortcut) and its output never reaches memory (set keep_outputs to run "
                                  "every layer on its own)", index);
            const size_t cnt = (size_t)h->last_batch * t.C * t.H * t.W;
            TRY(need(cnt * sizeof(float)));
            float* d_tmp;
            CK(cudaDeviceSynchronize());
            if (!h->keep_outputs) {
                // Buffers are reused once their last reader has run, so the tensor may have been overwritten since:
                // run the forward's launches up to this operator again (same input, same kernels) and stop there.
                if (!h->last_input) return fail(FP_ERR_ARG, "fp_query: no forward has run yet");
                for (int j = 0; j <= index; ++j) launch_op(h, j, h->last_input, h->last_batch, h->d_logits_stage, 0);
                CK(cudaDeviceSynchronize());
            }
            TRY(dev_alloc_raw(h, (void**)&d_tmp, cnt * sizeof(float)));
            fp::launch_planar_to_nchw_f32(t.d, h->act_is_bf16(), d_tmp, h->last_batch, t.H, t.W, t.C_pad, t.C, t.split, 0);
            cudaError_t e = cudaMemcpy(h_out, d_tmp, cnt * sizeof(float), cudaMemcpyDeviceToHost);
            dev_free(h, d_tmp);
            if (e != cudaSuccess) return fail(FP_ERR_CUDA, "fp_query: copy failed: %s", cudaGetErrorString(e));
            return FP_OK;
        }
        case FP_Q_DEVICE_STATUS: {
            TRY(need(4));
            int v = 0;
            CK(cudaMemcpy(&v, h->d_status, sizeof(int), cudaMemcpyDeviceToHost));
            if (v) CK(cudaMemset(h->d_status, 0, sizeof(int)));          // reported once
            *(int32_t*)h_out = v ? FP_ERR_TIMEOUT : 0;
            return FP_OK;
        }
        case FP_Q_OP_TIMES: {
            const int n = (int)h->ops.size();
            TRY(need((size_t)n * sizeof(float)));
            if (h->last_batch <= 0 || !h->last_input) return fail(FP_ERR_ARG, "fp_query: no forward has run yet");
            TRY(need_plan(h, "fp_query"));
            // Operator i's time = (time of the launches 0..i) - (time of the launches 0..i-1), each prefix of the forward
            // captured as a CUDA graph - the way fp_forward runs them, programmatic dependent launch included - and
            // replayed `reps` times back to back between two events.  An event between two kernels would cost more
            // than the short kernels it is meant to time.
            const int reps = index > 0 ? index : 10;
            cudaStream_t st;
            CK(cudaStreamCreate(&st));
            cudaEvent_t e0, e1;
            CK(cudaEventCreate(&e0));
            CK(cudaEventCreate(&e1));
            std::vector<float> prefix(n, 0.f);
            fp_status rc = FP_OK;
            for (int i = 0; i < n && rc == FP_OK; ++i) {
                // an operator without a launch of its own (a layer inside a fused run, a layout conversion done by the
                // first run) adds nothing to the prefix
                const Op& op = h->ops[i];
                const bool silent = (op.kind == 0 && h->op_chain[i] >= 0 && h->chains[h->op_chain[i]].first_op != i) ||
                                    (op.kind == 3 && (h->input_fused || h->stem_fused)) || (h->stem_fused && i == 2) ||
                                    (op.kind == 0 && h->convs[op.idx].absorbed);
                if (silent) { prefix[i] = i ? prefix[i - 1] : 0.f; continue; }
                cudaGraph_t g = nullptr;
                cudaGraphExec_t ge = nullptr;
                if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { rc = fail(FP_ERR_CUDA, "fp_query: capture failed"); break; }
                for (int j = 0; j <= i; ++j) launch_op(h, j, h->last_input, h->last_batch, h->d_logits_stage, st);
                if (cudaStreamEndCapture(st, &g) != cudaSuccess || g == nullptr) { rc = fail(FP_ERR_CUDA, "fp_query: capture failed"); break; }
                size_t n_nodes = 0;
                cudaGraphGetNodes(g, nullptr, &n_nodes);
                if (n_nodes == 0) {                      // nothing launched yet (e.g. a layout conversion done inside the first run)
                    prefix[i] = i ? prefix[i - 1] : 0.f;
                    cudaGraphDestroy(g);
                    continue;
                }
                if (cudaGraphInstantiate(&ge, g, 0) != cudaSuccess) { cudaGraphDestroy(g); rc = fail(FP_ERR_CUDA, "fp_query: graph instantiate failed"); break; }
                for (int k = 0; k < 3; ++k) cudaGraphLaunch(ge, st);          // warm-up
                cudaEventRecord(e0, st);
                for (int k = 0; k < reps; ++k) cudaGraphLaunch(ge, st);
                cudaEventRecord(e1, st);
                cudaError_t e = cudaStreamSynchronize(st);
                float ms = 0.f;
                if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
                cudaGraphExecDestroy(ge);
                cudaGraphDestroy(g);
                if (e != cudaSuccess) { rc = fail(FP_ERR_CUDA, "fp_query: timing failed: %s", cudaGetErrorString(e)); break; }
                prefix[i] = ms / reps;
            }
            cudaEventDestroy(e0);
            cudaEventDestroy(e1);
            cudaStreamDestroy(st);
            cudaGetLastError();
            if (rc != FP_OK) return rc;
            for (int i = 0; i < n; ++i) {
                const float d = prefix[i] - (i ? prefix[i - 1] : 0.f);
                ((float*)h_out)[i] = d > 0.f ? d : 0.f;
            }
            return FP_OK;
        }
        default: return fail(FP_ERR_ARG, "fp_query: unknown query %d", what);
    }
}
