/*
 * fupruner - fused + pruned residual-network inference for NVIDIA B200 (sm_100a).
 *
 * C ABI.  The three main calls follow the paper's statement of the problem (Sec. IV-A:
 * given a pre-trained model, a fusion option and a pruning rate, produce the optimised
 * model; Algorithm 1: inputs W and p, output W*), and the inference that the paper times
 * on its devices (Sec. V-C):
 *
 *   fp_fuse     model description + weights + BN statistics  ->  equivalent fused graph
 *   fp_prune    per-layer ratios or masks                    ->  smaller fused graph
 *   fp_forward  input batch                                  ->  logits
 *
 * Conventions
 *   - Every call returns an fp_status, never throws, never exits the process.  On error the
 *     outputs are untouched and fp_last_error() holds a message (thread local).
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller owns every
 *     buffer it passes; the library copies what it keeps during fp_fuse.
 *   - Filter weights are fp32 in K,C,R,S order (the paper's k x c x r x s, Sec. IV-B.1);
 *     BN parameters are [gamma | beta | running mean | running variance], 4*K fp32 per BN.
 *   - Masks: 1 = keep, 0 = pruned.  Convolutions are numbered in the order their FP_CONV
 *     nodes appear in the description.
 *   - The library needs a B200 (compute capability 10.0); there is no CPU fallback.
 */
#ifndef FUPRUNER_H_
#define FUPRUNER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fp_handle_s* fp_handle;

typedef enum {
    FP_OK = 0,
    FP_ERR_ARG = -1,          /* NULL / out-of-range argument                                  */
    FP_ERR_DESC = -2,         /* description is not a supported residual-network pattern        */
    FP_ERR_SHAPE = -3,        /* inconsistent channel counts or spatial sizes                   */
    FP_ERR_NONFINITE = -4,    /* NaN/Inf in weights or BN statistics                            */
    FP_ERR_CUDA = -5,         /* a CUDA runtime/driver call failed (message has the CUDA error) */
    FP_ERR_NOMEM = -6,        /* device allocation failed                                       */
    FP_ERR_UNSUPPORTED = -7,  /* valid request the library cannot run (e.g. an aggressive block that is neither
                                 3x3-3x3 nor 1x1-3x3-1x1, an image wider than 512 pixels)            */
    FP_ERR_TIMEOUT = -8,      /* a bounded device-side wait ran out; results are invalid        */
    FP_ERR_EMPTY_LAYER = -9,  /* a mask or ratio would remove every filter of a convolution     */
    FP_ERR_BOUNDS = -10       /* batch larger than max_batch, size beyond a stated maximum      */
} fp_status;

/* ---- model description: flat node list in topological order ------------------------------- */

typedef enum {
    FP_CONV = 0,        /* in0 -> K x C x R x S convolution, stride, zero padding `pad`        */
    FP_BN = 1,          /* inference batch norm over K channels (Eq. 3-5)                        */
    FP_RELU = 2,
    FP_ADD = 3,         /* in0 = main branch (BN of the block's last conv), in1 = shortcut      */
    FP_SHORTCUT_A = 4,  /* parameter-free shortcut: spatial subsample by `stride`, C -> K channels
                           with `pad_lo` zero channels before and K-C-pad_lo after the copy     */
    FP_MAXPOOL = 5,     /* R x R window, stride, pad; padded positions never win                */
    FP_GAVGPOOL = 6,    /* mean over all spatial positions                                      */
    FP_FC = 7,          /* K x C matrix + K bias                                                */
    FP_CONCAT = 8       /* channel concatenation [in0 ; in1] of the concatenation structure of Sec. IV-B.1:
                           in0 = the BN (or ReLU) of a stride-1 "same" convolution with K - C filters, in1 =
                           that convolution's input with C channels.  Always fused: the convolution gets C
                           identity filters (the auxiliary convolution xconv-C) and no concatenation remains */
} fp_op;

typedef struct {
    int32_t op;                         /* fp_op                                                */
    int32_t in0, in1;                   /* producer node ids; -1 = network input                */
    int32_t K, C, R, S, stride, pad;    /* geometry (see fp_op)                                 */
    int32_t pad_lo;                     /* FP_SHORTCUT_A only                                   */
    int32_t block_id;                   /* residual building block this node belongs to, -1 none */
    int32_t aggressive;                 /* 1: fuse this block the paper's way (Sec. IV-B): identity
                                           filters stacked under conv1, shortcut filters stacked
                                           beside conv2, add removed.  0: the add becomes a residual
                                           operand of conv2's epilogue.                         */
    int32_t reserved;
    int64_t w_off;                      /* element offset into `weights` (CONV: KCRS, FC: KC), -1 none */
    int64_t b_off;                      /* element offset of the FC bias in `weights`, -1 none  */
    int64_t bn_off;                     /* element offset into `bn` of this BN's 4*K values     */
} fp_node;

enum { FP_DTYPE_F32 = 0, FP_DTYPE_BF16 = 1 };
enum { FP_COMPUTE_BF16_TC = 0,     /* BF16 tensor-core path, fp32 accumulation (the product)   */
       FP_COMPUTE_FP32 = 1,        /* plain fp32 CUDA-core path, for validation only            */
       FP_COMPUTE_BF16_SIMT = 2 }; /* BF16 storage, CUDA-core convolutions: validation only     */
enum { FP_NORM_L1 = 0,             /* sum of |w|                                                */
       FP_NORM_L2 = 1 };           /* sum of w^2 (Eq. 6 without its monotone square root)       */

typedef struct {
    int32_t n_nodes;
    const fp_node* nodes;               /* host                                                 */
    int32_t in_C, in_H, in_W;           /* network input is N x in_C x in_H x in_W (NCHW)       */
    int32_t in_dtype;                   /* FP_DTYPE_F32 or FP_DTYPE_BF16                        */
    int32_t compute;                    /* FP_COMPUTE_*                                         */
    float bn_eps;                       /* the epsilon of Eq. 4                                 */
    int32_t use_graph;                  /* 1: fp_forward replays a captured CUDA graph          */
    int32_t keep_outputs;               /* 1: every operator keeps its own output buffer (needed for
                                           FP_Q_OP_OUTPUT on any operator; default 0 reuses memory) */
    int32_t scatter;                    /* pruned convolutions that write a residual stream (their output is a shortcut
                                           operand, so the tensor keeps its full width): 0 = compute only the kept
                                           filters and scatter them into the full-width tensor where that pays (wide
                                           layers with a long reduction), zero filter rows elsewhere; 1 = scatter
                                           wherever it saves accumulator columns; -1 = always zero rows.  The
                                           result is the same in every case (Algorithm 1's removal of masked filters) */
} fp_model_desc;

/*
 * fp_fuse - build the equivalent fused graph (Sec. IV-B; BN merged as in the "*" models of
 * Table VI): fold every BN into its convolution on the device (fp32, fixed operation order
 * t=var+eps, r=sqrt(t), omega=gamma/r, W'=omega*W, lambda=beta-omega*mean), rewrite each
 * residual block as two convolutions with a fused bias/shortcut/ReLU epilogue or, where
 * `aggressive` is set, as the paper's dilated convolutions without an add, pack weights for
 * the tensor cores and plan activation memory for up to `max_batch` images.
 *   desc        host; copied.
 *   d_weights   device fp32, all CONV/FC weights at the w_off/b_off offsets; n_weights elements.
 *   d_bn        device fp32, all BN parameters at the bn_off offsets; n_bn elements.
 *   out         receives the handle; release with fp_destroy.
 * Errors: FP_ERR_ARG, FP_ERR_DESC, FP_ERR_SHAPE, FP_ERR_NONFINITE, FP_ERR_UNSUPPORTED,
 *         FP_ERR_NOMEM, FP_ERR_CUDA.  Synchronous (returns after the device work finished).
 */
fp_status fp_fuse(const fp_model_desc* desc, const float* d_weights, size_t n_weights,
                  const float* d_bn, size_t n_bn, int32_t max_batch, fp_handle* out);

/*
 * fp_fuse_with_allocator - fp_fuse with the caller's device allocator (Sec. IV-A's problem statement leaves memory
 * to the host framework): every device buffer of the handle - fused and packed filter banks, activations, scratch,
 * now and in later fp_prune / fp_soft_prune_finish / fp_query calls - is taken with alloc(bytes, user) and given
 * back with dealloc(ptr, user), e.g. a framework's caching allocator, so the library itself never calls cudaMalloc.
 *   alloc     returns a device pointer aligned to 256 bytes, or NULL (reported as FP_ERR_NOMEM); may be called from
 *             any thread that calls into the library; must stay valid until fp_destroy.
 *   dealloc   called once for every pointer alloc returned, at the latest in fp_destroy.
 * alloc == dealloc == NULL is fp_fuse.
 */
fp_status fp_fuse_with_allocator(const fp_model_desc* desc, const float* d_weights, size_t n_weights,
                                 const float* d_bn, size_t n_bn, int32_t max_batch,
                                 void* (*alloc)(size_t bytes, void* user), void (*dealloc)(void* ptr, void* user),
                                 void* user, fp_handle* out);

/*
 * fp_prune - filter pruning (Sec. IV-C, Algorithm 1 selection + final extraction).  Scores
 * every convolution's filters on the device on the fused, unpruned fp32 weights (Eq. 6 or
 * the l1 sum), ranks ascending by (score, filter index), masks the lowest q, then removes
 * masked filters and the matching input channels of their consumers and repacks.
 *   q = n - m for an aggressively fused operator (n filters now, m originally),
 *   q = floor(ratio * n + 1e-9) otherwise.
 *   h_ratios    host, one double per convolution, or NULL (= all 0).  Ignored where masks given.
 *   h_masks     host, array of n_convs pointers (entries may be NULL = use the ratio), each to K
 *               bytes (1 keep / 0 prune) for that convolution; or NULL.
 * Always starts from the unpruned fused weights, so ratios of 0 restore the unpruned model.
 * Errors: FP_ERR_ARG, FP_ERR_EMPTY_LAYER, FP_ERR_NOMEM, FP_ERR_CUDA.  Synchronous.
 * Arguments are checked, and every mask selected, before anything is changed: FP_ERR_ARG and
 * FP_ERR_EMPTY_LAYER leave the previous graph running.  A failure while the new graph is being built
 * (FP_ERR_NOMEM, FP_ERR_CUDA) leaves the handle without a graph: fp_forward then returns FP_ERR_ARG
 * until a later fp_prune succeeds.
 */
fp_status fp_prune(fp_handle h, int32_t norm, const double* h_ratios, const uint8_t* const* h_masks);

/*
 * fp_forward - run the fused (and pruned) network on `batch` images (the inference the paper
 * times, Sec. V-C).  Asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default
 * stream); performs no allocation and no host synchronisation.
 *   d_input     device, batch x in_C x in_H x in_W, NCHW, dtype as given in the description.
 *   d_logits    device fp32, batch x classes, row major.
 * Errors: FP_ERR_ARG, FP_ERR_BOUNDS (batch > max_batch), FP_ERR_CUDA.  A device-side wait that
 * ran out is reported by the next fp_query(FP_Q_DEVICE_STATUS) as FP_ERR_TIMEOUT.
 */
fp_status fp_forward(fp_handle h, const void* d_input, int32_t batch, float* d_logits, void* stream);

/* fp_forward_host - same, with HOST input and output buffers: copies the input to the device,
 * runs the network, copies the logits back and waits.  (The end-to-end call.) */
fp_status fp_forward_host(fp_handle h, const void* h_input, int32_t batch, float* h_logits, void* stream);

/* fp_forward_host_async - fp_forward_host without the wait: the input copy, the network and the copy of the logits are
 * queued and the call returns.  Where the graph starts with a kernel of its own that takes the input in (the ImageNet
 * networks), the input crosses the bus on a second stream - in pieces of at least 8 MB, each handed to that kernel as it
 * arrives - and waits only for the PREVIOUS call's first kernel, the one reader of the staging buffer: a caller who
 * queues the next call before this one has finished has the next input copied while this forward still runs.
 *   h_input     host (pinned for the copy to be asynchronous), same layout and type as fp_forward's d_input; must stay
 *               unchanged until the work queued by this call has finished.
 *   h_logits    host, batch x n_classes floats; valid once `stream` has been synchronised (or an event recorded on it
 *               after the call has completed).  Calls on one handle are ordered on `stream`.
 * Errors: as fp_forward.  Asynchronous on `stream` (and an internal copy stream). */
fp_status fp_forward_host_async(fp_handle h, const void* h_input, int32_t batch, float* h_logits, void* stream);

/*
 * fp_score - filter scores of one convolution of the fused, unpruned graph (Eq. 6 / l1),
 * computed on the device in fp64 with a fixed summation order: filter flattened in (c,r,s)
 * order, 32 partial sums over elements l, l+32, ..., combined pairwise at distances 16,8,4,2,1.
 *   h_scores    host, K doubles (K = fp_query FP_Q_CONV_K_FUSED).
 */
fp_status fp_score(fp_handle h, int32_t conv_index, int32_t norm, double* h_scores);

typedef enum {
    FP_Q_N_CONVS = 0,        /* int32: number of FP_CONV nodes in the description                */
    FP_Q_CONV_K_FUSED = 1,   /* int32: filters of conv `index` after fusion, before pruning (0 if the
                                conv was absorbed into another by aggressive fusion)             */
    FP_Q_CONV_K_KEPT = 2,    /* int32: filters kept by the last fp_prune                          */
    FP_Q_CONV_C_KEPT = 3,    /* int32: input channels left after its producers were pruned        */
    FP_Q_MASK = 4,           /* uint8[K_FUSED]                                                    */
    FP_Q_RANK = 5,           /* int32[K_FUSED]: position in ascending (score, index) order        */
    FP_Q_N_CLASSES = 6,      /* int32                                                             */
    FP_Q_FLOPS = 7,          /* double: 2*MACs per image of the current graph, unpadded kept sizes */
    FP_Q_BYTES = 8,          /* double[2]: algorithmic bytes of one forward = per image part, batch-
                                independent part (weights): each op reads inputs/residual, writes output once */
    FP_Q_N_OPS = 9,          /* int32: fused operators in execution order                         */
    FP_Q_OP_INFO = 10,       /* fp_op_info of fused operator `index`                              */
    FP_Q_OP_OUTPUT = 11,     /* float[batch*C*H*W] NCHW, logical channels: output of fused operator
                                `index` for the input of the last fp_forward (debug; synchronises the device).
                                Without keep_outputs the launches up to that operator are run again first (the
                                last input must still be alive), and a layer inside a fused run, whose output
                                never reaches memory, is refused with FP_ERR_UNSUPPORTED - the run's last
                                layer can be read */
    FP_Q_DEVICE_STATUS = 12, /* int32: 0, or FP_ERR_TIMEOUT if a bounded device wait ran out since the last query
                                (the flag is cleared by the query that reports it); synchronises with the device's
                                earlier work through the copy that reads it                             */
    FP_Q_N_LAUNCHES = 13,    /* int32: kernels one fp_forward launches                             */
    FP_Q_OP_TIMES = 14       /* float[N_OPS]: milliseconds per fused operator of a forward of the last batch size,
                                measured now as differences of the times of the forward's prefixes (launches 0..i
                                minus launches 0..i-1), each prefix replayed as a CUDA graph `index` times (0 = 10)
                                between two events; a layer inside a fused run reports 0 except the run's first;
                                synchronises */,
    FP_Q_CONV_BANK_ELEMS = 15 /* int64: weights in the fused fp32 bank of conv `index` (K_fused*C_fused*R*S), 0 if absorbed */
} fp_query_what;

typedef struct {
    int32_t kind;            /* 0 conv, 1 maxpool, 2 avgpool+fc head, 3 input layout conversion     */
    int32_t conv_index;      /* description conv number, -1 for non-conv operators                  */
    int32_t K, C, R, S, stride, pad;   /* kept (unpadded) sizes                                     */
    int32_t K_pad, C_pad;    /* sizes the kernel computes with                                      */
    int32_t H, W, P, Q;      /* input / output spatial size                                         */
    int32_t res_mode;        /* 0 none, 1 same-shape tensor, 2 subsample + zero-channel pad          */
    int32_t relu;
    double flops_per_image;  /* 2*MACs, unpadded                                                    */
    double bytes_per_image;  /* algorithmic activation bytes (in + residual + out)                   */
    double bytes_fixed;      /* weight + bias bytes                                                  */
    int32_t chain;           /* >= 0: the operator is a layer of fused run number `chain` (one kernel for the
                                whole run, activations in shared memory; FP_Q_OP_TIMES reports the run's time
                                at its first layer and 0 at the others); -1: launched on its own          */
    int32_t reserved;
} fp_op_info;

fp_status fp_query(fp_handle h, int32_t what, int32_t index, void* h_out, size_t bytes);

/*
 * fp_soft_prune_epoch - one pass of the loop body of Algorithm 1 (dynamic filter pruning, Sec. IV-C): the
 * fused fp32 filter banks are updated, every convolution's filters are scored on the updated weights (Eq. 6
 * or the l1 sum, same fixed summation order as fp_score), and the lowest n - m (fused operator) or
 * floor(ratio * n + 1e-9) filters are ZEROIZED in place - weights only; they stay in the bank, and the next
 * epoch's update can bring them back.  The masks of the epoch are kept (FP_Q_MASK / FP_Q_RANK); the graph
 * that fp_forward runs is NOT changed until fp_soft_prune_finish.
 *   d_updates   device fp32 or NULL.  Stands for "update the parameters W by using data X" (the library has no
 *               trainer): the concatenation, over the convolutions of the description in order (convolutions
 *               absorbed by aggressive fusion skipped), of one addend per weight of the fused bank,
 *               K_fused x C_fused x R x S each (FP_Q_CONV_BANK_ELEMS gives the count); W <- W + update, one
 *               fp32 addition per weight.
 *   h_ratios    host, one double per convolution, or NULL (= all 0); ignored for fused operators.
 * After the first epoch the banks no longer hold the original fused weights, so a later fp_prune scores the
 * updated, partly zeroized weights.
 * Errors: FP_ERR_ARG, FP_ERR_EMPTY_LAYER, FP_ERR_CUDA.  Synchronous.
 */
fp_status fp_soft_prune_epoch(fp_handle h, int32_t norm, const double* h_ratios, const float* d_updates);

/*
 * fp_soft_prune_finish - the last step of Algorithm 1: the pruned model is obtained from the updated weights
 * according to the masks of the last epoch: masked filters (and the matching input channels of their
 * consumers) are removed, filters repacked, activation memory and launch plans rebuilt, as fp_prune does.
 * Errors: FP_ERR_ARG (no epoch has run), FP_ERR_EMPTY_LAYER, FP_ERR_NOMEM, FP_ERR_CUDA.  Synchronous.
 */
fp_status fp_soft_prune_finish(fp_handle h);

/*
 * fp_rank_filters_static - score, rank and mask the filters of ONE filter bank without allocating.
 * (No counterpart in the paper: it is the selection step of fp_prune offered in a form for callers
 * that must not allocate.)
 *
 * Who needs it: code that runs where device allocation is off limits - a serving loop that has handed
 * all device memory to its own pool, a real-time path that cannot afford cudaMalloc's implicit
 * device synchronisation, a plug-in that is only given buffers.  fp_fuse/fp_prune allocate (packed
 * banks, score buffers); this call does not: it calls no cudaMalloc/cudaFree and no allocating
 * library routine.  Its one intermediate, an fp64 score per filter, lives in a fixed array inside the
 * library image (32 KB, present on every GPU that loads the library, until the process exits).
 *
 *   d_filters   device fp32, K filters of per_filter elements each, filter-major (a K x C x R x S bank).
 *   norm        FP_NORM_L1 or FP_NORM_L2; scores and order exactly as fp_score / fp_prune define them.
 *   q           number of filters to mask: the q lowest by (score, index) get mask 0.  0 <= q <= K.
 *   d_rank      device int32[K]  out: position of each filter in ascending (score, index) order.
 *   d_mask      device uint8[K]  out: 1 keep, 0 pruned.
 *   stream      cudaStream_t as void*, NULL = default stream.  Asynchronous.
 *
 * Limit: K <= FP_STATIC_RANK_MAX_FILTERS (4096); larger banks are rejected with FP_ERR_BOUNDS.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) and keeps it;
 * make that first call outside any stream capture.  All calls on a device share the array: two calls
 * whose kernels overlap on the GPU (different streams, no ordering between them) race on it - order
 * them.  The array keeps the previous call's scores; every call overwrites the part it reads, so
 * nothing needs clearing.
 * Errors: FP_ERR_ARG, FP_ERR_BOUNDS, FP_ERR_CUDA.
 */
#define FP_STATIC_RANK_MAX_FILTERS 4096
fp_status fp_rank_filters_static(const float* d_filters, int32_t K, int32_t per_filter, int32_t norm, int32_t q,
                                 int32_t* d_rank, uint8_t* d_mask, void* stream);

/*
 * fp_debug_expire_wait - diagnostic (no counterpart in the paper): makes one bounded device-side wait run out on
 * purpose, to show that the kernels' way out works.  Every wait inside the tensor-core kernels (for a bulk copy, for
 * the tensor cores, for the other warps) has a time limit; when one runs out the CTA raises the handle's status word,
 * all of its roles leave their loops, tensor memory is released and the kernel returns.  This call launches the first
 * stride-1 convolution of the graph that runs as a kernel of its own with the first round of its activation copies
 * left out and a limit of one millisecond, so exactly that happens; nothing faults and nothing hangs.  The
 * activations of the handle are garbage afterwards (run fp_forward again), and the next
 * fp_query(FP_Q_DEVICE_STATUS) reports FP_ERR_TIMEOUT, once.  Asynchronous on `stream`.
 * Errors: FP_ERR_ARG, FP_ERR_UNSUPPORTED (no such convolution in the graph), FP_ERR_CUDA.
 */
fp_status fp_debug_expire_wait(fp_handle h, void* stream);

fp_status fp_destroy(fp_handle h);

const char* fp_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FUPRUNER_H_ */
