"""Thin ctypes binding over the C-ABI library (include/fupruner.h).

Argument marshalling only: every step of fusing, pruning and running the network happens
inside the library's CUDA kernels.  PyTorch is used for device memory and streams.
The library is required - there is no fallback; a missing build raises ImportError here.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libfupruner.so")

FP_OK = 0
FP_ERR_ARG, FP_ERR_DESC, FP_ERR_SHAPE, FP_ERR_NONFINITE, FP_ERR_CUDA = -1, -2, -3, -4, -5
FP_ERR_NOMEM, FP_ERR_UNSUPPORTED, FP_ERR_TIMEOUT, FP_ERR_EMPTY_LAYER, FP_ERR_BOUNDS = -6, -7, -8, -9, -10
FP_DTYPE_F32, FP_DTYPE_BF16 = 0, 1
FP_COMPUTE_BF16_TC, FP_COMPUTE_FP32, FP_COMPUTE_BF16_SIMT = 0, 1, 2
FP_NORM_L1, FP_NORM_L2 = 0, 1
(FP_Q_N_CONVS, FP_Q_CONV_K_FUSED, FP_Q_CONV_K_KEPT, FP_Q_CONV_C_KEPT, FP_Q_MASK, FP_Q_RANK, FP_Q_N_CLASSES,
 FP_Q_FLOPS, FP_Q_BYTES, FP_Q_N_OPS, FP_Q_OP_INFO, FP_Q_OP_OUTPUT, FP_Q_DEVICE_STATUS, FP_Q_N_LAUNCHES,
 FP_Q_OP_TIMES, FP_Q_CONV_BANK_ELEMS) = range(16)

EXPORTS = ["fp_fuse", "fp_prune", "fp_forward", "fp_forward_host", "fp_forward_host_async", "fp_score", "fp_query", "fp_destroy",
           "fp_last_error", "fp_rank_filters_static", "fp_soft_prune_epoch", "fp_soft_prune_finish",
           "fp_debug_expire_wait", "fp_fuse_with_allocator"]
FP_STATIC_RANK_MAX_FILTERS = 4096


class fp_node(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("op", "in0", "in1", "K", "C", "R", "S", "stride", "pad", "pad_lo", "block_id", "aggressive",
                 "reserved")] + [("pad_", ctypes.c_int32)] + \
               [("w_off", ctypes.c_int64), ("b_off", ctypes.c_int64), ("bn_off", ctypes.c_int64)]


class fp_model_desc(ctypes.Structure):
    _fields_ = [("n_nodes", ctypes.c_int32), ("nodes", ctypes.POINTER(fp_node)),
                ("in_C", ctypes.c_int32), ("in_H", ctypes.c_int32), ("in_W", ctypes.c_int32),
                ("in_dtype", ctypes.c_int32), ("compute", ctypes.c_int32), ("bn_eps", ctypes.c_float),
                ("use_graph", ctypes.c_int32), ("keep_outputs", ctypes.c_int32), ("scatter", ctypes.c_int32)]


class fp_op_info(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("kind", "conv_index", "K", "C", "R", "S", "stride", "pad", "K_pad", "C_pad", "H", "W", "P", "Q",
                 "res_mode", "relu")] + \
               [("flops_per_image", ctypes.c_double), ("bytes_per_image", ctypes.c_double),
                ("bytes_fixed", ctypes.c_double), ("chain", ctypes.c_int32), ("reserved", ctypes.c_int32)]


ALLOC_FN = ctypes.CFUNCTYPE(ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p)
DEALLOC_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_void_p)


class TorchAllocator:
    """PyTorch's caching allocator as the library's device allocator (argument marshalling only: the two callbacks hand
    sizes and pointers through).  Keep the object alive as long as the handle."""

    def __init__(self):
        import torch
        self.n_alloc = self.n_free = 0
        self.live = {}

        def _alloc(nbytes, _user):
            try:
                ptr = torch.cuda.caching_allocator_alloc(int(nbytes))
            except Exception:
                return None
            self.n_alloc += 1
            self.live[ptr] = int(nbytes)
            return ptr

        def _free(ptr, _user):
            self.n_free += 1
            self.live.pop(ptr, None)
            torch.cuda.caching_allocator_delete(ptr)

        self.alloc, self.dealloc = ALLOC_FN(_alloc), DEALLOC_FN(_free)


class FpError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"fupruner status {status}: {message}")
        self.status = status


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2010_16165_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(_LIB_PATH)
        L.fp_last_error.restype = ctypes.c_char_p
        L.fp_fuse.argtypes = [ctypes.POINTER(fp_model_desc), ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p,
                              ctypes.c_size_t, ctypes.c_int32, ctypes.POINTER(ctypes.c_void_p)]
        L.fp_fuse_with_allocator.argtypes = [ctypes.POINTER(fp_model_desc), ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p,
                                             ctypes.c_size_t, ctypes.c_int32, ALLOC_FN, DEALLOC_FN, ctypes.c_void_p,
                                             ctypes.POINTER(ctypes.c_void_p)]
        L.fp_prune.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        L.fp_forward.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        L.fp_forward_host.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        L.fp_forward_host_async.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        L.fp_score.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
        L.fp_query.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t]
        L.fp_destroy.argtypes = [ctypes.c_void_p]
        L.fp_soft_prune_epoch.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        L.fp_soft_prune_finish.argtypes = [ctypes.c_void_p]
        L.fp_debug_expire_wait.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        L.fp_rank_filters_static.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                             ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib = L
    return _lib


def _check(status):
    if status != FP_OK:
        raise FpError(status, lib().fp_last_error().decode())


def make_nodes(node_dicts):
    arr = (fp_node * len(node_dicts))()
    for a, n in zip(arr, node_dicts):
        for k in ("op", "in0", "in1", "K", "C", "R", "S", "stride", "pad", "pad_lo", "block_id", "aggressive",
                  "w_off", "b_off", "bn_off"):
            setattr(a, k, int(n[k]))
    return arr


def fp_fuse(net, d_weights, d_bn, max_batch, compute=FP_COMPUTE_BF16_TC, in_dtype=FP_DTYPE_F32, use_graph=0,
            keep_outputs=0, scatter=0, allocator=None):
    """net: workloads.Net; d_weights/d_bn: CUDA float32 torch tensors; allocator: None (the library uses cudaMalloc) or an
    object with ctypes callbacks `alloc` / `dealloc` (TorchAllocator).  Returns an opaque handle."""
    nodes = make_nodes(net.nodes)
    desc = fp_model_desc(len(net.nodes), nodes, net.in_C, net.in_H, net.in_W, in_dtype, compute,
                         float(net.bn_eps), use_graph, keep_outputs, scatter)
    h = ctypes.c_void_p()
    if allocator is None:
        _check(lib().fp_fuse(ctypes.byref(desc), d_weights.data_ptr(), d_weights.numel(), d_bn.data_ptr(),
                             d_bn.numel(), max_batch, ctypes.byref(h)))
    else:
        _check(lib().fp_fuse_with_allocator(ctypes.byref(desc), d_weights.data_ptr(), d_weights.numel(), d_bn.data_ptr(),
                                            d_bn.numel(), max_batch, allocator.alloc, allocator.dealloc, None, ctypes.byref(h)))
    return h


def fp_prune(h, ratios=None, masks=None, norm=FP_NORM_L1):
    """ratios: sequence of one float per convolution, or None.  masks: dict/list conv -> uint8 array, or None."""
    r = None
    if ratios is not None:
        r = np.ascontiguousarray(ratios, dtype=np.float64)
    mptr = None
    keep = []
    if masks is not None:
        n = fp_query_int(h, FP_Q_N_CONVS)
        mptr = (ctypes.c_void_p * n)()
        for ci in range(n):
            m = masks.get(ci) if isinstance(masks, dict) else masks[ci]
            if m is None:
                mptr[ci] = None
            else:
                m = np.ascontiguousarray(m, dtype=np.uint8)
                keep.append(m)
                mptr[ci] = m.ctypes.data
    _check(lib().fp_prune(h, norm, r.ctypes.data if r is not None else None, mptr))


def fp_forward(h, d_input, batch, d_logits, stream=None):
    """d_input / d_logits: CUDA torch tensors; stream: torch.cuda.Stream or None (default stream)."""
    _check(lib().fp_forward(h, d_input.data_ptr(), batch, d_logits.data_ptr(),
                            stream.cuda_stream if stream is not None else None))


def fp_forward_host(h, h_input, batch, h_logits, stream=None):
    """h_input / h_logits: host buffers (numpy arrays or pinned CPU torch tensors)."""
    pin = h_input.ctypes.data if isinstance(h_input, np.ndarray) else h_input.data_ptr()
    pout = h_logits.ctypes.data if isinstance(h_logits, np.ndarray) else h_logits.data_ptr()
    _check(lib().fp_forward_host(h, pin, batch, pout, stream.cuda_stream if stream is not None else None))


def fp_forward_host_async(h, h_input, batch, h_logits, stream=None):
    """fp_forward_host without the wait: h_logits is valid once `stream` has been synchronised."""
    pin = h_input.ctypes.data if isinstance(h_input, np.ndarray) else h_input.data_ptr()
    pout = h_logits.ctypes.data if isinstance(h_logits, np.ndarray) else h_logits.data_ptr()
    _check(lib().fp_forward_host_async(h, pin, batch, pout, stream.cuda_stream if stream is not None else None))


def fp_score(h, conv_index, norm=FP_NORM_L1):
    K = fp_query_int(h, FP_Q_CONV_K_FUSED, conv_index)
    out = np.empty(K, dtype=np.float64)
    _check(lib().fp_score(h, conv_index, norm, out.ctypes.data))
    return out


def fp_query_int(h, what, index=0):
    v = ctypes.c_int32()
    _check(lib().fp_query(h, what, index, ctypes.byref(v), 4))
    return v.value


def fp_query_array(h, what, index, dtype, count):
    out = np.empty(count, dtype=dtype)
    _check(lib().fp_query(h, what, index, out.ctypes.data, out.nbytes))
    return out


def fp_query_op(h, index):
    o = fp_op_info()
    _check(lib().fp_query(h, FP_Q_OP_INFO, index, ctypes.byref(o), ctypes.sizeof(o)))
    return o


def fp_rank_filters_static(d_filters, K, per_filter, norm, q, d_rank, d_mask, stream=None):
    """Allocation-free selection for one bank: d_filters fp32 CUDA tensor (K*per_filter), d_rank int32[K] and
    d_mask uint8[K] CUDA tensors provided by the caller.  Asynchronous on `stream`."""
    _check(lib().fp_rank_filters_static(d_filters.data_ptr(), K, per_filter, norm, q, d_rank.data_ptr(),
                                        d_mask.data_ptr(), stream.cuda_stream if stream is not None else None))


def fp_soft_prune_epoch(h, ratios=None, d_updates=None, norm=FP_NORM_L2):
    """One pass of Algorithm 1's loop body.  d_updates: CUDA float32 tensor (concatenated addends of all fused
    banks, see conv_bank_elems) or None."""
    r = np.ascontiguousarray(ratios, dtype=np.float64) if ratios is not None else None
    _check(lib().fp_soft_prune_epoch(h, norm, r.ctypes.data if r is not None else None,
                                     d_updates.data_ptr() if d_updates is not None else None))


def fp_soft_prune_finish(h):
    _check(lib().fp_soft_prune_finish(h))


def fp_debug_expire_wait(h, stream=None):
    """Diagnostic: lets one bounded device-side wait run out (see the header); the next FP_Q_DEVICE_STATUS reports it."""
    _check(lib().fp_debug_expire_wait(h, stream.cuda_stream if stream is not None else None))


def conv_bank_elems(h):
    """Weights in the fused fp32 bank of every convolution of the description (0 where absorbed)."""
    out = []
    for ci in range(fp_query_int(h, FP_Q_N_CONVS)):
        v = ctypes.c_int64()
        _check(lib().fp_query(h, FP_Q_CONV_BANK_ELEMS, ci, ctypes.byref(v), 8))
        out.append(int(v.value))
    return out


def fp_destroy(h):
    _check(lib().fp_destroy(h))


def masks_and_ranks(h):
    out = {}
    for ci in range(fp_query_int(h, FP_Q_N_CONVS)):
        K = fp_query_int(h, FP_Q_CONV_K_FUSED, ci)
        if K == 0:
            out[ci] = (None, None)
            continue
        out[ci] = (fp_query_array(h, FP_Q_MASK, ci, np.uint8, K), fp_query_array(h, FP_Q_RANK, ci, np.int32, K))
    return out


def op_infos(h):
    return [fp_query_op(h, i) for i in range(fp_query_int(h, FP_Q_N_OPS))]
