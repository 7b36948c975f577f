"""CPU oracle for fused + pruned residual-network inference (fp64).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It shares no code with the CUDA library and
never touches a GPU.  The heavy loops live in ``fpo.c`` (plain C, fp64,
NCHW/KCRS); this file holds the graph logic, written with numpy.

What is defined here, and where the paper states it:

* ``unfused_forward``  - the network exactly as described by the node list:
  conv, batch norm (textbook inference form), ReLU, add, shortcut, pooling, FC.
  This is the plain definition of the result; the paper's fusion is an
  equivalence transformation (Sec. IV-C, first paragraph), so every fused or
  fused-and-unpruned graph must reproduce it.
* ``fuse``  - BN as the affine map of Eq. 3-5 merged into the preceding
  convolution (the "*" models of Table VI), and per building block either the
  element-wise add kept as a residual operand of the second convolution
  ("epilogue" form) or the paper's aggressive fusion (Sec. IV-B): an identity
  convolution xconv-C stacked under conv1 along K, an xconv-F / padded pconv-F
  stacked beside conv2 along C, the add removed.
* ``scores`` / ``rank_mask``  - Eq. 6 and the selection rule of Algorithm 1
  (zero the lowest n-m filters of a fused operator, the lowest p*n of the others).
* ``prune_remove`` / ``prune_zero``  - the final extraction step of Algorithm 1
  (masked filters are removed), realised both by physically removing filters and
  the matching consumer channels and by zeroing them.

Parity status: every function below is pinned by tests/test_oracle_*.py (brute-force
convolution, library convolution as a special case, closed forms, the equivalence
invariants the paper states).  End-to-end activations have no printed values in the
paper; they are pinned only through those invariants.  The accuracy tables of the
paper are out of reach (datasets, training): parity unpinned for them, not computed here.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

OP_CONV, OP_BN, OP_RELU, OP_ADD, OP_SHORTCUT_A, OP_MAXPOOL, OP_GAVGPOOL, OP_FC, OP_CONCAT = range(9)

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None
_dp = ctypes.POINTER(ctypes.c_double)
_fp = ctypes.POINTER(ctypes.c_float)


def build(force=False):
    """Compile fpo.c into libfpo.so next to it (gcc, -O2, OpenMP, no fp contraction)."""
    src = os.path.join(_HERE, "fpo.c")
    out = os.path.join(_HERE, "libfpo.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
                               src, "-o", out, "-lm"])
    return out


def lib():
    global _LIB
    if _LIB is None:
        _LIB = ctypes.CDLL(build())
        _LIB.fpo_score_filter.restype = ctypes.c_double
        _LIB.fpo_num_threads.restype = ctypes.c_int
    return _LIB


def num_threads():
    return int(lib().fpo_num_threads())


def _d(a):
    return a.ctypes.data_as(_dp)


def _f(a):
    return a.ctypes.data_as(_fp)


def _c64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


# ------------------------------------------------------------------------------------
# operators (thin wrappers over the C loops)
# ------------------------------------------------------------------------------------

def conv2d(x, w, stride=1, pad=0):
    x, w = _c64(x), _c64(w)
    N, C, H, W = x.shape
    K, C2, R, S = w.shape
    assert C == C2, (x.shape, w.shape)
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    y = np.empty((N, K, P, Q), dtype=np.float64)
    if K == 0 or N == 0:
        return y
    if C == 0:
        y[:] = 0.0
        return y
    lib().fpo_conv2d(_d(x), _d(w), _d(y), N, C, H, W, K, R, S, stride, pad)
    return y


def batchnorm(x, gamma, beta, mean, var, eps):
    x = _c64(x)
    N, C = x.shape[:2]
    y = np.empty_like(x)
    lib().fpo_bn(_d(x), _d(y), N, C, int(np.prod(x.shape[2:])), _d(_c64(gamma)), _d(_c64(beta)),
                 _d(_c64(mean)), _d(_c64(var)), ctypes.c_double(eps))
    return y


def add_bias(y, b):
    y = _c64(y)
    N, C = y.shape[:2]
    if y.size:
        lib().fpo_bias(_d(y), N, C, int(np.prod(y.shape[2:])), _d(_c64(b)))
    return y


def relu(x):
    x = _c64(x)
    y = np.empty_like(x)
    lib().fpo_relu(_d(x), _d(y), ctypes.c_size_t(x.size))
    return y


def add(a, b):
    a, b = _c64(a), _c64(b)
    assert a.shape == b.shape, (a.shape, b.shape)
    y = np.empty_like(a)
    lib().fpo_add(_d(a), _d(b), _d(y), ctypes.c_size_t(a.size))
    return y


def shortcut_a(x, K, stride, pad_lo=0):
    x = _c64(x)
    N, C, H, W = x.shape
    P, Q = (H + stride - 1) // stride, (W + stride - 1) // stride
    y = np.empty((N, K, P, Q), dtype=np.float64)
    lib().fpo_shortcut_a(_d(x), _d(y), N, C, H, W, K, stride, pad_lo)
    return y


def maxpool(x, R=3, stride=2, pad=1):
    x = _c64(x)
    N, C, H, W = x.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - R) // stride + 1
    y = np.empty((N, C, P, Q), dtype=np.float64)
    if x.size:
        lib().fpo_maxpool(_d(x), _d(y), N, C, H, W, R, stride, pad)
    return y


def gavgpool(x):
    x = _c64(x)
    N, C = x.shape[:2]
    y = np.empty((N, C), dtype=np.float64)
    lib().fpo_gavgpool(_d(x), _d(y), N, C, int(np.prod(x.shape[2:])))
    return y


def fc(x, w, b=None):
    x, w = _c64(x), _c64(w)
    N, C = x.shape
    K = w.shape[0]
    y = np.empty((N, K), dtype=np.float64)
    bb = _c64(b) if b is not None else None
    lib().fpo_fc(_d(x), _d(w), _d(bb) if bb is not None else None, _d(y), N, C, K)
    return y


# ------------------------------------------------------------------------------------
# the network as described: node-by-node evaluation
# ------------------------------------------------------------------------------------

def _conv_w(n, weights):
    cnt = n["K"] * n["C"] * n["R"] * n["S"]
    return weights[n["w_off"]:n["w_off"] + cnt].reshape(n["K"], n["C"], n["R"], n["S"])


def _bn_params(n, bn):
    K, o = n["K"], n["bn_off"]
    return bn[o:o + K], bn[o + K:o + 2 * K], bn[o + 2 * K:o + 3 * K], bn[o + 3 * K:o + 4 * K]


def unfused_forward(net, weights, bn, x, return_all=False):
    """Evaluate the descriptor node by node in fp64.  x: (N,C,H,W).  Returns logits (N,classes)."""
    weights = np.asarray(weights, dtype=np.float64)
    bn = np.asarray(bn, dtype=np.float64)
    vals = {-1: _c64(x)}
    for i, n in enumerate(net.nodes):
        a = vals[n["in0"]]
        op = n["op"]
        if op == OP_CONV:
            v = conv2d(a, _conv_w(n, weights), n["stride"], n["pad"])
        elif op == OP_BN:
            g, b, m, s2 = _bn_params(n, bn)
            v = batchnorm(a, g, b, m, s2, net.bn_eps)
        elif op == OP_RELU:
            v = relu(a)
        elif op == OP_ADD:
            v = add(a, vals[n["in1"]])
        elif op == OP_CONCAT:
            v = np.concatenate([a, vals[n["in1"]]], axis=1)
        elif op == OP_SHORTCUT_A:
            v = shortcut_a(a, n["K"], n["stride"], n["pad_lo"])
        elif op == OP_MAXPOOL:
            v = maxpool(a, n["R"], n["stride"], n["pad"])
        elif op == OP_GAVGPOOL:
            v = gavgpool(a)
        elif op == OP_FC:
            w = weights[n["w_off"]:n["w_off"] + n["K"] * n["C"]].reshape(n["K"], n["C"])
            b = weights[n["b_off"]:n["b_off"] + n["K"]] if n["b_off"] >= 0 else None
            v = fc(a, w, b)
        else:
            raise ValueError(f"unknown op {op}")
        vals[i] = v
    return vals if return_all else vals[len(net.nodes) - 1]


# ------------------------------------------------------------------------------------
# BN folding (Eq. 3-5) in two precisions
# ------------------------------------------------------------------------------------

def fold64(w, gamma, beta, mean, var, eps):
    """omega = gamma/sqrt(var+eps), lambda = beta - omega*mean; W' = omega*W (per filter), fp64."""
    omega = np.asarray(gamma, np.float64) / np.sqrt(np.asarray(var, np.float64) + eps)
    lam = np.asarray(beta, np.float64) - omega * np.asarray(mean, np.float64)
    return np.asarray(w, np.float64) * omega[:, None, None, None], lam, omega


def fold32(w, gamma, beta, mean, var, eps):
    """Same map in fp32 with the fixed operation order that filter scoring is defined on."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    K = w.shape[0]
    per = int(np.prod(w.shape[1:]))
    g, b, m, v = (np.ascontiguousarray(t, dtype=np.float32) for t in (gamma, beta, mean, var))
    wo = np.empty_like(w)
    bo = np.empty(K, dtype=np.float32)
    om = np.empty(K, dtype=np.float32)
    lib().fpo_fold_bn_f32(_f(w), K, per, _f(g), _f(b), _f(m), _f(v), ctypes.c_float(eps), _f(wo), _f(bo), _f(om))
    return wo, bo, om


# ------------------------------------------------------------------------------------
# fusion: descriptor -> list of fused operators
# ------------------------------------------------------------------------------------

class FusedGraph:
    """ops: list of dicts.  Tensor ids: 0 = network input, op['out'] = id of its result.

    conv op:  src, W (K,C,R,S), b (K), stride, pad, relu, res (None or dict(mode, tid, pad_lo, stride)),
              conv (index among the descriptor's CONV nodes), n_orig (filter count of the original
              operator: Algorithm 1's m), role ('plain' | 'aggr1' | 'aggr2'), absorbed (conv indices
              merged into this one), K_full and scatter (set by prune_remove for stream writers)
    pool op:  src, R, stride, pad
    head op:  src, Wfc (classes,C), bfc      (global average pool + FC)
    """

    def __init__(self):
        self.ops = []
        self.n_convs = 0
        self.conv_op = {}     # descriptor conv index -> op (absent if absorbed)
        self.absorbed = {}    # descriptor conv index -> conv index it was merged into

    def consumers(self, tid):
        out = []
        for op in self.ops:
            if op.get("src") == tid:
                out.append((op, "main"))
            if op["kind"] == "conv" and op["res"] is not None and op["res"]["tid"] == tid:
                out.append((op, "res"))
        return out


def _consumer_map(net):
    cons = {i: [] for i in range(-1, len(net.nodes))}
    for i, n in enumerate(net.nodes):
        cons[n["in0"]].append(i)
        if n["op"] in (OP_ADD, OP_CONCAT):
            cons[n["in1"]].append(i)
    return cons


def _identity_filters(K, C, R, S, shift=0, dtype=np.float64):
    """W~[k][c] centre tap = 1 where c == k - shift: the auxiliary identity convolution (Sec. IV-B.1)."""
    w = np.zeros((K, C, R, S), dtype=dtype)
    for k in range(K):
        c = k - shift
        if 0 <= c < C:
            w[k, c, R // 2, S // 2] = 1.0
    return w


def _pad_to(w, R, S):
    """pconv: zero-pad a filter bank to a larger R x S footprint, original taps centred (Sec. IV-B.1)."""
    K, C, r, s = w.shape
    out = np.zeros((K, C, R, S), dtype=w.dtype)
    r0, s0 = (R - r) // 2, (S - s) // 2
    out[:, :, r0:r0 + r, s0:s0 + s] = w
    return out


def fuse(net, weights, bn, precision="f64"):
    """Build the fused operator list.  precision 'f64': exact-as-possible fold from the raw parameters
    (used for activations); 'f32': the fixed-order single-precision fold that scores are defined on."""
    if precision == "f64":
        fold, dt = fold64, np.float64
        weights_t, bn_t = np.asarray(weights, np.float64), np.asarray(bn, np.float64)
    else:
        fold, dt = fold32, np.float32
        weights_t, bn_t = np.asarray(weights, np.float32), np.asarray(bn, np.float32)
    eps = net.bn_eps
    cons = _consumer_map(net)
    nodes = net.nodes
    conv_index = {nid: ci for ci, nid in enumerate(net.conv_ids())}
    g = FusedGraph()
    g.n_convs = len(conv_index)
    tensor_of = {-1: 0}     # node id -> tensor id once materialised
    producer = {}           # tensor id -> op
    next_tid = [1]

    def new_tid():
        next_tid[0] += 1
        return next_tid[0] - 1

    def folded(conv_id):
        n = nodes[conv_id]
        (bn_id,) = cons[conv_id]
        assert nodes[bn_id]["op"] == OP_BN, "every convolution must be followed by batch norm"
        gm, bt, mu, var = _bn_params(nodes[bn_id], bn_t)
        W, b, omega = fold(_conv_w(n, weights_t), gm, bt, mu, var, eps)
        return W, b, bn_id

    def emit_conv(conv_id, W, b, src_tid, relu_flag, res, role="plain", n_orig=None, absorbed=()):
        n = nodes[conv_id]
        op = dict(kind="conv", src=src_tid, W=W, b=b, stride=n["stride"], pad=n["pad"], relu=relu_flag,
                  res=res, conv=conv_index[conv_id], n_orig=n["K"] if n_orig is None else n_orig,
                  role=role, absorbed=[conv_index[a] for a in absorbed], out=new_tid(),
                  K_full=W.shape[0], scatter=None)
        g.ops.append(op)
        g.conv_op[op["conv"]] = op
        for a in absorbed:
            g.absorbed[conv_index[a]] = op["conv"]
        producer[op["out"]] = op
        return op

    for i, n in enumerate(nodes):
        op = n["op"]
        if op == OP_CONV:
            W, b, bn_id = folded(i)
            nxt = cons[bn_id]
            # the concatenation structure (Sec. IV-B.1): y = concat(conv(x), x) becomes one convolution with the
            # identity filters of xconv-C stacked under W: y = new_conv(x, [W ; I])
            last = nxt[0] if (len(nxt) == 1 and nodes[nxt[0]]["op"] == OP_RELU) else bn_id
            cc = cons[last]
            if len(cc) == 1 and nodes[cc[0]]["op"] == OP_CONCAT and nodes[cc[0]]["in0"] == last \
                    and nodes[cc[0]]["in1"] == n["in0"]:
                K, C, R, S = W.shape
                if n["stride"] != 1 or R != S or R % 2 == 0 or n["pad"] != R // 2:
                    raise ValueError("the concatenation structure needs a stride-1 'same' convolution")
                relu_flag = last != bn_id
                xp = producer.get(tensor_of[n["in0"]])
                if relu_flag and (xp is None or (xp["kind"] == "conv" and not xp["relu"])):
                    raise ValueError("fusing concat(relu(conv(x)), x) needs x to be a ReLU output")
                Wc = np.concatenate([W, _identity_filters(C, C, R, S, 0, dt)], axis=0)
                bc = np.concatenate([b, np.zeros(C, dtype=dt)])
                o = emit_conv(i, Wc, bc, tensor_of[n["in0"]], relu_flag, None, role="aggr1", n_orig=K)
                tensor_of[cc[0]] = o["out"]
            elif len(nxt) == 1 and nodes[nxt[0]]["op"] == OP_RELU:
                o = emit_conv(i, W, b, tensor_of[n["in0"]], True, None)
                tensor_of[nxt[0]] = o["out"]
            elif len(nxt) == 1 and nodes[nxt[0]]["op"] == OP_ADD:
                pass  # handled when the add is reached
            else:
                o = emit_conv(i, W, b, tensor_of[n["in0"]], False, None)
                tensor_of[bn_id] = o["out"]
        elif op == OP_ADD:
            (relu_id,) = cons[i]
            assert nodes[relu_id]["op"] == OP_RELU
            main_bn = n["in0"]
            conv2_id = nodes[main_bn]["in0"]
            assert nodes[main_bn]["op"] == OP_BN and nodes[conv2_id]["op"] == OP_CONV
            W2, b2, _ = folded(conv2_id)
            sc = nodes[n["in1"]] if n["in1"] >= 0 else None
            # classify the shortcut operand
            if n["in1"] in tensor_of:
                mode, x_node = "id", n["in1"]
            elif sc["op"] == OP_SHORTCUT_A:
                mode, x_node = "A", sc["in0"]
            else:
                assert sc["op"] == OP_BN and nodes[sc["in0"]]["op"] == OP_CONV
                mode, x_node = "proj", nodes[sc["in0"]]["in0"]
            x_tid = tensor_of[x_node]
            h_tid = tensor_of[nodes[conv2_id]["in0"]]
            if not n["aggressive"]:
                if mode == "id":
                    res = dict(mode="id", tid=x_tid, pad_lo=0, stride=1)
                elif mode == "A":
                    res = dict(mode="A", tid=x_tid, pad_lo=sc["pad_lo"], stride=sc["stride"])
                else:
                    ps = sc["in0"]
                    Ws, bs, _ = folded(ps)
                    po = emit_conv(ps, Ws, bs, x_tid, False, None)
                    res = dict(mode="id", tid=po["out"], pad_lo=0, stride=1)
                o = emit_conv(conv2_id, W2, b2, h_tid, True, res)
            else:
                # ---- aggressive fusion of the block (Sec. IV-B) ---------------------------
                f1 = producer[h_tid]
                n2 = nodes[conv2_id]
                fa = producer.get(f1["src"]) if f1["kind"] == "conv" else None
                if (fa is not None and fa["kind"] == "conv" and fa["src"] == x_tid and n2["R"] == 1 and n2["S"] == 1):
                    # ---- bottleneck block (not in the paper, which stops at basic blocks): the block input is
                    #      carried through all three convolutions.  conv1'' = [W1 ; I] (1x1), conv2'' = diag(W2, I at
                    #      the centre tap) so that the pass-through is subsampled with conv2's stride, conv3'' =
                    #      [W3 | S] with S the identity or the projection's 1x1 filters; no add remains. ----
                    fb = f1                                               # the 3x3 convolution
                    if not (fa["relu"] and fb["relu"] and fa["res"] is None and fb["res"] is None
                            and fa["W"].shape[2:] == (1, 1) and fa["stride"] == 1 and fa["pad"] == 0
                            and fb["W"].shape[2:] == (3, 3) and fb["pad"] == 1
                            and n2["stride"] == 1 and n2["pad"] == 0 and mode in ("id", "proj")):
                        raise ValueError("aggressive fusion of a three-convolution block needs 1x1 - 3x3 - 1x1")
                    xp = producer.get(x_tid)
                    if xp is None or (xp["kind"] == "conv" and not xp["relu"]):
                        raise ValueError("aggressive fusion needs a block input that is a ReLU output")
                    Kw, C = fa["W"].shape[0], fa["W"].shape[1]
                    K3 = W2.shape[0]
                    fa["W"] = np.concatenate([fa["W"], _identity_filters(C, C, 1, 1, 0, dt)], axis=0)
                    fa["b"] = np.concatenate([fa["b"], np.zeros(C, dtype=dt)])
                    fa["role"], fa["K_full"] = "aggr1", Kw + C
                    Wd = np.zeros((Kw + C, Kw + C, 3, 3), dtype=dt)
                    Wd[:Kw, :Kw] = fb["W"]
                    Wd[Kw:, Kw:] = _identity_filters(C, C, 3, 3, 0, dt)
                    fb["W"] = Wd
                    fb["b"] = np.concatenate([fb["b"], np.zeros(C, dtype=dt)])
                    fb["role"], fb["K_full"] = "aggr1", Kw + C
                    absorbed = ()
                    if mode == "id":
                        Sw, bsum = _identity_filters(K3, C, 1, 1, 0, dt), b2
                    else:
                        ps = sc["in0"]
                        Ws, bs, _ = folded(ps)
                        if nodes[ps]["stride"] != fb["stride"] or nodes[ps]["pad"] != 0 or Ws.shape[2:] != (1, 1):
                            raise ValueError("projection shortcut must be 1x1 with the 3x3 convolution's stride")
                        Sw, bsum, absorbed = Ws, (b2 + bs).astype(dt), (ps,)
                    o = emit_conv(conv2_id, np.concatenate([W2, Sw], axis=1), bsum, h_tid, True, None, role="aggr2",
                                  absorbed=absorbed)
                    tensor_of[relu_id] = o["out"]
                    continue
                if not (f1["kind"] == "conv" and f1["src"] == x_tid and f1["relu"] and f1["res"] is None
                        and f1["W"].shape[2:] == (3, 3) and f1["pad"] == 1
                        and n2["R"] == 3 and n2["S"] == 3 and n2["stride"] == 1 and n2["pad"] == 1):
                    raise ValueError("aggressive fusion needs a two-convolution 3x3 block")
                xp = producer.get(x_tid)
                if xp is None or (xp["kind"] == "conv" and not xp["relu"]):
                    raise ValueError("aggressive fusion needs a block input that is a ReLU output")
                K1, C = f1["W"].shape[0], f1["W"].shape[1]
                K2 = W2.shape[0]
                # xconv-C: identity filters under conv1, unit BN scale and zero shift for them
                f1["W"] = np.concatenate([f1["W"], _identity_filters(C, C, 3, 3, 0, dt)], axis=0)
                f1["b"] = np.concatenate([f1["b"], np.zeros(C, dtype=dt)])
                f1["role"], f1["K_full"] = "aggr1", K1 + C
                absorbed = ()
                if mode == "id":
                    Sw = _identity_filters(K2, C, 3, 3, 0, dt)            # xconv-F
                    bsum = b2
                elif mode == "A":
                    if sc["stride"] != f1["stride"]:
                        raise ValueError("shortcut stride differs from conv1 stride")
                    Sw = _identity_filters(K2, C, 3, 3, sc["pad_lo"], dt)  # padded identity
                    bsum = b2
                else:
                    ps = sc["in0"]
                    Ws, bs, _ = folded(ps)
                    if nodes[ps]["stride"] != f1["stride"] or nodes[ps]["pad"] != 0 or Ws.shape[2:] != (1, 1):
                        raise ValueError("projection shortcut must be 1x1 with conv1's stride")
                    Sw = _pad_to(Ws, 3, 3)                                 # pconv-F
                    bsum = (b2 + bs).astype(dt)
                    absorbed = (ps,)
                W2f = np.concatenate([W2, Sw], axis=1)
                o = emit_conv(conv2_id, W2f, bsum, h_tid, True, None, role="aggr2", absorbed=absorbed)
            tensor_of[relu_id] = o["out"]
        elif op == OP_MAXPOOL:
            o = dict(kind="pool", src=tensor_of[n["in0"]], R=n["R"], stride=n["stride"], pad=n["pad"],
                     out=new_tid())
            g.ops.append(o)
            producer[o["out"]] = o
            tensor_of[i] = o["out"]
        elif op == OP_GAVGPOOL:
            (fc_id,) = cons[i]
            f = nodes[fc_id]
            assert f["op"] == OP_FC
            Wfc = weights_t[f["w_off"]:f["w_off"] + f["K"] * f["C"]].reshape(f["K"], f["C"]).astype(dt)
            bfc = weights_t[f["b_off"]:f["b_off"] + f["K"]].astype(dt) if f["b_off"] >= 0 else np.zeros(f["K"], dt)
            o = dict(kind="head", src=tensor_of[n["in0"]], Wfc=Wfc, bfc=bfc, out=new_tid())
            g.ops.append(o)
            producer[o["out"]] = o
        elif op in (OP_BN, OP_RELU, OP_SHORTCUT_A, OP_FC, OP_CONCAT):
            pass  # consumed by the patterns above
        else:
            raise ValueError(f"unknown op {op}")
    return g


def aggressive_block_paper_order(x, W1, bn1, W2, bn2, eps, stride=1, shift=0):
    """One basic block evaluated the way Sec. IV-B.2 orders it, with BN kept as an operator:
    conv1 and the identity xconv-C stacked along K; the 'new bn' = bn1 extended by an auxiliary
    BN with unit scale and zero shift on the pass-through channels; ReLU; conv2 and xconv-F
    stacked along C with the xconv-F taps divided by bn2's scale (the inverse of bn2 applied
    to the identity weights); bn2 unchanged; ReLU.  No add operator.  bn1/bn2 = (gamma, beta,
    mean, var).  shift > 0 gives the zero-channel-padded identity of a downsampling shortcut."""
    K1, C = W1.shape[0], W1.shape[1]
    K2 = W2.shape[0]
    Wa = np.concatenate([np.asarray(W1, np.float64), _identity_filters(C, C, 3, 3)], axis=0)
    g1, b1, m1, v1 = (np.asarray(t, np.float64) for t in bn1)
    new_bn = (np.concatenate([g1, np.ones(C)]), np.concatenate([b1, np.zeros(C)]),
              np.concatenate([m1, np.zeros(C)]), np.concatenate([v1, np.full(C, 1.0 - eps)]))
    h = relu(batchnorm(conv2d(x, Wa, stride, 1), *new_bn, eps))
    g2, b2, m2, v2 = (np.asarray(t, np.float64) for t in bn2)
    omega2 = g2 / np.sqrt(v2 + eps)
    J = _identity_filters(K2, C, 3, 3, shift) / omega2[:, None, None, None]
    Wb = np.concatenate([np.asarray(W2, np.float64), J], axis=1)
    return relu(batchnorm(conv2d(h, Wb, 1, 1), g2, b2, m2, v2, eps))


def fused_forward(g, x, return_all=False):
    """Evaluate a fused (possibly pruned) operator list in fp64."""
    t = {0: _c64(x)}
    for op in g.ops:
        a = t[op["src"]]
        if op["kind"] == "conv":
            y = add_bias(conv2d(a, op["W"], op["stride"], op["pad"]), op["b"])
            if op["scatter"] is not None:
                full = np.zeros((y.shape[0], op["K_full"]) + y.shape[2:], dtype=np.float64)
                full[:, op["scatter"]] = y
                y = full
            r = op["res"]
            if r is not None:
                s = t[r["tid"]]
                if r["mode"] == "A":
                    s = shortcut_a(s, y.shape[1], r["stride"], r["pad_lo"])
                y = add(y, s)
            if op["relu"]:
                y = relu(y)
        elif op["kind"] == "pool":
            y = maxpool(a, op["R"], op["stride"], op["pad"])
        else:
            y = fc(gavgpool(a), op["Wfc"], op["bfc"])
        t[op["out"]] = y
    return t if return_all else t[g.ops[-1]["out"]]


# ------------------------------------------------------------------------------------
# scoring, ranking, masks (Eq. 6, Algorithm 1)
# ------------------------------------------------------------------------------------

NORM_L1, NORM_L2 = 0, 1


def score_filters(w_f32, norm=NORM_L1):
    """Per-filter sum of |w| (l1) or w^2 (l2, the square root of Eq. 6 dropped: it is monotone)."""
    w = np.ascontiguousarray(w_f32, dtype=np.float32)
    K = w.shape[0]
    per = int(np.prod(w.shape[1:]))
    out = np.empty(K, dtype=np.float64)
    lib().fpo_score(_f(w), K, per, int(norm), _d(out))
    return out


def exact_scores(w_f32, norm=NORM_L1):
    """The same sums, exactly rounded (math.fsum), to check that summation order cannot change a ranking."""
    w = np.asarray(w_f32, dtype=np.float32).astype(np.float64)
    w = w.reshape(w.shape[0], -1)
    terms = w * w if norm == NORM_L2 else np.abs(w)
    return np.array([math.fsum(row) for row in terms])


def num_pruned(n, ratio):
    """Algorithm 1: 'the lowest p*n filters' - taken as floor(p*n) (tiny slack for p*n that is integral)."""
    return int(math.floor(ratio * n + 1e-9))


def rank_mask(scores, q):
    """Ascending by (score, index); the first q are pruned.  Returns (mask uint8 1=keep, rank int32)."""
    n = len(scores)
    order = sorted(range(n), key=lambda k: (scores[k], k))
    rank = np.empty(n, dtype=np.int32)
    for pos, k in enumerate(order):
        rank[k] = pos
    mask = (rank >= q).astype(np.uint8)
    return mask, rank


def select_masks(g32, ratios, norm=NORM_L1):
    """Masks for every convolution of a fused graph built with precision='f32'.

    Fused operators lose exactly n-m filters (back to the original count), the others
    floor(p*n); a conv absorbed into another has no filters of its own (mask None).
    All scores are taken on the unpruned fused weights, before any removal.
    """
    masks, ranks, all_scores = {}, {}, {}
    for ci in range(g32.n_convs):
        op = g32.conv_op.get(ci)
        if op is None:
            masks[ci] = ranks[ci] = all_scores[ci] = None
            continue
        s = score_filters(op["W"], norm)
        n = op["W"].shape[0]
        if op["role"] in ("aggr1", "aggr2"):
            q = n - op["n_orig"]
        else:
            q = num_pruned(n, float(ratios[ci]))
        if q >= n:
            raise ValueError(f"conv {ci}: pruning {q} of {n} filters leaves an empty layer")
        masks[ci], ranks[ci] = rank_mask(s, q)
        all_scores[ci] = s
    return masks, ranks, all_scores


# ------------------------------------------------------------------------------------
# pruning: removal and zeroing
# ------------------------------------------------------------------------------------

def _compactable(g, tid):
    """A tensor's channels can be physically dropped iff everything that reads it is a convolution's
    main input (or a max pool whose own result is compactable).  A tensor read as a residual operand,
    or produced into a residual stream, keeps its full width."""
    cons = g.consumers(tid)
    if not cons:
        return False
    for op, how in cons:
        if how == "res":
            return False
        if op["kind"] == "conv":
            continue
        if op["kind"] == "pool":
            if not _compactable(g, op["out"]):
                return False
        else:
            return False
    return True


def _drop_input_channels(g, tid, keep):
    for op, how in g.consumers(tid):
        if op["kind"] == "conv":
            op["W"] = op["W"][:, keep]
        elif op["kind"] == "pool":
            _drop_input_channels(g, op["out"], keep)


def _copy_graph(g):
    h = FusedGraph()
    h.n_convs = g.n_convs
    h.absorbed = dict(g.absorbed)
    for op in g.ops:
        o = dict(op)
        for key in ("W", "b", "Wfc", "bfc"):
            if key in o:
                o[key] = o[key].copy()
        if o.get("res") is not None:
            o["res"] = dict(o["res"])
        h.ops.append(o)
        if o["kind"] == "conv":
            h.conv_op[o["conv"]] = o
    return h


def prune_remove(g, masks):
    """Final extraction of Algorithm 1: masked filters are removed.  A removed filter contributes
    nothing downstream: where every reader is a convolution the matching input-channel slices are
    removed too; a convolution that writes a residual stream computes only its kept filters and
    scatters them into the full-width stream (the other channels carry the shortcut alone)."""
    h = _copy_graph(g)
    for ci, mask in masks.items():
        if mask is None:
            continue
        op = h.conv_op[ci]
        mask = np.asarray(mask).astype(bool)
        assert mask.shape[0] == op["K_full"]
        if mask.all():
            continue
        keep = np.nonzero(mask)[0]
        # the rows of W that survive; W may already have lost input channels, never rows
        op["W"] = op["W"][keep]
        op["b"] = op["b"][keep]
        if op["res"] is None and _compactable(h, op["out"]):
            _drop_input_channels(h, op["out"], keep)
            op["K_full"] = len(keep)
        else:
            op["scatter"] = keep
    return h


def prune_zero(g, masks):
    """Same selection realised by zeroing: the filter and its folded bias become 0, shapes unchanged."""
    h = _copy_graph(g)
    for ci, mask in masks.items():
        if mask is None:
            continue
        op = h.conv_op[ci]
        dead = ~np.asarray(mask).astype(bool)
        op["W"][dead] = 0.0
        op["b"][dead] = 0.0
    return h


def zero_unfused(net, weights, bn, masks):
    """Zeroing expressed on the original description: pruned filters get zero weights and their BN
    channel gamma = beta = 0, so the channel is exactly 0 for every consumer."""
    w = np.array(weights, dtype=np.float64)
    b = np.array(bn, dtype=np.float64)
    cons = _consumer_map(net)
    for ci, nid in enumerate(net.conv_ids()):
        mask = masks.get(ci)
        if mask is None:
            continue
        n = net.nodes[nid]
        per = n["C"] * n["R"] * n["S"]
        (bn_id,) = cons[nid]
        o, K = net.nodes[bn_id]["bn_off"], n["K"]
        for k in np.nonzero(~np.asarray(mask).astype(bool))[0]:
            w[n["w_off"] + k * per:n["w_off"] + (k + 1) * per] = 0.0
            b[o + k] = 0.0
            b[o + K + k] = 0.0
    return w, b


def pruned_model(net, weights, bn, ratios, norm=NORM_L1, masks=None):
    """fuse -> score -> mask -> remove.  Returns (fp64 pruned graph, masks, ranks, scores)."""
    g32 = fuse(net, weights, bn, "f32")
    ranks = scores = None
    if masks is None:
        masks, ranks, scores = select_masks(g32, ratios, norm)
    g64 = fuse(net, weights, bn, "f64")
    return prune_remove(g64, masks), masks, ranks, scores


# ------------------------------------------------------------------------------------
# dynamic (soft) filter pruning: the per-epoch loop of Algorithm 1
# ------------------------------------------------------------------------------------

def soft_prune_epoch(g32, ratios, norm=NORM_L2, updates=None):
    """One pass of Algorithm 1's loop body over a fused graph built with precision='f32', in place.

    `updates`: dict conv -> array shaped like that convolution's fused bank, standing for "update the
    parameters W by using data X" (there is no trainer here): W <- W + update, one fp32 addition per
    weight.  Then, for every convolution, the filters are scored on the updated weights, the lowest
    n - m (fused operator) or floor(p*n) filters are zeroized - weights only, they stay in the bank and
    the next epoch's update can bring them back - and the mask is returned.
    Returns (masks, ranks, scores), scores taken before zeroizing.
    """
    if updates is not None:
        for ci, dw in updates.items():
            op = g32.conv_op.get(ci)
            if op is None or dw is None:
                continue
            assert dw.shape == op["W"].shape
            op["W"] = (op["W"].astype(np.float32) + np.asarray(dw, np.float32)).astype(np.float32)
    masks, ranks, scores = select_masks(g32, ratios, norm)
    for ci, mask in masks.items():
        if mask is not None:
            g32.conv_op[ci]["W"][~np.asarray(mask).astype(bool)] = 0.0
    return masks, ranks, scores


def soft_prune_extract(g32, masks):
    """The last step of Algorithm 1: the model is obtained from the updated weights according to the masks
    of the last epoch - masked filters are removed.  Returns an fp64 graph for fused_forward."""
    g = _copy_graph(g32)
    for op in g.ops:
        for key in ("W", "b", "Wfc", "bfc"):
            if key in op and op[key] is not None:
                op[key] = np.asarray(op[key], dtype=np.float64)
    return prune_remove(g, masks)


def flops_and_params(g, in_hw):
    """Multiply-accumulate count per image and parameter count of a fused graph (bookkeeping pin)."""
    shapes = {0: in_hw}
    macs = params = 0
    for op in g.ops:
        H, W = shapes[op["src"]]
        if op["kind"] == "conv":
            K, C, R, S = op["W"].shape
            P = (H + 2 * op["pad"] - R) // op["stride"] + 1
            Q = (W + 2 * op["pad"] - S) // op["stride"] + 1
            macs += P * Q * K * C * R * S
            params += K * C * R * S
            shapes[op["out"]] = (P, Q)
        elif op["kind"] == "pool":
            P = (H + 2 * op["pad"] - op["R"]) // op["stride"] + 1
            Q = (W + 2 * op["pad"] - op["R"]) // op["stride"] + 1
            shapes[op["out"]] = (P, Q)
        else:
            macs += op["Wfc"].size
            params += op["Wfc"].size + op["bfc"].size
            shapes[op["out"]] = (1, 1)
    return macs, params
