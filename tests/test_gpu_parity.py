"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Tolerances (stated by the workload definition):
  masks / ranks / scores              bit-exact
  BF16 tensor-core activations        max|err| <= 2e-2 * max|ref|
  FP32 validation path                max|err| <= 1e-4 * max|ref|
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2010_16165_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_FP32 = 1e-4
# Activations deep inside a network (not the logits the stated tolerance is about): every layer rounds its output and
# its weights to bf16 (relative step 2^-9), the errors add up like a random walk over the layers, and where a sum of
# products cancels the relative error grows further.  Both GPU paths (layer by layer and the fused run) measure about
# 3.3e-3 * sqrt(L) rms after L convolutions (1.4e-2 after the 19 layers of ResNet-56's first stage, 2.5e-2 after 73
# layers of ResNet-110) and up to twice that at the worst element, so a tensor after L convolutions is held to
# max(2e-2, 6e-3 * sqrt(L)) in the rms sense and to twice that at the worst element.  A wrong tap, channel or shortcut
# is off by tens of percent.  The logits keep the stated 2e-2.


def inner_tolerances(n_convs_before):
    rms = max(2e-2, 6e-3 * np.sqrt(max(n_convs_before, 1)))
    return rms, 2.0 * rms


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2010_16165_b200 import binding
    binding.lib()
    return binding


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


class Gpu:
    """One fused model on the device."""

    def __init__(self, B, w, compute, max_batch=None, use_graph=0, keep_outputs=0, in_bf16=None, scatter=0):
        self.B, self.w = B, w
        self.dw, self.dbn = to_dev(w.weights), to_dev(w.bn)
        self.in_bf16 = w.in_bf16 if in_bf16 is None else in_bf16
        self.h = B.fp_fuse(w.net, self.dw, self.dbn, max_batch or w.batch, compute,
                           B.FP_DTYPE_BF16 if self.in_bf16 else B.FP_DTYPE_F32, use_graph, keep_outputs, scatter)
        self.n_classes = B.fp_query_int(self.h, B.FP_Q_N_CLASSES)

    def forward(self, x, stream=None):
        dx = to_dev(x)
        if self.in_bf16:
            dx = dx.to(torch.bfloat16)
        self.last_dx = dx                 # FP_Q_OP_OUTPUT may run the forward's prefix again on this input
        out = torch.full((x.shape[0], self.n_classes), float("nan"), device="cuda", dtype=torch.float32)
        if stream is not None:
            stream.wait_stream(torch.cuda.current_stream())
        self.B.fp_forward(self.h, dx, x.shape[0], out, stream)
        torch.cuda.synchronize()
        assert self.B.fp_query_int(self.h, self.B.FP_Q_DEVICE_STATUS) == 0, "a device-side wait timed out"
        return out.cpu().numpy().astype(np.float64)

    def close(self):
        self.B.fp_destroy(self.h)


def err(got, ref):
    return np.abs(got - ref).max() / np.abs(ref).max()


def oracle_pruned(fpo, w, masks=None):
    gp, m, ranks, scores = fpo.pruned_model(w.net, w.weights, w.bn, w.ratios, masks=masks)
    return gp, m, ranks, scores


TINY = {
    "cifar": lambda **k: wl.tiny_cifar(**k),
    "cifar_odd": lambda **k: wl.tiny_cifar(widths=(7, 12, 23), in_hw=12, batch=3, **k),
    "cifar_centered": lambda **k: wl.tiny_cifar(pad_lo_centered=True, n_per_stage=2, **k),
    "cifar_wide": lambda **k: wl.tiny_cifar(widths=(16, 48, 80), in_hw=16, batch=5, **k),
    "imagenet_basic": lambda **k: wl.tiny_imagenet_basic(**k),
    "imagenet_wide": lambda **k: wl.tiny_imagenet_basic(widths=(32, 64, 96), in_hw=48, batch=3, **k),
}


# ------------------------------------------------------------------------------------------
# scoring, ranking, masks: bit-exact
# ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("name", ["cifar", "cifar_odd", "imagenet_basic"])
@pytest.mark.parametrize("aggressive", [False, True])
@pytest.mark.parametrize("norm", [0, 1])
def test_scores_masks_bit_exact_tiny(B, fpo, name, aggressive, norm):
    w = TINY[name](aggressive=aggressive, p=0.3)
    g = Gpu(B, w, B.FP_COMPUTE_FP32)
    try:
        g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
        masks, ranks, scores = fpo.select_masks(g32, w.ratios, norm)
        B.fp_prune(g.h, w.ratios, None, norm)
        got = B.masks_and_ranks(g.h)
        for ci in range(w.net.n_convs()):
            if masks[ci] is None:
                assert got[ci][0] is None
                continue
            s = B.fp_score(g.h, ci, norm)
            assert s.tobytes() == scores[ci].tobytes(), f"conv {ci}: scores differ"
            np.testing.assert_array_equal(got[ci][1], ranks[ci])
            np.testing.assert_array_equal(got[ci][0], masks[ci])
    finally:
        g.close()


def test_masks_bit_exact_resnet20_and_bottleneck(B, fpo):
    for w in (wl.workload(1), wl.tiny_bottleneck(p=0.4)):
        g = Gpu(B, w, B.FP_COMPUTE_FP32, max_batch=2)
        try:
            g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
            masks, ranks, scores = fpo.select_masks(g32, w.ratios, 0)
            B.fp_prune(g.h, w.ratios)
            got = B.masks_and_ranks(g.h)
            for ci in range(w.net.n_convs()):
                np.testing.assert_array_equal(got[ci][0], masks[ci])
                np.testing.assert_array_equal(got[ci][1], ranks[ci])
                assert B.fp_score(g.h, ci, 0).tobytes() == scores[ci].tobytes()
                assert B.fp_query_int(g.h, B.FP_Q_CONV_K_KEPT, ci) == int(masks[ci].sum())
        finally:
            g.close()


def test_caller_masks_are_used(B, fpo):
    w = wl.tiny_cifar(p=0.0)
    rng = np.random.default_rng(5)
    masks = {}
    for ci, nid in enumerate(w.net.conv_ids()):
        m = (rng.random(w.net.nodes[nid]["K"]) > 0.4).astype(np.uint8)
        m[0] = 1
        masks[ci] = m
    g = Gpu(B, w, B.FP_COMPUTE_FP32)
    try:
        B.fp_prune(g.h, None, masks)
        got = g.forward(w.x)
        gp, _, _, _ = oracle_pruned(fpo, w, masks)
        assert err(got, fpo.fused_forward(gp, w.x)) < TOL_FP32
    finally:
        g.close()


# ------------------------------------------------------------------------------------------
# activations, tiny networks, every compute path
# ------------------------------------------------------------------------------------------

def _compare_ops(B, g, w, gp, fpo, tol):
    """Per-operator comparison (needs keep_outputs=1): reports the first operator that is off."""
    ref_all = fpo.fused_forward(gp, w.x, return_all=True)
    infos = B.op_infos(g.h)
    conv_ops = [op for op in gp.ops]
    oi = 0
    for i, info in enumerate(infos):
        if info.kind in (2, 3):
            continue
        ref = ref_all[conv_ops[oi]["out"]]
        oi += 1
        cnt = w.x.shape[0] * info.K_pad * info.P * info.Q   # upper bound
        C = ref.shape[1]
        got = B.fp_query_array(g.h, B.FP_Q_OP_OUTPUT, i, np.float32, w.x.shape[0] * C * info.P * info.Q)
        got = got.reshape(ref.shape).astype(np.float64)
        e = np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30)
        assert e < tol, f"operator {i} (kind {info.kind}, conv {info.conv_index}, K={info.K} C={info.C} " \
                        f"R={info.R} stride={info.stride} res={info.res_mode}): rel err {e:.3e}"


@pytest.mark.parametrize("name", list(TINY))
@pytest.mark.parametrize("aggressive", [False, True])
@pytest.mark.parametrize("p", [0.0, 0.3])
@pytest.mark.parametrize("compute", ["fp32", "simt", "tc"])
def test_tiny_networks(B, fpo, name, aggressive, p, compute):
    w = TINY[name](aggressive=aggressive, p=p)
    mode = {"fp32": B.FP_COMPUTE_FP32, "simt": B.FP_COMPUTE_BF16_SIMT, "tc": B.FP_COMPUTE_BF16_TC}[compute]
    tol = TOL_FP32 if compute == "fp32" else TOL_BF16
    g = Gpu(B, w, mode, keep_outputs=1)
    try:
        if p == 0.0:
            # fusion alone is an equivalence: the fused graph reproduces the network as described
            assert err(g.forward(w.x), fpo.unfused_forward(w.net, w.weights, w.bn, w.x)) < tol
        B.fp_prune(g.h, w.ratios)
        got = g.forward(w.x)
        gp, masks, _, _ = oracle_pruned(fpo, w)
        ref = fpo.fused_forward(gp, w.x)
        if not err(got, ref) < tol:
            _compare_ops(B, g, w, gp, fpo, tol)
        assert err(got, ref) < tol
    finally:
        g.close()


@pytest.mark.parametrize("compute", ["fp32", "tc"])
def test_tiny_bottleneck(B, fpo, compute):
    w = wl.tiny_bottleneck(p=0.4)
    mode = B.FP_COMPUTE_FP32 if compute == "fp32" else B.FP_COMPUTE_BF16_TC
    tol = TOL_FP32 if compute == "fp32" else TOL_BF16
    g = Gpu(B, w, mode, keep_outputs=1)
    try:
        B.fp_prune(g.h, w.ratios)
        got = g.forward(w.x)
        gp, _, _, _ = oracle_pruned(fpo, w)
        ref = fpo.fused_forward(gp, w.x)
        if not err(got, ref) < tol:
            _compare_ops(B, g, w, gp, fpo, tol)
        assert err(got, ref) < tol
    finally:
        g.close()


@pytest.mark.parametrize("compute", ["fp32", "tc"])
def test_tiny_bottleneck_aggressive(B, fpo, compute):
    """Three-convolution blocks fused the paper's way: the pass-through rides through 1x1 - 3x3 - 1x1, no add."""
    w = wl.tiny_bottleneck(aggressive=True)
    mode = B.FP_COMPUTE_FP32 if compute == "fp32" else B.FP_COMPUTE_BF16_TC
    tol = TOL_FP32 if compute == "fp32" else TOL_BF16
    g = Gpu(B, w, mode, keep_outputs=1)
    try:
        assert all(o.res_mode == 0 for o in B.op_infos(g.h)), "an add survived"
        assert err(g.forward(w.x), fpo.unfused_forward(w.net, w.weights, w.bn, w.x)) < tol
        zeros = np.zeros(w.net.n_convs())
        B.fp_prune(g.h, zeros)                       # fused operators go back to their original filter counts
        gp, masks, ranks, _ = fpo.pruned_model(w.net, w.weights, w.bn, zeros)
        for ci, (m, r) in B.masks_and_ranks(g.h).items():
            if masks[ci] is None:
                assert m is None
            else:
                np.testing.assert_array_equal(m, masks[ci])
                np.testing.assert_array_equal(r, ranks[ci])
        got = g.forward(w.x)
        ref = fpo.fused_forward(gp, w.x)
        if not err(got, ref) < tol:
            _compare_ops(B, g, w, gp, fpo, tol)
        assert err(got, ref) < tol
    finally:
        g.close()


@pytest.mark.parametrize("compute", ["fp32", "tc"])
def test_concat_structures(B, fpo, compute):
    """y = concat(conv(x), x) (Sec. IV-B.1) runs as one convolution with identity filters; pruned back by n - m."""
    w = wl.tiny_concat()
    mode = B.FP_COMPUTE_FP32 if compute == "fp32" else B.FP_COMPUTE_BF16_TC
    tol = TOL_FP32 if compute == "fp32" else TOL_BF16
    g = Gpu(B, w, mode, keep_outputs=1)
    try:
        infos = [o for o in B.op_infos(g.h) if o.kind == 0]
        assert [o.K for o in infos] == [8, 14, 24, 29]
        assert err(g.forward(w.x), fpo.unfused_forward(w.net, w.weights, w.bn, w.x)) < tol
        zeros = np.zeros(w.net.n_convs())
        B.fp_prune(g.h, zeros)
        gp, masks, ranks, _ = fpo.pruned_model(w.net, w.weights, w.bn, zeros)
        for ci, (m, r) in B.masks_and_ranks(g.h).items():
            np.testing.assert_array_equal(m, masks[ci])
            np.testing.assert_array_equal(r, ranks[ci])
        got = g.forward(w.x)
        ref = fpo.fused_forward(gp, w.x)
        if not err(got, ref) < tol:
            _compare_ops(B, g, w, gp, fpo, tol)
        assert err(got, ref) < tol
    finally:
        g.close()


@pytest.mark.parametrize("name", ["cifar_wide", "cifar_odd", "imagenet_basic", "imagenet_wide"])
@pytest.mark.parametrize("p", [0.3, 0.6])
@pytest.mark.parametrize("scatter", [1, -1])
def test_stream_writers_scattered_or_zero_rows(B, fpo, name, p, scatter):
    """Algorithm 1's removal for convolutions that write a residual stream: only the kept filters are computed and
    scattered into the full-width tensor (scatter=1, forced here on every such layer: strided and 1x1 projections,
    option-A and same-shape shortcuts, the first convolution), or the pruned filters stay as zero rows (-1).  Both
    against the oracle, operator by operator."""
    w = TINY[name](p=p)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, keep_outputs=1, scatter=scatter)
    try:
        B.fp_prune(g.h, w.ratios)
        got = g.forward(w.x)
        gp, _, _, _ = oracle_pruned(fpo, w)
        _compare_ops(B, g, w, gp, fpo, TOL_BF16)
        assert err(got, fpo.fused_forward(gp, w.x)) < TOL_BF16
        writers = [o for o in B.op_infos(g.h) if o.kind == 0 and
                   o.K < B.fp_query_int(g.h, B.FP_Q_CONV_K_FUSED, o.conv_index) and
                   (o.res_mode != 0 or o.conv_index == 0)]
        assert writers, "the case must contain pruned stream writers"
        narrower = [o for o in writers if o.K_pad < (B.fp_query_int(g.h, B.FP_Q_CONV_K_FUSED, o.conv_index) + 15) // 16 * 16]
        if scatter == 1:
            assert narrower or all((o.K + 15) // 16 == (B.fp_query_int(g.h, B.FP_Q_CONV_K_FUSED, o.conv_index) + 15) // 16
                                   for o in writers), "no stream writer computes fewer columns than its tensor is wide"
        else:
            assert not narrower
    finally:
        g.close()


def test_per_operator_outputs_tc(B, fpo):
    """Every fused operator's activation, not only the logits (several tiles, ragged tails)."""
    w = wl.tiny_cifar(widths=(16, 32, 64), in_hw=20, batch=3, n_per_stage=2, p=0.3)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, keep_outputs=1)
    try:
        B.fp_prune(g.h, w.ratios)
        g.forward(w.x)
        gp, _, _, _ = oracle_pruned(fpo, w)
        _compare_ops(B, g, w, gp, fpo, TOL_BF16)
    finally:
        g.close()


def test_prune_ratio_zero_restores_unpruned(B, fpo):
    w = wl.tiny_cifar(n_per_stage=2, p=0.5)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        before = g.forward(w.x)
        B.fp_prune(g.h, w.ratios)
        pruned = g.forward(w.x)
        B.fp_prune(g.h, np.zeros_like(w.ratios))
        after = g.forward(w.x)
        np.testing.assert_array_equal(before, after)
        assert np.abs(before - pruned).max() > 1e-3
    finally:
        g.close()


def test_batch_edges_and_graph_and_host(B, fpo):
    w = wl.tiny_cifar(batch=7, p=0.3)
    gp, _, _, _ = oracle_pruned(fpo, w)
    ref = fpo.fused_forward(gp, w.x)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, max_batch=9, use_graph=1)
    try:
        B.fp_prune(g.h, w.ratios)
        full = g.forward(w.x)
        assert err(full, ref) < TOL_BF16
        # images are independent: any sub-batch reproduces its rows bit for bit
        for b in (1, 2, 5):
            np.testing.assert_array_equal(g.forward(w.x[:b]), full[:b])
        # CUDA-graph replay on a side stream gives the same bits, twice
        st = torch.cuda.Stream()
        a1 = g.forward(w.x, st)
        a2 = g.forward(w.x, st)
        np.testing.assert_array_equal(a1, full)
        np.testing.assert_array_equal(a2, full)
        # host-buffer entry point
        out = np.empty((7, g.n_classes), dtype=np.float32)
        B.fp_forward_host(g.h, w.x, 7, out)
        np.testing.assert_array_equal(out.astype(np.float64), full)
        with pytest.raises(B.FpError) as e:
            B.fp_forward(g.h, to_dev(w.x), 10, torch.empty(10, g.n_classes, device="cuda"))
        assert e.value.status == B.FP_ERR_BOUNDS
    finally:
        g.close()


def test_a_device_wait_that_runs_out_is_reported_and_survived(B, fpo):
    """Every wait inside the tensor-core kernels is bounded.  A diagnostic launch leaves out one round of a convolution's
    activation copies with a limit of a millisecond: the waiting thread gives up, the status word is raised, all roles of the
    CTA leave, tensor memory is released, the kernel returns.  The status is reported once, and the same handle then runs a
    forward with the bits it produced before."""
    w = wl.tiny_cifar(widths=(16, 32, 64), in_hw=16, batch=4, p=0.3)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, keep_outputs=1)            # every layer is a kernel of its own
    try:
        B.fp_prune(g.h, w.ratios)
        before = g.forward(w.x)
        B.fp_debug_expire_wait(g.h)
        torch.cuda.synchronize()                                   # returns: nothing hangs, nothing faults
        assert B.fp_query_int(g.h, B.FP_Q_DEVICE_STATUS) == B.FP_ERR_TIMEOUT
        assert B.fp_query_int(g.h, B.FP_Q_DEVICE_STATUS) == 0      # reported once
        after = g.forward(w.x)                                     # forward() checks the status too
        np.testing.assert_array_equal(before, after)
        gp, _, _, _ = oracle_pruned(fpo, w)
        assert err(after, fpo.fused_forward(gp, w.x)) < TOL_BF16
    finally:
        g.close()


def test_callers_allocator_serves_every_buffer(B, fpo):
    """fp_fuse_with_allocator: the library takes all of its device memory from the caller's allocator (here PyTorch's
    caching allocator through two callbacks) - at fuse time, when fp_prune rebuilds the graph and for debug dumps - and
    gives all of it back by fp_destroy; results are the same bits as with its own cudaMalloc."""
    w = wl.tiny_cifar(widths=(16, 32, 64), in_hw=16, batch=3, n_per_stage=2, p=0.3)
    ref_g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        B.fp_prune(ref_g.h, w.ratios)
        want = ref_g.forward(w.x)
    finally:
        ref_g.close()
    alloc = B.TorchAllocator()
    dw, dbn = to_dev(w.weights), to_dev(w.bn)
    h = B.fp_fuse(w.net, dw, dbn, w.batch, B.FP_COMPUTE_BF16_TC, B.FP_DTYPE_F32, 0, 0, 0, alloc)
    try:
        n_fuse = alloc.n_alloc
        assert n_fuse > 10
        B.fp_prune(h, w.ratios)
        assert alloc.n_alloc > n_fuse and alloc.n_free > 0          # the graph was rebuilt out of the same allocator
        out = torch.empty(w.batch, 5, device="cuda")
        dx = to_dev(w.x)
        B.fp_forward(h, dx, w.batch, out)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(out.cpu().numpy().astype(np.float64), want)
        info = [o for o in B.op_infos(h)]
        last_conv = max(i for i, o in enumerate(info) if o.kind == 0)
        o = info[last_conv]
        B.fp_query_array(h, B.FP_Q_OP_OUTPUT, last_conv, np.float32, w.batch * 64 * o.P * o.Q)    # the dump's scratch too
    finally:
        B.fp_destroy(h)
    assert alloc.n_alloc == alloc.n_free and not alloc.live


def test_error_codes(B):
    w = wl.tiny_cifar()
    dw, dbn = to_dev(w.weights), to_dev(w.bn)
    # NaN in the weights
    bad = w.weights.copy(); bad[3] = np.nan
    with pytest.raises(B.FpError) as e:
        B.fp_fuse(w.net, to_dev(bad), dbn, 2, B.FP_COMPUTE_FP32)
    assert e.value.status == B.FP_ERR_NONFINITE
    # a convolution whose channel count does not match its producer
    import copy
    net = copy.deepcopy(w.net)
    net.nodes[net.conv_ids()[1]]["C"] += 1
    with pytest.raises(B.FpError) as e:
        B.fp_fuse(net, dw, dbn, 2, B.FP_COMPUTE_FP32)
    assert e.value.status in (B.FP_ERR_SHAPE, B.FP_ERR_DESC)
    # forward reference
    net = copy.deepcopy(w.net)
    net.nodes[2]["in0"] = 5
    with pytest.raises(B.FpError) as e:
        B.fp_fuse(net, dw, dbn, 2, B.FP_COMPUTE_FP32)
    assert e.value.status == B.FP_ERR_DESC
    # pruning everything
    h = B.fp_fuse(w.net, dw, dbn, 2, B.FP_COMPUTE_FP32)
    try:
        with pytest.raises(B.FpError) as e:
            B.fp_prune(h, np.ones(w.net.n_convs()))
        assert e.value.status == B.FP_ERR_EMPTY_LAYER
        with pytest.raises(B.FpError) as e:
            B.fp_prune(h, np.full(w.net.n_convs(), -0.5))
        assert e.value.status == B.FP_ERR_ARG
    finally:
        B.fp_destroy(h)
    # a valid description the kernels cannot run: images wider than 512 pixels
    wb = wl.tiny_cifar()
    net = copy.deepcopy(wb.net)
    net.in_W = 600
    with pytest.raises(B.FpError) as e:
        B.fp_fuse(net, to_dev(wb.weights), to_dev(wb.bn), 2, B.FP_COMPUTE_FP32)
    assert e.value.status == B.FP_ERR_UNSUPPORTED


# ------------------------------------------------------------------------------------------
# the benchmark-shaped workloads at full size
# ------------------------------------------------------------------------------------------

def _sample_images(n, k):
    idx = sorted(set([0, n - 1] + list(range(0, n, 37))))
    return idx[:k] if len(idx) > k else idx


def _compare_stored_ops(B, g, w, gp, fpo, idx):
    """Full-size run without keep_outputs: every operator whose output reaches memory (single layers, pools, the
    last layer of each fused run) against the oracle on the sampled images `idx`.  Returns how many were compared."""
    ref_all = fpo.fused_forward(gp, w.x[idx], return_all=True)
    infos = B.op_infos(g.h)
    n_img = w.x.shape[0]
    oi, compared = 0, 0
    for i, info in enumerate(infos):
        if info.kind in (2, 3):
            continue
        ref = ref_all[gp.ops[oi]["out"]]
        oi += 1
        C = ref.shape[1]
        try:
            got = B.fp_query_array(g.h, B.FP_Q_OP_OUTPUT, i, np.float32, n_img * C * info.P * info.Q)
        except B.FpError as e:
            assert e.status == B.FP_ERR_UNSUPPORTED      # inside a fused run, or pooled inside the first convolution's kernel: never stored
            continue
        got = got.reshape((n_img,) + ref.shape[1:])[idx].astype(np.float64)
        e = np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30)
        rms = np.sqrt(((got - ref) ** 2).mean()) / max(np.sqrt((ref ** 2).mean()), 1e-30)
        tol_rms, tol_max = inner_tolerances(oi)          # oi operators (convolutions, but for a pool) come before it
        assert e < tol_max and rms < tol_rms, \
            f"{w.name}: operator {i} (kind {info.kind}, conv {info.conv_index}, K={info.K} C={info.C} R={info.R} " \
            f"stride={info.stride} res={info.res_mode} chain={info.chain}): max err {e:.3e}, rms err {rms:.3e}"
        compared += 1
    return compared


def _full_config(B, fpo, w, n_oracle, also_fp32=True, stored_ops=False):
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, use_graph=1)
    try:
        B.fp_prune(g.h, w.ratios)
        st = torch.cuda.Stream()
        got = g.forward(w.x, st)
        assert np.isfinite(got).all()
        # masks bit-exact at full size
        g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
        masks, ranks, _ = fpo.select_masks(g32, w.ratios, 0)
        mr = B.masks_and_ranks(g.h)
        for ci in range(w.net.n_convs()):
            if masks[ci] is not None:
                np.testing.assert_array_equal(mr[ci][0], masks[ci])
                np.testing.assert_array_equal(mr[ci][1], ranks[ci])
        # sampled images against the oracle
        idx = _sample_images(w.batch, n_oracle)
        gp = fpo.prune_remove(fpo.fuse(w.net, w.weights, w.bn), masks)
        ref = fpo.fused_forward(gp, w.x[idx])
        e = err(got[idx], ref)
        assert e < TOL_BF16, f"{w.name}: bf16 tensor-core path rel err {e:.3e}"
        if stored_ops:
            assert _compare_stored_ops(B, g, w, gp, fpo, idx) >= 2
    finally:
        g.close()
    if also_fp32:
        # every image: FP32 validation path (itself within 1e-4 of the oracle on the samples)
        g = Gpu(B, w, B.FP_COMPUTE_FP32)
        try:
            B.fp_prune(g.h, w.ratios)
            got32 = g.forward(w.x)
            assert err(got32[idx], ref) < TOL_FP32
            assert err(got, got32) < TOL_BF16
        finally:
            g.close()


def test_config1_resnet20_b8(B, fpo):
    w = wl.workload(1)
    _full_config(B, fpo, w, 8)


@pytest.mark.parametrize("p", [0.0, 0.3, 0.5])
def test_config2_resnet56_b256(B, fpo, p):
    w = wl.workload(2, prune=p)
    _full_config(B, fpo, w, 12, stored_ops=True)   # fused runs are compared at their last layer, not only through the head


def test_config3_resnet110_b1024(B, fpo):
    w = wl.workload(3)
    _full_config(B, fpo, w, 6, stored_ops=True)


def test_config4_resnet18_b64(B, fpo):
    w = wl.workload(4)
    _full_config(B, fpo, w, 2, stored_ops=True)


def test_wide_stream_writers_compute_kept_filters_only(B, fpo):
    """ResNet-18 at batch 256: the last stage's second convolutions keep 359 of 512 filters and, with enough position
    tiles to fill the GPU several times over, compute only those (scattered output); the result still equals the oracle's
    removal.  (At batch 64 the same layers have 41 position tiles and keep zero rows: fewer columns would only idle SMs.)"""
    w = wl.workload(4, batch=256)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, use_graph=1)
    try:
        B.fp_prune(g.h, w.ratios)
        got = g.forward(w.x, torch.cuda.Stream())
        wide = [o for o in B.op_infos(g.h) if o.kind == 0 and o.res_mode == 1 and o.K == 359]
        assert wide and all(o.K_pad <= 384 for o in wide), [(o.K, o.K_pad) for o in wide]
        idx = [0, 255]
        gp, _, _, _ = oracle_pruned(fpo, w)
        assert err(got[idx], fpo.fused_forward(gp, w.x[idx])) < TOL_BF16
        assert _compare_stored_ops(B, g, w, gp, fpo, idx) >= 2
    finally:
        g.close()


def test_config5_resnet50_b128(B, fpo):
    """The benchmarked batch: its launch plans (tile counts decide them) are the ones compared with the oracle."""
    w = wl.workload(5)
    assert w.batch == 128
    _full_config(B, fpo, w, 2, stored_ops=True)


def test_config5_resnet50_small_batches(B, fpo):
    w = wl.workload(5, batch=16)     # the oracle covers two images; all 16 go through both GPU paths
    _full_config(B, fpo, w, 2)
    w1 = wl.workload(5, batch=1)     # the latency configuration
    _full_config(B, fpo, w1, 1, also_fp32=False, stored_ops=True)


def test_paper_models_resnet32_and_resnet34(B, fpo):
    """The two networks of the paper's Table II that the five workloads do not cover, at the benchmarked batches."""
    _full_config(B, fpo, wl.workload(6), 6)
    w = wl.workload(7)
    assert w.batch == 64
    _full_config(B, fpo, w, 1, stored_ops=True)
    _full_config(B, fpo, wl.workload(7, batch=8), 1, also_fp32=False)


def test_config1_aggressive_fused_unpruned_and_pruned(B, fpo):
    """The paper's own graph: dilated convolutions, no add; then pruned back by n-m filters."""
    w = wl.workload(1, aggressive=True)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        got = g.forward(w.x)
        ref = fpo.unfused_forward(w.net, w.weights, w.bn, w.x)
        assert err(got, ref) < TOL_BF16
        B.fp_prune(g.h, np.zeros(w.net.n_convs()))          # conservative: fused operators lose n-m
        gp, masks, _, _ = fpo.pruned_model(w.net, w.weights, w.bn, np.zeros(w.net.n_convs()))
        assert err(g.forward(w.x), fpo.fused_forward(gp, w.x)) < TOL_BF16
        for ci, m in B.masks_and_ranks(g.h).items():
            np.testing.assert_array_equal(m[0], masks[ci])
    finally:
        g.close()


def _stem_net(H, W, K, in_C=3, name="stem_pool"):
    net = wl.Net(in_C, H, W, name)
    x = net.relu(net.bn(net.conv(-1, K, in_C, 7, 2, 3), K))
    x = net.maxpool(x, K)
    x = net.relu(net.bn(net.conv(x, 24, K, 3, 1, 1), 24))
    x = net.gavgpool(x, 24)
    net.fc(x, 6, 24)
    net.n_blocks = 0
    return net


@pytest.mark.parametrize("shape", [(32, 32, 16, 3, 2), (36, 64, 40, 3, 5), (24, 112, 64, 3, 3), (16, 8, 16, 1, 2), (224, 224, 64, 3, 2)])
@pytest.mark.parametrize("p", [0.0, 0.3])
def test_first_convolution_and_pooling_in_one_kernel(B, fpo, shape, p):
    """7x7 / 2 convolution + ReLU + 3x3 / 2 max pooling from the NCHW bf16 input in one kernel: one, two and three position
    tiles per unit, an odd number of pooled rows, one input channel, the 224 x 224 size; the pooled tensor and the logits
    against the oracle, and a smaller batch than the handle was built for."""
    H, W, K, C, batch = shape
    w = wl.Workload("stem_pool", _stem_net(H, W, K, C), batch, 31, True, wl.uniform_ratios(p), f"uniform {p}")
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, max_batch=batch + 1)
    try:
        B.fp_prune(g.h, w.ratios)
        assert B.fp_query_int(g.h, B.FP_Q_N_LAUNCHES) == 4          # stem + pooling, convolution, two head kernels
        got = g.forward(w.x)
        gp, _, _, _ = oracle_pruned(fpo, w)
        ref_all = fpo.fused_forward(gp, w.x, return_all=True)
        pooled_ref = ref_all[gp.ops[1]["out"]]
        info = B.op_infos(g.h)[2]
        pooled = B.fp_query_array(g.h, B.FP_Q_OP_OUTPUT, 2, np.float32, batch * pooled_ref.shape[1] * info.P * info.Q)
        assert err(pooled.reshape(pooled_ref.shape).astype(np.float64), pooled_ref) < TOL_BF16
        assert err(got, fpo.fused_forward(gp, w.x)) < TOL_BF16
        np.testing.assert_array_equal(g.forward(w.x[:1]), got[:1])
        out = np.empty((batch, g.n_classes), dtype=np.float32)
        x_host = torch.from_numpy(w.x).to(torch.bfloat16)            # host buffer in the network's input type
        B.fp_forward_host(g.h, x_host, batch, out)                   # the input arrives in pieces, one kernel launch per piece
        np.testing.assert_array_equal(out.astype(np.float64), got)
    finally:
        g.close()


def test_queued_host_calls_overlap_copies_without_mixing_inputs(B, fpo):
    """fp_forward_host_async: three calls with three different pinned inputs queued back to back on one stream (the
    second and third inputs are copied while the forward before them still runs - they wait only for its first
    kernel); every call's logits equal those of the blocking call on the same input."""
    H, W, K, C, batch = 64, 64, 32, 3, 6
    w = wl.Workload("stem_pool", _stem_net(H, W, K, C), batch, 37, True, wl.uniform_ratios(0.3), "uniform 0.3")
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, max_batch=batch)
    try:
        B.fp_prune(g.h, w.ratios)
        rng = np.random.default_rng(5)
        xs = [torch.from_numpy((w.x * s + rng.standard_normal(w.x.shape).astype(np.float32) * 0.1)).to(torch.bfloat16).pin_memory()
              for s in (1.0, -0.5, 0.25)]
        want = []
        for x in xs:
            out = np.empty((batch, g.n_classes), dtype=np.float32)
            B.fp_forward_host(g.h, x, batch, out)
            want.append(out)
        assert not np.array_equal(want[0], want[1])
        outs = [torch.empty((batch, g.n_classes), dtype=torch.float32).pin_memory() for _ in xs]
        stream = torch.cuda.Stream()
        for rep in range(3):
            for x, o in zip(xs, outs):
                B.fp_forward_host_async(g.h, x, batch, o, stream)
            stream.synchronize()
            for o, ref in zip(outs, want):
                np.testing.assert_array_equal(o.numpy(), ref)
        assert B.fp_query_int(g.h, B.FP_Q_DEVICE_STATUS) == 0
    finally:
        g.close()


def test_maxpool_windows_of_negative_values(B, fpo):
    """Max pooling right after a batch norm without ReLU, every other channel shifted far below zero, so a padded
    position that took part in a window as 0 (instead of being ignored) would win it.  Odd height, a width that
    leaves the second warp of a row partly empty; compared operator by operator."""
    net = wl.Net(3, 37, 70, "pool_negative")
    x = net.bn(net.conv(-1, 16, 3, 3, 1, 1), 16)
    x = net.maxpool(x, 16)
    x = net.gavgpool(x, 16)
    net.fc(x, 5, 16)
    net.n_blocks = 0
    w = wl.Workload("pool_negative", net, 2, 23, True, wl.uniform_ratios(0.0), "none")
    node = [n for n in net.nodes if n["op"] == wl.OP_BN][0]
    w.bn[node["bn_off"] + 16:node["bn_off"] + 32:2] = -3.0        # beta of every other channel: all-negative windows
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, keep_outputs=1)
    try:
        got = g.forward(w.x)
        gp, _, _, _ = oracle_pruned(fpo, w)
        ref_all = fpo.fused_forward(gp, w.x, return_all=True)
        pooled = [ref_all[op["out"]] for op in gp.ops][1]
        assert (pooled < 0).mean() > 0.05, "the case must contain windows whose maximum is negative"
        _compare_ops(B, g, w, gp, fpo, TOL_BF16)
        assert err(got, fpo.fused_forward(gp, w.x)) < TOL_BF16
    finally:
        g.close()
