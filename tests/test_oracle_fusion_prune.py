"""Pins for the oracle's fusion, scoring, ranking and pruning: the invariants the paper fixes."""
import os

import numpy as np
import pytest

from paper_2010_16165_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rel(a, b):
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-300)


def tiny_sets():
    return [
        ("cifar", wl.tiny_cifar, dict()),
        ("cifar_centered_pad", wl.tiny_cifar, dict(pad_lo_centered=True)),
        ("cifar_deeper", wl.tiny_cifar, dict(n_per_stage=2, widths=(4, 6, 10))),
        ("imagenet_basic", wl.tiny_imagenet_basic, dict()),
        ("imagenet_basic_3x3stem", wl.tiny_imagenet_basic, dict(stem_k=3, in_hw=16)),
    ]


# ---------------------------------------------------------------------------------------
# fusion is an equivalence transformation (Sec. IV-B.1 end of first paragraph; Sec. IV-C)
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("name,make,kw", tiny_sets())
@pytest.mark.parametrize("aggressive", [False, True])
def test_fused_equals_unfused_tiny(fpo, name, make, kw, aggressive):
    w = make(aggressive=aggressive, **kw)
    ref = fpo.unfused_forward(w.net, w.weights, w.bn, w.x)
    g = fpo.fuse(w.net, w.weights, w.bn)
    got = fpo.fused_forward(g, w.x)
    assert rel(got, ref) < 1e-12
    if aggressive:
        assert all(op["res"] is None for op in g.ops if op["kind"] == "conv"), "an add survived"
        assert any(op["role"] == "aggr1" for op in g.ops if op["kind"] == "conv")


def test_fused_equals_unfused_bottleneck(fpo):
    w = wl.tiny_bottleneck()
    ref = fpo.unfused_forward(w.net, w.weights, w.bn, w.x)
    assert rel(fpo.fused_forward(fpo.fuse(w.net, w.weights, w.bn), w.x), ref) < 1e-12


@pytest.mark.parametrize("aggressive", [False, True, {0, 1, 2, 3}])
def test_fused_equals_unfused_resnet20(fpo, aggressive):
    # fusion option x/n: all blocks, or only the first stage plus the first downsampling block
    net = wl.resnet_cifar(3, aggressive=aggressive)
    rng = np.random.default_rng(1)
    weights, bn = wl.make_params(net, rng)
    x = wl.make_input(net, 2, rng)
    ref = fpo.unfused_forward(net, weights, bn, x)
    got = fpo.fused_forward(fpo.fuse(net, weights, bn), x)
    assert rel(got, ref) < 1e-12


def test_fused_filter_bookkeeping(fpo):
    # a fused conv1 has n = K1 + C filters where the original had m = K1 (Algorithm 1, n and m)
    w = wl.tiny_cifar(aggressive=True)
    g = fpo.fuse(w.net, w.weights, w.bn)
    seen = 0
    for op in g.ops:
        if op["kind"] == "conv" and op["role"] == "aggr1":
            K, C = op["W"].shape[:2]
            assert K == op["n_orig"] + C
            seen += 1
        if op["kind"] == "conv" and op["role"] == "aggr2":
            assert op["W"].shape[0] == op["n_orig"]
    assert seen == 3


def test_both_bn_orders_agree(fpo):
    # Sec. IV-B.2: auxiliary BN (scale 1, shift 0) on the pass-through channels does not change the
    # result, and the xconv-F weights carry the inverse of bn2.  Compare with the plain block.
    rng = np.random.default_rng(2)
    C = 5
    x = np.abs(rng.standard_normal((2, C, 6, 6)))            # block inputs are ReLU outputs
    W1 = rng.standard_normal((7, C, 3, 3)); W2 = rng.standard_normal((C, 7, 3, 3))
    bn1 = (rng.uniform(0.5, 1.5, 7), rng.standard_normal(7), rng.standard_normal(7), rng.uniform(0.5, 1.5, 7))
    bn2 = (rng.uniform(0.5, 1.5, C), rng.standard_normal(C), rng.standard_normal(C), rng.uniform(0.5, 1.5, C))
    eps = 1e-5
    h = fpo.relu(fpo.batchnorm(fpo.conv2d(x, W1, 1, 1), *bn1, eps))
    plain = fpo.relu(fpo.add(fpo.batchnorm(fpo.conv2d(h, W2, 1, 1), *bn2, eps), x))
    paper = fpo.aggressive_block_paper_order(x, W1, bn1, W2, bn2, eps)
    assert rel(paper, plain) < 1e-12
    # downsampling block with zero-channel padding: shortcut = x[::2, ::2] in channels shift..shift+C
    K = 9
    W1 = rng.standard_normal((K, C, 3, 3)); W2 = rng.standard_normal((K, K, 3, 3))
    bn1 = (rng.uniform(0.5, 1.5, K), rng.standard_normal(K), rng.standard_normal(K), rng.uniform(0.5, 1.5, K))
    bn2 = (rng.uniform(0.5, 1.5, K), rng.standard_normal(K), rng.standard_normal(K), rng.uniform(0.5, 1.5, K))
    h = fpo.relu(fpo.batchnorm(fpo.conv2d(x, W1, 2, 1), *bn1, eps))
    plain = fpo.relu(fpo.add(fpo.batchnorm(fpo.conv2d(h, W2, 1, 1), *bn2, eps), fpo.shortcut_a(x, K, 2, 2)))
    paper = fpo.aggressive_block_paper_order(x, W1, bn1, W2, bn2, eps, stride=2, shift=2)
    assert rel(paper, plain) < 1e-12


def test_architecture_counts(fpo):
    want = {}
    for line in open(os.path.join(GOLDEN, "architectures.txt")):
        if line.strip() and not line.startswith("#"):
            name, p, m = line.split()
            want[name] = (int(m), int(p))
    nets = {
        "resnet20": (wl.resnet_cifar(3), 32), "resnet32": (wl.resnet_cifar(5), 32),
        "resnet56": (wl.resnet_cifar(9), 32), "resnet110": (wl.resnet_cifar(18), 32),
        "resnet18": (wl.resnet_imagenet_basic(), 224), "resnet34": (wl.resnet_imagenet_basic((3, 4, 6, 3)), 224),
        "resnet50": (wl.resnet_imagenet_bottleneck(), 224),
    }
    for name, (net, hw) in nets.items():
        g = fpo.fuse(net, np.zeros(net.n_weights, np.float32), np.ones(net.n_bn, np.float32), "f32")
        assert fpo.flops_and_params(g, (hw, hw)) == want[name], name


# ---------------------------------------------------------------------------------------
# scoring (Eq. 6) and selection (Algorithm 1)
# ---------------------------------------------------------------------------------------

def test_scores_hand_example(fpo):
    w = np.array([[[[1.0]], [[-2.0]]], [[[0.5]], [[0.25]]]], dtype=np.float32)   # 2 x 2 x 1 x 1
    np.testing.assert_array_equal(fpo.score_filters(w, fpo.NORM_L1), [3.0, 0.75])
    np.testing.assert_array_equal(fpo.score_filters(w, fpo.NORM_L2), [5.0, 0.3125])


def test_identity_filters_score_exactly_one(fpo):
    # auxiliary filters are a single unit tap (Sec. IV-B.1, Sec. IV-C "dramatically sparse")
    w = wl.tiny_cifar(aggressive=True)
    g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
    for op in g32.ops:
        if op["kind"] == "conv" and op["role"] == "aggr1":
            for norm in (fpo.NORM_L1, fpo.NORM_L2):
                s = fpo.score_filters(op["W"], norm)
                np.testing.assert_array_equal(s[op["n_orig"]:], 1.0)
                assert (s[:op["n_orig"]] != 1.0).all()


@pytest.mark.parametrize("norm", [0, 1])
def test_scores_vs_exact_and_numpy(fpo, norm):
    rng = np.random.default_rng(3)
    for shape in [(5, 3, 3, 3), (7, 16, 3, 3), (4, 70, 1, 1), (3, 3, 7, 7), (2, 1, 1, 1)]:
        w = rng.standard_normal(shape).astype(np.float32)
        s = fpo.score_filters(w, norm)
        e = fpo.exact_scores(w, norm)
        np.testing.assert_allclose(s, e, rtol=1e-14)
        w64 = w.astype(np.float64).reshape(shape[0], -1)
        ref = (w64 ** 2).sum(1) if norm else np.abs(w64).sum(1)
        np.testing.assert_allclose(s, ref, rtol=1e-13)


def test_score_summation_order(fpo):
    # values chosen so that the fixed order (32 strided partial sums, then pairwise 16,8,4,2,1)
    # gives a different double than left-to-right summation: 2^53 in slot 0, ones elsewhere
    w = np.zeros((1, 64, 1, 1), dtype=np.float32)
    w[0, 0] = 2.0 ** 53
    w[0, 32] = 1.0          # same partial sum as slot 0: 2^53 + 1 rounds to 2^53
    w[0, 1] = 1.0
    w[0, 33] = 1.0          # partial sum 1 = 2, then combined: 2^53 + 2 is representable
    s = fpo.score_filters(w, fpo.NORM_L1)[0]
    assert s == 2.0 ** 53 + 2.0
    assert fpo.exact_scores(w, 0)[0] == 2.0 ** 53 + 3.0 or fpo.exact_scores(w, 0)[0] == 2.0 ** 53 + 4.0


def test_rank_mask_brute_force_and_ties(fpo):
    rng = np.random.default_rng(4)
    s = rng.standard_normal(37)
    s[5] = s[20] = s[11]                      # a three-way tie
    for q in (0, 1, 11, 36):
        mask, rank = fpo.rank_mask(s, q)
        brute = np.array([sum(1 for j in range(37) if (s[j] < s[k]) or (s[j] == s[k] and j < k)) for k in range(37)])
        np.testing.assert_array_equal(rank, brute)
        assert mask.sum() == 37 - q
        np.testing.assert_array_equal(mask, (brute >= q).astype(np.uint8))
    assert rank[5] < rank[11] < rank[20]      # equal scores: lower index is pruned first


def test_num_pruned(fpo):
    assert fpo.num_pruned(16, 0.3) == 4 and fpo.num_pruned(32, 0.3) == 9 and fpo.num_pruned(64, 0.3) == 19
    assert fpo.num_pruned(10, 0.3) == 3       # 0.3*10 = 2.9999999999999996 in binary
    assert fpo.num_pruned(64, 0.5) == 32 and fpo.num_pruned(64, 0.0) == 0 and fpo.num_pruned(64, 0.4) == 25


def test_mask_popcounts_resnet20(fpo):
    w = wl.workload(1)
    g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
    masks, ranks, scores = fpo.select_masks(g32, w.ratios, fpo.NORM_L1)
    kept = sorted({int(m.sum()) for m in masks.values()})
    assert kept == [12, 23, 45]
    # the fixed summation order never changes a ranking relative to exactly rounded sums
    for ci, op in g32.conv_op.items():
        e = fpo.exact_scores(op["W"], 0)
        m2, r2 = fpo.rank_mask(e, int((masks[ci] == 0).sum()))
        np.testing.assert_array_equal(r2, ranks[ci])


# ---------------------------------------------------------------------------------------
# pruning
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("make,kw", [(wl.tiny_cifar, dict(n_per_stage=2)), (wl.tiny_imagenet_basic, dict()),
                                     (wl.tiny_bottleneck, dict())])
def test_ratio_zero_is_unpruned(fpo, make, kw):
    w = make(p=0.0, **kw)
    g = fpo.fuse(w.net, w.weights, w.bn)
    gp, masks, _, _ = fpo.pruned_model(w.net, w.weights, w.bn, w.ratios)
    assert all(m.all() for m in masks.values())
    np.testing.assert_array_equal(fpo.fused_forward(gp, w.x), fpo.fused_forward(g, w.x))


@pytest.mark.parametrize("make,kw", [(wl.tiny_cifar, dict(n_per_stage=2, p=0.3)),
                                     (wl.tiny_cifar, dict(p=0.5, widths=(7, 12, 23))),
                                     (wl.tiny_imagenet_basic, dict(p=0.3)),
                                     (wl.tiny_bottleneck, dict(p=0.4))])
def test_removal_equals_zeroing(fpo, make, kw):
    w = make(**kw)
    gp, masks, _, _ = fpo.pruned_model(w.net, w.weights, w.bn, w.ratios)
    assert any(not m.all() for m in masks.values())
    removed = fpo.fused_forward(gp, w.x)
    zeroed_fused = fpo.fused_forward(fpo.prune_zero(fpo.fuse(w.net, w.weights, w.bn), masks), w.x)
    wz, bz = fpo.zero_unfused(w.net, w.weights, w.bn, masks)
    zeroed_unfused = fpo.unfused_forward(w.net, wz, bz, w.x)
    assert rel(removed, zeroed_fused) < 1e-12
    assert rel(removed, zeroed_unfused) < 1e-12
    # something was really removed
    ref = fpo.unfused_forward(w.net, w.weights, w.bn, w.x)
    assert rel(removed, ref) > 1e-3
    n_small = sum(op["W"].size for op in gp.ops if op["kind"] == "conv")
    n_full = sum(op["W"].size for op in fpo.fuse(w.net, w.weights, w.bn).ops if op["kind"] == "conv")
    assert n_small < n_full


def test_inner_channels_are_physically_removed(fpo):
    w = wl.tiny_bottleneck(p=0.5)
    gp, masks, _, _ = fpo.pruned_model(w.net, w.weights, w.bn, w.ratios)
    for op in gp.ops:
        if op["kind"] != "conv":
            continue
        prod = [o for o in gp.ops if o["out"] == op["src"]]
        if prod and prod[0]["kind"] == "conv" and prod[0]["scatter"] is None:
            assert op["W"].shape[1] == prod[0]["W"].shape[0]


def test_aggressive_prune_back_equals_plain_chain(fpo):
    """Fused operators lose n-m filters.  With these weights the lowest scores are exactly the
    auxiliary identity filters (score 1), so what remains is the original network with its
    shortcuts gone: a plain convolution chain, evaluated here from a description without adds."""
    w = wl.tiny_cifar(n_per_stage=2, aggressive=True)
    gp, masks, _, scores = fpo.pruned_model(w.net, w.weights, w.bn, w.ratios)
    for ci, op in fpo.fuse(w.net, w.weights, w.bn, "f32").conv_op.items():
        if op["role"] == "aggr1":
            assert masks[ci][:op["n_orig"]].all() and not masks[ci][op["n_orig"]:].any()
            assert scores[ci][:op["n_orig"]].min() > 1.0
    got = fpo.fused_forward(gp, w.x)
    # the same parameters, description rebuilt without shortcuts (same draw order => same offsets)
    plain = wl.Net(3, 8, 8)
    widths, C = (8, 16, 24), 8
    x = plain.relu(plain.bn(plain.conv(-1, 8, 3, 3, 1, 1), 8))
    for si, K in enumerate(widths):
        for bi in range(2):
            st = 2 if (bi == 0 and si > 0) else 1
            x = plain.relu(plain.bn(plain.conv(x, K, C, 3, st, 1), K))
            x = plain.relu(plain.bn(plain.conv(x, K, K, 3, 1, 1), K))
            C = K
    plain.fc(plain.gavgpool(x, C), 5, C)
    assert plain.n_weights == w.net.n_weights and plain.n_bn == w.net.n_bn
    ref = fpo.unfused_forward(plain, w.weights, w.bn, w.x)
    assert rel(got, ref) < 1e-12


def test_planted_mistakes_are_caught(fpo):
    """Each plausible slip in the fusion changes the output by far more than the tolerance the
    equivalence tests use - so those tests would fail if the oracle contained it."""
    w = wl.tiny_cifar(aggressive=True)
    ref = fpo.unfused_forward(w.net, w.weights, w.bn, w.x)
    g = fpo.fuse(w.net, w.weights, w.bn)
    # (a) identity tap off-centre
    h = fpo._copy_graph(g)
    op = [o for o in h.ops if o["kind"] == "conv" and o["role"] == "aggr1"][0]
    K1 = op["n_orig"]
    op["W"][K1:] = np.roll(op["W"][K1:], 1, axis=3)
    assert rel(fpo.fused_forward(h, w.x), ref) > 1e-3
    # (b) folded shift dropped
    h = fpo._copy_graph(g)
    h.ops[0]["b"][:] = 0
    assert rel(fpo.fused_forward(h, w.x), ref) > 1e-3
    # (c) zero-channel padding on the wrong side
    w2 = wl.tiny_cifar(aggressive=False)
    h = fpo.fuse(w2.net, w2.weights, w2.bn)
    for o in h.ops:
        if o["kind"] == "conv" and o["res"] is not None and o["res"]["mode"] == "A":
            o["res"]["pad_lo"] = 3
    assert rel(fpo.fused_forward(h, w2.x), ref) > 1e-3


# ------------------------------------------------------------------------------------------
# dynamic (soft) pruning: the loop of Algorithm 1
# ------------------------------------------------------------------------------------------

def _soft_setup(fpo, p=0.4, aggressive=False):
    w = wl.tiny_cifar(widths=(6, 10, 14), in_hw=8, batch=2, n_per_stage=1, p=p, aggressive=aggressive)
    g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
    return w, g32


def test_soft_epoch_without_update_is_static_selection_plus_zeroing(fpo):
    """With no weight update one epoch selects exactly the masks of the static scheme, zeroizes those filters
    and nothing else; a second epoch then finds the same filters again (their score is exactly 0)."""
    w, g32 = _soft_setup(fpo)
    ref_masks, _, _ = fpo.select_masks(fpo.fuse(w.net, w.weights, w.bn, "f32"), w.ratios, fpo.NORM_L2)
    before = {ci: op["W"].copy() for ci, op in g32.conv_op.items()}
    masks, _, scores = fpo.soft_prune_epoch(g32, w.ratios, fpo.NORM_L2)
    for ci, m in masks.items():
        np.testing.assert_array_equal(m, ref_masks[ci])
        W = g32.conv_op[ci]["W"]
        assert (W[m == 0] == 0).all()
        np.testing.assert_array_equal(W[m == 1], before[ci][m == 1])
    masks2, _, scores2 = fpo.soft_prune_epoch(g32, w.ratios, fpo.NORM_L2)
    for ci in masks:
        np.testing.assert_array_equal(masks2[ci], masks[ci])
        assert (scores2[ci][masks[ci] == 0] == 0).all()


def test_soft_pruned_filter_can_recover(fpo):
    """The point of the dynamic scheme: a zeroized filter that receives a large update is kept in the next epoch,
    and another one takes its place (the number of pruned filters is the same every epoch)."""
    w, g32 = _soft_setup(fpo)
    masks, _, _ = fpo.soft_prune_epoch(g32, w.ratios, fpo.NORM_L2)
    ci = 1
    victim = int(np.nonzero(masks[ci] == 0)[0][0])
    upd = {c: np.zeros_like(op["W"]) for c, op in g32.conv_op.items()}
    upd[ci][victim] = 10.0
    masks2, _, _ = fpo.soft_prune_epoch(g32, w.ratios, fpo.NORM_L2, upd)
    assert masks2[ci][victim] == 1
    assert masks2[ci].sum() == masks[ci].sum()
    assert (masks2[ci] != masks[ci]).sum() == 2


def test_soft_extraction_equals_zeroed_model(fpo):
    """Removing the masked filters of the last epoch gives the same outputs as running the unshrunk model with
    those filters (and their folded shifts) zeroed."""
    w, g32 = _soft_setup(fpo)
    rng = np.random.default_rng(3)
    for _ in range(3):
        upd = {c: (0.05 * rng.standard_normal(op["W"].shape)).astype(np.float32) for c, op in g32.conv_op.items()}
        masks, _, _ = fpo.soft_prune_epoch(g32, w.ratios, fpo.NORM_L2, upd)
    removed = fpo.soft_prune_extract(g32, masks)
    full = fpo.soft_prune_extract(g32, {ci: None for ci in masks})
    zeroed = fpo.prune_zero(full, masks)
    a, b = fpo.fused_forward(removed, w.x), fpo.fused_forward(zeroed, w.x)
    assert np.abs(a - b).max() <= 1e-12 * max(np.abs(b).max(), 1.0)


def test_soft_epoch_fused_operators_lose_n_minus_m(fpo):
    w, g32 = _soft_setup(fpo, p=0.0, aggressive=True)
    masks, _, _ = fpo.soft_prune_epoch(g32, w.ratios, fpo.NORM_L2)
    for ci, m in masks.items():
        if m is None:
            continue
        op = g32.conv_op[ci]
        if op["role"] in ("aggr1", "aggr2"):
            assert int(m.sum()) == op["n_orig"]


# ------------------------------------------------------------------------------------------
# aggressive fusion of bottleneck blocks (the pass-through carried through three convolutions)
# ------------------------------------------------------------------------------------------

def test_aggressive_bottleneck_equals_unfused(fpo):
    w = wl.tiny_bottleneck(aggressive=True)
    g = fpo.fuse(w.net, w.weights, w.bn)
    assert not any(op["kind"] == "conv" and op["res"] is not None for op in g.ops), "an add survived"
    ref = fpo.unfused_forward(w.net, w.weights, w.bn, w.x)
    got = fpo.fused_forward(g, w.x)
    assert np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()
    # and the same as the epilogue form of the same network
    w0 = wl.tiny_bottleneck(aggressive=False)
    np.testing.assert_array_equal(w0.weights, w.weights)
    g0 = fpo.fuse(w0.net, w0.weights, w0.bn)
    assert np.abs(fpo.fused_forward(g0, w.x) - got).max() <= 1e-12 * np.abs(ref).max()


def test_aggressive_bottleneck_loses_n_minus_m(fpo):
    w = wl.tiny_bottleneck(aggressive=True)
    g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
    masks, _, _ = fpo.select_masks(g32, np.zeros(w.net.n_convs()), fpo.NORM_L1)
    n_fused = 0
    for ci, m in masks.items():
        if m is None:
            continue
        op = g32.conv_op[ci]
        if op["role"] in ("aggr1", "aggr2"):
            n_fused += 1
            assert int(m.sum()) == op["n_orig"] and len(m) >= op["n_orig"]
    assert n_fused == 9          # three blocks x three convolutions
    # removal and zeroing of that selection agree
    g = fpo.fuse(w.net, w.weights, w.bn)
    a = fpo.fused_forward(fpo.prune_remove(g, masks), w.x)
    b = fpo.fused_forward(fpo.prune_zero(g, masks), w.x)
    assert np.abs(a - b).max() <= 1e-12 * max(np.abs(b).max(), 1.0)


# ------------------------------------------------------------------------------------------
# the concatenation structure (Sec. IV-B.1): y = concat(conv(x), x)  ->  new_conv(x, [W ; I])
# ------------------------------------------------------------------------------------------

def test_concat_structure_fused_equals_unfused(fpo):
    w = wl.tiny_concat()
    g = fpo.fuse(w.net, w.weights, w.bn)
    convs = [op for op in g.ops if op["kind"] == "conv"]
    assert [op["W"].shape[0] for op in convs] == [8, 6 + 8, 10 + 14, 5 + 24]       # filters: own + pass-through
    assert len(g.ops) == 5                                                          # 4 convolutions + head: no concat left
    ref = fpo.unfused_forward(w.net, w.weights, w.bn, w.x)
    got = fpo.fused_forward(g, w.x)
    assert np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()


def test_concat_identity_filters_reproduce_the_input(fpo):
    """x = xconv(x, W~): the stacked identity filters alone return the block input, channel for channel."""
    rng = np.random.default_rng(2)
    x = np.abs(rng.standard_normal((2, 5, 6, 7)))
    Wt = fpo._identity_filters(5, 5, 3, 3)
    np.testing.assert_array_equal(fpo.conv2d(x, Wt, 1, 1), x)


def test_concat_structure_conservative_pruning(fpo):
    """A fused concatenation operator has n = K + C filters and m = K originally: it loses n - m."""
    w = wl.tiny_concat()
    g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
    masks, _, _ = fpo.select_masks(g32, np.zeros(w.net.n_convs()), fpo.NORM_L1)
    kept = [int(masks[ci].sum()) for ci in sorted(masks)]
    assert kept == [8, 6, 10, 5]
    g = fpo.fuse(w.net, w.weights, w.bn)
    a = fpo.fused_forward(fpo.prune_remove(g, masks), w.x)
    b = fpo.fused_forward(fpo.prune_zero(g, masks), w.x)
    assert np.abs(a - b).max() <= 1e-12 * max(np.abs(b).max(), 1.0)
