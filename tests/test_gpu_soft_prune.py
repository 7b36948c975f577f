"""GPU parity of the dynamic (soft) filter pruning loop of Algorithm 1: fp_soft_prune_epoch / fp_soft_prune_finish
against the oracle's soft_prune_epoch / soft_prune_extract on the same seeded weight updates.

Masks, ranks and scores are bit-exact (one fp32 addition per weight, the fixed-order fp64 score); the forward of
the extracted model is within the BF16 tolerance.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2010_16165_b200 import workloads as wl
from test_gpu_parity import Gpu, err, TOL_BF16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2010_16165_b200 import binding
    binding.lib()
    return binding


def _updates(g32, rng, scale=0.05):
    return {ci: (scale * rng.standard_normal(op["W"].shape)).astype(np.float32) for ci, op in sorted(g32.conv_op.items())}


def _to_device(upd):
    flat = np.concatenate([upd[ci].ravel() for ci in sorted(upd)])
    return torch.from_numpy(flat).cuda()


def _check_epoch(B, fpo, g, g32, masks, ranks, norm):
    mr = B.masks_and_ranks(g.h)
    for ci, m in masks.items():
        if m is None:
            assert mr[ci][0] is None
            continue
        np.testing.assert_array_equal(mr[ci][0], m)
        np.testing.assert_array_equal(mr[ci][1], ranks[ci])
        # the bank after update + zeroizing: its scores are the same doubles on both sides
        got = B.fp_score(g.h, ci, norm)
        ref = fpo.score_filters(g32.conv_op[ci]["W"], norm)
        assert got.tobytes() == ref.tobytes()
        assert (got[m == 0] == 0).all()


@pytest.mark.parametrize("aggressive", [False, True])
@pytest.mark.parametrize("norm", [0, 1])
def test_soft_pruning_loop_matches_oracle(B, fpo, aggressive, norm):
    w = wl.tiny_cifar(widths=(16, 24, 40), in_hw=16, batch=3, n_per_stage=2, p=0.0 if aggressive else 0.4,
                      aggressive=aggressive)
    g32 = fpo.fuse(w.net, w.weights, w.bn, "f32")
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        sizes = B.conv_bank_elems(g.h)
        for ci in range(w.net.n_convs()):
            assert sizes[ci] == (g32.conv_op[ci]["W"].size if ci in g32.conv_op else 0)
        before = g.forward(w.x)
        rng = np.random.default_rng(17)
        masks = ranks = None
        for epoch in range(3):
            upd = _updates(g32, rng)
            if epoch == 1:                      # bring one zeroized filter of one convolution back
                ci = sorted(g32.conv_op)[1]
                dead = np.nonzero(masks[ci] == 0)[0]
                if len(dead):
                    upd[ci][dead[0]] = 5.0
                    victim = (ci, int(dead[0]))
            B.fp_soft_prune_epoch(g.h, w.ratios, _to_device(upd), norm)
            masks, ranks, _ = fpo.soft_prune_epoch(g32, w.ratios, norm, upd)
            _check_epoch(B, fpo, g, g32, masks, ranks, norm)
            if epoch == 1 and len(dead):
                assert masks[victim[0]][victim[1]] == 1
            # the running graph is untouched until the extraction
            np.testing.assert_array_equal(g.forward(w.x), before)
        B.fp_soft_prune_finish(g.h)
        got = g.forward(w.x)
        ref = fpo.fused_forward(fpo.soft_prune_extract(g32, masks), w.x)
        assert err(got, ref) < TOL_BF16
        assert np.abs(got - before).max() > 1e-3
    finally:
        g.close()


def test_soft_epoch_without_update_selects_like_fp_prune(B, fpo):
    w = wl.tiny_cifar(widths=(16, 32, 64), in_hw=32, batch=2, n_per_stage=1, p=0.3)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    g2 = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        B.fp_prune(g2.h, w.ratios, norm=B.FP_NORM_L1)
        B.fp_soft_prune_epoch(g.h, w.ratios, None, B.FP_NORM_L1)
        a, b = B.masks_and_ranks(g.h), B.masks_and_ranks(g2.h)
        for ci in a:
            np.testing.assert_array_equal(a[ci][0], b[ci][0])
            np.testing.assert_array_equal(a[ci][1], b[ci][1])
        B.fp_soft_prune_finish(g.h)
        # zeroized-then-removed filters: same network as the static scheme
        np.testing.assert_array_equal(g.forward(w.x), g2.forward(w.x))
    finally:
        g.close()
        g2.close()


def test_soft_prune_errors(B):
    w = wl.tiny_cifar(p=0.3)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        with pytest.raises(B.FpError) as e:
            B.fp_soft_prune_finish(g.h)
        assert e.value.status == B.FP_ERR_ARG
        with pytest.raises(B.FpError) as e:
            B.fp_soft_prune_epoch(g.h, np.full(w.net.n_convs(), 1.0), None)
        assert e.value.status == B.FP_ERR_EMPTY_LAYER
        with pytest.raises(B.FpError) as e:
            B.fp_soft_prune_epoch(g.h, np.full(w.net.n_convs(), -0.1), None)
        assert e.value.status == B.FP_ERR_ARG
    finally:
        g.close()
