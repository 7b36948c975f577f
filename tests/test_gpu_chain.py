"""GPU parity of the fused run-of-layers kernel (a whole stage of 3x3 convolutions with the activations in
shared memory): against the CPU oracle, and against the library's own layer-by-layer path.

The fused kernel is chosen by the library when `keep_outputs` is 0 and a run of stride-1 3x3 convolutions
works on images 8, 16 or 32 pixels wide; with `keep_outputs` = 1 every layer runs on its own.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2010_16165_b200 import workloads as wl
from test_gpu_parity import Gpu, err, oracle_pruned, TOL_BF16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2010_16165_b200 import binding
    binding.lib()
    return binding


CASES = {
    # name: (workload factory, expected number of fused runs at least)
    "cifar32": lambda **k: wl.tiny_cifar(widths=(16, 32, 64), in_hw=32, batch=3, n_per_stage=2, **k),
    "cifar32_odd_widths": lambda **k: wl.tiny_cifar(widths=(7, 12, 23), in_hw=32, batch=5, n_per_stage=1, **k),
    "cifar32_centered_pad": lambda **k: wl.tiny_cifar(widths=(8, 20, 44), in_hw=32, batch=2, n_per_stage=2,
                                                      pad_lo_centered=True, **k),
    "cifar16": lambda **k: wl.tiny_cifar(widths=(16, 24, 40), in_hw=16, batch=9, n_per_stage=3, **k),
    "cifar8_one_stage": lambda **k: wl.tiny_cifar(in_hw=8, batch=2, n_per_stage=2, **k),
    "imagenet_projection": lambda **k: wl.tiny_imagenet_basic(layers=(2, 1, 2), widths=(8, 16, 24), in_hw=128,
                                                              batch=2, **k),
}


def _runs(B, h):
    return sorted({o.chain for o in B.op_infos(h) if o.chain >= 0})


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("p", [0.0, 0.3])
def test_fused_runs_match_oracle_and_layerwise(B, fpo, name, p):
    w = CASES[name](p=p)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, keep_outputs=0)
    g1 = Gpu(B, w, B.FP_COMPUTE_BF16_TC, keep_outputs=1)
    try:
        B.fp_prune(g.h, w.ratios)
        B.fp_prune(g1.h, w.ratios)
        assert len(_runs(B, g.h)) >= 1, "the fused kernel was not selected"
        assert _runs(B, g1.h) == []
        got = g.forward(w.x)
        layerwise = g1.forward(w.x)
        gp, _, _, _ = oracle_pruned(fpo, w)
        ref = fpo.fused_forward(gp, w.x)
        assert err(got, ref) < TOL_BF16
        # same roundings to bf16 at the same places; only the fp32 summation order differs
        assert err(got, layerwise) < 1e-2
        # fewer launches than operators
        assert B.fp_query_int(g.h, B.FP_Q_N_LAUNCHES) < B.fp_query_int(g1.h, B.FP_Q_N_LAUNCHES)
    finally:
        g.close()
        g1.close()


def test_fused_runs_aggressive_fusion(B, fpo):
    """The paper's dilated convolutions (identity filters stacked under conv1, shortcut filters beside conv2)
    run through the fused kernel too: wider layers, no shortcut operand."""
    w = wl.tiny_cifar(widths=(16, 24, 40), in_hw=32, batch=2, n_per_stage=2, aggressive=True, p=0.0)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        assert len(_runs(B, g.h)) >= 1
        assert err(g.forward(w.x), fpo.unfused_forward(w.net, w.weights, w.bn, w.x)) < TOL_BF16
        B.fp_prune(g.h, w.ratios)
        gp, _, _, _ = oracle_pruned(fpo, w)
        assert err(g.forward(w.x), fpo.fused_forward(gp, w.x)) < TOL_BF16
    finally:
        g.close()


def test_fused_runs_batches_and_groups(B, fpo):
    """Batches that do not fill the last group of images, a batch smaller than planned, graph replay."""
    w = wl.tiny_cifar(widths=(16, 32, 64), in_hw=32, batch=11, n_per_stage=1, p=0.3)
    gp, _, _, _ = oracle_pruned(fpo, w)
    ref = fpo.fused_forward(gp, w.x)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC, max_batch=600, use_graph=1)     # 600 images: several images per group
    try:
        B.fp_prune(g.h, w.ratios)
        full = g.forward(w.x)
        assert err(full, ref) < TOL_BF16
        for b in (1, 2, 7):
            np.testing.assert_array_equal(g.forward(w.x[:b]), full[:b])
        st = torch.cuda.Stream()
        np.testing.assert_array_equal(g.forward(w.x, st), full)
        np.testing.assert_array_equal(g.forward(w.x, st), full)
        # many groups per CTA: 600 images, every image a copy of one of the 11
        reps = np.concatenate([w.x] * 55)[:600]
        big = g.forward(reps, st)
        np.testing.assert_array_equal(big, np.concatenate([full] * 55)[:600])
    finally:
        g.close()


def test_intermediate_output_query_is_refused(B):
    w = wl.tiny_cifar(widths=(16, 32, 64), in_hw=32, batch=2, n_per_stage=1)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        g.forward(w.x)
        inside = [i for i, o in enumerate(B.op_infos(g.h)) if o.chain >= 0]
        with pytest.raises(B.FpError) as e:
            B.fp_query_array(g.h, B.FP_Q_OP_OUTPUT, inside[0], np.float32, 2 * 16 * 32 * 32)
        assert e.value.status == B.FP_ERR_UNSUPPORTED
    finally:
        g.close()


def test_fused_runs_non_square_images_and_bf16_input(B, fpo):
    """Images that are not square (24 x 32, then 12 x 16 and 6 x 8), network input given as bf16 NCHW: the first
    fused run converts the layout while it loads."""
    net = wl.resnet_cifar(2, (16, 32, 64), in_hw=32, n_classes=5, name="rect_cifar")
    net.in_H = 24
    w = wl.Workload("rect_cifar", net, 3, 5, True, wl.uniform_ratios(0.3), "uniform 0.3")
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    g1 = Gpu(B, w, B.FP_COMPUTE_BF16_TC, keep_outputs=1)
    try:
        B.fp_prune(g.h, w.ratios)
        B.fp_prune(g1.h, w.ratios)
        assert len(_runs(B, g.h)) == 3
        got = g.forward(w.x)
        gp, _, _, _ = oracle_pruned(fpo, w)
        assert err(got, fpo.fused_forward(gp, w.x)) < TOL_BF16
        assert err(got, g1.forward(w.x)) < 1e-2
        # no layout-conversion launch: 3 runs + 2 strided convolutions + 2 head kernels
        assert B.fp_query_int(g.h, B.FP_Q_N_LAUNCHES) == 7
    finally:
        g.close()
        g1.close()


def test_operator_times_add_up(B):
    """FP_Q_OP_TIMES: one non-negative time per operator, layers inside a run report 0 except the run's first."""
    w = wl.tiny_cifar(widths=(16, 32, 64), in_hw=32, batch=4, n_per_stage=2, p=0.3)
    g = Gpu(B, w, B.FP_COMPUTE_BF16_TC)
    try:
        B.fp_prune(g.h, w.ratios)
        g.forward(w.x)
        ops = B.op_infos(g.h)
        ms = B.fp_query_array(g.h, B.FP_Q_OP_TIMES, 3, np.float32, len(ops))
        assert (ms >= 0).all() and ms.sum() > 0
        seen = set()
        for o, t in zip(ops, ms):
            if o.kind == 0 and o.chain >= 0:
                if o.chain in seen:
                    assert t == 0
                seen.add(o.chain)
    finally:
        g.close()
