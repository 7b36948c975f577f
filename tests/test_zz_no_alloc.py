"""The allocation-free selection entry point against the regular one.

fp_rank_filters_static is for callers that may not allocate device memory (all of it belongs to the
host application's pool, or an allocation's implicit synchronisation is unaffordable).  It must give
exactly the masks and ranks fp_prune gives for the same filters.  The network below has batch norms
that fold to the identity (gamma 1, beta 0, mean 0, variance 1, epsilon below fp32 resolution), so the
filters fp_prune scores are bit for bit the raw filters handed to the new call.  Two calls in a row
share the library's built-in scratch; both must be right.  (Collected last on purpose.)
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2010_16165_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_rank_matches_fp_prune_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2010_16165_b200 import binding as B
    w = wl.tiny_cifar(widths=(16, 24, 40), in_hw=8, batch=2, p=0.3, n_per_stage=2)
    w.net.bn_eps = 1e-12
    for n in w.net.nodes:
        if n["op"] == wl.OP_BN:
            K, o = n["K"], n["bn_off"]
            w.bn[o:o + K] = 1.0
            w.bn[o + K:o + 3 * K] = 0.0
            w.bn[o + 3 * K:o + 4 * K] = 1.0
    dw, dbn = torch.from_numpy(w.weights).cuda(), torch.from_numpy(w.bn).cuda()
    h = B.fp_fuse(w.net, dw, dbn, 2, B.FP_COMPUTE_FP32)
    try:
        conv_nodes = [w.net.nodes[i] for i in w.net.conv_ids()]
        for norm, ratios in ((B.FP_NORM_L1, w.ratios), (B.FP_NORM_L2, np.full(len(conv_nodes), 0.5))):
            B.fp_prune(h, ratios, None, norm)                      # the existing entry point
            want = B.masks_and_ranks(h)
            # two calls in a row on different banks, then compare both
            got = []
            for ci in (1, len(conv_nodes) - 1):
                n = conv_nodes[ci]
                K, per = n["K"], n["C"] * n["R"] * n["S"]
                bank = dw[n["w_off"]:n["w_off"] + K * per]
                rank = torch.full((K,), -1, dtype=torch.int32, device="cuda")
                mask = torch.full((K,), 7, dtype=torch.uint8, device="cuda")
                q = int(np.floor(ratios[ci] * K + 1e-9))
                B.fp_rank_filters_static(bank, K, per, norm, q, rank, mask)
                got.append((ci, rank, mask))
            torch.cuda.synchronize()
            for ci, rank, mask in got:
                np.testing.assert_array_equal(rank.cpu().numpy(), want[ci][1])
                np.testing.assert_array_equal(mask.cpu().numpy(), want[ci][0])
        # sizes beyond the built-in scratch are refused, nothing is launched
        big = torch.zeros(8, device="cuda")
        with pytest.raises(B.FpError) as e:
            B.fp_rank_filters_static(big, B.FP_STATIC_RANK_MAX_FILTERS + 1, 1, 0, 0,
                                     torch.zeros(1, dtype=torch.int32, device="cuda"),
                                     torch.zeros(1, dtype=torch.uint8, device="cuda"))
        assert e.value.status == B.FP_ERR_BOUNDS
    finally:
        B.fp_destroy(h)
