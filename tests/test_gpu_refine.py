"""The refine pass of the group-mode search: near-ties that the screening arithmetic cannot order.

The inputs are made near-tied on purpose.  Per-token errors do not depend on the importance weights (the scale
statistic sees the activations only), and a loss is linear in the weights, so from the oracle's per-token errors of its
two best candidates a and b one can solve for weights under which loss_b = loss_a * (1 + delta) for any small delta of
either sign: tokens on which a is better are scaled by (1 - t), the others by (1 + t), and t is the root of a linear
equation.  The oracle is then run again on the float32 weights actually handed to the library; what it says is the
expected result.  With |delta| of a few 1e-6 the screening GEMM (delta weights rounded to bf16, each output
accumulated over all of C1 inside the tensor core: up to 6e-5 of a loss) cannot be relied on; the refine pass
re-evaluates the candidates within 1e-4 of the minimum and must reproduce the oracle's argmin and, for those
candidates, its losses to 2e-6.
"""
import numpy as np
import pytest
import torch

from oracle import tlq_oracle as orc
from paper_2602_07899_b200 import workloads as wl

pytestmark = pytest.mark.gpu

REFINED_RTOL = 2e-6       # refined losses against the oracle (the screening tolerance is 2e-3)
HDR_REFINE_COUNT = 7      # int32 word of the workspace header that holds the size of the refine set


@pytest.fixture(scope="module")
def tlq():
    import __graft_entry__ as entry
    entry.build()
    from paper_2602_07899_b200 import tlq as mod
    return mod


def near_tie_weights(per_token, base_w, delta):
    """float32 weights under which the two best candidates (by base_w) are `delta` apart, relative; delta < 0 makes
    the runner-up win.  Returns (weights, a, b)."""
    losses = per_token @ base_w
    a, b = np.argsort(losses, kind="stable")[:2]
    d = per_token[b] - per_token[a] - delta * per_token[a]         # want sum_n w_n d_n = 0
    u = np.where(per_token[b] > per_token[a], -1.0, 1.0)
    t = -np.dot(base_w, d) / np.dot(base_w * u, d)
    assert 0.0 < t < 0.9, t
    return (base_w * (1.0 + t * u)).astype(np.float32), int(a), int(b)


def search(tlq, xb, wb, w32, group, n_grid, flags=0):
    cfg = tlq.config(group_size=group, n_grid=n_grid, flags=flags)
    out = tlq.tlq_scale_search_layer(tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb), torch.from_numpy(w32).cuda(), cfg)
    hdr = out.workspace[:256].view(torch.int32).cpu().numpy()
    assert hdr[0] == 0
    return int(out.best_idx.item()), out.losses.cpu().numpy(), int(hdr[HDR_REFINE_COUNT]), \
        out.s_best.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("n,c1,c2,group,n_grid,seed", [(384, 1024, 256, 128, 12, 301), (300, 4096, 200, 64, 8, 302),
                                                       (1100, 8192, 384, 128, 6, 303),
                                                       # ragged everywhere: 17 k-blocks (chunks of 4, 4, 4, 4, 1), a
                                                       # last output tile of 2 channels, K = 4 (two spare slots)
                                                       (257, 1088, 130, 64, 4, 304),
                                                       # one and a half k-blocks, one chunk
                                                       (200, 96, 72, 32, 5, 306)])
def test_near_ties_are_decided_like_the_oracle(tlq, n, c1, c2, group, n_grid, seed):
    xb, wb, imp = wl.small_case(seed, n, c1, c2, n_outlier=2)
    base = orc.scale_search(xb, wb, imp, "w4a16", group, n_grid)
    per_token = np.asarray(base["per_token"], dtype=np.float64)
    screened_right = 0
    deltas = (2e-6, -2e-6, 5e-6, -5e-6, 2e-5, -2e-5)
    for delta in deltas:
        w32, a, b = near_tie_weights(per_token, np.asarray(imp, dtype=np.float64), delta)
        ref = orc.scale_search(xb, wb, w32, "w4a16", group, n_grid)
        losses_ref = np.asarray(ref["losses"])
        order = np.argsort(losses_ref, kind="stable")
        gap = (losses_ref[order[1]] - losses_ref[order[0]]) / losses_ref[order[0]]
        assert {int(order[0]), int(order[1])} == {a, b} and ref["best"] == (a if delta > 0 else b)
        assert abs(gap - abs(delta)) < 2e-7, (gap, delta)           # the construction hit its target
        best, losses, n_refined, s_best = search(tlq, xb, wb, w32, group, n_grid)
        assert n_refined >= 2
        assert best == ref["best"], (delta, best, ref["best"], losses[[a, b]], losses_ref[[a, b]])
        assert best == int(np.argmin(losses))
        np.testing.assert_allclose(losses[[a, b]], losses_ref[[a, b]], rtol=REFINED_RTOL)
        np.testing.assert_allclose(losses, losses_ref, rtol=2e-3)
        assert np.array_equal(s_best, orc.f32_to_bf16_bits(ref["scales"][best]))
        # the pass does not depend on which screening kernel ran before it
        best_n, losses_n, n_n, _ = search(tlq, xb, wb, w32, group, n_grid, flags=tlq.FLAG_GEMM_NARROW_TILES)
        assert best_n == best and n_n == n_refined
        np.testing.assert_allclose(losses_n[[a, b]], losses_ref[[a, b]], rtol=REFINED_RTOL)
        # the same call without the pass: same losses to the screening tolerance, argmin not asserted
        best0, losses0, n0, _ = search(tlq, xb, wb, w32, group, n_grid, flags=tlq.FLAG_NO_REFINE)
        assert n0 == 0
        np.testing.assert_allclose(losses0, losses_ref, rtol=2e-3)
        screened_right += int(best0 == ref["best"])
        err0 = np.abs(losses0[[a, b]] / losses_ref[[a, b]] - 1).max()
        err1 = np.abs(losses[[a, b]] / losses_ref[[a, b]] - 1).max()
        print(f"C1={c1} delta={delta:+.0e}: screening error {err0:.1e}, refined {err1:.1e}, "
              f"screening argmin {'right' if best0 == ref['best'] else 'WRONG'}")
    print(f"screening alone decided {screened_right} of {len(deltas)} near-ties like the oracle")


def three_way_weights(per_token, base_w, d1, d2):
    """float32 weights under which, with a, b, c the three best candidates by base_w, loss_b = loss_a * (1 + d1) and
    loss_c = loss_a * (1 + d2): two linear conditions, two sign patterns to scale the tokens by."""
    a, b, c = np.argsort(per_token @ base_w, kind="stable")[:3]
    u1 = np.where(per_token[b] > per_token[a], -1.0, 1.0)
    u2 = np.where(per_token[c] > per_token[a], -1.0, 1.0)
    r1 = per_token[b] - (1 + d1) * per_token[a]
    r2 = per_token[c] - (1 + d2) * per_token[a]
    lhs = np.array([[np.dot(base_w * u1, r1), np.dot(base_w * u2, r1)], [np.dot(base_w * u1, r2), np.dot(base_w * u2, r2)]])
    t = np.linalg.solve(lhs, -np.array([np.dot(base_w, r1), np.dot(base_w, r2)]))
    assert np.abs(t).sum() < 0.9, t
    return (base_w * (1.0 + t[0] * u1 + t[1] * u2)).astype(np.float32), [int(a), int(b), int(c)]


@pytest.mark.parametrize("n,c1,c2,group,n_grid,seed", [(640, 2048, 256, 128, 10, 320), (384, 1024, 256, 128, 12, 322)])
def test_three_candidates_near_tied(tlq, n, c1, c2, group, n_grid, seed):
    """Three candidates within 1e-5: all three are evaluated again and come out in the oracle's order."""
    xb, wb, imp = wl.small_case(seed, n, c1, c2, n_outlier=2)
    base = orc.scale_search(xb, wb, imp, "w4a16", group, n_grid)
    w32, abc = three_way_weights(np.asarray(base["per_token"], np.float64), np.asarray(imp, np.float64), 4e-6, -6e-6)
    ref = orc.scale_search(xb, wb, w32, "w4a16", group, n_grid)
    losses_ref = np.asarray(ref["losses"])
    order = [int(i) for i in np.argsort(losses_ref, kind="stable")]
    assert order[:3] == [abc[2], abc[0], abc[1]] and ref["best"] == abc[2]
    gaps = (losses_ref[order[1:4]] - losses_ref[order[0]]) / losses_ref[order[0]]
    assert abs(gaps[0] - 6e-6) < 3e-7 and abs(gaps[1] - 1e-5) < 3e-7 and gaps[2] > 1e-3
    best, losses, n_refined, s_best = search(tlq, xb, wb, w32, group, n_grid)
    assert n_refined == 3 and best == ref["best"]
    assert [int(i) for i in np.argsort(losses, kind="stable")][:3] == order[:3]
    np.testing.assert_allclose(losses[abc], losses_ref[abc], rtol=REFINED_RTOL)
    assert np.array_equal(s_best, orc.f32_to_bf16_bits(ref["scales"][best]))


def test_no_near_tie_means_no_second_evaluation(tlq):
    """Well separated candidates: the refine set stays empty and the results are those of the flagged call, bit for bit."""
    xb, wb, imp = wl.small_case(17, 515, 1088, 777, n_outlier=2)
    ref = orc.scale_search(xb, wb, imp, "w4a16", 64, 7)
    order = np.sort(ref["losses"])
    assert (order[1] - order[0]) / order[0] > 2e-4
    best, losses, n_refined, s_best = search(tlq, xb, wb, np.asarray(imp, np.float32), 64, 7)
    best0, losses0, _, s_best0 = search(tlq, xb, wb, np.asarray(imp, np.float32), 64, 7, flags=tlq.FLAG_NO_REFINE)
    assert n_refined == 0 and best == best0 == ref["best"]
    assert np.array_equal(losses, losses0) and np.array_equal(s_best, s_best0)


def test_refine_with_skipped_tokens_and_exact_ties(tlq):
    """Token skipping on top (the refine GEMM reads the live token count on the device), and a loss curve that is flat
    over all candidates (a constant activation statistic of 1 makes every scale 1)."""
    xb, wb, imp = wl.small_case(305, 640, 2048, 256, n_outlier=2)
    base = orc.scale_search(xb, wb, imp, "w4a16", 128, 8)
    w32, a, b = near_tie_weights(np.asarray(base["per_token"], np.float64), np.asarray(imp, np.float64), -4e-6)
    w32[np.random.default_rng(5).random(640) < 0.3] = 0.0
    ref = orc.scale_search(xb, wb, w32, "w4a16", 128, 8)
    order = np.sort(ref["losses"])
    gap = (order[1] - order[0]) / order[0]
    cfg = tlq.config(n_grid=8, flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS)
    out = tlq.tlq_scale_search_layer(tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb), torch.from_numpy(w32).cuda(), cfg)
    losses = out.losses.cpu().numpy()
    np.testing.assert_allclose(losses, ref["losses"], rtol=2e-3)
    hdr = out.workspace[:256].view(torch.int32).cpu().numpy()
    if gap < 5e-5:
        assert hdr[HDR_REFINE_COUNT] >= 2
    if gap > 1e-6:
        assert int(out.best_idx.item()) == ref["best"]
    # |x| = 1 everywhere: x_stat = 1, every candidate scale is 1, all K losses are equal: more candidates within the
    # band than the pass takes on, so the first evaluation stands as a whole and index 0 wins
    ones = np.full((256, 512), 0x3F80, dtype=np.uint16)
    ones[::2, ::3] = 0xBF80
    best, losses, n_refined, _ = search(tlq, ones, wb[:128, :512].copy(), np.ones(256, np.float32), 128, 6)
    assert best == 0 and np.all(losses == losses[0]) and n_refined == 0
