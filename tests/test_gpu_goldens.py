"""GPU parity at the benchmark's full sizes against stored oracle results, every linear of the layer.

tests/golden/fullsize/<cell>_<linear>.npz was written by tests/golden/make_goldens.py, which calls only the
CPU oracle on the seeded workloads: all K losses, the argmin, the relative gap between the two smallest
losses and the per-token errors of a seeded token sample.  Here the same tensors are generated again, the
search runs once through the C ABI in the launch configuration bench.py times (default flags, all K
candidates in one call), and the results must agree: argmin and winning scale exactly, losses and the
sampled per-token errors within the stated 2e-3.  No argmin other than the oracle's is accepted; that this
is a fair demand (the oracle's own two best candidates are never closer than the arithmetic can resolve) is
asserted on the stored gaps by the CPU test at the end of the file.
"""
import glob
import os

import numpy as np
import pytest
import torch

from oracle import tlq_oracle as orc
from paper_2602_07899_b200 import workloads as wl

LOSS_RTOL = 2e-3
# What decides whether the CUDA path can reproduce an argmin is how differently its arithmetic (bf16 rounding of the
# delta-weight operand, fp32 accumulation in tensor memory) shifts the losses of the oracle's two best candidates.
# Measured on every stored linear: that difference is at most 2.3e-5 relative (the 256-row key / value projections of
# the 2B-class sweep) and at most 6e-6 for projections of 1536 rows and more, never more than a seventh of the
# oracle's own gap.  An oracle gap below the floor would make "identical argmin" a coin toss rather than a property
# of the method.
GAP_FLOOR = 4e-5
REFINED_RTOL = 2e-6        # losses of candidates the refine pass re-evaluated
HDR_REFINE_COUNT = 7       # int32 word of the workspace header that holds the size of the refine set
GOLDEN_DIR = os.path.join(os.path.dirname(__file__), "golden", "fullsize")
ORDER = {n: i for i, n in enumerate(("q", "k", "v", "o", "gate", "up", "down"))}


def golden_cases():
    out = []
    for path in sorted(glob.glob(os.path.join(GOLDEN_DIR, "*.npz"))):
        cell, lin = os.path.basename(path)[:-4].rsplit("_", 1)
        out.append((cell, lin))
    return sorted(out, key=lambda c: (c[0], ORDER[c[1]]))


CASES = golden_cases()


def load_golden(cell, lin):
    with np.load(os.path.join(GOLDEN_DIR, f"{cell}_{lin}.npz")) as z:
        return {k: z[k] for k in z.files}


def cell_config(cell, g):
    n_tokens, _, _, n_grid = (int(v) for v in g["shape"])
    return wl.config(cell.split("_")[0], n_tokens=n_tokens, mode=str(g["mode"]), group=int(g["group"]),
                     imp_kind=str(g["imp_kind"]), n_grid=n_grid)


@pytest.fixture(scope="module")
def tlq():
    import __graft_entry__ as entry
    entry.build()
    from paper_2602_07899_b200 import tlq as mod
    return mod


@pytest.fixture(scope="module")
def layer_data():
    """One LayerData per cell at a time: sibling linears share their activation tensor, the previous cell's
    tensors are dropped."""
    cache = {}

    def get(cell, cfgw):
        if cell not in cache:
            cache.clear()
            cache[cell] = wl.LayerData(cfgw)
        return cache[cell]
    return get


@pytest.mark.gpu
@pytest.mark.parametrize("cell,lin_name", CASES, ids=[f"{c}-{l}" for c, l in CASES])
def test_full_size_search_matches_stored_oracle(tlq, layer_data, cell, lin_name):
    g = load_golden(cell, lin_name)
    cfgw = cell_config(cell, g)
    lin = cfgw.linear(lin_name)
    assert [cfgw.n_tokens, lin.c_in, lin.c_out, cfgw.n_grid] == [int(v) for v in g["shape"]]
    data = layer_data(cell, cfgw)
    xb, wb, imp = data.x(lin), data.w(lin), data.imp()
    mode = tlq.W4A16_ASYM_GROUP if cfgw.mode == "w4a16" else tlq.W8A8_SYM
    cfg = tlq.config(mode=mode, group_size=cfgw.group, n_grid=cfgw.n_grid)
    out = tlq.tlq_scale_search_layer(tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb), torch.from_numpy(imp).cuda(), cfg,
                                     per_token=True)
    losses = out.losses.cpu().numpy()
    best = int(out.best_idx.item())
    n_refined = int(out.workspace[:256].view(torch.int32).cpu().numpy()[HDR_REFINE_COUNT])
    tokens = g["tokens"]
    per_token = out.per_token[:, torch.from_numpy(tokens).cuda()].cpu().numpy()
    s_best = out.s_best.view(torch.int16).cpu().numpy().view(np.uint16)
    del out
    data.drop(lin)
    torch.cuda.empty_cache()
    np.testing.assert_allclose(losses, g["losses"], rtol=LOSS_RTOL)
    np.testing.assert_allclose(per_token, g["per_token"], rtol=LOSS_RTOL, atol=1e-30)
    assert best == int(g["best"]), (best, int(g["best"]), float(g["gap"]))
    assert best == int(np.argmin(losses))
    assert np.array_equal(s_best, g["scale_best"])
    # the refine pass takes on candidates within this relative distance of the screened minimum
    band = max(1e-4, 3.2e-3 / np.sqrt(lin.c_out))
    if cfgw.mode == "w4a16" and float(g["gap"]) < band - 3e-5:
        # close enough for the second, more exact evaluation to have run on the two best candidates: their losses
        # must then match the oracle's to its accuracy, not just to the screening tolerance
        assert n_refined >= 2
        top2 = np.argsort(g["losses"], kind="stable")[:2]
        np.testing.assert_allclose(losses[top2], g["losses"][top2], rtol=REFINED_RTOL)
    if cfgw.mode != "w4a16" or float(g["gap"]) > band + 1e-4:
        assert n_refined == 0


def test_stored_goldens_are_complete_and_their_argmin_is_resolvable():
    """CPU check of the stored files themselves: every linear of the 7B-class layer in both settings is there,
    the stored argmin is the lowest index of the stored minimum, and no stored top-2 gap is below the floor."""
    have = set(CASES)
    for cell in ("cfg1", "cfg2"):
        for lin in ORDER:
            assert (cell, lin) in have, f"missing golden {cell}_{lin}: run tests/golden/make_goldens.py"
    smallest = None
    for cell, lin in CASES:
        g = load_golden(cell, lin)
        losses = g["losses"]
        assert np.all(np.isfinite(losses)) and np.all(losses > 0)
        assert int(g["best"]) == orc.argmin_lowest(losses)
        order = np.sort(losses)
        gap = float((order[1] - order[0]) / order[0])
        assert gap == pytest.approx(float(g["gap"]), rel=1e-12)
        assert gap > GAP_FLOOR, (cell, lin, gap)
        assert g["per_token"].shape == (len(losses), len(g["tokens"]))
        if smallest is None or gap < smallest[0]:
            smallest = (gap, cell, lin)
    print("smallest stored top-2 gap:", smallest)
