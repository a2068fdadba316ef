"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot evaluate 20 candidates of an 8192 x 3584 x 18944 layer in fp64 in test time, so the
large linears are checked on sampled outputs it can compute one by one (a token's squared output error
for a given candidate needs only that token's row and the candidate's quantized weights), on whole
weight matrices for the integer codes, and through properties that hold at any size; the small
projections are compared in full."""
import numpy as np
import pytest
import torch

from oracle import tlq_oracle as orc
from paper_2602_07899_b200 import workloads as wl

pytestmark = pytest.mark.gpu
LOSS_RTOL = 2e-3


@pytest.fixture(scope="module")
def tlq():
    import __graft_entry__ as entry
    entry.build()
    from paper_2602_07899_b200 import tlq as mod
    return mod


def assert_same_argmin(best, ref, floor=1e-4):
    """No argmin but the oracle's is accepted; that the oracle's own two best candidates are far enough apart for
    this to be a fair demand is asserted on the seeded data first."""
    order = np.sort(ref["losses"])
    gap = (order[1] - order[0]) / order[0]
    assert gap > floor, f"the oracle's top-2 gap is {gap:.2e}: ambiguous seeded case"
    assert best == ref["best"]


def bits_of(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def gpu_search(tlq, cfgw, xb, wb, imp):
    mode = tlq.W4A16_ASYM_GROUP if cfgw.mode == "w4a16" else tlq.W8A8_SYM
    cfg = tlq.config(mode=mode, group_size=cfgw.group, n_grid=cfgw.n_grid)
    X, W = tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb)
    w_dev = torch.from_numpy(imp).cuda()
    out = tlq.tlq_scale_search_layer(X, W, w_dev, cfg, per_token=True)
    res = dict(best=int(out.best_idx.item()), losses=out.losses.cpu().numpy(), per_token=out.per_token.cpu().numpy(),
               s_best=bits_of(out.s_best), X=X, W=W, cfg=cfg)
    del out
    return res


def check_properties(got, imp, c_out):
    """What must hold at any size: the losses are the weighted means of the per-token table and the
    argmin is the lowest index of the minimum."""
    w = imp.astype(np.float64)
    ref = (got["per_token"].astype(np.float64) * w[None, :]).sum(axis=1) / (c_out * w.sum())
    np.testing.assert_allclose(got["losses"], ref, rtol=2e-5)
    assert got["best"] == int(np.argmin(got["losses"]))
    assert np.all(np.isfinite(got["losses"])) and np.all(got["losses"] > 0)


def check_sampled(got, cfgw, xb, wb, scales, tokens, cands):
    for k in cands:
        e = orc.candidate_error(xb[tokens], wb, scales[k], cfgw.mode, cfgw.group)
        np.testing.assert_allclose(got["per_token"][k, tokens], e, rtol=LOSS_RTOL, atol=1e-30)


def full_compare(tlq, cfgw, lin_name):
    data = wl.LayerData(cfgw)
    lin = cfgw.linear(lin_name)
    xb, wb, imp = data.x(lin), data.w(lin), data.imp()
    ref = orc.scale_search(xb, wb, imp, cfgw.mode, cfgw.group, cfgw.n_grid)
    got = gpu_search(tlq, cfgw, xb, wb, imp)
    np.testing.assert_allclose(got["per_token"], ref["per_token"], rtol=LOSS_RTOL, atol=1e-30)
    np.testing.assert_allclose(got["losses"], ref["losses"], rtol=LOSS_RTOL)
    assert_same_argmin(got["best"], ref)
    assert np.array_equal(got["s_best"], orc.f32_to_bf16_bits(ref["scales"][got["best"]]))
    check_properties(got, imp, lin.c_out)
    return ref, got


@pytest.mark.parametrize("key", ["cfg1", "cfg2"])
def test_7b_k_projection_full(tlq, key):
    full_compare(tlq, wl.config(key), "k")


@pytest.mark.parametrize("key,lin_name,cands,n_tok", [("cfg1", "gate", (0, 9, 19), 48), ("cfg1", "down", (0, 11), 32),
                                                      ("cfg2", "up", (0, 13), 48), ("cfg2", "down", (7,), 32)])
def test_7b_large_linears_sampled(tlq, key, lin_name, cands, n_tok):
    cfgw = wl.config(key)
    data = wl.LayerData(cfgw)
    lin = cfgw.linear(lin_name)
    xb, wb, imp = data.x(lin), data.w(lin), data.imp()
    got = gpu_search(tlq, cfgw, xb, wb, imp)
    check_properties(got, imp, lin.c_out)
    scales = orc.scale_table(orc.channel_stat(xb), cfgw.n_grid)
    assert np.array_equal(got["s_best"], orc.f32_to_bf16_bits(scales[got["best"]]))
    rng = np.random.default_rng(5)
    tokens = np.sort(np.concatenate([rng.choice(cfgw.n_visual, n_tok // 2, replace=False),
                                     cfgw.n_visual + rng.choice(cfgw.n_tokens - cfgw.n_visual, n_tok // 2, replace=False)]))
    check_sampled(got, cfgw, xb, wb, scales, tokens, cands)
    # integer codes of the whole matrix for one candidate, bit for bit
    k = cands[-1]
    s_dev = tlq.bf16_from_bits(orc.f32_to_bf16_bits(scales[k]))
    q = tlq.tlq_quantize_weights(got["W"], s_dev, got["cfg"])
    if cfgw.mode == "w4a16":
        codes, step, zero, _ = orc.quantize_weights_group_asym(wb, scales[k], cfgw.group)
        assert np.array_equal(q["zeros"].cpu().numpy(), zero)
    else:
        codes, step = orc.quantize_weights_row_sym(wb, scales[k])
        qa, ta = tlq.tlq_quantize_activations(got["X"][:2048], s_dev, got["cfg"])
        qx, t = orc.quantize_activations_token_sym(xb[:2048], scales[k])
        assert np.array_equal(qa.cpu().numpy(), qx) and np.array_equal(ta.cpu().numpy(), t)
    assert np.array_equal(q["codes"].cpu().numpy(), codes)
    assert np.array_equal(q["steps"].cpu().numpy(), step)


def test_72b_shapes_sampled(tlq):
    cfgw = wl.config("cfg3")
    data = wl.LayerData(cfgw)
    # kv projection: all candidates on sampled tokens; gate (ragged last output tile: 29568 = 115.5 x 256):
    # properties + one candidate on a few tokens
    for lin_name, cands, n_tok in (("k", tuple(range(20)), 64), ("gate", (6,), 16)):
        lin = cfgw.linear(lin_name)
        xb, wb, imp = data.x(lin), data.w(lin), data.imp()
        got = gpu_search(tlq, cfgw, xb, wb, imp)
        check_properties(got, imp, lin.c_out)
        scales = orc.scale_table(orc.channel_stat(xb), cfgw.n_grid)
        tokens = np.sort(np.random.default_rng(9).choice(cfgw.n_tokens, n_tok, replace=False))
        check_sampled(got, cfgw, xb, wb, scales, tokens, cands)
        if lin_name == "k":
            # with every candidate evaluated on the sample, the sample's own argmin must agree
            sub = np.stack([orc.candidate_error(xb[tokens], wb, scales[k], "w4a16", 128) for k in range(20)])
            w = imp[tokens].astype(np.float64)
            np.testing.assert_allclose((got["per_token"][:, tokens] * w).sum(axis=1), (sub * w).sum(axis=1), rtol=LOSS_RTOL)
        del got
        data.drop(lin)
        torch.cuda.empty_cache()


@pytest.mark.parametrize("mode,group,imp_kind", [("w4a16", 64, "uniform"), ("w4a16", 128, "onehot"),
                                                 ("w4a16", 64, "lognormal"), ("w8a8", 128, "lognormal"),
                                                 ("w8a8", 128, "onehot")])
@pytest.mark.parametrize("n_tokens", [1024, 4096])
def test_2b_sweep_cells_full(tlq, mode, group, imp_kind, n_tokens):
    cfgw = wl.config("cfg4", mode=mode, group=group, imp_kind=imp_kind, n_tokens=n_tokens)
    for lin_name in ("k", "o"):
        if lin_name == "o" and n_tokens > 1024:
            continue
        full_compare(tlq, cfgw, lin_name)


@pytest.mark.parametrize("mode", ["w4a16", "w8a8"])
def test_2b_64k_tokens_sampled(tlq, mode):
    cfgw = wl.config("cfg4", mode=mode, n_tokens=65536)
    data = wl.LayerData(cfgw)
    lin = cfgw.linear("down")                      # 8960 -> 1536: the largest activation tensor of the sweep
    xb, wb, imp = data.x(lin), data.w(lin), data.imp()
    got = gpu_search(tlq, cfgw, xb, wb, imp)
    check_properties(got, imp, lin.c_out)
    scales = orc.scale_table(orc.channel_stat(xb), cfgw.n_grid)
    assert np.array_equal(got["s_best"], orc.f32_to_bf16_bits(scales[got["best"]]))
    tokens = np.sort(np.random.default_rng(3).choice(cfgw.n_tokens, 96, replace=False))
    check_sampled(got, cfgw, xb, wb, scales, tokens, (0, 8, 19))


def test_7b_k_projection_full_paper_settings(tlq):
    """The paper's own setting on the 7B k-projection at full size: W4A8 with the top-50 % token set as 0/1
    weights, zero-weight tokens skipped on the device."""
    cfgw = wl.config("cfg1", mode="w4a8")
    data = wl.LayerData(cfgw)
    lin = cfgw.linear("k")
    xb, wb, imp = data.x(lin), data.w(lin), data.imp()
    mask = (imp >= np.sort(imp)[len(imp) // 2]).astype(np.float32)
    ref = orc.scale_search(xb, wb, mask, "w4a8", 0, cfgw.n_grid)
    cfg = tlq.config(tlq.WA_SYM_CHANNEL, w_bits=4, a_bits=8, n_grid=cfgw.n_grid, flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS)
    out = tlq.tlq_scale_search_layer(tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb), torch.from_numpy(mask).cuda(), cfg)
    np.testing.assert_allclose(out.losses.cpu().numpy(), ref["losses"], rtol=LOSS_RTOL)
    assert_same_argmin(int(out.best_idx.item()), ref)


@pytest.mark.parametrize("key", ["cfg1", "cfg2"])
def test_7b_k_projection_full_two_streams(tlq, key):
    """Two activation streams at full size: the quantized stream is the full-precision one with a 2 % relative
    perturbation (rounded to bf16)."""
    cfgw = wl.config(key)
    data = wl.LayerData(cfgw)
    lin = cfgw.linear("k")
    xf, wb, imp = data.x(lin), data.w(lin), data.imp()
    noise = np.random.default_rng(9).standard_normal(xf.shape).astype(np.float32)
    xq = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(xf) * (1.0 + 0.02 * noise))
    ref = orc.scale_search(xq, wb, imp, cfgw.mode, cfgw.group, cfgw.n_grid, x_fp_bits=xf)
    mode = tlq.W4A16_ASYM_GROUP if cfgw.mode == "w4a16" else tlq.W8A8_SYM
    cfg = tlq.config(mode=mode, group_size=cfgw.group, n_grid=cfgw.n_grid)
    out = tlq.tlq_scale_search_layer(tlq.bf16_from_bits(xq), tlq.bf16_from_bits(wb), torch.from_numpy(imp).cuda(), cfg,
                                     per_token=True, X_fp=tlq.bf16_from_bits(xf))
    np.testing.assert_allclose(out.per_token.cpu().numpy(), ref["per_token"], rtol=LOSS_RTOL, atol=1e-30)
    np.testing.assert_allclose(out.losses.cpu().numpy(), ref["losses"], rtol=LOSS_RTOL)
    assert_same_argmin(int(out.best_idx.item()), ref)
