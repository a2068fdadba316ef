"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle itself.

Each test is chosen so that a plausible slip in oracle/tlq_oracle.py (a dropped term, a wrong sign or
axis, a transposed operand, a wrong rounding rule) fails it.  No GPU, no CUDA library.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import brute
from oracle import tlq_oracle as orc
from paper_2602_07899_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")


def paper_facts():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = [t.strip() for t in line.split("=")]
                out[k] = float(v)
    return out


def bits(a):
    return wl.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


# ------------------------------------------------------------------ bf16 rounding / scale table


def test_round_to_bf16_ties_and_library():
    # ties go to the even significand; 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -30, 3.0, 0.1])
    r = orc.round_to_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 + 2.0 ** -6 and r[2] == 1.0 + 2.0 ** -7 and r[3] == 3.0
    # special case that reduces to a library routine: float32 inputs through torch's conversion
    v = np.random.default_rng(1).standard_normal(20000).astype(np.float32) * 37.0
    ref = torch.from_numpy(v).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(orc.round_to_bf16(v.astype(np.float64)), ref)
    # and the scalar integer-arithmetic rounding of the brute-force program
    for t in np.abs(v[:500]).astype(np.float64) + 1e-3:
        assert brute.to_bf16(float(t)) == float(orc.round_to_bf16(np.array([t]))[0])


def test_channel_stat_closed_forms():
    n, c = 12, 8
    sign = np.where(np.arange(n)[:, None] % 2 == 0, 1.0, -1.0)
    x = sign * (np.arange(c)[None, :] + 1.0) * np.where(np.arange(n)[:, None] < 4, 2.0, 1.0)
    xb = bits(x)
    # rows 0..3 are doubled: mean |x_c| = (c+1) * (4*2 + 8*1)/12, max = 2(c+1)
    assert np.allclose(orc.channel_stat(xb, orc.STAT_MEAN_ABS), (np.arange(c) + 1) * 16.0 / 12.0, rtol=0, atol=1e-15)
    assert np.array_equal(orc.channel_stat(xb, orc.STAT_MAX_ABS), 2.0 * (np.arange(c) + 1))
    mask = np.zeros(n, np.uint8)
    mask[6:] = 1   # only undoubled rows selected
    assert np.array_equal(orc.channel_stat(xb, orc.STAT_MASKED_MAX, mask), 1.0 * (np.arange(c) + 1))


def test_scale_table_grid_and_exponent():
    stat = np.array([4.0, 16.0, 0.25, 1.0, 0.0])
    tab = orc.scale_table(stat, 4)           # r = 0, 1/4, 1/2, 3/4
    assert np.array_equal(tab[0], np.ones(5, np.float32))        # r = 0 -> scale 1 (plain RTN row)
    assert np.array_equal(tab[2][:4], np.array([2.0, 4.0, 0.5, 1.0], np.float32))   # square roots
    assert tab[1][1] == 2.0 and tab[3][1] == 8.0                  # 16^(1/4), 16^(3/4)
    assert tab[2][4] == np.float32(2.0 ** -10)                    # dead channel floored at 2^-20
    assert orc.grid_ratio(19, 20) == 19 / 20 and orc.grid_ratio(0, 20) == 0.0
    # every entry is a bfloat16 value
    t = orc.scale_table(np.abs(np.random.default_rng(0).standard_normal(64)) + 0.01, 20)
    assert np.array_equal(wl.bf16_bits_to_f32(orc.f32_to_bf16_bits(t)), t)


# ------------------------------------------------------------------ quantizers


def test_symmetric_quantizer_matches_paper_definition():
    facts = paper_facts()
    rng = np.random.default_rng(3)
    v = rng.standard_normal((16, 40)).astype(np.float32)
    q, step = orc.quantize_sym_rows(v, 8)
    assert q.min() >= facts["int8_range_lo"] and q.max() <= facts["int8_range_hi"]
    amax_pos = np.abs(v).argmax(axis=1)
    for i in range(16):
        # s_i = max_j |X_ij| / (2^(n-1)-1); the largest element lands on +-127
        assert math.isclose(step[i], np.abs(v[i]).max() / facts["sym_levels_n8"], rel_tol=1e-6)
        assert abs(int(q[i, amax_pos[i]])) == int(facts["sym_levels_n8"])
        # round(X / s): independent scalar evaluation in binary64 (off by at most rounding of the quotient)
        for j in range(40):
            assert abs(int(q[i, j]) - v[i, j] / step[i]) <= 0.5 + 1e-4
    # other widths: 6-bit activations use [-32, 31], largest at +-31
    q6, _ = orc.quantize_sym_rows(v, 6)
    assert q6.min() >= -32 and q6.max() <= 31 and np.all(np.abs(q6).max(axis=1) == 31)


def test_exactly_representable_inputs_have_zero_error():
    # weights already on a 16-level grid with power-of-two step: the group quantizer must return them
    rng = np.random.default_rng(5)
    c2, c1, g = 6, 64, 32
    lvl = rng.integers(0, 16, size=(c2, c1))
    lvl[:, ::g] = 0
    lvl[:, 1::g] = 15                       # each group spans the whole grid
    w = (lvl - 5) * 2.0 ** -6
    codes, step, zero, w_hat = orc.quantize_weights_group_asym(bits(w), None, g)
    assert np.all(step == np.float32(2.0 ** -6)) and np.all(zero == 5)
    assert np.array_equal(codes, lvl.astype(np.uint8))
    assert np.array_equal(w_hat.astype(np.float64), w)
    x = rng.standard_normal((9, c1))
    e = orc.per_token_error(orc.layer_fp(bits(x), bits(w)), orc.layer_q_w4a16(bits(x), w_hat))
    assert np.all(e == 0.0)
    # int8 rows: integers times 2^-7 with +-127 present -> step exactly 2^-7, codes = the integers
    li = rng.integers(-127, 128, size=(c2, c1))
    li[:, 0] = 127
    qw, u = orc.quantize_weights_row_sym(bits(li * 2.0 ** -7), None)
    assert np.all(u == np.float32(2.0 ** -7)) and np.array_equal(qw, li.astype(np.int8))
    xi = rng.integers(-127, 128, size=(9, c1))
    xi[:, 3] = -127
    qx, t = orc.quantize_activations_token_sym(bits(xi * 2.0 ** -5), None)
    assert np.all(t == np.float32(2.0 ** -5)) and np.array_equal(qx, xi.astype(np.int8))
    yq = orc.layer_q_w8a8(qx, t, qw, u)
    assert np.array_equal(yq, (xi * 2.0 ** -5) @ (li * 2.0 ** -7).T)


def test_group_quantizer_codes_are_nearest_levels_brute_force():
    # exhaustive: for the step / zero-point the oracle reports, its code is the closest level among all 2^n
    x, w, _ = wl.small_case(11, 8, 16, 5)
    s = orc.scale_table(orc.channel_stat(x), 4)[2]
    for nbits in (3, 4):
        codes, step, zero, w_hat = orc.quantize_weights_group_asym(w, s, 8, nbits)
        p = (orc.bf16_to_f64(w) * s.astype(np.float64)[None, :])
        qmax = (1 << nbits) - 1
        for o in range(5):
            for c in range(16):
                g = c // 8
                best = brute.nearest_level(float(p[o, c]), float(step[o, g]), int(zero[o, g]), qmax)
                assert int(codes[o, c]) in best
                # dequantized weight is (q - z) * step / s
                assert math.isclose(float(w_hat[o, c]), (int(codes[o, c]) - int(zero[o, g])) * float(step[o, g]) / float(s[c]),
                                    rel_tol=3e-7, abs_tol=1e-12)
            # affine grid covers the group's range: min maps to code 0 or the zero-point clamps
            for g in range(2):
                pg = p[o, g * 8:(g + 1) * 8]
                assert math.isclose(float(step[o, g]), max(pg.max() - pg.min(), 1e-5) / qmax, rel_tol=2e-7)


def test_all_positive_group_clamps_zero_point():
    # reading: the zero-point is an n-bit integer; a group without sign change clips at the range ends
    w = np.linspace(0.5, 1.0, 16)[None, :]
    codes, step, zero, w_hat = orc.quantize_weights_group_asym(bits(w), None, 16)
    assert zero[0, 0] == 0 and codes.max() == 15
    wneg = -w
    codes, step, zero, w_hat = orc.quantize_weights_group_asym(bits(wneg), None, 16)
    assert zero[0, 0] == 15 and codes.min() == 0


def test_fixed_parameter_idempotency_and_requantization():
    x, w, _ = wl.small_case(7, 64, 256, 24)
    s = orc.scale_table(orc.channel_stat(x), 20)[9]
    codes, step, zero, w_hat = orc.quantize_weights_group_asym(w, s, 128)
    g = 128
    dq = (codes.astype(np.int64).reshape(24, 2, g) - zero[:, :, None]).astype(np.float32) * step[:, :, None]
    # quantize(dequantize(codes)) with the same step / zero-point returns the codes
    again = np.clip(np.rint((dq / step[:, :, None]).astype(np.float32)).astype(np.int64) + zero[:, :, None], 0, 15)
    assert np.array_equal(again.reshape(24, 256), codes.astype(np.int64))
    # quantize -> dequantize -> quantize with re-estimated parameters: groups whose codes span [0,15]
    # reproduce codes and zero-point (dq is exactly representable in bf16? no -> feed float values through p directly)
    full = (codes.reshape(24, 2, g).min(axis=2) == 0) & (codes.reshape(24, 2, g).max(axis=2) == 15)
    assert full.mean() > 0.9
    mx, mn = dq.max(axis=2), dq.min(axis=2)
    step2 = ((mx - mn).astype(np.float32) / np.float32(15)).astype(np.float32)
    zero2 = np.clip(-np.rint((mn / step2).astype(np.float32)).astype(np.int64), 0, 15)
    codes2 = np.clip(np.rint((dq / step2[:, :, None]).astype(np.float32)).astype(np.int64) + zero2[:, :, None], 0, 15)
    assert np.array_equal(zero2[full], zero[full])
    assert np.array_equal(codes2[full], codes.reshape(24, 2, g).astype(np.int64)[full])
    # symmetric int8: same property (the amax element is +-127 so the step is reproduced)
    qw, u = orc.quantize_weights_row_sym(w, s)
    deq = qw.astype(np.float32) * u[:, None]
    qw2, u2 = orc.quantize_sym_rows(deq, 8)
    assert np.array_equal(qw2, qw) and np.allclose(u2, u, rtol=2e-7)


def test_rounding_error_variance_is_step_squared_over_12():
    facts = paper_facts()
    rng = np.random.default_rng(9)
    c2, c1, g = 64, 1024, 128
    w = rng.uniform(-1, 1, size=(c2, c1))
    wb = bits(w)
    codes, step, zero, w_hat = orc.quantize_weights_group_asym(wb, None, g, 4)
    err = (orc.bf16_to_f64(wb) - w_hat.astype(np.float64)).reshape(c2, c1 // g, g)
    ratio = (err ** 2).mean(axis=2) / (step.astype(np.float64) ** 2)
    assert abs(ratio.mean() - facts["rtn_error_var_over_step2"]) < 0.004
    # more bits -> error shrinks with the square of the step (15/255)^2
    _, step8, _, w_hat8 = orc.quantize_weights_group_asym(wb, None, g, 8)
    e8 = ((orc.bf16_to_f64(wb) - w_hat8.astype(np.float64)) ** 2).mean()
    assert abs(e8 / (err ** 2).mean() / (15.0 / 255.0) ** 2 - 1.0) < 0.1


def test_power_of_two_rescale_of_scale_is_invisible():
    x, w, imp = wl.small_case(13, 48, 128, 16)
    s = orc.scale_table(orc.channel_stat(x), 20)[11]
    c1, s1, z1, wh1 = orc.quantize_weights_group_asym(w, s, 64)
    c2, s2, z2, wh2 = orc.quantize_weights_group_asym(w, s * np.float32(8.0), 64)
    assert np.array_equal(c1, c2) and np.array_equal(z1, z2) and np.array_equal(s1 * np.float32(8), s2)
    assert np.array_equal(wh1, wh2)
    e1 = orc.candidate_error(x, w, s, "w8a8", 0)
    e2 = orc.candidate_error(x, w, s * np.float32(0.25), "w8a8", 0)
    assert np.allclose(e1, e2, rtol=1e-12)


# ------------------------------------------------------------------ smoothing identity, objective


def test_smoothing_identity_and_scale_axis():
    # Y = (X diag(s)^-1)(diag(s) W): the scale multiplies W's input-channel axis (columns of W in C2 x C1)
    rng = np.random.default_rng(2)
    x = rng.standard_normal((7, 12))
    w = rng.standard_normal((5, 12))
    s = np.abs(rng.standard_normal(12)) + 0.5
    xb, wb = bits(x), bits(w)
    y = orc.layer_fp(xb, wb)
    xv, wv = orc.bf16_to_f64(xb), orc.bf16_to_f64(wb)
    for n in range(7):
        for o in range(5):
            acc = 0.0
            for c in range(12):
                acc += (xv[n, c] / s[c]) * (s[c] * wv[o, c])
            assert math.isclose(acc, y[n, o], rel_tol=1e-12, abs_tol=1e-12)
    b = rng.standard_normal(5)
    assert np.allclose(orc.layer_fp(xb, wb, b) - y, b[None, :], atol=1e-12)
    # a quantizer that returns its input leaves no error: w_hat = W
    assert np.all(orc.per_token_error(y, orc.layer_q_w4a16(xb, wv)) == 0.0)


def _direct_mse(x, w, s, group):
    """Plain MSE from the integer outputs only (codes, step, zero-point), explicit dequantization."""
    codes, step, zero, _ = orc.quantize_weights_group_asym(w, s, group)
    c2, c1 = codes.shape
    deq = (codes.astype(np.float64).reshape(c2, c1 // group, group) - zero[:, :, None]) * step.astype(np.float64)[:, :, None]
    w_eff = deq.reshape(c2, c1) / s.astype(np.float64)[None, :]
    xv = orc.bf16_to_f64(x)
    d = xv @ orc.bf16_to_f64(w).T - xv @ w_eff.T
    return d


def test_uniform_onehot_and_subset_importance():
    x, w, imp = wl.small_case(21, 40, 128, 24)
    res_u = orc.scale_search(x, w, np.full(40, 3.7, np.float32), group=64, n_grid=6)
    res_n = orc.scale_search(x, w, None, group=64, n_grid=6)
    assert np.allclose(res_u["losses"], res_n["losses"], rtol=1e-13)
    for k in range(6):
        d = _direct_mse(x, w, res_u["scales"][k], 64)
        assert math.isclose(res_u["losses"][k], (d ** 2).mean(), rel_tol=2e-6)    # uniform -> plain MSE
        assert np.allclose(res_u["per_token"][k], (d ** 2).sum(axis=1), rtol=2e-6)
    j = 17
    hot = np.zeros(40, np.float32)
    hot[j] = 5.0
    res_h = orc.scale_search(x, w, hot, group=64, n_grid=6)
    assert np.allclose(res_h["losses"], res_u["per_token"][:, j] / 24.0, rtol=1e-13)   # one-hot -> that token
    sel = np.zeros(40, np.float32)
    sel[5:25] = 1.0
    res_s = orc.scale_search(x, w, sel, group=64, n_grid=6)
    assert np.allclose(res_s["losses"], res_u["per_token"][:, 5:25].mean(axis=1) / 24.0, rtol=1e-13)
    # weights act linearly and the normalisation removes their overall size
    res_w = orc.scale_search(x, w, imp, group=64, n_grid=6)
    ref = (res_u["per_token"] * imp.astype(np.float64)[None, :]).sum(axis=1) / (24.0 * imp.astype(np.float64).sum())
    assert np.allclose(res_w["losses"], ref, rtol=1e-13)
    assert res_w["best"] == int(np.argmin(ref))


def test_gram_route_agrees_with_direct_route():
    # sum_n w_n ||x_n dW^T||^2 = tr(dW H dW^T), H = sum_n w_n x_n x_n^T (linear in dW when Q_a = id)
    x, w, imp = wl.small_case(31, 96, 128, 20)
    res = orc.scale_search(x, w, imp, group=128, n_grid=5)
    xv, wv = orc.bf16_to_f64(x), orc.bf16_to_f64(w)
    h = (xv * imp.astype(np.float64)[:, None]).T @ xv
    for k in range(5):
        _, _, _, w_hat = orc.quantize_weights_group_asym(w, res["scales"][k], 128)
        dw = wv - w_hat.astype(np.float64)
        gram = np.trace(dw @ h @ dw.T) / (20.0 * imp.astype(np.float64).sum())
        assert math.isclose(gram, res["losses"][k], rel_tol=1e-9)


def test_first_candidate_is_plain_rtn():
    x, w, imp = wl.small_case(41, 32, 128, 12)
    res = orc.scale_search(x, w, imp, group=64, n_grid=4)
    assert np.all(res["scales"][0] == 1.0)
    e0 = orc.candidate_error(x, w, None, "w4a16", 64)
    assert np.array_equal(e0, res["per_token"][0])
    res8 = orc.scale_search(x, w, imp, mode="w8a8", n_grid=4)
    assert np.array_equal(orc.candidate_error(x, w, None, "w8a8", 0), res8["per_token"][0])


@pytest.mark.parametrize("mode", ["w4a16", "w8a8", "w4a8", "w4a6"])
def test_search_agrees_with_scalar_brute_force(mode):
    x, w, imp = wl.small_case(51, 5, 8, 3)
    res = orc.scale_search(x, w, imp, mode=mode, group=4, n_grid=4, w_bits_n=3 if mode == "w4a16" else 4)
    best, losses, table = brute.search(x.tolist(), w.tolist(), [float(v) for v in imp], 4, 4, 3, mode)
    assert best == res["best"]
    assert np.allclose(losses, res["losses"], rtol=1e-11)
    assert np.allclose(np.array(table), res["per_token"], rtol=1e-11, atol=1e-18)


def test_w8a8_error_matches_explicit_dequantization():
    x, w, imp = wl.small_case(61, 24, 64, 10)
    s = orc.scale_table(orc.channel_stat(x), 20)[10]
    qw, u = orc.quantize_weights_row_sym(w, s)
    qx, t = orc.quantize_activations_token_sym(x, s)
    xv, wv = orc.bf16_to_f64(x), orc.bf16_to_f64(w)
    # dequantized operands approximate the smoothed ones to half a step
    assert np.all(np.abs(qx * t[:, None].astype(np.float64) - xv / s[None, :]) <= 0.5 * t[:, None] * (1 + 1e-5))
    assert np.all(np.abs(qw * u[:, None].astype(np.float64) - wv * s[None, :]) <= 0.5 * u[:, None] * (1 + 1e-5))
    e = orc.candidate_error(x, w, s, "w8a8", 0)
    d = xv @ wv.T - (qx * t[:, None].astype(np.float64)) @ (qw * u[:, None].astype(np.float64)).T
    assert np.allclose(e, (d ** 2).sum(axis=1), rtol=1e-10)
    # 8-bit error is far below 4-bit group error on the same data
    assert e.sum() < 0.05 * orc.candidate_error(x, w, s, "w4a16", 64).sum()


def test_paper_bit_widths_w4a8_w4a6():
    """The paper's own settings (Experiments: W4A8 and W4A6, per-token symmetric activations, per-channel
    symmetric weights): integer ranges follow [-2^(n-1), 2^(n-1)-1], the largest element of a row sits on
    +-(2^(n-1)-1), and fewer bits can only cost accuracy on the same data."""
    x, w, imp = wl.small_case(67, 32, 64, 12)
    s = orc.scale_table(orc.channel_stat(x), 20)[10]
    assert orc.symmetric_bits("w4a8") == (4, 8) and orc.symmetric_bits("w4a6") == (4, 6)
    qw, u = orc.quantize_weights_row_sym(w, s, 4)
    assert qw.min() >= -8 and qw.max() <= 7 and np.all(np.abs(qw).max(axis=1) == 7)
    qx, t = orc.quantize_activations_token_sym(x, s, 6)
    assert qx.min() >= -32 and qx.max() <= 31 and np.all(np.abs(qx).max(axis=1) == 31)
    p = (orc.bf16_to_f64(w) * s[None, :].astype(np.float64))
    assert np.allclose(u, np.abs(p).max(axis=1) / 7.0, rtol=1e-6)
    e88 = orc.candidate_error(x, w, s, "w8a8", 0).sum()
    e48 = orc.candidate_error(x, w, s, "w4a8", 0).sum()
    e46 = orc.candidate_error(x, w, s, "w4a6", 0).sum()
    assert e88 < e48 < e46
    # the error of W4A8 is dominated by the 4-bit weights: explicit dequantization gives the same number
    qx8, t8 = orc.quantize_activations_token_sym(x, s, 8)
    d = orc.bf16_to_f64(x) @ orc.bf16_to_f64(w).T - (qx8 * t8[:, None].astype(np.float64)) @ (qw * u[:, None].astype(np.float64)).T
    assert np.allclose(orc.candidate_error(x, w, s, "w4a8", 0), (d ** 2).sum(axis=1), rtol=1e-10)
    with pytest.raises(ValueError):
        orc.symmetric_bits("w9a8")


def test_argmin_takes_lowest_index_on_ties():
    assert orc.argmin_lowest(np.array([3.0, 1.0, 1.0, 2.0])) == 1
    assert orc.argmin_lowest(np.array([float("inf"), 5.0, 5.0])) == 1
    assert orc.weighted_loss(np.array([float("nan"), 1.0]), None, 2) == float("inf")


# ------------------------------------------------------------------ token importance


def test_token_importance_closed_forms():
    facts = paper_facts()
    b, n, c = 6, 10, 16
    g = np.full((b, n, c), -0.75)
    imp, mask = orc.token_importance(bits(g), orc.NORM_MEAN_ABS)
    assert np.allclose(imp, b * 0.75, rtol=0, atol=1e-15) and mask is None       # constant gradient
    hot = np.zeros((b, n, c))
    hot[:, :, 3] = 2.0                                                            # one live channel
    assert np.allclose(orc.token_importance(bits(hot), orc.NORM_MEAN_ABS)[0], b * 2.0 / c)
    assert np.allclose(orc.token_importance(bits(hot), orc.NORM_L2)[0], b * 2.0)
    rng = np.random.default_rng(4)
    gr = bits(rng.standard_normal((b, n, c)))
    i1, m1 = orc.token_importance(gr, orc.NORM_MEAN_ABS, facts["top_fraction"])
    i2, m2 = orc.token_importance(gr[::-1].copy(), orc.NORM_MEAN_ABS, facts["top_fraction"])
    assert np.allclose(i1, i2, rtol=1e-14) and np.array_equal(m1, m2)            # sample order is irrelevant
    assert m1.sum() == n // 2
    assert set(np.flatnonzero(m1)) == set(np.argsort(-i1, kind="stable")[: n // 2])
    # ties keep the lower index; count is floor(frac * N) but never zero
    tie = np.array([1.0, 2.0, 2.0, 2.0, 0.5])
    assert orc.top_mask(tie, 0.4).tolist() == [0, 1, 1, 0, 0]
    assert orc.top_mask(tie, 0.01).tolist() == [0, 1, 0, 0, 0]
    # linear in per-sample contributions: doubling one sample's gradient adds its share once more
    g2 = rng.standard_normal((2, n, c))
    a = orc.token_importance(bits(g2), orc.NORM_MEAN_ABS)[0]
    a0 = orc.token_importance(bits(g2[:1]), orc.NORM_MEAN_ABS)[0]
    a1 = orc.token_importance(bits(g2[1:]), orc.NORM_MEAN_ABS)[0]
    assert np.allclose(a, a0 + a1, rtol=1e-14)


def test_paper_shapes_of_gradient_workload():
    facts = paper_facts()
    g = wl.token_gradients(1, "g", 2, 64, 32, 48)
    assert g.shape == (2, 64, 32)
    assert int(facts["grad_tokens"]) == 1058 and int(facts["grad_channels"]) == 3584 and int(facts["calib_samples_B"]) == 128


def test_apply_layer_equals_search_candidate():
    x, w, imp = wl.small_case(71, 16, 128, 8)
    res = orc.scale_search(x, w, imp, group=128, n_grid=4)
    s = res["scales"][res["best"]]
    bias = bits(np.linspace(-1, 1, 8))
    yq, (codes, step, zero) = orc.apply_layer(x, w, s, bias, "w4a16", 128)
    e = orc.per_token_error(orc.layer_fp(x, w, orc.bf16_to_f64(bias)), yq)   # the bias cancels in the error
    assert np.allclose(e, res["per_token"][res["best"]], rtol=1e-9)


def test_shared_scale_of_sibling_linears_is_the_search_on_stacked_rows():
    """Linears fed by the same activations (q/k/v, gate/up) must share one scale, because the scale is folded
    into the layer before them (Sec. 2.2, last sentence on fusing the smoothing factor).  Quantizers act per
    output row (or per group inside a row), so stacking the weight matrices row-wise changes no code, and the
    loss of the stack is the row-count-weighted mean of the single losses: per_token adds up."""
    x, wq, imp = wl.small_case(91, 40, 64, 24)
    _, wk, _ = wl.small_case(92, 40, 64, 8)
    stack = np.concatenate([wq, wk], axis=0)
    for mode, group in (("w4a16", 32), ("w4a8", 0)):
        a = orc.scale_search(x, wq, imp, mode=mode, group=group, n_grid=5)
        b = orc.scale_search(x, wk, imp, mode=mode, group=group, n_grid=5)
        c = orc.scale_search(x, stack, imp, mode=mode, group=group, n_grid=5)
        assert np.allclose(c["per_token"], a["per_token"] + b["per_token"], rtol=1e-12)
        assert np.allclose(c["losses"], (24 * a["losses"] + 8 * b["losses"]) / 32, rtol=1e-12)
        assert np.array_equal(c["scales"], a["scales"])


@pytest.mark.parametrize("mode", ["w4a16", "w4a8"])
def test_two_stream_objective(mode):
    """First propagation strategy of Sec. 3.2.1: || f_fp(x_fp) - f_q(x_q) ||^2.  With equal streams it is the
    plain search; in general the error splits into a candidate-independent part (x_fp - x_q) W^T plus the
    single-stream error term, checked through that second route and against the scalar brute force."""
    xq, w, imp = wl.small_case(111, 6, 8, 3)
    xf, _, _ = wl.small_case(112, 6, 8, 3)
    same = orc.scale_search(xq, w, imp, mode=mode, group=4, n_grid=3, x_fp_bits=xq)
    plain = orc.scale_search(xq, w, imp, mode=mode, group=4, n_grid=3)
    assert np.array_equal(same["per_token"], plain["per_token"]) and same["best"] == plain["best"]
    two = orc.scale_search(xq, w, imp, mode=mode, group=4, n_grid=3, x_fp_bits=xf)
    assert np.array_equal(two["scales"], plain["scales"])          # the scale follows the quantized stream
    best, losses, table = brute.search(xq.tolist(), w.tolist(), [float(v) for v in imp], 4, 3, 4, mode, xf.tolist())
    assert best == two["best"]
    assert np.allclose(losses, two["losses"], rtol=1e-11)
    assert np.allclose(np.array(table), two["per_token"], rtol=1e-11, atol=1e-18)
    if mode == "w4a16":
        d = (orc.bf16_to_f64(xf) - orc.bf16_to_f64(xq)) @ orc.bf16_to_f64(w).T
        for k in range(3):
            _, _, _, w_hat = orc.quantize_weights_group_asym(w, two["scales"][k], 4)
            e = d + orc.bf16_to_f64(xq) @ (orc.bf16_to_f64(w) - w_hat.astype(np.float64)).T
            assert np.allclose(two["per_token"][k], (e ** 2).sum(axis=1), rtol=1e-9)


def test_four_bit_packing_round_trips():
    x, w, _ = wl.small_case(151, 8, 64, 6)
    s = orc.scale_table(orc.channel_stat(x), 20)[9]
    codes, _, _, _ = orc.quantize_weights_group_asym(w, s, 32, 4)
    packed = orc.pack_codes4(codes)
    assert packed.shape == (6, 32) and packed.dtype == np.uint8
    assert np.array_equal(orc.unpack_codes4(packed, signed=False), codes)
    assert packed[0, 0] == (int(codes[0, 0]) | (int(codes[0, 1]) << 4))          # even channel in the low nibble
    qw, _ = orc.quantize_weights_row_sym(w, s, 4)
    assert np.array_equal(orc.unpack_codes4(orc.pack_codes4(qw), signed=True), qw)


# ------------------------------------------------------------------ delta-weight operand, symmetric apply, reciprocal reading


def test_delta_weights_bf16_hand_values():
    """W - W_hat, one rounding to binary32 and one to bfloat16 (ties to even), checked on values worked out by hand:
    operand order and sign, a value already representable, both kinds of bfloat16 tie, and a case where the
    binary32 rounding lands on a tie that a single rounding from the exact difference would not see."""
    def one(w, w_hat):
        return int(orc.delta_weights_bf16(bits([[w]]), np.array([[w_hat]], dtype=np.float32))[0, 0])
    assert one(1.0, 0.75) == 0x3E80                       # +0.25
    assert one(0.5, 0.75) == 0xBE80                       # -0.25: W minus W_hat, not the reverse
    assert one(-1.0, -0.75) == 0xBE80
    assert one(0.25, 0.25) == 0x0000                      # no error -> +0
    # 2^-4 (1 + 2^-8): halfway between mantissas 0 and 1 -> even mantissa 0
    assert one(1.0, 1.0 - 2.0 ** -4 - 2.0 ** -12) == 0x3D80
    # 2^-4 (1 + 3 * 2^-8): halfway between mantissas 1 and 2 -> even mantissa 2
    assert one(1.0, 1.0 - 2.0 ** -4 - 3 * 2.0 ** -12) == 0x3D82
    # just above / below the first tie
    assert one(1.0, 1.0 - 2.0 ** -4 - 2.0 ** -12 - 2.0 ** -20) == 0x3D81
    assert one(1.0, 1.0 - 2.0 ** -4 - 2.0 ** -12 + 2.0 ** -20) == 0x3D80
    # exact difference 1 + 2^-8 + 2^-26: binary32 drops the 2^-26 (below half an ulp of 2^-23), leaving the tie
    # 1 + 2^-8, which goes to the even mantissa 0; one rounding from the exact value would give 1 + 2^-7
    w_hat = np.float32(2.0 ** -8 - 2.0 ** -26)
    assert float(w_hat) == 2.0 ** -8 - 2.0 ** -26
    assert one(1.0 + 2.0 ** -7, float(w_hat)) == 0x3F80
    # the same through a library conversion chain on random data (float32 subtraction, then torch's bf16 rounding)
    rng = np.random.default_rng(12)
    wb = bits(rng.standard_normal((16, 64)) * 0.02)
    w_hat = (wl.bf16_bits_to_f32(wb) + rng.standard_normal((16, 64)).astype(np.float32) * np.float32(1e-3)).astype(np.float32)
    ref = torch.from_numpy(wl.bf16_bits_to_f32(wb) - w_hat).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.delta_weights_bf16(wb, w_hat), ref)


def test_delta_weights_reproduce_the_candidate_error():
    """The bf16 delta-weight operand is a rounding of W - W_hat: X dW^T reproduces the search's per-token error to
    the operand's rounding (half an ulp of an 8-bit significand: 2^-8 relative) (a sign or transposition slip would be off by orders of magnitude)."""
    x, w, imp = wl.small_case(181, 48, 128, 24)
    res = orc.scale_search(x, w, imp, group=64, n_grid=4)
    for k in range(4):
        _, _, _, w_hat = orc.quantize_weights_group_asym(w, res["scales"][k], 64)
        dw = orc.bf16_to_f64(orc.delta_weights_bf16(w, w_hat))
        exact = orc.bf16_to_f64(w) - w_hat.astype(np.float64)
        assert np.all(np.abs(dw - exact) <= 2.0 ** -8 * np.abs(exact) + 1e-30)
        e = ((orc.bf16_to_f64(x) @ dw.T) ** 2).sum(axis=1)
        assert np.allclose(e, res["per_token"][k], rtol=5e-3)


@pytest.mark.parametrize("mode", ["w8a8", "w4a8", "w4a6"])
def test_apply_layer_symmetric_modes_with_bias(mode):
    """f_q = Q_w(W scale) Q_a(x / scale) + b in the symmetric settings, against scalar loops over the integer codes:
    the bias is added per output channel after the two steps have rescaled the integer product, it cancels in the
    search error, and the quantizer outputs returned are those of the candidate."""
    x, w, imp = wl.small_case(191, 7, 16, 5)
    wn, an = orc.symmetric_bits(mode)
    s = orc.scale_table(orc.channel_stat(x), 4)[2]
    bias_bits = bits(np.array([0.5, -1.0, 0.0, 2.0, -0.25]))
    b = orc.bf16_to_f64(bias_bits)
    yq, (qw, u, none) = orc.apply_layer(x, w, s, bias_bits, mode)
    assert none is None and yq.shape == (7, 5)
    qw_ref, u_ref = orc.quantize_weights_row_sym(w, s, wn)
    qx, t = orc.quantize_activations_token_sym(x, s, an)
    assert np.array_equal(qw, qw_ref) and np.array_equal(u, u_ref)
    for n in range(7):
        for o in range(5):
            acc = 0
            for c in range(16):
                acc += int(qx[n, c]) * int(qw[o, c])
            assert math.isclose(yq[n, o], float(t[n]) * float(u[o]) * acc + float(b[o]), rel_tol=1e-13, abs_tol=1e-15)
    # layer_q_w8a8 alone: bias per output channel (second axis), nothing else changes
    y0 = orc.layer_q_w8a8(qx, t, qw, u)
    y1 = orc.layer_q_w8a8(qx, t, qw, u, b)
    assert np.allclose(y1 - y0, np.broadcast_to(b[None, :], (7, 5)), rtol=0, atol=1e-15)
    # the bias cancels in the search error
    e = orc.per_token_error(orc.layer_fp(x, w, b), yq)
    assert np.allclose(e, orc.candidate_error(x, w, s, mode, 0), rtol=1e-9)
    # without a scale the activations are quantized as they are
    yq_plain, _ = orc.apply_layer(x, w, None, None, mode)
    qx0, t0 = orc.quantize_sym_rows(orc.bf16_to_f64(x).astype(np.float32), an)
    qw0, u0 = orc.quantize_weights_row_sym(w, None, wn)
    assert np.allclose(yq_plain, orc.layer_q_w8a8(qx0, t0, qw0, u0), rtol=0, atol=0)


def _search_with_exact_division(x, w, imp, group, n_grid):
    """The group-mode search with the other reading of diag(scale)^-1 in the smoothing identity of Sec. 2.2: the
    dequantized weight divided by the scale in one IEEE binary32 division, where the oracle multiplies by the
    rounded reciprocal.  Codes, steps and zero-points are the oracle's (they do not depend on the reading)."""
    scales = orc.scale_table(orc.channel_stat(x), n_grid)
    y_fp = orc.layer_fp(x, w)
    losses, per_token, ints = [], [], []
    for k in range(n_grid):
        codes, step, zero, _ = orc.quantize_weights_group_asym(w, scales[k], group)
        c2, c1 = codes.shape
        dq = ((codes.astype(np.int64).reshape(c2, c1 // group, group) - zero[:, :, None]).astype(np.float32)
              * step[:, :, None]).astype(np.float32).reshape(c2, c1)
        w_hat = (dq / scales[k][None, :].astype(np.float32)).astype(np.float32)
        e = orc.per_token_error(y_fp, orc.layer_q_w4a16(x, w_hat))
        per_token.append(e)
        losses.append(orc.weighted_loss(e, imp, c2))
        ints.append((codes, step, zero))
    return np.array(losses), np.array(per_token), ints


@pytest.mark.parametrize("shape", ["cfg0", (300, 192, 320, 64, 5), (515, 1088, 777, 64, 7), (128, 64, 256, 32, 3)])
def test_reciprocal_and_division_readings_give_the_same_search(shape):
    """Sec. 2.2 writes the smoothing as diag(scale)^-1; the oracle takes that as a product with the binary32
    reciprocal (the same factor that smooths the activations).  Dividing by the scale instead changes W_hat by at
    most an ulp, so the integers are untouched and every loss moves by far less than the stated tolerance; the
    argmin is the same."""
    if shape == "cfg0":
        cfgw = wl.config("cfg0")
        data = wl.LayerData(cfgw)
        lin = cfgw.linear("q")
        x, w, imp, group, n_grid = data.x(lin), data.w(lin), data.imp(), cfgw.group, cfgw.n_grid
    else:
        n, c1, c2, group, n_grid = shape
        x, w, imp = wl.small_case(17, n, c1, c2, n_outlier=2)
    ref = orc.scale_search(x, w, imp, "w4a16", group, n_grid)
    losses, per_token, ints = _search_with_exact_division(x, w, imp, group, n_grid)
    assert np.max(np.abs(losses - ref["losses"]) / ref["losses"]) < 1e-6
    assert np.allclose(per_token, ref["per_token"], rtol=1e-5)
    assert orc.argmin_lowest(losses) == ref["best"]
    # the reading cannot reach the integers: they are computed before any division by the scale
    for k in (0, n_grid - 1):
        codes, step, zero, _ = orc.quantize_weights_group_asym(w, ref["scales"][k], group)
        assert np.array_equal(codes, ints[k][0]) and np.array_equal(step, ints[k][1]) and np.array_equal(zero, ints[k][2])


def test_reciprocal_and_division_readings_symmetric_activations():
    """For quantized activations the reading reaches an integer decision: x * fl32(1/scale) against fl32(x / scale)
    differ by an ulp in about a quarter of the elements, which moves a code only when the quotient sits within
    that ulp of a rounding boundary.  Counted here: a few codes in a hundred thousand, losses equal to 1e-4."""
    x, w, imp = wl.small_case(43, 256, 512, 512, n_outlier=2)
    scales = orc.scale_table(orc.channel_stat(x), 20)
    y_fp = orc.layer_fp(x, w)
    xv = orc.bf16_to_f64(x).astype(np.float32)
    flipped, total = 0, 0
    for k in (5, 12, 19):
        qx, t = orc.quantize_activations_token_sym(x, scales[k], 8)
        qx_div, t_div = orc.quantize_sym_rows((xv / scales[k][None, :]).astype(np.float32), 8)
        flipped += int((qx != qx_div).sum())
        total += qx.size
        assert np.max(np.abs(qx.astype(np.int64) - qx_div.astype(np.int64))) <= 1
        qw, u = orc.quantize_weights_row_sym(w, scales[k], 8)
        l_mul = orc.weighted_loss(orc.per_token_error(y_fp, orc.layer_q_w8a8(qx, t, qw, u)), imp, 512)
        l_div = orc.weighted_loss(orc.per_token_error(y_fp, orc.layer_q_w8a8(qx_div, t_div, qw, u)), imp, 512)
        assert abs(l_mul - l_div) / l_mul < 1e-4
    assert flipped / total < 1e-3
