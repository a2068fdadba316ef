"""GPU parity: the CUDA path (through the C ABI binding) against the CPU oracle, element by element on
the same seeded inputs.  Integer work (codes, zero-points, scale bits, argmin) must match bit for bit;
weighted losses and per-token errors within 2e-3 relative."""
import numpy as np
import pytest
import torch

from oracle import tlq_oracle as orc
from paper_2602_07899_b200 import workloads as wl

pytestmark = pytest.mark.gpu

LOSS_RTOL = 2e-3   # the stated tolerance on weighted losses (and per-token errors)


@pytest.fixture(scope="module")
def tlq():
    import __graft_entry__ as entry
    entry.build()
    from paper_2602_07899_b200 import tlq as mod
    return mod


def dev_bf16(tlq, bits):
    return tlq.bf16_from_bits(bits)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


# ----------------------------------------------------------------------------------- (a) statistics + scale table


@pytest.mark.parametrize("n,c1", [(256, 512), (300, 264), (1, 8), (4100, 1544), (8192, 3584)])
@pytest.mark.parametrize("stat", [0, 1, 2])
def test_scale_candidates_bit_exact(tlq, n, c1, stat):
    if stat == 2 and n == 8192:
        pytest.skip("covered by the smaller shapes")
    xb = wl.activations(5, f"sc/{n}x{c1}", n, c1, (3 * n) // 4, "normal", min(4, c1))
    mask_np = (np.random.default_rng(n + c1).random(n) < 0.5).astype(np.uint8)
    mask_np[0] = 1
    cfg = tlq.config(stat_mode=stat, n_grid=20)
    mask = torch.from_numpy(mask_np).cuda() if stat == 2 else None
    x_stat, s = tlq.tlq_scale_candidates(dev_bf16(tlq, xb), cfg, mask)
    torch.cuda.synchronize()
    ref_stat = orc.channel_stat(xb, stat, mask_np)
    ref_s = orc.scale_table(ref_stat, 20)
    np.testing.assert_allclose(x_stat.cpu().numpy(), ref_stat, rtol=1e-14, atol=0)
    assert np.array_equal(bits_of(s), orc.f32_to_bf16_bits(ref_s))


# ----------------------------------------------------------------------------------- (b) fake-quant


@pytest.mark.parametrize("c2,c1,group,bits", [(512, 512, 128, 4), (37, 384, 64, 4), (130, 1024, 256, 3),
                                              (16, 96, 32, 8), (1, 128, 128, 2), (1000, 3584, 128, 4)])
def test_group_quantizer_bit_exact(tlq, c2, c1, group, bits):
    xb = wl.activations(7, f"gq/x{c1}", 64, c1, 48, "normal", 4)
    wb = wl.weights(7, f"gq/w{c2}x{c1}", c2, c1)
    s_np = orc.scale_table(orc.channel_stat(xb), 20)[13]
    cfg = tlq.config(w_bits=bits, group_size=group)
    for s_vec in (None, s_np):
        s_dev = None if s_vec is None else dev_bf16(tlq, orc.f32_to_bf16_bits(s_vec))
        out = tlq.tlq_quantize_weights(dev_bf16(tlq, wb), s_dev, cfg, want_dw=True)
        torch.cuda.synchronize()
        codes, step, zero, w_hat = orc.quantize_weights_group_asym(wb, s_vec, group, bits)
        assert np.array_equal(out["codes"].cpu().numpy(), codes)
        assert np.array_equal(out["zeros"].cpu().numpy(), zero)
        assert np.array_equal(out["steps"].cpu().numpy().view(np.uint32), step.view(np.uint32))
        assert np.array_equal(bits_of(out["dW"]), orc.delta_weights_bf16(wb, w_hat))


def test_degenerate_groups(tlq):
    # flat group, zero group, all-positive group, huge and tiny magnitudes
    w = np.zeros((4, 256), dtype=np.float32)
    w[0, :128] = 0.25
    w[1, :128] = np.linspace(0.5, 1.0, 128)
    w[2, 128:] = -np.linspace(1e-3, 2e-3, 128)
    w[3, :] = np.random.default_rng(0).standard_normal(256) * 1e4
    wb = wl.f32_to_bf16_bits(w)
    cfg = tlq.config()
    out = tlq.tlq_quantize_weights(dev_bf16(tlq, wb), None, cfg, want_dw=True)
    torch.cuda.synchronize()
    codes, step, zero, w_hat = orc.quantize_weights_group_asym(wb, None, 128)
    assert np.array_equal(out["codes"].cpu().numpy(), codes)
    assert np.array_equal(out["zeros"].cpu().numpy(), zero)
    assert np.array_equal(out["steps"].cpu().numpy(), step)
    assert np.array_equal(bits_of(out["dW"]), orc.delta_weights_bf16(wb, w_hat))


@pytest.mark.parametrize("c2,c1", [(64, 512), (33, 1040), (512, 3584)])
def test_int8_row_quantizer_bit_exact(tlq, c2, c1):
    xb = wl.activations(9, f"i8/x{c1}", 32, c1, 24, "normal", 4)
    wb = wl.weights(9, f"i8/w{c2}x{c1}", c2, c1)
    s_np = orc.scale_table(orc.channel_stat(xb), 20)[7]
    cfg = tlq.config(tlq.W8A8_SYM)
    for s_vec in (None, s_np):
        s_dev = None if s_vec is None else dev_bf16(tlq, orc.f32_to_bf16_bits(s_vec))
        out = tlq.tlq_quantize_weights(dev_bf16(tlq, wb), s_dev, cfg)
        torch.cuda.synchronize()
        qw, u = orc.quantize_weights_row_sym(wb, s_vec)
        assert np.array_equal(out["codes"].cpu().numpy(), qw)
        assert np.array_equal(out["steps"].cpu().numpy().view(np.uint32), u.view(np.uint32))


# ----------------------------------------------------------------------------------- (d) token importance


@pytest.mark.parametrize("b,n,c,norm", [(6, 100, 64, 0), (3, 257, 520, 1), (1, 50, 8, 0), (16, 1058, 512, 0)])
def test_token_importance(tlq, b, n, c, norm):
    gb = wl.token_gradients(3, f"g/{b}x{n}x{c}", b, n, c, (3 * n) // 4)
    imp, mask = tlq.tlq_token_importance(dev_bf16(tlq, gb), norm, 0.5)
    torch.cuda.synchronize()
    ref_imp, ref_mask = orc.token_importance(gb, norm, 0.5)
    got = imp.cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(got, ref_imp, rtol=1e-5, atol=1e-30)
    m = mask.cpu().numpy()
    k_sel = max(1, n // 2)
    assert m.sum() == k_sel
    # the mask is exactly the top-k (ties: lower index) of the values the kernel itself produced
    assert np.array_equal(m, orc.top_mask(imp.cpu().numpy(), 0.5))
    # and agrees with the oracle's selection except where two importances are within rounding of the cut
    diff = np.flatnonzero(m != ref_mask)
    if diff.size:
        cut = np.sort(ref_imp)[::-1][k_sel - 1]
        assert np.all(np.abs(ref_imp[diff] - cut) <= 1e-5 * cut)
    # float32 gradients take the same path
    gf = torch.from_numpy(wl.bf16_bits_to_f32(gb)).cuda()
    imp32, _ = tlq.tlq_token_importance(gf, norm, 0.0)
    np.testing.assert_allclose(imp32.cpu().numpy(), got, rtol=1e-6)


# ----------------------------------------------------------------------------------- (c) the search


def run_search(tlq, xb, wb, imp, group=128, n_grid=20, w_bits=4, stat=0, mask=None):
    cfg = tlq.config(w_bits=w_bits, group_size=group, n_grid=n_grid, stat_mode=stat)
    w_dev = None if imp is None else torch.from_numpy(np.asarray(imp, dtype=np.float32)).cuda()
    m_dev = None if mask is None else torch.from_numpy(mask).cuda()
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), w_dev, cfg, mask=m_dev, per_token=True)
    return dict(best=int(out.best_idx.item()), losses=out.losses.cpu().numpy(), per_token=out.per_token.cpu().numpy(),
                s_best=bits_of(out.s_best))


GAP_FLOOR = 1e-4   # the seeded cases keep the oracle's two best losses at least this far apart (asserted), so
                   # the CUDA path's loss error (at most 4e-5 relative) cannot excuse a different argmin


def assert_same_argmin(best, ref):
    """The argmin must be the oracle's; the oracle's own top-2 gap is asserted to be resolvable first."""
    order = np.sort(ref["losses"])
    if len(order) > 1:
        gap = (order[1] - order[0]) / order[0]
        assert gap > GAP_FLOOR, f"seeded case is ambiguous in the oracle itself (top-2 gap {gap:.2e}): pick another seed"
    assert best == ref["best"]


def check_against_oracle(got, ref, n_grid):
    np.testing.assert_allclose(got["per_token"], ref["per_token"], rtol=LOSS_RTOL, atol=1e-30)
    np.testing.assert_allclose(got["losses"], ref["losses"], rtol=LOSS_RTOL)
    assert_same_argmin(got["best"], ref)
    assert got["best"] == int(np.argmin(got["losses"]))
    assert np.array_equal(got["s_best"], orc.f32_to_bf16_bits(ref["scales"][got["best"]]))


def test_search_cfg0(tlq):
    cfgw = wl.config("cfg0")
    data = wl.LayerData(cfgw)
    lin = cfgw.linear("q")
    ref = orc.scale_search(data.x(lin), data.w(lin), data.imp(), "w4a16", 128, 20)
    got = run_search(tlq, data.x(lin), data.w(lin), data.imp())
    check_against_oracle(got, ref, 20)


@pytest.mark.parametrize("n,c1,c2,group,n_grid", [(300, 192, 320, 64, 5), (128, 64, 256, 32, 3), (1, 128, 64, 128, 2),
                                                  (515, 1088, 777, 64, 7), (257, 512, 256, 256, 1)])
def test_search_ragged_shapes(tlq, n, c1, c2, group, n_grid):
    xb, wb, imp = wl.small_case(17, n, c1, c2, n_outlier=2)
    ref = orc.scale_search(xb, wb, imp, "w4a16", group, n_grid)
    got = run_search(tlq, xb, wb, imp, group, n_grid)
    check_against_oracle(got, ref, n_grid)


def test_search_importance_special_cases(tlq):
    xb, wb, imp = wl.small_case(23, 384, 256, 512)
    ref = orc.scale_search(xb, wb, None, "w4a16", 128, 6)
    uni = run_search(tlq, xb, wb, None, 128, 6)
    check_against_oracle(uni, ref, 6)
    const = run_search(tlq, xb, wb, np.full(384, 2.5, np.float32), 128, 6)
    np.testing.assert_allclose(const["losses"], uni["losses"], rtol=1e-6)            # uniform importance = plain MSE
    hot = np.zeros(384, np.float32)
    hot[201] = 3.0
    one = run_search(tlq, xb, wb, hot, 128, 6)
    np.testing.assert_allclose(one["losses"], uni["per_token"][:, 201].astype(np.float64) / 512.0, rtol=1e-6)
    np.testing.assert_allclose(one["losses"], ref["per_token"][:, 201] / 512.0, rtol=LOSS_RTOL)
    sel = np.zeros(384, np.float32)
    sel[100:292] = 1.0                                                                # a 0/1 token selection
    sub = run_search(tlq, xb, wb, sel, 128, 6)
    np.testing.assert_allclose(sub["losses"], ref["per_token"][:, 100:292].mean(axis=1) / 512.0, rtol=LOSS_RTOL)


def test_search_masked_max_statistic(tlq):
    xb, wb, imp = wl.small_case(29, 200, 256, 256)
    mask = orc.top_mask(imp.astype(np.float64), 0.5)
    ref = orc.scale_search(xb, wb, imp, "w4a16", 128, 8, orc.STAT_MASKED_MAX, mask)
    got = run_search(tlq, xb, wb, imp, 128, 8, stat=2, mask=mask)
    check_against_oracle(got, ref, 8)


def test_search_is_deterministic(tlq):
    xb, wb, imp = wl.small_case(31, 640, 512, 768)
    a = run_search(tlq, xb, wb, imp)
    b = run_search(tlq, xb, wb, imp)
    assert np.array_equal(a["losses"].view(np.uint64), b["losses"].view(np.uint64))
    assert np.array_equal(a["per_token"].view(np.uint32), b["per_token"].view(np.uint32))


def apply_reference_and_bound(xb, wb, w_hat, bias_bits):
    """What tlq_apply_layer's 16-bit-activation path computes, in float64: X W^T - X bf16(dW)^T + b with the oracle's
    bf16 delta weights, and the bound on the kernel's distance from it.  Two sources remain: the fp32 accumulation
    of 2*C1 products in tensor memory (error at most 2*C1 * 2^-23 * sum |x| (|w| + |dw|), the standard
    running-sum bound with a unit roundoff that also covers a truncating adder) and one rounding of the result
    to bf16 (half an ulp: 2^-8 relative to the exact value plus the accumulation error)."""
    x, w = orc.bf16_to_f64(xb), orc.bf16_to_f64(wb)
    dw = orc.bf16_to_f64(orc.delta_weights_bf16(wb, w_hat))
    y = x @ w.T - x @ dw.T
    if bias_bits is not None:
        y = y + orc.bf16_to_f64(bias_bits)[None, :]
    acc = 2.0 * x.shape[1] * 2.0 ** -23 * (np.abs(x) @ (np.abs(w) + np.abs(dw)).T)
    return y, acc + 2.0 ** -8 * (np.abs(y) + acc) + 1e-30


def test_apply_layer(tlq):
    xb, wb, imp = wl.small_case(37, 300, 256, 328)
    ref = orc.scale_search(xb, wb, imp, "w4a16", 128, 8)
    s = ref["scales"][ref["best"]]
    bias_bits = wl.f32_to_bf16_bits(np.linspace(-0.5, 0.5, 328).astype(np.float32))
    yq_ref, (codes, step, zero) = orc.apply_layer(xb, wb, s, bias_bits, "w4a16", 128)
    out = tlq.tlq_apply_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), dev_bf16(tlq, orc.f32_to_bf16_bits(s)),
                              dev_bf16(tlq, bias_bits), tlq.config())
    assert np.array_equal(out["codes"].cpu().numpy(), codes)
    assert np.array_equal(out["zeros"].cpu().numpy(), zero)
    yq = out["Yq"].float().cpu().numpy().astype(np.float64)
    _, _, _, w_hat = orc.quantize_weights_group_asym(wb, s, 128)
    y_op, bound = apply_reference_and_bound(xb, wb, w_hat, bias_bits)
    assert np.all(np.abs(yq - y_op) <= bound)
    # and the operand's own bf16 rounding keeps that reference close to the oracle's f_q: per token the squared
    # distance is a 2^-8-relative perturbation of every delta weight, far below the token's output error
    d2 = ((y_op - yq_ref) ** 2).sum(axis=1)
    assert np.all(d2 <= 2.0 ** -14 * ref["per_token"][ref["best"]])
    # without scale and bias
    out0 = tlq.tlq_apply_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), None, None, tlq.config(), want_codes=False)
    _, _, _, w_hat0 = orc.quantize_weights_group_asym(wb, None, 128)
    y0_op, bound0 = apply_reference_and_bound(xb, wb, w_hat0, None)
    y0 = out0["Yq"].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(y0 - y0_op) <= bound0)


def test_device_errors_are_reported_not_raised_as_faults(tlq):
    # host-side refusals on a live device: nothing is launched, the context stays usable
    import ctypes
    x = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    c = tlq.config()
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    rc = tlq.lib.tlq_scale_search_layer(x.data_ptr(), 4, 128, x.data_ptr(), 4, None, None, ctypes.byref(c),
                                        ws.data_ptr(), 1024, ws.data_ptr(), ws.data_ptr(), ws.data_ptr(), None, None)
    assert rc == tlq.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert tlq.tlq_kernel_launch_count() >= 0


def test_bounded_wait_runs_out_and_is_reported(tlq):
    """The device-side error path without a fault: a wait with a short limit on a barrier nothing arrives on gives
    up, the status word says TLQ_ERR_TIMEOUT, and the very next search on the same workspace memory is normal."""
    xb, wb, imp = wl.small_case(201, 200, 128, 96)
    cfg = tlq.config(group_size=64, n_grid=4)
    bufs = tlq.SearchBuffers(200, 128, 96, cfg, torch.device("cuda"))
    assert tlq.tlq_selftest_bounded_wait(bufs.workspace, 1_000_000) == tlq.ERR_TIMEOUT
    hdr = bufs.workspace[:256].view(torch.int32).cpu().numpy()
    assert hdr[1] == 99 and hdr[4] == 1          # which wait gave up; the abort flag reached the other lanes
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.from_numpy(imp).cuda(), cfg, bufs)
    assert tlq.tlq_read_status(out.workspace) == tlq.OK
    ref = orc.scale_search(xb, wb, imp, "w4a16", 64, 4)
    np.testing.assert_allclose(out.losses.cpu().numpy(), ref["losses"], rtol=LOSS_RTOL)
    # host-side refusals of the self-test itself
    import ctypes
    assert tlq.lib.tlq_selftest_bounded_wait(bufs.workspace.data_ptr(), 16, 1000, None) == tlq.ERR_WORKSPACE
    assert tlq.lib.tlq_selftest_bounded_wait(bufs.workspace.data_ptr(), 256, 0, None) == tlq.ERR_INVALID_ARG
    assert tlq.lib.tlq_selftest_bounded_wait(bufs.workspace.data_ptr(), 256, 3_000_000_000, None) == tlq.ERR_INVALID_ARG


# ----------------------------------------------------------------------------------- W8A8


@pytest.mark.parametrize("n,c1", [(64, 512), (130, 1040), (1000, 3584)])
def test_int8_activation_quantizer_bit_exact(tlq, n, c1):
    xb = wl.activations(11, f"a8/x{n}x{c1}", n, c1, (3 * n) // 4, "normal", 4)
    s_np = orc.scale_table(orc.channel_stat(xb), 20)[11]
    cfg = tlq.config(tlq.W8A8_SYM)
    for s_vec in (None, s_np):
        s_dev = None if s_vec is None else dev_bf16(tlq, orc.f32_to_bf16_bits(s_vec))
        codes, steps = tlq.tlq_quantize_activations(dev_bf16(tlq, xb), s_dev, cfg)
        torch.cuda.synchronize()
        qx, t = orc.quantize_activations_token_sym(xb, s_vec)
        assert np.array_equal(codes.cpu().numpy(), qx)
        assert np.array_equal(steps.cpu().numpy().view(np.uint32), t.view(np.uint32))


def run_search_w8a8(tlq, xb, wb, imp, n_grid=20):
    cfg = tlq.config(tlq.W8A8_SYM, n_grid=n_grid)
    w_dev = None if imp is None else torch.from_numpy(np.asarray(imp, dtype=np.float32)).cuda()
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), w_dev, cfg, per_token=True)
    return dict(best=int(out.best_idx.item()), losses=out.losses.cpu().numpy(), per_token=out.per_token.cpu().numpy(),
                s_best=bits_of(out.s_best))


@pytest.mark.parametrize("n,c1,c2,n_grid", [(256, 512, 512, 20), (300, 208, 320, 5), (128, 128, 256, 3), (1, 256, 64, 2),
                                            (515, 1088, 777, 6)])
def test_search_w8a8(tlq, n, c1, c2, n_grid):
    xb, wb, imp = wl.small_case(43, n, c1, c2, n_outlier=2)
    ref = orc.scale_search(xb, wb, imp, "w8a8", 0, n_grid)
    got = run_search_w8a8(tlq, xb, wb, imp, n_grid)
    check_against_oracle(got, ref, n_grid)


def test_search_w8a8_importance_special_cases_and_determinism(tlq):
    xb, wb, imp = wl.small_case(47, 384, 256, 512)
    ref = orc.scale_search(xb, wb, None, "w8a8", 0, 6)
    uni = run_search_w8a8(tlq, xb, wb, None, 6)
    check_against_oracle(uni, ref, 6)
    hot = np.zeros(384, np.float32)
    hot[77] = 1.0
    one = run_search_w8a8(tlq, xb, wb, hot, 6)
    np.testing.assert_allclose(one["losses"], uni["per_token"][:, 77].astype(np.float64) / 512.0, rtol=1e-6)
    again = run_search_w8a8(tlq, xb, wb, None, 6)
    assert np.array_equal(uni["losses"].view(np.uint64), again["losses"].view(np.uint64))
    assert np.array_equal(uni["per_token"].view(np.uint32), again["per_token"].view(np.uint32))


def test_apply_layer_w8a8(tlq):
    xb, wb, imp = wl.small_case(53, 300, 256, 328)
    ref = orc.scale_search(xb, wb, imp, "w8a8", 0, 8)
    s = ref["scales"][ref["best"]]
    bias_bits = wl.f32_to_bf16_bits(np.linspace(-0.5, 0.5, 328).astype(np.float32))
    yq_ref, (qw, u, _) = orc.apply_layer(xb, wb, s, bias_bits, "w8a8")
    out = tlq.tlq_apply_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), dev_bf16(tlq, orc.f32_to_bf16_bits(s)),
                              dev_bf16(tlq, bias_bits), tlq.config(tlq.W8A8_SYM))
    assert np.array_equal(out["codes"].cpu().numpy(), qw)
    assert np.array_equal(out["steps"].cpu().numpy().view(np.uint32), u.view(np.uint32))
    yq = out["Yq"].float().cpu().numpy().astype(np.float64)
    # integer accumulation is exact; what remains is the bf16 rounding of the output (2^-9 relative, doubled)
    assert np.all(np.abs(yq - yq_ref) <= 2.0 ** -8 * np.abs(yq_ref) + 1e-6)


# ----------------------------------------------------------------------------------- W4A8 / W4A6 (the paper's settings)


@pytest.mark.parametrize("w_bits,a_bits", [(4, 8), (4, 6), (6, 4), (2, 8)])
def test_symmetric_quantizers_other_widths_bit_exact(tlq, w_bits, a_bits):
    xb = wl.activations(71, "sym/x", 130, 1040, 96, "normal", 4)
    wb = wl.weights(71, "sym/w", 77, 1040)
    s_np = orc.scale_table(orc.channel_stat(xb), 20)[9]
    cfg = tlq.config(tlq.WA_SYM_CHANNEL, w_bits=w_bits, a_bits=a_bits)
    for s_vec in (None, s_np):
        s_dev = None if s_vec is None else dev_bf16(tlq, orc.f32_to_bf16_bits(s_vec))
        out = tlq.tlq_quantize_weights(dev_bf16(tlq, wb), s_dev, cfg)
        codes, steps = tlq.tlq_quantize_activations(dev_bf16(tlq, xb), s_dev, cfg)
        torch.cuda.synchronize()
        qw, u = orc.quantize_weights_row_sym(wb, s_vec, w_bits)
        qx, t = orc.quantize_activations_token_sym(xb, s_vec, a_bits)
        assert np.array_equal(out["codes"].cpu().numpy(), qw)
        assert np.array_equal(out["steps"].cpu().numpy().view(np.uint32), u.view(np.uint32))
        assert np.array_equal(codes.cpu().numpy(), qx)
        assert np.array_equal(steps.cpu().numpy().view(np.uint32), t.view(np.uint32))
        assert qw.min() >= -(1 << (w_bits - 1)) and qx.max() <= (1 << (a_bits - 1)) - 1


def run_search_sym(tlq, xb, wb, imp, w_bits, a_bits, n_grid=20):
    cfg = tlq.config(tlq.WA_SYM_CHANNEL, w_bits=w_bits, a_bits=a_bits, n_grid=n_grid)
    w_dev = None if imp is None else torch.from_numpy(np.asarray(imp, dtype=np.float32)).cuda()
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), w_dev, cfg, per_token=True)
    return dict(best=int(out.best_idx.item()), losses=out.losses.cpu().numpy(), per_token=out.per_token.cpu().numpy(),
                s_best=bits_of(out.s_best))


@pytest.mark.parametrize("mode,n,c1,c2,n_grid", [("w4a8", 256, 512, 512, 20), ("w4a6", 256, 512, 512, 20),
                                                 ("w4a8", 515, 1088, 777, 6), ("w4a6", 300, 208, 320, 5)])
def test_search_w4a8_w4a6(tlq, mode, n, c1, c2, n_grid):
    xb, wb, imp = wl.small_case(73, n, c1, c2, n_outlier=2)
    wn, an = orc.symmetric_bits(mode)
    ref = orc.scale_search(xb, wb, imp, mode, 0, n_grid)
    got = run_search_sym(tlq, xb, wb, imp, wn, an, n_grid)
    check_against_oracle(got, ref, n_grid)


def test_apply_layer_w4a8(tlq):
    xb, wb, imp = wl.small_case(79, 300, 256, 328)
    ref = orc.scale_search(xb, wb, imp, "w4a8", 0, 8)
    s = ref["scales"][ref["best"]]
    yq_ref, (qw, u, _) = orc.apply_layer(xb, wb, s, None, "w4a8")
    out = tlq.tlq_apply_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), dev_bf16(tlq, orc.f32_to_bf16_bits(s)), None,
                              tlq.config(tlq.WA_SYM_CHANNEL, w_bits=4, a_bits=8))
    assert np.array_equal(out["codes"].cpu().numpy(), qw)
    assert np.array_equal(out["steps"].cpu().numpy().view(np.uint32), u.view(np.uint32))
    yq = out["Yq"].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(yq - yq_ref) <= 2.0 ** -8 * np.abs(yq_ref) + 1e-6)


# ----------------------------------------------------------------------------------- host-side pipeline


def test_host_layer_search_overlapped_copies_match_direct_calls(tlq):
    """Inputs in pinned host memory, copies on a side stream: same argmin and bit-identical losses as the direct
    call on resident tensors, also when the staging buffers are re-used for new data right away."""
    from paper_2602_07899_b200 import calibrate
    dev = torch.device("cuda", 0)
    cfg = tlq.config(n_grid=6)
    shapes = [("a", "x0", 300, 256, 320), ("b", "x0", 300, 256, 64), ("c", "x1", 300, 512, 256)]
    pipe = calibrate.HostLayerSearch(shapes, cfg, dev)
    rounds = []
    for seed in (81, 82, 83):
        hx, hw = {}, {}
        for name, x_name, n, c1, c2 in shapes:
            xb, wb, imp = wl.small_case(seed + c1, n, c1, c2)
            hx.setdefault(x_name, torch.from_numpy(xb.view(np.int16)).pin_memory())
            hw[name] = torch.from_numpy(wb.view(np.int16)).pin_memory()
        himp = torch.from_numpy(wl.importance(seed, "pipe/imp", 300, 225)).pin_memory()
        out = {name: (torch.empty(1, dtype=torch.int32).pin_memory(), torch.empty(6, dtype=torch.float64).pin_memory())
               for name, *_ in shapes}
        pipe.run(hx, hw, himp, out)       # three rounds back to back, no host synchronisation in between
        rounds.append((hx, hw, himp, out))
    pipe.check()
    for hx, hw, himp, out in rounds:
        for name, x_name, n, c1, c2 in shapes:
            ref = tlq.tlq_scale_search_layer(hx[x_name].cuda().view(torch.bfloat16), hw[name].cuda().view(torch.bfloat16),
                                             himp.cuda(), cfg)
            assert int(out[name][0].item()) == int(ref.best_idx.item())
            assert np.array_equal(out[name][1].numpy().view(np.uint64), ref.losses.cpu().numpy().view(np.uint64))


def test_shared_scale_search_on_stacked_sibling_weights(tlq):
    """q/k/v-style siblings searched as one row-stacked matrix: parity with the oracle on the stack, and the
    stack's per-token error is the sum of the siblings' (one scale for all of them)."""
    xb, wq, imp = wl.small_case(93, 300, 256, 320)
    _, wk, _ = wl.small_case(94, 300, 256, 72)
    stack = np.concatenate([wq, wk], axis=0)
    ref = orc.scale_search(xb, stack, imp, "w4a16", 64, 6)
    got = run_search(tlq, xb, stack, imp, group=64, n_grid=6)
    check_against_oracle(got, ref, 6)
    parts = run_search(tlq, xb, wq, imp, group=64, n_grid=6)["per_token"] + run_search(tlq, xb, wk, imp, group=64, n_grid=6)["per_token"]
    np.testing.assert_allclose(got["per_token"], parts, rtol=1e-5)


# ----------------------------------------------------------------------------------- zero-weight tokens skipped


def _search_losses(tlq, xb, wb, imp, cfg):
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.from_numpy(imp).cuda(), cfg)
    return int(out.best_idx.item()), out.losses.cpu().numpy(), bits_of(out.s_best)


@pytest.mark.parametrize("mode", ["w4a16", "w8a8", "w4a6"])
@pytest.mark.parametrize("n,c1,c2,kind", [(300, 256, 320, "top50"), (515, 1088, 777, "sparse"), (256, 512, 512, "onehot"),
                                          (384, 256, 256, "dense"), (130, 128, 64, "first_tile_only")])
def test_search_skipping_zero_weight_tokens(tlq, mode, n, c1, c2, kind):
    """The paper's token-level calibration set is a 0/1 weight vector (top half by gradient importance);
    tokens of weight zero are packed away before the quantized layer is applied.  Same losses as the
    oracle (which multiplies by the zeros) and as the unflagged call."""
    xb, wb, imp = wl.small_case(97, n, c1, c2)
    imp = imp.copy()
    if kind == "top50":
        gb = wl.token_gradients(97, "skip/g", 2, n, 64, (3 * n) // 4)
        imp = orc.top_mask(orc.token_importance(gb)[0], 0.5).astype(np.float32)
        assert imp.sum() == n // 2
    elif kind == "sparse":
        imp[np.random.default_rng(5).random(n) < 0.7] = 0.0
    elif kind == "onehot":
        imp = wl.importance(97, "skip/onehot", n, (3 * n) // 4, "onehot")
    elif kind == "first_tile_only":
        imp[100:] = 0.0
    n_grid = 5
    if mode == "w4a16":
        base = dict(group_size=64, n_grid=n_grid)
        ref = orc.scale_search(xb, wb, imp, "w4a16", 64, n_grid)
    else:
        wn, an = orc.symmetric_bits(mode)
        base = dict(mode=tlq.WA_SYM_CHANNEL, w_bits=wn, a_bits=an, n_grid=n_grid)
        ref = orc.scale_search(xb, wb, imp, mode, 0, n_grid)
    best0, loss0, s0 = _search_losses(tlq, xb, wb, imp, tlq.config(**base))
    best1, loss1, s1 = _search_losses(tlq, xb, wb, imp, tlq.config(flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS, **base))
    np.testing.assert_allclose(loss1, ref["losses"], rtol=LOSS_RTOL)
    np.testing.assert_allclose(loss1, loss0, rtol=1e-5)
    assert_same_argmin(best1, ref)
    assert best0 == best1
    assert np.array_equal(s1, orc.f32_to_bf16_bits(ref["scales"][best1]))


def test_skipping_needs_weights_and_has_no_per_token_table(tlq):
    xb, wb, imp = wl.small_case(98, 64, 128, 64)
    cfg = tlq.config(n_grid=3, flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS)
    with pytest.raises(tlq.TlqError) as e:
        tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), None, cfg)
    assert e.value.status == tlq.ERR_INVALID_ARG
    with pytest.raises(tlq.TlqError) as e:
        tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.from_numpy(imp).cuda(), cfg, per_token=True)
    assert e.value.status == tlq.ERR_INVALID_ARG
    # every weight zero: no loss is defined, reported through the status word, not as a fault
    with pytest.raises(tlq.TlqError) as e:
        tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.zeros(64).cuda(), cfg)
    assert e.value.status == tlq.ERR_NONFINITE


# ----------------------------------------------------------------------------------- the CTA-pair GEMM


@pytest.mark.parametrize("n,c1,c2,group,n_grid", [(256, 512, 512, 128, 20), (300, 288, 320, 32, 5), (130, 128, 100, 64, 3),
                                                  (1, 64, 8, 32, 2), (515, 1088, 777, 64, 6), (1000, 512, 256, 128, 4)])
@pytest.mark.parametrize("variant", ["pairs", "narrow"])
def test_search_on_cta_pairs(tlq, n, c1, c2, group, n_grid, variant):
    """The search with the other variants of the fused GEMM (the default is one CTA per 256-token tile): 256-token
    tiles across two SMs (CTA pairs) and 128-token tiles; oracle parity, including the odd-tile and ragged cases
    where the second half of a 256-token tile has no tokens."""
    gemm_flag = tlq.FLAG_GEMM_CTA_PAIRS if variant == "pairs" else tlq.FLAG_GEMM_NARROW_TILES
    xb, wb, imp = wl.small_case(101, n, c1, c2)
    ref = orc.scale_search(xb, wb, imp, "w4a16", group, n_grid)
    cfg = tlq.config(group_size=group, n_grid=n_grid, flags=gemm_flag)
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.from_numpy(imp).cuda(), cfg, per_token=True)
    got = dict(best=int(out.best_idx.item()), losses=out.losses.cpu().numpy(), per_token=out.per_token.cpu().numpy(),
               s_best=bits_of(out.s_best))
    check_against_oracle(got, ref, n_grid)
    # with token skipping on top (half of the tokens dead)
    imp2 = imp.copy()
    imp2[::2] = 0.0
    if imp2.sum() == 0.0:
        return
    ref2 = orc.scale_search(xb, wb, imp2, "w4a16", group, n_grid)
    cfg2 = tlq.config(group_size=group, n_grid=n_grid, flags=gemm_flag | tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS)
    out2 = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.from_numpy(imp2).cuda(), cfg2)
    np.testing.assert_allclose(out2.losses.cpu().numpy(), ref2["losses"], rtol=LOSS_RTOL)


# ----------------------------------------------------------------------------------- two activation streams


def _perturbed_stream(xb, seed, rel):
    """A second activation stream: the same tokens with a relative perturbation (what the quantized layers
    before this one would have done to them), rounded to bf16."""
    x = wl.bf16_bits_to_f32(xb)
    noise = np.random.default_rng(seed).standard_normal(x.shape).astype(np.float32)
    return wl.f32_to_bf16_bits(x * (1.0 + rel * noise))


@pytest.mark.parametrize("mode", ["w4a16", "w8a8", "w4a8"])
@pytest.mark.parametrize("n,c1,c2,n_grid,rel", [(256, 512, 512, 20, 0.02), (300, 288, 320, 5, 0.1), (130, 128, 100, 3, 0.5),
                                                (515, 1088, 777, 6, 0.02), (1, 64, 8, 2, 0.1)])
def test_two_stream_search(tlq, mode, n, c1, c2, n_grid, rel):
    """First propagation strategy of Sec. 3.2.1: reference output from x_fp, quantized layer (and scale) from x_q."""
    xf, wb, imp = wl.small_case(121, n, c1, c2)
    xq = _perturbed_stream(xf, 7, rel)
    if mode == "w4a16":
        cfg = tlq.config(group_size=32, n_grid=n_grid)
        ref = orc.scale_search(xq, wb, imp, "w4a16", 32, n_grid, x_fp_bits=xf)
    else:
        wn, an = orc.symmetric_bits(mode)
        cfg = tlq.config(tlq.WA_SYM_CHANNEL, w_bits=wn, a_bits=an, n_grid=n_grid)
        ref = orc.scale_search(xq, wb, imp, mode, 0, n_grid, x_fp_bits=xf)
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xq), dev_bf16(tlq, wb), torch.from_numpy(imp).cuda(), cfg,
                                     per_token=True, X_fp=dev_bf16(tlq, xf))
    got = dict(best=int(out.best_idx.item()), losses=out.losses.cpu().numpy(), per_token=out.per_token.cpu().numpy(),
               s_best=bits_of(out.s_best))
    check_against_oracle(got, ref, n_grid)


def test_two_stream_with_equal_streams_is_the_plain_search(tlq):
    xb, wb, imp = wl.small_case(123, 384, 256, 320)
    cfg = tlq.config(group_size=64, n_grid=6)
    w_dev = torch.from_numpy(imp).cuda()
    one = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), w_dev, cfg, per_token=True)
    two = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), w_dev, cfg, per_token=True, X_fp=dev_bf16(tlq, xb))
    assert int(one.best_idx.item()) == int(two.best_idx.item())
    # X W^T - X W^T cancels exactly in the fp32 accumulator, what remains is the same X dW^T
    np.testing.assert_allclose(two.per_token.cpu().numpy(), one.per_token.cpu().numpy(), rtol=1e-5)
    with pytest.raises(tlq.TlqError) as e:
        tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), w_dev,
                                   tlq.config(group_size=64, n_grid=6, flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS),
                                   X_fp=dev_bf16(tlq, xb))
    assert e.value.status == tlq.ERR_INVALID_ARG


# ----------------------------------------------------------------------------------- grid extremes


@pytest.mark.parametrize("mode", ["w4a16", "w8a8"])
@pytest.mark.parametrize("n_grid", [1, 64])
def test_grid_of_one_and_of_the_maximum(tlq, mode, n_grid):
    """K = 1 (only scale = 1, plain round-to-nearest) and K = 64 (TLQ_MAX_GRID); K = 65 is refused."""
    xb, wb, imp = wl.small_case(141, 200, 128, 96)
    if mode == "w4a16":
        cfg = tlq.config(group_size=64, n_grid=n_grid)
        ref = orc.scale_search(xb, wb, imp, "w4a16", 64, n_grid)
    else:
        cfg = tlq.config(tlq.W8A8_SYM, n_grid=n_grid)
        ref = orc.scale_search(xb, wb, imp, "w8a8", 0, n_grid)
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.from_numpy(imp).cuda(), cfg, per_token=True)
    got = dict(best=int(out.best_idx.item()), losses=out.losses.cpu().numpy(), per_token=out.per_token.cpu().numpy(),
               s_best=bits_of(out.s_best))
    check_against_oracle(got, ref, n_grid)
    if n_grid == 1:
        assert got["best"] == 0 and np.all(wl.bf16_bits_to_f32(got["s_best"]) == 1.0)
    assert tlq.tlq_scale_search_workspace_bytes(200, 128, 96, tlq.config(n_grid=65)) == 0


def test_four_bit_packing_bit_exact(tlq):
    wb = wl.weights(161, "pack/w", 77, 1056)
    s_np = orc.scale_table(orc.channel_stat(wl.activations(161, "pack/x", 64, 1056, 48)), 20)[7]
    s_dev = dev_bf16(tlq, orc.f32_to_bf16_bits(s_np))
    out = tlq.tlq_quantize_weights(dev_bf16(tlq, wb), s_dev, tlq.config(group_size=32))
    codes, _, _, _ = orc.quantize_weights_group_asym(wb, s_np, 32, 4)
    assert np.array_equal(tlq.tlq_pack_codes4(out["codes"]).cpu().numpy(), orc.pack_codes4(codes))
    sym = tlq.tlq_quantize_weights(dev_bf16(tlq, wb), s_dev, tlq.config(tlq.WA_SYM_CHANNEL, w_bits=4, a_bits=8))
    qw, _ = orc.quantize_weights_row_sym(wb, s_np, 4)
    packed = tlq.tlq_pack_codes4(sym["codes"]).cpu().numpy()
    assert np.array_equal(packed, orc.pack_codes4(qw))
    assert np.array_equal(orc.unpack_codes4(packed, signed=True), qw)


# ----------------------------------------------------------------------------------- chained layers, row shards


@pytest.mark.parametrize("mode", ["w4a16", "w4a8"])
def test_chain_search_apply_then_search_of_the_next_linear(tlq, mode):
    """Quantization-exposed calibration of two linears in a row (Sec. 3.2.1): search linear A, apply it with the
    winning scale, and calibrate linear B on what A's quantized form produced, once under the second propagation
    strategy (B sees only the quantized stream) and once under the first (reference output from the full-precision
    stream).  The oracle is fed the very bf16 bits the CUDA path produced for the quantized stream."""
    xa, wa, imp = wl.small_case(131, 300, 256, 512)
    _, wb, _ = wl.small_case(132, 300, 512, 320)
    n_grid = 6
    if mode == "w4a16":
        cfg, group = tlq.config(group_size=64, n_grid=n_grid), 64
    else:
        wn, an = orc.symmetric_bits(mode)
        cfg, group = tlq.config(tlq.WA_SYM_CHANNEL, w_bits=wn, a_bits=an, n_grid=n_grid), 0
    w_dev = torch.from_numpy(imp).cuda()
    Xa, Wa, Wb = dev_bf16(tlq, xa), dev_bf16(tlq, wa), dev_bf16(tlq, wb)
    # linear A
    ref_a = orc.scale_search(xa, wa, imp, mode, group, n_grid)
    out_a = tlq.tlq_scale_search_layer(Xa, Wa, w_dev, cfg)
    assert_same_argmin(int(out_a.best_idx.item()), ref_a)
    assert np.array_equal(bits_of(out_a.s_best), orc.f32_to_bf16_bits(ref_a["scales"][ref_a["best"]]))
    # its quantized form applied to the calibration tokens: the next linear's input
    applied = tlq.tlq_apply_layer(Xa, Wa, out_a.s_best, None, cfg, want_codes=False)
    yq_bits = bits_of(applied["Yq"])
    yq_ref, _ = orc.apply_layer(xa, wa, ref_a["scales"][ref_a["best"]], None, mode, group if group else 128)
    e_a = ref_a["per_token"][ref_a["best"]]
    d2 = ((orc.bf16_to_f64(yq_bits) - yq_ref) ** 2).sum(axis=1)
    y2 = (yq_ref ** 2).sum(axis=1)
    assert np.all(d2 <= 2.0 ** -14 * (y2 + e_a))          # bf16 output rounding: 2^-8 relative per element, squared
    # the full-precision stream of the same tokens (what the unquantized layer A produces), as bf16
    yfp_bits = wl.f32_to_bf16_bits(orc.layer_fp(xa, wa).astype(np.float32))
    # second strategy: B calibrated on the quantized stream alone
    ref_b = orc.scale_search(yq_bits, wb, imp, mode, group, n_grid)
    out_b = tlq.tlq_scale_search_layer(applied["Yq"], Wb, w_dev, cfg, per_token=True)
    got_b = dict(best=int(out_b.best_idx.item()), losses=out_b.losses.cpu().numpy(), per_token=out_b.per_token.cpu().numpy(),
                 s_best=bits_of(out_b.s_best))
    check_against_oracle(got_b, ref_b, n_grid)
    # first strategy: reference from the full-precision stream, quantized layer from the quantized stream
    ref_two = orc.scale_search(yq_bits, wb, imp, mode, group, n_grid, x_fp_bits=yfp_bits)
    out_two = tlq.tlq_scale_search_layer(applied["Yq"], Wb, w_dev, cfg, per_token=True, X_fp=dev_bf16(tlq, yfp_bits))
    got_two = dict(best=int(out_two.best_idx.item()), losses=out_two.losses.cpu().numpy(),
                   per_token=out_two.per_token.cpu().numpy(), s_best=bits_of(out_two.s_best))
    check_against_oracle(got_two, ref_two, n_grid)
    # the two-stream loss contains the error A already made, so it can only be larger
    assert np.all(got_two["losses"] > got_b["losses"])


@pytest.mark.parametrize("mode", ["w4a16", "w8a8"])
def test_row_sharded_search_combines_to_the_unsharded_result(tlq, mode):
    """One linear cut by output rows over two ranks (run one after the other on this GPU): quantizers never cross
    rows, so the slices' losses, weighted by their row counts, add up to the unsharded search."""
    from paper_2602_07899_b200 import replicas
    xb, wb, imp = wl.small_case(171, 300, 256, 333)
    n_grid = 6
    if mode == "w4a16":
        cfg, group = tlq.config(group_size=64, n_grid=n_grid), 64
    else:
        cfg, group = tlq.config(tlq.W8A8_SYM, n_grid=n_grid), 0
    w_dev = torch.from_numpy(imp).cuda()
    X = dev_bf16(tlq, xb)
    ref = orc.scale_search(xb, wb, imp, mode, group, n_grid)
    whole = tlq.tlq_scale_search_layer(X, dev_bf16(tlq, wb), w_dev, cfg, per_token=True)
    summed, per_token, rows = None, None, 0
    for rank in range(2):
        info = replicas.RankInfo(rank, 2, 0)
        r0, r1 = replicas.shard_rows(333, info)
        part = tlq.tlq_scale_search_layer(X, dev_bf16(tlq, wb[r0:r1]), w_dev, cfg, per_token=True)
        t = replicas.weighted_slice_losses(part.losses, r1 - r0)
        summed = t if summed is None else summed + t        # stands in for the SUM reduction over the ranks
        per_token = part.per_token.double() if per_token is None else per_token + part.per_token.double()
        rows += r1 - r0
        assert bits_of(part.s_best).shape == (256,)
    assert rows == 333
    losses, best = replicas.finish_sharded_losses(summed, 333)
    np.testing.assert_allclose(losses.cpu().numpy(), whole.losses.cpu().numpy(), rtol=2e-6)
    np.testing.assert_allclose(per_token.cpu().numpy(), whole.per_token.double().cpu().numpy(), rtol=2e-6)
    np.testing.assert_allclose(losses.cpu().numpy(), ref["losses"], rtol=LOSS_RTOL)
    assert best == int(whole.best_idx.item())
    assert_same_argmin(best, ref)


def test_row_quantizers_on_very_wide_rows(tlq):
    """A few rows of more than a hundred thousand channels (224 column tiles per row, every row maximum combined
    from that many partial maxima): same contract."""
    c1 = 114688
    xb = wl.activations(191, "wide/x", 6, c1, 4, "normal", 4)
    wb = wl.weights(191, "wide/w", 5, c1)
    s_np = orc.scale_table(orc.channel_stat(xb), 20)[9]
    s_dev = dev_bf16(tlq, orc.f32_to_bf16_bits(s_np))
    cfg = tlq.config(tlq.W8A8_SYM)
    out = tlq.tlq_quantize_weights(dev_bf16(tlq, wb), s_dev, cfg)
    codes, steps = tlq.tlq_quantize_activations(dev_bf16(tlq, xb), s_dev, cfg)
    qw, u = orc.quantize_weights_row_sym(wb, s_np)
    qx, t = orc.quantize_activations_token_sym(xb, s_np)
    assert np.array_equal(out["codes"].cpu().numpy(), qw) and np.array_equal(out["steps"].cpu().numpy(), u)
    assert np.array_equal(codes.cpu().numpy(), qx) and np.array_equal(steps.cpu().numpy(), t)


@pytest.mark.parametrize("n,c2", [(2048, 2048), (2304, 1792), (2100, 2000)])
def test_search_with_the_l2_partition_aware_tile_walk(tlq, n, c2):
    """Large enough for the 256-token kernel to run one CTA per SM with the tile space split between the two L2
    partitions (when the device's partition table could be measured): same results, every slot claimed once.
    The whole per-token table is compared, so a tile that no CTA visited would show as a missing share of 256
    tokens' errors.  Even, odd and ragged tile counts (the cut between the partitions moves with the candidate)."""
    xb, wb, imp = wl.small_case(211, n, 512, c2)
    ref = orc.scale_search(xb, wb, imp, "w4a16", 128, 20)
    for _ in range(2):      # the first large call on a device also measures the table
        got = run_search(tlq, xb, wb, imp)
        check_against_oracle(got, ref, 20)
    cfg = tlq.config()
    out = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.from_numpy(imp).cuda(), cfg)
    hdr = out.workspace[:256].view(torch.int32).cpu().numpy()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert hdr[0] == 0 and int(hdr[5]) + int(hdr[6]) in (0, sms), hdr[:8]
    print("tile-walk slots claimed per L2 partition:", int(hdr[5]), int(hdr[6]))
    info = tlq.tlq_l2_partition_info()
    if info["valid"]:      # the walk used the table: as many slots per partition as the table has SMs
        assert info["n_sms"] == sms and sum(info["count"]) == sms and min(info["count"]) * 4 >= sms
        assert (int(hdr[5]), int(hdr[6])) == info["count"]
        assert int(info["part"][:].max()) == 1
    else:
        assert int(hdr[5]) + int(hdr[6]) == 0
    # token skipping on top: the live token count, and with it the split, is only known on the device
    imp2 = imp.copy()
    imp2[np.random.default_rng(3).random(n) < 0.4] = 0.0
    ref2 = orc.scale_search(xb, wb, imp2, "w4a16", 128, 20)
    cfg2 = tlq.config(flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS)
    out2 = tlq.tlq_scale_search_layer(dev_bf16(tlq, xb), dev_bf16(tlq, wb), torch.from_numpy(imp2).cuda(), cfg2)
    np.testing.assert_allclose(out2.losses.cpu().numpy(), ref2["losses"], rtol=LOSS_RTOL)
    assert_same_argmin(int(out2.best_idx.item()), ref2)
