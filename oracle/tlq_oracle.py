"""CPU oracle for the token-importance-weighted, quantization-exposed scale search (TLQ).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the hot path computes,
written from the paper; only tests, the smoke check and the benchmark's CPU-baseline leg may import
it.  It shares no code with the CUDA path and never imports it.  numpy only; float64 everywhere
except at the named contract points below.

What the paper fixes, and where each function comes from:
  * quantizer: X_hat = round(X / s_i), s_i = max_j |X_ij| / (2^(n-1) - 1), integers in
    [-2^(n-1), 2^(n-1)-1]; per token for activations, per output channel for weights
    (Sec. 2.2, first two equations and the integer-range sentence).  The asymmetric variant
    is only said to be handled analogously (same section); its formula here is a reading (min/max affine grid).
  * smoothing: Y = (X diag(scale)^-1)(diag(scale) W) (Sec. 2.2, per-channel smoothing equation);
    scale indexes the input channels of W in R^{C2 x C1}.
  * scale = x_stat^r (Sec. 3.1.2, first equation), x_stat_c = max over the selected tokens of
    |X_ic| (second equation), with mean / max over all tokens as the ablation variants (Table 2).
  * search: r* = argmin_r E || f_fp(x) - f_q(x; scale) ||^2, f_fp = W x + b,
    f_q = Q_w(W * scale) Q_a(x / scale) + b (Sec. 3.2.1).
  * token importance: sum_n = sum_b ||g_{b,n}||, where the surrounding text describes the norm as the
    channel mean of the absolute gradient; I = the top half of the tokens by sum_n (Sec. 3.1.2, last two
    equations).

Contract points (where floating point decides an integer the decision is taken in binary32, the
precision of the CUDA kernels; everything else is float64): the product scale*w (exact in binary32
for bf16 factors), the group range, the step, the zero-point quotient, the code quotient, the
dequantized value, the reciprocal of the scale and the product with it.  They are written with
numpy float32 arrays, one IEEE operation per statement.

Readings of points the paper leaves open, each stated where it is used below: the grid r_k = k/K
(grid_ratio), bfloat16 storage of the scale (scale_table), half-to-even rounding (np.rint), the floors
on degenerate statistics (_STAT_FLOOR, _RANGE_FLOOR), diag(scale)^-1 taken as a product with the
binary32 reciprocal (quantize_weights_group_asym, quantize_activations_token_sym) and the loss
normalisation by C2 * sum(w) (weighted_loss).

Parity pins: tests/test_oracle_pins.py holds, for every function here, closed forms, hand-computed
values, invariants, library conversions or a scalar brute force on tiny inputs.  The paper prints no
worked numeric example, so absolute values are pinned by those tests alone.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
F64 = np.float64

STAT_MEAN_ABS = 0
STAT_MAX_ABS = 1
STAT_MASKED_MAX = 2

NORM_MEAN_ABS = 0
NORM_L2 = 1

_STAT_FLOOR = 2.0 ** -20      # floor on x_stat (silent in the paper: a dead channel keeps scale finite)
_RANGE_FLOOR = F32(1e-5)      # floor on a group's range / a row's amax (flat group, zero row)


# ----------------------------------------------------------------------------- bf16


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Values denoted by bfloat16 bit patterns, as float64 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(F64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (ties to even); returns float32 values.

    float64 -> bfloat16 is done in one rounding: bfloat16 keeps 8 significand bits, so the value is
    split at that bit directly in the float64 encoding (52 - 7 = 45 dropped bits).  Inputs are
    assumed finite and within bfloat16's normal range.
    """
    u = np.ascontiguousarray(x, dtype=F64).view(np.uint64)
    drop = np.uint64(45)
    half = (np.uint64(1) << (drop - np.uint64(1))) - np.uint64(1)
    lsb = (u >> drop) & np.uint64(1)
    r = ((u + half + lsb) >> drop) << drop
    return r.view(F64).astype(F32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bfloat16-representable."""
    return (np.ascontiguousarray(x, dtype=F32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# ----------------------------------------------------------------------------- scale candidates


def channel_stat(x_bits: np.ndarray, stat_mode: int = STAT_MEAN_ABS, mask: np.ndarray | None = None) -> np.ndarray:
    """x_stat_c over tokens: mean |X| (AWQ-style; the paper's x_mean ablation row), max |X| (x_max
    row) or max over the selected tokens I (Sec. 3.1.2, second equation).  float64 [C1]."""
    a = np.abs(bf16_to_f64(x_bits))
    if stat_mode == STAT_MEAN_ABS:
        return a.sum(axis=0) / F64(a.shape[0])
    if stat_mode == STAT_MAX_ABS:
        return a.max(axis=0)
    if stat_mode == STAT_MASKED_MAX:
        sel = np.asarray(mask).astype(bool)
        if not sel.any():
            raise ValueError("empty token selection")
        return a[sel].max(axis=0)
    raise ValueError(stat_mode)


def grid_ratio(k: int, n_grid: int) -> float:
    """r_k = k / K, k = 0..K-1 (the paper only says r is found by a search; this is the grid reading)."""
    return float(k) / float(n_grid)


def scale_table(x_stat: np.ndarray, n_grid: int) -> np.ndarray:
    """scale_{k,c} = x_stat_c ^ r_k (Sec. 3.1.2 first equation / Sec. 3.2.1 first equation), rounded
    once to bfloat16 (the scale is stored in the model's 16-bit type when it is folded into the
    preceding layer).  float32 values [K, C1]; row 0 is exactly 1."""
    m = np.maximum(np.asarray(x_stat, dtype=F64), F64(_STAT_FLOOR))
    tab = np.empty((n_grid, m.shape[0]), dtype=F32)
    for k in range(n_grid):
        tab[k] = round_to_bf16(np.power(m, F64(grid_ratio(k, n_grid))))
    return tab


# ----------------------------------------------------------------------------- weight quantizers


def quantize_weights_group_asym(w_bits: np.ndarray, s: np.ndarray | None, group: int, bits: int = 4):
    """Q_w(W * scale) for the group-wise asymmetric setting: every `group` consecutive input channels
    of one output row share a step and an integer zero-point.

    Returns (codes uint8 [C2,C1], step float32 [C2,C1/G], zero int32 [C2,C1/G], w_hat float32 [C2,C1])
    where w_hat = dequant * (1/scale) is the weight the quantized layer effectively applies to the
    unscaled activations (Sec. 2.2 smoothing identity); 1/scale is the same binary32 reciprocal that
    smooths the activations in quantize_activations_token_sym.
    """
    w = bf16_to_f64(w_bits)
    c2, c1 = w.shape
    if c1 % group:
        raise ValueError("C1 must be a multiple of the group size")
    sv = np.ones(c1, dtype=F64) if s is None else np.asarray(s, dtype=F64)
    qmax = (1 << bits) - 1
    p = (w * sv[None, :]).astype(F32)                     # exact: 8-bit x 8-bit significands
    pg = p.reshape(c2, c1 // group, group)
    mx = pg.max(axis=2)
    mn = pg.min(axis=2)
    rng = (mx - mn).astype(F32)                           # binary32 subtraction
    rng = np.maximum(rng, _RANGE_FLOOR)
    step = (rng / F32(qmax)).astype(F32)                  # binary32 division
    zq = (mn / step).astype(F32)                          # binary32 division
    zero = np.clip(-np.rint(zq).astype(np.int64), 0, qmax).astype(np.int32)
    cq = (pg / step[:, :, None]).astype(F32)              # binary32 division
    codes = np.clip(np.rint(cq).astype(np.int64) + zero[:, :, None], 0, qmax)
    dq = ((codes - zero[:, :, None]).astype(F32) * step[:, :, None]).astype(F32)   # binary32 product
    rs = (F32(1.0) / sv.astype(F32)).astype(F32)                                   # binary32 reciprocal of the scale
    w_hat = (dq.reshape(c2, c1) * rs[None, :]).astype(F32)                         # binary32 product
    return codes.reshape(c2, c1).astype(np.uint8), step, zero, w_hat


def delta_weights_bf16(w_bits: np.ndarray, w_hat: np.ndarray) -> np.ndarray:
    """W - W_hat rounded to binary32 and then to bfloat16 (bit patterns): the operand a fused kernel
    may feed its tensor cores.  Not used by the search below; provided so tests can check that
    operand bit for bit."""
    d = (bf16_to_f64(w_bits).astype(F32) - np.asarray(w_hat, dtype=F32)).astype(F32)
    return f32_to_bf16_bits(round_to_bf16(d.astype(F64)))


def quantize_sym_rows(v: np.ndarray, bits: int = 8):
    """X_hat = round(X / s_i), s_i = max_j |X_ij| / (2^(n-1)-1) for every row i of a float32 matrix
    (Sec. 2.2 first two equations); integers clamped to [-2^(n-1), 2^(n-1)-1].
    Returns (codes int8 [R,C], step float32 [R])."""
    v = np.asarray(v, dtype=F32)
    qpos = (1 << (bits - 1)) - 1
    amax = np.maximum(np.abs(v).max(axis=1), _RANGE_FLOOR)
    step = (amax / F32(qpos)).astype(F32)                 # binary32 division
    q = (v / step[:, None]).astype(F32)                   # binary32 division
    codes = np.clip(np.rint(q).astype(np.int64), -(qpos + 1), qpos)
    return codes.astype(np.int8), step


def quantize_weights_row_sym(w_bits: np.ndarray, s: np.ndarray | None, bits: int = 8):
    """Per-output-channel symmetric Q_w(W * scale). Returns (codes int8 [C2,C1], step u float32 [C2])."""
    w = bf16_to_f64(w_bits)
    sv = np.ones(w.shape[1], dtype=F64) if s is None else np.asarray(s, dtype=F64)
    p = (w * sv[None, :]).astype(F32)                     # exact
    return quantize_sym_rows(p, bits)


def quantize_activations_token_sym(x_bits: np.ndarray, s: np.ndarray | None, bits: int = 8):
    """Per-token symmetric Q_a(x / scale).  The smoothed activation is x * (1/scale) with the
    reciprocal and the product each rounded to binary32 (the scale's reciprocal is what gets folded
    into the preceding layer).  Returns (codes int8 [N,C1], step t float32 [N])."""
    x = bf16_to_f64(x_bits).astype(F32)
    if s is None:
        xt = x
    else:
        rs = (F32(1.0) / np.asarray(s, dtype=F32)).astype(F32)     # binary32 reciprocal
        xt = (x * rs[None, :]).astype(F32)                         # binary32 product
    return quantize_sym_rows(xt, bits)


def pack_codes4(codes: np.ndarray) -> np.ndarray:
    """Two 4-bit codes per byte, the even channel in the low nibble (a storage format: with n = 4 the
    integer range of Sec. 2.2 has sixteen levels).  Signed codes keep their two's-complement nibble."""
    c = np.asarray(codes).astype(np.int64) & 15
    return (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)


def unpack_codes4(packed: np.ndarray, signed: bool) -> np.ndarray:
    """Inverse of pack_codes4: [R,C/2] bytes -> [R,C] integers in 0..15, or -8..7 when `signed`."""
    p = np.asarray(packed, dtype=np.uint8).astype(np.int64)
    out = np.empty((p.shape[0], 2 * p.shape[1]), dtype=np.int64)
    out[:, 0::2] = p & 15
    out[:, 1::2] = p >> 4
    return np.where(out >= 8, out - 16, out) if signed else out


# ----------------------------------------------------------------------------- the layer, its error, the search


def layer_fp(x_bits: np.ndarray, w_bits: np.ndarray, bias: np.ndarray | None = None) -> np.ndarray:
    """f_fp(x) = W x + b for every token: Y = X W^T + b, float64 [N,C2] (Sec. 3.2.1)."""
    y = bf16_to_f64(x_bits) @ bf16_to_f64(w_bits).T
    return y if bias is None else y + np.asarray(bias, dtype=F64)[None, :]


def layer_q_w4a16(x_bits: np.ndarray, w_hat: np.ndarray, bias: np.ndarray | None = None) -> np.ndarray:
    """f_q with 16-bit activations (Q_a = identity): Y_q = X W_hat^T + b, float64."""
    y = bf16_to_f64(x_bits) @ np.asarray(w_hat, dtype=F64).T
    return y if bias is None else y + np.asarray(bias, dtype=F64)[None, :]


def layer_q_w8a8(qx: np.ndarray, t: np.ndarray, qw: np.ndarray, u: np.ndarray,
                 bias: np.ndarray | None = None) -> np.ndarray:
    """f_q = Q_w(W*scale) Q_a(x/scale) + b with integer codes: Y_q[n,o] = t_n u_o sum_c qx qw, float64."""
    acc = qx.astype(F64) @ qw.astype(F64).T               # integers < 2^53: exact
    y = acc * np.asarray(t, dtype=F64)[:, None] * np.asarray(u, dtype=F64)[None, :]
    return y if bias is None else y + np.asarray(bias, dtype=F64)[None, :]


def per_token_error(y_fp: np.ndarray, y_q: np.ndarray) -> np.ndarray:
    """e_n = || f_fp(x_n) - f_q(x_n) ||_2^2 (the norm inside the search objective), float64 [N]."""
    d = y_fp - y_q
    return np.einsum("no,no->n", d, d)


def weighted_loss(e: np.ndarray, w_imp: np.ndarray | None, c_out: int) -> float:
    """sum_n w_n e_n / (C2 sum_n w_n): with constant w this is the plain expectation of Sec. 3.2.1
    (mean squared output error); with a 0/1 selection it is that expectation over the selected
    tokens.  Non-finite results are reported as +inf."""
    e = np.asarray(e, dtype=F64)
    w = np.ones_like(e) if w_imp is None else np.asarray(w_imp, dtype=F64)
    v = float((w * e).sum() / (F64(c_out) * w.sum()))
    return v if np.isfinite(v) else float("inf")


def argmin_lowest(losses: np.ndarray) -> int:
    """Index of the minimum, the lowest index on ties."""
    best, idx = float("inf"), -1
    for k, v in enumerate(losses):
        if v < best:
            best, idx = float(v), k
    return idx


def symmetric_bits(mode: str) -> tuple[int, int]:
    """(weight bits, activation bits) of a per-channel / per-token symmetric setting named "w<n>a<m>":
    "w8a8", and the paper's main settings "w4a8" and "w4a6" (Experiments, quantization settings:
    per-token symmetric activations, per-channel symmetric weights)."""
    if not (mode.startswith("w") and "a" in mode[1:]):
        raise ValueError(mode)
    n, m = mode[1:].split("a", 1)
    n, m = int(n), int(m)
    if not (2 <= n <= 8 and 2 <= m <= 8):
        raise ValueError(mode)
    return n, m


def candidate_error(x_bits, w_bits, s_k, mode: str, group: int, y_fp: np.ndarray | None = None,
                    w_bits_n: int = 4) -> np.ndarray:
    """Per-token squared output error of one scale candidate, float64 [N].
    mode "w4a16": group-wise asymmetric `w_bits_n`-bit weights, activations untouched;
    mode "w<n>a<m>" otherwise: symmetric n-bit weights per output channel, m-bit activations per token."""
    if y_fp is None:
        y_fp = layer_fp(x_bits, w_bits)
    if mode == "w4a16":
        _, _, _, w_hat = quantize_weights_group_asym(w_bits, s_k, group, w_bits_n)
        y_q = layer_q_w4a16(x_bits, w_hat)
    else:
        wn, an = symmetric_bits(mode)
        qw, u = quantize_weights_row_sym(w_bits, s_k, wn)
        qx, t = quantize_activations_token_sym(x_bits, s_k, an)
        y_q = layer_q_w8a8(qx, t, qw, u)
    return per_token_error(y_fp, y_q)


def scale_search(x_bits: np.ndarray, w_bits: np.ndarray, w_imp: np.ndarray | None, mode: str = "w4a16",
                 group: int = 128, n_grid: int = 20, stat_mode: int = STAT_MEAN_ABS,
                 mask: np.ndarray | None = None, w_bits_n: int = 4, x_fp_bits: np.ndarray | None = None):
    """The layer-wise search of Sec. 3.2.1 over the grid r_k = k/K, in the paper's order:
    x_stat -> scale(r) -> quantize the scaled weights (and smoothed activations) -> apply the
    quantized layer to the calibration tokens -> squared output error per token -> importance-
    weighted mean -> argmin.

    `x_fp_bits` selects the paper's first propagation strategy (Sec. 3.2.1, PassAct1): two activation
    streams, the full-precision layer sees x_fp (output of the full-precision layers before it) while the
    quantized layer, and the statistic behind its scale, see `x_bits` (output of the already quantized
    layers): loss = || f_fp(x_fp) - f_q(x_q; scale) ||^2.  Without it both see `x_bits`.

    Returns dict(best, losses float64 [K], per_token float64 [K,N], scales float32 [K,C1], x_stat).
    """
    x_stat = channel_stat(x_bits, stat_mode, mask)
    scales = scale_table(x_stat, n_grid)
    y_fp = layer_fp(x_bits if x_fp_bits is None else x_fp_bits, w_bits)
    c_out = w_bits.shape[0]
    per_token = np.empty((n_grid, x_bits.shape[0]), dtype=F64)
    losses = np.empty(n_grid, dtype=F64)
    for k in range(n_grid):
        per_token[k] = candidate_error(x_bits, w_bits, scales[k], mode, group, y_fp, w_bits_n)
        losses[k] = weighted_loss(per_token[k], w_imp, c_out)
    return dict(best=argmin_lowest(losses), losses=losses, per_token=per_token, scales=scales, x_stat=x_stat)


def apply_layer(x_bits, w_bits, s, bias_bits, mode: str = "w4a16", group: int = 128, w_bits_n: int = 4):
    """f_q(x; scale) for the chosen scale (what the next layer receives under the paper's second
    propagation strategy, Sec. 3.2.1 PassAct2).  Returns (Y_q float64 [N,C2], quantizer outputs)."""
    b = None if bias_bits is None else bf16_to_f64(bias_bits)
    if mode == "w4a16":
        codes, step, zero, w_hat = quantize_weights_group_asym(w_bits, s, group, w_bits_n)
        return layer_q_w4a16(x_bits, w_hat, b), (codes, step, zero)
    wn, an = symmetric_bits(mode)
    qw, u = quantize_weights_row_sym(w_bits, s, wn)
    qx, t = quantize_activations_token_sym(x_bits, s, an)
    return layer_q_w8a8(qx, t, qw, u, b), (qw, u, None)


# ----------------------------------------------------------------------------- token importance


def token_importance(g_bits: np.ndarray, norm_kind: int = NORM_MEAN_ABS, top_frac: float = 0.0,
                     g_is_f32: bool = False):
    """sum_n = sum_b || g_{b,n} || (Sec. 3.1.2): per sample the absolute gradient averaged over the
    channel dimension (text) or the L2 norm (equation), summed over the B samples; then the
    top `top_frac` of the positions form the selection I (count floor(frac*N), at least 1; equal
    values keep the lower index).  Returns (imp float64 [N], mask uint8 [N] or None)."""
    g = np.asarray(g_bits, dtype=F64) if g_is_f32 else bf16_to_f64(g_bits)
    if g.ndim == 2:
        g = g[None]
    if norm_kind == NORM_MEAN_ABS:
        per = np.abs(g).sum(axis=2) / F64(g.shape[2])
    elif norm_kind == NORM_L2:
        per = np.sqrt((g * g).sum(axis=2))
    else:
        raise ValueError(norm_kind)
    imp = per.sum(axis=0)
    if top_frac <= 0.0:
        return imp, None
    return imp, top_mask(imp, top_frac)


def top_mask(imp: np.ndarray, top_frac: float) -> np.ndarray:
    """I = Top_frac({sum_n}) as a 0/1 vector."""
    n = imp.shape[0]
    k_sel = max(1, int(np.floor(top_frac * n)))
    order = sorted(range(n), key=lambda i: (-float(imp[i]), i))
    mask = np.zeros(n, dtype=np.uint8)
    mask[order[:k_sel]] = 1
    return mask
