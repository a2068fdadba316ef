"""Seeded synthetic calibration workloads (inputs only; none of the method's arithmetic).

The paper calibrates on 128 image-caption pairs pushed through a VLM (Experiments, "Calibration
Datasets"); neither the pairs nor the models exist here, so these generators stand in for the
*shapes and distributions* of one decoder layer's calibration activations, weights, token
importance and token gradients.  Every tensor is a pure function of (seed, tensor name, shape):
a Philox counter-based stream keyed by the seed and a per-tensor id, drawn on the host in a fixed
chunk order and rounded to bfloat16 (round-to-nearest-even) where the tensor is bf16.

The module serves both the CPU oracle's tests and the CUDA path's tests/bench, so it must stay
free of anything the method computes (no scales, quantizers, errors or reductions).
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Dict, List, Optional, Tuple

import numpy as np

BASE_SEED = 20260207

# ----------------------------------------------------------------------------- bf16 containers


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest, ties to even) and return the uint16 bits."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to the float32 values they denote (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, name: str) -> np.random.Generator:
    tid = zlib.crc32(name.encode("utf-8"))
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(tid)]))


_CHUNK_ROWS = 1024  # fixed draw order: row blocks of this height, row-major inside a block


# ----------------------------------------------------------------------------- tensors


def activations(seed: int, name: str, n_tokens: int, channels: int, n_visual: int,
                dist: str = "normal", n_outlier: int = 4,
                text_gain: float = 20.0, visual_gain: float = 5.0) -> np.ndarray:
    """bf16 bits [n_tokens, channels]: rows [0, n_visual) are visual tokens, the rest text.

    dist "normal" is N(0,1); "student3" is Student-t with 3 degrees of freedom (a normal over the
    root of a chi-square/3).  `n_outlier` seeded channels are multiplied by `text_gain` on text
    rows and `visual_gain` on visual rows.
    """
    g = _rng(seed, name)
    picks = _rng(seed, name + "/outlier_channels").permutation(channels)[:n_outlier]
    out = np.empty((n_tokens, channels), dtype=np.uint16)
    for r0 in range(0, n_tokens, _CHUNK_ROWS):
        r1 = min(n_tokens, r0 + _CHUNK_ROWS)
        blk = g.standard_normal((r1 - r0, channels), dtype=np.float32)
        if dist == "student3":
            chi = np.zeros_like(blk)
            for _ in range(3):
                z = g.standard_normal(blk.shape, dtype=np.float32)
                chi += z * z
            blk = blk / np.sqrt(chi / np.float32(3.0))
        elif dist != "normal":
            raise ValueError(dist)
        rows = np.arange(r0, r1)
        gain = np.where(rows < n_visual, np.float32(visual_gain), np.float32(text_gain)).astype(np.float32)
        blk[:, picks] *= gain[:, None]
        out[r0:r1] = f32_to_bf16_bits(blk)
    return out


def weights(seed: int, name: str, c_out: int, c_in: int, std: float = 0.02) -> np.ndarray:
    """bf16 bits [c_out, c_in] ~ N(0, std^2)."""
    g = _rng(seed, name)
    out = np.empty((c_out, c_in), dtype=np.uint16)
    for r0 in range(0, c_out, _CHUNK_ROWS):
        r1 = min(c_out, r0 + _CHUNK_ROWS)
        out[r0:r1] = f32_to_bf16_bits(g.standard_normal((r1 - r0, c_in), dtype=np.float32) * np.float32(std))
    return out


def importance(seed: int, name: str, n_tokens: int, n_visual: int, kind: str = "lognormal",
               visual_factor: float = 0.2) -> np.ndarray:
    """fp32 [n_tokens] token-importance weights.

    "lognormal": exp(N(0,1)), visual rows times `visual_factor`; "uniform": all ones;
    "onehot": a single seeded token has weight 1.
    """
    g = _rng(seed, name)
    if kind == "lognormal":
        w = np.exp(g.standard_normal(n_tokens)).astype(np.float32)
        w[:n_visual] *= np.float32(visual_factor)
        return w
    if kind == "uniform":
        return np.ones(n_tokens, dtype=np.float32)
    if kind == "onehot":
        w = np.zeros(n_tokens, dtype=np.float32)
        w[int(g.integers(0, n_tokens))] = 1.0
        return w
    raise ValueError(kind)


def token_gradients(seed: int, name: str, n_samples: int, n_tokens: int, channels: int,
                    n_visual: int, zero_frac: float = 0.6) -> np.ndarray:
    """bf16 bits [n_samples, n_tokens, channels] standing in for per-sample output gradients.

    Each token row is N(0,1) times a log-normal token magnitude exp(N(0, 2^2)); a seeded
    `zero_frac` of the visual rows of every sample is exactly zero (the paper's gradient figure
    shows many visual tokens with zero gradient).
    """
    g = _rng(seed, name)
    out = np.empty((n_samples, n_tokens, channels), dtype=np.uint16)
    for b in range(n_samples):
        blk = g.standard_normal((n_tokens, channels), dtype=np.float32)
        mag = np.exp(2.0 * g.standard_normal(n_tokens)).astype(np.float32)
        dead = g.random(n_tokens) < zero_frac
        dead[n_visual:] = False
        mag[dead] = 0.0
        out[b] = f32_to_bf16_bits(blk * mag[:, None])
    return out


# ----------------------------------------------------------------------------- layer configs


@dataclasses.dataclass(frozen=True)
class Linear:
    name: str       # q, k, v, o, gate, up, down
    c_in: int
    c_out: int
    x_name: str     # which activation tensor feeds it (siblings share one)


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    key: str
    hidden: int
    inter: int
    kv: int
    n_tokens: int
    visual_frac: float
    dist: str = "normal"
    n_outlier: int = 4
    mode: str = "w4a16"       # "w4a16" (group-wise asymmetric weights) | "w8a8", "w4a8", "w4a6" (symmetric)
    group: int = 128
    n_grid: int = 20
    imp_kind: str = "lognormal"
    seed: int = BASE_SEED

    @property
    def n_visual(self) -> int:
        return int(self.visual_frac * self.n_tokens)

    def linears(self) -> List[Linear]:
        h, i, kv = self.hidden, self.inter, self.kv
        return [Linear("q", h, h, "x_attn_in"), Linear("k", h, kv, "x_attn_in"),
                Linear("v", h, kv, "x_attn_in"), Linear("o", h, h, "x_o_in"),
                Linear("gate", h, i, "x_mlp_in"), Linear("up", h, i, "x_mlp_in"),
                Linear("down", i, h, "x_down_in")]

    def linear(self, name: str) -> Linear:
        for l in self.linears():
            if l.name == name:
                return l
        raise KeyError(name)

    def flops_per_candidate(self, lin: Linear) -> float:
        return 2.0 * self.n_tokens * lin.c_in * lin.c_out


def config(key: str, **over) -> LayerConfig:
    """The benchmark configurations: cfg0 (one 512x512 linear), cfg1/cfg2 (7B-class layer, W4A16 /
    W8A8), cfg3 (72B-class, Student-t), cfg4 (2B-class sweep cell; pass n_tokens/imp_kind/group/mode)."""
    base: Dict[str, LayerConfig] = {
        "cfg0": LayerConfig("cfg0", 512, 512, 512, 256, 0.75),
        "cfg1": LayerConfig("cfg1", 3584, 18944, 512, 8192, 0.85),
        "cfg2": LayerConfig("cfg2", 3584, 18944, 512, 8192, 0.85, mode="w8a8"),
        "cfg3": LayerConfig("cfg3", 8192, 29568, 1024, 16384, 0.90, dist="student3", n_outlier=8),
        "cfg4": LayerConfig("cfg4", 1536, 8960, 256, 4096, 0.85),
    }
    return dataclasses.replace(base[key], **over)


class LayerData:
    """Lazily generated, cached tensors of one configuration (bf16 as uint16 bits, fp32 weights)."""

    def __init__(self, cfg: LayerConfig):
        self.cfg = cfg
        self._x: Dict[str, np.ndarray] = {}
        self._w: Dict[str, np.ndarray] = {}
        self._imp: Optional[np.ndarray] = None

    def x(self, lin: Linear) -> np.ndarray:
        if lin.x_name not in self._x:
            c = self.cfg
            self._x[lin.x_name] = activations(c.seed, f"{c.key}/{lin.x_name}", c.n_tokens, lin.c_in,
                                              c.n_visual, c.dist, c.n_outlier)
        return self._x[lin.x_name]

    def w(self, lin: Linear) -> np.ndarray:
        if lin.name not in self._w:
            c = self.cfg
            self._w[lin.name] = weights(c.seed, f"{c.key}/w_{lin.name}", lin.c_out, lin.c_in)
        return self._w[lin.name]

    def imp(self) -> np.ndarray:
        if self._imp is None:
            c = self.cfg
            self._imp = importance(c.seed, f"{c.key}/w_imp/{c.imp_kind}", c.n_tokens, c.n_visual, c.imp_kind)
        return self._imp

    def drop(self, lin: Linear) -> None:
        self._w.pop(lin.name, None)


def small_case(seed: int, n_tokens: int, c_in: int, c_out: int, n_visual: Optional[int] = None,
               n_outlier: int = 2, imp_kind: str = "lognormal") -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """(X bits, W bits, importance) for an arbitrary small shape, same recipe as the configs."""
    nv = (3 * n_tokens) // 4 if n_visual is None else n_visual
    tag = f"small/{n_tokens}x{c_in}x{c_out}"
    return (activations(seed, tag + "/x", n_tokens, c_in, nv, "normal", min(n_outlier, c_in)),
            weights(seed, tag + "/w", c_out, c_in),
            importance(seed, tag + "/imp/" + imp_kind, n_tokens, nv, imp_kind))
