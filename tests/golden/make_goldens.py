"""Writes the full-size expected values under tests/golden/fullsize/ from the CPU oracle alone.

Run from the repository root (CPU only; nothing of the CUDA path is imported or needed):

    python tests/golden/make_goldens.py              # every cell listed in CELLS that has no file yet
    python tests/golden/make_goldens.py cfg1 cfg2    # only cells whose name starts with one of these
    python tests/golden/make_goldens.py --force ...  # overwrite existing files

For every (configuration cell, linear) it runs oracle.tlq_oracle.scale_search on the seeded synthetic
tensors of paper_2602_07899_b200.workloads (input generators only, none of the method's arithmetic)
and stores what a GPU test needs to compare the search of Sec. 3.2.1 at the benchmark's full size
without re-running hours of float64 on the test machine:

    losses      float64 [K]      the importance-weighted objective of every grid point
    best        int              lowest index of the minimum (the argmin of Sec. 3.2.1)
    gap         float            relative distance of the two smallest losses (how unique the argmin is)
    tokens      int64 [T]        a seeded sample of token rows (half visual, half text, plus the tokens
                                 that carry a one-hot importance)
    per_token   float64 [K, T]   squared output error of those tokens for every grid point
    scale_best  uint16 [C1]      bfloat16 bits of the winning scale
    seconds     float            oracle wall time for this linear, cores = threads numpy used

One .npz per linear (about 45 KB), so an interrupted run resumes where it stopped.
"""
from __future__ import annotations

import argparse
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import tlq_oracle as orc                      # noqa: E402
from paper_2602_07899_b200 import workloads as wl         # noqa: E402

OUT_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "fullsize")
N_SAMPLED_TOKENS = 256
ALL = ("q", "k", "v", "o", "gate", "up", "down")

# name -> (config key, overrides, linears).  Cell names are the file prefixes the GPU tests look for.
CELLS = {
    "cfg1": ("cfg1", {}, ALL),
    "cfg2": ("cfg2", {}, ALL),
    "cfg4_n16384_w4a16_g64_lognormal": ("cfg4", dict(n_tokens=16384, mode="w4a16", group=64, imp_kind="lognormal"), ALL),
    "cfg4_n16384_w4a16_g128_uniform": ("cfg4", dict(n_tokens=16384, mode="w4a16", group=128, imp_kind="uniform"), ALL),
    "cfg4_n16384_w8a8_onehot": ("cfg4", dict(n_tokens=16384, mode="w8a8", imp_kind="onehot"), ALL),
    "cfg4_n65536_w8a8_lognormal": ("cfg4", dict(n_tokens=65536, mode="w8a8", imp_kind="lognormal"), ("k", "down")),
    "cfg4_n65536_w4a16_g64_lognormal": ("cfg4", dict(n_tokens=65536, mode="w4a16", group=64, imp_kind="lognormal"), ("v", "down")),
    "cfg3": ("cfg3", {}, ("k", "v", "q", "o", "down", "gate", "up")),
}


def sample_tokens(cfgw: wl.LayerConfig, imp: np.ndarray, cell: str) -> np.ndarray:
    """Seeded token sample: half from the visual block, half from the text block, plus every token that
    holds all of a one-hot importance vector."""
    rng = np.random.default_rng([cfgw.seed, len(cell), cfgw.n_tokens])
    half = N_SAMPLED_TOKENS // 2
    nv, nt = cfgw.n_visual, cfgw.n_tokens - cfgw.n_visual
    vis = rng.choice(nv, min(half, nv), replace=False)
    txt = nv + rng.choice(nt, min(half, nt), replace=False)
    tok = np.concatenate([vis, txt])
    if cfgw.imp_kind == "onehot":
        tok = np.concatenate([tok, np.flatnonzero(imp)])
    return np.unique(tok).astype(np.int64)


def golden_path(cell: str, lin_name: str) -> str:
    return os.path.join(OUT_DIR, f"{cell}_{lin_name}.npz")


def make_one(cell: str, cfgw: wl.LayerConfig, data: wl.LayerData, lin_name: str) -> None:
    lin = cfgw.linear(lin_name)
    xb, wb, imp = data.x(lin), data.w(lin), data.imp()
    t0 = time.time()
    ref = orc.scale_search(xb, wb, imp, cfgw.mode, cfgw.group, cfgw.n_grid)
    dt = time.time() - t0
    order = np.sort(ref["losses"])
    gap = float((order[1] - order[0]) / order[0]) if len(order) > 1 else float("inf")
    tokens = sample_tokens(cfgw, imp, cell)
    np.savez(golden_path(cell, lin_name),
             losses=ref["losses"], best=np.int64(ref["best"]), gap=np.float64(gap), tokens=tokens,
             per_token=np.ascontiguousarray(ref["per_token"][:, tokens]),
             scale_best=orc.f32_to_bf16_bits(ref["scales"][ref["best"]]),
             seconds=np.float64(dt), cores=np.int64(os.cpu_count() or 1),
             shape=np.array([cfgw.n_tokens, lin.c_in, lin.c_out, cfgw.n_grid], dtype=np.int64),
             mode=np.array(cfgw.mode), group=np.int64(cfgw.group), imp_kind=np.array(cfgw.imp_kind))
    print(f"{cell}/{lin_name}: best={ref['best']} gap={gap:.3e} {dt:.1f}s", flush=True)
    data.drop(lin)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("prefixes", nargs="*", help="cell-name prefixes (default: all)")
    ap.add_argument("--force", action="store_true")
    args = ap.parse_args()
    os.makedirs(OUT_DIR, exist_ok=True)
    for cell, (key, over, linears) in CELLS.items():
        if args.prefixes and not any(cell.startswith(p) for p in args.prefixes):
            continue
        cfgw = wl.config(key, **over)
        data = wl.LayerData(cfgw)
        for lin_name in linears:
            if os.path.exists(golden_path(cell, lin_name)) and not args.force:
                continue
            make_one(cell, cfgw, data, lin_name)


if __name__ == "__main__":
    main()
