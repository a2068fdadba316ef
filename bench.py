#!/usr/bin/env python
"""Benchmark of the TLQ scale-search hot path on B200.

One "step" = the whole hot path over one decoder layer's seven linears (q, k, v, o, gate, up, down):
per linear, activation statistics -> K scale candidates -> fake-quant of all candidates -> fused
tensor-core GEMM with the importance-weighted error epilogue -> losses + argmin.  The metric is
scale-grid candidates per second (7 linears x K candidates per step) plus the fused GEMM's TFLOP/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg1] [--impl ours|reference]

N > 1 (torchrun): every rank calibrates its own layer (own seed), no data-path collective: weak scaling.
`--impl reference` times the CPU oracle on a bounded sample of the same workload (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "scale_grid_candidates_per_sec"
UNIT = "candidates/s"
SAMPLE_LINEAR = "k"            # reference arm: k-projection, first SAMPLE_TOKENS tokens per step (about a second)
SAMPLE_TOKENS = 2048
BASELINE_LINEAR = "q"          # the one-shot cpu_baseline leg of the GPU arm: q-projection, first BASELINE_TOKENS
BASELINE_TOKENS = 4096         # tokens (about 10-25 s of CPU work on 16 cores)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(bf16_sustained=float(p.get("bf16_tflops_sustained", 1400.0)), bf16_burst=float(p["bf16_tflops"]),
                    hbm=float(p["hbm_gbs"]), source="measured")
    return dict(bf16_sustained=1400.0, bf16_burst=1590.0, hbm=6650.0, source="fallback")


def layer_flops(cfgw):
    return sum(cfgw.flops_per_candidate(l) for l in cfgw.linears()) * cfgw.n_grid


# --------------------------------------------------------------------------------------------- CPU oracle legs


def oracle_sample_seconds(cfgw, data, tokens=SAMPLE_TOKENS, linear=SAMPLE_LINEAR):
    """One pass of the oracle over the bounded sample: one projection, the first `tokens` tokens,
    all K candidates.  Returns (seconds, flops of the sample)."""
    from oracle import tlq_oracle as orc
    lin = cfgw.linear(linear)
    n = min(tokens, cfgw.n_tokens)
    x, w, imp = data.x(lin)[:n], data.w(lin), data.imp()[:n]
    t0 = time.perf_counter()
    orc.scale_search(x, w, imp, cfgw.mode, cfgw.group, cfgw.n_grid)
    dt = time.perf_counter() - t0
    return dt, 2.0 * n * lin.c_in * lin.c_out * cfgw.n_grid


def sample_description(cfgw, tokens=SAMPLE_TOKENS, linear=SAMPLE_LINEAR):
    lin = cfgw.linear(linear)
    n = min(tokens, cfgw.n_tokens)
    return (f"{linear}-projection {lin.c_in}->{lin.c_out}, first {n} of {cfgw.n_tokens} tokens, all "
            f"{cfgw.n_grid} candidates; scaled to the whole layer by 2*N*C1*C2*K (extrapolated)")


def candidates_per_sec_from_sample(cfgw, seconds, flops):
    n_cand = len(cfgw.linears()) * cfgw.n_grid
    return n_cand * (flops / layer_flops(cfgw)) / seconds


def run_reference(args, cfgw):
    from paper_2602_07899_b200 import replicas, workloads as wl
    if not replicas.rank_info_from_env().is_root:
        return      # rank 0 alone runs and prints the reference arm
    data = wl.LayerData(cfgw)
    for _ in range(args.warmup):
        oracle_sample_seconds(cfgw, data)
    times = []
    for _ in range(args.steps):
        dt, flops = oracle_sample_seconds(cfgw, data)
        times.append(dt)
    total = sum(times)
    value = candidates_per_sec_from_sample(cfgw, total / len(times), flops)
    cores = os.cpu_count()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(cfgw), "sample": sample_description(cfgw)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample_description(cfgw)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_name(cfgw):
    return (f"{cfgw.key}: decoder layer hidden={cfgw.hidden} inter={cfgw.inter} kv={cfgw.kv}, {cfgw.n_tokens} tokens, "
            f"{cfgw.mode} group={cfgw.group}, K={cfgw.n_grid}, 7 linears per step")


# --------------------------------------------------------------------------------------------- clocks


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for nme, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw), "samples": len(sm),
                "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------------- GPU arm


def side_legs(tlq, torch, dev, cfgr, cfg, lins, dev_x, dev_w, bufs, peaks):
    """tlq_apply_layer with each linear's winning scale (quantized output for the next layer) and
    tlq_token_importance on the paper's gradient shape (128 samples x 1058 tokens x 3584 channels, bf16)."""
    def timed(fn, reps):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    def apply_all():
        for l in lins:
            tlq.tlq_apply_layer(dev_x[l.x_name], dev_w[l.name], bufs[l.name].s_best, None, cfg, want_codes=True,
                                check=False)
    ms_apply = timed(apply_all, 3)
    flops = sum(cfgr.flops_per_candidate(l) for l in lins) * (2.0 if cfgr.mode == "w4a16" else 1.0)
    torch.cuda.empty_cache()
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfgr.seed)
    B, N, C = 128, 1058, 3584
    G = torch.randn((B, N, C), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    imp = torch.empty(N, dtype=torch.float32, device=dev)
    mask = torch.empty(N, dtype=torch.uint8, device=dev)
    ms_imp = timed(lambda: tlq.tlq_token_importance(G, tlq.NORM_MEAN_ABS, 0.5, imp, mask), 5)
    gbs = G.numel() * 2 / (ms_imp * 1e-3) / 1e9
    del G
    torch.cuda.empty_cache()
    return {"apply_winner": {"ms_per_layer": round(ms_apply, 3), "tensor_tflops": round(flops / (ms_apply * 1e-3) / 1e12, 1),
                             "note": "fake-quant with the winning scale + one GEMM per linear (two K passes for W4A16: "
                                     "X W^T - X dW^T), bf16 Y_q stored; includes the binding's output allocations"},
            "token_importance": {"shape": [B, N, C], "ms": round(ms_imp, 4), "gbs": round(gbs, 1),
                                 "frac_of_hbm_peak": round(gbs / peaks["hbm"], 3), "peak_gbs": peaks["hbm"],
                                 "peak_source": peaks["source"]}}


def library_int8_probe(torch, dev, seconds=2.0):
    """Rate of the library's own int8 GEMM (torch._int_mm, 8192^3) on this GPU, outside every timed region:
    best single launch after idling (burst) and a back-to-back loop of `seconds` (sustained, power-capped).
    Context for the int8 roofline only; nothing on the measured path calls it."""
    n = 8192
    try:
        a = torch.randint(-128, 127, (n, n), dtype=torch.int8, device=dev)
        b = torch.randint(-128, 127, (n, n), dtype=torch.int8, device=dev).t().contiguous().t()
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        best = None
        for _ in range(10):
            e0.record(); torch._int_mm(a, b); e1.record()
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1)
            best = t if best is None or t < best else best
        iters = max(10, int(seconds * 1e3 / best))
        e0.record()
        for _ in range(iters):
            torch._int_mm(a, b)
        e1.record()
        torch.cuda.synchronize()
        ops = 2.0 * n ** 3
        return {"kind": "torch._int_mm 8192^3", "burst_tops": round(ops / best / 1e9, 1),
                "sustained_tops": round(ops * iters / e0.elapsed_time(e1) / 1e9, 1), "sustained_seconds": seconds}
    except Exception as exc:      # the probe is context, never a reason to lose the bench line
        return {"kind": "torch._int_mm 8192^3", "unavailable": str(exc)[:200]}
    finally:
        torch.cuda.empty_cache()


def search_config(tlq, cfgr, flags=0):
    if cfgr.mode == "w4a16":
        return tlq.config(mode=tlq.W4A16_ASYM_GROUP, group_size=cfgr.group, n_grid=cfgr.n_grid, flags=flags)
    # "w<n>a<m>": symmetric per-channel weights / per-token activations on the int8 tensor-core path
    wn, an = (int(v) for v in cfgr.mode[1:].split("a"))
    return tlq.config(mode=tlq.WA_SYM_CHANNEL, w_bits=wn, a_bits=an, n_grid=cfgr.n_grid, flags=flags)


def kernel_leg(tlq, torch, cfgr, cfg, lins, dev_x, dev_w, dev_imp, dev, local, steps, warmup, barrier):
    """The timed HBM-resident leg: `steps` passes over all linears, per-stage CUDA events on the launching
    stream, clocks sampled meanwhile.  Returns the raw measurements."""
    ws_bytes = max(tlq.tlq_scale_search_workspace_bytes(cfgr.n_tokens, l.c_in, l.c_out, cfg) for l in lins)
    workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    bufs = {l.name: tlq.SearchBuffers(cfgr.n_tokens, l.c_in, l.c_out, cfg, dev, False, workspace) for l in lins}
    torch.cuda.synchronize()

    def step():
        for l in lins:
            tlq.tlq_scale_search_layer(dev_x[l.x_name], dev_w[l.name], dev_imp, cfg, bufs[l.name], check=False)

    for _ in range(warmup):
        step()
    st = tlq.tlq_read_status(workspace)
    if st != tlq.OK:
        raise SystemExit(f"device status after warm-up: {tlq.status_string(st)}")
    sampler = ClockSampler(local)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    tlq.tlq_stage_timing_enable(True)
    launches0 = tlq.tlq_kernel_launch_count()
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    barrier()
    clocks = sampler.stop()
    launches = tlq.tlq_kernel_launch_count() - launches0
    stage_ms = tlq.tlq_stage_timing_drain(512)
    tlq.tlq_stage_timing_enable(False)
    st = tlq.tlq_read_status(workspace)
    if st != tlq.OK:
        raise SystemExit(f"device status after the timed region: {tlq.status_string(st)}")
    best = {l.name: int(bufs[l.name].best_idx.item()) for l in lins}
    return {"ms_total": ev0.elapsed_time(ev1), "stage_ms": stage_ms, "launches": launches, "clocks": clocks,
            "best": best, "bufs": bufs, "workspace": workspace}


def stage_report(tlq, cfgr, lins, leg, live_frac, peaks):
    """Per-linear figures and the fused GEMM's achieved rate from the per-stage events of a timed leg."""
    per_linear = {}
    gemm_ms_sum, gemm_flops_sum = 0.0, 0.0
    stage_tot = [0.0] * tlq.N_STAGES
    stage_ms, best = leg["stage_ms"], leg["best"]
    for i, rec in enumerate(stage_ms):
        l = lins[i % len(lins)]
        fl = cfgr.flops_per_candidate(l) * cfgr.n_grid * live_frac
        d = per_linear.setdefault(l.name, {"gemm_ms": [], "flops": fl, "stages_ms": [0.0] * tlq.N_STAGES})
        d["gemm_ms"].append(rec[2])
        for j in range(tlq.N_STAGES):
            d["stages_ms"][j] += rec[j]
            stage_tot[j] += rec[j]
        gemm_ms_sum += rec[2]
        gemm_flops_sum += fl
    n_rec = max(1, len(stage_ms) // len(lins))
    lin_report = {}
    stream_tot = {"stats": [0.0, 0.0], "fakequant": [0.0, 0.0]}     # algorithmic bytes, ms per step
    for name, d in per_linear.items():
        g = statistics.mean(d["gemm_ms"])
        l = next(x for x in lins if x.name == name)
        K = cfgr.n_grid
        # algorithmic bytes of the two streaming stages: X read once (+ the two K x C1 scale tables);
        # W read once and K operands written (bf16 delta weights, or int8 weights + int8 activations)
        stat_bytes = 2.0 * cfgr.n_tokens * l.c_in + 6.0 * K * l.c_in
        if cfgr.mode == "w4a16":
            fq_bytes = (2.0 + 2.0 * K) * l.c_out * l.c_in
        else:
            fq_bytes = (2.0 + K) * l.c_out * l.c_in + (2.0 + K) * cfgr.n_tokens * l.c_in
        stream_tot["stats"][0] += stat_bytes
        stream_tot["stats"][1] += d["stages_ms"][0] / n_rec
        stream_tot["fakequant"][0] += fq_bytes
        stream_tot["fakequant"][1] += d["stages_ms"][1] / n_rec
        lin_report[name] = {"gemm_ms": round(g, 4), "gemm_tflops": round(d["flops"] / (g * 1e-3) / 1e12, 1),
                            "stats_gbs": round(stat_bytes / (d["stages_ms"][0] / n_rec * 1e-3) / 1e9, 1),
                            "fakequant_gbs": round(fq_bytes / (d["stages_ms"][1] / n_rec * 1e-3) / 1e9, 1),
                            "stages_ms": [round(v / n_rec, 4) for v in d["stages_ms"]],
                            "candidates_per_s": round(cfgr.n_grid / (sum(d["stages_ms"]) / n_rec * 1e-3), 1),
                            "best_idx": best[name]}
    achieved = gemm_flops_sum / (gemm_ms_sum * 1e-3) / 1e12 if gemm_ms_sum > 0 else None
    share = {n: round(v / max(sum(stage_tot), 1e-9), 4) for n, v in zip(tlq.STAGE_NAMES, stage_tot)}
    streaming = {n: {"bound": "hbm", "achieved": round(b / (ms * 1e-3) / 1e9, 1) if ms > 0 else None,
                     "peak": peaks["hbm"], "unit": "GB/s",
                     "frac": round(b / (ms * 1e-3) / 1e9 / peaks["hbm"], 3) if ms > 0 else None,
                     "note": "algorithmic bytes of the stage over its in-step time (events between stages: "
                             "includes launch gaps)"}
                 for n, (b, ms) in stream_tot.items()}
    return lin_report, achieved, share, streaming, len(stage_ms)


def roofline_record(kernel, i8, achieved, peaks, clocks, traffic, launches_timed, share, lib_int8=None):
    """Roofline of the fused search GEMM.  The comparator follows the run's own clock record: a region whose
    median SM clock sat below 85 % of the maximum (the power cap of a long run) is compared with the sustained
    library rate, a short region at full clock with the burst rate.  int8 takes the measured bf16
    peak times the nominal int8 : bf16 ratio of 2."""
    ratio = 2.0 if i8 else 1.0
    sm, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    # the median clock decides (the power-cap reason alone also shows up for a moment when a 300 W run starts)
    capped = sm is None or not mx or sm < 0.85 * mx
    comparator = "sustained" if capped else "burst"
    peak = peaks["bf16_sustained" if capped else "bf16_burst"] * ratio
    nominal = 2250.0 * ratio
    rec = {"kernel": kernel, "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TOP/s" if i8 else "TFLOP/s",
           "frac": (achieved / peak) if achieved else None, "comparator": comparator,
           "traffic": traffic["bytes"] if traffic else None, "traffic_source": traffic["source"] if traffic else None,
           "peak_source": (f"{peaks['source']}: library bf16 GEMM, {comparator} ({peaks['bf16_sustained']} sustained, "
                           f"{peaks['bf16_burst']} burst){' x2 nominal int8:bf16 ratio' if i8 else ''}"),
           "frac_of_sustained": (achieved / (peaks["bf16_sustained"] * ratio)) if achieved else None,
           "frac_of_burst": (achieved / (peaks["bf16_burst"] * ratio)) if achieved else None,
           "frac_of_nominal": (achieved / nominal) if achieved else None, "nominal_peak": nominal,
           "launches_timed": launches_timed, "stage_share": share}
    if lib_int8 is not None:
        rec["library_int8"] = lib_int8
        ref = lib_int8.get("sustained_tops" if capped else "burst_tops")
        rec["frac_of_library_int8"] = (achieved / ref) if (achieved and ref) else None
    return rec


def stored_traffic(cfg_key):
    """DRAM bytes per launch of the fused GEMM from the committed ncu summary (not measured by this run)."""
    tpath = os.path.join(ROOT, "profiles", "search_gemm_traffic.json")
    if not os.path.exists(tpath):
        return None
    with open(tpath) as f:
        rec = json.load(f)
    if rec.get(cfg_key) is None:
        return None
    return {"bytes": rec[cfg_key], "source": "profiles/search_gemm_traffic.json: " + rec.get("note", "")}


def run_ours(args, cfgw):
    import dataclasses

    import torch
    import torch.distributed as dist
    from paper_2602_07899_b200 import calibrate, replicas, tlq, workloads as wl

    info = replicas.rank_info_from_env()
    world, rank, local = info.world, info.rank, info.local_rank
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    replicas.init_process_group(info, "nccl", dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank calibrates its own layer: same shapes, its own seed
    cfgr = dataclasses.replace(cfgw, seed=replicas.replica_seed(cfgw.seed, rank))
    data = wl.LayerData(cfgr)
    lins = [l for l in cfgr.linears() if args.linears is None or l.name in args.linears.split(",")]
    n_linears = len(lins)
    stacked = {}
    if args.shared_scale:
        # linears fed by the same activations share one scale (it is folded into the layer before them): their
        # weight matrices are stacked row-wise and searched as one; the step still covers all seven linears
        groups = {}
        for l in lins:
            groups.setdefault(l.x_name, []).append(l)
        lins = []
        for x_name, members in groups.items():
            name = "+".join(m.name for m in members)
            lins.append(wl.Linear(name, members[0].c_in, sum(m.c_out for m in members), x_name))
            stacked[name] = members

    def weights_of(l):
        if l.name in stacked:
            return np.concatenate([data.w(m) for m in stacked[l.name]], axis=0)
        return data.w(l)

    flags = tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS if args.skip_zero_weight else 0
    flags |= {"default": 0, "pairs": tlq.FLAG_GEMM_CTA_PAIRS, "narrow": tlq.FLAG_GEMM_NARROW_TILES}[args.gemm]
    if args.no_refine:
        flags |= tlq.FLAG_NO_REFINE
    cfg = search_config(tlq, cfgr, flags)

    # host (pinned) copies for the end-to-end leg, device-resident copies for the kernel leg
    host_x, host_w, dev_x, dev_w = {}, {}, {}, {}
    for l in lins:
        if l.x_name not in host_x:
            host_x[l.x_name] = torch.from_numpy(data.x(l).view(np.int16)).pin_memory()
            dev_x[l.x_name] = host_x[l.x_name].to(dev, non_blocking=True).view(torch.bfloat16)
        host_w[l.name] = torch.from_numpy(weights_of(l).view(np.int16)).pin_memory()
        dev_w[l.name] = host_w[l.name].to(dev, non_blocking=True).view(torch.bfloat16)
    imp_np = data.imp()
    if args.importance == "top50":      # the paper's token set: 1 for the top half by importance, 0 for the rest
        imp_np = (imp_np >= np.sort(imp_np)[len(imp_np) // 2]).astype(np.float32)
    host_imp = torch.from_numpy(imp_np).pin_memory()
    dev_imp = host_imp.to(dev, non_blocking=True)
    peaks = measured_peaks()
    live_frac = float((imp_np > 0).mean()) if args.skip_zero_weight else 1.0   # tokens the GEMM really processes

    # ---- kernel leg: inputs resident in HBM
    leg = kernel_leg(tlq, torch, cfgr, cfg, lins, dev_x, dev_w, dev_imp, dev, local, args.steps, args.warmup, barrier)
    ms_total, best = leg["ms_total"], leg["best"]
    if args.profile:
        print(json.dumps({"profile_run": True, "ms_per_step": ms_total / args.steps,
                          "stage_ms": leg["stage_ms"][-len(lins):]}))
        return

    # ---- the two path steps outside the search call, timed on their own (not part of `value`):
    #      applying the winner (Y_q for the next layer) and the token-importance reduction
    extra = side_legs(tlq, torch, dev, cfgr, cfg, lins, dev_x, dev_w, leg["bufs"], peaks)
    plain = (args.linears is None and args.mode is None and not args.skip_zero_weight and args.gemm == "default"
             and not args.shared_scale and args.importance == "config" and not args.no_refine)
    del leg["bufs"], leg["workspace"]
    torch.cuda.empty_cache()

    # ---- the same layer in the W8A8 setting (the metric is quoted for bf16 and for int8): a second kernel leg on the
    #      resident tensors, reported as a sub-record; the headline stays on the configured workload
    int8_leg = None
    if plain and cfgr.key == "cfg1" and not args.no_int8:
        cfg8w = dataclasses.replace(cfgr, key="cfg2", mode="w8a8")
        cfg8 = search_config(tlq, cfg8w)
        int8_leg = kernel_leg(tlq, torch, cfg8w, cfg8, lins, dev_x, dev_w, dev_imp, dev, local, args.steps, args.warmup,
                              barrier)
        del int8_leg["bufs"], int8_leg["workspace"]
        torch.cuda.empty_cache()

    # ---- end-to-end leg: host buffers in, results out, every step, through the public host-side entry:
    #      inputs in pinned host memory, copies overlapped with the previous linear's kernels
    del dev_x, dev_w
    torch.cuda.empty_cache()
    pipe = calibrate.HostLayerSearch([(l.name, l.x_name, cfgr.n_tokens, l.c_in, l.c_out) for l in lins], cfg, dev)
    out_host = {l.name: (torch.empty(1, dtype=torch.int32).pin_memory(),
                         torch.empty(cfgr.n_grid, dtype=torch.float64).pin_memory()) for l in lins}
    h2d = sum(v.numel() * 2 for v in host_x.values()) + sum(v.numel() * 2 for v in host_w.values()) + host_imp.numel() * 4
    d2h = len(lins) * (4 + 8 * cfgr.n_grid)

    def e2e_step():
        pipe.run(host_x, host_w, host_imp, out_host)

    for _ in range(2):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        e2e_step()
    e1.record()
    barrier()
    ms_e2e = e0.elapsed_time(e1)
    pipe.check()
    assert all(int(out_host[l.name][0].item()) == best[l.name] for l in lins)
    del pipe
    torch.cuda.empty_cache()

    # ---- max over ranks
    ms_int8 = int8_leg["ms_total"] if int8_leg else 0.0
    ms_total, ms_e2e, ms_int8 = replicas.max_over_ranks([ms_total, ms_e2e, ms_int8], info, dev)

    n_cand_step = n_linears * cfgr.n_grid
    value = replicas.whole_job_rate(n_cand_step, args.steps, info, ms_total)
    e2e_value = replicas.whole_job_rate(n_cand_step, args.steps, info, ms_e2e)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the fused search GEMM), from the per-stage events of the timed region
    i8 = cfgr.mode != "w4a16"
    lib_int8 = library_int8_probe(torch, dev) if (world == 1 and (i8 or int8_leg)) else None
    lin_report, achieved, share, streaming, n_timed = stage_report(tlq, cfgr, lins, leg, live_frac, peaks)
    kernel = "gemm_w8a8_kernel<search>" if i8 else {"default": "gemm_bf16_wide_kernel", "pairs": "gemm_bf16_pair_kernel",
                                                     "narrow": "gemm_bf16_kernel<search>"}[args.gemm]
    roofline = roofline_record(kernel, i8, achieved, peaks, leg["clocks"], stored_traffic(cfgr.key) if plain else None,
                               n_timed, share, lib_int8 if i8 else None)
    int8_record = None
    if int8_leg:
        rep8, ach8, share8, stream8, n8 = stage_report(tlq, cfg8w, lins, int8_leg, 1.0, peaks)
        int8_record = {"workload": workload_name(cfg8w) + " [the tensors of the headline workload, W8A8 setting]",
                       "value": replicas.whole_job_rate(n_cand_step, args.steps, info, ms_int8), "unit": UNIT,
                       "ms_per_step": ms_int8 / args.steps, "dtype": "int8", "gemm_tops": ach8,
                       "roofline": roofline_record("gemm_w8a8_kernel<search>", True, ach8, peaks, int8_leg["clocks"],
                                                   stored_traffic("cfg2"), n8, share8, lib_int8),
                       "gpu_launches": int8_leg["launches"], "clocks": int8_leg["clocks"], "per_linear": rep8,
                       "streaming_stages": stream8}

    cpu = None
    if world == 1:
        dt, fl = oracle_sample_seconds(cfgw, data, BASELINE_TOKENS, BASELINE_LINEAR)
        cpu = {"value": candidates_per_sec_from_sample(cfgw, dt, fl), "unit": UNIT, "cores": os.cpu_count(),
               "kind": "oracle", "sample": sample_description(cfgw, BASELINE_TOKENS, BASELINE_LINEAR), "sample_seconds": round(dt, 3),
               "oracle_gflops": round(fl / dt / 1e9, 1)}

    part = tlq.tlq_l2_partition_info()       # whether the bf16 GEMM ran its L2-partition-aware tile order on this device
    l2_partitions = {"measured": part["valid"], "sms_per_partition": list(part["count"])}

    notes = (("" if args.linears is None else f" [subset: {args.linears}]")
             + ("" if args.importance == "config" else f" [importance: {args.importance}]")
             + (" [zero-weight tokens skipped]" if args.skip_zero_weight else "")
             + (" [refine pass off]" if args.no_refine else "")
             + (" [shared scale: " + ", ".join(l.name for l in lins) + "]" if args.shared_scale else ""))
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if cfgr.mode == "w4a16" else "int8", "data": "synthetic",
            "config": {"workload": workload_name(cfgr) + notes, "l2": "inputs_exceed_l2 (operands of one linear: 0.1-2.9 GB)",
                       "parallelism": f"replicas x{world} (one layer per rank, no collective)"},
            "gemm_tflops": achieved, "roofline": roofline, "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": leg["launches"], "clocks": leg["clocks"], "per_linear": lin_report, "other_path_steps": extra,
            "streaming_stages": streaming, "l2_partitions": l2_partitions, "int8": int8_record}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg1")
    ap.add_argument("--mode", default=None, help="override the config's setting: w4a16, w8a8, w4a8, w4a6")
    ap.add_argument("--importance", default="config", choices=["config", "top50"],
                    help="token weights: the config's (log-normal) or a 0/1 top-50%% mask (the paper's token set)")
    ap.add_argument("--skip-zero-weight", action="store_true",
                    help="set TLQ_FLAG_SKIP_ZERO_WEIGHT_TOKENS (tensor FLOP/s then count the live tokens only)")
    ap.add_argument("--gemm", default="default", choices=["default", "pairs", "narrow"],
                    help="variant of the bf16 search GEMM (TLQ_FLAG_GEMM_*), for A/B measurements")
    ap.add_argument("--shared-scale", action="store_true",
                    help="stack linears that share their input (q/k/v, gate/up) and search one scale for each stack")
    ap.add_argument("--linears", default=None, help="comma-separated subset of q,k,v,o,gate,up,down (profiling)")
    ap.add_argument("--profile", action="store_true", help="kernel leg only: skip the end-to-end and CPU legs")
    ap.add_argument("--no-refine", action="store_true",
                    help="set TLQ_FLAG_NO_REFINE (the second evaluation of near-tied candidates), for A/B measurements")
    ap.add_argument("--no-int8", action="store_true", help="skip the W8A8 sub-record of the default (cfg1) run")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2602_07899_b200 import workloads as wl
    cfgw = wl.config(args.config) if args.mode is None else wl.config(args.config, mode=args.mode)
    if args.impl == "reference":
        run_reference(args, cfgw)
    else:
        run_ours(args, cfgw)


if __name__ == "__main__":
    main()
