"""The multi-process path (one replica per rank) on CPU ranks over gloo, world size 2.

The search has no data-path collective, so what more than one rank adds is host logic only: which
data a rank calibrates, the MAX reduction of the measured times, the whole-job rate, and that the
reference arm runs on rank 0 alone.  All of it runs here without a GPU.
"""
import json
import os
import socket
import subprocess
import sys
import zlib

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str) -> None:
    sys.path.insert(0, ROOT)
    from paper_2602_07899_b200 import replicas, workloads as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    info = replicas.rank_info_from_env()
    assert (info.rank, info.world, info.local_rank) == (rank, world, rank)
    assert replicas.init_process_group(info, "gloo")
    try:
        # every rank draws its own layer: same shapes, different bits
        seed = replicas.replica_seed(wl.BASE_SEED, info.rank)
        x, w, imp = wl.small_case(seed, 64, 32, 16)
        digest = zlib.crc32(x.tobytes() + w.tobytes() + imp.tobytes())
        digests = [None] * world
        dist.all_gather_object(digests, (seed, x.shape, w.shape, digest))
        assert len({d[0] for d in digests}) == world and len({d[3] for d in digests}) == world
        assert len({(d[1], d[2]) for d in digests}) == 1

        # the slowest rank defines the step time, for both timed legs at once
        mine = [10.0 + 5.0 * rank, 30.0 - 7.0 * rank]
        got = replicas.max_over_ranks(mine, info)
        assert got == [10.0 + 5.0 * (world - 1), 30.0]
        # whole-job aggregate: all ranks' units over the max time
        assert replicas.whole_job_rate(140, 5, info, 1000.0) == world * 140 * 5

        # layers of a model are dealt out without overlap or gaps
        mine_layers = replicas.assign_layers(7, info)
        all_layers = [None] * world
        dist.all_gather_object(all_layers, mine_layers)
        assert sorted(sum(all_layers, [])) == list(range(7))
        dist.barrier()
        with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
            f.write("ok")
    finally:
        dist.destroy_process_group()


def _shard_worker(rank: int, world: int, port: int, out_dir: str) -> None:
    """One linear cut by output rows over the ranks: slice losses from the oracle, combined over gloo."""
    sys.path.insert(0, ROOT)
    from oracle import tlq_oracle as orc
    from paper_2602_07899_b200 import replicas, workloads as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    info = replicas.rank_info_from_env()
    replicas.init_process_group(info, "gloo")
    try:
        x, w, imp = wl.small_case(131, 48, 64, 37)           # 37 rows: uneven slices
        r0, r1 = replicas.shard_rows(37, info)
        spans = [None] * world
        dist.all_gather_object(spans, (r0, r1))
        assert spans[0][0] == 0 and spans[-1][1] == 37 and all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
        for mode, group in (("w4a16", 32), ("w4a8", 0)):
            mine = orc.scale_search(x, w[r0:r1], imp, mode=mode, group=group, n_grid=5)
            total, best = replicas.combine_sharded_losses(torch.from_numpy(mine["losses"]), r1 - r0, 37, info)
            full = orc.scale_search(x, w, imp, mode=mode, group=group, n_grid=5)
            assert np.allclose(total.numpy(), full["losses"], rtol=1e-12)
            assert best == full["best"]
        with open(os.path.join(out_dir, f"shard{rank}"), "w") as f:
            f.write("ok")
    finally:
        dist.destroy_process_group()


def test_row_sharded_search_combines_exactly(tmp_path):
    mp.spawn(_shard_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    assert sorted(os.listdir(tmp_path)) == ["shard0", "shard1"]


def test_two_gloo_ranks_host_logic(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert sorted(os.listdir(tmp_path)) == ["ok0", "ok1"]


def test_single_process_is_the_degenerate_group():
    sys.path.insert(0, ROOT)
    from paper_2602_07899_b200 import replicas
    info = replicas.rank_info_from_env({})
    assert info.world == 1 and info.is_root
    assert not replicas.init_process_group(info, "gloo")
    assert replicas.max_over_ranks([1.5, 2.5], info) == [1.5, 2.5]
    assert replicas.assign_layers(3, info) == [0, 1, 2]


def test_reference_arm_prints_once_under_two_ranks():
    """`bench.py --impl reference` launched as two ranks: rank 0 runs the oracle sample and prints the one
    JSON line, rank 1 exits 0 without work."""
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference",
           "--gpus", "2", "--steps", "1", "--warmup", "0", "--config", "cfg0"]
    r = subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=ROOT, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["gpu_launches"] == 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["value"] > 0
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and np.isfinite(rec["ms_per_step"])
