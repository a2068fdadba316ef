"""CPU-side checks: the C ABI library builds, loads and exports every declared symbol; host-side
argument validation answers with error codes (no compute call reaches a GPU here)."""
import ctypes
import os
import re

import pytest
import torch

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tlq():
    entry.build()
    from paper_2602_07899_b200 import tlq as mod
    return mod


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tlq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tlq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(tlq):
    names = declared_symbols()
    assert len(names) >= 12 and "tlq_scale_search_layer" in names
    for n in names:
        assert hasattr(tlq.lib, n), n
    assert sorted(tlq.EXPORTS) == names
    assert tlq.lib.tlq_version() == 1009
    assert tlq.status_string(0) == "ok" and "workspace" in tlq.status_string(tlq.ERR_WORKSPACE)


def test_config_struct_layout(tlq):
    c = tlq.config()
    assert ctypes.sizeof(tlq.Config) == 32 and c.struct_size == 32
    assert (c.mode, c.w_bits, c.a_bits, c.group_size, c.n_grid) == (0, 4, 16, 128, 20)
    c8 = tlq.config(tlq.W8A8_SYM)
    assert (c8.w_bits, c8.a_bits) == (8, 8)


def test_workspace_queries_and_shape_validation(tlq):
    c = tlq.config()
    n = tlq.tlq_scale_search_workspace_bytes(8192, 3584, 18944, c)
    dW = 20 * 18944 * 3584 * 2
    assert dW < n < dW + 400 * 2 ** 20
    assert tlq.tlq_scale_search_workspace_bytes(256, 512, 512, c) % 256 == 0
    assert tlq.tlq_scale_search_workspace_bytes(256, 500, 512, c) == 0          # C1 % 8
    assert tlq.tlq_scale_search_workspace_bytes(256, 576, 512, c) == 0          # C1 % group
    assert tlq.tlq_scale_search_workspace_bytes(0, 512, 512, c) == 0
    bad = tlq.config(n_grid=65)
    assert tlq.tlq_scale_search_workspace_bytes(256, 512, 512, bad) == 0
    # fp64 column partials: one row of C1 doubles per chunk of 256 tokens
    assert tlq.lib.tlq_scale_candidates_workspace_bytes(8192, 3584) == 32 * 3584 * 8
    assert tlq.lib.tlq_scale_candidates_workspace_bytes(1, 8) == 256


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device error path")
def test_compute_calls_fail_loudly_without_a_device(tlq):
    c = tlq.config()
    buf = (ctypes.c_uint8 * 4096)()
    addr = (ctypes.addressof(buf) + 255) // 256 * 256
    rc = tlq.lib.tlq_quantize_weights(addr, None, 8, 128, ctypes.byref(c), addr, addr, addr, None, None)
    assert rc == tlq.ERR_CUDA
    rc = tlq.lib.tlq_token_importance(addr, 0, 1, 4, 8, 0, 0.0, addr, None, None)
    assert rc == tlq.ERR_CUDA


def test_host_validation_error_codes(tlq):
    c = tlq.config()
    buf = (ctypes.c_uint8 * 8192)()
    a = (ctypes.addressof(buf) + 255) // 256 * 256
    L = tlq.lib
    assert L.tlq_quantize_weights(None, None, 8, 128, ctypes.byref(c), a, a, a, None, None) == tlq.ERR_INVALID_ARG
    assert L.tlq_quantize_weights(a + 2, None, 8, 128, ctypes.byref(c), a, a, a, None, None) == tlq.ERR_ALIGN
    assert L.tlq_quantize_weights(a, None, 8, 100, ctypes.byref(c), a, a, a, None, None) == tlq.ERR_SHAPE
    c3 = tlq.config(group_size=48)
    assert L.tlq_quantize_weights(a, None, 8, 96, ctypes.byref(c3), a, a, a, None, None) == tlq.ERR_UNSUPPORTED
    c.struct_size = 8
    assert L.tlq_quantize_weights(a, None, 8, 128, ctypes.byref(c), a, a, a, None, None) == tlq.ERR_INVALID_ARG
    c = tlq.config()
    assert L.tlq_scale_search_layer(a, 4, 128, a, 8, None, None, ctypes.byref(c), a, 16, a, a, a, None,
                                    None) == tlq.ERR_WORKSPACE
    assert L.tlq_scale_search_layer(a, 4, 128, a, 8, None, None, ctypes.byref(c), None, 1 << 30, a, a, a, None,
                                    None) == tlq.ERR_INVALID_ARG
    cm = tlq.config(stat_mode=tlq.STAT_MASKED_MAX)
    assert L.tlq_scale_search_layer(a, 4, 128, a, 8, None, None, ctypes.byref(cm), a, 1 << 30, a, a, a, None,
                                    None) == tlq.ERR_INVALID_ARG
    # flags: unknown bits, token skipping without weights or with a per-token table, options the two-stream call rejects
    assert L.tlq_scale_search_layer(a, 4, 128, a, 8, None, None, ctypes.byref(tlq.config(flags=32)), a, 1 << 30, a, a, a,
                                    None, None) == tlq.ERR_INVALID_ARG
    skip = tlq.config(flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS)
    assert L.tlq_scale_search_layer(a, 4, 128, a, 8, None, None, ctypes.byref(skip), a, 1 << 30, a, a, a, None,
                                    None) == tlq.ERR_INVALID_ARG
    assert L.tlq_scale_search_layer(a, 4, 128, a, 8, a, None, ctypes.byref(skip), a, 1 << 30, a, a, a, a,
                                    None) == tlq.ERR_INVALID_ARG
    assert L.tlq_scale_search_layer_two_stream(a, None, 4, 128, a, 8, None, None, ctypes.byref(c), a, 1 << 30, a, a, a,
                                               None, None) == tlq.ERR_INVALID_ARG
    assert L.tlq_scale_search_layer_two_stream(a, a, 4, 128, a, 8, a, None, ctypes.byref(skip), a, 1 << 30, a, a, a,
                                               None, None) == tlq.ERR_INVALID_ARG
    assert L.tlq_scale_search_layer_two_stream(a, a + 4, 4, 128, a, 8, None, None, ctypes.byref(c), a, 1 << 30, a, a, a,
                                               None, None) == tlq.ERR_ALIGN
    # the symmetric mode takes 2..8 bits on either side, nothing else
    assert tlq.tlq_scale_search_workspace_bytes(64, 128, 64, tlq.config(tlq.WA_SYM_CHANNEL, w_bits=4, a_bits=6)) > 0
    assert tlq.tlq_scale_search_workspace_bytes(64, 128, 64, tlq.config(tlq.WA_SYM_CHANNEL, w_bits=4, a_bits=16)) == 0
    assert tlq.tlq_scale_search_workspace_bytes(64, 128, 64, tlq.config(tlq.WA_SYM_CHANNEL, w_bits=1, a_bits=8)) == 0
    assert L.tlq_token_importance(a, 7, 1, 4, 8, 0, 0.0, a, None, None) == tlq.ERR_INVALID_ARG
    assert L.tlq_token_importance(a, 0, 1, 4, 12, 0, 0.0, a, None, None) == tlq.ERR_SHAPE
    assert L.tlq_token_importance(a, 0, 1, 4, 8, 0, 1.5, a, None, None) == tlq.ERR_INVALID_ARG
    assert L.tlq_read_status(None, None) == tlq.ERR_INVALID_ARG
    arr = (ctypes.c_float * 4)()
    assert L.tlq_stage_timing_drain(arr, 1) == tlq.ERR_INVALID_ARG  # timing never enabled


def test_oracle_never_imports_the_cuda_path():
    for fn in ("tlq_oracle.py", "brute.py"):
        src = open(os.path.join(ROOT, "oracle", fn)).read()
        assert "paper_2602_07899_b200" not in src and "ctypes" not in src and "torch" not in src
    for fn in os.listdir(os.path.join(ROOT, "paper_2602_07899_b200")):
        if fn.endswith(".py"):
            text = open(os.path.join(ROOT, "paper_2602_07899_b200", fn)).read()
            assert not re.search(r"^\s*(from|import)\s+oracle", text, flags=re.M), fn


def test_tile_walk_visits_every_tile_exactly_once(tlq):
    """The order in which the persistent CTAs of the fused GEMM take their tiles, replayed on the host: whole grid
    (plain and blocked) and split over two L2 partitions of unequal size, whose token cut moves from candidate to
    candidate.  Every (candidate, output tile, token tile) must be visited exactly once."""
    import numpy as np
    for mtiles, otiles, K in ((32, 74, 20), (32, 2, 20), (9, 7, 20), (4, 1, 1), (5, 3, 64), (64, 116, 3)):
        for n0, n1 in ((72, 76), (70, 78), (74, 74), (40, 108)):
            v = tlq.tlq_debug_tile_walk(mtiles, otiles, K, n0, n1)
            assert v.min() == 1 and v.max() == 1, (mtiles, otiles, K, n0, n1)
        for grid in (148, 7, 1):
            assert np.all(tlq.tlq_debug_tile_walk(mtiles, otiles, K, grid) == 1)
            assert np.all(tlq.tlq_debug_tile_walk(mtiles, otiles, K, grid, blocked=True, block_a=8) == 1)
            assert np.all(tlq.tlq_debug_tile_walk(mtiles, otiles, K, grid, blocked=True, block_a=16) == 1)
    # the partitions' shares follow their SM counts: both need about the same number of rounds
    mt, ot, K, n0, n1 = 32, 74, 20, 72, 76
    c0 = (K * mt * n0) // (n0 + n1)                  # token tiles of partition 0 summed over the candidates
    rounds0 = -(-c0 * ot // n0)
    rounds1 = -(-(K * mt - c0) * ot // n1)
    assert abs(rounds0 - rounds1) <= 1
    # refusals: a split needs an unblocked walk, four token tiles and partitions of comparable size
    v = np.zeros(4 * 4, dtype=np.int32)
    args = v.ctypes.data_as(__import__("ctypes").c_void_p)
    assert tlq.lib.tlq_debug_tile_walk(4, 4, 1, 72, 76, 1, 8, args) == tlq.ERR_UNSUPPORTED
    assert tlq.lib.tlq_debug_tile_walk(3, 4, 1, 72, 76, 0, 8, args) == tlq.ERR_UNSUPPORTED
    assert tlq.lib.tlq_debug_tile_walk(4, 4, 1, 10, 138, 0, 8, args) == tlq.ERR_UNSUPPORTED
    assert tlq.lib.tlq_debug_tile_walk(4, 4, 0, 72, 76, 0, 8, args) == tlq.ERR_SHAPE
    assert tlq.lib.tlq_debug_tile_walk(4, 4, 1, 72, 76, 0, 8, None) == tlq.ERR_INVALID_ARG


def test_resident_kernel_work_items_cover_every_candidate_of_every_tile_once(tlq):
    """The tile-resident kernels: whole waves of tiles keep all K candidates, the tiles of the last partial wave are
    split by candidates over the CTAs that would idle; with more CTAs than tiles everything is a tail."""
    import numpy as np
    for mtiles, otiles, K in ((64, 14, 20), (64, 2, 20), (64, 74, 20), (1, 1, 1), (3, 5, 7), (128, 6, 64), (33, 1, 2)):
        for grid in (148, 132, 7, 1):
            for blocked in (False, True):
                v = tlq.tlq_debug_resident_walk(mtiles, otiles, K, min(grid, mtiles * otiles), blocked)
                assert v.min() == 1 and v.max() == 1, (mtiles, otiles, K, grid, blocked)


def test_guard_word_layout_is_consistent(tlq):
    """Host only: the guards of a flagged layout are ascending, 16-byte aligned, 256 bytes apart at least, inside
    the workspace size the flagged configuration reports; an unflagged configuration has none to report."""
    for mode, kw in ((tlq.W4A16_ASYM_GROUP, dict(group_size=128)), (tlq.W8A8_SYM, {})):
        for flags in (0, tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS):
            plain = tlq.config(mode, flags=flags, **kw)
            guarded = tlq.config(mode, flags=flags | tlq.FLAG_DEBUG_CANARIES, **kw)
            for kind, size_of in ((0, tlq.lib.tlq_scale_search_workspace_bytes), (1, tlq.lib.tlq_apply_layer_workspace_bytes)):
                n, c1, c2 = 1000, 512, 264
                offs = tlq.tlq_debug_canary_offsets(kind, n, c1, c2, guarded)
                total = int(size_of(n, c1, c2, ctypes.byref(guarded)))
                assert len(offs) >= (8 if kind == 0 else 2)
                assert all(o % 16 == 0 for o in offs)
                assert all(b - a >= 256 for a, b in zip(offs, offs[1:]))
                assert offs[0] >= 256 and offs[-1] + 256 <= total
                assert total > int(size_of(n, c1, c2, ctypes.byref(plain)))      # some guards fit into alignment gaps
                assert tlq.lib.tlq_debug_canary_offsets(kind, n, c1, c2, ctypes.byref(plain), None, 0) == tlq.ERR_INVALID_ARG
    assert tlq.lib.tlq_debug_canary_offsets(2, 8, 128, 8, ctypes.byref(tlq.config(flags=tlq.FLAG_DEBUG_CANARIES)), None,
                                            0) == tlq.ERR_INVALID_ARG
