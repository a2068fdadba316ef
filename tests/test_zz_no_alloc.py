"""The allocation-free scale-candidate call against the workspace version.

Some callers of the library cannot give it a workspace because they are not allowed to allocate device
memory at the point of the call (allocator callbacks, fixed memory pools, plug-ins that only receive their
tensors).  tlq_scale_candidates_noalloc keeps its partial sums in an array built into the library; this
test checks, through the C ABI, that it returns what tlq_scale_candidates returns, on two calls in a row
that share that array (the second smaller than the first, so stale partials would show), and that sizes
beyond the array are refused.  Collected last so that a failure here cannot hide any other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2602_07899_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tlq():
    import __graft_entry__ as entry
    entry.build()
    from paper_2602_07899_b200 import tlq as mod
    return mod


def bits_of(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def free_device_bytes():
    """Free memory as the driver reports it: unlike torch's own counters it also sees allocations made behind
    torch's back (a cudaMalloc inside the library would show here)."""
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_noalloc_matches_workspace_version_twice_in_a_row(tlq):
    # (tokens, channels, statistic).  In the third and fifth case the 4 MiB array holds fewer row chunks than the
    # workspace version would use (32 against room for 27, 17 against 16), so the call runs with taller chunks; the
    # fifth also sits on the largest channel count accepted.  Each of them is followed by a smaller call that
    # re-uses the array.
    cases = [(9000, 3584, 0), (2000, 18944, 0), (8192, 18944, 0), (300, 264, 1), (4352, 32768, 1), (4100, 1544, 2)]
    for n, c1, stat in cases:
        xb = wl.activations(61, f"na/{n}x{c1}", n, c1, (3 * n) // 4, "normal", 4)
        X = tlq.bf16_from_bits(xb)
        mask = torch.from_numpy((np.random.default_rng(n).random(n) < 0.5).astype(np.uint8)).cuda() if stat == 2 else None
        cfg = tlq.config(stat_mode=stat, n_grid=20)
        ref_stat, ref_s = tlq.tlq_scale_candidates(X, cfg, mask)
        x_stat = torch.empty(c1, dtype=torch.float64, device="cuda")
        s = torch.empty((20, c1), dtype=torch.bfloat16, device="cuda")
        tlq.tlq_scale_candidates_noalloc(X, cfg, x_stat, s, mask)      # first call on this shape (and device): set-up done
        x_stat.zero_()
        s.zero_()
        free_before = free_device_bytes()
        torch.cuda.reset_peak_memory_stats()
        peak_before = torch.cuda.max_memory_allocated()
        tlq.tlq_scale_candidates_noalloc(X, cfg, x_stat, s, mask)
        # neither the driver's free-memory figure nor torch's allocation peak moves: nothing was allocated
        assert free_device_bytes() == free_before and torch.cuda.max_memory_allocated() == peak_before
        # same tolerances as the parity tests of the workspace version: scale bits exact, x_stat to 1e-14
        assert np.array_equal(bits_of(s), bits_of(ref_s))
        np.testing.assert_allclose(x_stat.cpu().numpy(), ref_stat.cpu().numpy(), rtol=1e-14, atol=0)
        del X, x_stat, s, ref_stat, ref_s


def test_noalloc_rejects_sizes_beyond_its_scratch(tlq):
    cfg = tlq.config()
    x = torch.zeros((2, 8), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(64, dtype=torch.float64, device="cuda")
    rc = tlq.lib.tlq_scale_candidates_noalloc(x.data_ptr(), 2, 32768 + 8, None, ctypes.byref(cfg), None, out.data_ptr(), None)
    assert rc == tlq.ERR_SHAPE
    assert "shape" in tlq.status_string(rc)
