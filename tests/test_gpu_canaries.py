"""TLQ_FLAG_DEBUG_CANARIES: guard words between the regions of a workspace.

A flagged call lays its workspace out with 256 guard bytes after every region, writes them when it starts and
compares them when it ends.  Here: (1) on ragged shapes, in every mode and variant of the search and for the apply
call, no kernel touches a guard and the results are those of the unflagged call, bit for bit; (2) the comparison does
notice a changed guard: the test itself flips one byte of a guard inside its own workspace tensor (an ordinary,
in-bounds write from the host's point of view) and asks the library to compare again.
"""
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


def variants(tlq):
    g, s = tlq.W4A16_ASYM_GROUP, tlq.W8A8_SYM
    return {
        "w4a16": dict(mode=g, group_size=64),
        "w4a16-narrow": dict(mode=g, group_size=64, flags=tlq.FLAG_GEMM_NARROW_TILES),
        "w4a16-pairs": dict(mode=g, group_size=64, flags=tlq.FLAG_GEMM_CTA_PAIRS),
        "w4a16-skip": dict(mode=g, group_size=64, flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS),
        "w4a16-two-stream": dict(mode=g, group_size=64),
        "w8a8": dict(mode=s),
        "w4a6": dict(mode=s, w_bits=4, a_bits=6),
        "w4a8-two-stream": dict(mode=s, w_bits=4, a_bits=8),
        "w8a8-skip": dict(mode=s, flags=tlq.FLAG_SKIP_ZERO_WEIGHT_TOKENS),
    }


@pytest.mark.parametrize("name", ["w4a16", "w4a16-narrow", "w4a16-pairs", "w4a16-skip", "w4a16-two-stream", "w8a8",
                                  "w4a6", "w4a8-two-stream", "w8a8-skip"])
@pytest.mark.parametrize("n,c1,c2", [(515, 1088, 777), (300, 192, 320), (129, 64, 8)])
def test_no_kernel_writes_outside_its_workspace_region(tlq, name, n, c1, c2):
    kw = dict(variants(tlq)[name])
    if kw["mode"] == tlq.W8A8_SYM and c1 % 16:
        pytest.skip("symmetric mode needs C1 % 16 == 0")
    xb, wb, imp = wl.small_case(411, n, c1, c2, n_outlier=2)
    imp = np.asarray(imp, np.float32)
    if "skip" in name:
        imp[np.random.default_rng(1).random(n) < 0.35] = 0.0
    x, w, wi = tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb), torch.from_numpy(imp).cuda()
    x_fp = tlq.bf16_from_bits(wl.small_case(412, n, c1, c2)[0]) if "two-stream" in name else None
    per_token = "skip" not in name
    flags = kw.pop("flags", 0)
    results = []
    for extra in (0, tlq.FLAG_DEBUG_CANARIES):
        cfg = tlq.config(n_grid=7, flags=flags | extra, **kw)
        out = tlq.tlq_scale_search_layer(x, w, wi, cfg, per_token=per_token, X_fp=x_fp)       # raises on a device status
        results.append((int(out.best_idx.item()), out.losses.cpu().numpy(), out.s_best.view(torch.int16).cpu().numpy(),
                        None if not per_token else out.per_token.cpu().numpy(), out.workspace.numel()))
    (b0, l0, s0, p0, bytes0), (b1, l1, s1, p1, bytes1) = results
    assert b0 == b1 and np.array_equal(l0, l1) and np.array_equal(s0, s1)
    assert p0 is None or np.array_equal(p0, p1)
    offs = tlq.tlq_debug_canary_offsets(0, n, c1, c2, cfg)
    assert len(offs) >= 8 and bytes1 > bytes0


@pytest.mark.parametrize("mode_name", ["w4a16", "w8a8"])
def test_apply_layer_with_guard_words(tlq, mode_name):
    n, c1, c2 = 300, 192, 320
    xb, wb, _ = wl.small_case(413, n, c1, c2)
    x, w = tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb)
    kw = dict(mode=tlq.W4A16_ASYM_GROUP, group_size=64) if mode_name == "w4a16" else dict(mode=tlq.W8A8_SYM)
    plain = tlq.tlq_apply_layer(x, w, None, None, tlq.config(**kw))
    guarded = tlq.tlq_apply_layer(x, w, None, None, tlq.config(flags=tlq.FLAG_DEBUG_CANARIES, **kw))
    assert torch.equal(plain["Yq"].view(torch.int16), guarded["Yq"].view(torch.int16))
    assert torch.equal(plain["codes"], guarded["codes"])


def test_a_changed_guard_word_is_reported(tlq):
    n, c1, c2 = 300, 192, 320
    xb, wb, imp = wl.small_case(414, n, c1, c2)
    cfg = tlq.config(group_size=64, n_grid=5, flags=tlq.FLAG_DEBUG_CANARIES)
    out = tlq.tlq_scale_search_layer(tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb), torch.from_numpy(imp).cuda(), cfg)
    ws = out.workspace
    offs = tlq.tlq_debug_canary_offsets(0, n, c1, c2, cfg)
    assert all(o % 16 == 0 for o in offs) and offs == sorted(offs) and offs[-1] + 256 <= ws.numel()
    tlq.tlq_debug_check_canaries(0, n, c1, c2, cfg, ws)
    assert tlq.tlq_read_status(ws) == 0                     # untouched since the call: still intact
    for j in (0, len(offs) // 2, len(offs) - 1):
        for byte in (0, 17, 255):
            saved = int(ws[offs[j] + byte].item())
            ws[offs[j] + byte] = saved ^ 0x40               # the test scribbles on its own buffer
            tlq.tlq_debug_check_canaries(0, n, c1, c2, cfg, ws)
            assert tlq.tlq_read_status(ws) == tlq.ERR_OVERRUN
            hdr = ws[:256].view(torch.int32).cpu().numpy()
            assert int(hdr[1]) == 100 + j
            ws[offs[j] + byte] = saved
            ws[:8] = 0                                      # clear status and position, as the next call would
            tlq.tlq_debug_check_canaries(0, n, c1, c2, cfg, ws)
            assert tlq.tlq_read_status(ws) == 0
    # and the workspace still serves a normal call afterwards
    again = tlq.tlq_scale_search_layer(tlq.bf16_from_bits(xb), tlq.bf16_from_bits(wb), torch.from_numpy(imp).cuda(), cfg, out)
    assert int(again.best_idx.item()) == int(out.best_idx.item())
