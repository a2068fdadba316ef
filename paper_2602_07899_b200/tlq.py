"""ctypes binding of libtlq.so: same names as the C ABI (include/tlq.h), argument marshalling only.

Tensors are torch CUDA tensors used purely as device-memory handles (bf16 tensors may be passed as
torch.bfloat16 or as int16/uint16 bit patterns); the stream is torch's current stream unless given.
Every step of the path runs in the library's kernels.  Importing this module loads the library and
raises if it has not been built: there is no fallback implementation.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtlq.so")

OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_ALIGN, ERR_UNSUPPORTED = -1, -2, -3, -4
ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE, ERR_OVERRUN = -5, -6, -7, -8, -9
W4A16_ASYM_GROUP, W8A8_SYM = 0, 1
WA_SYM_CHANNEL = W8A8_SYM     # symmetric per-channel weights / per-token activations, w_bits and a_bits in 2..8
STAT_MEAN_ABS, STAT_MAX_ABS, STAT_MASKED_MAX = 0, 1, 2
NORM_MEAN_ABS, NORM_L2 = 0, 1
DTYPE_BF16, DTYPE_F32 = 0, 1
N_STAGES = 4
STAGE_NAMES = ("stats", "fakequant", "gemm", "reduce")

EXPORTS = (
    "tlq_status_string", "tlq_version", "tlq_token_importance", "tlq_scale_candidates_workspace_bytes",
    "tlq_scale_candidates", "tlq_scale_candidates_noalloc", "tlq_quantize_weights", "tlq_pack_codes4", "tlq_quantize_activations", "tlq_scale_search_workspace_bytes", "tlq_scale_search_layer", "tlq_scale_search_layer_two_stream",
    "tlq_apply_layer_workspace_bytes", "tlq_apply_layer", "tlq_read_status", "tlq_stage_timing_enable",
    "tlq_stage_timing_drain", "tlq_kernel_launch_count", "tlq_selftest_bounded_wait", "tlq_debug_tile_walk", "tlq_debug_resident_walk", "tlq_l2_partition_info", "tlq_debug_canary_offsets",
    "tlq_debug_check_canaries",
)


class TlqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


class Config(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("mode", ctypes.c_int32), ("w_bits", ctypes.c_int32),
                ("a_bits", ctypes.c_int32), ("group_size", ctypes.c_int32), ("n_grid", ctypes.c_int32),
                ("stat_mode", ctypes.c_int32), ("flags", ctypes.c_uint32)]


FLAG_SKIP_ZERO_WEIGHT_TOKENS = 1
FLAG_GEMM_CTA_PAIRS = 2
FLAG_GEMM_NARROW_TILES = 4
FLAG_NO_REFINE = 8
FLAG_DEBUG_CANARIES = 16


def config(mode: int = W4A16_ASYM_GROUP, w_bits: Optional[int] = None, a_bits: Optional[int] = None,
           group_size: int = 128, n_grid: int = 20, stat_mode: int = STAT_MEAN_ABS, flags: int = 0) -> Config:
    if w_bits is None:
        w_bits = 4 if mode == W4A16_ASYM_GROUP else 8
    if a_bits is None:
        a_bits = 16 if mode == W4A16_ASYM_GROUP else 8
    return Config(ctypes.sizeof(Config), mode, w_bits, a_bits, group_size, n_grid, stat_mode, flags)


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_07899_b200.build` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
    cfgp = ctypes.POINTER(Config)
    lib.tlq_status_string.restype = ctypes.c_char_p
    lib.tlq_status_string.argtypes = [i32]
    lib.tlq_version.restype = i32
    lib.tlq_kernel_launch_count.restype = i64
    lib.tlq_token_importance.argtypes = [vp, i32, i64, i64, i64, i32, ctypes.c_float, vp, vp, vp]
    lib.tlq_scale_candidates_workspace_bytes.restype = sz
    lib.tlq_scale_candidates_workspace_bytes.argtypes = [i64, i64]
    lib.tlq_scale_candidates.argtypes = [vp, i64, i64, vp, cfgp, vp, sz, vp, vp, vp]
    lib.tlq_scale_candidates_noalloc.argtypes = [vp, i64, i64, vp, cfgp, vp, vp, vp]
    lib.tlq_scale_candidates_noalloc.restype = i32
    lib.tlq_quantize_weights.argtypes = [vp, vp, i64, i64, cfgp, vp, vp, vp, vp, vp]
    lib.tlq_pack_codes4.argtypes = [vp, i64, i64, vp, vp]
    lib.tlq_pack_codes4.restype = i32
    lib.tlq_quantize_activations.argtypes = [vp, vp, i64, i64, cfgp, vp, vp, vp]
    lib.tlq_quantize_activations.restype = i32
    lib.tlq_scale_search_workspace_bytes.restype = sz
    lib.tlq_scale_search_workspace_bytes.argtypes = [i64, i64, i64, cfgp]
    lib.tlq_scale_search_layer.argtypes = [vp, i64, i64, vp, i64, vp, vp, cfgp, vp, sz, vp, vp, vp, vp, vp]
    lib.tlq_scale_search_layer_two_stream.argtypes = [vp, vp, i64, i64, vp, i64, vp, vp, cfgp, vp, sz, vp, vp, vp, vp, vp]
    lib.tlq_scale_search_layer_two_stream.restype = i32
    lib.tlq_apply_layer_workspace_bytes.restype = sz
    lib.tlq_apply_layer_workspace_bytes.argtypes = [i64, i64, i64, cfgp]
    lib.tlq_apply_layer.argtypes = [vp, i64, i64, vp, i64, vp, vp, cfgp, vp, sz, vp, vp, vp, vp, vp]
    lib.tlq_read_status.argtypes = [vp, vp]
    lib.tlq_selftest_bounded_wait.argtypes = [vp, sz, i64, vp]
    lib.tlq_selftest_bounded_wait.restype = i32
    lib.tlq_debug_tile_walk.argtypes = [i64, i64, i32, i32, i32, i32, i32, vp]
    lib.tlq_debug_tile_walk.restype = i32
    lib.tlq_debug_canary_offsets.argtypes = [i32, i64, i64, i64, vp, vp, i32]
    lib.tlq_debug_canary_offsets.restype = i32
    lib.tlq_debug_check_canaries.argtypes = [i32, i64, i64, i64, vp, vp, sz, vp]
    lib.tlq_debug_check_canaries.restype = i32
    lib.tlq_l2_partition_info.argtypes = [vp, vp]
    lib.tlq_l2_partition_info.restype = i32
    lib.tlq_debug_resident_walk.argtypes = [i64, i64, i32, i32, i32, vp]
    lib.tlq_debug_resident_walk.restype = i32
    lib.tlq_stage_timing_enable.argtypes = [i32]
    lib.tlq_stage_timing_drain.argtypes = [ctypes.POINTER(ctypes.c_float), i32]
    for fn in ("tlq_token_importance", "tlq_scale_candidates", "tlq_scale_candidates_noalloc", "tlq_quantize_weights", "tlq_pack_codes4", "tlq_quantize_activations", "tlq_scale_search_layer",
               "tlq_apply_layer", "tlq_read_status", "tlq_stage_timing_enable", "tlq_stage_timing_drain"):
        getattr(lib, fn).restype = i32
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.tlq_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(status: int, what: str) -> None:
    if status != OK:
        raise TlqError(status, what)


def tlq_token_importance(G: torch.Tensor, norm_kind: int = NORM_MEAN_ABS, top_frac: float = 0.0,
                         imp_out: Optional[torch.Tensor] = None, mask_out: Optional[torch.Tensor] = None, stream=None):
    """G [B,N,C] (bf16 / int16 bits / float32) -> (imp float32 [N], mask uint8 [N] or None)."""
    if G.dim() == 2:
        G = G.unsqueeze(0)
    B, N, C = G.shape
    dt = DTYPE_F32 if G.dtype == torch.float32 else DTYPE_BF16
    if imp_out is None:
        imp_out = torch.empty(N, dtype=torch.float32, device=G.device)
    if mask_out is None and top_frac > 0:
        mask_out = torch.empty(N, dtype=torch.uint8, device=G.device)
    _check(lib.tlq_token_importance(_ptr(G), dt, B, N, C, norm_kind, float(top_frac), _ptr(imp_out), _ptr(mask_out),
                                    _stream(stream)), "tlq_token_importance")
    return imp_out, mask_out


def tlq_scale_candidates(X: torch.Tensor, cfg: Config, mask: Optional[torch.Tensor] = None, stream=None):
    """X [N,C1] bf16 -> (x_stat float64 [C1], s bf16 [K,C1])."""
    N, C1 = X.shape
    nbytes = lib.tlq_scale_candidates_workspace_bytes(N, C1)
    ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=X.device)
    x_stat = torch.empty(C1, dtype=torch.float64, device=X.device)
    s = torch.empty((cfg.n_grid, C1), dtype=torch.bfloat16, device=X.device)
    _check(lib.tlq_scale_candidates(_ptr(X), N, C1, _ptr(mask), ctypes.byref(cfg), _ptr(ws), nbytes, _ptr(x_stat),
                                    _ptr(s), _stream(stream)), "tlq_scale_candidates")
    return x_stat, s


def tlq_scale_candidates_noalloc(X: torch.Tensor, cfg: Config, x_stat: torch.Tensor, s: torch.Tensor,
                                 mask: Optional[torch.Tensor] = None, stream=None) -> None:
    """Same result as tlq_scale_candidates, written into the caller's x_stat [C1] float64 and s [K,C1] bf16;
    the library uses its built-in scratch array, so nothing is allocated here or in the library."""
    N, C1 = X.shape
    _check(lib.tlq_scale_candidates_noalloc(_ptr(X), N, C1, _ptr(mask), ctypes.byref(cfg), _ptr(x_stat), _ptr(s),
                                            _stream(stream)), "tlq_scale_candidates_noalloc")


def tlq_quantize_weights(W: torch.Tensor, s: Optional[torch.Tensor], cfg: Config, want_dw: bool = False, stream=None):
    """W [C2,C1] bf16, s [C1] bf16 or None -> dict(codes, steps, zeros, dW)."""
    C2, C1 = W.shape
    dev = W.device
    if cfg.mode == W4A16_ASYM_GROUP:
        ng = C1 // cfg.group_size
        codes = torch.empty((C2, C1), dtype=torch.uint8, device=dev)
        steps = torch.empty((C2, ng), dtype=torch.float32, device=dev)
        zeros = torch.empty((C2, ng), dtype=torch.int32, device=dev)
        dW = torch.empty((C2, C1), dtype=torch.bfloat16, device=dev) if want_dw else None
    else:
        codes = torch.empty((C2, C1), dtype=torch.int8, device=dev)
        steps = torch.empty((C2,), dtype=torch.float32, device=dev)
        zeros, dW = None, None
    _check(lib.tlq_quantize_weights(_ptr(W), _ptr(s), C2, C1, ctypes.byref(cfg), _ptr(codes), _ptr(steps), _ptr(zeros),
                                    _ptr(dW), _stream(stream)), "tlq_quantize_weights")
    return dict(codes=codes, steps=steps, zeros=zeros, dW=dW)


def tlq_pack_codes4(codes: torch.Tensor, stream=None) -> torch.Tensor:
    """codes uint8/int8 [R,C] (one 4-bit code per byte) -> uint8 [R,C/2], even channel in the low nibble."""
    R, C = codes.shape
    packed = torch.empty((R, C // 2), dtype=torch.uint8, device=codes.device)
    _check(lib.tlq_pack_codes4(_ptr(codes), R, C, _ptr(packed), _stream(stream)), "tlq_pack_codes4")
    return packed


def tlq_quantize_activations(X: torch.Tensor, s: Optional[torch.Tensor], cfg: Config, stream=None):
    """X [N,C1] bf16, s [C1] bf16 or None -> (codes int8 [N,C1], steps float32 [N]) (W8A8 mode)."""
    N, C1 = X.shape
    codes = torch.empty((N, C1), dtype=torch.int8, device=X.device)
    steps = torch.empty((N,), dtype=torch.float32, device=X.device)
    _check(lib.tlq_quantize_activations(_ptr(X), _ptr(s), N, C1, ctypes.byref(cfg), _ptr(codes), _ptr(steps),
                                        _stream(stream)), "tlq_quantize_activations")
    return codes, steps


def tlq_scale_search_workspace_bytes(N: int, C1: int, C2: int, cfg: Config) -> int:
    return int(lib.tlq_scale_search_workspace_bytes(N, C1, C2, ctypes.byref(cfg)))


class SearchBuffers:
    """Caller-owned device buffers of one tlq_scale_search_layer call (reusable across calls)."""

    def __init__(self, N: int, C1: int, C2: int, cfg: Config, device, per_token: bool = False,
                 workspace: Optional[torch.Tensor] = None):
        self.nbytes = tlq_scale_search_workspace_bytes(N, C1, C2, cfg)
        if self.nbytes == 0:
            raise TlqError(ERR_SHAPE, "tlq_scale_search_workspace_bytes")
        if workspace is None or workspace.numel() < self.nbytes:
            workspace = torch.empty(self.nbytes, dtype=torch.uint8, device=device)
        self.workspace = workspace
        self.best_idx = torch.empty(1, dtype=torch.int32, device=device)
        self.losses = torch.empty(cfg.n_grid, dtype=torch.float64, device=device)
        self.s_best = torch.empty(C1, dtype=torch.bfloat16, device=device)
        self.per_token = torch.empty((cfg.n_grid, N), dtype=torch.float32, device=device) if per_token else None


def tlq_scale_search_layer(X: torch.Tensor, W: torch.Tensor, w_imp: Optional[torch.Tensor], cfg: Config,
                           buffers: Optional[SearchBuffers] = None, mask: Optional[torch.Tensor] = None,
                           per_token: bool = False, stream=None, check: bool = True,
                           X_fp: Optional[torch.Tensor] = None) -> SearchBuffers:
    """Enqueue the search; with check=True also synchronise and raise on a device-side error.
    X_fp selects tlq_scale_search_layer_two_stream (X is then the quantized stream)."""
    N, C1 = X.shape
    C2 = W.shape[0]
    if buffers is None:
        buffers = SearchBuffers(N, C1, C2, cfg, X.device, per_token)
    st = _stream(stream)
    if X_fp is None:
        _check(lib.tlq_scale_search_layer(_ptr(X), N, C1, _ptr(W), C2, _ptr(w_imp), _ptr(mask), ctypes.byref(cfg),
                                          _ptr(buffers.workspace), buffers.nbytes, _ptr(buffers.best_idx),
                                          _ptr(buffers.losses), _ptr(buffers.s_best), _ptr(buffers.per_token), st),
               "tlq_scale_search_layer")
    else:
        if X_fp.shape != X.shape:
            raise ValueError("X_fp must have the shape of X")
        _check(lib.tlq_scale_search_layer_two_stream(_ptr(X), _ptr(X_fp), N, C1, _ptr(W), C2, _ptr(w_imp), _ptr(mask),
                                                     ctypes.byref(cfg), _ptr(buffers.workspace), buffers.nbytes,
                                                     _ptr(buffers.best_idx), _ptr(buffers.losses), _ptr(buffers.s_best),
                                                     _ptr(buffers.per_token), st),
               "tlq_scale_search_layer_two_stream")
    if check:
        _check(lib.tlq_read_status(_ptr(buffers.workspace), st), "tlq_scale_search_layer (device)")
    return buffers


def tlq_apply_layer(X: torch.Tensor, W: torch.Tensor, s: Optional[torch.Tensor], bias: Optional[torch.Tensor],
                    cfg: Config, want_codes: bool = True, stream=None, check: bool = True):
    """-> dict(Yq bf16 [N,C2], codes, steps, zeros)."""
    N, C1 = X.shape
    C2 = W.shape[0]
    dev = X.device
    nbytes = int(lib.tlq_apply_layer_workspace_bytes(N, C1, C2, ctypes.byref(cfg)))
    if nbytes == 0:
        raise TlqError(ERR_SHAPE, "tlq_apply_layer_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    Yq = torch.empty((N, C2), dtype=torch.bfloat16, device=dev)
    codes = steps = zeros = None
    if want_codes:
        if cfg.mode == W4A16_ASYM_GROUP:
            ng = C1 // cfg.group_size
            codes = torch.empty((C2, C1), dtype=torch.uint8, device=dev)
            steps = torch.empty((C2, ng), dtype=torch.float32, device=dev)
            zeros = torch.empty((C2, ng), dtype=torch.int32, device=dev)
        else:
            codes = torch.empty((C2, C1), dtype=torch.int8, device=dev)
            steps = torch.empty((C2,), dtype=torch.float32, device=dev)
    st = _stream(stream)
    _check(lib.tlq_apply_layer(_ptr(X), N, C1, _ptr(W), C2, _ptr(s), _ptr(bias), ctypes.byref(cfg), _ptr(ws), nbytes,
                               _ptr(codes), _ptr(steps), _ptr(zeros), _ptr(Yq), st), "tlq_apply_layer")
    if check:
        _check(lib.tlq_read_status(_ptr(ws), st), "tlq_apply_layer (device)")
    return dict(Yq=Yq, codes=codes, steps=steps, zeros=zeros)


def tlq_read_status(workspace: torch.Tensor, stream=None) -> int:
    return int(lib.tlq_read_status(_ptr(workspace), _stream(stream)))


def tlq_selftest_bounded_wait(workspace: torch.Tensor, limit_cycles: int = 2_000_000, stream=None) -> int:
    """Run the bounded-wait self-test on `workspace` and return the device status it left (TLQ_ERR_TIMEOUT when
    the error path works).  Synchronises the stream."""
    st = _stream(stream)
    _check(lib.tlq_selftest_bounded_wait(_ptr(workspace), workspace.numel() * workspace.element_size(), int(limit_cycles), st),
           "tlq_selftest_bounded_wait")
    return int(lib.tlq_read_status(_ptr(workspace), st))


def tlq_debug_canary_offsets(kind: int, N: int, C1: int, C2: int, cfg: Config):
    """-> list of byte offsets of the guard words of a workspace laid out with FLAG_DEBUG_CANARIES (host only)."""
    buf = (ctypes.c_uint64 * 32)()
    n = int(lib.tlq_debug_canary_offsets(kind, N, C1, C2, ctypes.byref(cfg), buf, 32))
    _check(min(n, 0), "tlq_debug_canary_offsets")
    return [int(buf[i]) for i in range(n)]


def tlq_debug_check_canaries(kind: int, N: int, C1: int, C2: int, cfg: Config, workspace: torch.Tensor,
                             stream=None) -> None:
    """Enqueue one more comparison of the guard words; read the outcome with tlq_read_status."""
    _check(lib.tlq_debug_check_canaries(kind, N, C1, C2, ctypes.byref(cfg), _ptr(workspace), workspace.numel(),
                                        _stream(stream)), "tlq_debug_check_canaries")


def tlq_l2_partition_info():
    """-> dict(valid, n_sms, count=(n0, n1), part=numpy uint8 [256]): the current device's SM -> L2 partition table."""
    import numpy as np
    info = (ctypes.c_int32 * 4)()
    part = np.zeros(256, dtype=np.uint8)
    _check(lib.tlq_l2_partition_info(info, part.ctypes.data_as(ctypes.c_void_p)), "tlq_l2_partition_info")
    return dict(valid=bool(info[0]), n_sms=int(info[1]), count=(int(info[2]), int(info[3])), part=part)


def tlq_debug_tile_walk(mtiles: int, otiles: int, K: int, n0: int, n1: int = 0, blocked: bool = False, block_a: int = 8):
    """Host-side replay of the fused GEMM's tile walk -> numpy int32 [K, otiles, mtiles] of visit counts."""
    import numpy as np
    visits = np.zeros((K, otiles, mtiles), dtype=np.int32)
    _check(lib.tlq_debug_tile_walk(mtiles, otiles, K, n0, n1, 1 if blocked else 0, block_a,
                                   visits.ctypes.data_as(ctypes.c_void_p)), "tlq_debug_tile_walk")
    return visits


def tlq_debug_resident_walk(mtiles: int, otiles: int, K: int, grid: int, blocked: bool = True):
    """Host-side replay of the tile-resident kernels' work items -> numpy int32 [K, otiles, mtiles] of visit counts."""
    import numpy as np
    visits = np.zeros((K, otiles, mtiles), dtype=np.int32)
    _check(lib.tlq_debug_resident_walk(mtiles, otiles, K, grid, 1 if blocked else 0,
                                       visits.ctypes.data_as(ctypes.c_void_p)), "tlq_debug_resident_walk")
    return visits


def tlq_stage_timing_enable(on: bool) -> None:
    _check(lib.tlq_stage_timing_enable(1 if on else 0), "tlq_stage_timing_enable")


def tlq_stage_timing_drain(max_calls: int = 512):
    """-> list of per-call [stats, fakequant, gemm, reduce] milliseconds, oldest call first."""
    arr = (ctypes.c_float * (N_STAGES * max_calls))()
    n = lib.tlq_stage_timing_drain(arr, max_calls)
    if n < 0:
        raise TlqError(n, "tlq_stage_timing_drain")
    return [[float(arr[c * N_STAGES + i]) for i in range(N_STAGES)] for c in range(n)]


def tlq_kernel_launch_count() -> int:
    return int(lib.tlq_kernel_launch_count())


def bf16_from_bits(bits, device="cuda") -> torch.Tensor:
    """numpy uint16 bit patterns -> torch.bfloat16 device tensor (no arithmetic)."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)
