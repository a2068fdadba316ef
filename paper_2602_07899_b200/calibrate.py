"""Scale search of a layer's linears whose inputs live in (pinned) host memory.

The searches themselves are the library's kernels (`tlq_scale_search_layer`); what this module adds is
plumbing only: per-linear staging buffers on the device, a side stream for the host-to-device copies,
and events, so that the copy of the next linear's weights (and of the next layer's activations) runs
while the tensor cores work on the current linear.  The calibration inputs of a 7B-class layer are
about 1 GB per layer; at PCIe rates that is a quarter of the layer's compute time when done in line,
and nothing when overlapped.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence, Tuple

import torch

from . import tlq

# (name, activation tensor name, N, C1, C2)
LinearShape = Tuple[str, str, int, int, int]


class HostLayerSearch:
    """Repeatedly searches the same set of linears; every `run` takes fresh host tensors.

    shapes    one entry per linear, in execution order; linears naming the same activation tensor share it
    cfg       tlq.Config
    Device memory held: one staging buffer per activation tensor and per weight matrix, the importance
    vector, one workspace sized for the largest linear, and the small result buffers.
    """

    def __init__(self, shapes: Sequence[LinearShape], cfg: tlq.Config, device: torch.device):
        self.shapes = list(shapes)
        self.cfg = cfg
        self.device = device
        self.copy_stream = torch.cuda.Stream(device=device)
        n_tokens = {s[2] for s in self.shapes}
        if len(n_tokens) != 1:
            raise ValueError("all linears of one layer see the same tokens")
        self.n_tokens = n_tokens.pop()
        self.x_stage: Dict[str, torch.Tensor] = {}
        self.w_stage: Dict[str, torch.Tensor] = {}
        for name, x_name, n, c1, c2 in self.shapes:
            if x_name not in self.x_stage:
                self.x_stage[x_name] = torch.empty((n, c1), dtype=torch.bfloat16, device=device)
            self.w_stage[name] = torch.empty((c2, c1), dtype=torch.bfloat16, device=device)
        self.imp_stage = torch.empty(self.n_tokens, dtype=torch.float32, device=device)
        ws_bytes = max(tlq.tlq_scale_search_workspace_bytes(n, c1, c2, cfg) for _, _, n, c1, c2 in self.shapes)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
        self.bufs = {name: tlq.SearchBuffers(n, c1, c2, cfg, device, False, self.workspace)
                     for name, _, n, c1, c2 in self.shapes}
        # events: inputs of a linear have landed / the kernels that read a staging buffer have finished
        self.ready = {name: torch.cuda.Event() for name, *_ in self.shapes}
        self.w_free = {name: None for name, *_ in self.shapes}
        self.x_free: Dict[str, Optional[torch.cuda.Event]] = {k: None for k in self.x_stage}
        self.imp_free: Optional[torch.cuda.Event] = None
        self.last_user = {}
        for name, x_name, *_ in self.shapes:
            self.last_user[x_name] = name

    @staticmethod
    def _as_bf16(t: torch.Tensor) -> torch.Tensor:
        return t if t.dtype == torch.bfloat16 else t.view(torch.bfloat16)

    def run(self, host_x: Dict[str, torch.Tensor], host_w: Dict[str, torch.Tensor],
            host_imp: Optional[torch.Tensor],
            out_host: Optional[Dict[str, Tuple[torch.Tensor, torch.Tensor]]] = None) -> Dict[str, tlq.SearchBuffers]:
        """Enqueue copies and searches of all linears; returns the per-linear result buffers (device).
        If `out_host` gives pinned (best_idx int32[1], losses float64[K]) pairs, results are copied there too.
        Nothing here synchronises with the host: call `check()` (or synchronise) before reading results."""
        compute = torch.cuda.current_stream(self.device)
        cs = self.copy_stream
        copied_x = set()
        with torch.cuda.stream(cs):
            if host_imp is not None:
                if self.imp_free is not None:
                    cs.wait_event(self.imp_free)
                self.imp_stage.copy_(host_imp, non_blocking=True)
            for name, x_name, *_ in self.shapes:
                if x_name not in copied_x:
                    if self.x_free[x_name] is not None:
                        cs.wait_event(self.x_free[x_name])
                    self.x_stage[x_name].copy_(self._as_bf16(host_x[x_name]), non_blocking=True)
                    copied_x.add(x_name)
                if self.w_free[name] is not None:
                    cs.wait_event(self.w_free[name])
                self.w_stage[name].copy_(self._as_bf16(host_w[name]), non_blocking=True)
                self.ready[name].record(cs)
        imp = self.imp_stage if host_imp is not None else None
        for name, x_name, *_ in self.shapes:
            compute.wait_event(self.ready[name])
            tlq.tlq_scale_search_layer(self.x_stage[x_name], self.w_stage[name], imp, self.cfg, self.bufs[name],
                                       check=False)
            ev = torch.cuda.Event()
            ev.record(compute)
            self.w_free[name] = ev
            if self.last_user[x_name] == name:
                self.x_free[x_name] = ev
            if out_host is not None:
                out_host[name][0].copy_(self.bufs[name].best_idx, non_blocking=True)
                out_host[name][1].copy_(self.bufs[name].losses, non_blocking=True)
        self.imp_free = self.w_free[self.shapes[-1][0]]
        return self.bufs

    def check(self) -> None:
        """Synchronise and raise if a kernel reported a device-side error."""
        st = tlq.tlq_read_status(self.workspace)
        if st != tlq.OK:
            raise tlq.TlqError(st, "HostLayerSearch")
