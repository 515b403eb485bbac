"""Device-resident synthetic workloads shaped like the paper's evaluation models (Section 6): the
linear layers of a decoder stack, packed once (packing happens once, at model load,
Section 5.1) and then driven token by token (decode) or prompt by prompt (prefill).

Only plumbing lives here: seeded arrays from ``inputs`` are packed with the library's host packer,
copied to the GPU, and the launches of one step are issued through the C ABI.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

from . import binding as B
from . import inputs

# which linears of a decoder layer read the same activations: (q, k, v), (o), (gate, up), (down)
_INPUT_OF = {"q": 0, "k": 0, "v": 0, "o": 1, "gate": 2, "up": 2, "down": 3}
_INPUT_SEED_ID = {0: 0, 1: 3, 2: 4, 3: 6}


w4_bytes = inputs.w4_bytes
linear_bytes = inputs.linear_bytes


@dataclass
class _Layer:
    packed: Dict[str, torch.Tensor] = field(default_factory=dict)
    x_off: Dict[int, Tuple[int, int]] = field(default_factory=dict)   # input id -> (offset, K) in halfs
    y_off: Dict[str, Tuple[int, int]] = field(default_factory=dict)   # linear -> (offset, N) in halfs


class LinearStack:
    """All linears of ``layers`` decoder layers of ``model`` for ``M`` tokens.

    ``xin`` holds every layer's four input activations back to back ([M, K] each), ``yout`` every
    linear's output ([M, N] each); ``xin_host`` / ``yout_host`` are pinned mirrors for end-to-end
    timing.  ``run_w4a16`` issues the decode launches of one step: per layer one batched launch
    for q, k, v (same input), one for o, one batched for gate and up, one for down.
    """

    def __init__(self, model: dict, config: int, M: int, group: int = 64, layers: Optional[int] = None,
                 outliers: bool = False, device: str = "cuda", weights_from: "Optional[LinearStack]" = None,
                 distinct: Optional[int] = None):
        """``distinct`` = d < layers: only the first d layers get arrays of their own; layer l reuses
        the packed weights and the input activations of layer l mod d (outputs stay separate).  With
        d layers of weights well above the L2 size every pass still streams from DRAM; it bounds the
        host time spent drawing random numbers for the large models."""
        self.model, self.config, self.M, self.group = model, config, M, group
        self.n_layers = model["layers"] if layers is None else layers
        self.linears = inputs.stack(model)
        self.device = torch.device(device)
        xs: List[np.ndarray] = []
        x_total = y_total = 0
        self.layers: List[_Layer] = []
        self.weight_bytes = 0
        self.algorithmic_bytes_w4a16 = 0
        self.ops = 0
        self.distinct = self.n_layers if distinct is None else max(1, min(distinct, self.n_layers))
        for l in range(self.n_layers):
            L = _Layer()
            src = self.layers[l % self.distinct] if l >= self.distinct else None
            for lin in self.linears:
                if weights_from is not None:   # same packed weights, other activations
                    L.packed[lin.name] = weights_from.layers[l].packed[lin.name]
                elif src is not None:
                    L.packed[lin.name] = src.packed[lin.name]
                else:
                    W = inputs.weights(inputs.seed_for(config, l, lin.matrix_id, 0), lin.N, lin.K)
                    L.packed[lin.name] = torch.from_numpy(B.pack_w4(W, group)).to(self.device)
                    del W
                iid = _INPUT_OF[lin.name]
                if src is not None:
                    L.x_off[iid] = src.x_off[iid]
                if iid not in L.x_off:
                    x = inputs.activations(inputs.seed_for(config, l, _INPUT_SEED_ID[iid], 1), M, lin.K,
                                           outliers=outliers)
                    L.x_off[iid] = (x_total, lin.K)
                    xs.append(x.reshape(-1))
                    x_total += M * lin.K
                L.y_off[lin.name] = (y_total, lin.N)
                y_total += M * lin.N
                self.weight_bytes += w4_bytes(lin.N, lin.K, group)
                self.algorithmic_bytes_w4a16 += linear_bytes(lin.N, lin.K, group, M)
                self.ops += 2 * M * lin.N * lin.K
            self.layers.append(L)
        self.xin_host = torch.from_numpy(np.concatenate(xs)).pin_memory()
        self.xin = self.xin_host.to(self.device)
        self.yout = torch.zeros(y_total, dtype=torch.float16, device=self.device)
        self.yout_host = torch.empty(y_total, dtype=torch.float16).pin_memory()
        self._launches = None
        self._workspace = None

    # ---- views ----
    def x_view(self, layer: int, name: str) -> torch.Tensor:
        off, K = self.layers[layer].x_off[_INPUT_OF[name]]
        return self.xin[off:off + self.M * K].view(self.M, K)

    def y_view(self, layer: int, name: str) -> torch.Tensor:
        off, N = self.layers[layer].y_off[name]
        return self.yout[off:off + self.M * N].view(self.M, N)

    # ---- decode ----
    def _decode_launches(self):
        if self._launches is None:
            out = []
            for l, L in enumerate(self.layers):
                for names in (("q", "k", "v"), ("o",), ("gate", "up"), ("down",)):
                    probs = []
                    for name in names:
                        lin = next(t for t in self.linears if t.name == name)
                        probs.append(dict(x=self.x_view(l, name), packed=L.packed[name], y=self.y_view(l, name),
                                          N=lin.N, K=lin.K, group=self.group, y_dtype=B.F16))
                    out.append(B.make_batch(probs))
            self._launches = out
        return self._launches

    @property
    def launches_per_step_w4a16(self) -> int:
        return 4 * self.n_layers * ((self.M + 7) // 8)

    def run_w4a16(self, stream=None) -> None:
        for arr in self._decode_launches():
            B.linear_w4a16_batch(arr, self.M, stream)

    def _stack_plan(self):
        """The whole stack as ONE launch.  The dependency list is the decoder's: q, k, v wait for the
        previous layer's down projection, o for q, k, v, gate and up for o, down for gate and up."""
        if getattr(self, "_plan", None) is None:
            probs, prev_down = [], None
            for l, L in enumerate(self.layers):
                idx = {}
                for lin in self.linears:
                    deps = {"q": [prev_down], "k": [prev_down], "v": [prev_down], "o": [idx.get("q"), idx.get("k"), idx.get("v")],
                            "gate": [idx.get("o")], "up": [idx.get("o")], "down": [idx.get("gate"), idx.get("up")]}[lin.name]
                    idx[lin.name] = len(probs)
                    probs.append(dict(x=self.x_view(l, lin.name), packed=L.packed[lin.name], y=self.y_view(l, lin.name),
                                      N=lin.N, K=lin.K, y_dtype=B.F16, deps=[d for d in deps if d is not None]))
                prev_down = idx["down"]
            plan = B.stack_plan_w4a16(probs, self.M, self.group)
            plan_dev = torch.from_numpy(plan).to(self.device)
            nbytes = B.stack_workspace_size(plan)
            ws = torch.zeros(nbytes, dtype=torch.uint8, device=self.device)
            self._plan = (plan, plan_dev, ws, nbytes)
        return self._plan

    def run_w4a16_stack(self, stream=None) -> None:
        plan, plan_dev, ws, nbytes = self._stack_plan()
        B.linear_w4a16_stack(plan, plan_dev, ws, nbytes, stream)

    # ---- prefill ----
    @property
    def launches_per_step_w4a8(self) -> int:
        return 2 * 4 * self.n_layers   # per layer: q+k+v, o, gate+up, down; quantiser + GEMM each

    def _prefill_launches(self):
        if getattr(self, "_pre", None) is None:
            out = []
            for l, L in enumerate(self.layers):
                for names in (("q", "k", "v"), ("o",), ("gate", "up"), ("down",)):
                    lins = [next(t for t in self.linears if t.name == n) for n in names]
                    arr = B.make_batch_w4a8([dict(packed=L.packed[t.name], y=self.y_view(l, t.name), N=t.N, y_dtype=B.F16)
                                             for t in lins])
                    out.append((arr, self.x_view(l, names[0]), lins[0].K))
            self._pre = out
        return self._pre

    def run_w4a8(self, stream=None) -> None:
        """One prefill step: per layer the matrices that share their input go in one call (one
        quantiser pass, one GEMM launch): q+k+v, o, gate+up, down."""
        if self._workspace is None:
            need = max(B.workspace_size_w4a8(self.M, t.N, t.K, self.group) for t in self.linears)
            self._workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        ws, nbytes = self._workspace, self._workspace.numel()
        for arr, x, K in self._prefill_launches():
            B.linear_w4a8_batch(arr, x, self.M, K, self.group, ws, nbytes, stream=stream)
