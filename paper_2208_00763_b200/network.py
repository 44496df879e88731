"""The compact quantised CNN workload as a chain of library calls (marshalling only).

Every arithmetic step (convolution, requantisation, pooling) runs in the CUDA library; this
class only keeps the device buffers and issues the calls layer by layer on one stream.
"""
from __future__ import annotations

from typing import List, Optional

import torch

from . import binding as hk
from . import inputs


class CompactCnn:
    """conv3x3 -> shift/clamp -> optional 2x2 max-pool, repeated; then a 1x1 head with int32 output."""

    def __init__(self, layers: List[dict], head_w, device="cuda"):
        self.device = torch.device(device)
        self.layers = []
        ws_bytes = 0
        for L in layers:
            w = torch.from_numpy(inputs.to_storage(L["w"])).to(self.device)
            self.layers.append({**{k: v for k, v in L.items() if k != "w"}, "d_w": w})
            Co, Ci, K, _ = w.shape
            ws_bytes = max(ws_bytes, hk.conv2d_workspace_bytes(Ci, Co, K))
        self.head_w = torch.from_numpy(inputs.to_storage(head_w)).to(self.device)
        Co, Ci, K, _ = self.head_w.shape
        ws_bytes = max(ws_bytes, hk.conv2d_workspace_bytes(Ci, Co, K))
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)

    def forward(self, d_x: torch.Tensor, algo: int = hk.ALGO_PACKED32, keep_activations: bool = False, stream=None):
        acts = []
        a = d_x
        for L in self.layers:
            a = hk.conv2d(a, L["d_w"], L["pad"], L["p"], L["q"], L["x_signed"], L["w_signed"],
                          requant=(L["shift"], L["lo"], L["hi"]), algo=algo, workspace=self.workspace, stream=stream)
            if L["pool"]:
                a = hk.maxpool2x2_i8(a, is_signed=L["lo"] < 0, stream=stream)
            if keep_activations:
                acts.append(a)
        last = self.layers[-1]
        head = hk.conv2d(a, self.head_w, 0, 4, 4, last["lo"] < 0, True, requant=None, algo=algo,
                         workspace=self.workspace, stream=stream)
        return head, acts
