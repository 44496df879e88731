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
        for L in layers:
            w = torch.from_numpy(inputs.to_storage(L["w"])).to(self.device)
            self.layers.append({**{k: v for k, v in L.items() if k != "w"}, "d_w": w})
        self.head_w = torch.from_numpy(inputs.to_storage(head_w)).to(self.device)
        self.workspace = None
        self._ws_shape = None
        self._tiles = {}          # (algo, fused_pool, input shape) -> per-layer tuning records found by tune_tiles()

    def _ensure_workspace(self, shape):
        """One workspace large enough for every layer of a batch of this input shape."""
        if self._ws_shape == tuple(shape):
            return
        B, _, H, W = shape
        need = 0
        for L in self.layers:
            Co, Ci, K, _ = L["d_w"].shape
            need = max(need, hk.conv2d_workspace_bytes(B, Ci, H, W, Co, K, L["pad"]))
            H, W = H + 2 * L["pad"] - K + 1, W + 2 * L["pad"] - K + 1
            if L["pool"]:
                H, W = H // 2, W // 2
        Co, Ci, K, _ = self.head_w.shape
        need = max(need, hk.conv2d_workspace_bytes(B, Ci, H, W, Co, K, 0))
        self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
        self._ws_shape = tuple(shape)

    def _layer(self, a, L, algo, fused_pool, tune, stream):
        """One conv3x3 layer with its requantisation and, if it has one, its pool."""
        rq = (L["shift"], L["lo"], L["hi"])
        if L["pool"] and fused_pool:
            B, Ci, H, W = a.shape
            return hk.conv2d_dense(a.reshape(-1), (B, Ci, H, W), 8, L["d_w"].reshape(-1), tuple(L["d_w"].shape), 8, L["pad"], L["p"],
                                   L["q"], L["x_signed"], L["w_signed"], requant=rq, out_store_bits=8, pool=True, algo=algo,
                                   tune=tune, workspace=self.workspace, stream=stream)
        a = hk.conv2d(a, L["d_w"], L["pad"], L["p"], L["q"], L["x_signed"], L["w_signed"], requant=rq, algo=algo, tune=tune,
                      workspace=self.workspace, stream=stream)
        if L["pool"]:
            a = hk.maxpool2x2_i8(a, is_signed=L["lo"] < 0, stream=stream)
        return a

    def tune_tiles(self, d_x: torch.Tensor, algo: int = hk.ALGO_PACKED32, fused_pool: bool = True, repeats: int = 3) -> List[Optional[dict]]:
        """Lets the library time, layer by layer on this input, every tile shape it accepts against its own choice
        (``hikonv_conv2d_tune``) and keeps a forced tile where it measures at least 3 % faster; later ``forward`` calls
        on inputs of this shape and these options use the kept tiles.  Results do not depend on the tile.  Returns the
        per-layer tuning records (None: the library's choice stays)."""
        self._ensure_workspace(d_x.shape)
        kept: List[Optional[dict]] = []
        a = d_x
        for L in self.layers:
            B, Ci, H, W = a.shape
            rq = (L["shift"], L["lo"], L["hi"])
            pool_here = bool(L["pool"] and fused_pool)
            found = hk.conv2d_tune(a.reshape(-1), (B, Ci, H, W), 8, L["d_w"].reshape(-1), tuple(L["d_w"].shape), 8, L["pad"], L["p"],
                                   L["q"], L["x_signed"], L["w_signed"], requant=rq, out_store_bits=8, pool=pool_here, algo=algo,
                                   workspace=self.workspace, repeats=repeats)
            kept.append(found["tune"])
            a = found["out"]
            if L["pool"] and not fused_pool:
                a = hk.maxpool2x2_i8(a, is_signed=L["lo"] < 0)
        torch.cuda.synchronize()
        self._tiles[(algo, bool(fused_pool), tuple(d_x.shape))] = kept
        return kept

    def set_tiles(self, shape, tiles: List[Optional[dict]], algo: int = hk.ALGO_PACKED32, fused_pool: bool = True) -> None:
        """Tuning records found earlier (``tune_tiles``) for inputs of this shape, one per layer (None: automatic)."""
        if len(tiles) != len(self.layers):
            raise ValueError("one tuning record per layer")
        self._tiles[(algo, bool(fused_pool), tuple(shape))] = list(tiles)

    def forward(self, d_x: torch.Tensor, algo: int = hk.ALGO_PACKED32, keep_activations: bool = False, stream=None,
                fused_pool: bool = True):
        """``fused_pool``: layers followed by a pool run it inside their epilogue (``hikonv_conv2d_dense`` with one code
        per byte; the default: four launches fewer, 0.651 against 0.654 ms on the benchmark network); otherwise the pool
        is a launch of its own."""
        self._ensure_workspace(d_x.shape)
        tiles = self._tiles.get((algo, bool(fused_pool), tuple(d_x.shape)))
        acts = []
        a = d_x
        for i, L in enumerate(self.layers):
            a = self._layer(a, L, algo, fused_pool, tiles[i] if tiles else None, stream)
            if keep_activations:
                acts.append(a)
        last = self.layers[-1]
        head = hk.conv2d(a, self.head_w, 0, 4, 4, last["lo"] < 0, True, requant=None, algo=algo,
                         workspace=self.workspace, stream=stream)
        return head, acts
