"""User-facing wrapper: a quantised layer resident on the GPU and its V step.

All computation happens in the CUDA library (``binding``); this class only owns
the device tensors, the workspace and the call order
select -> encode -> dequantise of one step (Algorithm 3, V-step lines and
``dequantize_weights``).
"""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as B
from .synth import SynthLayer


def _codes_to_torch(codes: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(codes))


class VStepLayer:
    def __init__(self, rows, cols, W, g, scale, codebooks, codes, *, eta=1.0, beam=8, max_k=None, group_dim=8):
        self.rows, self.cols = int(rows), int(cols)
        self.W, self.g, self.scale, self.codebooks, self.codes = W, g, scale, codebooks, codes
        self.eta, self.beam = float(eta), int(beam)
        self.group_dim = int(group_dim)
        self.num_groups = self.rows * (self.cols // self.group_dim)
        self.desc = B.make_layer(self.rows, self.cols, W, g, scale, codebooks, codes, eta=self.eta, beam=self.beam,
                                 group_dim=self.group_dim)
        self._ws = None
        self._ws_k = 0
        if max_k is not None:
            self.reserve(max_k)

    @classmethod
    def from_host(cls, L: SynthLayer, device="cuda", max_k=None) -> "VStepLayer":
        dev = torch.device(device)
        up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        return cls(L.rows, L.cols, up(L.W), up(L.g), up(L.scale), up(L.codebooks), _codes_to_torch(L.codes).to(dev),
                   eta=L.eta, beam=L.beam, max_k=max_k, group_dim=L.group_dim)

    def reserve(self, k: int) -> torch.Tensor:
        """Workspace large enough for select/encode with this k (grown on demand)."""
        need = B.pvt_workspace_bytes(self.desc, k)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.W.device)
            B.pvt_workspace_init(self._ws)
        return self._ws

    def select(self, k: int, idx_out: Optional[torch.Tensor] = None) -> torch.Tensor:
        ws = self.reserve(k)
        if idx_out is None:
            idx_out = torch.empty(k, dtype=torch.int32, device=self.W.device)
        B.pvt_vstep_select(self.desc, k, idx_out, ws)
        return idx_out

    def select_ste(self, buffer: torch.Tensor, k: int, idx_out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Selection while the straight-through buffer takes the step (Appendix E): buffer -= eta * g in place."""
        ws = self.reserve(k)
        if idx_out is None:
            idx_out = torch.empty(k, dtype=torch.int32, device=self.W.device)
        B.pvt_vstep_select_ste(self.desc, buffer, k, idx_out, ws)
        return idx_out

    def sample(self, k: int, rule: int, seed: int, idx_out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """A random subspace (B.PVT_SAMPLE_UNIFORM / B.PVT_SAMPLE_PROPORTIONAL) instead of the greedy one."""
        ws = self.reserve(k)
        if idx_out is None:
            idx_out = torch.empty(k, dtype=torch.int32, device=self.W.device)
        B.pvt_vstep_sample(self.desc, k, rule, seed, idx_out, ws)
        return idx_out

    def encode_against(self, buffer: torch.Tensor, idx: torch.Tensor, err_out: Optional[torch.Tensor] = None) -> None:
        """Re-encode the listed groups against buffer / scale (the V step's search with W = buffer, zero step)."""
        k = int(idx.numel())
        desc = B.make_layer(self.rows, self.cols, buffer, self.g, self.scale, self.codebooks, self.codes, eta=0.0,
                            beam=self.beam, group_dim=self.group_dim)
        B.pvt_vstep_encode(desc, idx, k, err_out, self.reserve(k))

    def encode(self, idx: torch.Tensor, err_out: Optional[torch.Tensor] = None) -> None:
        k = int(idx.numel())
        B.pvt_vstep_encode(self.desc, idx, k, err_out, self.reserve(k))

    def dequant(self, out: Optional[torch.Tensor] = None, dtype=torch.float32) -> torch.Tensor:
        if out is None:
            out = torch.empty(self.rows, self.cols, dtype=dtype, device=self.W.device)
        B.pvt_dequant(self.desc, out)
        return out

    def step(self, k: int, idx_out=None, W_hat=None, err_out=None):
        """One V step followed by the dequantisation that opens the next step."""
        idx = self.select(k, idx_out)
        self.encode(idx, err_out)
        return idx, self.dequant(W_hat) if W_hat is not None else None

    def step_trust(self, k_max: int, ratio: float = 0.01):
        """V step whose subspace size follows from the trust ratio (Section 4.3, Appendix J): returns the groups
        in rank order (int32 [k_max]), the number kept (int64 [1]) and float64 [2] = squared norm of the
        dequantised matrix before, squared change kept.  All three stay on the device."""
        need = B.pvt_trust_workspace_bytes(self.desc, k_max)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.W.device)
            B.pvt_workspace_init(self._ws)
        idx = torch.empty(k_max, dtype=torch.int32, device=self.W.device)
        n = torch.zeros(1, dtype=torch.int64, device=self.W.device)
        stats = torch.zeros(2, dtype=torch.float64, device=self.W.device)
        B.pvt_vstep_trust(self.desc, k_max, ratio, idx, n, stats, self._ws)
        return idx, n, stats

    def status(self) -> int:
        return B.pvt_status(self.reserve(1))
