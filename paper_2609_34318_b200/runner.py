"""Owns the device buffers of one attention problem and runs forward -> merge -> backward.

No arithmetic happens here: the class allocates torch CUDA tensors (device memory only), keeps the
pair list, and calls hydra_attn_fwd / hydra_lse_merge / hydra_attn_bwd on the current stream.
"""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as B


def bits_to_tensor(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on the device (a reinterpretation)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def tensor_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class AttnStep:
    def __init__(self, cu_seqlens, n_heads: int, pairs=None, part_rows: int = 0, causal: bool = True,
                 softmax_scale: Optional[float] = None, device="cuda"):
        self.cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
        self.h = int(n_heads)
        self.T = int(self.cu[-1])
        self.pairs = B.as_pairs(pairs)
        self.part_rows = int(part_rows)
        self.causal = bool(causal)
        self.scale = float(np.float32(1.0 / np.sqrt(np.float32(B.D_QK)))) if softmax_scale is None \
            else float(softmax_scale)
        dev = torch.device(device)
        bf, f32 = torch.bfloat16, torch.float32
        T, h = max(self.T, 1), self.h
        self.out = torch.empty((T, h, B.D_V), dtype=bf, device=dev)
        self.lse = torch.empty((h, T), dtype=f32, device=dev)
        self.o_part = torch.empty((max(self.part_rows, 1), h, B.D_V), dtype=bf, device=dev)
        self.lse_part = torch.empty((h, max(self.part_rows, 1)), dtype=f32, device=dev)
        self.dq = torch.empty((T, h, B.D_QK), dtype=bf, device=dev)
        self.dk = torch.empty((T, h, B.D_QK), dtype=bf, device=dev)
        self.dv = torch.empty((T, h, B.D_V), dtype=bf, device=dev)
        ws = max(B.hydra_workspace_bytes(w, self.cu, h, self.pairs)
                 for w in (B.HYDRA_WS_FWD, B.HYDRA_WS_MERGE, B.HYDRA_WS_BWD))
        self.workspace = torch.zeros(ws, dtype=torch.uint8, device=dev)    # status reads OK before the first launch
        self.has_partials = self.pairs is not None and bool((self.pairs["part_row"] >= 0).any())

    def forward(self, q, k, v, stream=None):
        B.hydra_attn_fwd(q, k, v, self.cu, self.h, self.pairs, self.causal, self.scale, self.out, self.lse,
                         self.o_part if self.has_partials else None,
                         self.lse_part if self.has_partials else None, self.part_rows, self.workspace,
                         stream=stream)
        if self.has_partials:
            B.hydra_lse_merge(self.o_part, self.lse_part, self.part_rows, self.cu, self.h, self.pairs,
                              self.out, self.lse, self.workspace, stream=stream)
        return self.out, self.lse

    def backward(self, q, k, v, dout, stream=None):
        B.hydra_attn_bwd(q, k, v, self.out, self.lse, dout, self.cu, self.h, self.pairs, self.causal,
                         self.scale, self.dq, self.dk, self.dv, self.workspace, stream=stream)
        return self.dq, self.dk, self.dv

    def poll(self, stream=None):
        return B.hydra_poll_status(self.workspace, stream)
