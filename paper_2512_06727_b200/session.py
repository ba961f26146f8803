"""Torch-side plumbing around a kvcar Context: device buffers and dtype helpers.
No arithmetic of the method happens here."""
from __future__ import annotations

from typing import Dict, Optional, Tuple

import numpy as np
import torch

from . import binding as B


def torch_dtype(storage: int):
    return torch.float32 if storage == B.F32 else torch.bfloat16


def storage_code(name: str) -> int:
    return {"f32": B.F32, "bf16": B.BF16}[name]


class Session:
    """Owns the three device buffers of one context and keeps them alive."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, page_tokens: int,
                 max_seqs: int, max_pages: int, max_pages_per_seq: int, storage: str,
                 src_k=None, src_v=None, autoencoders: Optional[Dict[Tuple[int, int], dict]] = None,
                 device: str = "cuda:0", kernel: int = B.KERNEL_AUTO, latent_quant: bool = False):
        self.storage = storage_code(storage)
        self.dtype = torch_dtype(self.storage)
        self.device = torch.device(device)
        self.ctx = B.Context(n_layers, n_q_heads, n_kv_heads, head_dim, page_tokens, max_seqs, max_pages,
                             max_pages_per_seq, self.storage, int(latent_quant))
        self.latent_quant = bool(latent_quant)
        if src_k is not None:
            self.ctx.set_reuse_map(src_k, src_v)
        for (layer, which), ae in (autoencoders or {}).items():
            self.ctx.set_autoencoder(layer, which, ae)
        nb = self.ctx.required_bytes()
        self.sizes = nb
        with torch.cuda.device(self.device):
            self.pool = torch.zeros(nb[0] + 256, dtype=torch.uint8, device=self.device)
            self.weights = torch.zeros(nb[1] + 256, dtype=torch.uint8, device=self.device)
            self.workspace = torch.zeros(nb[2] + 256, dtype=torch.uint8, device=self.device)
            torch.cuda.synchronize()
            self.ctx.bind_memory(self._aligned(self.pool), nb[0], self._aligned(self.weights), nb[1],
                                 self._aligned(self.workspace), nb[2], torch.cuda.current_stream().cuda_stream)
        if kernel != B.KERNEL_AUTO:
            self.ctx.set_kernel(kernel)

    @staticmethod
    def _aligned(t: torch.Tensor) -> int:
        return (t.data_ptr() + 255) // 256 * 256

    def stream(self) -> int:
        return torch.cuda.current_stream().cuda_stream

    def pool_rows(self, layer: int, which: int) -> torch.Tensor:
        """View of one layer's K or V cache rows [max_pages*page_tokens, width]."""
        off, pitch, width = self.ctx.pool_layout(layer, which)
        rows = self.ctx.cfg.max_pages * self.ctx.cfg.page_tokens
        base = self._aligned(self.pool) - self.pool.data_ptr() + off
        raw = self.pool[base:base + rows * pitch]
        if pitch == width and self.latent_quant:   # int8 codes (Eq. 4)
            return raw.view(torch.int8).view(rows, width)
        return raw.view(self.dtype).view(rows, width)

    def pool_quant_params(self, layer: int, which: int) -> torch.Tensor:
        """View of one layer's per-row (scale, zero-point) pairs [max_pages*page_tokens, 2] (int8 latent rows)."""
        rows = self.ctx.cfg.max_pages * self.ctx.cfg.page_tokens
        base = self._aligned(self.pool) - self.pool.data_ptr() + self.ctx.pool_quant_layout(layer, which)
        return self.pool[base:base + rows * 8].view(torch.float32).view(rows, 2)

    def to_device(self, x: np.ndarray) -> torch.Tensor:
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(self.device).to(self.dtype).contiguous()
