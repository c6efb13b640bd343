"""Convenience wrapper: prepared prefix + workspace + one call per decode step.

Marshalling only; every step of the path runs in the CUDA library.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as _b


class TyphoonMLADecoder:
    """Holds the expanded shared prefix and a workspace for batches up to ``max_batch``."""

    def __init__(self, num_heads: int, ckv_shared: torch.Tensor, kpe_shared: torch.Tensor,
                 w_uk: torch.Tensor, w_uv: torch.Tensor, softmax_scale: float,
                 max_batch: int, max_pages: int, page_size: int = 64, fp8_shared: bool = False):
        for t in (ckv_shared, kpe_shared, w_uk, w_uv):
            if not t.is_cuda or t.dtype != torch.bfloat16:
                raise ValueError("all tensors must be bf16 CUDA tensors")
        self.dims = _b.make_dims(num_heads)
        self.scale = float(softmax_scale)
        self.page_size = int(page_size)
        self.max_batch, self.max_pages = int(max_batch), int(max_pages)
        self.w_uk, self.w_uv = w_uk.contiguous(), w_uv.contiguous()
        prepare = _b.typhoon_mla_prepare_shared_fp8 if fp8_shared else _b.typhoon_mla_prepare_shared
        self.shared = prepare(self.dims, ckv_shared, kpe_shared, self.w_uk, self.w_uv)
        nbytes = _b.typhoon_mla_workspace_bytes(self.shared, self.max_batch, self.max_pages, self.page_size)
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        sbytes = _b.typhoon_mla_host_staging_bytes(self.shared, self.max_batch, self.max_pages)
        self.staging = torch.empty(max(sbytes, 256), dtype=torch.uint8, device="cuda")

    def decode(self, q_nope, q_pe, ckv_pages, kpe_pages, block_table, seq_lens,
               mode: int = _b.MODE_AUTO, out: Optional[torch.Tensor] = None,
               lse_out: Optional[torch.Tensor] = None) -> torch.Tensor:
        B, H = q_nope.shape[0], q_nope.shape[1]
        if B > self.max_batch or (block_table is not None and block_table.shape[1] > self.max_pages):
            raise ValueError("batch or page table larger than the decoder was sized for")
        if out is None:
            out = torch.empty(B, H, 128, dtype=torch.bfloat16, device="cuda")
        _b.typhoon_mla_decode(self.shared, q_nope, q_pe, ckv_pages, kpe_pages, self.page_size, block_table,
                              seq_lens, self.scale, out, self.workspace, mode=mode, lse_out=lse_out)
        return out

    def decode_host(self, q_nope_host, q_pe_host, ckv_pages, kpe_pages, block_table_host, seq_lens_host,
                    out_host, mode: int = _b.MODE_AUTO) -> None:
        """Per-step tensors in (pinned) host memory; result copied back to ``out_host``.
        Asynchronous on the current stream."""
        _b.typhoon_mla_decode_host(self.shared, q_nope_host, q_pe_host, ckv_pages, kpe_pages, self.page_size,
                                   block_table_host, seq_lens_host, self.scale, out_host, self.staging,
                                   self.workspace, mode=mode)

    def choose_mode(self, B: int, total_suffix_tokens: int = -1) -> int:
        return _b.typhoon_mla_choose_mode(self.shared, B, total_suffix_tokens)

    def close(self):
        self.shared.free()
