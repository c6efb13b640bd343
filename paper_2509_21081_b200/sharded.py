"""A decode step whose context is sharded over several GPUs (one process per GPU).

Two shardings, both with a single exchange after the attention itself:

* by sequence: rank r holds a contiguous slice of the shared prefix (prepared as its own handle) and
  the suffix pages of the requests it owns; every rank attends its tokens for all requests and heads
  (``typhoon_mla_decode_partial``: fp32 partial + LSE), the partials are all-gathered (B*H*129 floats
  per rank) and merged by ``typhoon_mla_combine_partials`` (the LSE combine of Algorithm 1 line 8);
* by head: rank r holds H / G heads (weights, queries and the expanded prefix sliced by head, latent
  caches replicated), runs the ordinary step on them and the bf16 outputs are all-gathered along the
  head axis.

The planning functions are pure host logic.  The exchange goes through a small ``Comm`` object:
``TorchDistComm`` wraps ``torch.distributed`` (NCCL on GPUs); a test can drive several ranks' decoders
in one process and stack their partials itself.  Marshalling only: every step of the attention runs
in the CUDA library.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch

from . import binding as _b

TILE = 64   # prefix slices start on a multiple of the expanded cache's 64-token block


def sequence_slices(Ls: int, world: int, align: int = TILE) -> List[Tuple[int, int]]:
    """Contiguous [begin, end) slices of a prefix of Ls tokens, one per rank: equal numbers of
    ``align``-token blocks (the first Ls_blocks % world ranks get one more), the ragged tail in the
    last non-empty slice.  Slices may be empty when there are fewer blocks than ranks."""
    if Ls < 0 or world < 1 or align < 1:
        raise ValueError("invalid arguments")
    blocks = -(-Ls // align)
    per, rem = divmod(blocks, world)
    out, b0 = [], 0
    for r in range(world):
        nb = per + (1 if r < rem else 0)
        out.append((min(b0 * align, Ls), min((b0 + nb) * align, Ls)))
        b0 += nb
    return out


def request_owner(b: int, world: int) -> int:
    """Rank that holds the suffix pages of request b (round robin)."""
    return b % world


def local_seq_lens(seq_lens: torch.Tensor, rank: int, world: int) -> torch.Tensor:
    """seq_lens with the entries of requests owned by other ranks set to 0."""
    idx = torch.arange(seq_lens.shape[0], device=seq_lens.device)
    return torch.where(idx % world == rank, seq_lens, torch.zeros_like(seq_lens))


def head_slice(H: int, rank: int, world: int) -> Tuple[int, int]:
    """Heads [h0, h1) of rank `rank`; H / world must be a multiple of 16 (the library's head granularity)."""
    if world < 1 or H % world or (H // world) % 16:
        raise ValueError("H / world must be a multiple of 16")
    per = H // world
    return rank * per, (rank + 1) * per


class TorchDistComm:
    """All-gather over a ``torch.distributed`` process group (NCCL for CUDA tensors, gloo for CPU)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        """[...] on every rank -> [world, ...], rank order."""
        t = t.contiguous()
        out = torch.empty((self.world,) + tuple(t.shape), dtype=t.dtype, device=t.device)
        self._dist.all_gather(list(out.unbind(0)), t, group=self.group)
        return out


class SequenceShardedDecoder:
    """Rank `rank` of `world`: its slice of the shared prefix plus the suffixes of the requests it owns."""

    def __init__(self, rank: int, world: int, num_heads: int, ckv_shared: torch.Tensor, kpe_shared: torch.Tensor,
                 w_uk: torch.Tensor, w_uv: torch.Tensor, softmax_scale: float, max_batch: int, max_pages: int,
                 page_size: int = 64, comm=None):
        self.rank, self.world, self.comm = int(rank), int(world), comm
        self.begin, self.end = sequence_slices(ckv_shared.shape[0], world)[rank]
        self.dims = _b.make_dims(num_heads)
        self.scale, self.page_size = float(softmax_scale), int(page_size)
        self.w_uk, self.w_uv = w_uk.contiguous(), w_uv.contiguous()
        self.shared = _b.typhoon_mla_prepare_shared(self.dims, ckv_shared[self.begin:self.end].contiguous(),
                                                    kpe_shared[self.begin:self.end].contiguous(), self.w_uk, self.w_uv)
        nbytes = _b.typhoon_mla_workspace_bytes(self.shared, int(max_batch), int(max_pages), self.page_size)
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")

    def partial(self, q_nope, q_pe, ckv_pages, kpe_pages, block_table, seq_lens, mode: int = _b.MODE_AUTO):
        """(o fp32 [B, H, 128], lse fp32 [B, H]) over this rank's tokens.  `seq_lens` are the full
        suffix lengths; the entries of requests this rank does not own are zeroed here."""
        B, H = q_nope.shape[0], q_nope.shape[1]
        o = torch.empty(B, H, 128, dtype=torch.float32, device="cuda")
        lse = torch.empty(B, H, dtype=torch.float32, device="cuda")
        lens = None if seq_lens is None else local_seq_lens(seq_lens, self.rank, self.world)
        _b.typhoon_mla_decode_partial(self.shared, q_nope, q_pe, ckv_pages, kpe_pages, self.page_size, block_table,
                                      lens, self.scale, o, lse, self.workspace, mode=mode)
        return o, lse

    def decode(self, q_nope, q_pe, ckv_pages, kpe_pages, block_table, seq_lens, mode: int = _b.MODE_AUTO,
               lse_out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """The full result on every rank: partial, all-gather, combine."""
        if self.comm is None:
            raise RuntimeError("no communicator: use partial() and merge_partials()")
        o, lse = self.partial(q_nope, q_pe, ckv_pages, kpe_pages, block_table, seq_lens, mode)
        return merge_partials(self.comm.all_gather(o), self.comm.all_gather(lse), lse_out)

    def close(self):
        self.shared.free()


def merge_partials(o_parts: torch.Tensor, lse_parts: torch.Tensor, lse_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """o_parts fp32 [n, B, H, 128], lse_parts fp32 [n, B, H] -> bf16 [B, H, 128]."""
    n, B, H = lse_parts.shape
    out = torch.empty(B, H, 128, dtype=torch.bfloat16, device=o_parts.device)
    _b.typhoon_mla_combine_partials(o_parts.contiguous(), lse_parts.contiguous(), out, lse_out)
    return out


class HeadShardedDecoder:
    """Rank `rank` of `world`: heads [h0, h1) of every request; latent caches replicated."""

    def __init__(self, rank: int, world: int, num_heads: int, ckv_shared: torch.Tensor, kpe_shared: torch.Tensor,
                 w_uk: torch.Tensor, w_uv: torch.Tensor, softmax_scale: float, max_batch: int, max_pages: int,
                 page_size: int = 64, comm=None):
        self.rank, self.world, self.comm = int(rank), int(world), comm
        self.h0, self.h1 = head_slice(num_heads, rank, world)
        self.dims = _b.make_dims(self.h1 - self.h0)
        self.scale, self.page_size = float(softmax_scale), int(page_size)
        self.w_uk, self.w_uv = w_uk[self.h0:self.h1].contiguous(), w_uv[self.h0:self.h1].contiguous()
        self.shared = _b.typhoon_mla_prepare_shared(self.dims, ckv_shared, kpe_shared, self.w_uk, self.w_uv)
        nbytes = _b.typhoon_mla_workspace_bytes(self.shared, int(max_batch), int(max_pages), self.page_size)
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")

    def local(self, q_nope, q_pe, ckv_pages, kpe_pages, block_table, seq_lens, mode: int = _b.MODE_AUTO) -> torch.Tensor:
        """bf16 [B, H / world, 128]: this rank's heads of the result (queries given for all H heads)."""
        qn = q_nope[:, self.h0:self.h1].contiguous()
        qp = q_pe[:, self.h0:self.h1].contiguous()
        out = torch.empty(qn.shape[0], self.h1 - self.h0, 128, dtype=torch.bfloat16, device="cuda")
        _b.typhoon_mla_decode(self.shared, qn, qp, ckv_pages, kpe_pages, self.page_size, block_table, seq_lens,
                              self.scale, out, self.workspace, mode=mode)
        return out

    def decode(self, q_nope, q_pe, ckv_pages, kpe_pages, block_table, seq_lens, mode: int = _b.MODE_AUTO) -> torch.Tensor:
        if self.comm is None:
            raise RuntimeError("no communicator: use local() and join_heads()")
        return join_heads(self.comm.all_gather(self.local(q_nope, q_pe, ckv_pages, kpe_pages, block_table, seq_lens, mode)))

    def close(self):
        self.shared.free()


def join_heads(parts: torch.Tensor) -> torch.Tensor:
    """[world, B, H / world, 128] in rank order -> [B, H, 128]."""
    G, B, Hl, D = parts.shape
    return parts.permute(1, 0, 2, 3).reshape(B, G * Hl, D)
