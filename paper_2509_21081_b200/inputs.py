"""Seeded synthetic inputs for MLA decode with a shared prefix.

This module only *draws* data and lays it out (dense per-request arrays for a
checker, a paged latent cache for the library).  It holds none of the method's
arithmetic: no attention, no projection, no softmax.  Both the CPU checker's
tests and the GPU tests/bench import it so that the two sides see identical
bits.

Recipe (all values bf16, rounded to nearest even from fp32 normal draws):

* ``ckv_shared [Ls, D_l]``, ``kpe_shared [Ls, D_r]``: N(0, 1)
* ``w_uk [H, D_n, D_l]``, ``w_uv [H, D_v, D_l]``: N(0, 1/D_l) (variance), i.e.
  fp32 ``randn * D_l**-0.5``
* suffix lengths: ``randint(lo, hi+1)`` (inclusive) from the global generator
* per request ``b`` (its own generator, so a smaller batch is a prefix of a
  larger one): ``q_nope [H, D_n]``, ``q_pe [H, D_r]``, ``ckv_suffix [Ln_b, D_l]``,
  ``kpe_suffix [Ln_b, D_r]``: N(0, 1)
* softmax scale ``(D_n + D_r) ** -0.5``
* pages: ``page_size`` tokens; physical page ids are a seeded permutation of
  ``sum_b ceil(Ln_b / page_size)`` pages plus ``spare_pages`` never-referenced
  ones; unused block-table slots are -1; token slots past a request's length in
  its last page and all spare pages hold NaN when ``poison`` is set.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import torch


@dataclass(frozen=True)
class MLAConfig:
    name: str
    B: int
    H: int
    Ls: int
    suffix_lo: int
    suffix_hi: int
    seed: int
    d_nope: int = 128
    d_rope: int = 64
    d_v: int = 128
    d_l: int = 512
    page_size: int = 64

    @property
    def scale(self) -> float:
        return float((self.d_nope + self.d_rope) ** -0.5)

    def with_batch(self, B: int) -> "MLAConfig":
        return replace(self, B=B, name=f"{self.name}_B{B}")


# The five benchmark configurations (config 4 is a batch sweep: use with_batch).
CONFIGS: Dict[str, MLAConfig] = {
    "cfg0": MLAConfig("cfg0", B=4, H=16, Ls=256, suffix_lo=64, suffix_hi=64, seed=0),
    "cfg1": MLAConfig("cfg1", B=64, H=128, Ls=4096, suffix_lo=512, suffix_hi=512, seed=1),
    "cfg2": MLAConfig("cfg2", B=128, H=128, Ls=26624, suffix_lo=256, suffix_hi=2048, seed=2),
    "cfg3": MLAConfig("cfg3", B=256, H=64, Ls=8192, suffix_lo=128, suffix_hi=4096, seed=3),
    "cfg4": MLAConfig("cfg4", B=128, H=128, Ls=16384, suffix_lo=256, suffix_hi=256, seed=4),
}
CFG4_BATCHES = (1, 8, 32, 128, 512, 1024)


@dataclass
class MLAInputs:
    cfg: MLAConfig
    q_nope: torch.Tensor            # bf16 [B, H, D_n]
    q_pe: torch.Tensor              # bf16 [B, H, D_r]
    ckv_shared: torch.Tensor        # bf16 [Ls, D_l]
    kpe_shared: torch.Tensor        # bf16 [Ls, D_r]
    suffix_lens: List[int]
    ckv_suffix: List[torch.Tensor]  # per request bf16 [Ln_b, D_l]
    kpe_suffix: List[torch.Tensor]  # per request bf16 [Ln_b, D_r]
    w_uk: torch.Tensor              # bf16 [H, D_n, D_l]
    w_uv: torch.Tensor              # bf16 [H, D_v, D_l]
    scale: float
    extra: dict = field(default_factory=dict)


def _randn_bf16(gen: torch.Generator, *shape: int, mul: float = 1.0) -> torch.Tensor:
    x = torch.randn(*shape, generator=gen, dtype=torch.float32)
    if mul != 1.0:
        x = x * mul
    return x.to(torch.bfloat16)


def _request_generator(seed: int, b: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 1_000_003 + 7919 * (b + 1))
    return g


def make_inputs(cfg: MLAConfig, suffix_lens: Optional[List[int]] = None) -> MLAInputs:
    """Draw one problem instance for ``cfg`` (CPU tensors)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.seed)
    ckv_shared = _randn_bf16(g, cfg.Ls, cfg.d_l)
    kpe_shared = _randn_bf16(g, cfg.Ls, cfg.d_rope)
    w_uk = _randn_bf16(g, cfg.H, cfg.d_nope, cfg.d_l, mul=cfg.d_l ** -0.5)
    w_uv = _randn_bf16(g, cfg.H, cfg.d_v, cfg.d_l, mul=cfg.d_l ** -0.5)
    # always draw a fixed-size pool of lengths so that a batch prefix keeps them
    pool = max(cfg.B, 1024)
    drawn = torch.randint(cfg.suffix_lo, cfg.suffix_hi + 1, (pool,), generator=g).tolist()
    if suffix_lens is None:
        suffix_lens = [int(x) for x in drawn[: cfg.B]]
    assert len(suffix_lens) == cfg.B
    q_nope = torch.empty(cfg.B, cfg.H, cfg.d_nope, dtype=torch.bfloat16)
    q_pe = torch.empty(cfg.B, cfg.H, cfg.d_rope, dtype=torch.bfloat16)
    ckv_suffix, kpe_suffix = [], []
    for b in range(cfg.B):
        gb = _request_generator(cfg.seed, b)
        q_nope[b] = _randn_bf16(gb, cfg.H, cfg.d_nope)
        q_pe[b] = _randn_bf16(gb, cfg.H, cfg.d_rope)
        ckv_suffix.append(_randn_bf16(gb, suffix_lens[b], cfg.d_l))
        kpe_suffix.append(_randn_bf16(gb, suffix_lens[b], cfg.d_rope))
    return MLAInputs(cfg, q_nope, q_pe, ckv_shared, kpe_shared, list(suffix_lens),
                     ckv_suffix, kpe_suffix, w_uk, w_uv, cfg.scale)


@dataclass
class PagedCache:
    ckv_pages: torch.Tensor    # bf16 [P, page_size, D_l]
    kpe_pages: torch.Tensor    # bf16 [P, page_size, D_r]
    block_table: torch.Tensor  # int32 [B, max_pages]
    seq_lens: torch.Tensor     # int32 [B]
    page_size: int


def build_pages(inp: MLAInputs, page_size: Optional[int] = None, seed: int = 12345,
                poison: bool = True, spare_pages: int = 2,
                min_max_pages: int = 0) -> PagedCache:
    """Scatter the dense per-request suffixes into a paged latent cache."""
    cfg = inp.cfg
    ps = page_size or cfg.page_size
    need = [(n + ps - 1) // ps for n in inp.suffix_lens]
    total = sum(need)
    P = total + spare_pages
    max_pages = max(max(need) if need else 0, min_max_pages)
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    perm = torch.randperm(P, generator=g).tolist()
    fill = float("nan") if poison else 0.0
    ckv_pages = torch.full((max(P, 1), ps, cfg.d_l), fill, dtype=torch.bfloat16)
    kpe_pages = torch.full((max(P, 1), ps, cfg.d_rope), fill, dtype=torch.bfloat16)
    block_table = torch.full((cfg.B, max(max_pages, 1)), -1, dtype=torch.int32)
    nxt = 0
    for b in range(cfg.B):
        n = inp.suffix_lens[b]
        for j in range(need[b]):
            pid = perm[nxt]
            nxt += 1
            block_table[b, j] = pid
            lo, hi = j * ps, min((j + 1) * ps, n)
            ckv_pages[pid, : hi - lo] = inp.ckv_suffix[b][lo:hi]
            kpe_pages[pid, : hi - lo] = inp.kpe_suffix[b][lo:hi]
    seq_lens = torch.tensor(inp.suffix_lens, dtype=torch.int32)
    return PagedCache(ckv_pages, kpe_pages, block_table, seq_lens, ps)


def to_f64(t: torch.Tensor):
    """Exact widening of a bf16/fp32 CPU tensor to a float64 numpy array."""
    return t.to(torch.float64).numpy()
