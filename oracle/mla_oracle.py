"""Float64 CPU checker for MLA decode attention with a shared prefix.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
CUDA library is compared against.  It is imported by the tests, by the smoke
check and by the benchmark's CPU-baseline leg, never by the library or its
Python binding, and it shares no code with them.

What it computes is the *definition* of Multi-Head Latent Attention in its
naive form (paper Section 2.1, "Naive"; Fig. 1a): every cached token's latent
vector is decompressed through the KV up-projection into a per-head key and
value, and standard softmax attention is taken per (request, head) over the
whole context at once.  The hybrid method (Algorithm 1) is stated by the paper
to be mathematically equal to this (Section 3.1, last sentence of "Decode"),
so the definition is the expected value.  No absorption, no prefix/suffix
split of the softmax, no online softmax, no paging.

Readings of points the paper leaves open (the same list is in the design
notes): the up-projection is given as two matrices W_UK = W_KVb1 [H, D_n, D_l]
and W_UV = W_KVb2 [H, D_v, D_l] (Algorithm 1, Require); q_pe and cached rope
keys arrive already rotated, so no RoPE is applied here; the softmax scale
multiplies the sum of the nope and rope logits; the log-sum-exp is the natural
log of the sum of exp(scaled logits); an empty context gives a zero output row
and lse = -inf; a single decode query attends to every cached token (no mask).

Pins (tests/test_oracle_pins.py): brute-force pure-Python loops on tiny
inputs; torch's CPU scaled_dot_product_attention after decompression; the
naive == absorb algebraic identity; LSE merge of any prefix/suffix split ==
single pass; row-stochastic weights; closed forms (zero query, one token,
identical tokens, dominant token, zero scale); Eq. 1 -> 61 and the Table 1
constants for the cost-model helpers.
"""
from __future__ import annotations

import math
from typing import Iterable, List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------
# Decompression (Section 2.1 "Naive": K and V are the up-projected latents)
# --------------------------------------------------------------------------
def decompress_head(ckv: np.ndarray, w_h: np.ndarray) -> np.ndarray:
    """[L, D_l] latents times one head's up-projection [D, D_l] -> [L, D]."""
    return ckv @ w_h.T


def expand_shared(ckv_shared: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Prefill-side expansion of the shared latent cache (Section 3.1 "Prefill").

    ckv_shared [Ls, D_l], w [H, D, D_l]  ->  [H, Ls, D]  (K_nope or V per head).
    """
    return np.stack([decompress_head(ckv_shared, w[h]) for h in range(w.shape[0])])


# --------------------------------------------------------------------------
# Softmax attention for one (request, head): the definition
# --------------------------------------------------------------------------
def attention_weights(s: np.ndarray) -> Tuple[np.ndarray, float]:
    """softmax(s) over a 1-D logit vector and ln(sum(exp(s)))."""
    if s.shape[0] == 0:
        return s.copy(), -math.inf
    m = float(np.max(s))
    p = np.exp(s - m)
    z = float(np.sum(p))
    return p / z, m + math.log(z)


def attend(q_nope_bh: np.ndarray, q_pe_bh: np.ndarray, K_nope: np.ndarray, R: np.ndarray,
           V: np.ndarray, scale: float) -> Tuple[np.ndarray, float]:
    """One query vector against L decompressed tokens.

    K_nope [L, D_n], R [L, D_r] (rope keys, shared by all heads), V [L, D_v].
    Returns (out [D_v], lse).  The key of a token is the concatenation
    [K_nope, R], the query is [q_nope, q_pe] (Algorithm 1, lines 1-4).
    """
    s = scale * (K_nope @ q_nope_bh + R @ q_pe_bh)
    p, lse = attention_weights(s)
    if s.shape[0] == 0:
        return np.zeros(V.shape[1], dtype=np.float64), lse
    return p @ V, lse


# --------------------------------------------------------------------------
# The whole operator
# --------------------------------------------------------------------------
def mla_decode(q_nope: np.ndarray, q_pe: np.ndarray,
               ckv_shared: np.ndarray, kpe_shared: np.ndarray,
               ckv_suffix: Sequence[np.ndarray], kpe_suffix: Sequence[np.ndarray],
               w_uk: np.ndarray, w_uv: np.ndarray, scale: float,
               pairs: Optional[Iterable[Tuple[int, int]]] = None):
    """MLA decode attention from the definition, float64.

    q_nope [B, H, D_n], q_pe [B, H, D_r]; shared latents [Ls, D_l] and rope keys
    [Ls, D_r] common to all requests; per-request suffix latents [Ln_b, D_l] and
    rope keys [Ln_b, D_r]; w_uk [H, D_n, D_l], w_uv [H, D_v, D_l].

    Returns (out [B, H, D_v], lse [B, H]).  With ``pairs`` given, only those
    (b, h) entries are computed and the rest of ``out``/``lse`` is NaN.

    The decompressed key/value of a token depends on the token and the head
    only, so the shared prefix is decompressed once per head and reused for
    every request; the softmax of each (b, h) still runs once over that
    request's whole context.
    """
    B, H, _ = q_nope.shape
    D_v = w_uv.shape[1]
    out = np.full((B, H, D_v), np.nan, dtype=np.float64)
    lse = np.full((B, H), np.nan, dtype=np.float64)
    if pairs is None:
        by_head = {h: list(range(B)) for h in range(H)}
    else:
        by_head = {}
        for b, h in pairs:
            by_head.setdefault(int(h), []).append(int(b))
    for h, bs in sorted(by_head.items()):
        Ks = decompress_head(ckv_shared, w_uk[h])
        Vs = decompress_head(ckv_shared, w_uv[h])
        for b in bs:
            Kn = decompress_head(ckv_suffix[b], w_uk[h])
            Vn = decompress_head(ckv_suffix[b], w_uv[h])
            K = np.concatenate([Ks, Kn], axis=0)
            V = np.concatenate([Vs, Vn], axis=0)
            R = np.concatenate([kpe_shared, kpe_suffix[b]], axis=0)
            out[b, h], lse[b, h] = attend(q_nope[b, h], q_pe[b, h], K, R, V, scale)
    return out, lse


# --------------------------------------------------------------------------
# Combine of normalised partial results by their log-sum-exps
# (Algorithm 1 line 8; Section 3.2 "CombineLSE")
# --------------------------------------------------------------------------
def combine_lse(outs: Sequence[np.ndarray], lses: Sequence[float]) -> Tuple[np.ndarray, float]:
    """Merge partial attention results over disjoint token sets.

    Each partial i is softmax-normalised over its own tokens with
    lse_i = ln sum exp(logits_i).  The merged result weighs partial i by
    exp(lse_i) / sum_j exp(lse_j).  Partials over no tokens carry lse = -inf
    and weight zero; if all are empty the result is zero with lse = -inf.
    """
    m = max(lses)
    if m == -math.inf:
        return np.zeros_like(outs[0], dtype=np.float64), -math.inf
    w = [math.exp(l - m) if l != -math.inf else 0.0 for l in lses]
    z = sum(w)
    acc = np.zeros_like(outs[0], dtype=np.float64)
    for wi, oi in zip(w, outs):
        if wi != 0.0:
            acc = acc + wi * oi
    return acc / z, m + math.log(z)


# --------------------------------------------------------------------------
# Cost model (Table 1) and batch threshold (Eq. 1)
# --------------------------------------------------------------------------
def macs(kind: str, B: int, S_q: int, L_s: int, L_n: int, H: int,
         D_qk: int, D_v: int, D_l: int, D_r: int) -> int:
    """Multiply-accumulates of the attention part (Table 1, upper half)."""
    naive_w = H * (D_qk + D_v)
    absorb_w = H * (2 * D_l + D_r)
    if kind == "naive":
        return B * S_q * L_s * naive_w + B * S_q * L_n * naive_w
    if kind == "absorb":
        return B * S_q * L_s * absorb_w + B * S_q * L_n * absorb_w
    if kind == "typhoon":
        return B * S_q * L_s * naive_w + B * S_q * L_n * absorb_w
    raise ValueError(kind)


def hbm_words(kind: str, B: int, L_s: int, L_n: int, H: int,
              D_qk: int, D_v: int, D_l: int, D_r: int) -> int:
    """Words read from HBM by the attention part (Table 1, lower half)."""
    naive_w = H * (D_qk + D_v)
    absorb_w = D_l + D_r
    if kind == "naive":
        return L_s * naive_w + B * L_n * naive_w
    if kind == "absorb":
        return L_s * absorb_w + B * L_n * absorb_w
    if kind == "typhoon":
        return L_s * naive_w + B * L_n * absorb_w
    raise ValueError(kind)


def batch_threshold(D_qk: int, D_v: int, D_l: int, D_r: int, S_q: int,
                    T: float, M: float) -> float:
    """Eq. 1: batch size at which reading the expanded shared cache (naive)
    takes as long as computing over it in absorb form.  The paper inserts T in
    operations/s (two per MAC) and M in bytes/s (two per 16-bit word); the two
    factors of two cancel, so MAC/s over words/s gives the same number."""
    return (D_qk + D_v) / (S_q * (2 * D_l + D_r)) * (T / M)
