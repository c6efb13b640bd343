"""Pins of the float64 CPU checker to things other than itself.

Each test is chosen so that a plausible slip in oracle/mla_oracle.py (dropped
rope term, wrong scale placement, transposed up-projection, softmax over the
wrong axis, wrong -inf handling in the merge) fails at least one of them.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import mla_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _tiny(seed=0, B=2, H=3, Ls=5, Ln=(3, 6), Dn=4, Dr=2, Dv=3, Dl=5):
    r = np.random.default_rng(seed)
    d = dict(
        q_nope=r.standard_normal((B, H, Dn)), q_pe=r.standard_normal((B, H, Dr)),
        ckv_shared=r.standard_normal((Ls, Dl)), kpe_shared=r.standard_normal((Ls, Dr)),
        ckv_suffix=[r.standard_normal((n, Dl)) for n in Ln],
        kpe_suffix=[r.standard_normal((n, Dr)) for n in Ln],
        w_uk=r.standard_normal((H, Dn, Dl)), w_uv=r.standard_normal((H, Dv, Dl)),
        scale=0.37,
    )
    return d


def _call(d, **kw):
    return O.mla_decode(d["q_nope"], d["q_pe"], d["ckv_shared"], d["kpe_shared"],
                        d["ckv_suffix"], d["kpe_suffix"], d["w_uk"], d["w_uv"], d["scale"], **kw)


# ---------------------------------------------------------------- brute force
def _brute(d):
    """Pure-Python loops, math.exp, no numpy arithmetic."""
    B = len(d["q_nope"]); H = len(d["q_nope"][0])
    Dn = len(d["q_nope"][0][0]); Dr = len(d["q_pe"][0][0])
    Dv = len(d["w_uv"][0]); Dl = len(d["w_uv"][0][0])
    out = [[[0.0] * Dv for _ in range(H)] for _ in range(B)]
    lse = [[0.0] * H for _ in range(B)]
    for b in range(B):
        toks_c = [list(map(float, row)) for row in d["ckv_shared"]] + \
                 [list(map(float, row)) for row in d["ckv_suffix"][b]]
        toks_r = [list(map(float, row)) for row in d["kpe_shared"]] + \
                 [list(map(float, row)) for row in d["kpe_suffix"][b]]
        for h in range(H):
            logits, vals = [], []
            for c, r in zip(toks_c, toks_r):
                k = [sum(float(d["w_uk"][h][i][j]) * c[j] for j in range(Dl)) for i in range(Dn)]
                v = [sum(float(d["w_uv"][h][i][j]) * c[j] for j in range(Dl)) for i in range(Dv)]
                s = sum(float(d["q_nope"][b][h][i]) * k[i] for i in range(Dn))
                s += sum(float(d["q_pe"][b][h][i]) * r[i] for i in range(Dr))
                logits.append(d["scale"] * s)
                vals.append(v)
            z = sum(math.exp(s) for s in logits)
            lse[b][h] = math.log(z)
            for i in range(Dv):
                out[b][h][i] = sum(math.exp(s) / z * v[i] for s, v in zip(logits, vals))
    return np.array(out), np.array(lse)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_brute_force(seed):
    d = _tiny(seed)
    out, lse = _call(d)
    bo, bl = _brute(d)
    assert np.max(np.abs(out - bo)) < 1e-13
    assert np.max(np.abs(lse - bl)) < 1e-13


# ------------------------------------------------ library routine (MHA == MLA)
def test_against_torch_sdpa():
    """After decompression MLA is standard multi-head attention
    (Section 2.1, "Naive"): compare with torch's CPU SDPA in float64."""
    d = _tiny(3, B=3, H=4, Ls=17, Ln=(9, 9, 9), Dn=8, Dr=4, Dv=6, Dl=10)
    out, _ = _call(d)
    for b in range(3):
        C = np.concatenate([d["ckv_shared"], d["ckv_suffix"][b]])
        R = np.concatenate([d["kpe_shared"], d["kpe_suffix"][b]])
        K = np.stack([np.concatenate([C @ d["w_uk"][h].T, R], axis=1) for h in range(4)])   # [H, L, Dn+Dr]
        V = np.stack([C @ d["w_uv"][h].T for h in range(4)])                                # [H, L, Dv]
        Q = np.concatenate([d["q_nope"][b], d["q_pe"][b]], axis=1)[:, None, :]             # [H, 1, Dqk]
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
            scale=d["scale"])[0, :, 0, :].numpy()
        assert np.max(np.abs(out[b] - ref)) < 1e-12


def test_identity_projection_is_multi_query_attention():
    """W_UK = W_UV = [I 0] makes every head attend over the raw latent."""
    d = _tiny(4, B=1, H=2, Ls=6, Ln=(5,), Dn=4, Dr=2, Dv=4, Dl=7)
    eye = np.zeros((4, 7)); eye[:4, :4] = np.eye(4)
    d["w_uk"] = np.stack([eye, eye]); d["w_uv"] = np.stack([eye, eye])
    out, _ = _call(d)
    C = np.concatenate([d["ckv_shared"], d["ckv_suffix"][0]])
    R = np.concatenate([d["kpe_shared"], d["kpe_suffix"][0]])
    for h in range(2):
        s = d["scale"] * (C[:, :4] @ d["q_nope"][0, h] + R @ d["q_pe"][0, h])
        p = np.exp(s) / np.exp(s).sum()
        assert np.max(np.abs(out[0, h] - p @ C[:, :4])) < 1e-13


# --------------------------------------------------- naive == absorb identity
def _absorb_form(d):
    """Algorithm 1 lines 5-7 applied to the whole context: the query is moved
    through W_UK into latent space, attention runs over latents, and the latent
    output is projected through W_UV."""
    B, H, _ = d["q_nope"].shape
    out = np.zeros((B, H, d["w_uv"].shape[1])); lse = np.zeros((B, H))
    for b in range(B):
        C = np.concatenate([d["ckv_shared"], d["ckv_suffix"][b]])
        R = np.concatenate([d["kpe_shared"], d["kpe_suffix"][b]])
        for h in range(H):
            qa = d["q_nope"][b, h] @ d["w_uk"][h]                 # [D_l]
            s = d["scale"] * (C @ qa + R @ d["q_pe"][b, h])
            m = s.max(); p = np.exp(s - m); z = p.sum()
            o_lat = (p / z) @ C
            out[b, h] = d["w_uv"][h] @ o_lat
            lse[b, h] = m + np.log(z)
    return out, lse


def test_naive_equals_absorb():
    d = _tiny(5, B=2, H=3, Ls=11, Ln=(4, 7), Dn=6, Dr=3, Dv=5, Dl=9)
    out, lse = _call(d)
    ao, al = _absorb_form(d)
    assert np.max(np.abs(out - ao)) < 1e-12
    assert np.max(np.abs(lse - al)) < 1e-12


# ------------------------------------------------------------------ LSE merge
def test_lse_merge_every_split_point():
    d = _tiny(6, B=1, H=2, Ls=0, Ln=(9,), Dn=4, Dr=2, Dv=3, Dl=5)
    d["ckv_shared"] = np.zeros((0, 5)); d["kpe_shared"] = np.zeros((0, 2))
    full, full_lse = _call(d)
    C, R = d["ckv_suffix"][0], d["kpe_suffix"][0]
    for k in range(0, 10):
        da = dict(d, ckv_suffix=[C[:k]], kpe_suffix=[R[:k]])
        db = dict(d, ckv_suffix=[C[k:]], kpe_suffix=[R[k:]])
        oa, la = _call(da); ob, lb = _call(db)
        for h in range(2):
            o, l = O.combine_lse([oa[0, h], ob[0, h]], [la[0, h], lb[0, h]])
            assert np.max(np.abs(o - full[0, h])) < 1e-12
            assert abs(l - full_lse[0, h]) < 1e-12


def test_lse_merge_prefix_suffix_and_three_way():
    d = _tiny(7)
    full, full_lse = _call(d)
    # shared prefix only / suffix only, merged (this is the hybrid method's split)
    dp = dict(d, ckv_suffix=[x[:0] for x in d["ckv_suffix"]], kpe_suffix=[x[:0] for x in d["kpe_suffix"]])
    ds = dict(d, ckv_shared=d["ckv_shared"][:0], kpe_shared=d["kpe_shared"][:0])
    op, lp = _call(dp); os_, ls = _call(ds)
    for b in range(2):
        for h in range(3):
            o, l = O.combine_lse([op[b, h], os_[b, h]], [lp[b, h], ls[b, h]])
            assert np.max(np.abs(o - full[b, h])) < 1e-12 and abs(l - full_lse[b, h]) < 1e-12
            # three-way with an empty partial in the middle
            o3, l3 = O.combine_lse([op[b, h], np.zeros(3), os_[b, h]], [lp[b, h], -math.inf, ls[b, h]])
            assert np.max(np.abs(o3 - full[b, h])) < 1e-12 and abs(l3 - full_lse[b, h]) < 1e-12


def test_combine_all_empty():
    o, l = O.combine_lse([np.zeros(3), np.zeros(3)], [-math.inf, -math.inf])
    assert np.all(o == 0) and l == -math.inf


def test_combine_two_way_closed_form():
    o1, o2 = np.array([1.0, 0.0]), np.array([0.0, 1.0])
    o, l = O.combine_lse([o1, o2], [math.log(3.0), math.log(1.0)])
    assert np.allclose(o, [0.75, 0.25], atol=1e-15) and abs(l - math.log(4.0)) < 1e-15


# ------------------------------------------------------------- weights / forms
def test_weights_row_stochastic():
    r = np.random.default_rng(8)
    for n in (1, 2, 50, 1000):
        s = r.standard_normal(n) * 5
        p, lse = O.attention_weights(s)
        assert np.all(p >= 0) and abs(p.sum() - 1.0) < 1e-14
        assert abs(lse - math.log(sum(math.exp(x) for x in s))) < 1e-12


def test_empty_context():
    d = _tiny(9, B=1, H=2, Ls=0, Ln=(0,))
    d["ckv_shared"] = np.zeros((0, 5)); d["kpe_shared"] = np.zeros((0, 2))
    out, lse = _call(d)
    assert np.all(out == 0) and np.all(lse == -math.inf)


def test_closed_forms():
    d = _tiny(10, B=2, H=3, Ls=7, Ln=(2, 5))
    # zero query -> uniform weights -> W_UV * mean latent, lse = ln L
    dz = dict(d, q_nope=np.zeros_like(d["q_nope"]), q_pe=np.zeros_like(d["q_pe"]))
    out, lse = _call(dz)
    for b in range(2):
        C = np.concatenate([d["ckv_shared"], d["ckv_suffix"][b]])
        for h in range(3):
            assert np.max(np.abs(out[b, h] - d["w_uv"][h] @ C.mean(0))) < 1e-13
            assert abs(lse[b, h] - math.log(C.shape[0])) < 1e-13
    # zero scale -> same uniform result with any query
    out0, _ = _call(dict(d, scale=0.0))
    assert np.max(np.abs(out0 - out)) < 1e-13
    # one token in total -> its value, whatever the query
    d1 = dict(d, ckv_shared=d["ckv_shared"][:1], kpe_shared=d["kpe_shared"][:1],
              ckv_suffix=[x[:0] for x in d["ckv_suffix"]], kpe_suffix=[x[:0] for x in d["kpe_suffix"]])
    out1, _ = _call(d1)
    for h in range(3):
        assert np.max(np.abs(out1[0, h] - d["w_uv"][h] @ d["ckv_shared"][0])) < 1e-13
    # all tokens identical -> that token's value
    c0, r0 = d["ckv_shared"][0], d["kpe_shared"][0]
    di = dict(d, ckv_shared=np.tile(c0, (7, 1)), kpe_shared=np.tile(r0, (7, 1)),
              ckv_suffix=[np.tile(c0, (2, 1)), np.tile(c0, (5, 1))],
              kpe_suffix=[np.tile(r0, (2, 1)), np.tile(r0, (5, 1))])
    outi, _ = _call(di)
    for h in range(3):
        assert np.max(np.abs(outi[1, h] - d["w_uv"][h] @ c0)) < 1e-12


def test_dominant_token():
    """One token 40 logits above the rest: output is its value up to L*e^-40.
    The dominant token sits in the suffix, so a dropped suffix fails here."""
    d = _tiny(11, B=1, H=1, Ls=6, Ln=(4,), Dn=4, Dr=2, Dv=3, Dl=6)
    d["w_uk"][0] = 0.0
    d["q_nope"][:] = 0.0                      # logits come from the rope part only
    d["q_pe"][0, 0] = [1.0, 0.0]
    d["kpe_shared"][:] = 0.0
    d["kpe_suffix"][0][:] = 0.0
    d["kpe_suffix"][0][2] = [40.0 / d["scale"], 123.0]
    out, lse = _call(d)
    v = d["w_uv"][0] @ d["ckv_suffix"][0][2]
    assert np.max(np.abs(out[0, 0] - v)) < 10 * math.exp(-40) * 10
    assert abs(lse[0, 0] - 40.0) < 1e-12


def test_rope_term_and_scale_placement():
    """The scale multiplies nope + rope logits together: doubling scale equals
    doubling both query parts."""
    d = _tiny(12)
    a, la = _call(dict(d, scale=2 * d["scale"]))
    b_, lb = _call(dict(d, q_nope=2 * d["q_nope"], q_pe=2 * d["q_pe"]))
    assert np.max(np.abs(a - b_)) < 1e-12 and np.max(np.abs(la - lb)) < 1e-12
    # the rope term matters
    c, _ = _call(dict(d, q_pe=np.zeros_like(d["q_pe"])))
    assert np.max(np.abs(c - _call(d)[0])) > 1e-3


def test_token_permutation_and_prefix_move_invariance():
    d = _tiny(13, B=2, H=2, Ls=8, Ln=(5, 3))
    base, base_l = _call(d)
    perm = np.random.default_rng(0).permutation(8)
    dp = dict(d, ckv_shared=d["ckv_shared"][perm], kpe_shared=d["kpe_shared"][perm])
    o, l = _call(dp)
    assert np.max(np.abs(o - base)) < 1e-13
    # move the last 3 shared tokens to the front of every suffix: same context
    dm = dict(d, ckv_shared=d["ckv_shared"][:5], kpe_shared=d["kpe_shared"][:5],
              ckv_suffix=[np.concatenate([d["ckv_shared"][5:], x]) for x in d["ckv_suffix"]],
              kpe_suffix=[np.concatenate([d["kpe_shared"][5:], x]) for x in d["kpe_suffix"]])
    o, l = _call(dm)
    assert np.max(np.abs(o - base)) < 1e-13 and np.max(np.abs(l - base_l)) < 1e-13


def test_pairs_subset_matches_full():
    d = _tiny(14)
    full, fl = _call(d)
    sub, sl = _call(d, pairs=[(1, 2), (0, 0)])
    assert np.array_equal(sub[1, 2], full[1, 2]) and np.array_equal(sub[0, 0], full[0, 0])
    assert np.isnan(sub[0, 1]).all() and sl[1, 2] == fl[1, 2]


def test_expand_shared_is_plain_matmul():
    r = np.random.default_rng(15)
    c = r.standard_normal((6, 5)); w = r.standard_normal((3, 4, 5))
    e = O.expand_shared(c, w)
    assert e.shape == (3, 6, 4)
    assert np.max(np.abs(e - np.einsum("tl,hdl->htd", c, w))) < 1e-14


# ------------------------------------------------------- cost model and Eq. 1
def test_eq1_printed_value():
    g = json.load(open(os.path.join(GOLD, "eq1_batch_threshold.json")))
    bt = O.batch_threshold(g["D_qk"], g["D_v"], g["D_l"], g["D_r"], g["S_q"], g["T"], g["M"])
    assert int(bt) == g["B_theta_printed"] and abs(bt - 61.44) < 0.01
    # S_q divides the threshold
    assert abs(O.batch_threshold(192, 128, 512, 64, 4, g["T"], g["M"]) - bt / 4) < 1e-12


def test_table1_printed_constants():
    g = json.load(open(os.path.join(GOLD, "table1_constants.json")))
    dm = g["dims"]
    kw = dict(H=dm["H"], D_qk=dm["D_qk"], D_v=dm["D_v"], D_l=dm["D_l"], D_r=dm["D_r"])
    B, Ls, Ln = 7, 1000, 300
    n = O.macs("naive", B, 1, Ls, Ln, **kw); a = O.macs("absorb", B, 1, Ls, Ln, **kw)
    t = O.macs("typhoon", B, 1, Ls, Ln, **kw)
    assert n == 40 * 1024 * B * (Ls + Ln) and a == 136 * 1024 * B * (Ls + Ln)
    assert t == 40 * 1024 * B * Ls + 136 * 1024 * B * Ln
    hn = O.hbm_words("naive", B, Ls, Ln, **kw); ha = O.hbm_words("absorb", B, Ls, Ln, **kw)
    ht = O.hbm_words("typhoon", B, Ls, Ln, **kw)
    assert hn == 40 * 1024 * (Ls + B * Ln)
    assert ha == int(0.5625 * 1024) * (Ls + B * Ln)
    assert ht == 40 * 1024 * Ls + 576 * B * Ln
    assert round(136 / 40, 1) == g["ratio_mac_absorb_over_naive_printed"]
    assert abs(40 * 1024 / 576 - g["ratio_hbm_naive_over_absorb_printed"]) < 1.5
    assert round(0.5625, 2) == g["hbm_per_token_x1024"]["absorb_printed"]
    # S_q scales MACs linearly
    assert O.macs("typhoon", B, 3, Ls, Ln, **kw) == 3 * t


def test_fig4_ratio_matches_mac_ratio():
    g = json.load(open(os.path.join(GOLD, "fig4_stage_ratio.json")))
    r = (g["baseline_ms"] - g["absorb_part_ms"]) / g["naive_part_ms"]
    assert round(r, 1) == g["ratio_printed"]
    kw = dict(H=64, D_qk=192, D_v=128, D_l=512, D_r=64)
    mr = O.macs("absorb", 1024, 1, 4096, 0, **kw) / O.macs("naive", 1024, 1, 4096, 0, **kw)
    assert abs(mr - r) < 0.15
