"""GPU parity of the 8-bit (E4M3) expanded shared-prefix cache: the stored codes against the checker's encoder, and the
decode step against the checker's operator over the decoded values.  The kernel widens the codes exactly and then
computes as the 16-bit path does, so the bars are the 16-bit path's (max-abs 2e-2, relative Frobenius 5e-3, LSE 2e-2);
what the encoding itself costs is measured against the unencoded definition and reported, not asserted tightly."""
import numpy as np
import pytest
import torch

from oracle import fp8_oracle as F
from oracle import mla_oracle as O
from paper_2509_21081_b200 import inputs as I
from tests import gpu_harness as G

pytestmark = pytest.mark.gpu

ABSORB, HYBRID, AUTO, NAIVE = 1, 2, 0, 3


def _cfg(name, B, H, Ls, lo, hi, seed, page_size=64):
    return I.MLAConfig(name, B=B, H=H, Ls=Ls, suffix_lo=lo, suffix_hi=hi, seed=seed, page_size=page_size)


@pytest.mark.parametrize("H,Ls", [(16, 200), (32, 777)])
def test_codes_and_scales_match_the_encoder(H, Ls):
    """Every stored code equals the checker's, except where the 16-bit expansion itself (fp32 accumulation on the GPU,
    exact in the checker) rounds to a neighbouring bfloat16: there the two codes must be adjacent, and such places must
    be rare.  Scales are equal exactly; padding tokens hold code 0."""
    from paper_2509_21081_b200 import binding as b
    inp = I.make_inputs(_cfg("codes", B=1, H=H, Ls=Ls, lo=0, hi=0, seed=77))
    dims = b.make_dims(H)
    w_uk, w_uv = inp.w_uk.cuda(), inp.w_uv.cuda()
    sh = b.typhoon_mla_prepare_shared_fp8(dims, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), w_uk, w_uv)
    kc, vc, sc = b.typhoon_mla_shared_export_fp8(sh)
    assert b.typhoon_mla_check_status(sh) == 0
    kc, vc, sc = kc.cpu().numpy(), vc.cpu().numpy(), sc.cpu().double().numpy()
    Lp = kc.shape[1]
    assert Lp % 128 == 0 and Lp >= Ls
    f = I.to_f64
    table = F.e4m3_decode_table()
    n_diff = 0
    for h in range(H):
        K = O.decompress_head(f(inp.ckv_shared), f(inp.w_uk)[h])          # [Ls, 128]
        V = O.decompress_head(f(inp.ckv_shared), f(inp.w_uv)[h])
        ck, sk = F.encode_head(K)
        cv, sv = F.encode_head(V)
        assert sc[0, h] == sk and sc[1, h] == sv
        got_k = kc[h, :Ls]                                                  # [Ls, 128]
        got_v = vc[h].transpose(0, 2, 1).reshape(Lp, 128)[:Ls]              # blocks [128 dims, 64 tok] -> [tok, dim]
        for got, want in ((got_k, ck), (got_v, cv)):
            d = got != want
            n_diff += int(d.sum())
            if d.any():   # neighbours in value: same sign (or a zero), magnitude codes one apart
                g, w = got[d].astype(int), want[d].astype(int)
                assert np.all(np.abs((g & 0x7F) - (w & 0x7F)) <= 1)
                assert np.all(((g ^ w) & 0x80 == 0) | ((g & 0x7F) + (w & 0x7F) <= 1))
        assert not kc[h, Ls:].any() and not vc[h].transpose(0, 2, 1).reshape(Lp, 128)[Ls:].any()
    assert n_diff <= 2e-3 * 2 * H * Ls * 128, n_diff
    sh.free()


@pytest.mark.parametrize("B,H,Ls,hi", [(4, 16, 256, 64), (9, 16, 331, 300), (64, 128, 520, 100), (37, 48, 1000, 70),
                                       (70, 64, 520, 90), (130, 16, 700, 50), (200, 32, 450, 0)])
@pytest.mark.parametrize("mode", [HYBRID, NAIVE])
def test_decode_matches_the_checker_over_decoded_values(B, H, Ls, hi, mode):
    """One and several 64-request row groups, ragged prefixes, several head counts; HYBRID and (no suffix) NAIVE."""
    cfg = _cfg("fp8", B=B, H=H, Ls=Ls, lo=0, hi=hi, seed=300 + B)
    inp = I.make_inputs(cfg)
    drop = mode == NAIVE
    ref, ref_lse = G.run_oracle_fp8(inp, drop_suffix=drop)
    out, lse, launches = G.run_gpu(inp, mode, fp8_shared=True, force_max_pages=0 if drop else None)
    assert launches > 0
    G.assert_parity(out, ref, lse, ref_lse, what=f"fp8 B={B} H={H} Ls={Ls} mode={mode}")
    # what the encoding costs against the unencoded definition: well above the kernel's own error, far below 1
    plain, _ = G.run_oracle(inp, drop_suffix=drop)
    _, rel = G.errors(ref, plain)
    assert 1e-3 < rel < 0.1, rel


@pytest.mark.parametrize("schedule", [1, 2])
def test_work_decompositions(schedule):
    from paper_2509_21081_b200 import binding as b
    b.typhoon_mla_set_naive_schedule(schedule)
    try:
        inp = I.make_inputs(_cfg("fp8s", B=100, H=32, Ls=1500, lo=0, hi=40, seed=311))
        ref, ref_lse = G.run_oracle_fp8(inp)
        out, lse, _ = G.run_gpu(inp, HYBRID, fp8_shared=True)
        G.assert_parity(out, ref, lse, ref_lse, what=f"fp8 schedule {schedule}")
    finally:
        b.typhoon_mla_set_naive_schedule(0)


def test_absorb_mode_and_empty_prefix_do_not_touch_the_codes():
    """ABSORB mode attends over the 16-bit latent copy of the prefix: the plain definition is the expected value.
    An empty prefix has nothing to encode."""
    inp = I.make_inputs(_cfg("fp8a", B=5, H=32, Ls=400, lo=1, hi=200, seed=312))
    ref, ref_lse = G.run_oracle(inp)
    out, lse, _ = G.run_gpu(inp, ABSORB, fp8_shared=True)
    G.assert_parity(out, ref, lse, ref_lse, what="fp8 handle, ABSORB")
    inp = I.make_inputs(_cfg("fp8e", B=3, H=16, Ls=0, lo=5, hi=100, seed=313))
    ref, ref_lse = G.run_oracle(inp)
    out, lse, _ = G.run_gpu(inp, HYBRID, fp8_shared=True)
    G.assert_parity(out, ref, lse, ref_lse, what="fp8 handle, no prefix")


def test_footprint_is_halved_and_other_paths_refuse():
    from paper_2509_21081_b200 import binding as b
    inp = I.make_inputs(_cfg("fp8f", B=2, H=16, Ls=1024, lo=0, hi=10, seed=314))
    dims = b.make_dims(16)
    args = (dims, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda())
    s16 = b.typhoon_mla_prepare_shared(*args)
    s8 = b.typhoon_mla_prepare_shared_fp8(*args)
    _, Lp, own16 = b.typhoon_mla_shared_view(s16)
    _, _, own8 = b.typhoon_mla_shared_view(s8)
    expanded16 = 2 * 16 * Lp * 128 * 2
    assert own16 - own8 == expanded16 // 2 - 16 * 3 * 4      # codes are half the bytes; plus the per-head scales
    with pytest.raises(b.TyphoonMLAError):
        b.typhoon_mla_shared_export(s8)
    with pytest.raises(b.TyphoonMLAError):
        b.typhoon_mla_shared_export_fp8(s16)
    # the warp-MMA cross-check kernels have no 8-bit path: refused, nothing launched
    pc = I.build_pages(inp)
    ws = torch.empty(b.typhoon_mla_workspace_bytes(s8, 2, pc.block_table.shape[1], 64), dtype=torch.uint8, device="cuda")
    out = torch.zeros(2, 16, 128, dtype=torch.bfloat16, device="cuda")
    b.typhoon_mla_set_kernel_path(b.PATH_WARP_MMA)
    try:
        with pytest.raises(b.TyphoonMLAError):
            b.typhoon_mla_decode(s8, inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), 64,
                                 pc.block_table.cuda(), pc.seq_lens.cuda(), inp.scale, out, ws, mode=HYBRID)
    finally:
        b.typhoon_mla_set_kernel_path(b.PATH_TCGEN05)
    torch.cuda.synchronize()
    assert not out.any()
    s16.free()
    s8.free()


def test_tree_with_an_8bit_root_and_16bit_branches():
    """Several shared prefixes per step, the root stored in 8 bits, the per-group prefixes in 16: the checker encodes
    the root only (the branches are part of each request's own context there)."""
    from paper_2509_21081_b200 import binding as b
    from tests.test_gpu_parity import _tree_problem
    B, H = 11, 32
    lens = [0, 3, 64, 65, 130, 7, 200, 1, 90, 64, 30]
    rows, inp, br = _tree_problem(B, H, 210, [(0, 150), (3, 0), (5, 333), (9, 70)], lens, seed=39)
    ref, ref_lse = G.run_oracle_fp8(rows)
    dev = "cuda"
    w_uk, w_uv = inp.w_uk.to(dev), inp.w_uv.to(dev)
    dims = b.make_dims(H)
    root = b.typhoon_mla_prepare_shared_fp8(dims, inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), w_uk, w_uv)
    handles = [root]
    prefixes = []
    for _, _, c, r in br:
        if c.shape[0] > 0:
            handles.append(b.typhoon_mla_prepare_shared(dims, c.to(dev), r.to(dev), w_uk, w_uv))
            prefixes.append(handles[-1])
        else:
            prefixes.append(None)
    levels = [([root], [0, B]), (prefixes, [b0 for b0, _, _, _ in br] + [B])]
    pc = I.build_pages(inp)
    ws = torch.empty(b.typhoon_mla_tree_workspace_bytes(levels, B, pc.block_table.shape[1], 64), dtype=torch.uint8, device=dev)
    out = torch.empty(B, H, 128, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(B, H, dtype=torch.float32, device=dev)
    b.typhoon_mla_decode_tree(levels, inp.q_nope.to(dev), inp.q_pe.to(dev), pc.ckv_pages.to(dev), pc.kpe_pages.to(dev), 64,
                              pc.block_table.to(dev), pc.seq_lens.to(dev), inp.scale, out, ws, lse_out=lse)
    for h in handles:
        assert b.typhoon_mla_check_status(h) == 0
    G.assert_parity(out.float().cpu().double().numpy(), ref, lse.cpu().double().numpy(), ref_lse, what="tree, 8-bit root")
    for h in handles:
        h.free()


@pytest.mark.parametrize("name,batch", [("cfg1", 0), ("cfg4", 512)])
def test_full_size_configurations(name, batch):
    """The benchmark's headline configuration (64-row instance, one tile range per head) and the fan-out sweep at
    B = 512 (128-row instance, four row groups, equal tile ranges over all SMs) on an 8-bit handle, in the launch
    configuration the benchmark times: all heads of at least 16 requests against the checker's operator."""
    from tests.test_gpu_parity import _checked_requests
    cfg = I.CONFIGS[name].with_batch(batch) if batch else I.CONFIGS[name]
    inp = I.make_inputs(cfg)
    reqs = _checked_requests(cfg, inp)
    reqs = sorted(set(reqs) | {r for g0 in range(0, cfg.B, 128) for r in (g0, min(g0 + 127, cfg.B - 1))})   # every 128-row group
    pairs = [(r, h) for r in reqs for h in range(cfg.H)]
    ref, ref_lse = G.run_oracle_fp8(inp, pairs=pairs)
    mask = ~np.isnan(ref_lse)
    assert mask.sum() == len(reqs) * cfg.H
    out, lse, _ = G.run_gpu(inp, HYBRID, fp8_shared=True)
    assert np.isfinite(out).all()
    G.assert_parity(out, ref, lse, ref_lse, mask=mask, what=f"fp8 {cfg.name} full size")


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes(seed):
    """Seeded random sizes, head counts, page sizes and work decompositions on an 8-bit handle (ring wrap-around with the
    staging and operand rings, several segments per CTA, odd tile counts, partial row groups)."""
    import random
    from paper_2509_21081_b200 import binding as b
    rnd = random.Random(7000 + seed)
    H = rnd.choice([16, 32, 48, 64, 128])
    B = rnd.choice([rnd.randint(1, 8), rnd.randint(9, 64), rnd.randint(65, 128), rnd.randint(129, 300)])
    Ls = rnd.choice([rnd.randint(1, 200), rnd.randint(200, 1500), rnd.randint(1500, 2600) if H <= 32 else rnd.randint(64, 900)])
    hi = rnd.choice([0, 5, 70, 200])
    page_size = rnd.choice([64, 128])
    b.typhoon_mla_set_naive_schedule(rnd.choice([0, 1, 2]))
    try:
        inp = I.make_inputs(_cfg("fp8rand", B=B, H=H, Ls=Ls, lo=0, hi=hi, seed=900 + seed, page_size=page_size))
        ref, ref_lse = G.run_oracle_fp8(inp)
        out, lse, _ = G.run_gpu(inp, HYBRID, page_size=page_size, fp8_shared=True)
        G.assert_parity(out, ref, lse, ref_lse, what=f"fp8 random {seed}: B={B} H={H} Ls={Ls} hi={hi} ps={page_size}")
    finally:
        b.typhoon_mla_set_naive_schedule(0)
