"""GPU parity: the CUDA library (through the C ABI) against the float64 CPU
checker on the same seeded inputs.  Bars (bf16 inputs, fp32 accumulation):
max-abs <= 2e-2 and relative Frobenius <= 5e-3 on the output, 2e-2 on the LSE.
"""
import math

import numpy as np
import pytest
import torch

from paper_2509_21081_b200 import inputs as I
from tests import gpu_harness as G

pytestmark = pytest.mark.gpu

ABSORB, HYBRID, AUTO, NAIVE = 1, 2, 0, 3


@pytest.fixture(autouse=True, params=["tcgen05", "warp_mma"])
def kernel_path(request):
    """Every test runs on both implementations of the tensor-core kernels."""
    from paper_2509_21081_b200 import binding as b
    b.typhoon_mla_set_kernel_path(b.PATH_TCGEN05 if request.param == "tcgen05" else b.PATH_WARP_MMA)
    yield request.param
    b.typhoon_mla_set_kernel_path(b.PATH_TCGEN05)


@pytest.fixture
def naive_schedule():
    """Selects the work decomposition of the shared-prefix kernel for one test."""
    from paper_2509_21081_b200 import binding as b
    yield lambda name: b.typhoon_mla_set_naive_schedule({"auto": 0, "split": 1, "streamk": 2}[name])
    b.typhoon_mla_set_naive_schedule(0)


def _cfg(name, B, H, Ls, lo, hi, seed, page_size=64):
    return I.MLAConfig(name, B=B, H=H, Ls=Ls, suffix_lo=lo, suffix_hi=hi, seed=seed, page_size=page_size)


@pytest.mark.parametrize("mode", [HYBRID, ABSORB, AUTO])
def test_cfg0_tiny(mode):
    inp = I.make_inputs(I.CONFIGS["cfg0"])
    ref, ref_lse = G.run_oracle(inp)
    out, lse, launches = G.run_gpu(inp, mode)
    assert launches > 0
    G.assert_parity(out, ref, lse, ref_lse, what=f"cfg0 mode {mode}")


@pytest.mark.parametrize("mode", [HYBRID, ABSORB])
@pytest.mark.parametrize("page_size", [64, 128])
def test_ragged_small(mode, page_size):
    """Ragged prefix (not a tile multiple), ragged suffixes with empty / one-token / page-edge lengths,
    NaN-poisoned page tails and spare pages, -1 in unused block-table slots."""
    cfg = _cfg("ragged", B=9, H=16, Ls=331, lo=0, hi=0, seed=21, page_size=page_size)
    inp = I.make_inputs(cfg, suffix_lens=[0, 1, 63, 64, 65, 127, 129, 300, 777])
    ref, ref_lse = G.run_oracle(inp)
    out, lse, _ = G.run_gpu(inp, mode, page_size=page_size)
    G.assert_parity(out, ref, lse, ref_lse, what=f"ragged mode {mode} ps {page_size}")


@pytest.mark.parametrize("H", [16, 48, 64, 128])
def test_head_counts_and_batch_tail(H):
    """B not a multiple of the row tile; several head counts (incl. a ragged head group)."""
    cfg = _cfg("heads", B=70 if H <= 64 else 37, H=H, Ls=520, lo=40, hi=200, seed=22 + H)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp)
    for mode in (HYBRID, ABSORB):
        out, lse, _ = G.run_gpu(inp, mode)
        G.assert_parity(out, ref, lse, ref_lse, what=f"H={H} mode {mode}")


@pytest.mark.parametrize("schedule", ["split", "streamk"])
@pytest.mark.parametrize("B,H,Ls", [(70, 64, 520), (5, 32, 1000), (150, 16, 1100), (300, 16, 700), (400, 32, 450)])
def test_naive_schedules(schedule, B, H, Ls, naive_schedule):
    """Both work decompositions of the shared-prefix kernel (every tile range inside one head; equal
    ranges that cross heads), for 64- and 128-token tiles, one and two query-row groups, a last
    row group with and without a second row tile."""
    naive_schedule(schedule)
    cfg = _cfg("sched", B=B, H=H, Ls=Ls, lo=0, hi=90, seed=40 + B)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp)
    out, lse, _ = G.run_gpu(inp, HYBRID)
    G.assert_parity(out, ref, lse, ref_lse, what=f"schedule {schedule} B={B} H={H} Ls={Ls}")


@pytest.mark.parametrize("seed", range(10))
def test_random_shapes(seed, naive_schedule):
    """Seeded random problem sizes, modes, page sizes and work decompositions: pipeline phase logic
    (ring wrap-around, segments per CTA, odd tile counts, partial row groups) against the checker."""
    import random
    rnd = random.Random(1000 + seed)
    H = rnd.choice([16, 32, 48, 64, 128])
    B = rnd.choice([rnd.randint(1, 8), rnd.randint(9, 128), rnd.randint(129, 300)])
    Ls = rnd.choice([rnd.randint(1, 200), rnd.randint(200, 1500), rnd.randint(1500, 2600) if H <= 32 else rnd.randint(64, 900)])
    hi = rnd.choice([0, 5, 70, 200])
    page_size = rnd.choice([64, 128])
    mode = rnd.choice([HYBRID, HYBRID, ABSORB, AUTO])
    naive_schedule(rnd.choice(["split", "streamk", "auto"]))
    cfg = _cfg("rand", B=B, H=H, Ls=Ls, lo=0, hi=hi, seed=500 + seed, page_size=page_size)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp)
    out, lse, _ = G.run_gpu(inp, mode, page_size=page_size)
    G.assert_parity(out, ref, lse, ref_lse, what=f"random {seed}: B={B} H={H} Ls={Ls} hi={hi} ps={page_size} mode={mode}")


def test_no_prefix():
    """Ls = 0: absorb path alone (Algorithm 1 lines 5-7)."""
    cfg = _cfg("noprefix", B=6, H=32, Ls=0, lo=1, hi=400, seed=23)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp)
    for mode in (HYBRID, ABSORB, AUTO):
        out, lse, _ = G.run_gpu(inp, mode)
        G.assert_parity(out, ref, lse, ref_lse, what=f"Ls=0 mode {mode}")


def test_no_suffix():
    """All suffixes empty: naive path alone (Algorithm 1 line 4) -- with a page table of zero
    lengths, with no page table at all, and in NAIVE mode."""
    cfg = _cfg("nosuffix", B=5, H=32, Ls=1000, lo=0, hi=0, seed=24)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp)
    out, lse, _ = G.run_gpu(inp, HYBRID, min_max_pages=3)
    G.assert_parity(out, ref, lse, ref_lse, what="Ln=0 hybrid")
    out, lse, _ = G.run_gpu(inp, AUTO, force_max_pages=0)
    G.assert_parity(out, ref, lse, ref_lse, what="Ln=0 auto, no page table")
    out, lse, _ = G.run_gpu(inp, NAIVE)
    G.assert_parity(out, ref, lse, ref_lse, what="Ln=0 naive")
    out, lse, _ = G.run_gpu(inp, ABSORB, min_max_pages=2)
    G.assert_parity(out, ref, lse, ref_lse, what="Ln=0 absorb")


def test_naive_mode_ignores_suffix():
    cfg = _cfg("naiveonly", B=4, H=16, Ls=300, lo=10, hi=90, seed=25)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp, drop_suffix=True)
    out, lse, _ = G.run_gpu(inp, NAIVE)
    G.assert_parity(out, ref, lse, ref_lse, what="naive mode")


def test_empty_context_rows():
    """No prefix and some empty suffixes: those rows are zero with lse = -inf, no NaN anywhere."""
    cfg = _cfg("empty", B=4, H=16, Ls=0, lo=0, hi=0, seed=26)
    inp = I.make_inputs(cfg, suffix_lens=[0, 5, 0, 70])
    ref, ref_lse = G.run_oracle(inp)
    out, lse, _ = G.run_gpu(inp, HYBRID)
    G.assert_parity(out, ref, lse, ref_lse, what="empty rows")
    assert np.all(out[0] == 0) and np.all(out[2] == 0) and np.all(np.isneginf(lse[0]))


@pytest.mark.parametrize("mult", [4.0, 8.0])
def test_peaked_softmax(mult):
    """Queries scaled up so that a few tokens dominate: sometimes in the prefix, sometimes in the
    suffix.  A mis-masked or dropped token shows here, where diffuse attention would hide it."""
    cfg = _cfg("peaked", B=8, H=16, Ls=700, lo=50, hi=600, seed=27)
    inp = I.make_inputs(cfg)
    inp.q_nope = (inp.q_nope.float() * mult).to(torch.bfloat16)
    inp.q_pe = (inp.q_pe.float() * mult).to(torch.bfloat16)
    ref, ref_lse = G.run_oracle(inp)
    for mode in (HYBRID, ABSORB):
        out, lse, _ = G.run_gpu(inp, mode)
        G.assert_parity(out, ref, lse, ref_lse, what=f"peaked x{mult} mode {mode}")


def test_dominant_token_in_suffix_and_prefix():
    """One token carries (almost) all the weight; output must be its decompressed value."""
    cfg = _cfg("dominant", B=2, H=16, Ls=200, lo=100, hi=100, seed=28)
    inp = I.make_inputs(cfg)
    inp.q_pe[:] = 0
    inp.q_pe[:, :, 0] = 8.0
    inp.kpe_shared[:] = 0
    for b in range(2):
        inp.kpe_suffix[b][:] = 0
    inp.kpe_suffix[0][77, 0] = 64.0      # request 0: winner in the suffix
    inp.kpe_shared[123, 0] = 0.0
    ref, ref_lse = G.run_oracle(inp)
    for mode in (HYBRID, ABSORB):
        out, lse, _ = G.run_gpu(inp, mode)
        G.assert_parity(out, ref, lse, ref_lse, what=f"dominant suffix mode {mode}")
    inp.kpe_suffix[0][77, 0] = 0.0
    inp.kpe_shared[123, 0] = 64.0        # both requests: winner in the prefix
    ref, ref_lse = G.run_oracle(inp)
    for mode in (HYBRID, ABSORB):
        out, lse, _ = G.run_gpu(inp, mode)
        G.assert_parity(out, ref, lse, ref_lse, what=f"dominant prefix mode {mode}")


def test_metamorphic_paging_and_modes():
    """Permuting physical pages, switching the page size and switching mode leave the result
    unchanged (within tolerance); repeating a call is bitwise identical."""
    cfg = _cfg("meta", B=6, H=32, Ls=450, lo=30, hi=500, seed=29)
    inp = I.make_inputs(cfg)
    ref, _ = G.run_oracle(inp)
    a, _, _ = G.run_gpu(inp, HYBRID, pages=I.build_pages(inp, 64, seed=1))
    b, _, _ = G.run_gpu(inp, HYBRID, pages=I.build_pages(inp, 64, seed=2))
    c, _, _ = G.run_gpu(inp, HYBRID, page_size=128, pages=I.build_pages(inp, 128, seed=3))
    d, _, _ = G.run_gpu(inp, ABSORB, pages=I.build_pages(inp, 64, seed=1))
    a2, _, _ = G.run_gpu(inp, HYBRID, pages=I.build_pages(inp, 64, seed=1))
    assert np.array_equal(a, a2), "run-to-run results differ bitwise"
    assert np.array_equal(a, b), "page permutation changed the result"
    for x, name in ((a, "a"), (c, "page128"), (d, "absorb")):
        G.assert_parity(x, ref, what=f"meta {name}")
    assert G.errors(d, a)[1] < G.REL_FRO_TOL


def test_moving_tokens_between_prefix_and_suffix():
    """The same total context split at a different point between shared prefix and suffixes."""
    cfg = _cfg("move", B=3, H=16, Ls=384, lo=64, hi=64, seed=30)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp)
    moved = I.make_inputs(cfg)
    k = 100
    moved.ckv_suffix = [torch.cat([inp.ckv_shared[-k:], x]) for x in inp.ckv_suffix]
    moved.kpe_suffix = [torch.cat([inp.kpe_shared[-k:], x]) for x in inp.kpe_suffix]
    moved.ckv_shared, moved.kpe_shared = inp.ckv_shared[:-k].contiguous(), inp.kpe_shared[:-k].contiguous()
    moved.suffix_lens = [n + k for n in inp.suffix_lens]
    out, lse, _ = G.run_gpu(moved, HYBRID)
    G.assert_parity(out, ref, lse, ref_lse, what="moved split")


def test_expansion_matches_plain_matmul():
    """Shared-prefix expansion against a float64 matmul: within one bf16 rounding of the exact value."""
    from oracle import mla_oracle as O
    from paper_2509_21081_b200 import binding as b
    cfg = _cfg("expand", B=1, H=16, Ls=333, lo=0, hi=0, seed=31)
    inp = I.make_inputs(cfg)
    dims = b.make_dims(cfg.H)
    w_uk, w_uv = inp.w_uk.cuda(), inp.w_uv.cuda()
    sh = b.typhoon_mla_prepare_shared(dims, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), w_uk, w_uv)
    assert b.typhoon_mla_check_status(sh) == 0
    k, vt = b.typhoon_mla_shared_export(sh)
    Ls, Lp, owned = b.typhoon_mla_shared_view(sh)
    torch.cuda.synchronize()
    assert (Ls, Lp) == (333, 384) and owned >= 2 * cfg.H * Lp * 128 * 2
    k = k.float().cpu().double().numpy().transpose(0, 1, 3, 2, 4).reshape(cfg.H, Lp, 128); v = vt.float().cpu().double().numpy().transpose(0, 1, 3, 2).reshape(cfg.H, Lp, 128)
    sh.free()
    kr = O.expand_shared(I.to_f64(inp.ckv_shared), I.to_f64(inp.w_uk))
    vr = O.expand_shared(I.to_f64(inp.ckv_shared), I.to_f64(inp.w_uv))
    for got, ref in ((k, kr), (v, vr)):
        assert np.all(got[:, 333:, :] == 0), "padding not zero"
        err = np.abs(got[:, :333, :] - ref)
        bound = np.abs(ref) * 2.0 ** -8 + 1e-6     # half-ulp of bf16 is 2^-9 relative; allow one ulp
        assert np.all(err <= bound), f"expansion error {err.max():.3e}"


def test_decode_host_matches_device_call():
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    cfg = _cfg("host", B=5, H=16, Ls=260, lo=10, hi=150, seed=32)
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp)
    dec = TyphoonMLADecoder(cfg.H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda(),
                            inp.scale, cfg.B, pc.block_table.shape[1])
    ckv_p, kpe_p = pc.ckv_pages.cuda(), pc.kpe_pages.cuda()
    ref = dec.decode(inp.q_nope.cuda(), inp.q_pe.cuda(), ckv_p, kpe_p, pc.block_table.cuda(), pc.seq_lens.cuda(),
                     mode=HYBRID).cpu()
    out_h = torch.empty(cfg.B, cfg.H, 128, dtype=torch.bfloat16).pin_memory()
    dec.decode_host(inp.q_nope.pin_memory(), inp.q_pe.pin_memory(), ckv_p, kpe_p, pc.block_table.pin_memory(),
                    pc.seq_lens.pin_memory(), out_h, mode=HYBRID)
    torch.cuda.synchronize()
    assert torch.equal(out_h, ref)
    dec.close()


def test_decode_captured_in_a_cuda_graph(kernel_path):
    """The decode call only enqueues kernels and event record/wait operations (on the given stream and
    on the handle's side stream), so it can be captured; replays see the buffers' current contents."""
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    cfg = _cfg("graph", B=7, H=32, Ls=300, lo=5, hi=200, seed=36)
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp, poison=False)
    dec = TyphoonMLADecoder(cfg.H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda(),
                            inp.scale, cfg.B, pc.block_table.shape[1])
    q_nope, q_pe = inp.q_nope.cuda(), inp.q_pe.cuda()
    args = (q_nope, q_pe, pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), pc.block_table.cuda(), pc.seq_lens.cuda())
    out = torch.empty(cfg.B, cfg.H, 128, dtype=torch.bfloat16, device="cuda")
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        dec.decode(*args, mode=HYBRID, out=out)      # an ordinary call first
        st.synchronize()
        direct = out.clone()
        with torch.cuda.graph(g, stream=st):
            dec.decode(*args, mode=HYBRID, out=out)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, direct)
    # new queries in the same buffers
    q_nope.copy_(torch.flip(q_nope, dims=[0]))
    q_pe.copy_(torch.flip(q_pe, dims=[0]))
    g.replay()
    torch.cuda.synchronize()
    replayed = out.clone()
    dec.decode(*args, mode=HYBRID, out=out)
    torch.cuda.synchronize()
    assert torch.equal(out, replayed) and not torch.equal(out, direct)
    assert b.typhoon_mla_check_status(dec.shared) == 0
    dec.close()


@pytest.mark.parametrize("S_q", [2, 3])
def test_several_query_tokens_per_request(S_q):
    """S_q query tokens per request (Table 1's S_q): rows = (request, query token) pairs sharing the
    request's pages, causal among the new tokens.  The checker sees each row as a request whose suffix is
    cut after its own token; one request is shorter than S_q (its first query sees the prefix only)."""
    import dataclasses
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    B, H = 6, 32
    cfg = _cfg("sq", B=B, H=H, Ls=300, lo=0, hi=0, seed=37)
    lens = [S_q - 1, 5, 64, 65, 130, 200]
    inp = I.make_inputs(cfg, suffix_lens=lens)
    pc = I.build_pages(inp)
    # queries of the B * S_q rows: a second draw with as many requests (same seed: same prefix and weights)
    rows = I.make_inputs(dataclasses.replace(cfg, B=B * S_q), suffix_lens=[0] * (B * S_q))
    row_lens = [max(lens[r // S_q] - (S_q - 1 - r % S_q), 0) for r in range(B * S_q)]
    rows.suffix_lens = row_lens
    rows.ckv_suffix = [inp.ckv_suffix[r // S_q][: row_lens[r]] for r in range(B * S_q)]
    rows.kpe_suffix = [inp.kpe_suffix[r // S_q][: row_lens[r]] for r in range(B * S_q)]
    assert torch.equal(rows.ckv_shared, inp.ckv_shared) and torch.equal(rows.w_uk, inp.w_uk)
    ref, ref_lse = G.run_oracle(rows)
    bt_rows, sl_rows = b.typhoon_mla_expand_query_rows(pc.block_table.cuda(), pc.seq_lens.cuda(), S_q)
    assert sl_rows.cpu().tolist() == row_lens
    assert torch.equal(bt_rows.cpu(), pc.block_table.repeat_interleave(S_q, dim=0))
    dec = TyphoonMLADecoder(H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda(),
                            inp.scale, B * S_q, pc.block_table.shape[1])
    for mode in (HYBRID, ABSORB):
        lse = torch.empty(B * S_q, H, dtype=torch.float32, device="cuda")
        out = dec.decode(rows.q_nope.cuda(), rows.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), bt_rows,
                         sl_rows, mode=mode, lse_out=lse)
        assert b.typhoon_mla_check_status(dec.shared) == 0
        G.assert_parity(out.float().cpu().double().numpy(), ref, lse.cpu().double().numpy(), ref_lse,
                        what=f"S_q={S_q} mode {mode}")
    dec.close()


def _tree_problem(B, H, root_len, branches, lens, seed):
    """Requests with a root prefix shared by all (may be 0 tokens = none) and one optional branch prefix per
    consecutive group.  `branches`: list of (first request, tokens); requests before the first branch and
    groups with 0 tokens have none.  Returns (rows for the checker, suffix-only inputs, branch latents)."""
    import dataclasses
    cfg = _cfg("tree", B=B, H=H, Ls=max(root_len, 1), lo=0, hi=0, seed=seed)
    inp = I.make_inputs(cfg, suffix_lens=lens)
    if root_len == 0:
        inp.ckv_shared, inp.kpe_shared = inp.ckv_shared[:0], inp.kpe_shared[:0]
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 77 + 1)
    starts = [b0 for b0, _ in branches] + [B]
    br = []
    for k, (b0, n) in enumerate(branches):
        br.append((b0, starts[k + 1], torch.randn(n, 512, generator=g).to(torch.bfloat16),
                   torch.randn(n, 64, generator=g).to(torch.bfloat16)))
    # checker: every request's own context = branch prefix + suffix (dense); the root stays shared
    rows = dataclasses.replace(inp, ckv_suffix=list(inp.ckv_suffix), kpe_suffix=list(inp.kpe_suffix))
    for b0, b1, c, r in br:
        for b in range(b0, b1):
            rows.ckv_suffix[b] = torch.cat([c, inp.ckv_suffix[b]])
            rows.kpe_suffix[b] = torch.cat([r, inp.kpe_suffix[b]])
    return rows, inp, br


@pytest.mark.parametrize("case", ["root+branches", "branches only", "root only, no pages"])
def test_tree_of_shared_prefixes(case, kernel_path):
    """Several shared prefixes per step: a root shared by all requests plus one prefix per group of
    requests, or flat groups, against the checker run on each request's whole context."""
    from paper_2509_21081_b200 import binding as b
    if kernel_path != "tcgen05":
        pytest.skip("row ranges need the tcgen05 kernel")
    B, H = 11, 32
    lens = [0, 3, 64, 65, 130, 7, 200, 1, 90, 64, 30]
    if case == "root+branches":
        root_len, branches = 210, [(0, 150), (3, 0), (5, 333), (9, 70)]
    elif case == "branches only":
        root_len, branches = 0, [(0, 100), (4, 260), (8, 0), (10, 65)]
    else:
        root_len, branches, lens = 500, [], [0] * B
    rows, inp, br = _tree_problem(B, H, root_len, branches, lens, seed=38)
    ref, ref_lse = G.run_oracle(rows)
    dev = "cuda"
    w_uk, w_uv = inp.w_uk.to(dev), inp.w_uv.to(dev)
    dims = b.make_dims(H)
    handles = []

    def prep(c, r):
        h = b.typhoon_mla_prepare_shared(dims, c.to(dev), r.to(dev), w_uk, w_uv)
        handles.append(h)
        return h

    levels = []
    if root_len > 0:
        levels.append(([prep(inp.ckv_shared, inp.kpe_shared)], [0, B]))
    if br:
        begins = [b0 for b0, _, _, _ in br] + [B]
        prefixes = [prep(c, r) if c.shape[0] > 0 else None for _, _, c, r in br]
        if begins[0] != 0:
            begins, prefixes = [0] + begins, [None] + prefixes
        levels.append((prefixes, begins))
    use_pages = case != "root only, no pages"
    pc = I.build_pages(inp)
    max_pages = pc.block_table.shape[1] if use_pages else 0
    ws = torch.empty(b.typhoon_mla_tree_workspace_bytes(levels, B, max_pages, 64), dtype=torch.uint8, device=dev)
    assert ws.numel() > 0
    out = torch.empty(B, H, 128, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(B, H, dtype=torch.float32, device=dev)
    args = (pc.ckv_pages.to(dev), pc.kpe_pages.to(dev), 64, pc.block_table.to(dev), pc.seq_lens.to(dev)) if use_pages \
        else (None, None, 64, None, None)
    b.typhoon_mla_decode_tree(levels, inp.q_nope.to(dev), inp.q_pe.to(dev), *args, inp.scale, out, ws, lse_out=lse)
    for h in handles:
        assert b.typhoon_mla_check_status(h) == 0
    G.assert_parity(out.float().cpu().double().numpy(), ref, lse.cpu().double().numpy(), ref_lse, what=f"tree: {case}")
    for h in handles:
        h.free()


def test_random_switches_repeatable_and_consistent(kernel_path):
    """Many small random problems with random work decomposition, stream overlap and launch mode: every
    call is bitwise repeatable, no in-kernel wait expires, and the hybrid and absorb-only paths agree."""
    import random
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    rnd = random.Random(77)
    try:
        for _ in range(40):
            H = rnd.choice([16, 32, 64, 128])
            B = rnd.choice([1, 2, 7, 33, 64, 65, 128, 129, 200, 300])
            Ls = rnd.choice([0, 1, 63, 64, 65, 500, 1000, 2049])
            hi = rnd.choice([0, 1, 64, 300])
            ps = rnd.choice([64, 128])
            b.typhoon_mla_set_naive_schedule(rnd.choice([0, 1, 2]))
            b.typhoon_mla_set_overlap(rnd.choice([True, True, False]))
            b.typhoon_mla_set_programmatic_launch(rnd.choice([True, True, False]))
            cfg = _cfg("switches", B=B, H=H, Ls=Ls, lo=0, hi=hi, seed=rnd.randint(0, 10 ** 6), page_size=ps)
            inp = I.make_inputs(cfg)
            if Ls == 0 and max(inp.suffix_lens) == 0:
                continue
            pc = I.build_pages(inp, page_size=ps)
            dec = TyphoonMLADecoder(H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda(),
                                    inp.scale, B, pc.block_table.shape[1], ps)
            args = (inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), pc.block_table.cuda(),
                    pc.seq_lens.cuda())
            outs = {}
            for mode in (HYBRID, ABSORB):
                o = [dec.decode(*args, mode=mode).clone() for _ in range(3)]
                assert b.typhoon_mla_check_status(dec.shared) == 0, f"{cfg} mode {mode}"
                assert all(torch.equal(x, o[0]) for x in o[1:]), f"not repeatable: {cfg} mode {mode}"
                assert torch.isfinite(o[0].float()).all(), f"non-finite: {cfg} mode {mode}"
                outs[mode] = o[0].float()
            d = (outs[HYBRID] - outs[ABSORB]).abs().max().item()
            assert d <= 3e-2 * max(1.0, outs[ABSORB].abs().max().item()), f"hybrid vs absorb {d}: {cfg}"
            dec.close()
    finally:
        b.typhoon_mla_set_naive_schedule(0)
        b.typhoon_mla_set_overlap(True)
        b.typhoon_mla_set_programmatic_launch(True)


def test_invalid_arguments():
    from paper_2509_21081_b200 import binding as b
    cfg = _cfg("inval", B=2, H=16, Ls=64, lo=8, hi=8, seed=33)
    inp = I.make_inputs(cfg)
    with pytest.raises(b.TyphoonMLAError) as e:
        b.typhoon_mla_prepare_shared(b.make_dims(17), inp.ckv_shared.cuda(), inp.kpe_shared.cuda(),
                                     inp.w_uk.cuda(), inp.w_uv.cuda())
    assert e.value.status == 2
    sh = b.typhoon_mla_prepare_shared(b.make_dims(16), inp.ckv_shared.cuda(), inp.kpe_shared.cuda(),
                                      inp.w_uk.cuda(), inp.w_uv.cuda())
    pc = I.build_pages(inp)
    out = torch.empty(2, 16, 128, dtype=torch.bfloat16, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.TyphoonMLAError) as e:
        b.typhoon_mla_decode(sh, inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), 64,
                             pc.block_table.cuda(), pc.seq_lens.cuda(), inp.scale, out, small, mode=HYBRID)
    assert e.value.status == 3
    with pytest.raises(b.TyphoonMLAError) as e:
        b.typhoon_mla_decode(sh, inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), 48,
                             pc.block_table.cuda(), pc.seq_lens.cuda(), inp.scale, out, small, mode=HYBRID)
    assert e.value.status == 1
    sh.free()


def test_fused_page_layout_and_strides():
    """Latent and rope keys interleaved in one 576-wide page array, passed through the token strides."""
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    cfg = _cfg("fused", B=5, H=32, Ls=200, lo=1, hi=300, seed=34)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp)
    pc = I.build_pages(inp)
    fused = torch.cat([pc.ckv_pages, pc.kpe_pages], dim=-1).contiguous().cuda()     # [P, 64, 576]
    ckv_view, kpe_view = fused[..., :512], fused[..., 512:]
    assert ckv_view.stride(-2) == 576 and kpe_view.data_ptr() == fused.data_ptr() + 1024
    dec = TyphoonMLADecoder(cfg.H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda(),
                            inp.scale, cfg.B, pc.block_table.shape[1])
    for mode in (HYBRID, ABSORB):
        lse = torch.empty(cfg.B, cfg.H, dtype=torch.float32, device="cuda")
        out = dec.decode(inp.q_nope.cuda(), inp.q_pe.cuda(), ckv_view, kpe_view, pc.block_table.cuda(),
                         pc.seq_lens.cuda(), mode=mode, lse_out=lse)
        assert b.typhoon_mla_check_status(dec.shared) == 0
        G.assert_parity(out.float().cpu().double().numpy(), ref, lse.cpu().double().numpy(), ref_lse,
                        what=f"fused layout mode {mode}")
    dec.close()


def test_order_by_length_is_a_stable_descending_sort():
    """Index work: bit-exact against numpy (descending length, ties by ascending index)."""
    from paper_2509_21081_b200 import binding as b
    rng = np.random.default_rng(3)
    for B in (1, 2, 5, 64, 257, 1000, 4096):
        lens = rng.integers(0, 40, size=B).astype(np.int32)        # many ties
        perm = b.typhoon_mla_order_by_length(torch.from_numpy(lens).cuda()).cpu().numpy()
        ref = np.lexsort((np.arange(B), -lens.astype(np.int64)))
        assert np.array_equal(perm, ref), f"B={B}"


# ------------------------------------------------------------ full-size configs
def _sampled_pairs(cfg, n, seed):
    r = np.random.default_rng(seed)
    pairs = {(int(r.integers(cfg.B)), int(r.integers(cfg.H))) for _ in range(n)}
    return sorted(pairs)


def _full_size_sampled(cfg, modes, n_pairs, extremes=False):
    inp = I.make_inputs(cfg)
    pairs = _sampled_pairs(cfg, n_pairs, cfg.seed)
    if extremes:  # always include the shortest and the longest suffix
        for b in (int(np.argmin(inp.suffix_lens)), int(np.argmax(inp.suffix_lens))):
            pairs += [(b, 0), (b, cfg.H - 1)]
    ref, ref_lse = G.run_oracle(inp, pairs=pairs)
    mask = ~np.isnan(ref_lse)
    res = {}
    for mode in modes:
        out, lse, launches = G.run_gpu(inp, mode)
        assert np.isfinite(out).all()
        res[mode] = G.assert_parity(out, ref, lse, ref_lse, mask=mask, what=f"{cfg.name} mode {mode}")
    return res


def _checked_requests(cfg, inp, n_min=16):
    """Requests whose rows the checker computes for ALL heads: the first and the last request of every
    query-row group of the shared-prefix kernel, the rows on either side of a row-tile boundary, the
    shortest and the longest suffix, and seeded random ones up to n_min."""
    B = cfg.B
    if B <= n_min:
        return list(range(B))
    chosen = {0, B - 1, int(np.argmin(inp.suffix_lens)), int(np.argmax(inp.suffix_lens))}
    for g0 in range(0, B, 256):                      # a CTA of the 128-token-tile kernel owns 256 query rows ...
        chosen |= {g0, min(g0 + 255, B - 1)}
    chosen |= {min(127, B - 1), min(128, B - 1)}     # ... as two row tiles of 128
    r = np.random.default_rng(cfg.seed + 17)
    while len(chosen) < n_min:
        chosen.add(int(r.integers(B)))
    return sorted(chosen)


def _full_size_all_heads(cfg, modes, kernel_path, all_rows=False):
    """A benchmark configuration at full size, in the launch configuration the benchmark times: the float64
    checker computes every head of the checked requests (every request with all_rows), so that every head,
    every tile range and partial slot of the shared-prefix kernel and every query-row group is compared;
    next to it the whole output tensor of the tcgen05 kernels is compared with that of the warp-MMA kernels
    (both are checked against the float64 rows): a second net over the rows the checker does not reach."""
    from paper_2509_21081_b200 import binding as b
    if kernel_path != "tcgen05":
        pytest.skip("both kernel paths run inside the tcgen05 parametrisation of this test")
    inp = I.make_inputs(cfg)
    reqs = list(range(cfg.B)) if all_rows else _checked_requests(cfg, inp)
    pairs = [(r, h) for r in reqs for h in range(cfg.H)]
    ref, ref_lse = G.run_oracle(inp, pairs=pairs)
    mask = ~np.isnan(ref_lse)
    assert mask.sum() == len(reqs) * cfg.H
    for mode in modes:
        outs = {}
        for path in (b.PATH_TCGEN05, b.PATH_WARP_MMA):
            b.typhoon_mla_set_kernel_path(path)
            out, lse, _ = G.run_gpu(inp, mode)
            assert np.isfinite(out).all()
            G.assert_parity(out, ref, lse, ref_lse, mask=mask, what=f"{cfg.name} mode {mode} path {path}")
            outs[path] = (out, lse)
        b.typhoon_mla_set_kernel_path(b.PATH_TCGEN05)
        (o_t, l_t), (o_w, l_w) = outs[b.PATH_TCGEN05], outs[b.PATH_WARP_MMA]
        # two implementations with different summation orders and both within the bars of the float64 rows:
        # their difference over the whole tensor stays within twice those bars, row by row as well
        d = np.abs(o_t - o_w)
        assert d.max() <= 2 * G.MAX_ABS_TOL
        rn = np.linalg.norm(o_w.reshape(-1, 128), axis=1)
        re = np.linalg.norm((o_t - o_w).reshape(-1, 128), axis=1)
        assert np.linalg.norm(o_t - o_w) / np.linalg.norm(o_w) <= 2 * G.REL_FRO_TOL
        assert np.max(re / np.maximum(rn, 1e-30)) <= 8 * G.REL_FRO_TOL, f"{cfg.name} mode {mode}: worst row tcgen05 vs warp-MMA"
        assert np.max(np.abs(l_t - l_w)) <= 2 * G.LSE_TOL


def test_cfg1_full_size_all_rows(kernel_path):
    """DeepSeek-v3 dims, B=64, Ls=4096, Ln=512 -- the benchmark's headline configuration: every
    (request, head) row against the float64 checker, in the hybrid mode AUTO resolves to and absorb-only."""
    _full_size_all_heads(I.CONFIGS["cfg1"], (AUTO, ABSORB), kernel_path, all_rows=True)


def test_cfg3_kimi_like_all_heads(kernel_path):
    _full_size_all_heads(I.CONFIGS["cfg3"], (HYBRID,), kernel_path)


def test_cfg2_long_prompt_all_heads(kernel_path):
    _full_size_all_heads(I.CONFIGS["cfg2"], (HYBRID,), kernel_path)


@pytest.mark.parametrize("B", [1, 8, 32, 128, 512, 1024])
def test_cfg4_fanout_all_heads(B, kernel_path):
    """The fan-out sweep at every batch size of the benchmark, in the mode AUTO picks (absorb-only at 1 and 8,
    hybrid above) and, up to 128 requests, in the other one as well."""
    modes = (AUTO,) if B > 128 else (AUTO, HYBRID if B <= 8 else ABSORB)
    _full_size_all_heads(I.CONFIGS["cfg4"].with_batch(B), modes, kernel_path)


def test_long_prefix_sampled():
    """A prefix of 70 001 tokens (1094 tiles per head, not a tile multiple): tile indexing over long ranges,
    many ring wrap-arounds per CTA, many absorb chunks in ABSORB mode."""
    cfg = _cfg("long", B=3, H=16, Ls=70001, lo=1, hi=300, seed=51)
    _full_size_sampled(cfg, (HYBRID, ABSORB), n_pairs=6)


def test_more_requests_than_the_ordering_block_sorts():
    """B = 4500 (> 4096): no longest-first order and no descriptors, 4500 CTAs per head group."""
    cfg = _cfg("wide", B=4500, H=16, Ls=100, lo=0, hi=70, seed=52)
    _full_size_sampled(cfg, (HYBRID, ABSORB), n_pairs=48, extremes=True)


def _upload(inp, pc):
    dev = "cuda"
    return (inp.q_nope.to(dev), inp.q_pe.to(dev), pc.ckv_pages.to(dev), pc.kpe_pages.to(dev), pc.block_table.to(dev),
            pc.seq_lens.to(dev))


@pytest.mark.parametrize("world,Ls", [(2, 1000), (3, 700), (4, 130)])
def test_sequence_sharded_ranks_one_after_the_other(world, Ls):
    """The context sharded by sequence over `world` ranks, the ranks' partial steps run one after the other
    on this GPU (no kernel waits for another): slices of the prefix (one of them empty when there are fewer
    64-token blocks than ranks), suffixes owned round robin, fp32 partials merged by the combine entry point."""
    from paper_2509_21081_b200 import binding as b, sharded as S
    cfg = _cfg("seqshard", B=11, H=32, Ls=Ls, lo=0, hi=260, seed=60 + world)
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp, poison=True)
    ref, ref_lse = G.run_oracle(inp)
    args = _upload(inp, pc)
    parts = []
    for r in range(world):
        dec = S.SequenceShardedDecoder(r, world, cfg.H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(),
                                       inp.w_uv.cuda(), inp.scale, cfg.B, pc.block_table.shape[1])
        parts.append(dec.partial(*args, mode=AUTO if r % 2 else HYBRID))
        assert b.typhoon_mla_check_status(dec.shared) == 0
        dec.close()
    lse = torch.empty(cfg.B, cfg.H, dtype=torch.float32, device="cuda")
    out = S.merge_partials(torch.stack([p[0] for p in parts]), torch.stack([p[1] for p in parts]), lse)
    G.assert_parity(out.float().cpu().double().numpy(), ref, lse.cpu().double().numpy(), ref_lse, what=f"sequence shards {world}")


@pytest.mark.parametrize("world,H", [(2, 64), (4, 128)])
def test_head_sharded_ranks_one_after_the_other(world, H):
    from paper_2509_21081_b200 import binding as b, sharded as S
    cfg = _cfg("headshard", B=6, H=H, Ls=300, lo=1, hi=150, seed=70 + world)
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp, poison=True)
    ref, _ = G.run_oracle(inp)
    args = _upload(inp, pc)
    parts = []
    for r in range(world):
        dec = S.HeadShardedDecoder(r, world, cfg.H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(),
                                   inp.w_uv.cuda(), inp.scale, cfg.B, pc.block_table.shape[1])
        parts.append(dec.local(*args, mode=HYBRID))
        assert b.typhoon_mla_check_status(dec.shared) == 0
        dec.close()
    out = S.join_heads(torch.stack(parts))
    G.assert_parity(out.float().cpu().double().numpy(), ref, what=f"head shards {world}")


def test_combine_partials_edge_cases():
    """Partials that are all empty give a zero row and -inf; an empty partial next to a live one has no weight
    even when its row holds NaN."""
    from paper_2509_21081_b200 import sharded as S
    g = torch.Generator().manual_seed(3)
    o = torch.randn(3, 4, 16, 128, generator=g).cuda()
    lse = torch.randn(3, 4, 16, generator=g).cuda()
    lse[:, 0, :] = -math.inf                     # request 0: nothing anywhere
    lse[1, 1, :] = -math.inf; o[1, 1] = math.nan   # request 1: rank 1 holds nothing, its row is garbage
    lse_out = torch.empty(4, 16, device="cuda")
    out = S.merge_partials(o, lse, lse_out).float().cpu()
    assert torch.all(out[0] == 0) and torch.all(lse_out[0].cpu() == -math.inf)
    o64, l64 = o.cpu().double(), lse.cpu().double()
    w = torch.softmax(l64[:, 1:], dim=0)
    w = torch.nan_to_num(w, nan=0.0)
    o64 = torch.nan_to_num(o64, nan=0.0)
    ref = (w.unsqueeze(-1) * o64[:, 1:]).sum(0)
    assert torch.allclose(out[1:].double(), ref, atol=2e-2, rtol=1e-2)
    assert torch.allclose(lse_out[1:].cpu().double(), torch.logsumexp(l64[:, 1:], dim=0), atol=1e-4)


@pytest.mark.parametrize("B", [1, 2, 3])
def test_absorb_only_one_or_two_requests(B):
    """Absorb-only steps of one or two requests take a single kernel for chunk merge, output projection and
    rounding; three requests take the GEMM form.  Long context (many chunks), one empty suffix, bf16 and fp32
    (partial) outputs."""
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    cfg = _cfg("fewreq", B=B, H=64, Ls=3000, lo=0, hi=0, seed=80 + B)
    inp = I.make_inputs(cfg, suffix_lens=[0, 333, 70][:B])
    ref, ref_lse = G.run_oracle(inp)
    out, lse, launches = G.run_gpu(inp, ABSORB)
    G.assert_parity(out, ref, lse, ref_lse, what=f"absorb-only B={B}")
    pc = I.build_pages(inp, poison=True)
    dec = TyphoonMLADecoder(cfg.H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda(), inp.scale,
                            cfg.B, pc.block_table.shape[1])
    o32 = torch.empty(B, cfg.H, 128, dtype=torch.float32, device="cuda")
    l32 = torch.empty(B, cfg.H, dtype=torch.float32, device="cuda")
    b.typhoon_mla_decode_partial(dec.shared, *_upload(inp, pc)[:4], cfg.page_size, *_upload(inp, pc)[4:], inp.scale, o32, l32,
                                 dec.workspace, mode=ABSORB)
    assert b.typhoon_mla_check_status(dec.shared) == 0
    G.assert_parity(o32.cpu().double().numpy(), ref, l32.cpu().double().numpy(), ref_lse, what=f"absorb-only fp32 B={B}")
    dec.close()


def test_partial_step_without_suffixes():
    """The fp32 partial of a rank that holds prefix tokens only (no page table): the stand-alone combine writes it."""
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    cfg = _cfg("partial_naive", B=70, H=16, Ls=900, lo=0, hi=0, seed=91)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp, drop_suffix=True)
    dec = TyphoonMLADecoder(cfg.H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda(), inp.scale,
                            cfg.B, 0)
    o32 = torch.empty(cfg.B, cfg.H, 128, dtype=torch.float32, device="cuda")
    l32 = torch.empty(cfg.B, cfg.H, dtype=torch.float32, device="cuda")
    b.typhoon_mla_decode_partial(dec.shared, inp.q_nope.cuda(), inp.q_pe.cuda(), None, None, cfg.page_size, None, None,
                                 inp.scale, o32, l32, dec.workspace, mode=NAIVE)
    assert b.typhoon_mla_check_status(dec.shared) == 0
    G.assert_parity(o32.cpu().double().numpy(), ref, l32.cpu().double().numpy(), ref_lse, what="fp32 partial, prefix only")
    dec.close()


def test_random_trees_against_per_group_steps(kernel_path):
    """Seeded random two-level trees (a root for all requests, branches for consecutive groups, some groups
    without a branch, some trees without a root): every group's rows equal an ordinary step of that group over
    the concatenation of root and branch (two runs of the library that share no launch plan)."""
    if kernel_path == "warp_mma":
        pytest.skip("row ranges need the tcgen05 kernel")
    import random
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    rng = random.Random(11)
    dev = "cuda"
    for it in range(24):
        H = rng.choice([16, 64, 128])
        B = rng.choice([2, 5, 16, 40, 64, 100, 130, 260])
        Ls = rng.choice([0, 64, 300, 1000, 3000])
        hi = rng.choice([0, 50, 400])
        n_groups = min(rng.choice([1, 2, 3, 5]), B)
        cfg = _cfg("rtree", B=B, H=H, Ls=Ls, lo=0, hi=hi, seed=500 + it)
        inp = I.make_inputs(cfg)
        pc = I.build_pages(inp, poison=True)
        gb = [0] + sorted(rng.sample(range(1, B), n_groups - 1)) + [B]
        branch_len = [rng.choice([0, 1, 70, 500, 1500]) for _ in range(n_groups)]
        gen = torch.Generator().manual_seed(it)
        br_ckv = [torch.randn(n, 512, generator=gen).to(torch.bfloat16) for n in branch_len]
        br_kpe = [torch.randn(n, 64, generator=gen).to(torch.bfloat16) for n in branch_len]
        dims = b.make_dims(H)
        w_uk, w_uv = inp.w_uk.to(dev), inp.w_uv.to(dev)
        root = b.typhoon_mla_prepare_shared(dims, inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), w_uk, w_uv) if Ls > 0 else None
        brs = [b.typhoon_mla_prepare_shared(dims, c.to(dev), k.to(dev), w_uk, w_uv) if c.shape[0] > 0 else None
               for c, k in zip(br_ckv, br_kpe)]
        levels = ([([root], [0, B])] if root is not None else []) + ([(brs, gb)] if any(x is not None for x in brs) else [])
        if not levels:
            continue
        args = _upload(inp, pc)
        out = torch.empty(B, H, 128, dtype=torch.bfloat16, device=dev)
        ws = torch.empty(b.typhoon_mla_tree_workspace_bytes(levels, B, pc.block_table.shape[1], 64), dtype=torch.uint8, device=dev)
        b.typhoon_mla_decode_tree(levels, args[0], args[1], args[2], args[3], 64, args[4], args[5], inp.scale, out, ws)
        handles = ([root] if root is not None else []) + [x for x in brs if x is not None]
        assert b.typhoon_mla_check_status(handles[0]) == 0
        for gi in range(n_groups):
            r0, r1 = gb[gi], gb[gi + 1]
            dec = TyphoonMLADecoder(H, torch.cat([inp.ckv_shared, br_ckv[gi]]).to(dev), torch.cat([inp.kpe_shared, br_kpe[gi]]).to(dev),
                                    w_uk, w_uv, inp.scale, r1 - r0, pc.block_table.shape[1])
            ref = dec.decode(args[0][r0:r1].contiguous(), args[1][r0:r1].contiguous(), args[2], args[3],
                             args[4][r0:r1].contiguous(), args[5][r0:r1].contiguous(), mode=AUTO).float()
            dec.close()
            o = out[r0:r1].float()
            assert torch.isfinite(o).all()
            err = float((o - ref).abs().max()) / max(1.0, float(ref.abs().max()))
            assert err < 2e-2, (it, gi, dict(H=H, B=B, Ls=Ls, hi=hi, groups=gb, branch=branch_len), err)
        for x in handles:
            x.free()


def test_random_shards_against_the_whole_step():
    """Seeded random sequence shardings (2 to 5 ranks, prefixes shorter than one block per rank included, ranks in
    different modes) and two-way head shardings: merged partials equal the single-device step."""
    import random
    from paper_2509_21081_b200 import binding as b, sharded as S
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    rng = random.Random(12)
    dev = "cuda"
    for it in range(30):
        B = rng.choice([1, 2, 3, 7, 16, 33, 64, 65, 130, 200])
        H = rng.choice([16, 32, 64, 128])
        Ls = rng.choice([0, 1, 63, 64, 65, 200, 513, 1500, 4000])
        hi = rng.choice([0, 1, 70, 300, 900])
        world = rng.choice([2, 3, 4, 5])
        if Ls == 0 and hi == 0:
            continue
        cfg = _cfg("rshard", B=B, H=H, Ls=Ls, lo=0, hi=hi, seed=1000 + it)
        inp = I.make_inputs(cfg)
        pc = I.build_pages(inp, poison=True)
        args = _upload(inp, pc)
        dev_in = (inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), inp.w_uk.to(dev), inp.w_uv.to(dev))
        dec = TyphoonMLADecoder(H, *dev_in, inp.scale, B, pc.block_table.shape[1])
        lse_ref = torch.empty(B, H, device=dev)
        ref = dec.decode(*args, mode=AUTO, lse_out=lse_ref).float()
        dec.close()
        parts = []
        for r in range(world):
            d = S.SequenceShardedDecoder(r, world, H, *dev_in, inp.scale, B, pc.block_table.shape[1])
            parts.append(d.partial(*args, mode=rng.choice([AUTO, HYBRID, ABSORB])))
            assert b.typhoon_mla_check_status(d.shared) == 0
            d.close()
        lse = torch.empty(B, H, device=dev)
        out = S.merge_partials(torch.stack([p[0] for p in parts]), torch.stack([p[1] for p in parts]), lse).float()
        scale = max(1.0, float(ref.abs().max()))
        fin = torch.isfinite(lse_ref)
        assert torch.isfinite(out).all() and torch.equal(torch.isfinite(lse), fin)
        assert float((out - ref).abs().max()) / scale < 2e-2, (it, dict(B=B, H=H, Ls=Ls, hi=hi, world=world))
        if fin.any():
            assert float((lse[fin] - lse_ref[fin]).abs().max()) < 2e-2
        if H % 32 == 0:
            halves = []
            for r in range(2):
                d = S.HeadShardedDecoder(r, 2, H, *dev_in, inp.scale, B, pc.block_table.shape[1])
                halves.append(d.local(*args, mode=AUTO))
                d.close()
            o2 = S.join_heads(torch.stack(halves)).float()
            assert float((o2 - ref).abs().max()) / scale < 2e-2, (it, "heads")


@pytest.mark.parametrize("H,B", [(16, 7), (16, 37), (48, 5), (32, 64), (64, 3)])
def test_absorb_row_groups_stacked_and_per_request(H, B, kernel_path):
    """Absorb-only steps over the shared prefix take 64-row groups of the stacked [B * H] query matrix (requests
    share a tile when a device has fewer than 64 heads) or, with the switch off, of every request: both against
    the checker, with ragged suffixes so that the per-request suffix items run next to the stacked prefix items."""
    from paper_2509_21081_b200 import binding as b
    if kernel_path != "tcgen05":
        pytest.skip("row groups are a property of the tcgen05 kernel")
    cfg = _cfg("stack", B=B, H=H, Ls=1100, lo=0, hi=150, seed=300 + H + B)
    inp = I.make_inputs(cfg)
    ref, ref_lse = G.run_oracle(inp)
    try:
        for stacked in (True, False):
            b.typhoon_mla_set_stacked_absorb(stacked)
            out, lse, _ = G.run_gpu(inp, ABSORB)
            G.assert_parity(out, ref, lse, ref_lse, what=f"H={H} B={B} stacked={stacked}")
    finally:
        b.typhoon_mla_set_stacked_absorb(True)
