"""The allocation-free entry point against the regular one and against the float64 checker.

typhoon_mla_naive_shared_noalloc serves callers that cannot allocate device memory when they call
(all HBM already pledged to a cache pool, or cudaMalloc banned on a latency-critical path): its
scratch is a fixed array inside the library.  Two calls in a row with different queries must each
match typhoon_mla_decode in NAIVE mode (which uses a caller workspace) and the checker's result for
the prefix alone, so stale contents of the shared array cannot leak from one call into the next; an
oversized problem and a bad scale must be refused with nothing written; a handle without a prefix
gives zero rows and lse = -inf.
This file sorts last so that a run stopping at the first failure has already run everything else.
"""
import math

import numpy as np
import pytest
import torch

from paper_2509_21081_b200 import inputs as I
from tests import gpu_harness as G

pytestmark = pytest.mark.gpu


def test_noalloc_matches_workspace_entry_point_twice():
    from paper_2509_21081_b200 import binding as b
    cfg = I.MLAConfig("noalloc", B=37, H=32, Ls=1500, suffix_lo=0, suffix_hi=0, seed=77)
    inp = I.make_inputs(cfg)
    dims = b.make_dims(cfg.H)
    w_uk, w_uv = inp.w_uk.cuda(), inp.w_uv.cuda()
    sh = b.typhoon_mla_prepare_shared(dims, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), w_uk, w_uv)
    ws = torch.empty(b.typhoon_mla_workspace_bytes(sh, cfg.B, 0, 64), dtype=torch.uint8, device="cuda")
    q1n, q1p = inp.q_nope.cuda(), inp.q_pe.cuda()
    g = torch.Generator(device="cpu").manual_seed(5)
    q2n = torch.randn(cfg.B, cfg.H, 128, generator=g).to(torch.bfloat16).cuda() * 3
    q2p = torch.randn(cfg.B, cfg.H, 64, generator=g).to(torch.bfloat16).cuda() * 3
    ora1, ora1_lse = G.run_oracle(inp, drop_suffix=True)      # the float64 checker over the prefix alone
    inp2 = I.make_inputs(cfg)
    inp2.q_nope, inp2.q_pe = q2n.cpu(), q2p.cpu()
    ora2, ora2_lse = G.run_oracle(inp2, drop_suffix=True)
    for (qn, qp), (ora, ora_lse) in zip(((q1n, q1p), (q2n, q2p)), ((ora1, ora1_lse), (ora2, ora2_lse))):
        ref = torch.empty(cfg.B, cfg.H, 128, dtype=torch.bfloat16, device="cuda")
        ref_lse = torch.empty(cfg.B, cfg.H, dtype=torch.float32, device="cuda")
        b.typhoon_mla_decode(sh, qn, qp, None, None, 64, None, None, inp.scale, ref, ws, mode=b.MODE_NAIVE,
                             lse_out=ref_lse)
        out = torch.full((cfg.B, cfg.H, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((cfg.B, cfg.H), float("nan"), dtype=torch.float32, device="cuda")
        b.typhoon_mla_naive_shared_noalloc(sh, qn, qp, inp.scale, out, lse)
        torch.cuda.synchronize()
        o, r = out.float().cpu().numpy(), ref.float().cpu().numpy()
        assert np.isfinite(o).all()
        # same kernels, possibly a different number of KV splits: same bars as the parity tests
        assert np.max(np.abs(o - r)) <= 2e-2 * max(1.0, float(np.max(np.abs(r))))
        assert np.linalg.norm(o - r) / np.linalg.norm(r) <= 5e-3
        assert torch.max(torch.abs(lse - ref_lse)).item() <= 2e-2
        G.assert_parity(out.float().cpu().double().numpy(), ora, lse.cpu().double().numpy(), ora_lse,
                        what="allocation-free entry point vs float64 checker")
    assert b.typhoon_mla_last_launch_count() == 2
    sh.free()


def test_noalloc_without_a_prefix_gives_empty_rows():
    from paper_2509_21081_b200 import binding as b
    cfg = I.MLAConfig("noalloc_empty", B=3, H=16, Ls=0, suffix_lo=0, suffix_hi=0, seed=79)
    inp = I.make_inputs(cfg)
    w_uk, w_uv = inp.w_uk.cuda(), inp.w_uv.cuda()
    sh = b.typhoon_mla_prepare_shared(b.make_dims(cfg.H), inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), w_uk, w_uv)
    out = torch.full((cfg.B, cfg.H, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((cfg.B, cfg.H), float("nan"), dtype=torch.float32, device="cuda")
    b.typhoon_mla_naive_shared_noalloc(sh, inp.q_nope.cuda(), inp.q_pe.cuda(), inp.scale, out, lse)
    torch.cuda.synchronize()
    assert bool((out == 0).all()) and bool((lse == -math.inf).all())
    sh.free()


def test_noalloc_rejects_oversized_problem():
    from paper_2509_21081_b200 import binding as b
    cfg = I.MLAConfig("noalloc_big", B=2, H=128, Ls=64, suffix_lo=0, suffix_hi=0, seed=78)
    inp = I.make_inputs(cfg)
    w_uk, w_uv = inp.w_uk.cuda(), inp.w_uv.cuda()
    sh = b.typhoon_mla_prepare_shared(b.make_dims(cfg.H), inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), w_uk, w_uv)
    B = 600                                    # 600 * 128 * 516 bytes > 32 MiB
    qn = torch.zeros(B, cfg.H, 128, dtype=torch.bfloat16, device="cuda")
    qp = torch.zeros(B, cfg.H, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.full((B, cfg.H, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, cfg.H), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(b.TyphoonMLAError) as e:
        b.typhoon_mla_naive_shared_noalloc(sh, qn, qp, inp.scale, out, lse)
    assert e.value.status == 7 and "scratch" in str(e.value)
    for bad_scale in (0.0, -0.5, float("nan")):
        with pytest.raises(b.TyphoonMLAError) as e:
            b.typhoon_mla_naive_shared_noalloc(sh, qn[:2], qp[:2], bad_scale, out[:2], lse[:2])
        assert e.value.status == 1
    torch.cuda.synchronize()
    assert bool((out == 7.0).all()) and bool((lse == 7.0).all()), "a refused call wrote to its outputs"
    assert b.typhoon_mla_last_launch_count() == 0
    sh.free()


def test_noalloc_with_an_8bit_expanded_cache():
    """The same entry point on a handle whose expanded cache is stored as E4M3 codes: against the checker's operator
    over the decoded values, prefix alone."""
    from paper_2509_21081_b200 import binding as b
    cfg = I.MLAConfig("noalloc8", B=70, H=16, Ls=900, suffix_lo=0, suffix_hi=0, seed=78)
    inp = I.make_inputs(cfg)
    w_uk, w_uv = inp.w_uk.cuda(), inp.w_uv.cuda()
    sh = b.typhoon_mla_prepare_shared_fp8(b.make_dims(cfg.H), inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), w_uk, w_uv)
    ora, ora_lse = G.run_oracle_fp8(inp, drop_suffix=True)
    out = torch.full((cfg.B, cfg.H, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((cfg.B, cfg.H), float("nan"), dtype=torch.float32, device="cuda")
    b.typhoon_mla_naive_shared_noalloc(sh, inp.q_nope.cuda(), inp.q_pe.cuda(), inp.scale, out, lse)
    assert b.typhoon_mla_check_status(sh) == 0
    G.assert_parity(out.float().cpu().double().numpy(), ora, lse.cpu().double().numpy(), ora_lse,
                    what="allocation-free entry point, 8-bit cache")
    sh.free()
