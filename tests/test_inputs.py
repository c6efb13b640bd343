"""The seeded input generator: determinism, batch-prefix property, paging."""
import numpy as np
import torch

from paper_2509_21081_b200 import inputs as I


def test_deterministic_and_bf16():
    a = I.make_inputs(I.CONFIGS["cfg0"]); b = I.make_inputs(I.CONFIGS["cfg0"])
    assert a.q_nope.dtype == torch.bfloat16 and torch.equal(a.q_nope, b.q_nope)
    assert torch.equal(a.ckv_suffix[3], b.ckv_suffix[3]) and a.suffix_lens == [64] * 4
    assert abs(a.scale - 192 ** -0.5) < 1e-12
    # W drawn with variance 1/512
    assert abs(float(a.w_uk.float().std()) - 512 ** -0.5) < 2e-3


def test_smaller_batch_is_prefix():
    c = I.MLAConfig("t", B=6, H=2, Ls=8, suffix_lo=1, suffix_hi=40, seed=4)
    big = I.make_inputs(c); small = I.make_inputs(c.with_batch(3))
    assert small.suffix_lens == big.suffix_lens[:3]
    assert torch.equal(small.q_nope, big.q_nope[:3])
    assert all(torch.equal(x, y) for x, y in zip(small.ckv_suffix, big.ckv_suffix))
    assert torch.equal(small.ckv_shared, big.ckv_shared)


def test_pages_roundtrip_and_poison():
    c = I.MLAConfig("t", B=5, H=2, Ls=8, suffix_lo=0, suffix_hi=150, seed=9)
    inp = I.make_inputs(c, suffix_lens=[0, 1, 64, 65, 150])
    for ps in (64, 128):
        pc = I.build_pages(inp, page_size=ps)
        assert pc.seq_lens.tolist() == [0, 1, 64, 65, 150]
        used = set()
        for b, n in enumerate(inp.suffix_lens):
            got = []
            for j in range((n + ps - 1) // ps):
                pid = int(pc.block_table[b, j]); assert pid >= 0 and pid not in used
                used.add(pid); got.append(pc.ckv_pages[pid])
            if n:
                dense = torch.cat(got)[:n]
                assert torch.equal(dense, inp.ckv_suffix[b])
                assert torch.isnan(torch.cat(got)[n:].float()).all()
            assert (pc.block_table[b, (n + ps - 1) // ps:] == -1).all()
        assert len(used) == pc.ckv_pages.shape[0] - 2
