"""GPU tests of the boundary's safety net: page ids outside the caller's cache, the bounded in-kernel
wait, the status word, planning queries from several threads while a switch flips, and argument checks
that need a device.  None of these tests faults, traps or hangs the GPU: the failure is either an input
the library is specified to survive, or a dedicated test kernel that waits on a barrier with a deadline
of a few hundred microseconds."""
import threading

import numpy as np
import pytest
import torch

from paper_2509_21081_b200 import inputs as I
from tests import gpu_harness as G

pytestmark = pytest.mark.gpu

ABSORB, HYBRID, AUTO, NAIVE = 1, 2, 0, 3


def _cfg(name, B, H, Ls, lo, hi, seed, page_size=64):
    return I.MLAConfig(name, B=B, H=H, Ls=Ls, suffix_lo=lo, suffix_hi=hi, seed=seed, page_size=page_size)


def _decoder(inp, pc, B=None):
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    return TyphoonMLADecoder(inp.cfg.H, inp.ckv_shared.cuda(), inp.kpe_shared.cuda(), inp.w_uk.cuda(), inp.w_uv.cuda(),
                             inp.scale, B or inp.cfg.B, pc.block_table.shape[1], pc.page_size)


@pytest.mark.parametrize("path", ["tcgen05", "warp_mma"])
@pytest.mark.parametrize("bad_id", ["num_pages", "minus_one", "huge"])
def test_page_id_outside_the_cache_is_not_dereferenced(path, bad_id):
    """A block-table entry inside a request's length that does not name a page of the cache: the step
    returns without a fault, the status word reports it, the other requests' rows still match the checker,
    and after clearing the word a step with a sound table is clean."""
    from paper_2509_21081_b200 import binding as b
    b.typhoon_mla_set_kernel_path(b.PATH_TCGEN05 if path == "tcgen05" else b.PATH_WARP_MMA)
    try:
        cfg = _cfg("badpage", B=5, H=32, Ls=300, lo=0, hi=0, seed=95)
        inp = I.make_inputs(cfg, suffix_lens=[100, 200, 330, 64, 10])
        pc = I.build_pages(inp, poison=True)
        ref, ref_lse = G.run_oracle(inp)
        dec = _decoder(inp, pc)
        n_pages = pc.ckv_pages.shape[0]
        bt = pc.block_table.clone()
        bt[2, 3] = {"num_pages": n_pages, "minus_one": -1, "huge": 1 << 22}[bad_id]   # request 2, tokens 192..255
        args = (inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda())
        for mode in (HYBRID, ABSORB):
            lse = torch.empty(cfg.B, cfg.H, dtype=torch.float32, device="cuda")
            out = dec.decode(*args, bt.cuda(), pc.seq_lens.cuda(), mode=mode, lse_out=lse)
            word = b.typhoon_mla_check_status(dec.shared, clear=True, raise_on_error=False)
            assert word == b.STATUS_BAD_PAGE, hex(word)
            o = out.float().cpu().double().numpy()
            keep = np.ones((cfg.B, cfg.H), dtype=bool)
            keep[2] = False                                  # that request's rows are unspecified (but finite)
            assert np.isfinite(o).all()
            G.assert_parity(o, ref, lse.cpu().double().numpy(), ref_lse, mask=keep, what=f"bad page {bad_id} mode {mode}")
            with pytest.raises(b.TyphoonMLAError):
                dec.decode(*args, bt.cuda(), pc.seq_lens.cuda(), mode=mode)
                b.typhoon_mla_check_status(dec.shared)        # raises ERR_DEVICE_CHECK
            assert b.typhoon_mla_check_status(dec.shared, clear=True, raise_on_error=False) == b.STATUS_BAD_PAGE
            # a sound table afterwards: clean word, all rows right
            out = dec.decode(*args, pc.block_table.cuda(), pc.seq_lens.cuda(), mode=mode, lse_out=lse)
            assert b.typhoon_mla_check_status(dec.shared) == 0
            G.assert_parity(out.float().cpu().double().numpy(), ref, lse.cpu().double().numpy(), ref_lse, what="sound table")
        # entries past a request's length may hold anything, also ids far outside the cache
        bt = pc.block_table.clone()
        bt[4, 1:] = 1 << 29
        bt[3, 1:] = -7
        out = dec.decode(*args, bt.cuda(), pc.seq_lens.cuda(), mode=HYBRID)
        assert b.typhoon_mla_check_status(dec.shared) == 0
        G.assert_parity(out.float().cpu().double().numpy(), ref, what="garbage past the length")
        dec.close()
    finally:
        b.typhoon_mla_set_kernel_path(b.PATH_TCGEN05)


def test_num_pages_is_required_with_a_page_table():
    from paper_2509_21081_b200 import binding as b
    cfg = _cfg("nopages", B=2, H=16, Ls=64, lo=8, hi=8, seed=96)
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp)
    dec = _decoder(inp, pc)
    out = torch.empty(2, 16, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.TyphoonMLAError) as e:
        b.typhoon_mla_decode(dec.shared, inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), 64,
                             pc.block_table.cuda(), pc.seq_lens.cuda(), inp.scale, out, dec.workspace, mode=HYBRID,
                             num_pages=0)
    assert e.value.status == 1
    dec.close()


def test_bounded_wait_runs_out_and_the_context_survives():
    """The wait every kernel of the library uses, on a barrier nothing arrives on (a test kernel: no copies, no
    tensor memory), with a deadline of about 0.2 ms: the kernel returns, the status word carries the code, the
    check call reports it, and an ordinary step afterwards is clean and right."""
    from paper_2509_21081_b200 import binding as b
    inp = I.make_inputs(I.CONFIGS["cfg0"])
    pc = I.build_pages(inp)
    ref, ref_lse = G.run_oracle(inp)
    dec = _decoder(inp, pc)
    assert b.typhoon_mla_check_status(dec.shared) == 0
    b.typhoon_mla_test_wait_expiry(dec.shared, 400_000, code=0x40)
    with pytest.raises(b.TyphoonMLAError) as e:
        b.typhoon_mla_check_status(dec.shared)
    assert e.value.status == 6
    word = b.typhoon_mla_check_status(dec.shared, clear=True, raise_on_error=False)
    assert word == 0x40 and (word & b.STATUS_WAIT_EXPIRED) and not (word & b.STATUS_BAD_PAGE)
    assert b.typhoon_mla_check_status(dec.shared) == 0
    lse = torch.empty(inp.cfg.B, inp.cfg.H, dtype=torch.float32, device="cuda")
    out = dec.decode(inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), pc.block_table.cuda(),
                     pc.seq_lens.cuda(), mode=HYBRID, lse_out=lse)
    assert b.typhoon_mla_check_status(dec.shared) == 0
    G.assert_parity(out.float().cpu().double().numpy(), ref, lse.cpu().double().numpy(), ref_lse, what="after an expired wait")
    dec.close()


def test_workspace_query_is_pure_while_switches_flip_and_steps_run():
    """typhoon_mla_workspace_bytes from two threads, a third thread flipping the kernel-path, schedule and
    overlap switches, the main thread decoding: the query always returns the same number (it reads no
    process-wide state), every step plans and launches from one snapshot of the switches (results stay
    right, nothing is written outside the workspace: a guard band behind it keeps its pattern)."""
    from paper_2509_21081_b200 import binding as b
    cfg = _cfg("threads", B=70, H=32, Ls=1500, lo=0, hi=300, seed=97)
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp, poison=True)
    ref, _ = G.run_oracle(inp)
    dec = _decoder(inp, pc)
    mp = pc.block_table.shape[1]
    expect = b.typhoon_mla_workspace_bytes(dec.shared, cfg.B, mp, 64)
    per_mode = [b.typhoon_mla_workspace_bytes(dec.shared, cfg.B, mp, 64, m) for m in (ABSORB, HYBRID, NAIVE)]
    assert expect == max(per_mode) and min(per_mode) > 0 and per_mode[2] < per_mode[1]
    guard = 1 << 16
    ws_all = torch.full((expect + guard,), 0x5A, dtype=torch.uint8, device="cuda")
    ws = ws_all[:expect]
    stop = threading.Event()
    bad = []

    def query():
        while not stop.is_set():
            if b.typhoon_mla_workspace_bytes(dec.shared, cfg.B, mp, 64) != expect:
                bad.append("size changed")

    def flip():
        k = 0
        while not stop.is_set():
            k += 1
            b.typhoon_mla_set_kernel_path(k % 2)
            b.typhoon_mla_set_naive_schedule(k % 3)
            b.typhoon_mla_set_overlap(bool(k % 5))

    threads = [threading.Thread(target=query), threading.Thread(target=query), threading.Thread(target=flip)]
    for t in threads:
        t.start()
    try:
        args = (inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), 64, pc.block_table.cuda(),
                pc.seq_lens.cuda(), inp.scale)
        out = torch.empty(cfg.B, cfg.H, 128, dtype=torch.bfloat16, device="cuda")
        for it in range(60):
            b.typhoon_mla_decode(dec.shared, *args, out, ws, mode=(HYBRID, ABSORB)[it % 2])
            if it % 10 == 9:
                assert b.typhoon_mla_check_status(dec.shared) == 0
                G.assert_parity(out.float().cpu().double().numpy(), ref, what=f"step {it} under flipping switches")
    finally:
        stop.set()
        for t in threads:
            t.join()
        b.typhoon_mla_set_kernel_path(b.PATH_TCGEN05)
        b.typhoon_mla_set_naive_schedule(0)
        b.typhoon_mla_set_overlap(True)
    torch.cuda.synchronize()
    assert not bad
    assert bool((ws_all[expect:] == 0x5A).all()), "a step wrote behind its workspace"
    dec.close()


def test_scale_and_mode_checks():
    from paper_2509_21081_b200 import binding as b
    cfg = _cfg("checks", B=2, H=16, Ls=64, lo=8, hi=8, seed=98)
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp)
    dec = _decoder(inp, pc)
    out = torch.empty(2, 16, 128, dtype=torch.bfloat16, device="cuda")
    args = (inp.q_nope.cuda(), inp.q_pe.cuda(), pc.ckv_pages.cuda(), pc.kpe_pages.cuda(), 64, pc.block_table.cuda(),
            pc.seq_lens.cuda())
    for scale in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(b.TyphoonMLAError) as e:
            b.typhoon_mla_decode(dec.shared, *args, scale, out, dec.workspace, mode=HYBRID)
        assert e.value.status == 1
    with pytest.raises(b.TyphoonMLAError) as e:
        b.typhoon_mla_decode(dec.shared, *args, inp.scale, out, dec.workspace, mode=7)
    assert e.value.status == 1
    assert b.typhoon_mla_workspace_bytes(dec.shared, 2, 1, 64, 9) == 0
    dec.close()
