"""The N > 1 path of bench.py on CPU: two gloo ranks.  The path shards by request with no data-path
collective; the only exchange is the MAX over ranks of the step time.  Checked here: ranks draw different
requests but the same shapes, the slowest rank's time is what every rank sees, the whole-job value counts
all ranks' queries, and the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_q):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2509_21081_b200 import inputs as I
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = I.MLAConfig("t", B=3, H=16, Ls=64, suffix_lo=1, suffix_hi=9, seed=5)
    rcfg = bench.rank_config(cfg, rank)
    inp = I.make_inputs(rcfg)
    my_ms = 10.0 + 5.0 * rank                      # rank 1 is slower
    worst = bench.max_over_ranks(my_ms, world, "cpu")
    value = bench.whole_job_value(cfg.B, world, worst)
    out_q.put((rank, rcfg.seed, tuple(inp.q_nope.shape), float(inp.q_nope.float().sum()), worst, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 500)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, shape0, sum0, worst0, val0), (r1, seed1, shape1, sum1, worst1, val1) = res
    assert (r0, r1) == (0, 1) and seed0 == 5 and seed1 == 1005
    assert shape0 == shape1 and sum0 != sum1            # same shapes, different requests
    assert worst0 == worst1 == 15.0                     # slowest rank decides
    assert abs(val0 - 2 * 3 / 15e-3) < 1e-9 and val0 == val1


def test_reference_arm_prints_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg0",
                        "--steps", "1", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg0",
                        "--steps", "1", "--warmup", "1", "--gpus", "2"], capture_output=True, text=True, env=env, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


def _shard_worker(rank, world, port, out_q):
    """One rank of a sequence-sharded step on CPU: the float64 checker stands in for the device's partial
    step, the library's planning functions and communicator do the rest."""
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import mla_oracle as O
    from paper_2509_21081_b200 import inputs as I, sharded as S
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    comm = S.TorchDistComm()
    cfg = I.MLAConfig("t", B=5, H=16, Ls=200, suffix_lo=0, suffix_hi=40, seed=9)
    inp = I.make_inputs(cfg)                         # every rank draws the same problem
    f = I.to_f64
    b0, b1 = S.sequence_slices(cfg.Ls, world)[rank]
    lens = S.local_seq_lens(torch.tensor([x.shape[0] for x in inp.ckv_suffix]), rank, world)
    ckv_suf = [f(x[:int(n)]) for x, n in zip(inp.ckv_suffix, lens)]
    kpe_suf = [f(x[:int(n)]) for x, n in zip(inp.kpe_suffix, lens)]
    o, lse = O.mla_decode(f(inp.q_nope), f(inp.q_pe), f(inp.ckv_shared)[b0:b1], f(inp.kpe_shared)[b0:b1], ckv_suf, kpe_suf,
                          f(inp.w_uk), f(inp.w_uv), inp.scale)
    o_parts = comm.all_gather(torch.from_numpy(o)).numpy()          # [world, B, H, 128]
    lse_parts = comm.all_gather(torch.from_numpy(lse)).numpy()
    merged = np.empty_like(o)
    for b in range(cfg.B):
        for h in range(cfg.H):
            merged[b, h], _ = O.combine_lse([o_parts[r, b, h] for r in range(world)], [float(lse_parts[r, b, h]) for r in range(world)])
    full, _ = O.mla_decode(f(inp.q_nope), f(inp.q_pe), f(inp.ckv_shared), f(inp.kpe_shared), [f(x) for x in inp.ckv_suffix],
                           [f(x) for x in inp.kpe_suffix], f(inp.w_uk), f(inp.w_uv), inp.scale)
    # head sharding: gather this rank's heads and put them back in order
    h0, h1 = S.head_slice(32, rank, world)
    heads = comm.all_gather(torch.arange(h0, h1).view(1, -1, 1).expand(2, -1, 3).contiguous())
    out_q.put((rank, (b0, b1), float(np.max(np.abs(merged - full))), S.join_heads(heads)[0, :, 0].tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_sequence_and_head_sharding_two_ranks_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 30100 + (os.getpid() % 500)
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [(0, 128), (128, 200)]
    assert all(r[2] < 1e-12 for r in res)                  # partials merged over ranks = the whole context
    assert all(r[3] == list(range(32)) for r in res)       # heads come back in order on every rank


def test_shard_plans():
    from paper_2509_21081_b200 import sharded as S
    for Ls in (0, 1, 63, 64, 65, 130, 1000, 4096, 26624):
        for world in (1, 2, 3, 4, 8):
            sl = S.sequence_slices(Ls, world)
            assert len(sl) == world and sl[0][0] == 0 and sl[-1][1] == Ls
            assert all(a[1] == b[0] for a, b in zip(sl, sl[1:]))           # contiguous, in order
            assert all((b0 % 64 == 0 or b0 == b1) and b0 <= b1 for b0, b1 in sl)   # empty slices may sit at Ls
            sizes = [-(-(b1 - b0) // 64) for b0, b1 in sl]
            assert max(sizes) - min(sizes) <= 1
    lens = torch.tensor([5, 0, 7, 9, 11])
    parts = [S.local_seq_lens(lens, r, 3) for r in range(3)]
    assert torch.equal(sum(parts), lens) and all(int((p > 0).sum()) <= 2 for p in parts)
    assert [S.request_owner(b, 3) for b in range(5)] == [0, 1, 2, 0, 1]
    assert S.head_slice(128, 3, 4) == (96, 128)
    import pytest
    with pytest.raises(ValueError):
        S.head_slice(64, 0, 8)    # 8 heads per rank: below the library's granularity
