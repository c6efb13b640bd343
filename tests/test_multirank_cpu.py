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
