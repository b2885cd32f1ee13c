"""The multi-GPU form of the benchmark is N independent replicas (rows never interact across
sequences), so the only cross-rank logic is host-side: the slowest rank's time, the whole-job value,
distinct input batches per rank, and the reference arm running on rank 0 only.  Checked here with two
gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    import workloads as W
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    cfg = W.tiny_config(N=64, n=8, rows=2)
    a = W.make_inputs(cfg, variant=0 + 100 * rank)["target"]
    gathered = [torch.zeros_like(a) for _ in range(world)]
    dist.all_gather(gathered, a)
    q.put((rank, ms, bool(torch.equal(gathered[0], gathered[1]))))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_timing_and_distinct_batches():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]          # both ranks see the slowest rank's time
    assert not res[0][2]                                # the ranks draw different batches
    sys.path.insert(0, ROOT)
    import bench
    assert bench.whole_job_value(320, 1, 10, 2, 15.0) == 2 * 320 * 10 / 0.015


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29611")
    outs = []
    for rank in (0, 1):
        env["RANK"] = str(rank)
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr[-500:]
        outs.append(r.stdout.strip())
    assert outs[1] == ""
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"


def test_timed_region_is_long_enough_whatever_the_step_count():
    """The benchmark repeats its K-step loop until half a second has been timed and at least five times,
    and reports the median; a handful of steps of a 50 microsecond kernel must not be the whole record."""
    import bench
    assert bench.repeats_for(0.05, 20) == 500          # 20 steps of 0.05 ms: 1 ms per loop
    assert bench.repeats_for(0.05, 2000) == 5          # 100 ms per loop: the minimum of five
    assert bench.repeats_for(0.4, 100) == 13
    assert bench.repeats_for(1e-9, 1) == 2000          # capped
    med, spread = bench.median_and_spread([1.0, 1.2, 0.9, 1.1, 1.0])
    assert med == 1.0 and abs(spread - 0.3) < 1e-12
    med, _ = bench.median_and_spread([2.0, 4.0])
    assert med == 3.0
