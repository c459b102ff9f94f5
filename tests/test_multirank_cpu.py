"""Host-side logic of the N > 1 bench path (independent replicas, max-over-ranks timing) on CPU:
two gloo ranks, no GPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = 10.0 + 5.0 * rank                       # rank 1 is slower: the job takes its time
        ms_max = bench.max_over_ranks(ms)
        # each replica draws its own seeded problem: different seeds, same shapes
        from paper_2510_13161_b200 import inputs as I
        x = I.gen_verify_inputs(I.CONFIGS["tiny"], 100 + rank, "cpu")
        sig = float(x.q.float().sum())
        sigs = [None] * world
        dist.all_gather_object(sigs, sig)
        out[rank] = (ms_max, bench.job_throughput(20, world, ms_max), sigs)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_time_and_sum_the_work():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        ms_max, thr, sigs = res[rank]
        assert ms_max == 15.0                          # max over ranks, seen by every rank
        assert abs(thr - 2 * 20 * 1e3 / 15.0) < 1e-9   # whole-job throughput: both replicas' steps over the max time
        assert sigs[0] != sigs[1]                      # replicas work on different problems


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.job_throughput(10, 1, 5.0) == 2000.0


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment re-runs itself under torch.distributed.run on
    127.0.0.1; the launch path (process group, barrier, max over ranks, one line from rank 0) is checked without a GPU."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "20", "--rendezvous-only"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                         # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["requested_gpus"] == 2
    assert line["ms_max"] == 15.0                                   # the slower rank's time
    assert abs(line["value"] - 2 * 20 * 1e3 / 15.0) < 1e-9
