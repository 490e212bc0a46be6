"""The N > 1 path of bench.py on CPU: two gloo ranks.  The data path has no collective (every
rank runs its own independent copy of the workload); what is shared is the bookkeeping: distinct
inputs per rank, the max-over-ranks time, the whole-job value, and rank 0 alone reporting."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    worst = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
    seeds = [bench.rank_layer_seed_offset(rank, layer) for layer in range(bench.LAYERS)]
    gathered = [None] * world
    dist.all_gather_object(gathered, seeds)
    if rank == 0:
        out.put((worst, gathered, bench.whole_job_value(1e12, worst, world)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_share_only_the_bookkeeping():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    worst, gathered, value = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert worst == 15.0                                   # the slowest rank sets the time
    assert not set(gathered[0]) & set(gathered[1])         # no two ranks draw the same layer inputs
    assert abs(value - 2 * 1e12 / 15e-3 / 1e12) < 1e-9     # both ranks' work over that time


def test_reference_arm_prints_one_line_from_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    r1 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--steps", "1", "--warmup", "0"], env=dict(env, RANK="1", LOCAL_RANK="1"),
                        capture_output=True, text=True, timeout=600)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                         "--steps", "1", "--warmup", "0"], env=dict(env, RANK="0", LOCAL_RANK="0"),
                        capture_output=True, text=True, timeout=600)
    assert r0.returncode == 0, r0.stderr
    lines = [x for x in r0.stdout.splitlines() if x.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


def test_bare_gpus_flag_spawns_its_own_ranks():
    """`bench.py --gpus 2` with no launcher around it starts two ranks itself (torch.distributed.run,
    rendezvous on 127.0.0.1); the reference arm needs no GPU, so this runs here: one line, n_gpus 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR",
                                                           "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [x for x in r.stdout.splitlines() if x.strip().startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
