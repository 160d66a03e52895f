"""World-size-2 plumbing on CPU (gloo): the path has no data-path collective, so what N > 1
needs is the rank bookkeeping around it - max-over-ranks timing, summed units, and the
reference arm printing from rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    # every rank scans the same number of units; the job's time is the slowest rank's
    ms = torch.tensor([10.0 + 5.0 * rank])
    agg = bench.aggregate_over_ranks(ms_local=float(ms), units_local=1000.0, dist=dist, device="cpu")
    out.put((rank, agg))
    dist.barrier()
    dist.destroy_process_group()


def test_weak_scaling_aggregation_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    ps = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    res = dict(q.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(2):
        ms, units = res[r]
        assert ms == 15.0 and units == 2000.0


def test_reference_arm_prints_once_under_two_ranks():
    """bench.py --impl reference with WORLD_SIZE=2: rank 0 prints the JSON line, rank 1 exits 0 silently."""
    outs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT="29999", CUDA_VISIBLE_DEVICES="")
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--steps", "1", "--warmup", "0", "--workload", "config1", "--ref-elements", "2e6"],
                           capture_output=True, text=True, env=env, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        outs.append(r.stdout.strip())
    assert outs[1] == ""
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
