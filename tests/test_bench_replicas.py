"""The N > 1 path of bench.py on CPU: the path shards over independent sequences
(replicas only), so what there is to test is the aggregation over ranks and the
launch contract of the reference arm.  gloo, world size 2, 127.0.0.1."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank r took (10 + 5 r) ms for (100 + r) tokens, and (1 + r) s end to end for (7 + r) tokens, with 1000 launches
    times, counts = bench.aggregate_over_ranks(dist, torch.device("cpu"), [10.0 + 5.0 * rank, 1.0 + rank],
                                               [100 + rank, 7 + rank, 1000])
    dist.barrier()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"times": times, "counts": counts}, f)
    dist.destroy_process_group()


def test_aggregation_is_max_time_and_summed_work(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        got = json.load(open(tmp_path / f"rank{rank}.json"))
        assert got["times"] == [15.0, 2.0]          # the slowest rank
        assert got["counts"] == [201, 15, 2000]     # all ranks' tokens and launches
    # whole-job throughput = summed tokens / slowest time, as bench.py prints it
    assert 201 / (15.0 / 1000.0) == 13400.0


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "sampler",
           "--gpus", "2", "--steps", "1", "--warmup", "0", "--cpu-budget", "0.5"]
    done = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert done.returncode == 0, done.stderr[-2000:]
    lines = [l for l in done.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["value"] > 0
    assert out["cpu_baseline"]["kind"] == "oracle" and out["e2e"]["h2d_bytes_per_step"] == 0
