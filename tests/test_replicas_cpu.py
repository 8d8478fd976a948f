"""The multi-process side of the benchmark, on CPU: with N > 1 the job is N independent replicas (the DDG iteration
does not shard across GPUs here), so the only cross-rank step is the maximum of the ranks' durations.  World size 2
over gloo checks that reduction and the whole-job throughput; a torchrun launch checks that the reference arm prints
one line, from rank 0 alone."""
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


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    mine = [1.0 + 0.5 * rank, 3.0 - rank]          # rank 0: 1.0, 3.0; rank 1: 1.5, 2.0
    got = bench.max_over_ranks(mine, dist, "cpu")
    dist.barrier()
    dist.destroy_process_group()
    json.dump(got, open(os.path.join(out_dir, "r%d.json" % rank), "w"))


def test_max_over_ranks_world_size_2(tmp_path):
    port = _free_port()
    mp.start_processes(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True, start_method="spawn")
    r0, r1 = (json.load(open(tmp_path / ("r%d.json" % r))) for r in (0, 1))
    assert r0 == r1 == [1.5, 3.0]                   # every rank holds the slowest replica's time


def test_single_process_is_the_identity_and_throughput_adds_up():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([0.25, 2.0], None, "cpu") == [0.25, 2.0]
    # two replicas of 128 images x 10 iterations in 0.5 s: 5120 images/s for the whole job
    assert bench.job_throughput(128, 10, 2, 0.5) == 5120.0


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--net", "resnet8", "--cpu-batch", "2", "--steps", "1", "--warmup", "0"]
    env = dict(os.environ, OMP_NUM_THREADS="2")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
