"""The N > 1 path of bench.py (independent replicas, max over ranks) on CPU: 2 gloo ranks."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 if rank == 0 else 20.0          # the timed region took 10 ms on rank 0, 20 ms on rank 1
    total = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    us = bench.us_per_layer_step(total, steps=5, world=world)
    dist.barrier()
    dist.destroy_process_group()
    open(os.path.join(out, f"r{rank}.txt"), "w").write(f"{total} {us}")


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_rank, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        total, us = map(float, open(tmp_path / f"r{r}.txt").read().split())
        assert total == 20.0                     # the slowest rank decides
        assert abs(us - 20.0e3 / (5 * 2)) < 1e-9 # 2 replicas x 5 layer-steps in 20 ms


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.us_per_layer_step(2.0, 4, 1) == 500.0


def test_bench_started_plainly_with_gpus_2_starts_two_ranks_itself():
    """`python bench.py --gpus 2` outside torchrun (how the single-GPU arm is invoked) must not run one
    replica and call it two: it starts the two ranks itself on 127.0.0.1.  Run here without a GPU through
    the CPU self-test mode, which goes through the same start-up, process group (gloo), barrier, max
    over ranks and aggregate; rank r pretends its timed region took 10 (r + 1) ms per step."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-cpu", "--steps", "5"],
                       capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                              # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["steps"] == 5
    assert line["slowest_rank_total_ms"] == 100.0       # rank 1: 5 steps x 20 ms
    assert abs(line["value"] - 100.0e3 / (5 * 2)) < 1e-9   # 2 replicas x 5 layer-steps in 100 ms
