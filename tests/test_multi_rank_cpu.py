"""The N > 1 path of bench.py on CPU: two gloo ranks.  The hot path has no exchange step (every rank
processes its own batches), so what the ranks share is the timing protocol: a barrier, the maximum
of the per-rank device times, and a whole-job throughput computed from it by rank 0."""
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


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2607_04302_b200 import synth
    cfg = synth.config("C2")
    my_ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
    dist.barrier()
    total = bench.max_over_ranks(dist, my_ms, torch.device("cpu"))
    value = bench.whole_job_tflops(cfg, world, 5, total)
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(f"{total} {value}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_slowest_time(tmp_path):
    world = 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    import bench
    from paper_2607_04302_b200 import synth
    cfg = synth.config("C2")
    vals = [open(tmp_path / f"r{r}.txt").read().split() for r in range(world)]
    assert all(float(v[0]) == 20.0 for v in vals)              # max over ranks, seen by both
    expect = 2 * bench.attn_flops(cfg) * 5 / 20e-3 / 1e12       # two copies of the workload in the slowest time
    assert all(abs(float(v[1]) - expect) < 1e-9 * expect for v in vals)
    # one rank alone: no collective, value halves for the same time
    assert bench.max_over_ranks(None, 20.0, None) == 20.0
    assert abs(bench.whole_job_tflops(cfg, 1, 5, 20.0) - expect / 2) < 1e-9 * expect
