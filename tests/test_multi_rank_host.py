"""Host-side logic of the multi-GPU bench (replicas, one independent long input per rank): two
gloo ranks on the CPU agree on the slowest rank's time, draw different inputs, and report the
whole-job value."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2506_01215_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    w = synth.WORKLOADS["tiny"]
    qkv = synth.chunk_qkv(w, 0, 0, seed=bench.rank_seed(w, rank))
    value = bench.job_throughput(w, world, ms)
    q.put((rank, ms, float(qkv[0].double().sum()), value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_slowest_time_and_use_distinct_inputs():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == 15.0                  # max over ranks
    assert res[0][2] != res[1][2]                          # independent inputs per rank
    w_tokens = 8192
    assert abs(res[0][3] - 2 * w_tokens / 15e-3) < 1e-6    # whole-job tokens/s
    assert res[0][3] == res[1][3]
