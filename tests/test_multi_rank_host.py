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


def _self_started_rank(out_dir):
    """Runs in every rank that bench.launch_ranks starts: the rendezvous variables are in the
    environment, as a launcher would have set them."""
    import json
    sys.path.insert(0, ROOT)
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert int(os.environ["LOCAL_RANK"]) == rank and os.environ["MASTER_ADDR"] == "127.0.0.1"
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(3.0 + rank, dist, torch.device("cpu"))
    with open(os.path.join(out_dir, f"{rank}.json"), "w") as f:
        json.dump({"rank": rank, "world": world, "ms": ms}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_bench_starts_its_own_ranks_when_no_launcher_did(tmp_path):
    """`python bench.py --gpus N` without torchrun: bench.launch_ranks starts the N ranks itself, each
    with RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* set, and they form one process group."""
    import json
    sys.path.insert(0, ROOT)
    import bench
    saved = {k: os.environ.get(k) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    bench.launch_ranks(2, _self_started_rank, (str(tmp_path),))
    assert {k: os.environ.get(k) for k in saved} == saved          # the parent's environment is untouched
    res = [json.load(open(tmp_path / f"{r}.json")) for r in range(2)]
    assert [r["rank"] for r in res] == [0, 1] and all(r["world"] == 2 for r in res)
    assert res[0]["ms"] == res[1]["ms"] == 4.0
