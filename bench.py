#!/usr/bin/env python
"""Benchmark of the REFORM compress-and-gather hot path on B200.

One "step" is one pass of the whole path over one synthetic long input of the
Llama-3-8B-shaped single-layer workload (131,072-token context): 4 recurrent
chunk steps (reform_chunk_step -> reform_embed_append -> reform_evict_topk),
then reform_retrieve_topk over the bank the pass just wrote and reform_gather
of the selected rows.  The headline value is context tokens per second per
layer; the JSON line also carries the retrieval+gather GB/s, the roofline of
the dominant kernel (the chunk-step attention) and the CPU oracle timed on a
bounded sample of the same workload.

  python bench.py --gpus N --steps K --warmup W          (this library)
  python bench.py --impl reference ...                    (the CPU oracle arm)
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2506_01215_b200 import synth  # noqa: E402

METRIC = "chunk-step context tokens/s/layer"
UNIT = "tokens/s/layer"
WORKLOAD = "llama8b_128k"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--force-simt", action="store_true", help="time the CUDA-core chunk step")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], tflops=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    source="measured (MEASURED_PEAKS.json, sustained bf16 / copy GB/s)")
    return dict(hbm_gbs=6650.0, tflops=1400.0, source="fallback")


# ------------------------------------------------------------------ work model

def attn_pairs(w, step):
    """Visible (query, key) pairs per query head in recurrence step `step`."""
    n_cache = 0 if step == 0 else w.budget
    return w.Lc * n_cache + w.Lc * (w.Lc + 1) // 2


def attn_flops(w, step):
    return 4 * w.B * w.Hq * w.d * attn_pairs(w, step)


# DRAM bytes the attention kernel moved per algorithmic byte (Q + K + V + O) in the ncu capture of
# the small case (profiles/attn2_sm100_kernel_lc8192.md): 174.7 MB / 201.3 MB.
ATTN_DRAM_RATIO = 0.87


def attn_bytes(w):
    sz = 2 if w.dtype == torch.bfloat16 else 4
    return w.B * sz * w.d * (2 * w.Hq * w.Lc + 2 * w.Hkv * (w.budget + w.Lc))


def retrieval_gather_bytes(w):
    sz = 2 if w.dtype == torch.bfloat16 else 4
    return w.B * (w.N * w.E * sz + 2 * w.k * w.D * sz)


# ------------------------------------------------------------------ ranks

def rank_seed(w, rank):
    """Each rank processes its own independent long input."""
    return w.seed + 1000 * rank


def max_over_ranks(ms, dist, device):
    """The job's step time is the slowest rank's."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def job_throughput(w, world, ms):
    """Whole-job context tokens per second per layer: every rank walked B*T tokens in ms."""
    return world * w.B * w.T / (ms * 1e-3)


# ------------------------------------------------------------------ clocks

class ClockSampler:
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the two wall-clock times (all if None)."""
        import datetime
        if self.proc is None:
            return None
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                clk, clk_max, power = float(f[1]), float(f[2]), float(f[3])
            except ValueError:
                continue
            if t_begin is not None and not (t_begin <= ts <= t_end):
                continue
            sm.append(clk)
            mx.append(clk_max)
            pw.append(power)
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w": statistics.median(pw),
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ our arm

class Pass:
    """Device-resident inputs and buffers of one pass, and the pass itself."""

    def __init__(self, w, dev, seed_offset=0, force_simt=False):
        import paper_2506_01215_b200 as R
        self.R, self.w, self.dev = R, w, dev
        self.flags = R.SCORE_ACCUMULATE | (R.FORCE_SIMT if force_simt else 0)
        seed = rank_seed(w, seed_offset)
        S = w.steps
        self.q, self.kc, self.vc = [], [], []
        # one K/V/score buffer set per recurrence step: the chunk's rows are already in place
        # behind the slot the previous eviction fills, so no copy sits in the timed region
        self.k = [torch.zeros(w.B, w.Hkv, w.cap, w.d, dtype=w.dtype, device=dev) for _ in range(S + 1)]
        self.v = [torch.zeros(w.B, w.Hkv, w.cap, w.d, dtype=w.dtype, device=dev) for _ in range(S + 1)]
        self.score = [torch.zeros(w.B, w.Hkv, w.cap, dtype=torch.float32, device=dev) for _ in range(S + 1)]
        for s in range(S):
            q, kc, vc = synth.chunk_qkv(w, 0, s, device=dev, seed=seed)
            n_cache = 0 if s == 0 else w.budget
            self.q.append(q)
            self.kc.append(kc)
            self.vc.append(vc)
            self.k[s][:, :, n_cache:n_cache + w.Lc] = kc
            self.v[s][:, :, n_cache:n_cache + w.Lc] = vc
        self.out = torch.empty(w.B, w.Hq, w.Lc, w.d, dtype=w.dtype, device=dev)
        self.lse = torch.empty(w.B, w.Hq, w.Lc, dtype=torch.float32, device=dev)
        self.kept = torch.empty(w.B, w.Hkv, w.budget, dtype=torch.int32, device=dev)
        self.bank = torch.zeros(w.B, w.N, w.E, dtype=w.dtype, device=dev)
        self.sel = synth.head_selection(w)
        _, self.queries, _ = synth.bank_and_queries(dataclasses.replace(w, N=256, n_planted=0),
                                                    device=dev, seed=seed)
        self.hidden = synth.hidden_rows(w, device=dev, seed=seed)
        self.idx = torch.zeros(w.B, w.k, dtype=torch.int32, device=dev)
        self.gathered = torch.empty(w.B, w.k, w.D, dtype=w.dtype, device=dev)
        self.events = []

    def _timed(self, name, fn, record):
        if record:
            a = torch.cuda.Event(enable_timing=True)
            b = torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            self.events.append((name, a, b))
        else:
            fn()

    def step(self, s, record=False):
        """Recurrence step s: chunk step, embedding append, eviction into the next buffer set."""
        R, w = self.R, self.w
        n_cache = 0 if s == 0 else w.budget
        self._timed(f"chunk_step{s}", lambda: R.chunk_step(
            self.q[s], self.k[s], self.v[s], self.out, self.score[s], n_cache, w.window,
            lse=self.lse, flags=self.flags), record)
        self._timed("embed_append", lambda: R.embed_append(
            self.bank, s * w.Lc, self.sel, q_state=self.q[s], k_state=self.kc[s],
            v_state=self.vc[s]), record)
        self._timed("evict_topk", lambda: R.evict_topk(
            self.k[s], self.v[s], self.score[s], self.k[s + 1], self.v[s + 1], self.score[s + 1],
            n_cache + w.Lc, w.budget, w.n_sink, w.n_recent, kept_idx=self.kept), record)

    def tail(self, record=False, hidden=None):
        """Gather phase: retrieval over the bank the steps wrote, then the row gather (from
        `hidden` if given: a pinned host copy of the rows, read in place by the kernel)."""
        R, w = self.R, self.w
        src = self.hidden if hidden is None else hidden
        self._timed("retrieve_topk", lambda: R.retrieve_topk(
            self.bank, self.queries, w.N, w.k, self.idx, scale=w.sim_scale,
            pool_window=w.pool_window, n_keep_head=w.keep_head, n_keep_tail=w.keep_tail), record)
        self._timed("gather", lambda: R.gather(src, self.idx, self.gathered), record)

    def run(self, record=False):
        for s in range(self.w.steps):
            self.step(s, record)
        self.tail(record)

    def breakdown(self):
        agg = {}
        for name, a, b in self.events:
            agg.setdefault(name, []).append(a.elapsed_time(b))
        self.events = []
        return agg


class HostPipeline:
    """The same pass driven from pinned host buffers: every recurrence step's Q/K/V and the query
    embeddings are copied to the device inside the timed region, the gather reads its rows
    straight out of the pinned host copy of the gather source (only the selected rows cross
    PCIe), and the gathered rows and their indices are read back.  Copies run on their own stream
    one step ahead of the kernels, and two device buffer sets alternate between consecutive
    passes, so a pass's transfers overlap the previous pass's kernels the way a serving loop
    streams inputs."""

    def __init__(self, passes):
        self.sets = passes
        p = passes[0]
        w = p.w
        pin = lambda t: t.cpu().pin_memory()
        self.hq = [pin(x) for x in p.q]
        self.hk = [pin(x) for x in p.kc]
        self.hv = [pin(x) for x in p.vc]
        self.hqueries = pin(p.queries)
        self.hhidden = pin(p.hidden)
        self.hout = torch.empty(p.gathered.shape, dtype=w.dtype).pin_memory()
        self.hidx = torch.empty(p.idx.shape, dtype=torch.int32).pin_memory()
        self.h2d = sum(t.numel() * t.element_size() for t in self.hq + self.hk + self.hv) + \
            self.hqueries.numel() * self.hqueries.element_size() + \
            p.gathered.numel() * p.gathered.element_size()      # the rows the gather kernel pulls
        self.d2h = self.hout.numel() * self.hout.element_size() + self.hidx.numel() * 4
        self.copy_stream = torch.cuda.Stream()
        self.done = [None] * len(passes)
        self.count = 0

    def run(self):
        i = self.count % len(self.sets)
        self.count += 1
        p, w = self.sets[i], self.sets[i].w
        main, cs = torch.cuda.current_stream(), self.copy_stream
        ready = [torch.cuda.Event() for _ in range(w.steps + 1)]
        with torch.cuda.stream(cs):
            if self.done[i] is not None:
                cs.wait_event(self.done[i])          # this buffer set's previous pass has finished
            else:
                cs.wait_stream(main)
            for s in range(w.steps):
                p.q[s].copy_(self.hq[s], non_blocking=True)
                p.kc[s].copy_(self.hk[s], non_blocking=True)
                p.vc[s].copy_(self.hv[s], non_blocking=True)
                ready[s].record(cs)
            p.queries.copy_(self.hqueries, non_blocking=True)
            ready[w.steps].record(cs)
        R = p.R
        for s in range(w.steps):
            n_cache = 0 if s == 0 else w.budget
            main.wait_event(ready[s])
            p.k[s][:, :, n_cache:n_cache + w.Lc].copy_(p.kc[s])
            p.v[s][:, :, n_cache:n_cache + w.Lc].copy_(p.vc[s])
            p.step(s)
        main.wait_event(ready[w.steps])
        p.tail(hidden=self.hhidden)
        self.hout.copy_(p.gathered, non_blocking=True)
        self.hidx.copy_(p.idx, non_blocking=True)
        self.done[i] = torch.cuda.Event()
        self.done[i].record(main)


def cpu_baseline(w, sample_rows=8192):
    """The oracle, as it stands, on a bounded sample: one KV-head group of recurrence step 1,
    every (Lc/sample_rows)-th query row for the attention output plus the full 128-row score
    window.  Extrapolated to the metric through (query, key) pairs per second."""
    import oracle
    G = w.Hq // w.Hkv
    ws = dataclasses.replace(w, B=1, Hq=G, Hkv=1)
    q, kc, vc = synth.chunk_qkv(ws, 0, 1)
    k0, v0, _ = synth.cache_state(ws, 0)
    k = torch.cat([k0, kc], 2).contiguous()
    v = torch.cat([v0, vc], 2).contiguous()
    stride = max(1, w.Lc // sample_rows)
    rows = list(range(0, w.Lc, stride))
    t0 = time.perf_counter()
    oracle.attention(q, k, v, w.budget, rows=rows)
    oracle.key_scores(q, k, w.budget, w.window)
    dt = time.perf_counter() - t0
    pairs = G * sum(w.budget + r + 1 for r in rows)
    pairs += 2 * G * sum(w.budget + (w.Lc - w.window + i) + 1 for i in range(w.window))
    pairs_per_s = pairs / dt
    total_pairs = w.B * w.Hq * sum(attn_pairs(w, s) for s in range(w.steps))
    value = w.B * w.T / (total_pairs / pairs_per_s)
    return {"value": value, "unit": UNIT, "cores": oracle.get_threads(), "kind": "oracle",
            "sample": (f"step 1 of {w.name}: 1 KV-head group ({G} query heads), {len(rows)} of {w.Lc} "
                       f"query rows (every {stride}th) + the {w.window}-row score window, "
                       f"{pairs / 1e9:.2f} G pairs in {dt:.1f} s; extrapolated by pairs/s to all heads and steps"),
            "seconds": dt}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(min(args.warmup, 1)):
        cpu_baseline(w, sample_rows=64)
    vals, secs = [], []
    for _ in range(args.steps):
        r = cpu_baseline(w, sample_rows=512)
        vals.append(r["value"])
        secs.append(r["seconds"])
    value = statistics.mean(vals)
    r["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.B * w.T / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": w.name, "note": "CPU oracle on a bounded sample per step"},
            "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    args = parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return
    import paper_2506_01215_b200 as R
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    R.lib()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # each rank processes its own independent long input (weak scaling, no data-path collective)
    p = Pass(w, dev, seed_offset=rank, force_simt=args.force_simt)
    for _ in range(max(args.warmup, 3)):
        p.run()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        t_up = time.time()
        while time.time() - t_up < 1.0:   # keep the GPU under load while the sampler comes up
            p.run()
            torch.cuda.synchronize()
    n0 = R.kernel_launch_count()
    start = torch.cuda.Event(enable_timing=True)
    end = torch.cuda.Event(enable_timing=True)
    barrier()
    n0 = R.kernel_launch_count()
    wall0 = time.time()
    start.record()
    for _ in range(args.steps):
        p.run(record=True)
    end.record()
    barrier()
    wall1 = time.time()
    ms_total = start.elapsed_time(end)
    launches = R.kernel_launch_count() - n0
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    ms_total = max_over_ranks(ms_total, dist, dev)
    ms = ms_total / args.steps
    bd = p.breakdown()

    # end-to-end arm: host buffers, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        hp = HostPipeline([p, Pass(w, dev, seed_offset=rank, force_simt=args.force_simt)])
        hp.run()
        hp.run()
        barrier()
        start.record()
        for _ in range(args.steps):
            hp.run()
        end.record()
        barrier()
        ms_e2e = start.elapsed_time(end)
        ms_e2e = max_over_ranks(ms_e2e, dist, dev) / args.steps
        e2e = {"value": job_throughput(w, world, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": hp.h2d, "d2h_bytes_per_step": hp.d2h,
               "gather_source": "pinned host memory; reform_gather reads the selected rows in place"}
    dev_err = R.device_error()
    if dev_err:
        raise RuntimeError(f"a kernel reported device error bits {dev_err} during the benchmark")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    pk = peaks()
    mean = lambda xs: sum(xs) / len(xs)
    chunk_ms = [mean(bd[f"chunk_step{s}"]) for s in range(w.steps)]
    flops = sum(attn_flops(w, s) for s in range(w.steps))
    achieved = flops / (sum(chunk_ms) * 1e-3) / 1e12
    t_rg = (mean(bd["retrieve_topk"]) + mean(bd["gather"])) * 1e-3
    sz = 2 if w.dtype == torch.bfloat16 else 4
    evict_bytes = w.B * w.Hkv * ((w.budget + w.Lc) * 4 + 4 * w.budget * w.d * sz + 8 * w.budget)
    embed_bytes = 2 * w.B * w.Lc * w.E * sz
    line = {
        "metric": METRIC, "value": job_throughput(w, world, ms), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.dtype == torch.bfloat16 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "context_tokens": w.T, "chunk": w.Lc, "kv_budget": w.budget,
                   "Hq": w.Hq, "Hkv": w.Hkv, "head_dim": w.d, "score_window": w.window,
                   "bank": [w.N, w.E], "nq": w.nq, "top_k": w.k, "gather_row": w.D,
                   "parallelism": f"replicas x{world}", "l2": "inputs_exceed_l2 (1.7 GB of Q/K/V per pass)",
                   "chunk_kernel": "simt" if args.force_simt else "auto"},
        "retrieval_gather": {"value": retrieval_gather_bytes(w) / t_rg / 1e9, "unit": "GB/s",
                             "frac_of_hbm_peak": retrieval_gather_bytes(w) / t_rg / 1e9 / pk["hbm_gbs"],
                             "ms": t_rg * 1e3},
        "breakdown_ms": {"chunk_step": chunk_ms, "embed_append": mean(bd["embed_append"]),
                         "evict_topk": mean(bd["evict_topk"]), "retrieve_topk": mean(bd["retrieve_topk"]),
                         "gather": mean(bd["gather"])},
        "hbm_gbs": {"evict_topk": evict_bytes / (mean(bd["evict_topk"]) * 1e-3) / 1e9,
                    "embed_append": embed_bytes / (mean(bd["embed_append"]) * 1e-3) / 1e9,
                    "retrieve_topk": w.B * w.N * w.E * sz / (mean(bd["retrieve_topk"]) * 1e-3) / 1e9,
                    "gather": 2 * w.B * w.k * w.D * sz / (mean(bd["gather"]) * 1e-3) / 1e9},
        "roofline": {"bound": "tensor", "kernel": "reform_chunk_step (attention + score pass)",
                     "achieved": achieved, "peak": pk["tflops"], "unit": "TFLOP/s",
                     "frac": achieved / pk["tflops"], "frac_of_nominal_2250": achieved / 2250.0,
                     "traffic": ATTN_DRAM_RATIO * attn_bytes(w), "traffic_unit": "bytes per launch (steps >= 1)",
                     "traffic_source": ("ncu dram__bytes_read+write of the small-case capture in profiles/, "
                                        "scaled by algorithmic bytes Q+K+V+O"),
                     "peak_source": pk["source"],
                     "flops_counted": "4*Hq*d*visible pairs (QK^T and PV of unmasked pairs only)"},
        "gpu_launches": launches,
        "device_error_bits": dev_err,
        "clocks": clocks,
    }
    if e2e:
        line["e2e"] = e2e
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = {k: v for k, v in cpu_baseline(w).items() if k != "seconds"}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
