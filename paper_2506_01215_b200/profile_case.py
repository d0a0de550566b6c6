"""Runs one entry point of the library a few times on a seeded synthetic case
of chosen size -- the command to put under a profiler (one kernel, few
launches, a footprint that exceeds L2 but stays small).

  python -m paper_2506_01215_b200.profile_case chunk_step --lc 8192 --reps 3
  python -m paper_2506_01215_b200.profile_case retrieve --n 262144 --nq 4
"""
from __future__ import annotations

import argparse
import dataclasses

import torch

import paper_2506_01215_b200 as R
from paper_2506_01215_b200 import synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["chunk_step", "evict", "embed", "retrieve", "gather", "rope"])
    ap.add_argument("--workload", default="llama8b_128k")
    ap.add_argument("--lc", type=int, default=8192)
    ap.add_argument("--budget", type=int, default=8192)
    ap.add_argument("--window", type=int, default=128)
    ap.add_argument("--n", type=int, default=262144, help="bank rows (retrieve / gather)")
    ap.add_argument("--nq", type=int, default=0)
    ap.add_argument("--k", type=int, default=0)
    ap.add_argument("--layers", type=int, default=1, help="evict: layers batched into one call")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--simt", action="store_true")
    ap.add_argument("--no-score", action="store_true", help="chunk_step without the key-score pass")
    ap.add_argument("--rope", action="store_true", help="chunk_step on un-rotated operands (REFORM_ROPE)")
    ap.add_argument("--in-place", action="store_true", help="evict: destinations are the sources")
    ap.add_argument("--graph", action="store_true",
                    help="capture the call in a CUDA graph and time its replays (device time without the "
                         "host's launch cost)")
    a = ap.parse_args()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    w = synth.WORKLOADS[a.workload]
    w = dataclasses.replace(w, Lc=a.lc, budget=a.budget, window=min(a.window, a.lc), T=2 * a.lc, N=a.n,
                            nq=a.nq or w.nq, k=a.k or w.k)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if a.op in ("chunk_step", "embed", "evict", "rope"):
        wb = dataclasses.replace(w, B=w.B * a.layers) if a.op == "evict" else w
        q, kc, vc = synth.chunk_qkv(wb, 0, 1, device=dev)
        k0, v0, s0 = synth.cache_state(wb, 0, device=dev)
        k = torch.cat([k0, kc], 2).contiguous()
        v = torch.cat([v0, vc], 2).contiguous()
        score = torch.cat([s0, torch.rand(wb.B, wb.Hkv, wb.Lc, device=dev)], 2).contiguous()
    if a.op == "chunk_step":
        out = torch.empty_like(q)
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=dev)
        flags = (R.NO_SCORE if a.no_score else R.SCORE_ACCUMULATE) | (R.FORCE_SIMT if a.simt else 0) | \
            (R.ROPE if a.rope else 0)
        fn = lambda: R.chunk_step(q, k, v, out, score, w.budget, w.window, lse=lse, flags=flags)
    elif a.op == "evict":
        kd, vd, sd = (k, v, score) if a.in_place else (torch.empty_like(k), torch.empty_like(v), torch.empty_like(score))
        kept = torch.empty(wb.B, wb.Hkv, wb.budget, dtype=torch.int32, device=dev)
        fn = lambda: R.evict_topk(k, v, score, kd, vd, sd, wb.cap, wb.budget, wb.n_sink, wb.n_recent,
                                  kept_idx=kept)
    elif a.op == "embed":
        bank = torch.zeros(w.B, w.Lc, w.E, dtype=w.dtype, device=dev)
        sel = synth.head_selection(w)
        fn = lambda: R.embed_append(bank, 0, sel, q_state=q, k_state=kc, v_state=vc)
    elif a.op == "rope":
        q_rot, k_rot = torch.empty_like(q), torch.empty_like(k)

        def fn():
            R.rope(q, q_rot, 0, w.Lc, w.budget)      # queries at positions n_cache + i
            R.rope(k, k_rot, 0, w.cap, 0)            # cache and chunk keys at positions 0 .. n-1
    elif a.op == "retrieve":
        bank, queries, _ = synth.bank_and_queries(w, device=dev)
        idx = torch.zeros(w.B, w.k, dtype=torch.int32, device=dev)
        fn = lambda: R.retrieve_topk(bank, queries, w.N, w.k, idx, scale=w.sim_scale,
                                     pool_window=w.pool_window, n_keep_head=w.keep_head,
                                     n_keep_tail=w.keep_tail)
    else:
        hidden = synth.hidden_rows(w, device=dev)
        g = torch.Generator(device=dev).manual_seed(1)
        idx = torch.sort(torch.randperm(w.N, generator=g, device=dev)[:w.k].to(torch.int32)).values
        idx = idx.expand(w.B, w.k).contiguous()
        dst = torch.empty(w.B, w.k, w.D, dtype=w.dtype, device=dev)
        fn = lambda: R.gather(hidden, idx, dst)
    fn()
    torch.cuda.synchronize()
    run = fn
    if a.graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fn()
        run = graph.replay
        run()
        torch.cuda.synchronize()
    ev0.record()
    for _ in range(a.reps):
        run()
    ev1.record()
    torch.cuda.synchronize()
    how = "graph replays" if a.graph else "calls"
    print(f"{a.op}: {ev0.elapsed_time(ev1) / a.reps:.4f} ms per call over {a.reps} {how}")


if __name__ == "__main__":
    main()
