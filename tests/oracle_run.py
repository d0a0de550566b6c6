"""The recurrence of Alg. 1 (ForwardChunk, one layer) run by the oracle alone:
chunk by chunk, key scores over [cache ; chunk], then the eviction's full
sort.  Shared by the CPU pin of the needle construction and by the GPU
free-running parity test.  Nothing here touches the CUDA library."""
import torch

import oracle
from paper_2506_01215_b200 import synth


def oracle_free_run(w, layer=0, accumulate=True, window=None):
    """Yields, after every recurrence step, a dict with the oracle's state:
    step, n (keys before the eviction), scores [B,Hkv,cap] fp64 before the
    eviction, and k, v, score, pos, kept_idx, n_kept after it."""
    window = window or w.window
    ck = torch.zeros(w.B, w.Hkv, w.cap, w.d, dtype=w.dtype)
    cv = torch.zeros_like(ck)
    cs = torch.zeros(w.B, w.Hkv, w.cap, dtype=torch.float64)
    pos = torch.zeros(w.B, w.Hkv, w.cap, dtype=torch.int32)
    n_cache = 0
    for step in range(w.steps):
        q, kc, vc = synth.chunk_qkv(w, layer, step)
        ck[:, :, n_cache:n_cache + w.Lc] = kc
        cv[:, :, n_cache:n_cache + w.Lc] = vc
        pos[:, :, n_cache:n_cache + w.Lc] = torch.arange(step * w.Lc, (step + 1) * w.Lc, dtype=torch.int32)
        n = n_cache + w.Lc
        scores = oracle.key_scores(q, ck, n_cache, window, score_in=cs, accumulate=accumulate)
        ref = oracle.evict_topk(ck, cv, scores, n, w.budget, w.n_sink, w.n_recent, cap_dst=w.cap, pos_src=pos)
        yield dict(step=step, n=n, n_cache_before=n_cache, scores=scores, pos_before=pos.clone(), **ref)
        ck, cv, cs, pos, n_cache = ref["k"], ref["v"], ref["score"], ref["pos"], ref["n_kept"]
