"""Caller-side bookkeeping of the recurrent chunked forwarding loop (Alg. 1,
ForwardChunk) for one layer: which buffer holds the compressed cache, where the
next chunk's K/V rows go, and the order of the three calls per chunk.  It owns
buffers and calls the binding; it computes nothing itself."""
from __future__ import annotations

from typing import List, Optional

import torch

from . import SCORE_ACCUMULATE, chunk_step, evict_topk


class LayerCache:
    """Compressed KV cache of one layer.

    ``n_buffers`` buffer sets of shape [B,Hkv,cap,d] are used round-robin: the
    chunk step of recurrence step s reads set s % n_buffers and the eviction
    writes the compacted rows into set (s+1) % n_buffers.  With ``n_buffers = 1``
    the eviction runs in place (destinations are the sources) and the layer
    holds one K/V buffer instead of two.
    """

    def __init__(self, B, Hkv, d, cap, budget, n_sink, n_recent, dtype, device, n_buffers=2):
        self.B, self.Hkv, self.d, self.cap = B, Hkv, d, cap
        self.budget, self.n_sink, self.n_recent = budget, n_sink, n_recent
        self.k = [torch.zeros(B, Hkv, cap, d, dtype=dtype, device=device) for _ in range(n_buffers)]
        self.v = [torch.zeros(B, Hkv, cap, d, dtype=dtype, device=device) for _ in range(n_buffers)]
        self.score = [torch.zeros(B, Hkv, cap, dtype=torch.float32, device=device) for _ in range(n_buffers)]
        self.kept_idx = torch.zeros(B, Hkv, budget, dtype=torch.int32, device=device)
        self.cur = 0
        self.n_cache = 0
        self.n_keys = 0

    @property
    def nxt(self) -> int:
        return (self.cur + 1) % len(self.k)

    def write_chunk(self, k_chunk: torch.Tensor, v_chunk: torch.Tensor):
        """Places the chunk's K/V rows behind the cache rows (the job of the
        model's K/V projection in a real forward pass)."""
        Lc = k_chunk.shape[2]
        self.k[self.cur][:, :, self.n_cache:self.n_cache + Lc].copy_(k_chunk)
        self.v[self.cur][:, :, self.n_cache:self.n_cache + Lc].copy_(v_chunk)
        self.n_keys = self.n_cache + Lc

    def attend(self, q, out, score_window, lse=None, flags=SCORE_ACCUMULATE, softmax_scale=0.0):
        chunk_step(q, self.k[self.cur], self.v[self.cur], out, self.score[self.cur], self.n_cache,
                   score_window, lse=lse, flags=flags, softmax_scale=softmax_scale)

    def evict(self):
        n_kept = evict_topk(self.k[self.cur], self.v[self.cur], self.score[self.cur],
                            self.k[self.nxt], self.v[self.nxt], self.score[self.nxt], self.n_keys,
                            self.budget, self.n_sink, self.n_recent, kept_idx=self.kept_idx)
        self.cur = self.nxt
        self.n_cache = n_kept
        self.n_keys = n_kept
        return n_kept
