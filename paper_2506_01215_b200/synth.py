"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors and plants structure in them; it holds
none of the method's arithmetic and is the one piece of code that both the
CUDA path's callers and the oracle's callers may use, so that both sides are
handed identical bytes.  The same (seed, ids, device type) always gives the
same tensor; CPU and CUDA generators give different streams, so a parity test
draws once and copies.

Recipe (stand-in for the long-context benchmarks the paper evaluates on):
  * Q/K/V states ~ N(0,1), rounded once to the config dtype.
  * Needle keys (Sec. 4.1 needle-in-a-haystack stand-in): a shared unit
    direction u is added with amplitude a = 2*d^(1/4) to every query and to
    each needle key, so a needle's logit is about +4 above an ordinary key's
    for every query and it must survive every eviction.
  * Embedding bank rows: each d-wide head slot is an independent unit vector;
    planted rows have cosine rho with one of the query embeddings in every
    slot (Sec. 3.3 stand-in for query-relevant context tokens).
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """One of the benchmark configurations (shapes only)."""
    name: str
    dtype: torch.dtype
    T: int            # context tokens
    layers: int
    B: int
    Hq: int
    Hkv: int
    d: int
    Lc: int           # chunk length
    budget: int       # kept keys per kv head
    n_sink: int
    n_recent: int
    window: int       # trailing queries of a chunk that score keys
    n_needles: int
    # retrieval
    N: int            # bank rows
    n_slots: int      # selected heads per row; E = n_slots * slot_dim
    slot_dim: int
    nq: int
    n_planted: int
    rho: float
    k: int            # gathered tokens
    pool_window: int
    keep_head: int
    keep_tail: int
    D: int            # gathered row width (elements of dtype)
    seed: int

    @property
    def E(self) -> int:
        return self.n_slots * self.slot_dim

    @property
    def steps(self) -> int:
        return self.T // self.Lc

    @property
    def cap(self) -> int:
        return self.budget + self.Lc

    @property
    def sim_scale(self) -> float:
        return 1.0 / self.n_slots


BF16, F32 = torch.bfloat16, torch.float32

WORKLOADS = {
    "tiny": Workload("tiny", F32, 8192, 1, 1, 4, 2, 64, 1024, 512, 32, 32, 128, 8,
                     8192, 1, 128, 1, 16, 0.9, 256, 17, 8, 8, 512, 0x5EF0),
    "llama8b_128k": Workload("llama8b_128k", BF16, 131072, 1, 1, 32, 8, 128, 32768, 8192, 256, 256,
                             128, 64, 131072, 8, 128, 4, 64, 0.9, 4096, 129, 256, 256, 4096, 0x5EF1),
    "llama8b_1m_32l": Workload("llama8b_1m_32l", BF16, 1048576, 32, 1, 32, 8, 128, 32768, 8192, 256,
                               256, 128, 64, 1048576, 8, 128, 4, 64, 0.9, 4096, 129, 256, 256, 4096,
                               0x5EF2),
    "retrieval_1m": Workload("retrieval_1m", BF16, 1048576, 1, 1, 32, 8, 128, 32768, 8192, 256, 256,
                             128, 64, 1048576, 8, 128, 64, 256, 0.9, 16384, 129, 256, 256, 4096,
                             0x5EF3),
    "mistral7b_4x256k": Workload("mistral7b_4x256k", BF16, 262144, 1, 4, 32, 8, 128, 16384, 4096, 256,
                                 256, 128, 64, 262144, 8, 128, 8, 64, 0.9, 8192, 129, 256, 256, 4096,
                                 0x5EF4),
}


def _mix(seed: int, *ids: int) -> int:
    """Fold integer ids into a 63-bit generator seed (splitmix-style)."""
    x = (seed & 0xFFFFFFFFFFFFFFFF) ^ 0x9E3779B97F4A7C15
    for i in ids:
        x = (x + 0x9E3779B97F4A7C15 + (int(i) & 0xFFFFFFFFFFFFFFFF)) & 0xFFFFFFFFFFFFFFFF
        x ^= x >> 30
        x = (x * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        x ^= x >> 27
        x = (x * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
        x ^= x >> 31
    return x & 0x7FFFFFFFFFFFFFFF


def generator(seed: int, *ids: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_mix(seed, *ids))
    return g


def randn(shape, seed, *ids, device="cpu", dtype=torch.float32) -> torch.Tensor:
    g = generator(seed, *ids, device=device)
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32).to(dtype)


# --------------------------------------------------------------------------
# chunk-step inputs
# --------------------------------------------------------------------------

def needle_direction(d: int, seed: int, device="cpu") -> torch.Tensor:
    u = randn((d,), seed, 101, device="cpu")
    return (u / u.norm()).to(device)


def needle_amplitude(d: int) -> float:
    return 2.0 * d ** 0.25


def needle_positions(w: Workload, b: int = 0, seed: Optional[int] = None) -> List[int]:
    """Distinct global token positions, one per equal stratum of the context,
    kept clear of the first n_sink tokens and the last chunk's recent tail."""
    seed = w.seed if seed is None else seed
    g = generator(seed, 202, b)
    lo, hi = w.n_sink, w.T - w.n_recent
    out = []
    for i in range(w.n_needles):
        a = lo + (hi - lo) * i // w.n_needles
        z = lo + (hi - lo) * (i + 1) // w.n_needles
        out.append(a + int(torch.randint(0, max(z - a, 1), (1,), generator=g).item()))
    return out


def chunk_qkv(w: Workload, layer: int, step: int, device="cpu", seed: Optional[int] = None,
              Lc: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Q [B,Hq,Lc,d], K and V [B,Hkv,Lc,d] of chunk ``step`` of ``layer``."""
    seed = w.seed if seed is None else seed
    Lc = Lc or w.Lc
    u = needle_direction(w.d, seed, device)
    a = needle_amplitude(w.d)
    q = randn((w.B, w.Hq, Lc, w.d), seed, 1, layer, step, device=device) + a * u
    k = randn((w.B, w.Hkv, Lc, w.d), seed, 2, layer, step, device=device)
    v = randn((w.B, w.Hkv, Lc, w.d), seed, 3, layer, step, device=device)
    for b in range(w.B):
        for p in needle_positions(w, b, seed):
            if step * Lc <= p < (step + 1) * Lc:
                k[b, :, p - step * Lc, :] += a * u
    return q.to(w.dtype), k.to(w.dtype), v.to(w.dtype)


def cache_state(w: Workload, layer: int, device="cpu", seed: Optional[int] = None,
                n_cache: Optional[int] = None):
    """A stand-alone compressed-cache state (K, V rows and carried scores) for
    checking one recurrent step in isolation: rows ~ N(0,1), scores uniform in
    [0, 4*window*G/cap)."""
    seed = w.seed if seed is None else seed
    n_cache = w.budget if n_cache is None else n_cache
    k = randn((w.B, w.Hkv, n_cache, w.d), seed, 11, layer, device=device, dtype=w.dtype)
    v = randn((w.B, w.Hkv, n_cache, w.d), seed, 12, layer, device=device, dtype=w.dtype)
    g = generator(seed, 13, layer, device=device)
    G = w.Hq // w.Hkv
    s = torch.rand((w.B, w.Hkv, n_cache), generator=g, device=device) * (4.0 * w.window * G / w.cap)
    return k, v, s


# --------------------------------------------------------------------------
# retrieval inputs
# --------------------------------------------------------------------------

def _unit_slots(x: torch.Tensor, n_slots: int) -> torch.Tensor:
    shp = x.shape
    y = x.reshape(*shp[:-1], n_slots, shp[-1] // n_slots)
    y = y / y.norm(dim=-1, keepdim=True).clamp_min(1e-20)
    return y.reshape(shp)


def planted_positions(N: int, n_planted: int, keep_head: int, keep_tail: int, seed: int, b: int = 0):
    g = generator(seed, 303, b)
    lo, hi = keep_head, N - keep_tail
    out = []
    for i in range(n_planted):
        a = lo + (hi - lo) * i // n_planted
        z = lo + (hi - lo) * (i + 1) // n_planted
        out.append(a + int(torch.randint(0, max(z - a, 1), (1,), generator=g).item()))
    return out


def bank_and_queries(w: Workload, device="cpu", seed: Optional[int] = None, N: Optional[int] = None,
                     rows_per_block: int = 65536):
    """Returns (bank [B,N,E], queries [B,nq,E], planted [B][n_planted]) in w.dtype.

    Every slot of every row is a unit vector (before the rounding to dtype).
    Planted row i of sequence b has cosine w.rho, in every slot, with query
    i % nq of that sequence.
    """
    seed = w.seed if seed is None else seed
    N = N or w.N
    E, ns = w.E, w.n_slots
    queries = _unit_slots(randn((w.B, w.nq, E), seed, 21, device=device), ns)
    bank = torch.empty((w.B, N, E), dtype=w.dtype, device=device)
    for b in range(w.B):
        for r0 in range(0, N, rows_per_block):
            r1 = min(N, r0 + rows_per_block)
            blk = randn((r1 - r0, E), seed, 22, b, r0, device=device)
            bank[b, r0:r1] = _unit_slots(blk, ns).to(w.dtype)
    planted = []
    for b in range(w.B):
        pos = planted_positions(N, w.n_planted, w.keep_head, w.keep_tail, seed, b)
        planted.append(pos)
        if not pos:
            continue
        qi = torch.arange(len(pos), device=device) % w.nq
        tgt = queries[b, qi].reshape(len(pos), ns, w.slot_dim)
        noise = randn((len(pos), ns, w.slot_dim), seed, 23, b, device=device)
        noise = noise - (noise * tgt).sum(-1, keepdim=True) * tgt
        noise = noise / noise.norm(dim=-1, keepdim=True)
        rows = w.rho * tgt + math.sqrt(1.0 - w.rho ** 2) * noise
        bank[b, torch.tensor(pos, device=device)] = rows.reshape(len(pos), E).to(w.dtype)
    return bank, queries.to(w.dtype), planted


def hidden_rows(w: Workload, device="cpu", seed: Optional[int] = None, N: Optional[int] = None,
                rows_per_block: int = 65536) -> torch.Tensor:
    """The [B,N,D] buffer the gather reads (input-embedding stand-in)."""
    seed = w.seed if seed is None else seed
    N = N or w.N
    out = torch.empty((w.B, N, w.D), dtype=w.dtype, device=device)
    for b in range(w.B):
        for r0 in range(0, N, rows_per_block):
            r1 = min(N, r0 + rows_per_block)
            out[b, r0:r1] = randn((r1 - r0, w.D), seed, 31, b, r0, device=device, dtype=w.dtype)
    return out


def head_selection(w: Workload) -> List[Tuple[int, int, int]]:
    """(kind, head, slot) triples feeding the bank: kinds cycle V, K, Q, V, ...
    over distinct heads, mirroring the paper's mix of query/key/value heads."""
    kinds = [2, 1, 0, 2, 2, 1, 0, 2, 2, 1, 0, 2, 2, 1, 0, 2]
    sel = []
    for s in range(w.n_slots):
        kind = kinds[s % len(kinds)]
        H = w.Hq if kind == 0 else w.Hkv
        sel.append((kind, (3 * s + 1) % H, s))
    return sel
