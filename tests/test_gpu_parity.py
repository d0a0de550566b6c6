"""GPU parity: every entry point of the C-ABI library against the fp64 CPU
oracle on identical seeded inputs (drawn once on the CPU, copied to the GPU)."""
import dataclasses

import pytest
import torch

import oracle
import paper_2506_01215_b200 as R
from paper_2506_01215_b200 import synth
from paper_2506_01215_b200.driver import LayerCache

from parity import assert_index_sets_match, assert_outputs_close, assert_scores_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(B, Hq, Hkv, d, Lc, n_cache, dtype, seed=0, extra=5):
    g = torch.Generator().manual_seed(seed)
    cap = n_cache + Lc + extra
    q = torch.randn(B, Hq, Lc, d, generator=g).to(dtype)
    k = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    v = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    carry = torch.rand(B, Hkv, cap, generator=g)
    return q, k, v, carry


def _run_chunk(q, k, v, carry, n_cache, W, flags=R.SCORE_ACCUMULATE, scale=0.0):
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    out = torch.full_like(qd, float("nan"))
    lse = torch.full(q.shape[:3], float("nan"), device=DEV)
    score = carry.to(DEV).clone()
    R.chunk_step(qd, kd, vd, out, score, n_cache, W, lse=lse, flags=flags, softmax_scale=scale)
    torch.cuda.synchronize()
    return out, lse, score


CHUNK_CASES = [
    # B, Hq, Hkv, d, Lc, n_cache, dtype, W
    (1, 4, 2, 64, 192, 100, torch.float32, 128),     # tiny-shaped, ragged everything
    (2, 4, 2, 64, 130, 0, torch.float32, 130),       # first step, W = Lc, ragged tail
    (1, 2, 1, 128, 200, 77, torch.float32, 1),       # TOVA-style window
    (1, 8, 2, 128, 300, 140, torch.bfloat16, 128),   # tensor-core path, several tiles
    (2, 4, 4, 128, 257, 0, torch.bfloat16, 257),     # no GQA sharing, W = Lc
    (1, 4, 1, 128, 128, 512, torch.bfloat16, 64),    # cache much longer than chunk
    (1, 4, 2, 64, 96, 40, torch.bfloat16, 32),       # bf16 on the CUDA-core path (d = 64)
    (3, 6, 2, 128, 300, 70, torch.bfloat16, 100),    # group of 3: tile pairs straddle heads, odd unit count
    (1, 2, 2, 128, 1000, 0, torch.bfloat16, 128),    # pairs of consecutive query tiles with different walks
]


@pytest.mark.parametrize("B,Hq,Hkv,d,Lc,n_cache,dtype,W", CHUNK_CASES)
def test_chunk_step_matches_oracle(B, Hq, Hkv, d, Lc, n_cache, dtype, W):
    q, k, v, carry = _case(B, Hq, Hkv, d, Lc, n_cache, dtype, seed=Lc)
    out, lse, score = _run_chunk(q, k, v, carry, n_cache, W)
    o_ref, lse_ref = oracle.attention(q, k, v, n_cache)
    assert_outputs_close(out, o_ref, dtype)
    assert (lse.cpu().double() - lse_ref).abs().max() < (2e-3 if dtype == torch.bfloat16 else 1e-4)
    s_ref = oracle.key_scores(q, k, n_cache, W, score_in=carry, accumulate=True)
    n = n_cache + Lc
    G = Hq // Hkv
    assert_scores_close(score[:, :, :n], s_ref[:, :, :n], W * G / n)
    # rows past the keys in use keep the caller's values
    assert torch.equal(score[:, :, n:].cpu(), carry[:, :, n:])
    # conservation: new mass sums to W*G
    new = score[:, :, :n].cpu().double().sum(-1) - carry[:, :, :n_cache].double().sum(-1)
    assert torch.allclose(new, torch.full_like(new, float(W * G)), rtol=2e-3)


def test_chunk_step_flags_and_scale():
    q, k, v, carry = _case(1, 4, 2, 128, 160, 64, torch.bfloat16, seed=5)
    out, lse, score = _run_chunk(q, k, v, carry, 64, 32, flags=0, scale=0.11)
    o_ref, _ = oracle.attention(q, k, v, 64, scale=0.11)
    assert_outputs_close(out, o_ref, torch.bfloat16)
    s_ref = oracle.key_scores(q, k, 64, 32, scale=0.11)
    assert_scores_close(score[:, :, :224], s_ref[:, :, :224], 32 * 2 / 224)
    out2, _, score2 = _run_chunk(q, k, v, carry, 64, 32, flags=R.NO_SCORE, scale=0.11)
    assert torch.equal(out2, out)
    assert torch.equal(score2.cpu(), carry)          # untouched
    out3, _, score3 = _run_chunk(q, k, v, carry, 64, 32, flags=R.FORCE_SIMT, scale=0.11)
    assert_outputs_close(out3, o_ref, torch.bfloat16)
    assert_scores_close(score3[:, :, :224], s_ref[:, :, :224], 32 * 2 / 224)


def test_recompute_phase_prefill_and_decode_shapes():
    """The steps right after the gather (Sec. 3.3, on-demand recomputation): a plain causal prefill
    of the gathered tokens is the chunk step with an empty cache and no score pass, and a decode
    step is a one-row chunk over the recomputed cache."""
    q, k, v, carry = _case(1, 8, 2, 128, 777, 0, torch.bfloat16, seed=21)
    out, lse, score = _run_chunk(q, k, v, carry, 0, 1, flags=R.NO_SCORE)
    o_ref, l_ref = oracle.attention(q, k, v, 0)
    assert_outputs_close(out, o_ref, torch.bfloat16)
    assert (lse.cpu().double() - l_ref).abs().max() < 2e-3
    assert torch.equal(score.cpu(), carry)
    q, k, v, carry = _case(2, 8, 2, 128, 1, 1500, torch.bfloat16, seed=22)
    out, lse, _ = _run_chunk(q, k, v, carry, 1500, 1, flags=R.NO_SCORE)
    o_ref, l_ref = oracle.attention(q, k, v, 1500)
    assert_outputs_close(out, o_ref, torch.bfloat16)
    assert (lse.cpu().double() - l_ref).abs().max() < 2e-3


@pytest.mark.parametrize("B,Hq,Hkv,Lc,n_cache,W", [
    (1, 32, 8, 1, 8192, 1),      # one new token over an 8k recomputed cache (the decode step)
    (2, 8, 2, 4, 1000, 4),       # four tokens at once: 16 packed rows, causal among themselves
    (1, 12, 4, 3, 77, 2),        # group of 3, ragged everything
    (1, 4, 4, 5, 0, 5),          # no sharing, empty cache
    (1, 16, 1, 1, 300, 1),       # all 16 heads on one KV head
])
def test_decode_shaped_steps_match_oracle(B, Hq, Hkv, Lc, n_cache, W):
    """Few query rows per KV head: the split-KV kernel (keys divided among warps, partials merged)."""
    q, k, v, carry = _case(B, Hq, Hkv, 128, Lc, n_cache, torch.bfloat16, seed=n_cache + Lc)
    out, lse, score = _run_chunk(q, k, v, carry, n_cache, W)
    o_ref, l_ref = oracle.attention(q, k, v, n_cache)
    assert_outputs_close(out, o_ref, torch.bfloat16)
    assert (lse.cpu().double() - l_ref).abs().max() < 2e-3
    n = n_cache + Lc
    s_ref = oracle.key_scores(q, k, n_cache, W, score_in=carry, accumulate=True)
    assert_scores_close(score[:, :, :n], s_ref[:, :, :n], W * (Hq // Hkv) / n)
    out2, lse2, _ = _run_chunk(q, k, v, carry, n_cache, W, flags=R.FORCE_SIMT | R.SCORE_ACCUMULATE)
    assert (out2.float() - out.float()).abs().max() < 2e-2


def test_alternative_compressors_through_the_same_calls():
    """Sec. 5.1 ablation: TOVA scores keys with the last query only and does not accumulate
    (score_window 1, no carry); StreamingLLM keeps only the initial and recent rows (budget =
    sink + recent).  Both are parameter settings of the same two entry points."""
    q, k, v, carry = _case(1, 8, 2, 128, 200, 300, torch.bfloat16, seed=23)
    out, lse, score = _run_chunk(q, k, v, carry, 300, 1, flags=0)
    s_ref = oracle.key_scores(q, k, 300, 1)
    assert_scores_close(score[:, :, :500], s_ref[:, :, :500], 1 * 4 / 500)
    ref = oracle.evict_topk(k, v, s_ref, 500, 128, 4, 4, cap_dst=128)
    kd = torch.zeros(1, 2, 128, 128, dtype=torch.bfloat16, device=DEV)
    vd, sd = torch.zeros_like(kd), torch.zeros(1, 2, 128, device=DEV)
    kept = torch.zeros(1, 2, 128, dtype=torch.int32, device=DEV)
    R.evict_topk(k.to(DEV), v.to(DEV), score, kd, vd, sd, 500, 128, 4, 4, kept_idx=kept)
    for h in range(2):
        assert_index_sets_match(kept[0, h].cpu(), ref["kept_idx"][0, h], s_ref[0, h])
    kept2 = torch.zeros(1, 2, 48, dtype=torch.int32, device=DEV)
    kd2 = torch.zeros(1, 2, 48, 128, dtype=torch.bfloat16, device=DEV)
    R.evict_topk(k.to(DEV), v.to(DEV), score, kd2, torch.zeros_like(kd2), torch.zeros(1, 2, 48, device=DEV),
                 500, 48, 16, 32, kept_idx=kept2)
    assert kept2.cpu()[0, 0].tolist() == list(range(16)) + list(range(468, 500))


def test_chunk_step_extreme_logits():
    """One key whose logit towers over everything seen before it (a jump of more than 100 in log2
    units in the middle of the walk): the running maximum must be re-based without overflow, rows
    that see the key return its value row, rows before it are untouched by it, nothing is NaN."""
    q, k, v, carry = _case(1, 4, 2, 128, 400, 200, torch.bfloat16, seed=77)
    q[..., 0] = 30.0
    k[..., 0] = 0.0
    j = 200 + 150                       # chunk row 150, in the second key tile of the chunk part
    k[:, :, j, 0] = 30.0
    out, lse, score = _run_chunk(q, k, v, carry, 200, 128, flags=0)
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all() and torch.isfinite(score[:, :, :600]).all()
    o_ref, l_ref = oracle.attention(q, k, v, 200)
    assert_outputs_close(out, o_ref, torch.bfloat16)
    assert (lse.cpu().double() - l_ref).abs().max() < 2e-3
    expect = v[:, :, j].double().repeat_interleave(2, dim=1)[:, :, None, :]
    assert (out[:, :, 150:].cpu().double() - expect).abs().max() < 2e-2
    s_ref = oracle.key_scores(q, k, 200, 128)
    assert_scores_close(score[:, :, :600], s_ref[:, :, :600], 128 * 2 / 600)
    assert abs(score[0, 0, j].item() - 256.0) < 0.3       # it takes all the mass of the 128 x 2 scoring rows


def test_chunk_step_is_deterministic():
    q, k, v, carry = _case(1, 8, 2, 128, 260, 130, torch.bfloat16, seed=9)
    a = _run_chunk(q, k, v, carry, 130, 128)
    b = _run_chunk(q, k, v, carry, 130, 128)
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_chunk_step_identical_keys_uniform_mass():
    """All keys equal: every query spreads its mass evenly, score[j] follows
    the harmonic-number closed form and out is the prefix mean of V."""
    q, k, v, carry = _case(1, 4, 2, 128, 140, 60, torch.bfloat16, seed=2)
    k[:] = k[:, :, :1]
    out, lse, score = _run_chunk(q, k, v, carry, 60, 140, flags=0)
    n = 200
    H = torch.cat([torch.zeros(1, dtype=torch.float64), (1.0 / torch.arange(1, n + 1, dtype=torch.float64)).cumsum(0)])
    expect = 2 * (H[n] - H[torch.clamp(torch.arange(n), min=60)])
    assert_scores_close(score[0, 0, :n], expect, 140 * 2 / n)
    pm = v[:, :, :n].double().cumsum(2)[:, :, 60:] / torch.arange(61, n + 1, dtype=torch.float64)[:, None]
    assert (out.cpu().double() - pm.repeat_interleave(2, dim=1)).abs().max() < 2e-2


# ------------------------------------------------------------------ evict

EVICT_CASES = [
    # B, Hkv, d, n_keys, budget, sink, recent, dtype
    (1, 2, 64, 1536, 512, 32, 32, torch.float32),
    (2, 3, 128, 5000, 1000, 0, 0, torch.bfloat16),
    (1, 2, 128, 9000, 4100, 256, 256, torch.bfloat16),    # more than two select tiles, ragged
    (1, 1, 64, 300, 40, 16, 24, torch.float32),            # no heavy hitters: sink + recent only
    (1, 2, 64, 100, 128, 8, 8, torch.float32),             # under budget: keep all
]


@pytest.mark.parametrize("B,Hkv,d,n_keys,budget,sink,recent,dtype", EVICT_CASES)
@pytest.mark.parametrize("ties", [False, True])
def test_evict_matches_oracle_bit_exactly(B, Hkv, d, n_keys, budget, sink, recent, dtype, ties):
    g = torch.Generator().manual_seed(n_keys)
    cap = n_keys + 7
    k = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    v = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    sc = torch.rand(B, Hkv, cap, generator=g)
    if ties:
        sc = (sc * 6).floor() / 4 - 0.5      # heavy ties, some negative, and a -0.0
        sc[..., 5] = -0.0
    pos = torch.randint(0, 1 << 20, (B, Hkv, cap), generator=g, dtype=torch.int32)
    ref = oracle.evict_topk(k, v, sc, n_keys, budget, sink, recent, cap_dst=budget + 3, pos_src=pos)
    kd = torch.zeros(B, Hkv, budget + 3, d, dtype=dtype, device=DEV)
    vd = torch.zeros_like(kd)
    sd = torch.zeros(B, Hkv, budget + 3, device=DEV)
    pd = torch.zeros(B, Hkv, budget + 3, dtype=torch.int32, device=DEV)
    kept = torch.full((B, Hkv, budget), -1, dtype=torch.int32, device=DEV)
    n_kept = R.evict_topk(k.to(DEV), v.to(DEV), sc.to(DEV), kd, vd, sd, n_keys, budget, sink, recent,
                          pos_src=pos.to(DEV), pos_dst=pd, kept_idx=kept)
    torch.cuda.synchronize()
    assert n_kept == ref["n_kept"]
    assert torch.equal(kept.cpu()[:, :, :n_kept], ref["kept_idx"][:, :, :n_kept])
    assert torch.equal(kd.cpu()[:, :, :n_kept].view(torch.uint8), ref["k"][:, :, :n_kept].view(torch.uint8))
    assert torch.equal(vd.cpu()[:, :, :n_kept].view(torch.uint8), ref["v"][:, :, :n_kept].view(torch.uint8))
    assert torch.equal(sd.cpu()[:, :, :n_kept].double(), ref["score"][:, :, :n_kept])
    assert torch.equal(pd.cpu()[:, :, :n_kept], ref["pos"][:, :, :n_kept])


def test_evict_many_segments():
    """384 segments in one call (layers x sequences x KV heads batched): one block per segment."""
    g = torch.Generator().manual_seed(4)
    B, Hkv, n, d, budget = 48, 8, 4200, 4, 1000
    k = torch.randn(B, Hkv, n, d, generator=g)
    sc = (torch.rand(B, Hkv, n, generator=g) * 50).floor()   # many ties
    ref = oracle.evict_topk(k, k, sc, n, budget, 16, 16, cap_dst=budget)
    kd = torch.zeros(B, Hkv, budget, d, device=DEV)
    vd = torch.zeros_like(kd)
    sd = torch.zeros(B, Hkv, budget, device=DEV)
    kept = torch.zeros(B, Hkv, budget, dtype=torch.int32, device=DEV)
    R.evict_topk(k.to(DEV), k.to(DEV).clone(), sc.to(DEV), kd, vd, sd, n, budget, 16, 16, kept_idx=kept)
    assert torch.equal(kept.cpu(), ref["kept_idx"])
    assert torch.equal(kd.cpu(), ref["k"])


@pytest.mark.parametrize("n", [70001, 140001])
def test_evict_long_segments(n):
    """Segments longer than one block handles alone: the selection runs as one cooperative launch
    over global-memory histograms (18 and 35 blocks per segment)."""
    g = torch.Generator().manual_seed(8)
    B, Hkv, d, budget = 1, 2, 4, 9000
    k = torch.randn(B, Hkv, n, d, generator=g)
    sc = (torch.rand(B, Hkv, n, generator=g) * 4000).floor()
    ref = oracle.evict_topk(k, k, sc, n, budget, 100, 100, cap_dst=budget)
    kd = torch.zeros(B, Hkv, budget, d, device=DEV)
    vd = torch.zeros_like(kd)
    sd = torch.zeros(B, Hkv, budget, device=DEV)
    kept = torch.zeros(B, Hkv, budget, dtype=torch.int32, device=DEV)
    R.evict_topk(k.to(DEV), k.to(DEV).clone(), sc.to(DEV), kd, vd, sd, n, budget, 100, 100, kept_idx=kept)
    assert torch.equal(kept.cpu(), ref["kept_idx"])
    assert torch.equal(kd.cpu(), ref["k"])


def test_retrieve_many_sequences_multi_launch_path():
    """More selection blocks than can be resident at once (10 sequences x 35 blocks): the selection
    falls back to one launch per pass; results must not change."""
    g = torch.Generator().manual_seed(6)
    B, N, E, nq, k = 10, 140000, 32, 2, 500
    bank = torch.randn(B, N, E, generator=g).bfloat16()
    qs = torch.randn(B, nq, E, generator=g).bfloat16()
    ref = oracle.retrieve_topk(bank, qs, N, k, scale=0.25, pool_window=9, n_keep_head=3, n_keep_tail=5)
    idx = torch.full((B, k), -1, dtype=torch.int32, device=DEV)
    pooled = torch.zeros(B, N, device=DEV)
    R.retrieve_topk(bank.to(DEV), qs.to(DEV), N, k, idx, scale=0.25, pool_window=9, n_keep_head=3,
                    n_keep_tail=5, pooled_score_out=pooled)
    assert_scores_close(pooled, ref["pooled"], 1.0)
    for b in range(B):
        assert_index_sets_match(idx[b].cpu(), ref["idx"][b], ref["pooled"][b])


def test_evict_all_scores_equal_and_two_level_ties():
    """Degenerate score distributions for the one-launch selection: every candidate in one
    histogram bin (all scores equal: the kept middle rows are the lowest indices), and scores that
    agree in their leading bits and differ only in the last ones."""
    g = torch.Generator().manual_seed(3)
    B, Hkv, n, d, budget = 1, 3, 13000, 8, 3000
    k = torch.randn(B, Hkv, n, d, generator=g)
    for sc in (torch.full((B, Hkv, n), 0.37),
               1.0 + torch.randint(0, 50, (B, Hkv, n), generator=g).float() * 2.0 ** -23,
               torch.zeros(B, Hkv, n)):
        ref = oracle.evict_topk(k, k, sc, n, budget, 7, 9, cap_dst=budget)
        kd = torch.zeros(B, Hkv, budget, d, device=DEV)
        vd, sd = torch.zeros_like(kd), torch.zeros(B, Hkv, budget, device=DEV)
        kept = torch.zeros(B, Hkv, budget, dtype=torch.int32, device=DEV)
        R.evict_topk(k.to(DEV), k.to(DEV).clone(), sc.to(DEV), kd, vd, sd, n, budget, 7, 9, kept_idx=kept)
        assert torch.equal(kept.cpu(), ref["kept_idx"])
        assert torch.equal(kd.cpu(), ref["k"]) and torch.equal(sd.cpu().double(), ref["score"])


def _score_kind(kind, shape, g):
    if kind == "uniform":
        return torch.rand(shape, generator=g)
    if kind == "ties":                       # heavy ties, some negative, a -0.0
        sc = (torch.rand(shape, generator=g) * 6).floor() / 4 - 0.5
        sc[..., 5] = -0.0
        return sc
    if kind == "equal":                      # every candidate in one bin of every pass
        return torch.full(shape, 0.37)
    if kind == "lowbits":                    # agree in the leading 22 bits, differ in the last ones
        return 1.0 + torch.randint(0, 50, shape, generator=g).float() * 2.0 ** -23
    if kind == "heavy":                      # attention-mass-like: a few large values over a small floor
        return torch.rand(shape, generator=g) ** 12 * 40 + torch.rand(shape, generator=g) * 1e-3
    raise ValueError(kind)


@pytest.mark.parametrize("B,Hkv,d,n_keys,budget,sink,recent,dtype,kind", [
    (4, 8, 64, 20480, 4096, 256, 256, torch.bfloat16, "uniform"),   # 32 clusters of 4 blocks
    (4, 8, 16, 20001, 4097, 7, 9, torch.float32, "ties"),           # ragged lengths, odd capacity: scalar loads
    (1, 12, 32, 40960, 8192, 256, 256, torch.bfloat16, "equal"),    # 12 clusters of 8
    (3, 4, 8, 60000, 20000, 0, 0, torch.float32, "lowbits"),        # 12 clusters of 8, no forced rows
    (3, 4, 8, 40963, 8192, 100, 3, torch.float32, "heavy"),
    (4, 8, 8, 20480, 30000, 256, 256, torch.float32, "uniform"),    # under budget: nothing to choose
    (4, 8, 8, 20480, 512, 256, 256, torch.float32, "uniform"),      # forced rows only
])
@pytest.mark.parametrize("in_place", [False, True])
def test_evict_by_cluster_matches_oracle(B, Hkv, d, n_keys, budget, sink, recent, dtype, kind, in_place):
    """Shapes that take the one-cluster-per-segment launch (checked through the path diagnostic):
    selection through distributed shared memory, then the compaction by the same cluster, out of
    place and in place, against the oracle's full sort bit for bit."""
    g = torch.Generator().manual_seed(n_keys + budget)
    cap = n_keys + (5 if n_keys % 2 else 8)
    k = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    v = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    sc = _score_kind(kind, (B, Hkv, cap), g)
    pos = torch.randint(0, 1 << 20, (B, Hkv, cap), generator=g, dtype=torch.int32)
    cap_dst = cap if in_place else min(budget, n_keys) + 3
    ref = oracle.evict_topk(k, v, sc, n_keys, budget, sink, recent, cap_dst=cap_dst, pos_src=pos)
    ks, vs, ss, ps = k.to(DEV), v.to(DEV), sc.to(DEV), pos.to(DEV)
    if in_place:
        kd, vd, sd, pd = ks, vs, ss, ps
    else:
        kd = torch.zeros(B, Hkv, cap_dst, d, dtype=dtype, device=DEV)
        vd, sd = torch.zeros_like(kd), torch.zeros(B, Hkv, cap_dst, device=DEV)
        pd = torch.zeros(B, Hkv, cap_dst, dtype=torch.int32, device=DEV)
    kept = torch.full((B, Hkv, budget), -1, dtype=torch.int32, device=DEV)
    n_kept = R.evict_topk(ks, vs, ss, kd, vd, sd, n_keys, budget, sink, recent, pos_src=ps, pos_dst=pd,
                          kept_idx=kept)
    assert R.debug_last_path() == R.PATH_CLUSTER
    torch.cuda.synchronize()
    assert R.device_error() == 0
    assert n_kept == ref["n_kept"]
    assert torch.equal(kept.cpu()[:, :, :n_kept], ref["kept_idx"][:, :, :n_kept])
    assert torch.equal(kd.cpu()[:, :, :n_kept].view(torch.uint8), ref["k"][:, :, :n_kept].view(torch.uint8))
    assert torch.equal(vd.cpu()[:, :, :n_kept].view(torch.uint8), ref["v"][:, :, :n_kept].view(torch.uint8))
    assert torch.equal(sd.cpu()[:, :, :n_kept].double(), ref["score"][:, :, :n_kept])
    assert torch.equal(pd.cpu()[:, :, :n_kept], ref["pos"][:, :, :n_kept])
    if in_place:
        assert torch.equal(kd.cpu()[:, :, n_keys:], k[:, :, n_keys:])   # rows past the keys in use are untouched


@pytest.mark.parametrize("B,N,E,nq,k,pool,keep,mode,quant", [
    (1, 131072, 64, 4, 4096, 129, 256, "max", 0),     # the largest bank one cluster takes: 16 blocks
    (2, 100003, 32, 3, 3000, 5, 0, "mean", 0),        # ragged, mean pooling
    (3, 9000, 32, 2, 700, 1, 8, "max", 0),            # no pooling, clusters of 2
    (1, 70001, 32, 2, 9000, 9, 100, "max", 8),        # quantised scores: heavy ties
    (4, 65536, 32, 8, 60000, 129, 256, "max", 0),     # nearly everything selected
])
def test_retrieve_by_cluster_matches_oracle(B, N, E, nq, k, pool, keep, mode, quant):
    """Banks of up to 131,072 tokens: pooling and selection by one cluster per sequence (checked
    through the path diagnostic), against the oracle."""
    g = torch.Generator().manual_seed(N + k)
    bank = torch.randn(B, N, E, generator=g)
    if quant:
        bank = (bank * quant).round() / quant
    bank = bank.bfloat16()
    qs = torch.randn(B, nq, E, generator=g).bfloat16()
    p = dict(scale=0.25, pool_window=pool, n_keep_head=keep, n_keep_tail=keep)
    ref = oracle.retrieve_topk(bank, qs, N, k, pool_mode=mode, **p)
    idx = torch.full((B, k), -1, dtype=torch.int32, device=DEV)
    pooled = torch.zeros(B, N, device=DEV)
    n_out = R.retrieve_topk(bank.to(DEV), qs.to(DEV), N, k, idx, pooled_score_out=pooled,
                            pool_mode=R.POOL_MEAN if mode == "mean" else R.POOL_MAX, **p)
    assert R.debug_last_path() == R.PATH_CLUSTER
    torch.cuda.synchronize()
    assert n_out == ref["n_out"]
    assert_scores_close(pooled, ref["pooled"], 1.0)
    for b in range(B):
        assert_index_sets_match(idx[b, :n_out].cpu(), ref["idx"][b], ref["pooled"][b])
    # the same call without the optional pooled-score output selects the same tokens
    idx2 = torch.full((B, k), -1, dtype=torch.int32, device=DEV)
    R.retrieve_topk(bank.to(DEV), qs.to(DEV), N, k, idx2,
                    pool_mode=R.POOL_MEAN if mode == "mean" else R.POOL_MAX, **p)
    assert torch.equal(idx2, idx)


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    """Failure detection without a fault: the eviction's one-launch form is made to wait, for
    about a millisecond, on a flag that nothing sets.  Every block gives up, the kernel returns,
    REFORM_DEV_TIMEOUT shows in the caller's status word and in the library's per-device word,
    and the next ordinary call on the same workspace is bit-exact against the oracle."""
    g = torch.Generator().manual_seed(17)
    B, Hkv, n, d, budget = 1, 4, 9000, 64, 2048
    k = torch.randn(B, Hkv, n, d, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, n, d, generator=g).to(torch.bfloat16)
    sc = torch.rand(B, Hkv, n, generator=g)
    kd = torch.zeros(B, Hkv, budget, d, dtype=torch.bfloat16, device=DEV)
    vd, sd = torch.zeros_like(kd), torch.zeros(B, Hkv, budget, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert R.device_error() == 0
    R.debug_evict_wait_expiry(k.to(DEV), v.to(DEV), sc.to(DEV), kd, vd, sd, n, budget, 64, 64,
                              wait_cycles=2_000_000, dev_status=status)
    torch.cuda.synchronize()                                  # returns: nothing hangs, nothing faults
    assert status.item() == R.DEV_TIMEOUT
    assert R.device_error() == R.DEV_TIMEOUT                  # kept by the library too; reading clears it
    assert R.device_error() == 0
    kept = torch.zeros(B, Hkv, budget, dtype=torch.int32, device=DEV)
    R.evict_topk(k.to(DEV), v.to(DEV), sc.to(DEV), kd, vd, sd, n, budget, 64, 64, kept_idx=kept)
    ref = oracle.evict_topk(k, v, sc, n, budget, 64, 64, cap_dst=budget)
    assert torch.equal(kept.cpu(), ref["kept_idx"])
    assert torch.equal(kd.cpu().view(torch.int16), ref["k"].view(torch.int16))
    assert torch.equal(vd.cpu().view(torch.int16), ref["v"].view(torch.int16))
    assert R.device_error() == 0


def test_evict_without_optional_outputs():
    g = torch.Generator().manual_seed(1)
    k = torch.randn(1, 2, 600, 64, generator=g)
    sc = torch.rand(1, 2, 600, generator=g)
    ref = oracle.evict_topk(k, k, sc, 600, 128, 4, 4, cap_dst=128)
    kd = torch.zeros(1, 2, 128, 64, device=DEV)
    vd = torch.zeros_like(kd)
    sd = torch.zeros(1, 2, 128, device=DEV)
    R.evict_topk(k.to(DEV), k.to(DEV).clone(), sc.to(DEV), kd, vd, sd, 600, 128, 4, 4)
    assert torch.equal(kd.cpu(), ref["k"])


# ------------------------------------------------------------------ embed

@pytest.mark.parametrize("dtype,d,n_slots", [(torch.float32, 64, 2), (torch.bfloat16, 128, 8),
                                               (torch.bfloat16, 256, 3)])
def test_embed_append_matches_oracle(dtype, d, n_slots):
    g = torch.Generator().manual_seed(d)
    B, Hq, Hkv, Lc = 2, 8, 4, 77
    qs = torch.randn(B, Hq, Lc, d, generator=g).to(dtype)
    ks = (torch.randn(B, Hkv, Lc, d, generator=g) * 5).to(dtype)
    vs = (torch.randn(B, Hkv, Lc, d, generator=g) * 0.01).to(dtype)
    vs[0, 1, 3] = 0                                      # a zero vector stays zero
    kinds = [2, 1, 0, 2, 2, 1, 0, 2]
    sel = [(kinds[s], (3 * s + 1) % (Hq if kinds[s] == 0 else Hkv), s) for s in range(n_slots)]
    E = n_slots * d
    ref = torch.full((B, 100, E), 7.0).to(dtype)
    f64 = oracle.embed_append(ref, 11, sel, qs, ks, vs, want_f64=True)
    bank = torch.full((B, 100, E), 7.0).to(dtype).to(DEV)
    R.embed_append(bank, 11, sel, q_state=qs.to(DEV), k_state=ks.to(DEV), v_state=vs.to(DEV))
    torch.cuda.synchronize()
    got = bank.cpu()
    assert torch.equal(got[:, :11], ref[:, :11]) and torch.equal(got[:, 11 + Lc:], ref[:, 11 + Lc:])
    rows = got[:, 11:11 + Lc].double()
    exact = f64[:, 11:11 + Lc]
    # within one unit in the last place of the exact quotient: bf16 banks take fp32 arithmetic and
    # one rounding, fp32 banks take an fp64 norm and quotient and one rounding
    tol = 2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -23
    assert ((rows - exact).abs() <= tol * exact.abs() + 1e-30).all()
    if dtype == torch.bfloat16:
        same = (got[:, 11:11 + Lc] == ref[:, 11:11 + Lc]).float().mean().item()
        assert same > 0.99, f"only {same:.4f} of elements equal the oracle's rounding"


# --------------------------------------------------------------- retrieve

def _retrieve_case(w, N, pool, keep, k, seed):
    w = dataclasses.replace(w, N=N, k=k, pool_window=pool, keep_head=keep, keep_tail=keep)
    bank, qs, planted = synth.bank_and_queries(w, seed=seed)
    ref = oracle.retrieve_topk(bank, qs, N, k, scale=w.sim_scale, pool_window=pool,
                               n_keep_head=keep, n_keep_tail=keep)
    idx = torch.full((w.B, k), -1, dtype=torch.int32, device=DEV)
    ts = torch.zeros(w.B, N, device=DEV)
    pooled = torch.zeros(w.B, N, device=DEV)
    n_out = R.retrieve_topk(bank.to(DEV), qs.to(DEV), N, k, idx, scale=w.sim_scale, pool_window=pool,
                            n_keep_head=keep, n_keep_tail=keep, token_score_out=ts,
                            pooled_score_out=pooled)
    torch.cuda.synchronize()
    return w, ref, idx.cpu(), ts.cpu(), pooled.cpu(), planted, n_out


RETRIEVE_CASES = [
    # workload, N, pool, keep, k
    ("tiny", 8192, 1, 0, 256),
    ("tiny", 8192, 17, 8, 256),
    ("tiny", 5000, 129, 8, 300),          # ragged N, paper's window
    ("llama8b_128k", 9001, 129, 256, 1024),   # bf16 MMA path, nq = 4, ragged
    ("retrieval_1m", 4099, 5, 16, 512),       # nq = 64
    ("mistral7b_4x256k", 3000, 129, 256, 700),  # batch 4, nq = 8
]


@pytest.mark.parametrize("name,N,pool,keep,k", RETRIEVE_CASES)
def test_retrieve_matches_oracle(name, N, pool, keep, k):
    w, ref, idx, ts, pooled, planted, n_out = _retrieve_case(synth.WORKLOADS[name], N, pool, keep, k, seed=N)
    assert n_out == ref["n_out"]
    assert_scores_close(ts, ref["ts"], 1.0)
    assert_scores_close(pooled, ref["pooled"], 1.0)
    for b in range(w.B):
        assert_index_sets_match(idx[b, :n_out], ref["idx"][b], ref["pooled"][b])
        if pool == 1:
            assert set(planted[b]) <= set(idx[b].tolist())


@pytest.mark.parametrize("name,N,pool,keep,k", [
    ("tiny", 8192, 21, 8, 256),                # fp32, the paper's 20 neighbours
    ("tiny", 5000, 5, 0, 300),
    ("llama8b_128k", 9001, 21, 256, 1024),     # bf16 tensor-core scan, ragged, several selection blocks
    ("mistral7b_4x256k", 3000, 129, 16, 700),  # batch 4, a window of 129
])
def test_retrieve_with_mean_pooling_matches_oracle(name, N, pool, keep, k):
    """The mean-pool scorer variant (Appendix, detailed head selection, Step 3) through the same call."""
    w = dataclasses.replace(synth.WORKLOADS[name], N=N, k=k, pool_window=pool, keep_head=keep, keep_tail=keep)
    bank, qs, planted = synth.bank_and_queries(w, seed=N + pool)
    p = dict(scale=w.sim_scale, pool_window=pool, n_keep_head=keep, n_keep_tail=keep)
    ref = oracle.retrieve_topk(bank, qs, N, k, pool_mode="mean", **p)
    idx = torch.full((w.B, k), -1, dtype=torch.int32, device=DEV)
    ts = torch.zeros(w.B, N, device=DEV)
    pooled = torch.zeros(w.B, N, device=DEV)
    R.retrieve_topk(bank.to(DEV), qs.to(DEV), N, k, idx, token_score_out=ts, pooled_score_out=pooled,
                    pool_mode=R.POOL_MEAN, **p)
    torch.cuda.synchronize()
    assert_scores_close(ts, ref["ts"], 1.0)
    assert_scores_close(pooled, ref["pooled"], 1.0)
    for b in range(w.B):
        assert_index_sets_match(idx[b].cpu(), ref["idx"][b], ref["pooled"][b])


def test_retrieve_window_wider_than_the_bank():
    g = torch.Generator().manual_seed(12)
    bank = torch.randn(2, 50, 64, generator=g).bfloat16()
    qs = torch.randn(2, 3, 64, generator=g).bfloat16()
    ref = oracle.retrieve_topk(bank, qs, 50, 7, scale=0.5, pool_window=129, n_keep_head=1, n_keep_tail=1)
    idx = torch.full((2, 7), -1, dtype=torch.int32, device=DEV)
    pooled = torch.zeros(2, 50, device=DEV)
    R.retrieve_topk(bank.to(DEV), qs.to(DEV), 50, 7, idx, scale=0.5, pool_window=129, n_keep_head=1,
                    n_keep_tail=1, pooled_score_out=pooled)
    assert_scores_close(pooled, ref["pooled"], 1.0)
    # every token has the same pooled score (the global maximum): ties go to the lowest indices
    assert idx.cpu().tolist() == ref["idx"].tolist() == [[0, 1, 2, 3, 4, 5, 49]] * 2


def test_retrieve_ties_take_lowest_index_and_k_ge_n():
    bank = torch.ones(1, 700, 32, dtype=torch.bfloat16)
    qs = torch.ones(1, 3, 32, dtype=torch.bfloat16)
    idx = torch.full((1, 50), -1, dtype=torch.int32, device=DEV)
    R.retrieve_topk(bank.to(DEV), qs.to(DEV), 700, 50, idx, pool_window=9, n_keep_head=2, n_keep_tail=3)
    assert idx.cpu()[0].tolist() == list(range(47)) + [697, 698, 699]
    idx = torch.full((1, 900), -1, dtype=torch.int32, device=DEV)
    n = R.retrieve_topk(bank.to(DEV), qs.to(DEV), 700, 900, idx)
    assert n == 700 and idx.cpu()[0, :700].tolist() == list(range(700))


# ----------------------------------------------------------------- gather

@pytest.mark.parametrize("D,dtype", [(512, torch.float32), (4096, torch.bfloat16), (8, torch.bfloat16),
                                     (136, torch.bfloat16)])
def test_gather_matches_oracle(D, dtype):
    g = torch.Generator().manual_seed(D)
    src = torch.randn(2, 999, D, generator=g).to(dtype)
    idx = torch.randint(0, 999, (2, 257), generator=g, dtype=torch.int32)
    ref = oracle.gather(src, idx)
    dst = torch.zeros(2, 257, D, dtype=dtype, device=DEV)
    R.gather(src.to(DEV), idx.to(DEV), dst)
    torch.cuda.synchronize()
    assert torch.equal(dst.cpu().view(torch.uint8), ref.view(torch.uint8))


def test_gather_flags_bad_index_without_faulting():
    src = torch.randn(1, 10, 64, device=DEV)
    idx = torch.tensor([[3, 10, -1, 9]], dtype=torch.int32, device=DEV)
    dst = torch.full((1, 4, 64), 5.0, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    R.gather(src, idx, dst, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == R.DEV_BAD_INDEX
    assert R.device_error() & R.DEV_BAD_INDEX          # also kept by the library itself
    assert R.device_error() == 0                       # cleared by the read above
    R.gather(src, idx, dst)                            # no status word passed: still not silent
    assert R.device_error() == R.DEV_BAD_INDEX
    assert torch.equal(dst[0, 0], src[0, 3]) and torch.equal(dst[0, 3], src[0, 9])
    assert torch.all(dst[0, 1:3] == 0)


# ------------------------------------------------- recurrent pipeline (Tiny)

@pytest.mark.parametrize("sink,window", [(32, 128), (0, 1024)])
def test_tiny_recurrence_matches_oracle_step_by_step(sink, window):
    """Config 1 end to end: 8 chunk steps with eviction, each step fed the
    oracle's pre-step state so every step is judged on its own; needles
    survive every eviction."""
    w = dataclasses.replace(synth.WORKLOADS["tiny"], n_sink=sink, n_recent=sink, window=window)
    G = w.Hq // w.Hkv
    needles = synth.needle_positions(w)
    # oracle-side state
    ck = torch.zeros(w.B, w.Hkv, w.cap, w.d)
    cv = torch.zeros_like(ck)
    cs = torch.zeros(w.B, w.Hkv, w.cap, dtype=torch.float64)
    pos = torch.zeros(w.B, w.Hkv, w.cap, dtype=torch.int32)
    n_cache = 0
    swaps = 0
    for step in range(w.steps):
        q, kc, vc = synth.chunk_qkv(w, 0, step)
        ck[:, :, n_cache:n_cache + w.Lc] = kc
        cv[:, :, n_cache:n_cache + w.Lc] = vc
        pos[:, :, n_cache:n_cache + w.Lc] = torch.arange(step * w.Lc, (step + 1) * w.Lc, dtype=torch.int32)
        n = n_cache + w.Lc
        # GPU step from the oracle's state
        out, lse, score = _run_chunk(q, ck, cv, cs.float(), n_cache, window)
        o_ref, _ = oracle.attention(q, ck, cv, n_cache)
        assert_outputs_close(out, o_ref, w.dtype)
        s_ref = oracle.key_scores(q, ck, n_cache, window, score_in=cs.float(), accumulate=True)
        assert_scores_close(score[:, :, :n], s_ref[:, :, :n], window * G / n)
        ref = oracle.evict_topk(ck, cv, s_ref, n, w.budget, sink, sink, cap_dst=w.cap, pos_src=pos)
        kd = torch.zeros(w.B, w.Hkv, w.cap, w.d, device=DEV)
        vd = torch.zeros_like(kd)
        sd = torch.zeros(w.B, w.Hkv, w.cap, device=DEV)
        kept = torch.zeros(w.B, w.Hkv, w.budget, dtype=torch.int32, device=DEV)
        R.evict_topk(ck.to(DEV), cv.to(DEV), score, kd, vd, sd, n, w.budget, sink, sink, kept_idx=kept)
        for h in range(w.Hkv):
            swaps += assert_index_sets_match(kept[0, h].cpu(), ref["kept_idx"][0, h], s_ref[0, h])
            kept_pos = set(ref["pos"][0, h, :w.budget].tolist())
            seen = [p for p in needles if p < (step + 1) * w.Lc]
            # with no recent rows kept, a key late in its chunk has been seen by few queries and
            # may rightly lose (the oracle drops it too); the needle claim needs the recent window
            if sink:
                assert set(seen) <= kept_pos, f"needle evicted at step {step}"
        ck, cv, cs, pos = ref["k"], ref["v"], ref["score"], ref["pos"]
        n_cache = ref["n_kept"]
    assert swaps <= 4


def test_tiny_free_running_pipeline_with_driver():
    """Config 1 free-running: the binding's driver runs all 8 steps on the GPU alone, the oracle
    runs them alone.  After every step the kept token positions of every KV head must equal the
    oracle's, up to swaps between candidates whose oracle scores lie within 1e-4 (relative) of the
    cutoff, and the carried scores of the kept rows must agree to 1e-3.  A tolerated swap makes the
    two caches differ from then on, so the comparison ends there and the step, head and score gap
    of that first divergence are reported."""
    import warnings
    from oracle_run import oracle_free_run
    w = synth.WORKLOADS["tiny"]
    G = w.Hq // w.Hkv
    cache = LayerCache(w.B, w.Hkv, w.d, w.cap, w.budget, w.n_sink, w.n_recent, w.dtype, DEV)
    out = torch.zeros(w.B, w.Hq, w.Lc, w.d, device=DEV)
    pos = torch.zeros(w.B, w.Hkv, w.cap, dtype=torch.int64)            # token position of every GPU cache row
    for st in oracle_free_run(w):
        step, n, n_cache = st["step"], st["n"], st["n_cache_before"]
        q, kc, vc = synth.chunk_qkv(w, 0, step)
        cache.write_chunk(kc.to(DEV), vc.to(DEV))
        cache.attend(q.to(DEV), out, w.window)
        pos[:, :, n_cache:n] = torch.arange(step * w.Lc, (step + 1) * w.Lc)
        gpu_scores = cache.score[cache.cur][:, :, :n].cpu()
        assert_scores_close(gpu_scores, st["scores"][:, :, :n], w.window * G / n)
        n_kept = cache.evict()
        assert n_kept == st["n_kept"]
        kept = cache.kept_idx.cpu().long()
        swaps = 0
        for h in range(w.Hkv):
            swaps += assert_index_sets_match(kept[0, h, :n_kept], st["kept_idx"][0, h, :n_kept],
                                             st["scores"][0, h])
        pos[:, :, :n_kept] = torch.gather(pos, 2, kept[:, :, :n_kept])
        if swaps:
            both = [sorted(set(kept[0, h].tolist()) ^ set(st["kept_idx"][0, h].tolist())) for h in range(w.Hkv)]
            gap = max(abs(float(st["scores"][0, h][a] - st["scores"][0, h][b]))
                      for h in range(w.Hkv) for a in both[h] for b in both[h])
            warnings.warn(f"free run diverged at step {step} by a tolerated swap (score gap {gap:.3e}); "
                          "later steps are judged by the step-by-step test only")
            return
        assert torch.equal(pos[:, :, :n_kept], st["pos"][:, :, :n_kept].long())
        kd = cache.k[cache.cur][:, :, :n_kept].cpu()
        assert torch.equal(kd, st["k"][:, :, :n_kept])                 # same rows, bit for bit
        assert torch.equal(cache.v[cache.cur][:, :, :n_kept].cpu(), st["v"][:, :, :n_kept])
        assert_scores_close(cache.score[cache.cur][:, :, :n_kept], st["score"][:, :, :n_kept], w.window * G / n)


def test_chunk_step_seeded_random_shapes():
    """Sixty seeded shapes of the tensor-core chunk step (group sizes 1-8, chunk lengths and cache
    sizes on and off the 128 tile grid, windows 1 .. Lc, padded capacity, both score modes), each
    compared with the oracle in full."""
    import random
    rnd = random.Random(20250601)
    for case in range(60):
        B = rnd.choice([1, 1, 2]); Hkv = rnd.choice([1, 2, 3]); G = rnd.choice([1, 2, 3, 4, 5, 8])
        Lc = rnd.choice([1, 2, 5, 17, 64, 127, 128, 129, 200, 256, 257, 300, 383, 384, 500, 641])
        n_cache = rnd.choice([0, 0, 1, 63, 128, 130, 255, 256, 300, 512, 777])
        if Lc * G <= 16:
            Lc += 17                                   # decode-shaped steps have tests of their own
        W = rnd.choice([1, min(Lc, 7), min(Lc, 128), Lc])
        cap = n_cache + Lc + rnd.choice([0, 5, 64])
        acc = rnd.choice([True, False])
        g = torch.Generator().manual_seed(case * 7919 + 13)
        q = (torch.randn(B, Hkv * G, Lc, 128, generator=g) * rnd.choice([1.0, 1.0, 3.0])).to(torch.bfloat16)
        k = torch.randn(B, Hkv, cap, 128, generator=g).to(torch.bfloat16)
        v = torch.randn(B, Hkv, cap, 128, generator=g).to(torch.bfloat16)
        carry = torch.rand(B, Hkv, cap, generator=g)
        qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
        score = carry.clone().to(DEV)
        out = torch.empty_like(qd)
        lse = torch.empty(B, Hkv * G, Lc, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        R.chunk_step(qd, kd, vd, out, score, n_cache, W, lse=lse,
                     flags=R.SCORE_ACCUMULATE if acc else 0, dev_status=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        n = n_cache + Lc
        o_ref, l_ref = oracle.attention(q, k[:, :, :n].contiguous(), v[:, :, :n].contiguous(), n_cache)
        assert_outputs_close(out, o_ref, torch.bfloat16)
        assert (lse.cpu().double() - l_ref).abs().max() < 3e-3, case
        s_ref = oracle.key_scores(q, k[:, :, :n].contiguous(), n_cache, W,
                                  score_in=carry[:, :, :n].contiguous(), accumulate=acc)
        assert_scores_close(score[:, :, :n], s_ref[:, :, :n], W * G / n)


def test_gather_reads_rows_out_of_pinned_host_memory():
    """The gather source may stay in page-locked host memory: same bytes as from device memory."""
    g = torch.Generator().manual_seed(11)
    src = torch.randn(2, 5000, 1024, generator=g).to(torch.bfloat16).pin_memory()
    idx = torch.stack([torch.sort(torch.randperm(5000, generator=g)[:300]).values for _ in range(2)]).to(torch.int32)
    dst = torch.zeros(2, 300, 1024, dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    R.gather(src, idx.to(DEV), dst, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.equal(dst.cpu().view(torch.int16), oracle.gather(src, idx).view(torch.int16))


# ------------------------------------------------------------------- rope

@pytest.mark.parametrize("dtype,d,interleaved,pos0", [
    (torch.bfloat16, 128, False, 0), (torch.bfloat16, 128, False, 1000000), (torch.bfloat16, 64, True, 40960),
    (torch.float32, 64, False, 8191), (torch.float32, 32, True, 5), (torch.float32, 128, False, 1000000),
])
def test_rope_matches_oracle(dtype, d, interleaved, pos0):
    g = torch.Generator().manual_seed(d + pos0 % 97)
    x = torch.randn(2, 3, 150, d, generator=g).to(dtype)
    ref = oracle.rope(x, 7, 131, pos0, base=500000.0, interleaved=interleaved)
    xd = x.to(DEV)
    yd = torch.full_like(xd, 3.0)
    R.rope(xd, yd, 7, 131, pos0, theta_base=500000.0, interleaved=interleaved)
    got = yd.cpu()
    assert torch.all(got[:, :, :7] == 3.0) and torch.all(got[:, :, 138:] == 3.0)   # untouched rows
    a, b = got[:, :, 7:138].double(), ref[:, :, 7:138].double()
    # both sides are rounded to dtype: they may land one unit in the last place apart (spacing is
    # up to 2^-7 of the value in bf16); the fp32 rotation itself is good to a few fp32 ulps
    ulp = 2.0 ** -7 if dtype == torch.bfloat16 else 2.0 ** -21
    assert ((a - b).abs() <= ulp * b.abs() + 1e-6).all()
    if dtype == torch.bfloat16:
        assert (got[:, :, 7:138] == ref[:, :, 7:138]).float().mean().item() > 0.99
    R.rope(xd, xd, 7, 131, pos0, theta_base=500000.0, interleaved=interleaved)          # in place
    assert torch.equal(xd[:, :, 7:138], yd[:, :, 7:138])
    assert torch.equal(xd.cpu()[:, :, :7], x[:, :, :7])


def test_chunk_step_on_rotated_operands():
    """One recurrence step as a model would run it: un-rotated cache and chunk keys are rotated at
    the consecutive ids of the moment (cache row r -> r, chunk row i -> n_cache + i), queries at
    n_cache + i, then the chunk step; against the oracle doing the same in fp64."""
    q, k, v, carry = _case(1, 8, 2, 128, 200, 300, torch.bfloat16, seed=41)
    n_cache, n = 300, 500
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    q_rot, k_rot = torch.empty_like(qd), kd.clone()
    R.rope(qd, q_rot, 0, 200, n_cache)
    R.rope(kd, k_rot, 0, n, 0)
    out = torch.empty_like(qd)
    score = carry.to(DEV).clone()
    R.chunk_step(q_rot, k_rot, vd, out, score, n_cache, 128, flags=R.SCORE_ACCUMULATE)
    qo, ko = oracle.rope(q, 0, 200, n_cache), oracle.rope(k, 0, n, 0)
    o_ref, _ = oracle.attention(qo, ko, v, n_cache)
    assert_outputs_close(out, o_ref, torch.bfloat16)
    s_ref = oracle.key_scores(qo, ko, n_cache, 128, score_in=carry, accumulate=True)
    assert_scores_close(score[:, :, :n], s_ref[:, :, :n], 128 * 4 / n)


@pytest.mark.parametrize("B,Hq,Hkv,d,Lc,n_cache,dtype,W,flags,theta", [
    (1, 8, 2, 128, 300, 200, torch.bfloat16, 128, 0, 0.0),                 # tensor-core path: query tiles rotated at load
    (2, 4, 2, 128, 257, 0, torch.bfloat16, 257, 0, 500000.0),              # first step, every row scores, Llama-3 base
    (1, 8, 2, 128, 200, 5000, torch.bfloat16, 64, R.ROPE_INTERLEAVED, 0.0),  # interleaved pairs, positions in the thousands
    (1, 4, 1, 128, 129, 77, torch.bfloat16, 1, R.NO_SCORE, 0.0),           # attention only
    (1, 4, 2, 64, 192, 100, torch.float32, 128, 0, 0.0),                   # CUDA-core path (Tiny's shapes)
    (1, 8, 2, 128, 1, 1500, torch.bfloat16, 1, 0, 0.0),                    # decode-shaped step
    (1, 4, 2, 64, 96, 40, torch.bfloat16, 32, R.ROPE_INTERLEAVED, 0.0),    # bf16 on the CUDA-core path
])
def test_chunk_step_applies_rope_inside_the_call(B, Hq, Hkv, d, Lc, n_cache, dtype, W, flags, theta):
    """REFORM_ROPE: the caller passes un-rotated queries and keys (the cache keeps them un-rotated,
    because every compression renumbers its rows) and the call rotates them at the ids of the moment
    -- cache and chunk keys at 0 .. n-1, chunk queries at n_cache + i -- before attending and
    scoring; q and k are left as they were.  Against the oracle rotating in fp64 and then attending."""
    q, k, v, carry = _case(B, Hq, Hkv, d, Lc, n_cache, dtype, seed=Lc + n_cache)
    n = n_cache + Lc
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    out = torch.full_like(qd, float("nan"))
    lse = torch.full(q.shape[:3], float("nan"), device=DEV)
    score = carry.to(DEV).clone()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    R.chunk_step(qd, kd, vd, out, score, n_cache, W, lse=lse, flags=R.SCORE_ACCUMULATE | R.ROPE | flags,
                 rope_theta=theta, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.equal(qd.cpu(), q) and torch.equal(kd.cpu(), k)          # inputs untouched
    base = theta or 10000.0
    inter = bool(flags & R.ROPE_INTERLEAVED)
    qo = oracle.rope(q, 0, Lc, n_cache, base=base, interleaved=inter)
    ko = oracle.rope(k, 0, n, 0, base=base, interleaved=inter)
    o_ref, l_ref = oracle.attention(qo, ko, v, n_cache)
    assert_outputs_close(out, o_ref, dtype)
    assert (lse.cpu().double() - l_ref).abs().max() < (3e-3 if dtype == torch.bfloat16 else 1e-4)
    if flags & R.NO_SCORE:
        assert torch.equal(score.cpu(), carry)
    else:
        s_ref = oracle.key_scores(qo, ko, n_cache, W, score_in=carry, accumulate=True)
        assert_scores_close(score[:, :, :n], s_ref[:, :, :n], W * (Hq // Hkv) / n)
    # and it equals the two-call form (reform_rope, then the plain step) bit for bit
    q_rot, k_rot = torch.empty_like(qd), kd.clone()
    R.rope(qd, q_rot, 0, Lc, n_cache, theta_base=theta, interleaved=inter)
    R.rope(kd, k_rot, 0, n, 0, theta_base=theta, interleaved=inter)
    out2 = torch.empty_like(qd)
    score2 = carry.to(DEV).clone()
    R.chunk_step(q_rot, k_rot, vd, out2, score2, n_cache, W, flags=R.SCORE_ACCUMULATE | (flags & R.NO_SCORE))
    assert torch.equal(out2, out) and torch.equal(score2, score)


def test_checkpoint_and_resume_is_bit_identical():
    """All recurrent state is caller-owned (cache K/V, carried scores, n_cache, bank rows written so
    far), so a checkpoint is a copy of those buffers: 8 chunk steps straight against 4 steps,
    copy-out to the host, copy-in to fresh buffers, 4 more steps -- the same bits everywhere."""
    w = synth.WORKLOADS["tiny"]
    sel = synth.head_selection(dataclasses.replace(w, n_slots=2, slot_dim=w.d))
    E = 2 * w.d

    def new_state():
        cache = LayerCache(w.B, w.Hkv, w.d, w.cap, w.budget, w.n_sink, w.n_recent, w.dtype, DEV)
        bank = torch.zeros(w.B, w.T, E, dtype=w.dtype, device=DEV)
        return cache, bank

    def run(cache, bank, steps):
        out = torch.zeros(w.B, w.Hq, w.Lc, w.d, device=DEV)
        outs = []
        for step in steps:
            q, kc, vc = synth.chunk_qkv(w, 0, step)
            q, kc, vc = q.to(DEV), kc.to(DEV), vc.to(DEV)
            cache.write_chunk(kc, vc)
            cache.attend(q, out, w.window)
            R.embed_append(bank, step * w.Lc, sel, q_state=q, k_state=kc, v_state=vc)
            cache.evict()
            outs.append(out.clone())
        return outs

    c1, b1 = new_state()
    outs1 = run(c1, b1, range(8))
    c2, b2 = new_state()
    outs2 = run(c2, b2, range(4))
    # checkpoint: everything the recurrence carries, to the host ...
    ck = dict(k=c2.k[c2.cur].cpu(), v=c2.v[c2.cur].cpu(), score=c2.score[c2.cur].cpu(), n_cache=c2.n_cache,
              bank=b2.cpu())
    del c2, b2
    # ... and back into fresh buffers
    c3, b3 = new_state()
    c3.k[c3.cur].copy_(ck["k"])
    c3.v[c3.cur].copy_(ck["v"])
    c3.score[c3.cur].copy_(ck["score"])
    c3.n_cache = c3.n_keys = ck["n_cache"]
    b3.copy_(ck["bank"])
    outs2 += run(c3, b3, range(4, 8))
    for a, b in zip(outs1, outs2):
        assert torch.equal(a, b)
    n = c1.n_cache
    assert c3.n_cache == n == w.budget
    assert torch.equal(c1.k[c1.cur][:, :, :n], c3.k[c3.cur][:, :, :n])
    assert torch.equal(c1.v[c1.cur][:, :, :n], c3.v[c3.cur][:, :, :n])
    assert torch.equal(c1.score[c1.cur][:, :, :n], c3.score[c3.cur][:, :, :n])
    assert torch.equal(b1, b3)
    # and the gather phase over the resumed bank picks the same tokens
    _, queries, _ = synth.bank_and_queries(dataclasses.replace(w, n_slots=2, slot_dim=w.d, N=256, n_planted=0))
    idx = [torch.zeros(w.B, w.k, dtype=torch.int32, device=DEV) for _ in range(2)]
    for bank, i in ((b1, idx[0]), (b3, idx[1])):
        R.retrieve_topk(bank, queries.to(DEV), w.T, w.k, i, scale=0.5, pool_window=w.pool_window,
                        n_keep_head=w.keep_head, n_keep_tail=w.keep_tail)
    assert torch.equal(idx[0], idx[1])


def test_evict_seeded_random_shapes():
    """Eighty seeded shapes of the cache compression (1 to 12 segments, 1 to 40,000 keys, budgets from
    a handful to nearly everything, sink / recent rows from none to most of the budget, score
    distributions from continuous to heavily tied, padded capacities so that vector and scalar key
    loads both occur, with and without the position map and the kept-index output), each compared
    bit for bit with the oracle's full sort.  Most take the one-launch form; shapes with many
    segments take the block-per-segment or per-pass forms."""
    import random
    rnd = random.Random(20250602)
    for case in range(80):
        B = rnd.choice([1, 1, 2, 3]); Hkv = rnd.choice([1, 2, 4])
        n = rnd.choice([1, 2, 7, 33, 500, 1023, 1024, 4095, 4096, 8191, 8192, 8193, 12000, 16385, 30000, 40000])
        budget = max(1, min(n + rnd.choice([-1, 0, 5]), rnd.choice([1, 8, 100, n // 5 + 1, n // 2 + 1, n - 1, n])))
        sink = rnd.choice([0, 0, 1, 4, budget // 3])
        recent = rnd.choice([0, 0, 1, 4, budget // 3])
        if sink + recent > budget or sink + recent > n:
            sink, recent = 0, min(recent, budget, n) // 2
        cap = n + rnd.choice([0, 1, 3, 4, 8])
        d = rnd.choice([4, 8, 64])
        dtype = rnd.choice([torch.float32, torch.bfloat16]) if d >= 8 else torch.float32
        g = torch.Generator().manual_seed(case * 104729 + 7)
        k = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
        v = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
        kind = rnd.choice(["uniform", "heavy_tail", "tied", "two_level", "constant", "signed"])
        u = torch.rand(B, Hkv, cap, generator=g)
        sc = {"uniform": u, "heavy_tail": torch.exp(8 * u) / 2981.0, "tied": (u * 7).floor() / 7,
              "two_level": 1.0 + (u * 40).floor() * 2.0 ** -23, "constant": torch.full_like(u, 0.25),
              "signed": (u - 0.5) * 3}[kind]
        with_pos, with_kept = rnd.random() < 0.5, rnd.random() < 0.7
        pos = torch.randint(0, 1 << 20, (B, Hkv, cap), generator=g, dtype=torch.int32) if with_pos else None
        ref = oracle.evict_topk(k, v, sc, n, budget, sink, recent, cap_dst=budget, pos_src=pos)
        kd = torch.zeros(B, Hkv, budget, d, dtype=dtype, device=DEV)
        vd, sd = torch.zeros_like(kd), torch.zeros(B, Hkv, budget, device=DEV)
        pd = torch.zeros(B, Hkv, budget, dtype=torch.int32, device=DEV) if with_pos else None
        kept = torch.full((B, Hkv, budget), -1, dtype=torch.int32, device=DEV) if with_kept else None
        status = "case %d: B %d Hkv %d n %d budget %d sink %d recent %d cap %d %s" % (
            case, B, Hkv, n, budget, sink, recent, cap, kind)
        n_kept = R.evict_topk(k.to(DEV), v.to(DEV), sc.to(DEV), kd, vd, sd, n, budget, sink, recent,
                              pos_src=pos.to(DEV) if with_pos else None, pos_dst=pd, kept_idx=kept)
        torch.cuda.synchronize()
        assert n_kept == ref["n_kept"], status
        if with_kept:
            assert torch.equal(kept.cpu()[:, :, :n_kept], ref["kept_idx"][:, :, :n_kept]), status
        assert torch.equal(kd.cpu()[:, :, :n_kept].view(torch.uint8), ref["k"][:, :, :n_kept].view(torch.uint8)), status
        assert torch.equal(vd.cpu()[:, :, :n_kept].view(torch.uint8), ref["v"][:, :, :n_kept].view(torch.uint8)), status
        assert torch.equal(sd.cpu()[:, :, :n_kept].double(), ref["score"][:, :, :n_kept]), status
        if with_pos:
            assert torch.equal(pd.cpu()[:, :, :n_kept], ref["pos"][:, :, :n_kept]), status
    assert R.device_error() == 0


def test_two_host_threads_on_their_own_streams():
    """The library's per-process state (launch-form caches, epochs, counters) under two host
    threads that call it at the same time, each on its own stream with its own buffers and
    workspaces: thirty rounds of cache compression (cooperative and cluster forms) and token
    selection per thread, every result equal to the oracle's."""
    import threading
    g = torch.Generator().manual_seed(31)
    cases = []
    for n, budget, B, Hkv in ((9000, 2048, 1, 4), (20480, 4096, 4, 8)):
        k = torch.randn(B, Hkv, n, 8, generator=g)
        sc = torch.rand(B, Hkv, n, generator=g)
        cases.append((k, sc, n, budget, oracle.evict_topk(k, k, sc, n, budget, 16, 16, cap_dst=budget)))
    N, E, kk = 20000, 32, 1500
    bank = torch.randn(1, N, E, generator=g).bfloat16()
    qs = torch.randn(1, 3, E, generator=g).bfloat16()
    rp = dict(scale=0.25, pool_window=9, n_keep_head=4, n_keep_tail=4)
    rref = oracle.retrieve_topk(bank, qs, N, kk, **rp)
    errors = []

    def worker(tid):
        try:
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                dev = [(k.to(DEV), sc.to(DEV)) for k, sc, _, _, _ in cases]
                bank_d, qs_d = bank.to(DEV), qs.to(DEV)
                ws = torch.empty(64 << 20, dtype=torch.uint8, device=DEV)
                for it in range(30):
                    for (k, sc, n, budget, ref), (kd_src, sc_d) in zip(cases, dev):
                        B, Hkv = k.shape[:2]
                        kd = torch.zeros(B, Hkv, budget, 8, device=DEV)
                        vd, sd = torch.zeros_like(kd), torch.zeros(B, Hkv, budget, device=DEV)
                        kept = torch.zeros(B, Hkv, budget, dtype=torch.int32, device=DEV)
                        R.evict_topk(kd_src, kd_src, sc_d, kd, vd, sd, n, budget, 16, 16, kept_idx=kept, ws=ws,
                                     stream=st)
                        st.synchronize()
                        assert torch.equal(kept.cpu(), ref["kept_idx"]), (tid, it, n)
                        assert torch.equal(kd.cpu(), ref["k"]), (tid, it, n)
                    idx = torch.full((1, kk), -1, dtype=torch.int32, device=DEV)
                    R.retrieve_topk(bank_d, qs_d, N, kk, idx, ws=ws, stream=st, **rp)
                    st.synchronize()
                    assert_index_sets_match(idx[0].cpu(), rref["idx"][0], rref["pooled"][0])
        except Exception as e:   # reported by the main thread
            errors.append((tid, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert R.device_error() == 0


def test_evict_in_place_seeded_random_shapes():
    """Fifty seeded shapes of the in-place cache compression (destinations == sources), which always
    takes the one-cluster-per-segment launch: 1 to 12 segments of 1 to 131,072 keys (clusters of 1
    to 16 blocks), capacities that allow and forbid vector key loads, all score distributions of
    the out-of-place fuzz, each compared bit for bit with the oracle."""
    import random
    rnd = random.Random(20250603)
    for case in range(50):
        B = rnd.choice([1, 1, 2, 3]); Hkv = rnd.choice([1, 2, 4])
        n = rnd.choice([1, 2, 9, 500, 4096, 8191, 8192, 8193, 16385, 30000, 40000, 65537, 100000, 131072])
        if n > 50000:
            B, Hkv = 1, rnd.choice([1, 2])
        budget = max(1, min(n + rnd.choice([-1, 0, 5]), rnd.choice([1, 8, 100, n // 5 + 1, n // 2 + 1, n - 1, n])))
        sink = rnd.choice([0, 0, 1, 4, budget // 3])
        recent = rnd.choice([0, 0, 1, 4, budget // 3])
        if sink + recent > budget or sink + recent > n:
            sink, recent = 0, min(recent, budget, n) // 2
        cap = n + rnd.choice([0, 1, 3, 4, 8])
        d = rnd.choice([4, 8, 64])
        dtype = rnd.choice([torch.float32, torch.bfloat16]) if d >= 8 else torch.float32
        g = torch.Generator().manual_seed(case * 7919 + 11)
        k = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
        v = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
        kind = rnd.choice(["uniform", "heavy_tail", "tied", "two_level", "constant", "signed"])
        u = torch.rand(B, Hkv, cap, generator=g)
        sc = {"uniform": u, "heavy_tail": torch.exp(8 * u) / 2981.0, "tied": (u * 7).floor() / 7,
              "two_level": 1.0 + (u * 40).floor() * 2.0 ** -23, "constant": torch.full_like(u, 0.25),
              "signed": (u - 0.5) * 3}[kind]
        with_pos, with_kept = rnd.random() < 0.5, rnd.random() < 0.7
        pos = torch.randint(0, 1 << 20, (B, Hkv, cap), generator=g, dtype=torch.int32) if with_pos else None
        ref = oracle.evict_topk(k, v, sc, n, budget, sink, recent, cap_dst=cap, pos_src=pos)
        kd, vd, sd = k.to(DEV), v.to(DEV), sc.to(DEV)
        pd = pos.to(DEV) if with_pos else None
        kept = torch.full((B, Hkv, budget), -1, dtype=torch.int32, device=DEV) if with_kept else None
        status = "case %d: B %d Hkv %d n %d budget %d sink %d recent %d cap %d d %d %s" % (
            case, B, Hkv, n, budget, sink, recent, cap, d, kind)
        n_kept = R.evict_topk(kd, vd, sd, kd, vd, sd, n, budget, sink, recent, pos_src=pd, pos_dst=pd,
                              kept_idx=kept)
        assert R.debug_last_path() == R.PATH_CLUSTER, status
        torch.cuda.synchronize()
        assert n_kept == ref["n_kept"], status
        if with_kept:
            assert torch.equal(kept.cpu()[:, :, :n_kept], ref["kept_idx"][:, :, :n_kept]), status
        assert torch.equal(kd.cpu()[:, :, :n_kept].view(torch.uint8), ref["k"][:, :, :n_kept].view(torch.uint8)), status
        assert torch.equal(vd.cpu()[:, :, :n_kept].view(torch.uint8), ref["v"][:, :, :n_kept].view(torch.uint8)), status
        assert torch.equal(sd.cpu()[:, :, :n_kept].double(), ref["score"][:, :, :n_kept]), status
        if with_pos:
            assert torch.equal(pd.cpu()[:, :, :n_kept], ref["pos"][:, :, :n_kept]), status
        assert torch.equal(kd.cpu()[:, :, n:], k[:, :, n:]), status
    assert R.device_error() == 0


def test_retrieve_seeded_random_shapes():
    """Forty seeded shapes of the retrieval (bank lengths on and off the tile grids, 1 to 64 queries,
    row widths that take the tensor-core scan and ones that do not, fp32 and bf16, pooling windows 1
    to 257 in both modes, forced head / tail rows, k from 1 to beyond N), each against the oracle
    in full."""
    import random
    rnd = random.Random(20250603)
    for case in range(40):
        B = rnd.choice([1, 1, 2, 3])
        N = rnd.choice([1, 5, 127, 128, 129, 1000, 4095, 4096, 4097, 9000, 20000])
        E = rnd.choice([32, 64, 128, 192, 1024])
        nq = rnd.choice([1, 2, 4, 8, 17, 64])
        dtype = rnd.choice([torch.bfloat16, torch.bfloat16, torch.float32])
        pool = rnd.choice([1, 3, 5, 21, 129, 257])
        mode = rnd.choice(["max", "mean"])
        k = rnd.choice([1, 8, 100, N // 3 + 1, N, N + 10])
        keep_h = rnd.choice([0, 0, 1, 3]); keep_t = rnd.choice([0, 0, 2, 5])
        if keep_h + keep_t > min(k, N):
            keep_h = keep_t = 0
        g = torch.Generator().manual_seed(case * 7907 + 3)
        bank = torch.randn(B, N + rnd.choice([0, 3]), E, generator=g).to(dtype)
        qs = torch.randn(B, nq, E, generator=g).to(dtype)
        scale = 1.0 / E ** 0.5
        status = "case %d: B %d N %d E %d nq %d %s pool %d %s k %d keep %d/%d" % (
            case, B, N, E, nq, dtype, pool, mode, k, keep_h, keep_t)
        p = dict(scale=scale, pool_window=pool, n_keep_head=keep_h, n_keep_tail=keep_t)
        ref = oracle.retrieve_topk(bank, qs, N, k, pool_mode=mode, **p)
        idx = torch.full((B, max(k, 1)), -1, dtype=torch.int32, device=DEV)
        ts = torch.zeros(B, N, device=DEV)
        pooled = torch.zeros(B, N, device=DEV)
        n_out = R.retrieve_topk(bank.to(DEV), qs.to(DEV), N, k, idx, token_score_out=ts, pooled_score_out=pooled,
                                pool_mode=R.POOL_MEAN if mode == "mean" else R.POOL_MAX, **p)
        torch.cuda.synchronize()
        assert n_out == ref["n_out"], status
        # bf16 products are exact in fp32 and the sums differ from fp64 only by fp32 rounding
        assert_scores_close(ts, ref["ts"], 1.0)
        assert_scores_close(pooled, ref["pooled"], 1.0)
        for b in range(B):
            assert_index_sets_match(idx[b, :n_out].cpu(), ref["idx"][b], ref["pooled"][b], rel=1e-4)
    assert R.device_error() == 0


@pytest.mark.parametrize("B,Hkv,d,n_keys,budget,sink,recent,dtype", [
    (1, 2, 64, 1536, 512, 32, 32, torch.float32),      # Tiny's shapes
    (1, 8, 128, 40960, 8192, 256, 256, torch.bfloat16),  # config 2: 65,536 rows, more than one wave of the copy
    (4, 8, 128, 20480, 4096, 256, 256, torch.bfloat16),  # config 5: 32 segments
    (2, 3, 8, 9001, 9000, 0, 0, torch.float32),        # nearly everything kept: rows barely move
    (1, 1, 32, 300, 40, 16, 24, torch.bfloat16),       # forced rows only
    (1, 2, 64, 100, 128, 8, 8, torch.float32),         # under budget: every row stays where it is
])
def test_evict_in_place_matches_oracle(B, Hkv, d, n_keys, budget, sink, recent, dtype):
    """Destinations == sources: the kept rows move down inside their own buffers (one K/V buffer per
    layer instead of two).  Same bits as the oracle's out-of-place result in rows [0, n_kept)."""
    g = torch.Generator().manual_seed(n_keys + budget)
    cap = n_keys + 5
    k = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    v = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    sc = torch.rand(B, Hkv, cap, generator=g)
    sc[:, :, ::5] = (sc[:, :, ::5] * 8).floor() / 8
    pos = torch.randint(0, 1 << 20, (B, Hkv, cap), generator=g, dtype=torch.int32)
    ref = oracle.evict_topk(k, v, sc, n_keys, budget, sink, recent, cap_dst=cap, pos_src=pos)
    kd, vd, sd, pd = k.to(DEV), v.to(DEV), sc.to(DEV), pos.to(DEV)
    kept = torch.full((B, Hkv, budget), -1, dtype=torch.int32, device=DEV)
    n_kept = R.evict_topk(kd, vd, sd, kd, vd, sd, n_keys, budget, sink, recent, pos_src=pd, pos_dst=pd,
                          kept_idx=kept)
    torch.cuda.synchronize()
    assert R.device_error() == 0
    assert n_kept == ref["n_kept"]
    assert torch.equal(kept.cpu()[:, :, :n_kept], ref["kept_idx"][:, :, :n_kept])
    assert torch.equal(kd.cpu()[:, :, :n_kept].view(torch.uint8), ref["k"][:, :, :n_kept].view(torch.uint8))
    assert torch.equal(vd.cpu()[:, :, :n_kept].view(torch.uint8), ref["v"][:, :, :n_kept].view(torch.uint8))
    assert torch.equal(sd.cpu()[:, :, :n_kept].double(), ref["score"][:, :, :n_kept])
    assert torch.equal(pd.cpu()[:, :, :n_kept], ref["pos"][:, :, :n_kept])
    # rows past the keys in use are untouched
    assert torch.equal(kd.cpu()[:, :, n_keys:], k[:, :, n_keys:])


def test_evict_in_place_recurrence_equals_ping_pong():
    """Tiny's 8 chunk steps through the driver with one buffer set per layer (in-place compaction)
    against the same recurrence with two (out of place): the same outputs and the same cache, bit
    for bit, after every step."""
    w = synth.WORKLOADS["tiny"]
    two = LayerCache(w.B, w.Hkv, w.d, w.cap, w.budget, w.n_sink, w.n_recent, w.dtype, DEV)
    one = LayerCache(w.B, w.Hkv, w.d, w.cap, w.budget, w.n_sink, w.n_recent, w.dtype, DEV, n_buffers=1)
    out2 = torch.zeros(w.B, w.Hq, w.Lc, w.d, device=DEV)
    out1 = torch.zeros_like(out2)
    for step in range(w.steps):
        q, kc, vc = (t.to(DEV) for t in synth.chunk_qkv(w, 0, step))
        for cache, out in ((two, out2), (one, out1)):
            cache.write_chunk(kc, vc)
            cache.attend(q, out, w.window)
            cache.evict()
        n = one.n_cache
        assert n == two.n_cache and one.cur == 0
        assert torch.equal(out1, out2)
        assert torch.equal(one.k[0][:, :, :n], two.k[two.cur][:, :, :n])
        assert torch.equal(one.v[0][:, :, :n], two.v[two.cur][:, :, :n])
        assert torch.equal(one.score[0][:, :, :n], two.score[two.cur][:, :, :n])
        assert torch.equal(one.kept_idx, two.kept_idx)
