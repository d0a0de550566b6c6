"""Parity at the full sizes of the benchmark configurations, in the launch
configuration bench.py times.  Inputs are drawn on the GPU (seeded); the oracle
gets device-to-host copies of exactly the slices it checks and computes sampled
outputs one by one; whole-tensor claims are checked through properties that
hold at any size (mass conservation, order, forced rows, planted structure)."""
import dataclasses

import pytest
import torch

import oracle
import paper_2506_01215_b200 as R
from paper_2506_01215_b200 import synth

from parity import assert_index_sets_match, assert_outputs_close, assert_scores_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _sample_rows(Lc, seed):
    g = torch.Generator().manual_seed(seed)
    edge = [0, 1, 127, 128, 129, 255, 256, Lc // 2 - 1, Lc // 2, Lc - 129, Lc - 128, Lc - 2, Lc - 1]
    rnd = torch.randint(0, Lc, (35,), generator=g).tolist()
    return sorted(set(r for r in edge + rnd if 0 <= r < Lc))


def _chunk_step_spot_check(name, seq, groups, flags=R.SCORE_ACCUMULATE):
    w = synth.WORKLOADS[name]
    G = w.Hq // w.Hkv
    q, kc, vc = synth.chunk_qkv(w, 0, 1, device=DEV)
    k0, v0, s0 = synth.cache_state(w, 0, device=DEV)
    k = torch.cat([k0, kc], 2).contiguous()
    v = torch.cat([v0, vc], 2).contiguous()
    carry = torch.cat([s0, torch.zeros(w.B, w.Hkv, w.Lc, device=DEV)], 2).contiguous()
    score = carry.clone()
    out = torch.empty_like(q)
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    R.chunk_step(q, k, v, out, score, w.budget, w.window, lse=lse, flags=flags, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    n = w.cap
    # whole tensor: every scored query hands out one unit of mass
    new = score[:, :, :n].double().sum(-1) - carry[:, :, :w.budget].double().sum(-1)
    assert torch.allclose(new, torch.full_like(new, float(w.window * G)), rtol=1e-3)
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    rows = _sample_rows(w.Lc, 7)
    for g in groups:
        qs = q[seq:seq + 1, g * G:(g + 1) * G].cpu().contiguous()
        ks = k[seq:seq + 1, g:g + 1].cpu().contiguous()
        vs = v[seq:seq + 1, g:g + 1].cpu().contiguous()
        o_ref, l_ref = oracle.attention(qs, ks, vs, w.budget, rows=rows)
        assert_outputs_close(out[seq:seq + 1, g * G:(g + 1) * G][:, :, rows], o_ref, w.dtype)
        assert (lse[seq:seq + 1, g * G:(g + 1) * G][:, :, rows].cpu().double() - l_ref).abs().max() < 2e-3
        s_ref = oracle.key_scores(qs, ks, w.budget, w.window, score_in=carry[seq:seq + 1, g:g + 1].cpu(),
                                  accumulate=True)
        assert_scores_close(score[seq:seq + 1, g:g + 1, :n], s_ref[:, :, :n], w.window * G / n)


def test_chunk_step_llama8b_full_size_spot_check():
    """Configs 2 and 3: Hq 32, Hkv 8, d 128, chunk 32,768 over an 8,192-row cache."""
    _chunk_step_spot_check("llama8b_128k", 0, groups=[0, 5])


def test_chunk_step_mistral_batched_full_size_spot_check():
    """Config 5: batch of 4, chunk 16,384 over a 4,096-row cache."""
    _chunk_step_spot_check("mistral7b_4x256k", 2, groups=[3])
    _chunk_step_spot_check("mistral7b_4x256k", 0, groups=[7])


def test_evict_full_size_bit_exact():
    """8 KV heads x 40,960 keys -> 8,192, sink/recent 256, seeded scores with ties."""
    w = synth.WORKLOADS["llama8b_128k"]
    g = torch.Generator(device=DEV).manual_seed(3)
    k = torch.randn(w.B, w.Hkv, w.cap, w.d, generator=g, device=DEV).to(w.dtype)
    v = torch.randn(w.B, w.Hkv, w.cap, w.d, generator=g, device=DEV).to(w.dtype)
    sc = torch.rand(w.B, w.Hkv, w.cap, generator=g, device=DEV)
    sc[:, :, ::7] = (sc[:, :, ::7] * 16).floor() / 16          # a seventh of the scores tie heavily
    kd, vd, sd = torch.zeros_like(k), torch.zeros_like(v), torch.zeros_like(sc)
    kept = torch.zeros(w.B, w.Hkv, w.budget, dtype=torch.int32, device=DEV)
    R.evict_topk(k, v, sc, kd, vd, sd, w.cap, w.budget, w.n_sink, w.n_recent, kept_idx=kept)
    ref = oracle.evict_topk(k.cpu(), v.cpu(), sc.cpu(), w.cap, w.budget, w.n_sink, w.n_recent, cap_dst=w.cap)
    assert torch.equal(kept.cpu(), ref["kept_idx"])
    b = w.budget
    assert torch.equal(kd.cpu()[:, :, :b].view(torch.int16), ref["k"][:, :, :b].view(torch.int16))
    assert torch.equal(vd.cpu()[:, :, :b].view(torch.int16), ref["v"][:, :, :b].view(torch.int16))
    assert torch.equal(sd.cpu()[:, :, :b].double(), ref["score"][:, :, :b])


def test_embed_append_full_chunk():
    w = synth.WORKLOADS["llama8b_128k"]
    q, kc, vc = synth.chunk_qkv(w, 0, 2, device=DEV)
    sel = synth.head_selection(w)
    bank = torch.zeros(w.B, w.Lc + 64, w.E, dtype=w.dtype, device=DEV)
    R.embed_append(bank, 64, sel, q_state=q, k_state=kc, v_state=vc)
    ref = torch.zeros(w.B, w.Lc + 64, w.E, dtype=w.dtype)
    f64 = oracle.embed_append(ref, 64, sel, q.cpu(), kc.cpu(), vc.cpu(), want_f64=True)
    got = bank.cpu()
    assert ((got.double() - f64).abs() <= 2.0 ** -8 * f64.abs() + 1e-30).all()
    assert (got == ref).float().mean().item() > 0.995
    assert torch.all(got[:, :64] == 0)


@pytest.mark.parametrize("name", ["llama8b_128k", "retrieval_1m", "mistral7b_4x256k"])
def test_retrieve_and_gather_full_size(name):
    """Configs 2, 4, 5: full bank scan, pool 129, forced 256/256, top-k, then the gather."""
    w = synth.WORKLOADS[name]
    bank, qs, planted = synth.bank_and_queries(w, device=DEV)
    idx = torch.full((w.B, w.k), -1, dtype=torch.int32, device=DEV)
    ts = torch.empty(w.B, w.N, device=DEV)
    pooled = torch.empty(w.B, w.N, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    p = dict(scale=w.sim_scale, pool_window=w.pool_window, n_keep_head=w.keep_head, n_keep_tail=w.keep_tail)
    R.retrieve_topk(bank, qs, w.N, w.k, idx, token_score_out=ts, pooled_score_out=pooled, **p)
    torch.cuda.synchronize()
    ref = oracle.retrieve_topk(bank.cpu(), qs.cpu(), w.N, w.k, **p)
    assert_scores_close(ts, ref["ts"], 1.0)
    assert_scores_close(pooled, ref["pooled"], 1.0)
    for b in range(w.B):
        assert_index_sets_match(idx[b].cpu(), ref["idx"][b], ref["pooled"][b])
        got = set(idx[b].tolist())
        assert set(range(w.keep_head)) <= got and set(range(w.N - w.keep_tail, w.N)) <= got
        pl = torch.tensor(planted[b])
        assert (ts[b].cpu()[pl] - w.rho).abs().max() < 5e-3           # cosine 0.9 by construction
        # pooling spreads each planted score over its 129 neighbours, and n_planted * 129 exceeds
        # k, so the chosen tokens are whole neighbourhoods of the best planted rows: every chosen
        # token outside the forced ranges lies within the pooling radius of a planted row
        r = (w.pool_window - 1) // 2
        chosen = idx[b].cpu().long()
        chosen = chosen[(chosen >= w.keep_head) & (chosen < w.N - w.keep_tail)]
        dist = (chosen[:, None] - pl[None, :]).abs().min(dim=1).values
        assert int(dist.max()) <= r
        assert len(set(planted[b]) & got) >= (w.k - w.keep_head - w.keep_tail) // w.pool_window - 1
    # without pooling every planted row must be among the selected tokens
    idx1 = torch.full((w.B, w.k), -1, dtype=torch.int32, device=DEV)
    R.retrieve_topk(bank, qs, w.N, w.k, idx1, scale=w.sim_scale, pool_window=1,
                    n_keep_head=w.keep_head, n_keep_tail=w.keep_tail)
    for b in range(w.B):
        assert set(planted[b]) <= set(idx1[b].tolist())
    # gather of the selected rows; the oracle copies the same rows from a host copy of their slice
    D = w.D
    hidden = synth.hidden_rows(dataclasses.replace(w, B=1), device=DEV)
    dst = torch.empty(1, w.k, D, dtype=w.dtype, device=DEV)
    R.gather(hidden, idx[:1].contiguous(), dst, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    lo, hi = int(idx[0, 0]), int(idx[0, -1]) + 1
    step = 1 << 16                                                     # host copies of 64K-row slices
    for r0 in range(lo, hi, step):
        r1 = min(hi, r0 + step)
        m = (idx[0] >= r0) & (idx[0] < r1)
        if not m.any():
            continue
        local = (idx[0][m] - r0).cpu().reshape(1, -1)
        exp = oracle.gather(hidden[:, r0:r1].cpu().contiguous(), local)
        assert torch.equal(dst[0][m].cpu().view(torch.int16), exp[0].view(torch.int16))


def test_retrieval_bank_beyond_2_to_31_elements():
    """Largest sizes: a ragged 2,500,037-row bank (2.56e9 elements, 5.1 GB) against the full oracle."""
    w = dataclasses.replace(synth.WORKLOADS["retrieval_1m"], N=2_500_037, nq=2, k=4096, n_planted=32)
    bank, qs, planted = synth.bank_and_queries(w, device=DEV)
    assert bank.numel() > 2 ** 31
    idx = torch.full((w.B, w.k), -1, dtype=torch.int32, device=DEV)
    ts = torch.empty(w.B, w.N, device=DEV)
    pooled = torch.empty(w.B, w.N, device=DEV)
    p = dict(scale=w.sim_scale, pool_window=w.pool_window, n_keep_head=w.keep_head, n_keep_tail=w.keep_tail)
    R.retrieve_topk(bank, qs, w.N, w.k, idx, token_score_out=ts, pooled_score_out=pooled, **p)
    torch.cuda.synchronize()
    assert R.device_error() == 0
    ref = oracle.retrieve_topk(bank.cpu(), qs.cpu(), w.N, w.k, **p)
    assert_scores_close(ts, ref["ts"], 1.0)
    assert_scores_close(pooled, ref["pooled"], 1.0)
    assert_index_sets_match(idx[0].cpu(), ref["idx"][0], ref["pooled"][0])
    assert (ts[0].cpu()[torch.tensor(planted[0])] - w.rho).abs().max() < 5e-3


def test_evict_32_layers_batched_bit_exact():
    """Largest sizes: the batched call of config 3 (32 layers x 8 KV heads x 40,960 keys; K and V
    of 2.7 GB each, byte offsets past 2^31) against the oracle's full sort."""
    w = dataclasses.replace(synth.WORKLOADS["llama8b_128k"], B=32)
    g = torch.Generator(device=DEV).manual_seed(5)
    k = torch.randn(w.B, w.Hkv, w.cap, w.d, generator=g, device=DEV).to(w.dtype)
    v = torch.randn(w.B, w.Hkv, w.cap, w.d, generator=g, device=DEV).to(w.dtype)
    sc = torch.rand(w.B, w.Hkv, w.cap, generator=g, device=DEV)
    kd = torch.zeros(w.B, w.Hkv, w.budget, w.d, dtype=w.dtype, device=DEV)
    vd = torch.zeros_like(kd)
    sd = torch.zeros(w.B, w.Hkv, w.budget, device=DEV)
    kept = torch.zeros(w.B, w.Hkv, w.budget, dtype=torch.int32, device=DEV)
    R.evict_topk(k, v, sc, kd, vd, sd, w.cap, w.budget, w.n_sink, w.n_recent, kept_idx=kept)
    torch.cuda.synchronize()
    assert R.device_error() == 0
    ref = oracle.evict_topk(k.cpu(), v.cpu(), sc.cpu(), w.cap, w.budget, w.n_sink, w.n_recent,
                            cap_dst=w.budget)
    assert torch.equal(kept.cpu(), ref["kept_idx"])
    assert torch.equal(kd.cpu().view(torch.int16), ref["k"].view(torch.int16))
    assert torch.equal(vd.cpu().view(torch.int16), ref["v"].view(torch.int16))
    assert torch.equal(sd.cpu().double(), ref["score"])


def test_chunk_step_beyond_2_to_31_elements():
    """Largest sizes: 5 sequences x 32 heads x 131,072 rows x 128 (2.7e9 elements of Q and of O) in
    one call; sampled rows of the last sequence and head group, whose offsets pass 2^31."""
    w = dataclasses.replace(synth.WORKLOADS["mistral7b_4x256k"], B=5, Lc=131072, budget=1024, T=262144)
    G = w.Hq // w.Hkv
    q, kc, vc = synth.chunk_qkv(w, 0, 1, device=DEV)
    k0, v0, s0 = synth.cache_state(w, 0, device=DEV)
    k = torch.cat([k0, kc], 2).contiguous()
    v = torch.cat([v0, vc], 2).contiguous()
    del kc, vc
    assert q.numel() > 2 ** 31
    carry = torch.cat([s0, torch.zeros(w.B, w.Hkv, w.Lc, device=DEV)], 2).contiguous()
    score = carry.clone()
    out = torch.empty_like(q)
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    R.chunk_step(q, k, v, out, score, w.budget, w.window, lse=lse, flags=R.SCORE_ACCUMULATE,
                 dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    n = w.budget + w.Lc
    new = score[:, :, :n].double().sum(-1) - carry[:, :, :w.budget].double().sum(-1)
    assert torch.allclose(new, torch.full_like(new, float(w.window * G)), rtol=1e-3)
    rows = [0, 1, 127, 128, 4095, 65535, 65536, 100000, w.Lc - 129, w.Lc - 2, w.Lc - 1]
    for seq, g in ((4, 7), (0, 0)):
        qs = q[seq:seq + 1, g * G:(g + 1) * G].cpu().contiguous()
        ks = k[seq:seq + 1, g:g + 1].cpu().contiguous()
        vs = v[seq:seq + 1, g:g + 1].cpu().contiguous()
        o_ref, l_ref = oracle.attention(qs, ks, vs, w.budget, rows=rows)
        assert_outputs_close(out[seq:seq + 1, g * G:(g + 1) * G][:, :, rows], o_ref, w.dtype)
        assert (lse[seq:seq + 1, g * G:(g + 1) * G][:, :, rows].cpu().double() - l_ref).abs().max() < 2e-3
        s_ref = oracle.key_scores(qs, ks, w.budget, w.window, score_in=carry[seq:seq + 1, g:g + 1].cpu(),
                                  accumulate=True)
        assert_scores_close(score[seq:seq + 1, g:g + 1, :n], s_ref[:, :, :n], w.window * G / n)


@pytest.mark.parametrize("name,accumulate,needles_must_survive", [
    ("llama8b_128k", True, True), ("llama8b_1m_32l", False, True), ("llama8b_1m_32l", True, False)])
def test_recurrent_pipeline_full_size_keeps_needles(name, accumulate, needles_must_survive):
    """Configs 2 and 3 (one layer) end to end on the GPU: 4 and 32 chunk steps with their evictions.
    Positions are carried through the compaction, mass is conserved, and every eviction equals the
    oracle's full sort of the scores the GPU held before it (teacher forcing).  Every needle seen so
    far is still in every KV head's cache after every step -- except in the 32-step run with
    accumulated scores, where rows that have collected mass for many steps out-score a needle that
    has been scored once (the oracle evicts it as well), so only the equality with the oracle is
    asserted there."""
    w = synth.WORKLOADS[name]
    flags = R.SCORE_ACCUMULATE if accumulate else 0
    G = w.Hq // w.Hkv
    needles = set(synth.needle_positions(w))
    bufs = [[torch.zeros(w.B, w.Hkv, w.cap, w.d, dtype=w.dtype, device=DEV) for _ in range(2)] for _ in range(2)]
    sc = [torch.zeros(w.B, w.Hkv, w.cap, device=DEV) for _ in range(2)]
    pos = [torch.zeros(w.B, w.Hkv, w.cap, dtype=torch.int32, device=DEV) for _ in range(2)]
    out = torch.empty(w.B, w.Hq, w.Lc, w.d, dtype=w.dtype, device=DEV)
    cur, n_cache = 0, 0
    for step in range(w.steps):
        q, kc, vc = synth.chunk_qkv(w, 0, step, device=DEV)
        bufs[cur][0][:, :, n_cache:n_cache + w.Lc] = kc
        bufs[cur][1][:, :, n_cache:n_cache + w.Lc] = vc
        pos[cur][:, :, n_cache:n_cache + w.Lc] = torch.arange(step * w.Lc, (step + 1) * w.Lc, device=DEV,
                                                             dtype=torch.int32)
        before = sc[cur][:, :, :n_cache].double().sum(-1) * (1 if accumulate else 0)
        R.chunk_step(q, bufs[cur][0], bufs[cur][1], out, sc[cur], n_cache, w.window, flags=flags)
        after = sc[cur][:, :, :n_cache + w.Lc].double().sum(-1)
        assert torch.allclose(after - before, torch.full_like(after, float(w.window * G)), rtol=1e-3)
        nxt = 1 - cur
        n_keys = n_cache + w.Lc
        kept_idx = torch.zeros(w.B, w.Hkv, w.budget, dtype=torch.int32, device=DEV)
        n_cache = R.evict_topk(bufs[cur][0], bufs[cur][1], sc[cur], bufs[nxt][0], bufs[nxt][1], sc[nxt],
                               n_keys, w.budget, w.n_sink, w.n_recent, pos_src=pos[cur], pos_dst=pos[nxt],
                               kept_idx=kept_idx)
        ref = oracle.evict_topk(torch.zeros(w.B, w.Hkv, n_keys, 8, dtype=w.dtype),
                                torch.zeros(w.B, w.Hkv, n_keys, 8, dtype=w.dtype), sc[cur][:, :, :n_keys].cpu(),
                                n_keys, w.budget, w.n_sink, w.n_recent, cap_dst=w.budget)
        assert torch.equal(kept_idx.cpu()[:, :, :n_cache], ref["kept_idx"][:, :, :n_cache])
        cur = nxt
        kept = pos[cur][:, :, :n_cache].cpu()
        assert (kept[:, :, 1:] > kept[:, :, :-1]).all()               # order preserved
        seen = {p for p in needles if p < (step + 1) * w.Lc}
        for h in range(w.Hkv):
            if needles_must_survive:
                assert seen <= set(kept[0, h].tolist()), f"needle lost in head {h} at step {step}"
