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


def test_chunk_step_with_rope_full_size_spot_check():
    """Config 2's step with the rotary embedding applied inside the call (un-rotated q and k in,
    positions 0 .. 40,959 for the keys and 8,192 .. 40,959 for the queries): sampled rows of one KV
    group against the oracle rotating in fp64, and the whole group's score row."""
    w = synth.WORKLOADS["llama8b_128k"]
    G = w.Hq // w.Hkv
    g = 6
    q, kc, vc = synth.chunk_qkv(w, 0, 2, device=DEV)
    k0, v0, s0 = synth.cache_state(w, 1, device=DEV)
    k = torch.cat([k0, kc], 2).contiguous()
    v = torch.cat([v0, vc], 2).contiguous()
    carry = torch.cat([s0, torch.zeros(w.B, w.Hkv, w.Lc, device=DEV)], 2).contiguous()
    score = carry.clone()
    out = torch.empty_like(q)
    lse = torch.empty(q.shape[:3], dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    R.chunk_step(q, k, v, out, score, w.budget, w.window, lse=lse, flags=R.SCORE_ACCUMULATE | R.ROPE,
                 rope_theta=500000.0, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0 and R.device_error() == 0
    n = w.cap
    new = score[:, :, :n].double().sum(-1) - carry[:, :, :w.budget].double().sum(-1)
    assert torch.allclose(new, torch.full_like(new, float(w.window * G)), rtol=1e-3)
    rows = _sample_rows(w.Lc, 11)
    qs = oracle.rope(q[:, g * G:(g + 1) * G].cpu().contiguous(), 0, w.Lc, w.budget, base=500000.0)
    ks = oracle.rope(k[:, g:g + 1].cpu().contiguous(), 0, n, 0, base=500000.0)
    vs = v[:, g:g + 1].cpu().contiguous()
    o_ref, l_ref = oracle.attention(qs, ks, vs, w.budget, rows=rows)
    assert_outputs_close(out[:, g * G:(g + 1) * G][:, :, rows], o_ref, w.dtype)
    assert (lse[:, g * G:(g + 1) * G][:, :, rows].cpu().double() - l_ref).abs().max() < 3e-3
    s_ref = oracle.key_scores(qs, ks, w.budget, w.window, score_in=carry[:, g:g + 1].cpu(), accumulate=True)
    assert_scores_close(score[:, g:g + 1, :n], s_ref[:, :, :n], w.window * G / n)


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


def _spot_check_live_step(w, q, k, v, carry, score, out, lse, n_cache, window, accumulate, pairs, seed):
    """Teacher-forced check of one recurrence step that has just run on the GPU: the oracle gets
    device-to-host copies of the pre-step state of the listed (sequence, KV head) pairs and
    computes sampled output rows, their LSE and the whole score row."""
    G = w.Hq // w.Hkv
    n = n_cache + w.Lc
    rows = _sample_rows(w.Lc, seed)
    for b, g in pairs:
        qs = q[b:b + 1, g * G:(g + 1) * G].cpu().contiguous()
        ks = k[b:b + 1, g:g + 1, :n].cpu().contiguous()
        vs = v[b:b + 1, g:g + 1, :n].cpu().contiguous()
        o_ref, l_ref = oracle.attention(qs, ks, vs, n_cache, rows=rows)
        assert_outputs_close(out[b:b + 1, g * G:(g + 1) * G][:, :, rows], o_ref, w.dtype)
        assert (lse[b:b + 1, g * G:(g + 1) * G][:, :, rows].cpu().double() - l_ref).abs().max() < 2e-3
        s_ref = oracle.key_scores(qs, ks, n_cache, window, score_in=carry[b:b + 1, g:g + 1, :n].cpu(),
                                  accumulate=accumulate)
        assert_scores_close(score[b:b + 1, g:g + 1, :n], s_ref[:, :, :n], window * G / n)


def _recurrence_at_stated_size(w, accumulate, needles_must_survive, spot_step, spot_pairs):
    """Alg. 1 (ForwardChunk for every layer of every chunk) at a configuration's stated size, all on
    the GPU: w.steps chunks x w.layers layers x w.B sequences.  Checked at every (chunk, layer):
    mass conservation of the new scores, the eviction against the oracle's full sort of the scores
    the GPU held (teacher forcing), positions carried in ascending order.  Checked once per layer,
    at chunk spot_step(layer): sampled outputs, LSE and scores of spot_pairs(layer) against the
    oracle.  Needles: every needle of a sequence seen so far is in every KV head's cache of every
    layer after every chunk, where needles_must_survive."""
    flags = R.SCORE_ACCUMULATE if accumulate else 0
    G = w.Hq // w.Hkv
    needles = [set(synth.needle_positions(w, b)) for b in range(w.B)]
    assert len(set(map(frozenset, needles))) == w.B                       # they differ per sequence
    mk = lambda *shape, dt=w.dtype: [torch.zeros(*shape, dtype=dt, device=DEV) for _ in range(2)]
    layers = [dict(k=mk(w.B, w.Hkv, w.cap, w.d), v=mk(w.B, w.Hkv, w.cap, w.d),
                   sc=mk(w.B, w.Hkv, w.cap, dt=torch.float32), pos=mk(w.B, w.Hkv, w.cap, dt=torch.int32),
                   cur=0) for _ in range(w.layers)]
    out = torch.empty(w.B, w.Hq, w.Lc, w.d, dtype=w.dtype, device=DEV)
    lse = torch.empty(w.B, w.Hq, w.Lc, dtype=torch.float32, device=DEV)
    kept_idx = torch.zeros(w.B, w.Hkv, w.budget, dtype=torch.int32, device=DEV)
    zeros_kv = None
    n_cache, spot_checks = 0, 0
    for step in range(w.steps):
        n_keys = n_cache + w.Lc
        new_pos = torch.arange(step * w.Lc, (step + 1) * w.Lc, device=DEV, dtype=torch.int32)
        seen = [{p for p in needles[b] if p < (step + 1) * w.Lc} for b in range(w.B)]
        for layer, st in enumerate(layers):
            cur, nxt = st["cur"], 1 - st["cur"]
            k, v, sc, pos = st["k"][cur], st["v"][cur], st["sc"][cur], st["pos"][cur]
            q, kc, vc = synth.chunk_qkv(w, layer, step, device=DEV)
            k[:, :, n_cache:n_keys] = kc
            v[:, :, n_cache:n_keys] = vc
            pos[:, :, n_cache:n_keys] = new_pos
            spot = step == spot_step(layer)
            carry = sc.clone() if spot else None
            before = sc[:, :, :n_cache].double().sum(-1) * (1 if accumulate else 0)
            R.chunk_step(q, k, v, out, sc, n_cache, w.window, lse=lse, flags=flags)
            after = sc[:, :, :n_keys].double().sum(-1)
            assert torch.allclose(after - before, torch.full_like(after, float(w.window * G)), rtol=1e-3), \
                f"mass not conserved at chunk {step}, layer {layer}"
            if spot:
                _spot_check_live_step(w, q, k, v, carry, sc, out, lse, n_cache, w.window, accumulate,
                                      spot_pairs(layer), seed=layer)
                spot_checks += 1
            n_kept = R.evict_topk(k, v, sc, st["k"][nxt], st["v"][nxt], st["sc"][nxt], n_keys, w.budget,
                                  w.n_sink, w.n_recent, pos_src=pos, pos_dst=st["pos"][nxt], kept_idx=kept_idx)
            if zeros_kv is None or zeros_kv.shape[2] != n_keys:
                zeros_kv = torch.zeros(w.B, w.Hkv, n_keys, 8, dtype=w.dtype)
            ref = oracle.evict_topk(zeros_kv, zeros_kv, sc[:, :, :n_keys].cpu(), n_keys, w.budget, w.n_sink,
                                    w.n_recent, cap_dst=w.budget)
            assert n_kept == ref["n_kept"]
            assert torch.equal(kept_idx.cpu()[:, :, :n_kept], ref["kept_idx"][:, :, :n_kept]), \
                f"eviction differs from the oracle's at chunk {step}, layer {layer}"
            st["cur"] = nxt
            kept = st["pos"][nxt][:, :, :n_kept].cpu()
            assert (kept[:, :, 1:] > kept[:, :, :-1]).all()               # order preserved
            # the compaction moved exactly the rows the kept list names
            assert torch.equal(kept, torch.gather(pos[:, :, :n_keys].cpu(), 2, ref["kept_idx"][:, :, :n_kept].long()))
            if needles_must_survive:
                for b in range(w.B):
                    for h in range(w.Hkv):
                        assert seen[b] <= set(kept[b, h].tolist()), \
                            f"needle lost: sequence {b}, layer {layer}, head {h}, chunk {step}"
        n_cache = n_kept
    assert spot_checks == w.layers
    torch.cuda.synchronize()
    assert R.device_error() == 0


@pytest.mark.parametrize("accumulate", [True, False])
def test_config3_32_layers_1m_tokens_at_stated_size(accumulate):
    """Config 3 as stated: 32 layers x 32 chunks of 32,768 tokens (1,048,576-token context), per-layer
    seeded Q/K/V, one oracle spot check per layer on 2 KV-head groups, every one of the 1,024
    evictions against the oracle's full sort.  With per-chunk scores every needle survives in every
    layer and head; with accumulated scores rows that have collected mass for many chunks out-score
    a needle that was scored once (the oracle evicts it as well), so that run asserts the equality
    with the oracle only."""
    w = synth.WORKLOADS["llama8b_1m_32l"]
    assert w.layers == 32 and w.steps == 32
    _recurrence_at_stated_size(
        w, accumulate, needles_must_survive=not accumulate,
        spot_step=lambda layer: (7 * layer + 3) % w.steps,                # a different chunk per layer; layer 27 checks chunk 0
        spot_pairs=lambda layer: [(0, layer % w.Hkv), (0, (layer + 3) % w.Hkv)])


@pytest.mark.parametrize("accumulate", [True, False])
def test_config5_four_sequences_16_chunks_at_stated_size(accumulate):
    """Config 5 as stated: 4 independent sequences of 262,144 tokens batched in every call, 16 chunks
    of 16,384 over a 4,096-row cache, needle positions that differ per sequence.  Every eviction of
    every sequence against the oracle, needle survival per sequence, and an oracle spot check of
    one chunk step on two (sequence, KV head) pairs."""
    w = synth.WORKLOADS["mistral7b_4x256k"]
    assert w.B == 4 and w.steps == 16
    _recurrence_at_stated_size(
        w, accumulate, needles_must_survive=not accumulate,
        spot_step=lambda layer: 9, spot_pairs=lambda layer: [(1, 2), (3, 6)])


def test_chunk_step_full_window_scores_at_full_size():
    """W = Lc at full size: all 32,768 queries of a config-2 chunk score the 40,960 keys (the
    stress reading of the score window); one KV-head group against the oracle in full."""
    w = synth.WORKLOADS["llama8b_128k"]
    G = w.Hq // w.Hkv
    g = 3
    q, kc, vc = synth.chunk_qkv(w, 0, 1, device=DEV)
    k0, v0, s0 = synth.cache_state(w, 0, device=DEV)
    k = torch.cat([k0, kc], 2).contiguous()
    v = torch.cat([v0, vc], 2).contiguous()
    carry = torch.cat([s0, torch.zeros(w.B, w.Hkv, w.Lc, device=DEV)], 2).contiguous()
    score = carry.clone()
    out = torch.empty_like(q)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    R.chunk_step(q, k, v, out, score, w.budget, w.Lc, flags=R.SCORE_ACCUMULATE, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    n = w.cap
    new = score[:, :, :n].double().sum(-1) - carry[:, :, :w.budget].double().sum(-1)
    assert torch.allclose(new, torch.full_like(new, float(w.Lc * G)), rtol=1e-3)
    s_ref = oracle.key_scores(q[:, g * G:(g + 1) * G].cpu().contiguous(), k[:, g:g + 1].cpu().contiguous(),
                              w.budget, w.Lc, score_in=carry[:, g:g + 1].cpu(), accumulate=True)
    assert_scores_close(score[:, g:g + 1, :n], s_ref[:, :, :n], w.Lc * G / n)


@pytest.mark.parametrize("name,accumulate,needles_must_survive", [
    ("llama8b_128k", True, True)])
def test_recurrent_pipeline_full_size_keeps_needles(name, accumulate, needles_must_survive):
    """Config 2 end to end on the GPU: 4 chunk steps with their evictions.  Positions are carried
    through the compaction, mass is conserved, every eviction equals the oracle's full sort of the
    scores the GPU held before it (teacher forcing), and every needle seen so far is still in every
    KV head's cache after every step."""
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
