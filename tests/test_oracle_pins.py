"""Pins for the CPU oracle: each check compares it with something that is not
the oracle itself -- a library routine on a special case, a closed form, an
invariant, or brute force on a tiny input -- chosen so that a dropped term, a
wrong sign or index, or a transposed operand fails at least one of them."""
import math

import pytest
import torch

import oracle

torch.manual_seed(0)


def _rand_case(B=2, Hq=4, Hkv=2, d=16, Lc=24, n_cache=10, extra=3, dtype=torch.float32, seed=0):
    g = torch.Generator().manual_seed(seed)
    cap = n_cache + Lc + extra
    q = torch.randn(B, Hq, Lc, d, generator=g).to(dtype)
    k = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    v = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    return q, k, v, n_cache


def _mask(Lc, n_cache):
    n = n_cache + Lc
    i = torch.arange(Lc)[:, None]
    j = torch.arange(n)[None, :]
    return j <= n_cache + i


# ---------------------------------------------------------------- attention

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n_cache", [0, 10])
def test_attention_matches_library_sdpa(dtype, n_cache):
    """Sec. 3.1 chunk forward == library scaled-dot-product attention with an
    explicit prefix-causal mask and the GQA head mapping h -> h // G."""
    q, k, v, _ = _rand_case(n_cache=n_cache, dtype=dtype)
    B, Hq, Lc, d = q.shape
    Hkv = k.shape[1]
    n = n_cache + Lc
    G = Hq // Hkv
    out, lse = oracle.attention(q, k, v, n_cache)
    q64 = q.double()
    k64 = k[:, :, :n].double().repeat_interleave(G, dim=1)
    v64 = v[:, :, :n].double().repeat_interleave(G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q64, k64, v64, attn_mask=_mask(Lc, n_cache))
    assert torch.allclose(out, ref, atol=1e-12, rtol=1e-12)
    s = (q64 @ k64.transpose(-1, -2)) / math.sqrt(d)
    s = s.masked_fill(~_mask(Lc, n_cache), float("-inf"))
    assert torch.allclose(lse, torch.logsumexp(s, -1), atol=1e-12)


def test_attention_custom_scale_and_row_subset():
    q, k, v, n_cache = _rand_case()
    full, lse_full = oracle.attention(q, k, v, n_cache, scale=0.37)
    rows = [0, 5, 23]
    sub, lse_sub = oracle.attention(q, k, v, n_cache, scale=0.37, rows=rows)
    assert torch.equal(sub, full[:, :, rows])
    assert torch.equal(lse_sub, lse_full[:, :, rows])
    other, _ = oracle.attention(q, k, v, n_cache)
    assert not torch.allclose(other, full)


def test_attention_identical_values_return_that_row():
    q, k, v, n_cache = _rand_case()
    v[:] = v[:, :, :1]
    out, _ = oracle.attention(q, k, v, n_cache)
    G = q.shape[1] // k.shape[1]
    expect = v[:, :, 0].double().repeat_interleave(G, dim=1)[:, :, None, :].expand_as(out)
    assert torch.allclose(out, expect, atol=1e-13)


def test_attention_identical_keys_give_prefix_mean():
    q, k, v, n_cache = _rand_case()
    k[:] = k[:, :, :1]
    out, lse = oracle.attention(q, k, v, n_cache)
    B, Hq, Lc, d = q.shape
    G = Hq // k.shape[1]
    csum = v.double().cumsum(dim=2)
    for i in range(Lc):
        nvis = n_cache + i + 1
        mean = (csum[:, :, nvis - 1] / nvis).repeat_interleave(G, dim=1)
        assert torch.allclose(out[:, :, i], mean, atol=1e-12)
    # lse = common logit + log(nvis)
    s0 = (q.double() * k[:, :, 0].double().repeat_interleave(G, dim=1)[:, :, None]).sum(-1) / math.sqrt(d)
    nvis = (n_cache + 1 + torch.arange(Lc)).double()
    assert torch.allclose(lse, s0 + nvis.log(), atol=1e-12)


def test_attention_dominant_key_returns_its_value():
    q, k, v, n_cache = _rand_case(d=8)
    j = 4  # a cache row, visible to every query
    q[:] = 0
    q[..., 0] = 30.0
    k[..., 0] = 0
    k[:, :, j, 0] = 30.0
    out, _ = oracle.attention(q, k, v, n_cache)
    G = q.shape[1] // k.shape[1]
    expect = v[:, :, j].double().repeat_interleave(G, dim=1)[:, :, None, :].expand_as(out)
    assert torch.allclose(out, expect, atol=1e-9)


# ------------------------------------------------------------------- scores

@pytest.mark.parametrize("W", [1, 7, 24])
@pytest.mark.parametrize("n_cache", [0, 10])
def test_scores_match_library_softmax_column_sums(W, n_cache):
    q, k, v, _ = _rand_case(n_cache=n_cache)
    B, Hq, Lc, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    n = n_cache + Lc
    sc = oracle.key_scores(q, k, n_cache, W)
    k64 = k[:, :, :n].double().repeat_interleave(G, dim=1)
    s = (q.double() @ k64.transpose(-1, -2)) / math.sqrt(d)
    p = torch.softmax(s.masked_fill(~_mask(Lc, n_cache), float("-inf")), -1)
    ref = p[:, :, Lc - W:].sum(2).reshape(B, Hkv, G, n).sum(2)
    assert torch.allclose(sc[:, :, :n], ref, atol=1e-12)
    assert torch.all(sc[:, :, n:] == 0)


@pytest.mark.parametrize("W", [1, 5, 24])
def test_scores_conserve_mass(W):
    """Every scored query hands out exactly one unit of attention."""
    q, k, v, n_cache = _rand_case(Hq=6, Hkv=2)
    sc = oracle.key_scores(q, k, n_cache, W)
    G = 3
    assert torch.allclose(sc.sum(-1), torch.full((2, 2), float(W * G), dtype=torch.float64), atol=1e-11)


@pytest.mark.parametrize("W", [3, 24])
def test_scores_identical_keys_closed_form(W):
    """With all keys equal every visible key of a query gets 1/nvis, so
    score[j] = G * (H(n) - H(max(n - W, j))) with H the harmonic numbers."""
    q, k, v, n_cache = _rand_case()
    k[:] = k[:, :, :1]
    Lc = q.shape[2]
    n = n_cache + Lc
    G = 2
    sc = oracle.key_scores(q, k, n_cache, W)
    H = [0.0]
    for t in range(1, n + 1):
        H.append(H[-1] + 1.0 / t)
    expect = torch.tensor([G * (H[n] - H[max(n - W, j)]) for j in range(n)], dtype=torch.float64)
    assert torch.allclose(sc[:, :, :n], expect.expand(2, 2, n), atol=1e-12)


def test_scores_identical_keys_without_mask_is_queries_over_keys():
    """Mask off: every scored query sees all n keys, score = W*G/n."""
    q, k, v, n_cache = _rand_case()
    k[:] = k[:, :, :1]
    n = n_cache + q.shape[2]
    sc = oracle.key_scores(q, k, n_cache, 8, causal=False)
    assert torch.allclose(sc[:, :, :n], torch.full((2, 2, n), 8 * 2 / n, dtype=torch.float64), atol=1e-13)


def test_scores_dominant_key_takes_all_mass():
    q, k, v, n_cache = _rand_case(d=8)
    q[:] = 0
    q[..., 0] = 30.0
    k[..., 0] = 0
    k[:, :, 2, 0] = 30.0
    sc = oracle.key_scores(q, k, n_cache, 6)
    assert torch.allclose(sc[:, :, 2], torch.full((2, 2), 12.0, dtype=torch.float64), atol=1e-9)


def test_scores_accumulate_adds_carry_only_on_cache_rows():
    q, k, v, n_cache = _rand_case()
    cap = k.shape[2]
    carry = torch.rand(2, 2, cap, dtype=torch.float64) + 1.0
    fresh = oracle.key_scores(q, k, n_cache, 9)
    acc = oracle.key_scores(q, k, n_cache, 9, score_in=carry, accumulate=True)
    n = n_cache + q.shape[2]
    assert torch.allclose(acc[:, :, :n_cache], fresh[:, :, :n_cache] + carry[:, :, :n_cache], atol=1e-14)
    assert torch.equal(acc[:, :, n_cache:n], fresh[:, :, n_cache:n])
    off = oracle.key_scores(q, k, n_cache, 9, score_in=carry, accumulate=False)
    assert torch.equal(off, fresh)


def test_scores_two_half_windows_sum_to_full_window():
    """Mass from window rows [Lc-2h, Lc-h) plus rows [Lc-h, Lc) equals the mass
    from the window of 2h rows (the first half is obtained by truncating the
    chunk, which leaves those rows' visible sets unchanged)."""
    q, k, v, n_cache = _rand_case()
    Lc, h = q.shape[2], 5
    full = oracle.key_scores(q, k, n_cache, 2 * h)
    last = oracle.key_scores(q, k, n_cache, h)
    q_cut = q[:, :, :Lc - h].contiguous()
    first = oracle.key_scores(q_cut, k, n_cache, h)
    n = n_cache + Lc
    assert torch.allclose(full[:, :, :n], (last + first)[:, :, :n], atol=1e-12)


# ---------------------------------------------------------------- eviction

def _py_topk(scores, lo, hi, m):
    cand = sorted(range(lo, hi), key=lambda j: (-scores[j], j))
    return cand[:m]


@pytest.mark.parametrize("n_sink,n_recent", [(0, 0), (3, 5), (8, 8)])
def test_evict_matches_bruteforce_and_library_sort(n_sink, n_recent):
    g = torch.Generator().manual_seed(3)
    B, Hkv, n, d, budget = 2, 3, 50, 4, 16
    k = torch.randn(B, Hkv, n + 4, d, generator=g)
    v = torch.randn(B, Hkv, n + 4, d, generator=g)
    sc = torch.randint(0, 6, (B, Hkv, n + 4), generator=g).float()  # many ties
    sc[0, 0, 7] = -0.0
    pos = torch.arange(n + 4, dtype=torch.int32).expand(B, Hkv, n + 4).contiguous() * 3
    r = oracle.evict_topk(k, v, sc, n, budget, n_sink, n_recent, cap_dst=budget + 2, pos_src=pos)
    assert r["n_kept"] == budget
    m = budget - n_sink - n_recent
    for b in range(B):
        for h in range(Hkv):
            kept = r["kept_idx"][b, h].tolist()
            s = sc[b, h].tolist()
            brute = sorted(list(range(n_sink)) + _py_topk(s, n_sink, n - n_recent, m)
                           + list(range(n - n_recent, n)))
            assert kept == brute
            # library: stable descending sort keeps lower indices first among ties
            mid = sc[b, h, n_sink:n - n_recent].double()
            order = torch.sort(mid, descending=True, stable=True).indices[:m] + n_sink
            lib = sorted(list(range(n_sink)) + order.tolist() + list(range(n - n_recent, n)))
            assert kept == lib
            kept_t = torch.tensor(kept)
            assert torch.equal(r["k"][b, h, :budget], k[b, h, kept_t])
            assert torch.equal(r["v"][b, h, :budget], v[b, h, kept_t])
            assert torch.equal(r["score"][b, h, :budget], sc[b, h, kept_t].double())
            assert torch.equal(r["pos"][b, h, :budget], pos[b, h, kept_t])
            assert all(a < c for a, c in zip(kept, kept[1:]))


def test_evict_keeps_everything_when_under_budget():
    k = torch.randn(1, 2, 12, 4)
    sc = torch.rand(1, 2, 12)
    r = oracle.evict_topk(k, k.clone(), sc, 9, 16, 2, 2, cap_dst=16)
    assert r["n_kept"] == 9
    assert r["kept_idx"][0, 0, :9].tolist() == list(range(9))
    assert torch.equal(r["k"][:, :, :9], k[:, :, :9])


def test_evict_without_heavy_hitters_is_sink_plus_recent():
    """Budget = sink + recent reproduces the StreamingLLM compressor (Sec. 5.1)."""
    k = torch.randn(1, 1, 40, 4)
    sc = torch.rand(1, 1, 40)
    r = oracle.evict_topk(k, k.clone(), sc, 40, 10, 4, 6, cap_dst=10)
    assert r["kept_idx"][0, 0].tolist() == [0, 1, 2, 3, 34, 35, 36, 37, 38, 39]


def test_evict_scale_invariance_and_threshold_property():
    g = torch.Generator().manual_seed(5)
    k = torch.randn(1, 2, 200, 4, generator=g)
    sc = torch.rand(1, 2, 200, generator=g)
    a = oracle.evict_topk(k, k.clone(), sc, 200, 64, 8, 8, cap_dst=64)
    b = oracle.evict_topk(k, k.clone(), sc * 7.5, 200, 64, 8, 8, cap_dst=64)
    assert torch.equal(a["kept_idx"], b["kept_idx"])
    for h in range(2):
        kept = set(a["kept_idx"][0, h].tolist())
        mid = [j for j in range(8, 192)]
        kept_mid = [sc[0, h, j].item() for j in mid if j in kept]
        drop_mid = [sc[0, h, j].item() for j in mid if j not in kept]
        assert min(kept_mid) >= max(drop_mid)
        assert set(range(8)) <= kept and set(range(192, 200)) <= kept


def test_evict_rejects_bad_budget():
    k = torch.randn(1, 1, 40, 4)
    with pytest.raises(ValueError):
        oracle.evict_topk(k, k.clone(), torch.rand(1, 1, 40), 40, 8, 5, 5, cap_dst=8)


# --------------------------------------------------------------- embeddings

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_embed_rows_are_unit_norm_per_slot_and_placed_by_slot(dtype):
    g = torch.Generator().manual_seed(7)
    B, Hq, Hkv, Lc, d = 2, 4, 2, 6, 16
    qs = torch.randn(B, Hq, Lc, d, generator=g).to(dtype)
    ks = torch.randn(B, Hkv, Lc, d, generator=g).to(dtype)
    vs = (torch.randn(B, Hkv, Lc, d, generator=g) * 9).to(dtype)
    sel = [(0, 3, 0), (2, 1, 2), (1, 0, 1)]
    bank = torch.zeros(B, 10, 3 * d, dtype=dtype)
    f64 = oracle.embed_append(bank, 2, sel, qs, ks, vs, want_f64=True)
    srcs = {0: qs, 1: ks, 2: vs}
    for kind, head, slot in sel:
        x = srcs[kind][:, head].double()
        ref = x / x.norm(dim=-1, keepdim=True)
        got = f64[:, 2:2 + Lc, slot * d:(slot + 1) * d]
        assert torch.allclose(got, ref, atol=1e-15)
        stored = bank[:, 2:2 + Lc, slot * d:(slot + 1) * d]
        assert torch.equal(stored, ref.to(dtype))            # one rounding, nearest-even
        tol = 2 ** -8 if dtype == torch.bfloat16 else 1e-6
        assert torch.all((stored.double().norm(dim=-1) - 1).abs() < tol)
    assert torch.all(bank[:, :2] == 0) and torch.all(bank[:, 2 + Lc:] == 0)


def test_embed_zero_vector_stays_zero():
    vs = torch.zeros(1, 1, 2, 8)
    bank = torch.ones(1, 2, 8)
    oracle.embed_append(bank, 0, [(2, 0, 0)], v_state=vs)
    assert torch.all(bank == 0)


def test_embed_concat_cosine_is_mean_of_per_head_cosines():
    """Sec. 3.2: cosine on the concatenation of normalised heads equals the
    mean of the per-head cosines."""
    g = torch.Generator().manual_seed(9)
    d, ns = 8, 4
    a = torch.randn(1, ns, 5, d, generator=g)
    sel = [(2, s, s) for s in range(ns)]
    bank = torch.zeros(1, 5, ns * d)
    f64 = oracle.embed_append(bank, 0, sel, v_state=a, want_f64=True)[0]
    x, y = f64[0], f64[3]
    cos_concat = (x @ y) / (x.norm() * y.norm())
    per_head = [torch.nn.functional.cosine_similarity(a[0, s, 0].double(), a[0, s, 3].double(), dim=0)
                for s in range(ns)]
    assert abs(cos_concat - sum(per_head) / ns) < 1e-14
    assert abs((x @ y) / ns - sum(per_head) / ns) < 1e-14


def test_bf16_rounding_is_nearest_even_without_double_rounding():
    # 1 + 2^-8 lies exactly between two bf16 values -> even mantissa (1.0);
    # 1 + 2^-8 + 2^-40 is above the tie -> rounds up; fp32 would have lost it.
    vs = torch.zeros(1, 1, 1, 2, dtype=torch.bfloat16)
    vs[..., 0] = 1.0
    bank = torch.zeros(1, 1, 2, dtype=torch.bfloat16)
    oracle.embed_append(bank, 0, [(2, 0, 0)], v_state=vs)
    assert bank[0, 0, 0].item() == 1.0
    x = torch.tensor([3.0, 4.0], dtype=torch.bfloat16).reshape(1, 1, 1, 2)
    oracle.embed_append(bank, 0, [(2, 0, 0)], v_state=x)
    assert bank[0, 0].tolist() == [torch.tensor(0.6).bfloat16().item(), torch.tensor(0.8).bfloat16().item()]


# ----------------------------------------------------------------- retrieve

@pytest.mark.parametrize("pool", [1, 5, 17])
def test_retrieve_matches_library_matmul_pool_and_sort(pool):
    g = torch.Generator().manual_seed(11)
    B, N, E, nq, k = 2, 300, 24, 3, 40
    bank = torch.randn(B, N + 5, E, generator=g).bfloat16()
    qs = torch.randn(B, nq, E, generator=g).bfloat16()
    r = oracle.retrieve_topk(bank, qs, N, k, scale=0.5, pool_window=pool, n_keep_head=4, n_keep_tail=6)
    sim = 0.5 * (qs.double() @ bank[:, :N].double().transpose(1, 2))
    ts = sim.max(dim=1).values
    assert torch.allclose(r["ts"], ts, atol=1e-13)
    pooled = torch.nn.functional.max_pool1d(ts[:, None], kernel_size=pool, stride=1, padding=pool // 2)[:, 0]
    assert torch.allclose(r["pooled"], pooled, atol=1e-13)
    for b in range(B):
        mid = r["pooled"][b, 4:N - 6]
        order = torch.sort(mid, descending=True, stable=True).indices[:k - 10] + 4
        expect = sorted(list(range(4)) + order.tolist() + list(range(N - 6, N)))
        assert r["idx"][b].tolist() == expect


@pytest.mark.parametrize("pool", [1, 5, 21, 601])
def test_retrieve_mean_pooling_matches_library_avg_pool(pool):
    """The mean-pool smoothing of the head-ranking procedure (Appendix, detailed head selection,
    Step 3): mean over the token and its neighbours, over the tokens that exist at the ends ==
    library avg_pool1d without counting the padding; selection by a stable sort of that."""
    g = torch.Generator().manual_seed(13)
    B, N, E, nq, k = 2, 300, 24, 3, 40
    bank = torch.randn(B, N + 5, E, generator=g).bfloat16()
    qs = torch.randn(B, nq, E, generator=g).bfloat16()
    r = oracle.retrieve_topk(bank, qs, N, k, scale=0.5, pool_window=pool, n_keep_head=4, n_keep_tail=6,
                             pool_mode="mean")
    ts = (0.5 * (qs.double() @ bank[:, :N].double().transpose(1, 2))).max(dim=1).values
    assert torch.allclose(r["ts"], ts, atol=1e-13)
    if pool // 2 < N:
        pooled = torch.nn.functional.avg_pool1d(ts[:, None], kernel_size=pool, stride=1, padding=pool // 2,
                                                count_include_pad=False)[:, 0]
    else:                                       # window wider than the bank: the mean of everything
        pooled = ts.mean(dim=1, keepdim=True).expand(B, N)
    assert torch.allclose(r["pooled"], pooled, atol=1e-12)
    # brute force at a few tokens, both ends included
    rad = pool // 2
    for t in (0, 1, min(rad, N - 1), N // 2, N - 2, N - 1):
        lo, hi = max(0, t - rad), min(N - 1, t + rad)
        assert abs(float(r["pooled"][1, t]) - float(ts[1, lo:hi + 1].sum() / (hi - lo + 1))) < 1e-12
    for b in range(B):
        mid = r["pooled"][b, 4:N - 6]
        order = torch.sort(mid, descending=True, stable=True).indices[:k - 10] + 4
        assert r["idx"][b].tolist() == sorted(list(range(4)) + order.tolist() + list(range(N - 6, N)))
    # a constant stays constant, and the mean never exceeds the max-pooled score
    rmax = oracle.retrieve_topk(bank, qs, N, k, scale=0.5, pool_window=pool, n_keep_head=4, n_keep_tail=6)
    assert (r["pooled"] <= rmax["pooled"] + 1e-15).all()


def test_retrieve_self_similarity_orthogonality_and_bound():
    E = 16
    eye = torch.eye(E)
    r = oracle.retrieve_topk(eye[None], eye[None, :1], E, 1)
    assert r["ts"][0, 0].item() == 1.0 and torch.all(r["ts"][0, 1:] == 0)
    assert r["idx"].tolist() == [[0]]
    g = torch.Generator().manual_seed(2)
    bank = torch.nn.functional.normalize(torch.randn(1, 100, E, generator=g), dim=-1)
    qs = torch.nn.functional.normalize(torch.randn(1, 4, E, generator=g), dim=-1)
    r = oracle.retrieve_topk(bank, qs, 100, 10)
    assert r["ts"].abs().max() <= 1.0 + 1e-6


def test_retrieve_pool_properties_and_ties():
    N = 64
    bank = torch.ones(1, N, 2)
    qs = torch.ones(1, 1, 2)
    r = oracle.retrieve_topk(bank, qs, N, 7, pool_window=9)
    assert torch.all(r["pooled"] == 2.0)
    assert r["idx"].tolist() == [list(range(7))]           # ties: lowest index first
    bank[0, 40] = 3.0
    r = oracle.retrieve_topk(bank, qs, N, 9, pool_window=9)
    assert r["idx"].tolist() == [list(range(36, 45))]      # the peak spreads +-4
    assert torch.all(r["pooled"] >= r["ts"])
    r1 = oracle.retrieve_topk(bank, qs, N, 9, pool_window=1)
    assert torch.equal(r1["pooled"], r1["ts"])


def test_retrieve_k_at_least_n_returns_all_tokens():
    bank = torch.randn(1, 12, 4)
    r = oracle.retrieve_topk(bank, bank[:, :2].contiguous(), 12, 20)
    assert r["n_out"] == 12 and r["idx"].tolist() == [list(range(12))]


def test_retrieve_finds_planted_rows():
    import dataclasses
    from paper_2506_01215_b200 import synth
    w = dataclasses.replace(synth.WORKLOADS["tiny"], N=2048, k=64)
    bank, qs, planted = synth.bank_and_queries(w)
    r = oracle.retrieve_topk(bank, qs, w.N, w.k, scale=w.sim_scale, pool_window=1)
    assert set(planted[0]) <= set(r["idx"][0].tolist())
    ts = r["ts"][0, torch.tensor(planted[0])]
    assert torch.all((ts - w.rho).abs() < 1e-5)


# ------------------------------------------------------------------- gather

def test_gather_copies_rows_bit_exactly():
    src = torch.randn(2, 30, 8).bfloat16()
    idx = torch.tensor([[0, 29, 3, 3], [7, 1, 2, 28]], dtype=torch.int32)
    out = oracle.gather(src, idx)
    for b in range(2):
        assert torch.equal(out[b].view(torch.int16), src[b, idx[b].long()].view(torch.int16))
    with pytest.raises(ValueError):
        oracle.gather(src, torch.tensor([[30], [0]], dtype=torch.int32))


# --------------------------------------------------------------------- rope

def _rope_ref_half(x, pos, base):
    """Independent statement of the rotate-half convention in torch fp64."""
    d = x.shape[-1]
    inv = base ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
    ang = pos[:, None].double() * inv[None, :]
    cos, sin = torch.cat([ang.cos(), ang.cos()], -1), torch.cat([ang.sin(), ang.sin()], -1)
    x = x.double()
    rot = torch.cat([-x[..., d // 2:], x[..., :d // 2]], -1)
    return x * cos + rot * sin


def test_rope_matches_rotate_half_and_complex_forms():
    g = torch.Generator().manual_seed(31)
    x = torch.randn(2, 3, 20, 16, generator=g)
    y = oracle.rope(x, 4, 10, 1000)
    pos = torch.arange(1000, 1010)
    ref = _rope_ref_half(x[:, :, 4:14], pos, 10000.0)
    assert torch.allclose(y[:, :, 4:14].double(), ref, atol=2e-7)          # one fp32 rounding
    assert torch.equal(y[:, :, :4], x[:, :, :4]) and torch.equal(y[:, :, 14:], x[:, :, 14:])
    # interleaved pairs = multiplication by e^{i pos theta} of the complex view
    yi = oracle.rope(x, 4, 10, 1000, base=500.0, interleaved=True)
    inv = 500.0 ** (-torch.arange(0, 16, 2, dtype=torch.float64) / 16)
    z = torch.view_as_complex(x[:, :, 4:14].double().reshape(2, 3, 10, 8, 2).contiguous())
    zr = z * torch.polar(torch.ones(10, 8, dtype=torch.float64), pos[:, None].double() * inv[None, :])
    assert torch.allclose(yi[:, :, 4:14].double(), torch.view_as_real(zr).reshape(2, 3, 10, 16), atol=2e-7)


def test_rope_position_zero_is_identity_and_norms_are_kept():
    g = torch.Generator().manual_seed(32)
    x = torch.randn(1, 2, 8, 32, generator=g)
    y = oracle.rope(x, 0, 8, 0)
    assert torch.equal(y[:, :, 0], x[:, :, 0])
    assert torch.allclose(y.double().norm(dim=-1), x.double().norm(dim=-1), rtol=1e-6)


def test_rope_scores_depend_on_relative_position_only():
    g = torch.Generator().manual_seed(33)
    q = torch.randn(1, 1, 1, 64, generator=g).double().float()
    k = torch.randn(1, 1, 1, 64, generator=g).double().float()
    dots = []
    for m, n in [(5, 2), (1005, 1002), (40963, 40960)]:
        qm, kn = oracle.rope(q, 0, 1, m), oracle.rope(k, 0, 1, n)
        dots.append((qm.double() * kn.double()).sum().item())
    assert abs(dots[0] - dots[1]) < 1e-4 and abs(dots[0] - dots[2]) < 1e-4
    assert abs(dots[0] - (q.double() * k.double()).sum().item()) > 1e-3   # and it is not the unrotated dot


# ------------------------------------------------- recurrence (needle pin)

@pytest.mark.parametrize("accumulate", [True, False])
def test_tiny_free_run_keeps_every_planted_needle(accumulate):
    """The Tiny configuration run by the oracle alone for its 8 chunk steps (Alg. 1 ForwardChunk;
    Sec. 3.1 compression with the first and last 32 rows kept): after every eviction every needle
    seen so far is still in every KV head's cache.  With per-chunk scores a needle scored among
    the candidates ranks within the first 2 x n_needles of them (only other needles and a few lucky
    keys out-score a +4 logit); with accumulated scores the survivors of earlier steps carry
    several chunks of mass, so the claim there is the weaker one that the needle ranks inside the
    kept set.  The planted keys are heavy by construction, so a selection that dropped one would
    be wrong by the definition itself."""
    from oracle_run import oracle_free_run
    from paper_2506_01215_b200 import synth
    w = synth.WORKLOADS["tiny"]
    needles = synth.needle_positions(w)
    assert len(set(needles)) == w.n_needles == 8
    m = w.budget - w.n_sink - w.n_recent
    steps = 0
    for st in oracle_free_run(w, accumulate=accumulate):
        steps += 1
        seen = [p for p in needles if p < (st["step"] + 1) * w.Lc]
        assert st["n_kept"] == w.budget
        for h in range(w.Hkv):
            kept = st["pos"][0, h, :w.budget]
            assert (kept[1:] > kept[:-1]).all()                           # order preserved
            assert set(seen) <= set(kept.tolist()), f"needle lost in head {h}, step {st['step']}"
            before = st["pos_before"][0, h, :st["n"]].tolist()
            sc = st["scores"][0, h, :st["n"]]
            cand = sc[w.n_sink:st["n"] - w.n_recent]
            for p in seen:
                r = before.index(p)
                if w.n_sink <= r < st["n"] - w.n_recent:                  # scored as a candidate
                    rank = int((cand > sc[r]).sum())
                    bound = m if accumulate else 2 * w.n_needles
                    assert rank < bound, f"needle {p} ranks {rank} of {cand.numel()} candidates"
    assert steps == w.steps == 8
