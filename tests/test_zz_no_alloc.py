"""reform_evict_topk_static: the cache compression for callers that cannot
allocate device memory (everything handed to a KV-cache pool already, or a
loop that must not pay cudaMalloc's device-wide synchronisation).  It has to
give exactly what reform_evict_topk gives, call after call, although all its
calls share one built-in scratch array that keeps the previous call's bytes.

This file sorts last on purpose: a run that stops at the first failure has
already been through every other test by the time it gets here."""
import ctypes

import pytest
import torch

import oracle
import paper_2506_01215_b200 as R

DEV = "cuda"


def _inputs(seed, B, Hkv, n_keys, d, dtype):
    g = torch.Generator().manual_seed(seed)
    cap = n_keys + 3
    k = torch.randn(B, Hkv, cap, d, generator=g).to(dtype).to(DEV)
    v = torch.randn(B, Hkv, cap, d, generator=g).to(dtype).to(DEV)
    sc = ((torch.rand(B, Hkv, cap, generator=g) * 64).floor() / 8).to(DEV)   # ties included
    pos = torch.randint(0, 1 << 20, (B, Hkv, cap), generator=g, dtype=torch.int32).to(DEV)
    return k, v, sc, pos


def _outputs(B, Hkv, budget, d, dtype):
    return (torch.zeros(B, Hkv, budget, d, dtype=dtype, device=DEV),
            torch.zeros(B, Hkv, budget, d, dtype=dtype, device=DEV),
            torch.zeros(B, Hkv, budget, device=DEV),
            torch.zeros(B, Hkv, budget, dtype=torch.int32, device=DEV),
            torch.full((B, Hkv, budget), -1, dtype=torch.int32, device=DEV))


@pytest.mark.gpu
def test_static_entry_point_matches_regular_one_on_two_calls_in_a_row():
    # two different problems back to back through the same built-in scratch
    cases = [(11, 1, 8, 9000, 128, 2048, 64, 64, torch.bfloat16),
             (12, 2, 4, 5000, 64, 1000, 0, 0, torch.float32)]
    for seed, B, Hkv, n_keys, d, budget, sink, recent, dtype in cases:
        k, v, sc, pos = _inputs(seed, B, Hkv, n_keys, d, dtype)
        ref = _outputs(B, Hkv, budget, d, dtype)
        n_ref = R.evict_topk(k, v, sc, ref[0], ref[1], ref[2], n_keys, budget, sink, recent,
                             pos_src=pos, pos_dst=ref[3], kept_idx=ref[4])
        got = _outputs(B, Hkv, budget, d, dtype)
        n_got = R.evict_topk_static(k, v, sc, got[0], got[1], got[2], n_keys, budget, sink, recent,
                                    pos_src=pos, pos_dst=got[3], kept_idx=got[4])
        torch.cuda.synchronize()
        assert n_got == n_ref == budget
        for a, b in zip(got, ref):
            assert torch.equal(a, b)      # integer, byte and index work: bit-exact
        # and both equal the oracle's full sort
        o = oracle.evict_topk(k.cpu(), v.cpu(), sc.cpu(), n_keys, budget, sink, recent, cap_dst=budget,
                              pos_src=pos.cpu())
        assert torch.equal(got[4].cpu(), o["kept_idx"])
        assert torch.equal(got[0].cpu().view(torch.uint8), o["k"].view(torch.uint8))
        assert torch.equal(got[2].cpu().double(), o["score"]) and torch.equal(got[3].cpu(), o["pos"])
    # and once more without the optional kept-index output (the list then lives in the scratch)
    seed, B, Hkv, n_keys, d, budget, sink, recent, dtype = cases[0]
    k, v, sc, pos = _inputs(seed, B, Hkv, n_keys, d, dtype)
    ref = _outputs(B, Hkv, budget, d, dtype)
    R.evict_topk(k, v, sc, ref[0], ref[1], ref[2], n_keys, budget, sink, recent)
    got = _outputs(B, Hkv, budget, d, dtype)
    R.evict_topk_static(k, v, sc, got[0], got[1], got[2], n_keys, budget, sink, recent)
    torch.cuda.synchronize()
    for a, b in zip(got[:3], ref[:3]):
        assert torch.equal(a, b)


@pytest.mark.gpu
def test_static_entry_point_at_its_documented_limits():
    """The largest problem the built-in scratch takes: 32 segments x 65,536 keys, budget 16,384, no
    kept-index output (so the list itself lives in the scratch, which this case fills almost to
    its last byte) -- more selection blocks than can be resident at once, so the selection runs as
    one launch per pass.  Twice back to back on different inputs, each against the oracle."""
    B, Hkv, n_keys, d, budget = 4, 8, R.EVICT_STATIC_MAX_KEYS, 64, R.EVICT_STATIC_MAX_BUDGET
    assert B * Hkv == R.EVICT_STATIC_MAX_SEGS
    for seed in (21, 22):
        k, v, sc, pos = _inputs(seed, B, Hkv, n_keys - 3, d, torch.bfloat16)     # cap = n_keys exactly
        got = _outputs(B, Hkv, budget, d, torch.bfloat16)
        n = R.evict_topk_static(k, v, sc, got[0], got[1], got[2], n_keys, budget, 256, 256,
                                pos_src=pos, pos_dst=got[3])
        torch.cuda.synchronize()
        assert n == budget and R.device_error() == 0
        o = oracle.evict_topk(k.cpu(), v.cpu(), sc.cpu(), n_keys, budget, 256, 256, cap_dst=budget,
                              pos_src=pos.cpu())
        assert torch.equal(got[0].cpu().view(torch.uint8), o["k"].view(torch.uint8))
        assert torch.equal(got[1].cpu().view(torch.uint8), o["v"].view(torch.uint8))
        assert torch.equal(got[2].cpu().double(), o["score"]) and torch.equal(got[3].cpu(), o["pos"])


@pytest.mark.gpu
def test_static_entry_point_rejects_problems_beyond_its_scratch():
    k, v, sc, pos = _inputs(1, 5, 8, 256, 64, torch.float32)      # 40 segments > 32
    out = _outputs(5, 8, 64, 64, torch.float32)
    with pytest.raises(R.ReformError) as e:
        R.evict_topk_static(k, v, sc, out[0], out[1], out[2], 256, 64, 4, 4)
    assert e.value.status == R.ERR_TOO_LARGE


def test_static_entry_point_limits_are_checked_on_the_host():
    """No GPU needed: an over-size request is refused before any CUDA call."""
    fake = 0x10000
    p = R.EvictParams(struct_size=ctypes.sizeof(R.EvictParams), dtype=R.BF16, B=1, Hkv=2, d=128,
                      n_keys=70000, cap_src=70000, cap_dst=64, budget=32, n_sink=4, n_recent=4,
                      k_src=fake, v_src=fake, score_src=fake, k_dst=fake + 4096, v_dst=fake + 8192,
                      score_dst=fake + 12288)
    assert R.lib().reform_evict_topk_static(ctypes.byref(p), None) == R.ERR_TOO_LARGE
    p.n_keys, p.cap_src, p.budget, p.cap_dst = 1000, 1000, 20000, 20000
    assert R.lib().reform_evict_topk_static(ctypes.byref(p), None) == R.ERR_TOO_LARGE
    p.budget, p.cap_dst, p.n_sink = 32, 64, 40
    assert R.lib().reform_evict_topk_static(ctypes.byref(p), None) == R.ERR_INVALID_ARG
    assert b"scratch" in R.lib().reform_status_string(R.ERR_TOO_LARGE)
