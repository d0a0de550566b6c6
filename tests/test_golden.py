"""The stored expected values of tests/golden/tiny_case.json (written by the oracle alone, see
make_golden.py) against the oracle as it stands (CPU) and against the CUDA path (GPU)."""
import importlib.util
import json
import os

import pytest
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
mg = importlib.util.module_from_spec(spec)
spec.loader.exec_module(mg)

with open(os.path.join(HERE, "golden", "tiny_case.json")) as f:
    GOLD = json.load(f)


def test_oracle_reproduces_stored_values():
    now = mg.compute(GOLD["case"])
    assert now["kept_idx"] == GOLD["kept_idx"]
    assert now["retrieve_idx"] == GOLD["retrieve_idx"]
    for key in ("out_row0_head0", "lse_head0", "score", "pooled"):
        a, b = torch.tensor(now[key], dtype=torch.float64), torch.tensor(GOLD[key], dtype=torch.float64)
        assert torch.allclose(a, b, rtol=1e-12, atol=1e-14), key


@pytest.mark.gpu
def test_cuda_path_matches_stored_values():
    import paper_2506_01215_b200 as R
    c = GOLD["case"]
    q, k, v, carry, bank, queries = mg.inputs(c)
    dev = "cuda"
    n = c["n_cache"] + c["Lc"]
    out = torch.empty_like(q, device=dev)
    lse = torch.empty(q.shape[:3], device=dev)
    score = carry.to(dev).clone()
    R.chunk_step(q.to(dev), k.to(dev), v.to(dev), out, score, c["n_cache"], c["window"], lse=lse,
                 flags=R.SCORE_ACCUMULATE)
    assert (out[0, 0, 0].cpu().double() - torch.tensor(GOLD["out_row0_head0"])).abs().max() < 1e-4
    assert (lse[0, 0].cpu().double() - torch.tensor(GOLD["lse_head0"])).abs().max() < 1e-4
    gs = torch.tensor(GOLD["score"], dtype=torch.float64)
    assert ((score.cpu().double() - gs).abs() <= 1e-3 * gs.abs() + 1e-7).all()
    kd = torch.zeros(c["B"], c["Hkv"], c["budget"], c["d"], device=dev)
    vd, sd = torch.zeros_like(kd), torch.zeros(c["B"], c["Hkv"], c["budget"], device=dev)
    kept = torch.zeros(c["B"], c["Hkv"], c["budget"], dtype=torch.int32, device=dev)
    R.evict_topk(k.to(dev), v.to(dev), score, kd, vd, sd, n, c["budget"], c["n_sink"], c["n_recent"],
                 kept_idx=kept)
    assert kept.cpu().tolist() == GOLD["kept_idx"]
    idx = torch.zeros(c["B"], c["k"], dtype=torch.int32, device=dev)
    pooled = torch.zeros(c["B"], c["N"], device=dev)
    R.retrieve_topk(bank.to(dev), queries.to(dev), c["N"], c["k"], idx, scale=1.0,
                    pool_window=c["pool_window"], n_keep_head=c["keep"], n_keep_tail=c["keep"],
                    pooled_score_out=pooled)
    assert idx.cpu().tolist() == GOLD["retrieve_idx"]
    gp = torch.tensor(GOLD["pooled"], dtype=torch.float64)
    assert ((pooled.cpu().double() - gp).abs() <= 1e-3 * gp.abs() + 1e-6).all()
