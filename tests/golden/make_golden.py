"""Writes tests/golden/tiny_case.json: expected values of a very small seeded case, computed by
the CPU oracle alone (this script imports only oracle/ and the seeded input generator).  The paper
prints no worked numerical example, so these are regression values of the oracle, each tied to the
passage whose definition it follows; the tests compare both the oracle and the CUDA path to them.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2506_01215_b200 import synth  # noqa: E402

CASE = dict(B=1, Hq=4, Hkv=2, d=64, Lc=32, n_cache=16, window=8, budget=20, n_sink=2, n_recent=4,
            N=96, E=128, nq=2, k=12, pool_window=5, keep=2, seed=0x5EF0)


def inputs(c=CASE):
    q = synth.randn((c["B"], c["Hq"], c["Lc"], c["d"]), c["seed"], 901)
    k = synth.randn((c["B"], c["Hkv"], c["n_cache"] + c["Lc"], c["d"]), c["seed"], 902)
    v = synth.randn((c["B"], c["Hkv"], c["n_cache"] + c["Lc"], c["d"]), c["seed"], 903)
    carry = synth.randn((c["B"], c["Hkv"], c["n_cache"] + c["Lc"]), c["seed"], 904).abs()
    bank = torch.nn.functional.normalize(synth.randn((c["B"], c["N"], c["E"]), c["seed"], 905), dim=-1)
    queries = torch.nn.functional.normalize(synth.randn((c["B"], c["nq"], c["E"]), c["seed"], 906), dim=-1)
    return q, k, v, carry, bank, queries


def compute(c=CASE):
    q, k, v, carry, bank, queries = inputs(c)
    out, lse = oracle.attention(q, k, v, c["n_cache"])
    score = oracle.key_scores(q, k, c["n_cache"], c["window"], score_in=carry, accumulate=True)
    ev = oracle.evict_topk(k, v, score, c["n_cache"] + c["Lc"], c["budget"], c["n_sink"], c["n_recent"],
                           cap_dst=c["budget"])
    r = oracle.retrieve_topk(bank, queries, c["N"], c["k"], scale=1.0, pool_window=c["pool_window"],
                             n_keep_head=c["keep"], n_keep_tail=c["keep"])
    return {
        "case": c,
        "citations": {
            "out_row0_head0, lse_head0": "Sec. 3.1 / Fig. 1 step (1): chunk attention over [cache ; chunk]",
            "score": "Sec. 3.1 + Sec. 4 common setup: attention mass from the last `window` queries, summed over the GQA group, carried scores added",
            "kept_idx": "Sec. 3.1 / Fig. 1 step (3): heavy hitters plus initial and recent rows, ascending",
            "retrieve_idx, pooled": "Sec. 3.3: cosine, max over queries, max-pool over adjacent tokens, top-k with first/last kept",
        },
        "out_row0_head0": out[0, 0, 0].tolist(),
        "lse_head0": lse[0, 0].tolist(),
        "score": score.tolist(),
        "kept_idx": ev["kept_idx"].tolist(),
        "retrieve_idx": r["idx"].tolist(),
        "pooled": r["pooled"].tolist(),
    }


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_case.json")
    with open(path, "w") as f:
        json.dump(compute(), f, indent=1)
    print("wrote", path)
