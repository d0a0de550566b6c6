"""Comparison rules shared by the GPU parity tests (tolerances of the build
target: index sets exact up to swaps between candidates whose oracle scores
differ by < 1e-4 relative; scores 1e-3 relative; bf16 outputs 2e-2 max-abs;
fp32 outputs 1e-4 max-abs)."""
import torch

OUT_TOL = {torch.bfloat16: 2e-2, torch.float32: 1e-4}


def assert_outputs_close(gpu_out, oracle_out, dtype):
    err = (gpu_out.detach().cpu().double() - oracle_out).abs().max().item()
    assert err <= OUT_TOL[dtype], f"attention output max-abs error {err:.3e} > {OUT_TOL[dtype]}"
    return err


def assert_scores_close(gpu, oracle, floor):
    """|g - o| <= 1e-3 |o| + 1e-6 * floor, elementwise."""
    g = gpu.detach().cpu().double()
    tol = 1e-3 * oracle.abs() + 1e-6 * floor
    bad = (g - oracle).abs() > tol
    assert not bad.any(), (
        f"{int(bad.sum())} scores outside tolerance; worst rel "
        f"{((g - oracle).abs() / oracle.abs().clamp_min(1e-30)).max().item():.3e}")


def assert_index_sets_match(gpu_idx, oracle_idx, oracle_vals, rel=1e-4):
    """Both are 1-D ascending index lists.  Any index chosen by only one side
    must have an oracle value within rel*|cutoff| of the cutoff (the smallest
    oracle value among the oracle's non-forced choices is not known here, so
    the cutoff is taken as the smallest oracle value over the oracle's set
    members that the GPU dropped or, failing that, over the symmetric
    difference)."""
    g = set(int(x) for x in gpu_idx.tolist())
    o = set(int(x) for x in oracle_idx.tolist())
    assert len(g) == len(gpu_idx), "duplicate indices"
    assert list(gpu_idx.tolist()) == sorted(g), "indices not ascending"
    assert len(g) == len(o), f"size {len(g)} != {len(o)}"
    diff = g ^ o
    if not diff:
        return 0
    vals = torch.tensor([float(oracle_vals[i]) for i in sorted(diff)], dtype=torch.float64)
    cutoff = vals.max().item()
    spread = (vals - cutoff).abs().max().item()
    assert spread <= rel * abs(cutoff), (
        f"{len(diff)} indices differ and their oracle values spread {spread:.3e} "
        f"around {cutoff:.6e} (> {rel} relative)")
    return len(diff)
