"""Host-side checks of the C-ABI library that need no GPU: it loads, exports
every symbol the header declares, the ctypes structs match the C layout, and
argument validation rejects bad calls before anything is launched."""
import ctypes
import os
import re

import pytest

import paper_2506_01215_b200 as R
from paper_2506_01215_b200 import build as rbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x10000  # a 16-byte aligned non-null address; never dereferenced (calls fail before launch)


@pytest.fixture(scope="module", autouse=True)
def _built():
    rbuild.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "reform.h")).read()
    declared = set(re.findall(r"\b(reform_[a-z_0-9]+)\s*\(", hdr))
    assert declared, "no declarations parsed"
    L = R.lib()
    for name in declared:
        assert hasattr(L, name), f"{name} declared in reform.h but not exported"
    assert declared == set(R.EXPORTS)


def test_version_and_status_strings():
    L = R.lib()
    assert L.reform_version() >= 100
    assert L.reform_status_string(0) == b"ok"
    for code in (-1, -2, -3, -4):
        assert L.reform_status_string(code) not in (b"ok", b"unknown status")
    assert L.reform_status_string(-99) == b"unknown status"


def _gather(**kw):
    base = dict(struct_size=ctypes.sizeof(R.GatherParams), B=1, k=4, n_rows=10, row_bytes=64,
                src=FAKE, idx=FAKE, dst=FAKE, dev_status=None)
    base.update(kw)
    return R.GatherParams(**base)


def _chunk(**kw):
    base = dict(struct_size=ctypes.sizeof(R.ChunkParams), dtype=R.BF16, B=1, Hq=4, Hkv=2, d=128,
                Lc=64, n_cache=0, cap=64, score_window=16, softmax_scale=0.0, flags=0, q=FAKE,
                k=FAKE, v=FAKE, out=FAKE, lse=FAKE, score=FAKE, workspace=None, workspace_bytes=0,
                dev_status=None)
    base.update(kw)
    return R.ChunkParams(**base)


def _evict(**kw):
    base = dict(struct_size=ctypes.sizeof(R.EvictParams), dtype=R.BF16, B=1, Hkv=2, d=128,
                n_keys=100, cap_src=128, cap_dst=64, budget=32, n_sink=4, n_recent=4, k_src=FAKE,
                v_src=FAKE, score_src=FAKE, pos_src=None, k_dst=FAKE + 4096, v_dst=FAKE + 8192,
                score_dst=FAKE + 12288, pos_dst=None, kept_idx=None, n_kept_host=None,
                workspace=None, workspace_bytes=0, dev_status=None)
    base.update(kw)
    return R.EvictParams(**base)


def _retrieve(**kw):
    base = dict(struct_size=ctypes.sizeof(R.RetrieveParams), dtype=R.BF16, B=1, N=1000, N_cap=1000,
                E=128, nq=2, scale=1.0, pool_window=5, n_keep_head=2, n_keep_tail=2, k=16,
                bank=FAKE, queries=FAKE, idx_out=FAKE, token_score_out=None, pooled_score_out=None,
                workspace=None, workspace_bytes=0, dev_status=None)
    base.update(kw)
    return R.RetrieveParams(**base)


def _embed(sel=((2, 0, 0),), **kw):
    arr = (R.HeadSel * len(sel))(*[R.HeadSel(*s) for s in sel])
    base = dict(struct_size=ctypes.sizeof(R.EmbedParams), dtype=R.BF16, B=1, Lc=8, d=128, Hq=4,
                Hkv=2, n_sel=len(sel), E=256, N_cap=64, token_offset=0, eps=0.0, sel=arr,
                q_state=FAKE, k_state=FAKE, v_state=FAKE, bank=FAKE, dev_status=None)
    base.update(kw)
    return R.EmbedParams(**base), arr


def test_struct_layouts_match_the_header():
    """A call whose only fault comes after the struct_size check returns that
    fault's code, not INVALID_ARG: the C sizeof equals the ctypes sizeof."""
    L = R.lib()
    assert L.reform_gather(ctypes.byref(_gather(row_bytes=24)), None) == R.ERR_UNSUPPORTED
    assert L.reform_chunk_step(ctypes.byref(_chunk(d=48)), None) == R.ERR_UNSUPPORTED
    assert L.reform_evict_topk(ctypes.byref(_evict(d=4)), None) == R.ERR_UNSUPPORTED
    assert L.reform_retrieve_topk(ctypes.byref(_retrieve(E=12)), None) == R.ERR_UNSUPPORTED
    p, _keep = _embed(d=6)
    assert L.reform_embed_append(ctypes.byref(p), None) == R.ERR_UNSUPPORTED
    assert L.reform_gather(ctypes.byref(_gather(struct_size=8)), None) == R.ERR_INVALID_ARG


@pytest.mark.parametrize("kw", [
    dict(Hq=5), dict(n_cache=8), dict(score_window=0), dict(score_window=65), dict(q=None),
    dict(score=None), dict(q=FAKE + 4), dict(softmax_scale=-1.0), dict(struct_size=0),
    dict(flags=R.ROPE_INTERLEAVED), dict(flags=R.ROPE, rope_theta=-2.0),
])
def test_chunk_step_rejects_bad_arguments(kw):
    assert R.lib().reform_chunk_step(ctypes.byref(_chunk(**kw)), None) == R.ERR_INVALID_ARG


def test_chunk_step_needs_workspace_for_lse():
    L = R.lib()
    p = _chunk(lse=None)
    assert L.reform_chunk_step_workspace_size(ctypes.byref(p)) >= 4 * 4 * 64
    assert L.reform_chunk_step(ctypes.byref(p), None) == R.ERR_WORKSPACE
    assert L.reform_chunk_step_workspace_size(ctypes.byref(_chunk())) == 0
    assert L.reform_chunk_step(ctypes.byref(_chunk(dtype=7)), None) == R.ERR_UNSUPPORTED


def test_chunk_step_size_query_validates_shapes():
    """The size query answers 0 for arguments the call would reject (it must not divide by a zero
    head count), and over-large batches are refused up front instead of failing at launch."""
    L = R.lib()
    for kw in (dict(Hkv=0), dict(Hq=5), dict(d=48), dict(dtype=7), dict(n_cache=8), dict(struct_size=0)):
        assert L.reform_chunk_step_workspace_size(ctypes.byref(_chunk(lse=None, **kw))) == 0
    assert L.reform_chunk_step_workspace_size(ctypes.byref(_chunk(lse=None, Lc=1, cap=1, score_window=1))) > 0
    assert L.reform_chunk_step(ctypes.byref(_chunk(B=20000, Hq=4)), None) == R.ERR_INVALID_ARG
    assert L.reform_evict_topk(ctypes.byref(_evict(B=40000)), None) == R.ERR_INVALID_ARG
    assert L.reform_retrieve_topk(ctypes.byref(_retrieve(B=70000)), None) == R.ERR_INVALID_ARG


@pytest.mark.parametrize("kw", [
    dict(n_sink=20, n_recent=20), dict(n_keys=200), dict(cap_dst=16), dict(k_dst=FAKE),
    dict(pos_src=FAKE), dict(score_src=None), dict(budget=-1),
    # in place means everything in place and one capacity: a mixture is refused
    dict(k_dst=FAKE, v_dst=FAKE, score_dst=FAKE),
    dict(k_dst=FAKE, v_dst=FAKE, score_dst=FAKE, cap_dst=128, pos_src=FAKE, pos_dst=FAKE + 64),
])
def test_evict_rejects_bad_arguments(kw):
    assert R.lib().reform_evict_topk(ctypes.byref(_evict(**kw)), None) == R.ERR_INVALID_ARG


def test_evict_in_place_is_accepted_by_the_validation():
    """All destinations equal to their sources with one capacity passes validation (it then asks for
    its workspace like any other call)."""
    p = _evict(k_dst=FAKE, v_dst=FAKE, score_dst=FAKE, cap_dst=128)
    assert R.lib().reform_evict_topk(ctypes.byref(p), None) == R.ERR_WORKSPACE


def test_evict_reports_n_kept_and_needs_workspace():
    L = R.lib()
    n = ctypes.c_int32(-1)
    p = _evict(n_kept_host=ctypes.addressof(n))
    assert L.reform_evict_topk_workspace_size(ctypes.byref(p)) > 0
    assert L.reform_evict_topk(ctypes.byref(p), None) == R.ERR_WORKSPACE
    assert n.value == 32
    p = _evict(n_keys=10, n_kept_host=ctypes.addressof(n))
    L.reform_evict_topk(ctypes.byref(p), None)
    assert n.value == 10


@pytest.mark.parametrize("kw", [
    dict(pool_window=4), dict(pool_window=0), dict(n_keep_head=10, n_keep_tail=10), dict(N=2000),
    dict(nq=0), dict(bank=None), dict(idx_out=FAKE + 8), dict(pool_mode=2), dict(pool_mode=-1),
])
def test_retrieve_rejects_bad_arguments(kw):
    assert R.lib().reform_retrieve_topk(ctypes.byref(_retrieve(**kw)), None) == R.ERR_INVALID_ARG


def test_retrieve_needs_workspace():
    L = R.lib()
    p = _retrieve()
    assert L.reform_retrieve_topk_workspace_size(ctypes.byref(p)) >= 2 * 4 * 1000
    assert L.reform_retrieve_topk(ctypes.byref(p), None) == R.ERR_WORKSPACE


@pytest.mark.parametrize("kw,sel", [
    (dict(), ((3, 0, 0),)), (dict(), ((2, 2, 0),)), (dict(), ((0, 4, 0),)), (dict(), ((2, 0, 2),)),
    (dict(v_state=None), ((2, 0, 0),)), (dict(token_offset=60), ((2, 0, 0),)),
    (dict(n_sel=17), ((2, 0, 0),)), (dict(bank=None), ((2, 0, 0),)),
])
def test_embed_rejects_bad_arguments(kw, sel):
    p, _keep = _embed(sel=sel, **kw)
    assert R.lib().reform_embed_append(ctypes.byref(p), None) == R.ERR_INVALID_ARG


@pytest.mark.parametrize("kw", [dict(src=None), dict(k=-1), dict(row_bytes=0), dict(dst=FAKE + 8)])
def test_gather_rejects_bad_arguments(kw):
    assert R.lib().reform_gather(ctypes.byref(_gather(**kw)), None) == R.ERR_INVALID_ARG


def test_binding_refuses_host_tensors():
    import torch
    t = torch.zeros(1, 4, 8)
    with pytest.raises(ValueError):
        R.gather(t, torch.zeros(1, 2, dtype=torch.int32), torch.zeros(1, 2, 8))


def _rope(**kw):
    base = dict(struct_size=ctypes.sizeof(R.RopeParams), dtype=R.BF16, B=1, H=2, d=128, interleaved=0, cap=64,
                row_begin=0, rows=64, pos_begin=0, theta_base=0.0, src=FAKE, dst=FAKE, dev_status=None)
    base.update(kw)
    return R.RopeParams(**base)


@pytest.mark.parametrize("kw,code", [
    (dict(rows=65), R.ERR_INVALID_ARG), (dict(row_begin=-1), R.ERR_INVALID_ARG), (dict(pos_begin=-5), R.ERR_INVALID_ARG),
    (dict(src=None), R.ERR_INVALID_ARG), (dict(theta_base=-1.0), R.ERR_INVALID_ARG), (dict(struct_size=4), R.ERR_INVALID_ARG),
    (dict(d=24), R.ERR_UNSUPPORTED), (dict(dtype=9), R.ERR_UNSUPPORTED),
])
def test_rope_rejects_bad_arguments(kw, code):
    assert R.lib().reform_rope(ctypes.byref(_rope(**kw)), None) == code


def test_empty_inputs_are_accepted_and_launch_nothing():
    """Degenerate sizes return REFORM_OK before any CUDA call (so this runs without a GPU)."""
    L = R.lib()
    n0 = R.kernel_launch_count()
    assert L.reform_chunk_step(ctypes.byref(_chunk(B=0)), None) == R.OK
    assert L.reform_chunk_step(ctypes.byref(_chunk(Lc=0, n_cache=0, score_window=0)), None) == R.OK
    assert L.reform_evict_topk(ctypes.byref(_evict(B=0)), None) == R.OK
    n = ctypes.c_int32(-1)
    assert L.reform_evict_topk(ctypes.byref(_evict(n_keys=0, n_kept_host=ctypes.addressof(n))), None) == R.OK
    assert n.value == 0
    assert L.reform_evict_topk(ctypes.byref(_evict(budget=0, n_sink=0, n_recent=0)), None) == R.OK
    p, _keep = _embed(Lc=0)
    assert L.reform_embed_append(ctypes.byref(p), None) == R.OK
    p, _keep = _embed(sel=(), n_sel=0)
    assert L.reform_embed_append(ctypes.byref(p), None) == R.OK
    assert L.reform_retrieve_topk(ctypes.byref(_retrieve(N=0)), None) == R.OK
    assert L.reform_retrieve_topk(ctypes.byref(_retrieve(k=0, n_keep_head=0, n_keep_tail=0)), None) == R.OK
    assert L.reform_retrieve_topk(ctypes.byref(_retrieve(B=0)), None) == R.OK
    assert L.reform_gather(ctypes.byref(_gather(k=0)), None) == R.OK
    assert L.reform_gather(ctypes.byref(_gather(B=0)), None) == R.OK
    assert L.reform_rope(ctypes.byref(_rope(rows=0)), None) == R.OK
    assert R.kernel_launch_count() == n0


def test_header_is_plain_c_and_struct_sizes_match_the_binding(tmp_path):
    """include/reform.h compiles as C99 on its own, and every params struct has the size the ctypes
    binding gives it (field order, widths and padding agree)."""
    import os
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    names = [("reform_chunk_params", R.ChunkParams), ("reform_evict_params", R.EvictParams),
             ("reform_embed_params", R.EmbedParams), ("reform_retrieve_params", R.RetrieveParams),
             ("reform_gather_params", R.GatherParams), ("reform_rope_params", R.RopeParams),
             ("reform_head_sel", R.HeadSel)]
    src = tmp_path / "sizes.c"
    src.write_text('#include <stdio.h>\n#include "reform.h"\nint main(void) {\n' +
                   "".join(f'  printf("%zu\\n", sizeof({n}));\n' for n, _ in names) + "  return 0;\n}\n")
    exe = tmp_path / "sizes"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror",
                           "-I", os.path.join(root, "include"), str(src), "-o", str(exe)])
    sizes = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    assert sizes == [ctypes.sizeof(t) for _, t in names]
