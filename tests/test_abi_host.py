"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, the Python struct mirrors the C struct, and invalid calls are refused before any CUDA work."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "clsa.h")


@pytest.fixture(scope="module")
def clsa():
    sys.path.insert(0, ROOT)
    import __graft_entry__ as entry

    entry._load_build_module().build()
    import paper_2606_06467_b200 as mod

    return mod


def _declared_functions():
    text = open(HEADER).read()
    return sorted(set(re.findall(r"CLSA_API\s+[\w\s\*]+?\b(clsa_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(clsa):
    names = _declared_functions()
    assert len(names) == 16 and set(names) == set(clsa.EXPORTS)
    lib = ctypes.CDLL(clsa.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert clsa.clsa_version() == 200
    assert clsa.clsa_status_string(0) == "ok" and "unsupported" in clsa.clsa_status_string(2)


def test_struct_layout_matches_the_header(clsa, tmp_path):
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "clsa.h"\nint main(void){printf("%zu", sizeof(clsa_params));\n'
                   + "".join(f'printf(" %zu", offsetof(clsa_params, {f}));\n' for f, _ in clsa.clsa_params._fields_)
                   + "return 0;}\n")
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    nums = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    assert nums[0] == ctypes.sizeof(clsa.clsa_params)
    assert nums[1:] == [getattr(clsa.clsa_params, f).offset for f, _ in clsa.clsa_params._fields_]


def _good(clsa, **kw):
    base = dict(num_seqs=2, num_q_heads=32, num_kv_heads=8, head_dim=128, idx_dim=128, top_k=64, num_layers=2,
                max_seq_len=1024, sm_scale=0.088, seq_start=0x1000, seq_len=0x2000, k_cache=0x10000, v_cache=0x20000,
                idx_k_cache=0x30000)
    base.update(kw)
    return clsa.make_params(**base)


def test_bad_arguments_are_refused_on_the_host(clsa):
    raw = clsa.raw()
    n = ctypes.c_size_t(0)
    P = ctypes.byref
    assert raw.clsa_workspace_bytes(None, P(n)) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_workspace_bytes(P(_good(clsa)), None) == clsa.CLSA_ERR_INVALID_ARG
    for kw, want in (
        (dict(num_seqs=0), clsa.CLSA_ERR_INVALID_ARG), (dict(top_k=0), clsa.CLSA_ERR_INVALID_ARG),
        (dict(num_q_heads=30), clsa.CLSA_ERR_INVALID_ARG), (dict(causal=2), clsa.CLSA_ERR_INVALID_ARG),
        (dict(max_seq_len=0), clsa.CLSA_ERR_INVALID_ARG), (dict(sm_scale=-1.0), clsa.CLSA_ERR_INVALID_ARG),
        (dict(sm_scale=float("nan")), clsa.CLSA_ERR_INVALID_ARG), (dict(sm_scale=0.0), clsa.CLSA_ERR_INVALID_ARG), (dict(num_layers=0), clsa.CLSA_ERR_INVALID_ARG),
        (dict(head_dim=64), clsa.CLSA_ERR_UNSUPPORTED), (dict(idx_dim=96), clsa.CLSA_ERR_UNSUPPORTED),
        (dict(num_q_heads=34, num_kv_heads=2), clsa.CLSA_ERR_UNSUPPORTED),
    ):
        assert raw.clsa_workspace_bytes(P(_good(clsa, **kw)), P(n)) == want, kw
    ws, wsb, st = 0x100000, 1 << 20, None
    good = _good(clsa)
    # index scores
    assert raw.clsa_index_scores(P(good), None, 0x40000, 1024, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_index_scores(P(good), 0x50008, 0x40000, 1024, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG  # q misaligned
    assert raw.clsa_index_scores(P(good), 0x50000, 0x40000, 1000, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG  # stride < max len
    assert raw.clsa_index_scores(P(_good(clsa, idx_k_cache=None)), 0x50000, 0x40000, 1024, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_index_scores(P(_good(clsa, idx_token_stride=100)), 0x50000, 0x40000, 1024, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_index_scores(P(_good(clsa, seq_len=None)), 0x50000, 0x40000, 1024, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_index_scores(P(good), 0x50000, 0x40000, 1024, None, wsb, st) == clsa.CLSA_ERR_WORKSPACE
    assert raw.clsa_index_scores(P(good), 0x50000, 0x40000, 1024, ws + 16, wsb, st) == clsa.CLSA_ERR_WORKSPACE
    assert raw.clsa_index_scores(P(good), 0x50000, 0x40000, 1024, ws, 8, st) == clsa.CLSA_ERR_WORKSPACE
    # top-k
    assert raw.clsa_topk(P(good), None, 1024, 0x60000, 0x70000, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_topk(P(good), 0x40000, 512, 0x60000, 0x70000, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_topk(P(good), 0x40000, 1024, 0x60002, 0x70000, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    # sparse attention
    assert raw.clsa_sparse_attn(P(good), None, 0x60000, 0x70000, 0x80000, None, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_sparse_attn(P(_good(clsa, k_cache=0x10004)), 0x50000, 0x60000, 0x70000, 0x80000, None, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_sparse_attn(P(_good(clsa, kv_head_stride=64)), 0x50000, 0x60000, 0x70000, 0x80000, None, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_sparse_attn(P(good), 0x50000, 0x60000, 0x70000, 0x80000, None, None, wsb, st) == clsa.CLSA_ERR_WORKSPACE
    # decode launches need their merge scratch, whose size depends on the device: without one the call stops at the device query
    too_small = (clsa.CLSA_ERR_WORKSPACE, clsa.CLSA_ERR_CUDA)
    assert raw.clsa_sparse_attn(P(good), 0x50000, 0x60000, 0x70000, 0x80000, None, ws, 256, st) in too_small
    for bad in (clsa.make_hints(reverse=2), clsa.make_hints(shared_gpu=-1), clsa.make_hints(shared_gpu=5), clsa.make_hints(keep_rows=7), clsa.make_hints(only_q_pending=2)):
        assert raw.clsa_sparse_attn_hinted(P(good), 0x50000, 0x60000, 0x70000, 0x80000, None, P(bad), ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
        assert raw.clsa_gather_probe(P(good), 0x60000, 0x70000, P(bad), ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_sparse_attn_hinted(P(good), None, 0x60000, 0x70000, 0x80000, None, None, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_gather_probe(P(good), None, 0x70000, None, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_gather_probe(P(good), 0x60000, 0x70000, None, ws, 256, st) in too_small
    assert raw.clsa_gather_probe(P(_good(clsa, q_per_seq=4, max_seq_len=1024)), 0x60000, 0x70000, None, ws, wsb, st) == clsa.CLSA_ERR_UNSUPPORTED
    # decode step
    L = good.num_layers
    qs = (ctypes.c_void_p * L)(0x50000, 0x51000)
    outs = (ctypes.c_void_p * L)(0x80000, None)
    assert raw.clsa_decode_step(P(good), 0x50000, qs, outs, 0x60000, 0x70000, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_decode_step(P(good), 0x50000, None, outs, 0x60000, 0x70000, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_sparse_attn_layers(P(good), qs, 0x60000, 0x70000, outs, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG  # null out
    assert raw.clsa_sparse_attn_layers(P(good), qs, None, 0x70000, qs, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_sparse_attn_layers(P(good), qs, 0x60000, 0x70000, qs, None, wsb, st) == clsa.CLSA_ERR_WORKSPACE
    # projections + append
    h, wq, wk, wkk, wv, qo = 0x90000, 0xA0000, 0xB0000, 0xC0000, 0xD0000, 0xE0000
    ko, kk, vv = 0x30000, 0x10000, 0x20000   # the writable cache pointers
    assert raw.clsa_project_append(P(good), 2560, None, wq, wk, wkk, wv, qo, ko, kk, vv, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_project_append(P(good), 2560, h, wq, wk, wkk, None, qo, ko, kk, vv, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG  # K without V
    assert raw.clsa_project_append(P(good), 2560, h, wq + 8, wk, None, None, qo, ko, None, None, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_project_append(P(good), 0, h, wq, wk, None, None, qo, ko, None, None, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_project_append(P(good), 2568, h, wq, wk, None, None, qo, ko, None, None, ws, wsb, st) == clsa.CLSA_ERR_UNSUPPORTED
    assert raw.clsa_project_append(P(good), 2560, h, wq, wk, wkk, wv, qo, ko, None, vv, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG  # weights without a cache to write
    assert raw.clsa_project_append(P(good), 2560, h, wq, wk, None, None, qo, ko, kk, vv, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG  # a cache without weights
    assert raw.clsa_project_append(P(good), 2560, h, wq, wk, None, None, qo, None, None, None, ws, wsb, st) == clsa.CLSA_ERR_INVALID_ARG
    assert raw.clsa_project_append(P(good), 2560, h, wq, wk, None, None, qo, ko, None, None, None, wsb, st) == clsa.CLSA_ERR_WORKSPACE
    assert raw.clsa_clear_status(None, 0, st) == clsa.CLSA_ERR_WORKSPACE
    assert raw.clsa_device_status(None, None, st) == clsa.CLSA_ERR_INVALID_ARG


def test_chain_planner_is_cheap_and_keyed_on_every_input(clsa):
    """clsa_chain_plan (the host-side choice of the chained layers' launch shapes) needs no GPU. Decode chains of groups
    of up to 8 query heads go two layers per launch. Wider groups keep one layer per launch and may end in a finer
    tail, chosen by a model of how the blocks fill the SMs: a shape that has not been seen must cost microseconds, not
    milliseconds -- a server whose batch size keeps changing pays it on the step that first sees a shape -- and shapes
    are remembered beyond a handful; two models that differ only in the number of KV heads must not share an entry."""
    import time

    def narrow(**kw):
        return clsa.clsa_chain_plan(_good(clsa, max_seq_len=131072, top_k=2048, **{"num_layers": 16, **kw}), 148, 1965000)

    def wide(**kw):   # 16 query heads per KV head: one layer per launch
        kw = {"num_layers": 16, "num_q_heads": 128, "num_kv_heads": 8, "max_seq_len": 131072, **kw}
        return clsa.clsa_chain_plan(_good(clsa, **kw), 148, 1965000)

    # two layers per launch: all of them, all but an odd last one, none for a single layer; prefill chunks,
    # paged caches and unknown devices alike
    assert narrow(num_seqs=16) == (0, 16) and narrow(num_seqs=16, num_layers=15) == (0, 14)
    assert narrow(num_seqs=16, num_layers=1) == (0, 0) and narrow(num_seqs=16, q_per_seq=4) == (0, 16)   # chunks pair too
    assert narrow(num_seqs=20) in ((2, 16), (4, 16), (6, 16))   # more blocks than one round of SMs holds: a finer tail of pairs
    assert narrow(num_seqs=3, block_table=0x5000, block_size=16, max_blocks_per_seq=8192) == (0, 16)
    assert clsa.clsa_chain_plan(_good(clsa, max_seq_len=131072, top_k=2048, num_layers=16, num_seqs=16), 132, 1755000) == (0, 16)
    # wide groups: a short finer tail at most, never pairs; a device the block model was not measured on keeps one shape
    fl, pl = wide(num_seqs=16, top_k=2048)
    assert 0 <= fl <= 3 and pl == 0
    assert clsa.clsa_chain_plan(_good(clsa, max_seq_len=131072, top_k=2048, num_layers=16, num_seqs=16, num_q_heads=128,
                                      num_kv_heads=8), 132, 1755000) == (0, 0)
    shapes = [dict(num_seqs=b, top_k=k) for b in range(1, 51) for k in (1024, 2048)]
    t0 = time.perf_counter()
    first = [wide(**sh) for sh in shapes]
    cold = (time.perf_counter() - t0) / len(shapes)
    t0 = time.perf_counter()
    again = [wide(**sh) for sh in shapes[-60:]]
    warm = (time.perf_counter() - t0) / 60
    assert again == first[-60:]
    assert any(f[0] > 0 for f in first), "the model never chose a finer tail"
    assert cold < 100e-6, f"{cold * 1e6:.1f} us per unseen shape (ctypes call included)"
    assert warm < 30e-6, f"{warm * 1e6:.1f} us per remembered shape"
    # The memo may never hand one model's answer to another (models that share heads per block and rows but differ in
    # the number of KV heads have different block counts): whatever was asked before, the answer is the same. Two
    # fresh processes ask the same 72 models in opposite orders and must agree on every one.
    code = (
        "import sys, json; sys.path.insert(0, %r); import paper_2606_06467_b200 as c\n"
        "cfgs = [(b, hq, hkv, k) for b in (4, 8, 12, 16, 20, 32) for hq, hkv in ((128, 8), (256, 16), (64, 4), (48, 4)) for k in (1024, 2048, 4096)]\n"
        "cfgs = cfgs[::-1] if sys.argv[1] == 'r' else cfgs\n"
        "out = {}\n"
        "for b, hq, hkv, k in cfgs:\n"
        "    p = c.make_params(num_seqs=b, num_q_heads=hq, num_kv_heads=hkv, idx_dim=128, top_k=k, num_layers=16, max_seq_len=131072, sm_scale=0.1)\n"
        "    out[str((b, hq, hkv, k))] = c.clsa_chain_plan(p, 148, 1965000)\n"
        "print(json.dumps(out, sort_keys=True))\n" % ROOT)
    fwd = subprocess.check_output([sys.executable, "-c", code, "f"])
    rev = subprocess.check_output([sys.executable, "-c", code, "r"])
    assert fwd == rev and len(fwd) > 500
    # paged caches, prefill chunks and single layers keep one shape
    assert wide(num_seqs=16, block_table=0x5000, block_size=16, max_blocks_per_seq=8192) == (0, 0)
    assert wide(num_seqs=16, q_per_seq=4) == (0, 0) and wide(num_seqs=16, num_layers=1) == (0, 0)
    n = ctypes.c_int32(0)
    raw = clsa.raw().clsa_chain_plan
    assert raw(ctypes.byref(_good(clsa)), 0, 1965000, ctypes.byref(n), ctypes.byref(n)) == clsa.CLSA_ERR_INVALID_ARG
    assert raw(ctypes.byref(_good(clsa)), 148, 1965000, None, ctypes.byref(n)) == clsa.CLSA_ERR_INVALID_ARG
    assert raw(ctypes.byref(_good(clsa)), 148, 1965000, ctypes.byref(n), None) == clsa.CLSA_ERR_INVALID_ARG


def test_binding_raises_with_the_status(clsa):
    with pytest.raises(clsa.ClsaError) as e:
        clsa.clsa_workspace_bytes(_good(clsa, head_dim=256))
    assert e.value.status == clsa.CLSA_ERR_UNSUPPORTED


def test_product_does_not_touch_the_oracle():
    """Neither the binding nor the CUDA sources may import, include or link anything under oracle/."""
    pkg = os.path.join(ROOT, "paper_2606_06467_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2606_06467_b200" not in text and "clsa.h" not in text
