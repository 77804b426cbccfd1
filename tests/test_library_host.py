"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, builds tree descriptors, and rejects bad arguments before launching anything."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2402_11131_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "ss_msa.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ss_[a-z_]+)\s*\(", header))
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None
    assert lib.ss_version() >= 100


def test_struct_sizes_match_the_header(lib):
    assert C.sizeof(api.TreeDesc) == 16 + 4 * 64 + 4 * 64 + 8 * 64
    assert C.sizeof(api.CacheLayout) == 40
    assert C.sizeof(api.AttnParams) == 24 + 8 * 8 + 3 * 8 + 8 * 8 + 8      # ... + flags (padded to 8)


def test_tree_build_paper_mask_example(lib):
    """Ancestor words of the App. A mask example: 'early' sees parameter, efficient and itself."""
    parent, vis = None, {}
    for line in open(os.path.join(GOLDEN, "mask_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split(":")
        if k == "parent":
            parent = [int(x) for x in v.split()]
        else:
            vis[int(k)] = {int(x) for x in v.split()}
    d = api.ss_tree_build(parent, 2)
    assert d.n_nodes == 5 and d.max_depth == 2 and d.gamma == 2
    for t in range(5):
        assert {a for a in range(64) if (d.anc_mask[t] >> a) & 1} == vis[t]
    assert list(d.depth[:5]) == [0, 1, 1, 2, 2]
    assert list(d.parent[:6]) == parent + [-1]


def test_tree_build_matches_oracle_on_random_trees(lib, oracle):
    from paper_2402_11131_b200 import workloads as W
    rng = np.random.default_rng(1)
    for _ in range(50):
        T = int(rng.integers(1, 65))
        parent = W.draw_tree(rng, T, 6, "uniform_parent")
        d = api.ss_tree_build(parent, 0)
        depth, anc, md = oracle.tree_build(parent)
        assert d.max_depth == md and list(d.depth[:T]) == list(depth)
        for t in range(T):
            assert d.anc_mask[t] == sum(1 << a for a in range(T) if anc[t, a])


def test_tree_build_errors(lib):
    for bad, code in (([0, 0], api.SS_ERR_BAD_TREE), ([-1, 1], api.SS_ERR_BAD_TREE), ([-1, 0, 2], api.SS_ERR_BAD_TREE),
                      ([-1, -1], api.SS_ERR_BAD_TREE), ([], api.SS_ERR_BAD_TREE),
                      ([-1] + [0] * 64, api.SS_ERR_UNSUPPORTED)):
        with pytest.raises(api.SsError) as e:
            api.ss_tree_build(bad, 0)
        assert e.value.status == code
    with pytest.raises(api.SsError) as e:
        api.ss_tree_build([-1], api.SS_MAX_GAMMA + 1)
    assert e.value.status == api.SS_ERR_UNSUPPORTED
    out = api.TreeDesc()
    assert lib.ss_tree_build(None, 1, 0, C.byref(out)) == api.SS_ERR_INVALID_ARG


def _fake_params(**kw):
    """ss_attn_params with plausible, 16-byte aligned but never dereferenced pointers."""
    p = api.AttnParams()
    p.batch, p.n_heads, p.head_dim, p.gamma, p.max_nodes, p.sm_scale = 1, 2, 64, 3, 6, 1.0
    for f in ("q_main", "o_main", "q_spec", "k_spec", "v_spec", "o_spec", "k_cache", "v_cache", "kv_start",
              "kv_len", "trees", "workspace"):
        setattr(p, f, 0x10000)
    p.kv_slot_stride, p.kv_head_stride, p.kv_total_slots = 128, 64, 128
    p.workspace_bytes = 1 << 40
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def test_attention_rejects_bad_arguments_before_any_launch(lib):
    ok_ws = lib.ss_msa_attention_workspace_bytes(C.byref(_fake_params()))
    assert ok_ws > 0
    cases = [
        (dict(head_dim=96), api.SS_ERR_UNSUPPORTED),
        (dict(max_nodes=65), api.SS_ERR_UNSUPPORTED),
        (dict(gamma=5), api.SS_ERR_UNSUPPORTED),
        (dict(batch=0), api.SS_ERR_INVALID_ARG),
        (dict(q_main=None), api.SS_ERR_INVALID_ARG),
        (dict(q_spec=None), api.SS_ERR_INVALID_ARG),
        (dict(k_cache=0x10008), api.SS_ERR_INVALID_ARG),      # misaligned
        (dict(kv_slot_stride=100), api.SS_ERR_INVALID_ARG),   # not a multiple of 8 elements
        (dict(kv_slot_stride=32), api.SS_ERR_INVALID_ARG),    # rows would overlap
        (dict(sm_scale=float("nan")), api.SS_ERR_INVALID_ARG),
        (dict(workspace_bytes=ok_ws - 1), api.SS_ERR_WORKSPACE),
        (dict(workspace=None), api.SS_ERR_INVALID_ARG),
    ]
    for kw, code in cases:
        assert lib.ss_msa_attention(C.byref(_fake_params(**kw)), None) == code, kw
    assert lib.ss_msa_attention(None, None) == api.SS_ERR_INVALID_ARG


def test_verify_and_compact_reject_bad_arguments_before_any_launch(lib):
    need = lib.ss_tree_verify_workspace_bytes(2, 6, 512)
    assert need >= 256 + 2 * 6 * 8
    a = 0x10000
    assert lib.ss_tree_verify(a, a, a, 2, 6, 512, a, a, a, a, None, a, need - 1, None) == api.SS_ERR_WORKSPACE
    assert lib.ss_tree_verify(None, a, a, 2, 6, 512, a, a, a, a, None, a, need, None) == api.SS_ERR_INVALID_ARG
    assert lib.ss_tree_verify(a, a, a, 2, 65, 512, a, a, a, a, None, a, 1 << 30, None) == api.SS_ERR_UNSUPPORTED
    assert lib.ss_tree_verify(a, a, a, 0, 6, 512, a, a, a, a, None, a, need, None) == api.SS_ERR_INVALID_ARG
    lo = api.CacheLayout()
    lo.n_layers, lo.n_heads, lo.head_dim, lo.layer_stride, lo.slot_stride, lo.head_stride = 2, 2, 64, 8192, 128, 64
    assert lib.ss_kv_compact(None, a, C.byref(lo), 1, a, a, a, a, a, None) == api.SS_ERR_INVALID_ARG
    lo.head_dim = 4
    assert lib.ss_kv_compact(a, a, C.byref(lo), 1, a, a, a, a, a, None) == api.SS_ERR_UNSUPPORTED
    lo.head_dim = 64
    assert lib.ss_kv_compact(a + 8, a, C.byref(lo), 1, a, a, a, a, a, None) == api.SS_ERR_INVALID_ARG


def test_error_strings(lib):
    assert lib.ss_error_string(0) == b"ok"
    assert b"workspace" in lib.ss_error_string(api.SS_ERR_WORKSPACE)
