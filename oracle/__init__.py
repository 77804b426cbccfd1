"""CPU oracle (fp64, plain C) for the Speculative-Streaming decode hot path.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library and its Python binding never do.  This file only
marshals numpy arrays into ``ss_oracle.c``; all arithmetic lives there.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ss_oracle.c")
_LIB = os.path.join(_HERE, "libss_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ss_oracle.c with gcc (-O2, OpenMP) into libss_oracle.so beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ssor_max_threads.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError("%s failed with status %d" % (what, rc))


def max_threads() -> int:
    return int(_load().ssor_max_threads())


def set_threads(n: int) -> None:
    _load().ssor_set_threads(C.c_int(int(n)))


def tree_build(parent: np.ndarray) -> Tuple[np.ndarray, np.ndarray, int]:
    """depth[T], is_anc[T][T] (ancestor-or-self), max_depth of the tree given by parent[]."""
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    n = parent.shape[0]
    depth = np.zeros(n, dtype=np.int32)
    anc = np.zeros((n, n), dtype=np.uint8)
    md = C.c_int32(0)
    _check(_load().ssor_tree_build(_p(parent), C.c_int32(n), _p(depth), _p(anc), C.byref(md)), "tree_build")
    return depth, anc, int(md.value)


def msa_attention(parent, L, gamma, sm_scale, q_main, k_cache, v_cache, q_spec=None, k_spec=None,
                  v_spec=None, node_sel=None, heads=None):
    """One layer, one sequence.  bf16 inputs as uint16 arrays:
    q_main [T][H][d]; k_cache/v_cache [>=L+T][H][d] views of this sequence's slots (may be strided
    in slot and head, contiguous in d); q_spec/k_spec/v_spec [T][gamma][H][d] when gamma > 0.
    Returns (o_main f64 [T][H][d], lse_main [T][H], o_spec [T][gamma][H][d] or None, lse_spec or None).
    Rows of unselected nodes / heads are NaN."""
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    T = parent.shape[0]
    q_main = np.ascontiguousarray(q_main, dtype=np.uint16)
    _, H, d = q_main.shape
    assert q_main.shape[0] == T
    for a in (k_cache, v_cache):
        assert a.dtype == np.uint16 and a.strides[2] == 2 and a.shape[0] >= L + T and a.shape[1:] == (H, d)
    assert k_cache.strides == v_cache.strides
    slot_stride, head_stride = k_cache.strides[0] // 2, k_cache.strides[1] // 2
    o_main = np.full((T, H, d), np.nan, dtype=np.float64)
    lse_main = np.full((T, H), np.nan, dtype=np.float64)
    o_spec = lse_spec = None
    if gamma > 0:
        q_spec = np.ascontiguousarray(q_spec, dtype=np.uint16)
        k_spec = np.ascontiguousarray(k_spec, dtype=np.uint16)
        v_spec = np.ascontiguousarray(v_spec, dtype=np.uint16)
        for a in (q_spec, k_spec, v_spec):
            assert a.shape == (T, gamma, H, d)
        o_spec = np.full((T, gamma, H, d), np.nan, dtype=np.float64)
        lse_spec = np.full((T, gamma, H), np.nan, dtype=np.float64)
    if node_sel is not None:
        node_sel = np.ascontiguousarray(node_sel, dtype=np.uint8)
        assert node_sel.shape == (T,)
    h0, h1 = (0, H) if heads is None else heads
    rc = _load().ssor_msa_attention(
        C.c_int32(H), C.c_int32(d), C.c_int32(int(L)), C.c_int32(T), C.c_int32(int(gamma)),
        C.c_double(float(sm_scale)), _p(parent), _p(q_main), _p(q_spec), _p(k_cache), _p(v_cache),
        C.c_int64(slot_stride), C.c_int64(head_stride), _p(k_spec), _p(v_spec), _p(o_main),
        _p(lse_main), _p(o_spec), _p(lse_spec), _p(node_sel), C.c_int32(h0), C.c_int32(h1))
    _check(rc, "msa_attention")
    return o_main, lse_main, o_spec, lse_spec


def tree_verify(logits, tokens, parent, path_cap: Optional[int] = None):
    """One sequence.  logits f32 [T][V], tokens/parent int32 [T].
    Returns dict(accept_len, path (int32[path_cap], -1 padded), last_node, bonus_token, node_argmax)."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    T, V = logits.shape
    cap = T if path_cap is None else int(path_cap)
    path = np.zeros(cap, dtype=np.int32)
    am = np.zeros(T, dtype=np.int32)
    ln, last, bonus = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    rc = _load().ssor_tree_verify(_p(logits), _p(tokens), _p(parent), C.c_int32(T), C.c_int32(V),
                                  C.byref(ln), _p(path), C.c_int32(cap), C.byref(last), C.byref(bonus),
                                  _p(am))
    _check(rc, "tree_verify")
    return dict(accept_len=int(ln.value), path=path, last_node=int(last.value),
                bonus_token=int(bonus.value), node_argmax=am)


def kv_compact(k_all, v_all, L, accept_len, path):
    """One sequence.  k_all/v_all uint16 [n_layers][slots][H][d] views (d contiguous).
    Returns (k_new, v_new, new_len): copies with slot L+i <- slot L+path[i] in every layer."""
    assert k_all.dtype == np.uint16 and v_all.dtype == np.uint16 and k_all.shape == v_all.shape
    k_src = np.ascontiguousarray(k_all)
    v_src = np.ascontiguousarray(v_all)
    k_dst, v_dst = k_src.copy(), v_src.copy()
    n_layers, slots, H, d = k_src.shape
    path = np.ascontiguousarray(path, dtype=np.int32)
    new_len = C.c_int32(0)
    rc = _load().ssor_kv_compact(_p(k_src), _p(v_src), _p(k_dst), _p(v_dst), C.c_int32(n_layers),
                                 C.c_int64(slots * H * d), C.c_int64(H * d), C.c_int64(d), C.c_int32(H),
                                 C.c_int32(d), C.c_int32(int(L)), C.c_int32(int(accept_len)), _p(path),
                                 C.byref(new_len))
    _check(rc, "kv_compact")
    return k_dst, v_dst, int(new_len.value)


def next_draft(stream_logits, k: int, bonus_token: int, max_nodes: int):
    """Next tree draft from the stream logits [gamma][V] of the last accepted node.
    Returns (tokens int32[n], parent int32[n])."""
    lg = np.ascontiguousarray(stream_logits, dtype=np.float32)
    gamma, V = lg.shape
    tokens = np.zeros(max_nodes, dtype=np.int32)
    parent = np.zeros(max_nodes, dtype=np.int32)
    n = C.c_int32(0)
    rc = _load().ssor_next_draft(_p(lg), C.c_int32(gamma), C.c_int32(V), C.c_int32(int(k)), C.c_int32(int(bonus_token)),
                                 C.c_int32(int(max_nodes)), C.byref(n), _p(tokens), _p(parent))
    _check(rc, "next_draft")
    return tokens[:n.value].copy(), parent[:n.value].copy()


def tree_prune(logits, tokens, parent, threshold: float, decide=None):
    """Prunes sub-trees below edges whose early-exit transition probability is under the threshold.
    logits f32 [T][V].  Returns dict(edge_prob f64[T], keep u8[T], new_index i32[T], kept_nodes i32[n],
    new_parent i32[n])."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    T, V = logits.shape
    prob = np.zeros(T, dtype=np.float64)
    keep = np.zeros(T, dtype=np.uint8)
    new_index = np.zeros(T, dtype=np.int32)
    kept = np.zeros(T, dtype=np.int32)
    new_parent = np.zeros(T, dtype=np.int32)
    n = C.c_int32(0)
    dec = None if decide is None else np.ascontiguousarray(decide, dtype=np.uint8)
    rc = _load().ssor_tree_prune(_p(logits), _p(tokens), _p(parent), C.c_int32(T), C.c_int32(V), C.c_double(float(threshold)),
                                 _p(dec), _p(prob), _p(keep), _p(new_index), C.byref(n), _p(kept), _p(new_parent))
    _check(rc, "tree_prune")
    return dict(edge_prob=prob, keep=keep, new_index=new_index, kept_nodes=kept[:n.value].copy(),
                new_parent=new_parent[:n.value].copy())


def tree_verify_soft(logits, tokens, parent, eps: float, delta: float, decide=None, path_cap: Optional[int] = None):
    """Verification with the soft (typical-acceptance) criterion.  Returns the dict of tree_verify plus
    edge_prob and node_entropy."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    T, V = logits.shape
    cap = T if path_cap is None else int(path_cap)
    path = np.zeros(cap, dtype=np.int32)
    prob = np.zeros(T, dtype=np.float64)
    ent = np.zeros(T, dtype=np.float64)
    ln, last, bonus = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    dec = None if decide is None else np.ascontiguousarray(decide, dtype=np.uint8)
    rc = _load().ssor_tree_verify_soft(_p(logits), _p(tokens), _p(parent), C.c_int32(T), C.c_int32(V), C.c_double(float(eps)),
                                       C.c_double(float(delta)), _p(dec), C.byref(ln), _p(path), C.c_int32(cap),
                                       C.byref(last), C.byref(bonus), _p(prob), _p(ent))
    _check(rc, "tree_verify_soft")
    return dict(accept_len=int(ln.value), path=path, last_node=int(last.value), bonus_token=int(bonus.value),
                edge_prob=prob, node_entropy=ent)


def tree_verify_sampled(logits, tokens, parent, k: int, u, drawn=None, path_cap: Optional[int] = None):
    """Verification against tokens drawn from the top-k softmax (temperature 1) with the uniforms u[T]."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    u = np.ascontiguousarray(u, dtype=np.float32)
    T, V = logits.shape
    cap = T if path_cap is None else int(path_cap)
    path = np.zeros(cap, dtype=np.int32)
    node_token = np.zeros(T, dtype=np.int32)
    ln, last, bonus = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    dr = None if drawn is None else np.ascontiguousarray(drawn, dtype=np.int32)
    rc = _load().ssor_tree_verify_sampled(_p(logits), _p(tokens), _p(parent), C.c_int32(T), C.c_int32(V), C.c_int32(int(k)),
                                          _p(u), _p(dr), C.byref(ln), _p(path), C.c_int32(cap), C.byref(last),
                                          C.byref(bonus), _p(node_token))
    _check(rc, "tree_verify_sampled")
    return dict(accept_len=int(ln.value), path=path, last_node=int(last.value), bonus_token=int(bonus.value),
                node_token=node_token)


def stream_insert(m, p):
    """S[t][j] = M[t] + P[j] (Eq. 3 with the identity transformation).  m uint16 [rows][hidden],
    p uint16 [gamma][hidden] (bf16 bit patterns).  Returns uint16 [rows][gamma][hidden]."""
    m = np.ascontiguousarray(m, dtype=np.uint16)
    p = np.ascontiguousarray(p, dtype=np.uint16)
    rows, hidden = m.shape
    gamma = p.shape[0]
    out = np.zeros((rows, gamma, hidden), dtype=np.uint16)
    _check(_load().ssor_stream_insert(_p(m), _p(p), _p(out), C.c_int64(rows), C.c_int32(gamma), C.c_int32(hidden)),
           "stream_insert")
    return out


def rotation_table(epsilon: float, gamma: int) -> np.ndarray:
    """cos / sin of epsilon * n, n = 1..gamma, evaluated in fp64 and rounded to fp32: [gamma][2]."""
    n = np.arange(1, gamma + 1, dtype=np.float64)
    return np.stack([np.cos(epsilon * n), np.sin(epsilon * n)], axis=1).astype(np.float32)


def value_rotate(v, gamma: int, epsilon: float):
    """V[t][n] = V[t] * exp(i * epsilon * n) on consecutive (re, im) pairs (Eq. 7).  v uint16 [rows][width].
    Returns uint16 [rows][gamma][width]."""
    v = np.ascontiguousarray(v, dtype=np.uint16)
    rows, width = v.shape
    out = np.zeros((rows, gamma, width), dtype=np.uint16)
    cs = np.ascontiguousarray(rotation_table(epsilon, gamma))
    _check(_load().ssor_value_rotate(_p(v), _p(out), C.c_int64(rows), C.c_int32(gamma), C.c_int32(width), _p(cs)),
           "value_rotate")
    return out
