"""ctypes binding of libss_msa.so: the same entry points as include/ss_msa.h.

Argument marshalling only: every step of the path runs in the CUDA library.  PyTorch is used for
device memory and streams.  There is no fallback: if the library is missing or cannot be loaded
this module raises, it never computes anything itself.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

SS_MAX_NODES = 64
SS_MAX_GAMMA = 4
SS_PATH_STRIDE = SS_MAX_NODES

SS_OK = 0
SS_ERR_INVALID_ARG = -1
SS_ERR_BAD_TREE = -2
SS_ERR_UNSUPPORTED = -3
SS_ERR_WORKSPACE = -4
SS_ERR_CAPACITY = -5
SS_ERR_CUDA = -6
SS_ERR_DEVICE_TIMEOUT = -7

SS_ATTN_PREFIX_STABLE = 1

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libss_msa.so")
_lib = None

# number of kernels each entry point enqueues per call (for launch accounting in the benchmark)
LAUNCHES_PER_CALL = {"ss_msa_attention": 1, "ss_tree_verify": 1, "ss_kv_compact": 2, "ss_next_draft": 1,
                     "ss_tree_prune": 1, "ss_tree_verify_soft": 1, "ss_tree_verify_sampled": 1, "ss_stream_insert": 1,
                     "ss_value_rotate": 1}


class SsError(RuntimeError):
    def __init__(self, what: str, status: int):
        self.status = status
        msg = lib().ss_error_string(C.c_int32(status)).decode() if _lib is not None else "?"
        super().__init__("%s failed: status %d (%s)" % (what, status, msg))


class TreeDesc(C.Structure):
    _fields_ = [("n_nodes", C.c_int32), ("gamma", C.c_int32), ("max_depth", C.c_int32), ("reserved", C.c_int32),
                ("parent", C.c_int32 * SS_MAX_NODES), ("depth", C.c_int32 * SS_MAX_NODES),
                ("anc_mask", C.c_uint64 * SS_MAX_NODES)]


class AttnParams(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("gamma", C.c_int32),
                ("max_nodes", C.c_int32), ("sm_scale", C.c_float),
                ("q_main", C.c_void_p), ("o_main", C.c_void_p), ("q_spec", C.c_void_p), ("k_spec", C.c_void_p),
                ("v_spec", C.c_void_p), ("o_spec", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
                ("kv_slot_stride", C.c_int64), ("kv_head_stride", C.c_int64), ("kv_total_slots", C.c_int64),
                ("kv_start", C.c_void_p), ("kv_len", C.c_void_p), ("kv_capacity", C.c_void_p),
                ("trees", C.c_void_p), ("lse_main", C.c_void_p), ("lse_spec", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("flags", C.c_uint32)]


class CacheLayout(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("reserved", C.c_int32),
                ("layer_stride", C.c_int64), ("slot_stride", C.c_int64), ("head_stride", C.c_int64)]


EXPORTS = ("ss_tree_build", "ss_msa_attention_workspace_bytes", "ss_msa_attention",
           "ss_tree_verify_workspace_bytes", "ss_tree_verify", "ss_tree_verify_static", "ss_kv_compact", "ss_status",
           "ss_version", "ss_error_string",
           "ss_next_draft_workspace_bytes", "ss_next_draft", "ss_tree_prune_workspace_bytes", "ss_tree_prune",
           "ss_tree_verify_soft", "ss_tree_verify_sampled_workspace_bytes", "ss_tree_verify_sampled",
           "ss_stream_insert", "ss_value_rotate", "ss_wait_selftest")
SS_MAX_TOPK = 8
SS_VERIFY_STATIC_SCRATCH_BYTES = 1 << 20


def lib() -> C.CDLL:
    """Loads libss_msa.so (built in-tree by paper_2402_11131_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: run `python -m paper_2402_11131_b200.build` "
                               "(there is no CPU fallback)" % _LIB_PATH)
        l = C.CDLL(_LIB_PATH)
        l.ss_tree_build.restype = C.c_int32
        l.ss_tree_build.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(TreeDesc)]
        l.ss_msa_attention_workspace_bytes.restype = C.c_size_t
        l.ss_msa_attention_workspace_bytes.argtypes = [C.POINTER(AttnParams)]
        l.ss_msa_attention.restype = C.c_int32
        l.ss_msa_attention.argtypes = [C.POINTER(AttnParams), C.c_void_p]
        l.ss_tree_verify_workspace_bytes.restype = C.c_size_t
        l.ss_tree_verify_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        l.ss_tree_verify.restype = C.c_int32
        l.ss_tree_verify.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.c_size_t, C.c_void_p]
        l.ss_tree_verify_static.restype = C.c_int32
        l.ss_tree_verify_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        l.ss_kv_compact.restype = C.c_int32
        l.ss_kv_compact.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(CacheLayout), C.c_int32, C.c_void_p,
                                    C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
        for name in ("ss_next_draft_workspace_bytes", "ss_tree_prune_workspace_bytes", "ss_tree_verify_sampled_workspace_bytes"):
            getattr(l, name).restype = C.c_size_t
            getattr(l, name).argtypes = [i32, i32, i32]
        l.ss_next_draft.restype = i32
        l.ss_next_draft.argtypes = [vp, i32, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, C.c_size_t, vp]
        l.ss_tree_prune.restype = i32
        l.ss_tree_prune.argtypes = [vp, vp, vp, i32, i32, i32, f32, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        l.ss_tree_verify_soft.restype = i32
        l.ss_tree_verify_soft.argtypes = [vp, vp, vp, i32, i32, i32, f32, f32, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        l.ss_tree_verify_sampled.restype = i32
        l.ss_tree_verify_sampled.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        l.ss_stream_insert.restype = i32
        l.ss_stream_insert.argtypes = [vp, vp, vp, C.c_int64, i32, i32, vp]
        l.ss_value_rotate.restype = i32
        l.ss_value_rotate.argtypes = [vp, vp, C.c_int64, i32, i32, f32, vp]
        l.ss_wait_selftest.restype = C.c_int32
        l.ss_wait_selftest.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
        l.ss_status.restype = C.c_int32
        l.ss_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
        l.ss_version.restype = C.c_int32
        l.ss_error_string.restype = C.c_char_p
        l.ss_error_string.argtypes = [C.c_int32]
        _lib = l
    return _lib


def _check(status: int, what: str) -> None:
    if status != SS_OK:
        raise SsError(what, status)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


# ---- host ---------------------------------------------------------------------------------------
def ss_tree_build(parent: Sequence[int], gamma: int) -> TreeDesc:
    """Host-side descriptor of one tree (depth, ancestor bit masks) from its parent array."""
    par = np.ascontiguousarray(parent, dtype=np.int32)
    out = TreeDesc()
    _check(lib().ss_tree_build(par.ctypes.data, C.c_int32(par.shape[0]), C.c_int32(gamma), C.byref(out)),
           "ss_tree_build")
    return out


def trees_to_device(descs: Sequence[TreeDesc], device="cuda") -> torch.Tensor:
    """Packs descriptors into one device byte tensor (the `trees` argument of the device calls)."""
    raw = b"".join(bytes(d) for d in descs)
    host = torch.frombuffer(bytearray(raw), dtype=torch.uint8)
    return host.to(device)


def workspace(n_bytes: int, device="cuda") -> torch.Tensor:
    """A zero-filled workspace of at least n_bytes (256-byte granularity)."""
    return torch.zeros((int(n_bytes) + 255) // 256 * 256, dtype=torch.uint8, device=device)


# ---- device -------------------------------------------------------------------------------------
def make_attn_params(*, q_main, o_main, k_cache, v_cache, kv_start, kv_len, trees, gamma, sm_scale,
                     q_spec=None, k_spec=None, v_spec=None, o_spec=None, kv_capacity=None, lse_main=None,
                     lse_spec=None, workspace=None, prefix_stable=False) -> AttnParams:
    """Fills ss_attn_params from tensors.  q_main/o_main: bf16 [B][Tmax][H][d]; *_spec: bf16
    [B][Tmax][gamma][H][d]; k_cache/v_cache: bf16 [slots][H][d] (any slot/head stride, d contiguous)."""
    B, Tmax, H, d = q_main.shape
    assert k_cache.dim() == 3 and k_cache.stride(2) == 1 and k_cache.stride() == v_cache.stride()
    p = AttnParams()
    p.batch, p.n_heads, p.head_dim, p.gamma, p.max_nodes = B, H, d, int(gamma), Tmax
    p.sm_scale = float(sm_scale)
    p.q_main, p.o_main = _ptr(q_main), _ptr(o_main)
    p.q_spec, p.k_spec, p.v_spec, p.o_spec = _ptr(q_spec), _ptr(k_spec), _ptr(v_spec), _ptr(o_spec)
    p.k_cache, p.v_cache = _ptr(k_cache), _ptr(v_cache)
    p.kv_slot_stride, p.kv_head_stride, p.kv_total_slots = k_cache.stride(0), k_cache.stride(1), k_cache.shape[0]
    p.kv_start, p.kv_len, p.kv_capacity = _ptr(kv_start), _ptr(kv_len), _ptr(kv_capacity)
    p.trees = _ptr(trees)
    p.lse_main, p.lse_spec = _ptr(lse_main), _ptr(lse_spec)
    p.workspace = _ptr(workspace)
    p.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    p.flags = SS_ATTN_PREFIX_STABLE if prefix_stable else 0
    return p


def ss_msa_attention_workspace_bytes(p: AttnParams) -> int:
    return int(lib().ss_msa_attention_workspace_bytes(C.byref(p)))


def ss_msa_attention(p: AttnParams, stream: Optional[torch.cuda.Stream] = None) -> None:
    """One layer of tree-masked multi-stream attention (asynchronous on `stream`)."""
    _check(lib().ss_msa_attention(C.byref(p), _stream(stream)), "ss_msa_attention")


def ss_tree_verify_workspace_bytes(batch: int, max_nodes: int, vocab: int) -> int:
    return int(lib().ss_tree_verify_workspace_bytes(batch, max_nodes, vocab))


def ss_tree_verify(logits, draft_tokens, trees, accept_len, accept_path, last_node, bonus_token,
                   node_argmax, workspace, stream=None) -> None:
    """Greedy verification.  logits f32 [B][Tmax][V]; the int32 outputs are written on the device."""
    B, Tmax, V = logits.shape
    _check(lib().ss_tree_verify(_ptr(logits), _ptr(draft_tokens), _ptr(trees), B, Tmax, V, _ptr(accept_len),
                                _ptr(accept_path), _ptr(last_node), _ptr(bonus_token), _ptr(node_argmax),
                                _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "ss_tree_verify")


def ss_tree_verify_static(logits, draft_tokens, trees, accept_len, accept_path, last_node, bonus_token,
                          node_argmax, stream=None) -> None:
    """ss_tree_verify for callers that cannot supply scratch memory (no allocator of their own, or
    allocation forbidden where they call): the scratch is a fixed array inside the library, shared
    by every call on the device, so overlapping calls race.  Raises SsError(SS_ERR_WORKSPACE) when
    the sizes need more than SS_VERIFY_STATIC_SCRATCH_BYTES.  Make the first call on a device
    outside any stream capture."""
    B, Tmax, V = logits.shape
    _check(lib().ss_tree_verify_static(_ptr(logits), _ptr(draft_tokens), _ptr(trees), B, Tmax, V,
                                       _ptr(accept_len), _ptr(accept_path), _ptr(last_node), _ptr(bonus_token),
                                       _ptr(node_argmax), _stream(stream)), "ss_tree_verify_static")


def _ws_bytes(t: torch.Tensor) -> int:
    return t.numel() * t.element_size()


def empty_trees(batch: int, device="cuda") -> torch.Tensor:
    """Device storage for `batch` tree descriptors (written by ss_next_draft / ss_tree_prune)."""
    return torch.zeros(batch * C.sizeof(TreeDesc), dtype=torch.uint8, device=device)


def trees_from_device(trees: torch.Tensor):
    """Descriptors back on the host (tests)."""
    raw = trees.cpu().numpy().tobytes()
    n = len(raw) // C.sizeof(TreeDesc)
    return [TreeDesc.from_buffer_copy(raw[i * C.sizeof(TreeDesc):(i + 1) * C.sizeof(TreeDesc)]) for i in range(n)]


def ss_next_draft_workspace_bytes(batch: int, gamma: int, vocab: int) -> int:
    return int(lib().ss_next_draft_workspace_bytes(batch, gamma, vocab))


def ss_next_draft(stream_logits, row_index, bonus_token, top_k: int, max_nodes: int, draft_tokens, trees, workspace,
                  stream=None) -> None:
    """Next tree draft.  stream_logits f32 [B][n_rows][gamma][V]; row_index int32 [B] or None; bonus_token int32 [B];
    draft_tokens int32 [B][max_nodes] and trees (empty_trees(B)) are written on the device."""
    B, n_rows, gamma, V = stream_logits.shape
    _check(lib().ss_next_draft(_ptr(stream_logits), n_rows, _ptr(row_index), _ptr(bonus_token), B, gamma, V, int(top_k),
                               int(max_nodes), _ptr(draft_tokens), _ptr(trees), _ptr(workspace), _ws_bytes(workspace),
                               _stream(stream)), "ss_next_draft")


def ss_tree_prune_workspace_bytes(batch: int, max_nodes: int, vocab: int) -> int:
    return int(lib().ss_tree_prune_workspace_bytes(batch, max_nodes, vocab))


def ss_tree_prune(exit_logits, draft_tokens, trees, threshold: float, edge_prob, new_index, kept_nodes, kept_tokens,
                  pruned_trees, workspace, stream=None) -> None:
    """Parallel tree pruning.  exit_logits f32 [B][Tmax][V]; outputs are written on the device."""
    B, Tmax, V = exit_logits.shape
    _check(lib().ss_tree_prune(_ptr(exit_logits), _ptr(draft_tokens), _ptr(trees), B, Tmax, V, float(threshold),
                               _ptr(edge_prob), _ptr(new_index), _ptr(kept_nodes), _ptr(kept_tokens), _ptr(pruned_trees),
                               _ptr(workspace), _ws_bytes(workspace), _stream(stream)), "ss_tree_prune")


def ss_tree_verify_soft(logits, draft_tokens, trees, eps: float, delta: float, accept_len, accept_path, last_node,
                        bonus_token, edge_prob, node_entropy, workspace, stream=None) -> None:
    """Verification with the soft (typical-acceptance) criterion; workspace of ss_tree_prune_workspace_bytes."""
    B, Tmax, V = logits.shape
    _check(lib().ss_tree_verify_soft(_ptr(logits), _ptr(draft_tokens), _ptr(trees), B, Tmax, V, float(eps), float(delta),
                                     _ptr(accept_len), _ptr(accept_path), _ptr(last_node), _ptr(bonus_token),
                                     _ptr(edge_prob), _ptr(node_entropy), _ptr(workspace), _ws_bytes(workspace),
                                     _stream(stream)), "ss_tree_verify_soft")


def ss_tree_verify_sampled_workspace_bytes(batch: int, max_nodes: int, vocab: int) -> int:
    return int(lib().ss_tree_verify_sampled_workspace_bytes(batch, max_nodes, vocab))


def ss_tree_verify_sampled(logits, draft_tokens, trees, uniforms, top_k: int, accept_len, accept_path, last_node,
                           bonus_token, node_token, workspace, stream=None) -> None:
    """Verification against tokens drawn from the top-k softmax (temperature 1) with the caller's uniforms f32 [B][Tmax]."""
    B, Tmax, V = logits.shape
    _check(lib().ss_tree_verify_sampled(_ptr(logits), _ptr(draft_tokens), _ptr(trees), _ptr(uniforms), B, Tmax, V,
                                        int(top_k), _ptr(accept_len), _ptr(accept_path), _ptr(last_node),
                                        _ptr(bonus_token), _ptr(node_token), _ptr(workspace), _ws_bytes(workspace),
                                        _stream(stream)), "ss_tree_verify_sampled")


def ss_stream_insert(main_hidden, stream_emb, out, stream=None) -> None:
    """out[t][j] = main_hidden[t] + stream_emb[j] (Eq. 3, identity transformation); bf16 [rows][hidden], [gamma][hidden]."""
    rows, hidden = main_hidden.shape
    gamma = stream_emb.shape[0]
    _check(lib().ss_stream_insert(_ptr(main_hidden), _ptr(stream_emb), _ptr(out), rows, gamma, hidden, _stream(stream)),
           "ss_stream_insert")


def ss_value_rotate(v_main, v_streams, epsilon: float, stream=None) -> None:
    """v_streams[t][n-1] = v_main[t] rotated by epsilon * n on (re, im) pairs (Eq. 7); bf16 [rows][width], [rows][gamma][width]."""
    rows, width = v_main.shape
    gamma = v_streams.shape[1]
    _check(lib().ss_value_rotate(_ptr(v_main), _ptr(v_streams), rows, gamma, width, float(epsilon), _stream(stream)),
           "ss_value_rotate")


def make_cache_layout(k_all: torch.Tensor) -> CacheLayout:
    """Layout of a bf16 cache tensor [n_layers][slots][H][d] (d contiguous)."""
    n_layers, _, H, d = k_all.shape
    assert k_all.stride(3) == 1
    lo = CacheLayout()
    lo.n_layers, lo.n_heads, lo.head_dim = n_layers, H, d
    lo.layer_stride, lo.slot_stride, lo.head_stride = k_all.stride(0), k_all.stride(1), k_all.stride(2)
    return lo


def ss_kv_compact(k_all, v_all, layout: CacheLayout, kv_start, kv_len_in, accept_len, accept_path, kv_len_out,
                  stream=None) -> None:
    """In-place gather of the accepted path's K/V in every layer (asynchronous on `stream`)."""
    _check(lib().ss_kv_compact(_ptr(k_all), _ptr(v_all), C.byref(layout), kv_start.shape[0], _ptr(kv_start),
                               _ptr(kv_len_in), _ptr(accept_len), _ptr(accept_path), _ptr(kv_len_out),
                               _stream(stream)), "ss_kv_compact")


def ss_wait_selftest(workspace: torch.Tensor, stream=None) -> None:
    """Diagnostic: one warp waits (bounded by workspace word 1) for a partial row that cannot arrive."""
    _check(lib().ss_wait_selftest(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "ss_wait_selftest")


def ss_status(workspace: torch.Tensor, stream=None) -> int:
    """Synchronises the stream and returns (and clears) the workspace's device status word."""
    out = C.c_int32(0)
    _check(lib().ss_status(_ptr(workspace), _stream(stream), C.byref(out)), "ss_status")
    return int(out.value)


# ---- numpy <-> device helpers for bf16 bit patterns ----------------------------------------------
def bf16_to_device(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bit patterns -> bf16 tensor on the device (no value conversion)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def bf16_to_host_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 device tensor -> uint16 bit patterns on the host."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
