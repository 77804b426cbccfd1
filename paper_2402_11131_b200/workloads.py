"""Seeded synthetic inputs for one Speculative-Streaming decode step.

This module only *draws inputs*: shapes, trees, bf16 tensors, logits.  It holds none of the
method's arithmetic (no attention, no mask construction, no argmax, no gather), so both the
CPU oracle and the CUDA path may consume its buffers.  It depends on numpy alone.

bf16 tensors are carried as ``numpy.uint16`` arrays holding the raw bit patterns.

The five named configurations stand in for the paper's workloads (OPT-1.3B / Phi-1.3B /
Phi-2-like / LLaMA-7B-like models decoding with a tree draft, Sec. 3.2.2 and App. A.1):
the KV prefix is the main-stream cache of the tokens decoded so far, the tree is the
flattened draft of the previous pass, and every tree node carries gamma speculative
streams in the last N_s layers (Sec. 3.2.1).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

# tensor ids used to derive independent random substreams
_TID_TREE, _TID_TOKENS, _TID_LOGITS, _TID_ACCEPT, _TID_LEN = 1, 2, 3, 4, 5
_TID_QM, _TID_QS, _TID_KS, _TID_VS, _TID_K, _TID_V, _TID_P = 10, 11, 12, 13, 14, 15, 16


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even) and return the bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float64."""
    u = b.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def _rng(seed: int, *key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, *key])))


def _normal_bf16(rng: np.random.Generator, shape, scale: float = 1.0) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if scale != 1.0:
        x *= np.float32(scale)
    return f32_to_bf16_bits(x)


@dataclass(frozen=True)
class StepConfig:
    """Shape of one decode step (one row of the configuration table)."""

    name: str
    config_id: int
    batch: int
    n_layers: int
    n_msa_layers: int           # N_s: the last N_s layers are multi-stream
    n_heads: int
    head_dim: int
    prefix_len: int             # L when fixed
    prefix_len_range: Optional[tuple]  # (lo, hi) inclusive when ragged
    n_nodes: int                # T
    max_depth: int
    gamma: int
    vocab: int
    p_accept: float
    p_accept_range: Optional[tuple]
    tree_kind: str              # "uniform_parent" (tiny) | "topk_growth"
    max_children: int = 4
    k_ramp: float = 0.0         # test inputs only: K of cache slot s is scaled by (1 + k_ramp * s), so the
                                # largest score of a row keeps growing along the keys

    @property
    def seed(self) -> int:
        return 0x5EED0000 + self.config_id


CONFIGS: Dict[str, StepConfig] = {
    "tiny": StepConfig("tiny", 1, 1, 1, 1, 2, 64, 64, None, 6, 2, 3, 512, 0.6, None, "uniform_parent"),
    "1.3b": StepConfig("1.3b", 2, 1, 24, 4, 32, 64, 512, None, 16, 3, 3, 51200, 0.7, None, "topk_growth"),
    "2.7b": StepConfig("2.7b", 3, 1, 32, 4, 32, 80, 1024, None, 32, 4, 3, 51200, 0.7, None, "topk_growth"),
    "7b": StepConfig("7b", 4, 1, 32, 4, 32, 128, 2048, None, 64, 4, 4, 32000, 0.6, None, "topk_growth"),
    "7b_ragged16": StepConfig("7b_ragged16", 5, 16, 32, 4, 32, 128, 0, (512, 4096), 64, 4, 4, 32000,
                              0.6, (0.4, 0.8), "topk_growth"),
}


def draw_tree(rng: np.random.Generator, n_nodes: int, max_depth: int, kind: str,
              max_children: int = 4) -> np.ndarray:
    """Parent array of a random draft tree; node 0 is the root, parent[i] < i."""
    parent = np.full(n_nodes, -1, dtype=np.int32)
    depth = np.zeros(n_nodes, dtype=np.int32)
    n_child = np.zeros(n_nodes, dtype=np.int32)
    for i in range(1, n_nodes):
        if kind == "uniform_parent":
            cand = [u for u in range(i) if depth[u] < max_depth]
        elif kind == "topk_growth":
            cand = [u for u in range(i) if depth[u] < max_depth and n_child[u] < max_children]
        elif kind == "chain":
            cand = [i - 1]
        else:
            raise ValueError(kind)
        if not cand:
            raise ValueError("tree cannot grow: depth/children limits too tight")
        u = int(cand[int(rng.integers(0, len(cand)))])
        parent[i] = u
        depth[i] = depth[u] + 1
        n_child[u] += 1
    return parent


@dataclass
class LayerInputs:
    """Per-layer tensors (bf16 bit patterns).  Layouts:

    q_main            [B][T][H][d]
    q_spec/k_spec/v_spec [B][T][gamma][H][d]   (None in plain layers)
    k_cache/v_cache   [slots][H][d]; sequence b owns slots kv_start[b] .. kv_start[b]+capacity[b)-1,
                      prefix at +0..L_b-1 and the tree nodes' K/V at +L_b .. +L_b+T-1.
    """

    layer: int
    is_msa: bool
    q_main: np.ndarray
    q_spec: Optional[np.ndarray]
    k_spec: Optional[np.ndarray]
    v_spec: Optional[np.ndarray]
    k_cache: Optional[np.ndarray]
    v_cache: Optional[np.ndarray]


@dataclass
class StepInputs:
    cfg: StepConfig
    kv_len: np.ndarray          # int32 [B]  L_b
    kv_start: np.ndarray        # int64 [B]
    kv_capacity: np.ndarray     # int32 [B]
    total_slots: int
    parent: np.ndarray          # int32 [B][T]
    draft_tokens: np.ndarray    # int32 [B][T]
    p_accept: np.ndarray        # float64 [B]
    sm_scale: float
    q_scale: float
    n_nodes_b: Optional[np.ndarray] = None   # per-sequence tree sizes T_b <= T (default: all T)
    _logits: Optional[np.ndarray] = field(default=None, repr=False)

    def nodes(self, b: int) -> int:
        return self.cfg.n_nodes if self.n_nodes_b is None else int(self.n_nodes_b[b])

    # ---- per-step tensors -------------------------------------------------------------
    def logits(self) -> np.ndarray:
        """fp32 main-stream logits [B][T][V]: N(0,1), then for every parent u its children (in
        index order) each draw Bernoulli(p); the first hit c gets logits[u][tok[c]] = 16."""
        if self._logits is not None:
            return self._logits
        c = self.cfg
        out = np.empty((c.batch, c.n_nodes, c.vocab), dtype=np.float32)
        for b in range(c.batch):
            r = _rng(c.seed, _TID_LOGITS, b)
            out[b] = r.standard_normal(size=(c.n_nodes, c.vocab), dtype=np.float32)
            ra = _rng(c.seed, _TID_ACCEPT, b)
            hit = ra.random(c.n_nodes) < self.p_accept[b]
            forced = np.zeros(c.n_nodes, dtype=bool)
            for ch in range(1, c.n_nodes):
                u = int(self.parent[b, ch])
                if hit[ch] and not forced[u]:
                    out[b, u, int(self.draft_tokens[b, ch])] = np.float32(16.0)
                    forced[u] = True
        self._logits = out
        return out

    # ---- per-layer tensors ------------------------------------------------------------
    def is_msa_layer(self, layer: int) -> bool:
        return layer >= self.cfg.n_layers - self.cfg.n_msa_layers

    def layer(self, layer: int, slab_seed: Optional[int] = None, with_slab: bool = True) -> LayerInputs:
        """Draw the tensors of one layer.  `slab_seed` (default: the layer index) selects the
        random substream of the KV slab, so a caller may reuse a few distinct slabs for many
        layers when host memory is short; with_slab=False skips the slab (k_cache = v_cache = None)."""
        c = self.cfg
        B, T, H, d, g = c.batch, c.n_nodes, c.n_heads, c.head_dim, c.gamma
        msa = self.is_msa_layer(layer)
        qm = _normal_bf16(_rng(c.seed, _TID_QM, layer), (B, T, H, d), self.q_scale)
        qs = ks = vs = None
        if msa and g > 0:
            qs = _normal_bf16(_rng(c.seed, _TID_QS, layer), (B, T, g, H, d), self.q_scale)
            ks = _normal_bf16(_rng(c.seed, _TID_KS, layer), (B, T, g, H, d))
            vs = _normal_bf16(_rng(c.seed, _TID_VS, layer), (B, T, g, H, d))
        s = layer if slab_seed is None else slab_seed
        kc = vc = None
        if with_slab:
            if c.k_ramp:
                x = _rng(c.seed, _TID_K, s).standard_normal(size=(self.total_slots, H, d), dtype=np.float32)
                x *= (1.0 + np.float32(c.k_ramp) * np.arange(self.total_slots, dtype=np.float32))[:, None, None]
                kc = f32_to_bf16_bits(x)
            else:
                kc = _normal_bf16(_rng(c.seed, _TID_K, s), (self.total_slots, H, d))
            vc = _normal_bf16(_rng(c.seed, _TID_V, s), (self.total_slots, H, d))
        return LayerInputs(layer, msa and g > 0, qm, qs, ks, vs, kc, vc)


def make_step(cfg: StepConfig, *, q_unit_variance: bool = False) -> StepInputs:
    """Draw the per-step structure of `cfg`: prefix lengths, slab layout, trees, draft tokens.

    Default: queries are N(0,1)/sqrt(d) and sm_scale = 1.  With `q_unit_variance` queries are
    N(0,1) and sm_scale = 1/sqrt(d); both give unit-variance scores."""
    B, T = cfg.batch, cfg.n_nodes
    if cfg.prefix_len_range is None:
        kv_len = np.full(B, cfg.prefix_len, dtype=np.int32)
    else:
        lo, hi = cfg.prefix_len_range
        kv_len = _rng(cfg.seed, _TID_LEN).integers(lo, hi + 1, size=B).astype(np.int32)
    cap = ((kv_len.astype(np.int64) + T + 63) // 64 * 64).astype(np.int32)
    kv_start = np.zeros(B, dtype=np.int64)
    kv_start[1:] = np.cumsum(cap.astype(np.int64))[:-1]
    total = int(cap.astype(np.int64).sum())
    parent = np.stack([draw_tree(_rng(cfg.seed, _TID_TREE, b), T, cfg.max_depth, cfg.tree_kind,
                                 cfg.max_children) for b in range(B)])
    tokens = np.stack([_rng(cfg.seed, _TID_TOKENS, b).integers(0, cfg.vocab, size=T).astype(np.int32)
                       for b in range(B)])
    if cfg.p_accept_range is None:
        p = np.full(B, cfg.p_accept, dtype=np.float64)
    else:
        lo, hi = cfg.p_accept_range
        p = _rng(cfg.seed, _TID_P).uniform(lo, hi, size=B)
    d = cfg.head_dim
    if q_unit_variance:
        q_scale, sm_scale = 1.0, 1.0 / float(np.sqrt(d))
    else:
        q_scale, sm_scale = 1.0 / float(np.sqrt(d)), 1.0
    return StepInputs(cfg, kv_len, kv_start, cap, total, parent, tokens, p, sm_scale, q_scale)


def custom_config(name: str, *, batch=1, n_layers=1, n_msa_layers=1, n_heads=2, head_dim=64,
                  prefix_len=64, prefix_len_range=None, n_nodes=6, max_depth=2, gamma=3, vocab=512,
                  p_accept=0.6, p_accept_range=None, tree_kind="uniform_parent", max_children=4,
                  config_id=100, k_ramp=0.0) -> StepConfig:
    """A free-form configuration for tests (edge cases, ragged tails, odd sizes)."""
    return StepConfig(name, config_id, batch, n_layers, n_msa_layers, n_heads, head_dim, prefix_len,
                      prefix_len_range, n_nodes, max_depth, gamma, vocab, p_accept, p_accept_range,
                      tree_kind, max_children, k_ramp)
