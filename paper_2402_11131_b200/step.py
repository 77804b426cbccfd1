"""Device-resident buffers of one decode step and the sequence of C-ABI calls that runs it.

Buffer management and argument marshalling only: attention, verification and compaction all run in
the CUDA library (see api.py).  Used by the tests, the smoke check and the benchmark.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

from . import api
from .workloads import StepInputs


class DeviceStep:
    """All inputs of one step on the device, with per-layer ss_attn_params prepared once.

    layers          layer indices of the workload to materialise (default: all of them)
    prefix_stable   pass SS_ATTN_PREFIX_STABLE to the attention calls (true for every use in this repo:
                    what runs before an attention call never writes the cached prefix)
    distinct_slabs  if set, layer l draws its KV slab from random substream (l % distinct_slabs):
                    every layer still owns its own device memory, only the host generation is shared
    """

    def __init__(self, st: StepInputs, layers: Optional[List[int]] = None, distinct_slabs: Optional[int] = None,
                 device: str = "cuda", with_lse: bool = False, pinned_host: bool = False, prefix_stable: bool = True):
        api.lib()
        c = st.cfg
        self.st, self.cfg, self.device = st, c, device
        # SS_ATTN_PREFIX_STABLE: nothing in flight before an attention call writes the prefix, lengths or trees
        self.prefix_stable = prefix_stable
        self.layers = list(range(c.n_layers)) if layers is None else list(layers)
        nl = len(self.layers)
        B, T, H, d, g = c.batch, c.n_nodes, c.n_heads, c.head_dim, c.gamma
        dev = device

        self.descs = [api.ss_tree_build(st.parent[b][:st.nodes(b)], g) for b in range(B)]
        self.trees = api.trees_to_device(self.descs, dev)
        self.kv_start = torch.from_numpy(st.kv_start.astype(np.int64)).to(dev)
        self.kv_len = torch.from_numpy(st.kv_len.astype(np.int32)).to(dev)
        self.kv_capacity = torch.from_numpy(st.kv_capacity.astype(np.int32)).to(dev)
        self.kv_len_out = torch.zeros(B, dtype=torch.int32, device=dev)

        self.k_all = torch.empty((nl, st.total_slots, H, d), dtype=torch.bfloat16, device=dev)
        self.v_all = torch.empty_like(self.k_all)
        # the main-stream queries of all layers lie in one allocation, so that a host copy can fill several layers at once
        self.q_main_all = torch.empty((nl, B, T, H, d), dtype=torch.bfloat16, device=dev)
        self.q_main, self.o_main, self.q_spec, self.k_spec, self.v_spec, self.o_spec = [], [], [], [], [], []
        self.lse_main, self.lse_spec = [], []
        self.is_msa: List[bool] = []
        self.host_inputs: List[Dict[str, torch.Tensor]] = []   # pinned host copies (end-to-end timing)
        slab_cache: Dict[int, tuple] = {}
        for i, layer in enumerate(self.layers):
            seed = layer if distinct_slabs is None else layer % distinct_slabs
            ly = st.layer(layer, slab_seed=seed, with_slab=seed not in slab_cache)
            if ly.k_cache is None:                      # slab already on the device: copy it there
                self.k_all[i].copy_(slab_cache[seed][0])
                self.v_all[i].copy_(slab_cache[seed][1])
            else:
                self.k_all[i].copy_(api.bf16_to_device(ly.k_cache, dev))
                self.v_all[i].copy_(api.bf16_to_device(ly.v_cache, dev))
                if distinct_slabs is not None:
                    slab_cache[seed] = (self.k_all[i], self.v_all[i])
            self.is_msa.append(ly.is_msa)
            self.q_main_all[i].copy_(api.bf16_to_device(ly.q_main, dev))
            self.q_main.append(self.q_main_all[i])
            self.o_main.append(torch.zeros((B, T, H, d), dtype=torch.bfloat16, device=dev))
            self.lse_main.append(torch.zeros((B, T, H), dtype=torch.float32, device=dev) if with_lse else None)
            if ly.is_msa:
                self.q_spec.append(api.bf16_to_device(ly.q_spec, dev))
                self.k_spec.append(api.bf16_to_device(ly.k_spec, dev))
                self.v_spec.append(api.bf16_to_device(ly.v_spec, dev))
                self.o_spec.append(torch.zeros((B, T, g, H, d), dtype=torch.bfloat16, device=dev))
                self.lse_spec.append(torch.zeros((B, T, g, H), dtype=torch.float32, device=dev) if with_lse else None)
            else:
                for lst in (self.q_spec, self.k_spec, self.v_spec, self.o_spec, self.lse_spec):
                    lst.append(None)
            if pinned_host:
                h = {}
                if ly.is_msa:
                    h.update(q_spec=self.q_spec[i].cpu().pin_memory(), k_spec=self.k_spec[i].cpu().pin_memory(),
                             v_spec=self.v_spec[i].cpu().pin_memory())
                self.host_inputs.append(h)

        self.host_q_main_all = self.q_main_all.cpu().pin_memory() if pinned_host else None
        if pinned_host:
            for i in range(nl):
                self.host_inputs[i]["q_main"] = self.host_q_main_all[i]

        # attention workspace: sized for the largest layer, shared by all (calls are stream-ordered)
        ws_bytes = 0
        for i in range(nl):
            ws_bytes = max(ws_bytes, api.ss_msa_attention_workspace_bytes(self._params(i, None)))
        self.attn_ws = api.workspace(ws_bytes, dev)
        self.params = [self._params(i, self.attn_ws) for i in range(nl)]

        # verification
        self.logits = torch.from_numpy(st.logits()).to(dev)
        self.tokens = torch.from_numpy(st.draft_tokens.astype(np.int32)).to(dev)
        self.accept_len = torch.zeros(B, dtype=torch.int32, device=dev)
        self.accept_path = torch.zeros((B, api.SS_PATH_STRIDE), dtype=torch.int32, device=dev)
        self.last_node = torch.zeros(B, dtype=torch.int32, device=dev)
        self.bonus_token = torch.zeros(B, dtype=torch.int32, device=dev)
        self.node_argmax = torch.zeros((B, T), dtype=torch.int32, device=dev)
        self.verify_ws = api.workspace(api.ss_tree_verify_workspace_bytes(B, T, c.vocab), dev)
        self.layout = api.make_cache_layout(self.k_all)
        torch.cuda.synchronize()

    def _params(self, i: int, ws) -> api.AttnParams:
        msa = self.is_msa[i]
        return api.make_attn_params(
            q_main=self.q_main[i], o_main=self.o_main[i], k_cache=self.k_all[i], v_cache=self.v_all[i],
            kv_start=self.kv_start, kv_len=self.kv_len, kv_capacity=self.kv_capacity, trees=self.trees,
            gamma=self.cfg.gamma if msa else 0, sm_scale=self.st.sm_scale,
            q_spec=self.q_spec[i], k_spec=self.k_spec[i], v_spec=self.v_spec[i], o_spec=self.o_spec[i],
            lse_main=self.lse_main[i], lse_spec=self.lse_spec[i], workspace=ws, prefix_stable=self.prefix_stable)

    # ---- the hot path -------------------------------------------------------------------------
    def run_attention(self, stream=None, only: Optional[List[int]] = None) -> int:
        idx = range(len(self.layers)) if only is None else only
        n = 0
        for i in idx:
            api.ss_msa_attention(self.params[i], stream)
            n += api.LAUNCHES_PER_CALL["ss_msa_attention"]
        return n

    def run_verify(self, stream=None) -> int:
        api.ss_tree_verify(self.logits, self.tokens, self.trees, self.accept_len, self.accept_path, self.last_node,
                           self.bonus_token, self.node_argmax, self.verify_ws, stream)
        return api.LAUNCHES_PER_CALL["ss_tree_verify"]

    def run_compact(self, stream=None) -> int:
        api.ss_kv_compact(self.k_all, self.v_all, self.layout, self.kv_start, self.kv_len, self.accept_len,
                          self.accept_path, self.kv_len_out, stream)
        return api.LAUNCHES_PER_CALL["ss_kv_compact"]

    def run_step(self, stream=None) -> int:
        """One pass of the whole hot path: every layer's attention, verification, compaction.
        Returns the number of kernels enqueued."""
        return self.run_attention(stream) + self.run_verify(stream) + self.run_compact(stream)

    # ---- algorithmic traffic (bytes each quantity must cross HBM once) -----------------------
    def attention_bytes(self, i: int) -> int:
        c = self.cfg
        g = c.gamma if self.is_msa[i] else 0
        H, d, T = c.n_heads, c.head_dim, c.n_nodes
        total = 0
        for b in range(c.batch):
            L, T = int(self.st.kv_len[b]), self.st.nodes(b)
            M = T * (1 + g)
            total += 4 * L * H * d + 4 * T * H * d + 4 * T * g * H * d + 4 * M * H * d
        return total

    def attention_flops(self, i: int) -> int:
        c = self.cfg
        g = c.gamma if self.is_msa[i] else 0
        H, d, T = c.n_heads, c.head_dim, c.n_nodes
        total = 0
        for b in range(c.batch):
            L, T = int(self.st.kv_len[b]), self.st.nodes(b)
            depth = np.array(self.descs[b].depth[:T])
            keys = int(((L + depth + 1) * (1 + g)).sum()) + T * g * (g + 1) // 2
            total += 4 * d * H * keys
        return total

    def verify_bytes(self) -> int:
        c = self.cfg
        return 4 * c.batch * c.n_nodes * c.vocab

    def compact_bytes(self, accept_len: np.ndarray) -> int:
        c = self.cfg
        return int(2 * 2 * int(accept_len.sum()) * c.n_heads * c.head_dim * 2 * len(self.layers))
