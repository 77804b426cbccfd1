"""The seeded input generator: shapes, determinism, tree constraints, bf16 round trip."""
import numpy as np
import pytest

from paper_2402_11131_b200 import workloads as W


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, -2.5, 3.140625, 1.00390625, 1.01171875, 0.0], dtype=np.float32)
    b = W.f32_to_bf16_bits(x)
    back = W.bf16_bits_to_f64(b)
    # 1.00390625 = 1 + 2^-8 is a tie -> rounds to even (1.0); 1.01171875 = 1 + 3*2^-8 -> 1 + 2^-6
    np.testing.assert_array_equal(back, [1.0, -2.5, 3.140625, 1.0, 1.015625, 0.0])
    torch = pytest.importorskip("torch")
    y = np.random.default_rng(0).standard_normal(4096).astype(np.float32)
    ref = torch.from_numpy(y).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(W.f32_to_bf16_bits(y), ref)


@pytest.mark.parametrize("name", list(W.CONFIGS))
def test_structure_of_named_configs(name):
    cfg = W.CONFIGS[name]
    st = W.make_step(cfg)
    assert st.parent.shape == (cfg.batch, cfg.n_nodes)
    for b in range(cfg.batch):
        par = st.parent[b]
        assert par[0] == -1 and all(0 <= par[i] < i for i in range(1, cfg.n_nodes))
        depth = np.zeros(cfg.n_nodes, dtype=int)
        for i in range(1, cfg.n_nodes):
            depth[i] = depth[par[i]] + 1
        assert depth.max() <= cfg.max_depth
        if cfg.tree_kind == "topk_growth":
            assert np.bincount(par[1:], minlength=cfg.n_nodes).max() <= 4
        assert st.kv_capacity[b] >= st.kv_len[b] + cfg.n_nodes
    if cfg.prefix_len_range:
        assert st.kv_len.min() >= 512 and st.kv_len.max() <= 4096 and len(set(st.kv_len)) > 1
    assert st.kv_start[0] == 0 and np.all(np.diff(st.kv_start) == st.kv_capacity[:-1])
    st2 = W.make_step(cfg)
    assert np.array_equal(st.parent, st2.parent) and np.array_equal(st.draft_tokens, st2.draft_tokens)


def test_layer_tensors_are_deterministic_and_unit_variance():
    st = W.make_step(W.CONFIGS["1.3b"])
    a, b = st.layer(21), st.layer(21)
    assert a.is_msa and np.array_equal(a.k_cache, b.k_cache) and np.array_equal(a.q_spec, b.q_spec)
    assert not st.layer(3).is_msa and st.layer(3).q_spec is None
    k = W.bf16_bits_to_f64(a.k_cache)
    assert abs(k.std() - 1.0) < 0.01 and abs(k.mean()) < 0.01
    q = W.bf16_bits_to_f64(a.q_main)
    assert abs(q.std() * np.sqrt(64) - 1.0) < 0.02
    assert a.q_spec.shape == (1, 16, 3, 32, 64) and a.k_cache.shape == (st.total_slots, 32, 64)


def test_logits_force_acceptance():
    st = W.make_step(W.CONFIGS["tiny"])
    lg = st.logits()
    assert lg.shape == (1, 6, 512) and lg.dtype == np.float32
    forced = (lg == 16.0)
    assert forced.sum(axis=2).max() <= 1
    for u in np.nonzero(forced.any(axis=2)[0])[0]:
        tok = int(np.argmax(lg[0, u]))
        assert tok in [int(st.draft_tokens[0, c]) for c in range(6) if st.parent[0, c] == u]
