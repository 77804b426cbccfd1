"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs.

Attention: max-abs <= 2e-2 and mean-abs <= 2e-3 (bf16 in, fp32 accumulate, bf16 out, unit-variance V).
Verification and compaction: bit-exact."""
import numpy as np
import pytest

from paper_2402_11131_b200 import workloads as W
from parity_util import assert_attention_close, oracle_layer

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cuda():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2402_11131_b200 import api, build
    build.build()
    api.lib()
    from paper_2402_11131_b200.step import DeviceStep
    return api, DeviceStep


def _layers_for(cfg):
    """>= 2 plain layers (when the config has any) and every MSA layer."""
    n_plain = cfg.n_layers - cfg.n_msa_layers
    plain = [0, n_plain - 1] if n_plain >= 2 else list(range(n_plain))
    return plain + list(range(n_plain, cfg.n_layers))


# ---- attention ------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["tiny", "1.3b", "2.7b"])
def test_attention_matches_oracle_all_rows(cuda, oracle, name):
    api, DeviceStep = cuda
    st = W.make_step(W.CONFIGS[name])
    layers = _layers_for(st.cfg)
    dev = DeviceStep(st, layers=layers, with_lse=True)
    dev.run_attention()
    assert api.ss_status(dev.attn_ws) == 0
    for i, layer in enumerate(layers):
        assert_attention_close(oracle, st, st.layer(layer), dev, i, check_lse=True)


def test_attention_7b_full_size(cuda, oracle):
    """Benchmark shape (7B-class): every MSA layer and two plain layers; all heads for a sample of
    nodes, and all rows for a sample of heads."""
    api, DeviceStep = cuda
    st = W.make_step(W.CONFIGS["7b"])
    layers = _layers_for(st.cfg)
    dev = DeviceStep(st, layers=layers)
    dev.run_attention()
    assert api.ss_status(dev.attn_ws) == 0
    rng = np.random.default_rng(0)
    for i, layer in enumerate(layers):
        ly = st.layer(layer)
        sel = np.zeros(st.cfg.n_nodes, dtype=np.uint8)
        sel[rng.choice(st.cfg.n_nodes, 8, replace=False)] = 1
        sel[[0, st.cfg.n_nodes - 1]] = 1
        assert_attention_close(oracle, st, ly, dev, i, node_sel=sel)
        h0 = int(rng.integers(0, st.cfg.n_heads - 2))
        assert_attention_close(oracle, st, ly, dev, i, heads=(h0, h0 + 2))


def test_attention_ragged_batch_sampled(cuda, oracle):
    """Ragged 16-sequence 7B-class batch: one plain and one MSA layer, sampled (sequence, node) rows."""
    api, DeviceStep = cuda
    st = W.make_step(W.CONFIGS["7b_ragged16"])
    layers = [0, st.cfg.n_layers - 1]
    dev = DeviceStep(st, layers=layers)
    dev.run_attention()
    assert api.ss_status(dev.attn_ws) == 0
    rng = np.random.default_rng(1)
    for i, layer in enumerate(layers):
        ly = st.layer(layer)
        sel = np.zeros(st.cfg.n_nodes, dtype=np.uint8)
        sel[rng.choice(st.cfg.n_nodes, 4, replace=False)] = 1
        seqs = [0, 15, int(np.argmin(st.kv_len)), int(np.argmax(st.kv_len))]
        assert_attention_close(oracle, st, ly, dev, i, seqs=seqs, node_sel=sel)


EDGE_CASES = {
    # name: dict(config kwargs)
    "no_prefix": dict(prefix_len=0, n_nodes=9, gamma=3, max_depth=3),
    "single_node": dict(prefix_len=50, n_nodes=1, gamma=4, max_depth=1),
    "single_node_no_prefix_no_streams": dict(prefix_len=0, n_nodes=1, gamma=0, max_depth=1),
    "ragged_tail_d64": dict(prefix_len=77, n_nodes=11, gamma=2, max_depth=4),
    "ragged_tail_d128": dict(prefix_len=333, n_nodes=64, gamma=4, max_depth=5, head_dim=128, n_heads=3,
                             tree_kind="topk_growth"),
    "d80_ragged": dict(prefix_len=1001, n_nodes=17, gamma=1, max_depth=4, head_dim=80, n_heads=5),
    "chain_63_deep": dict(prefix_len=130, n_nodes=64, gamma=1, max_depth=63, tree_kind="chain"),
    "gamma0_msa_layer": dict(prefix_len=200, n_nodes=20, gamma=0, max_depth=3),
    "batch_ragged_small": dict(batch=5, prefix_len_range=(0, 300), n_nodes=13, gamma=3, max_depth=3, n_heads=4),
    "many_pairs_short": dict(batch=24, prefix_len_range=(1, 40), n_nodes=8, gamma=2, max_depth=3, n_heads=8),
    "long_prefix_two_heads": dict(prefix_len=9000, n_nodes=16, gamma=3, max_depth=3, n_heads=2, head_dim=128),
    # the largest score of every row grows by far more than 2^8 from tile to tile: the running maximum is raised,
    # and the accumulator rescaled, on every tile (<= 64 rows per head, and three row blocks of 128)
    "growing_scores_small_head": dict(prefix_len=1500, n_nodes=12, gamma=0, max_depth=3, n_heads=40, head_dim=128,
                                      k_ramp=0.05),
    "growing_scores_row_blocks": dict(prefix_len=1500, n_nodes=64, gamma=4, max_depth=5, n_heads=40, head_dim=128,
                                      tree_kind="topk_growth", k_ramp=0.05),
    # later keys exceed the first tile's scores by hundreds of nats: unsplit 128-row blocks give up the reference they
    # share (the row maximum of the first tile) and run their tiles again with a running maximum
    "steep_scores_row_blocks": dict(prefix_len=700, n_nodes=64, gamma=4, max_depth=5, n_heads=40, head_dim=128,
                                    tree_kind="topk_growth", k_ramp=0.5),
    # the same in a ragged batch (sequences dispatched longest first) and at head_dim 64 with two row blocks
    "steep_scores_ragged_batch": dict(batch=3, prefix_len_range=(300, 1500), n_nodes=40, gamma=3, max_depth=4, n_heads=16,
                                      head_dim=128, tree_kind="topk_growth", k_ramp=0.3),
    "steep_scores_d64": dict(prefix_len=2000, n_nodes=64, gamma=2, max_depth=5, n_heads=48, head_dim=64,
                             tree_kind="topk_growth", k_ramp=0.4),
    "growing_scores_split_keys": dict(prefix_len=3000, n_nodes=40, gamma=2, max_depth=4, n_heads=3, head_dim=64,
                                      k_ramp=0.03),
}


@pytest.mark.parametrize("case", list(EDGE_CASES))
def test_attention_edge_cases(cuda, oracle, case):
    api, DeviceStep = cuda
    kw = dict(EDGE_CASES[case])
    cfg = W.custom_config(case, n_layers=2, n_msa_layers=1, config_id=500 + list(EDGE_CASES).index(case), **kw)
    st = W.make_step(cfg, q_unit_variance=(case in ("ragged_tail_d64", "d80_ragged")))
    dev = DeviceStep(st, with_lse=True)
    dev.run_attention()
    assert api.ss_status(dev.attn_ws) == 0
    started_over = int(dev.attn_ws.view(torch.int32)[2])
    if case.startswith("steep_scores"):
        assert started_over > 0                              # the multi-stream layer's blocks did start over
    for i in range(2):
        assert_attention_close(oracle, st, st.layer(i), dev, i, check_lse=True)


def test_attention_per_sequence_tree_sizes(cuda, oracle):
    """Sequences of one batch carry trees of different sizes T_b <= max_nodes."""
    api, DeviceStep = cuda
    cfg = W.custom_config("var_T", batch=4, n_layers=2, n_msa_layers=1, prefix_len_range=(20, 150), n_nodes=12,
                          gamma=3, max_depth=3, n_heads=3, config_id=600)
    st = W.make_step(cfg)
    st.n_nodes_b = np.array([12, 1, 7, 5], dtype=np.int32)
    dev = DeviceStep(st)
    for t in dev.o_main + [o for o in dev.o_spec if o is not None]:
        t.fill_(7.0)                                        # canary for rows of nodes >= T_b
    dev.run_attention()
    assert api.ss_status(dev.attn_ws) == 0
    for i in range(2):
        assert_attention_close(oracle, st, st.layer(i), dev, i)
        for b in range(4):
            assert (dev.o_main[i][b, st.nodes(b):] == 7.0).all()
    assert (dev.o_spec[1][1, 1:] == 7.0).all()


def test_attention_is_deterministic_and_leaves_inputs_alone(cuda):
    api, DeviceStep = cuda
    st = W.make_step(W.CONFIGS["1.3b"])
    layers = [0, 23]
    dev = DeviceStep(st, layers=layers)
    k0, v0 = dev.k_all.clone(), dev.v_all.clone()
    dev.run_attention()
    first = [dev.o_main[i].clone() for i in range(2)] + [dev.o_spec[1].clone()]
    for _ in range(3):
        dev.run_attention()
    torch.cuda.synchronize()
    again = [dev.o_main[i] for i in range(2)] + [dev.o_spec[1]]
    for a, b in zip(first, again):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert torch.equal(k0.view(torch.int16), dev.k_all.view(torch.int16))
    assert torch.equal(v0.view(torch.int16), dev.v_all.view(torch.int16))


def test_attention_ignores_slots_past_the_tree(cuda):
    """Poison (NaN) in slots >= L+T and in the rows of other sequences' unused capacity is never read."""
    api, DeviceStep = cuda
    cfg = W.custom_config("poison", batch=3, n_layers=1, n_msa_layers=1, prefix_len_range=(10, 90), n_nodes=10,
                          gamma=2, max_depth=3, n_heads=2, config_id=601)
    st = W.make_step(cfg)
    dev = DeviceStep(st)
    dev.run_attention()
    ref = [dev.o_main[0].clone(), dev.o_spec[0].clone()]
    for b in range(3):
        lo = int(st.kv_start[b]) + int(st.kv_len[b]) + cfg.n_nodes
        hi = int(st.kv_start[b]) + int(st.kv_capacity[b])
        dev.k_all[0, lo:hi] = float("nan")
        dev.v_all[0, lo:hi] = float("nan")
    dev.run_attention()
    torch.cuda.synchronize()
    assert torch.equal(ref[0].view(torch.int16), dev.o_main[0].view(torch.int16))
    assert torch.equal(ref[1].view(torch.int16), dev.o_spec[0].view(torch.int16))


def test_attention_reports_a_sequence_over_capacity(cuda, oracle):
    api, DeviceStep = cuda
    cfg = W.custom_config("overcap", batch=3, n_layers=1, n_msa_layers=1, prefix_len_range=(30, 60), n_nodes=6,
                          gamma=1, max_depth=2, n_heads=2, config_id=602)
    st = W.make_step(cfg)
    dev = DeviceStep(st)
    dev.kv_capacity[1] = int(st.kv_len[1]) + 5              # one slot short of L + T
    dev.o_main[0].fill_(3.0)
    dev.run_attention()
    assert api.ss_status(dev.attn_ws) == api.SS_ERR_CAPACITY
    assert api.ss_status(dev.attn_ws) == 0                  # reading clears it
    assert (dev.o_main[0][1] == 3.0).all()                  # the offending sequence was skipped
    assert_attention_close(oracle, st, st.layer(0), dev, 0, seqs=[0, 2])


def test_attention_strided_cache_views(cuda, oracle):
    """K/V given as a [slots][H][d] view of a [slots][2][H][d+pad] buffer (non-contiguous strides)."""
    api, DeviceStep = cuda
    cfg = W.custom_config("strided", n_layers=1, n_msa_layers=1, prefix_len=150, n_nodes=9, gamma=2, max_depth=3,
                          n_heads=3, head_dim=64, config_id=603)
    st = W.make_step(cfg)
    dev = DeviceStep(st)
    big = torch.zeros((st.total_slots, 2, 3, 64 + 8), dtype=torch.bfloat16, device="cuda")
    big[:, 0, :, :64] = dev.k_all[0]
    big[:, 1, :, :64] = dev.v_all[0]
    p = api.make_attn_params(q_main=dev.q_main[0], o_main=dev.o_main[0], k_cache=big[:, 0, :, :64],
                             v_cache=big[:, 1, :, :64], kv_start=dev.kv_start, kv_len=dev.kv_len, trees=dev.trees,
                             gamma=2, sm_scale=st.sm_scale, q_spec=dev.q_spec[0], k_spec=dev.k_spec[0],
                             v_spec=dev.v_spec[0], o_spec=dev.o_spec[0], workspace=dev.attn_ws)
    api.ss_msa_attention(p)
    assert api.ss_status(dev.attn_ws) == 0
    assert_attention_close(oracle, st, st.layer(0), dev, 0)


def test_attention_without_the_prefix_promise_gives_the_same_bits(cuda, oracle):
    """flags = 0 (nothing read before the dependency wait) and SS_ATTN_PREFIX_STABLE differ only in
    when the prefix tiles are requested: the outputs are bit-identical, for every kernel variant
    (<= 64 rows, one block of 65..128 rows, several blocks)."""
    api, DeviceStep = cuda
    cases = [dict(prefix_len=700, n_nodes=16, gamma=3, max_depth=3, n_heads=8, head_dim=128),      # 64 rows
             dict(prefix_len=500, n_nodes=32, gamma=3, max_depth=4, n_heads=6, head_dim=64),       # 128 rows
             dict(prefix_len=400, n_nodes=40, gamma=4, max_depth=4, n_heads=5, head_dim=80)]       # 200 rows
    for k, kw in enumerate(cases):
        cfg = W.custom_config("promise%d" % k, n_layers=2, n_msa_layers=1, config_id=640 + k, **kw)
        st = W.make_step(cfg)
        outs = []
        for promise in (False, True):
            dev = DeviceStep(st, prefix_stable=promise)
            for _ in range(2):                                  # back to back: the second call overlaps the first
                dev.run_attention()
            assert api.ss_status(dev.attn_ws) == 0
            outs.append([dev.o_main[0].clone(), dev.o_main[1].clone(), dev.o_spec[1].clone()])
            if promise:
                for i in range(2):
                    assert_attention_close(oracle, st, st.layer(i), dev, i)
        for x, y in zip(*outs):
            assert torch.equal(x.view(torch.int16), y.view(torch.int16))


@pytest.mark.parametrize("n_heads,expect_split", [(1, 8), (3, 8), (20, 4), (40, 2), (100, 1)])
def test_attention_every_split_factor(cuda, oracle, n_heads, expect_split):
    """The number of CTAs that share a row block's keys follows the head count (8, 4, 2, 1): every merge
    path, including CTAs that get no keys at all (8 CTAs, 5 key units).  The layers of a step share one
    workspace and may have different split factors and row counts (6 or 40 nodes, with and without stream
    rows); every call must leave the partial rows' area zero, which the second pass relies on."""
    api, DeviceStep = cuda
    for k, (L, T, g) in enumerate([(70, 6, 1), (900, 40, 4)]):
        cfg = W.custom_config("split%d_%d" % (n_heads, k), n_layers=2, n_msa_layers=1, prefix_len=L, n_nodes=T,
                              gamma=g, max_depth=3, n_heads=n_heads, head_dim=64, config_id=660 + k)
        st = W.make_step(cfg)
        dev = DeviceStep(st, with_lse=True)
        dev.run_attention()
        dev.run_attention()
        assert api.ss_status(dev.attn_ws) == 0
        assert int(dev.attn_ws.view(torch.int32)[2:].abs().max()) == 0
        for i in range(2):
            assert_attention_close(oracle, st, st.layer(i), dev, i, check_lse=True)


# ---- verification ---------------------------------------------------------------------------------
def _verify_and_compare(api, dev, st, oracle):
    dev.run_verify()
    assert api.ss_status(dev.verify_ws) == 0
    lg = st.logits()
    lens = dev.accept_len.cpu().numpy()
    for b in range(st.cfg.batch):
        T = st.nodes(b)
        r = oracle.tree_verify(lg[b][:T], st.draft_tokens[b][:T], st.parent[b][:T], path_cap=api.SS_PATH_STRIDE)
        assert int(lens[b]) == r["accept_len"]
        assert np.array_equal(dev.accept_path[b].cpu().numpy(), r["path"])
        assert int(dev.last_node[b]) == r["last_node"]
        assert int(dev.bonus_token[b]) == r["bonus_token"]
        assert np.array_equal(dev.node_argmax[b][:T].cpu().numpy(), r["node_argmax"])
    return lens


@pytest.mark.parametrize("name", list(W.CONFIGS))
def test_verify_is_bit_exact(cuda, oracle, name):
    api, DeviceStep = cuda
    st = W.make_step(W.CONFIGS[name])
    dev = DeviceStep(st, layers=[])
    lens = _verify_and_compare(api, dev, st, oracle)
    assert lens.min() >= 1 and lens.max() <= st.cfg.max_depth + 1
    lens2 = _verify_and_compare(api, dev, st, oracle)        # the workspace is left ready for reuse
    assert np.array_equal(lens, lens2)


@pytest.mark.parametrize("vocab", [1, 3, 127, 4096, 4097, 50001])
def test_verify_odd_vocab_sizes_and_ties(cuda, oracle, vocab):
    api, DeviceStep = cuda
    cfg = W.custom_config("v%d" % vocab, batch=3, n_layers=1, prefix_len=4, n_nodes=10, gamma=0, max_depth=4,
                          vocab=vocab, p_accept=0.8, config_id=700 + vocab % 97)
    st = W.make_step(cfg)
    lg = st.logits()
    # heavy ties: quantise the logits so that many entries share the maximum
    st._logits = np.round(lg * 2).astype(np.float32) / 2
    st.draft_tokens = np.minimum(st.draft_tokens, vocab - 1).astype(np.int32)
    dev = DeviceStep(st, layers=[])
    _verify_and_compare(api, dev, st, oracle)


def test_verify_duplicate_siblings_and_all_correct(cuda, oracle):
    api, DeviceStep = cuda
    cfg = W.custom_config("dups", batch=2, n_layers=1, prefix_len=4, n_nodes=12, gamma=0, max_depth=4, vocab=64,
                          p_accept=1.0, config_id=710)
    st = W.make_step(cfg)
    st.draft_tokens[0, :] = 5                                  # every sibling carries the same token
    dev = DeviceStep(st, layers=[])
    lens = _verify_and_compare(api, dev, st, oracle)
    assert lens[0] >= 2


# ---- compaction -----------------------------------------------------------------------------------
def _compact_and_compare(api, dev, st, oracle, host_layers):
    """host_layers: list of LayerInputs matching dev.layers (their slabs are the 'before' state)."""
    dev.run_verify()
    dev.run_compact()
    torch.cuda.synchronize()
    lens = dev.accept_len.cpu().numpy()
    paths = dev.accept_path.cpu().numpy()
    k_after = api.bf16_to_host_bits(dev.k_all)
    v_after = api.bf16_to_host_bits(dev.v_all)
    k_before = np.stack([ly.k_cache for ly in host_layers])
    v_before = np.stack([ly.v_cache for ly in host_layers])
    new_len = dev.kv_len_out.cpu().numpy()
    for b in range(st.cfg.batch):
        s0, cap, L = int(st.kv_start[b]), int(st.kv_capacity[b]), int(st.kv_len[b])
        ke, ve, nl = oracle.kv_compact(k_before[:, s0:s0 + cap], v_before[:, s0:s0 + cap], L, int(lens[b]), paths[b])
        assert nl == int(new_len[b]) == L + int(lens[b])
        assert np.array_equal(k_after[:, s0:s0 + nl], ke[:, :nl])
        assert np.array_equal(v_after[:, s0:s0 + nl], ve[:, :nl])
        assert np.array_equal(k_after[:, s0:s0 + L], k_before[:, s0:s0 + L])      # prefix bit-unchanged
    return lens


@pytest.mark.parametrize("name,layers", [("tiny", None), ("1.3b", None), ("2.7b", None), ("7b", None),
                                         ("7b_ragged16", [0, 9, 30, 31])])
def test_compaction_is_bit_exact(cuda, oracle, name, layers):
    api, DeviceStep = cuda
    st = W.make_step(W.CONFIGS[name])
    dev = DeviceStep(st, layers=layers)
    host = [st.layer(l) for l in dev.layers]
    lens = _compact_and_compare(api, dev, st, oracle, host)
    assert lens.max() >= 2          # the forced acceptances make some path longer than the root


def test_compaction_long_path_and_aliased_lengths(cuda, oracle):
    """Two interleaved chains (0-1-3-5-..-63 and 0-2-4-..-62) with every first child accepted: the
    accepted path has 33 nodes and skips every other slot, so a thread moves several batches of
    rows; kv_len_out aliases kv_len_in."""
    api, DeviceStep = cuda
    cfg = W.custom_config("deep", batch=2, n_layers=3, n_msa_layers=1, prefix_len=37, n_nodes=64, gamma=1,
                          max_depth=63, vocab=97, p_accept=1.0, n_heads=2, head_dim=80, tree_kind="chain",
                          config_id=720)
    st = W.make_step(cfg)
    st.parent[:] = np.array([-1, 0] + list(range(62)), dtype=np.int32)
    st.draft_tokens[:] = np.arange(64, dtype=np.int32)[None, :] % 97       # distinct sibling tokens
    dev = DeviceStep(st)
    host = [st.layer(l) for l in dev.layers]
    dev.kv_len_out = dev.kv_len                                  # alias
    lens = _compact_and_compare(api, dev, st, oracle, host)
    assert list(lens) == [33, 33]
    assert list(dev.accept_path[0, :4].cpu().numpy()) == [0, 1, 3, 5]


def test_two_steps_in_a_row_with_aliased_lengths(cuda, oracle):
    """A second step on the cache that the first step's compaction left behind: the lengths are updated in
    place (kv_len_out aliases kv_len), the accepted nodes have become prefix, new tree nodes are appended
    after them.  The first attention call after a compaction may not promise a stable prefix, so the step
    runs with flags = 0; its attention must match the oracle on the compacted cache and the new lengths."""
    api, DeviceStep = cuda
    cfg = W.custom_config("twostep", batch=2, n_layers=2, n_msa_layers=1, prefix_len=37, n_nodes=10, gamma=2,
                          max_depth=3, vocab=97, p_accept=0.9, n_heads=3, head_dim=64, config_id=730)
    st = W.make_step(cfg)
    dev = DeviceStep(st, prefix_stable=False)
    host = [st.layer(l) for l in dev.layers]
    dev.kv_len_out = dev.kv_len                                  # the compaction updates the lengths in place
    dev.run_attention()
    lens = _compact_and_compare(api, dev, st, oracle, host)
    assert api.ss_status(dev.attn_ws) == 0
    k_now = api.bf16_to_host_bits(dev.k_all)
    v_now = api.bf16_to_host_bits(dev.v_all)
    rng = np.random.default_rng(731)
    T, H, d = cfg.n_nodes, cfg.n_heads, cfg.head_dim
    for b in range(cfg.batch):
        s0, cap = int(st.kv_start[b]), int(st.kv_capacity[b])
        L2 = int(st.kv_len[b]) + int(lens[b])
        assert L2 + T <= cap
        for arr, dev_arr in ((k_now, dev.k_all), (v_now, dev.v_all)):         # this step's tree nodes, after the new prefix
            rows = W.f32_to_bf16_bits(rng.standard_normal((len(dev.layers), T, H, d)).astype(np.float32))
            arr[:, s0 + L2:s0 + L2 + T] = rows
            dev_arr[:, s0 + L2:s0 + L2 + T].copy_(api.bf16_to_device(rows))
        st.kv_len[b] = L2
    assert list(dev.kv_len.cpu().numpy()) == list(st.kv_len)
    dev.run_attention()
    assert api.ss_status(dev.attn_ws) == 0
    for i, ly in enumerate(host):
        now = W.LayerInputs(ly.layer, ly.is_msa, ly.q_main, ly.q_spec, ly.k_spec, ly.v_spec, k_now[i], v_now[i])
        assert_attention_close(oracle, st, now, dev, i)
