"""GPU checks that the parity tolerance alone would not make: which keys a row can see (one key at a time, at
long prefixes, across the row-block boundaries), the arg-max on special values, and the time-out path of a
bounded device wait."""
import numpy as np
import pytest

from paper_2402_11131_b200 import workloads as W
from parity_util import assert_attention_close

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

ONE, FORTY = 0x3F80, 0x4220            # bf16 bit patterns of 1.0 and 40.0


@pytest.fixture(scope="module")
def cuda():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2402_11131_b200 import api, build
    build.build()
    api.lib()
    from paper_2402_11131_b200.step import DeviceStep
    return api, DeviceStep


def _membership_sweep(api, DeviceStep, oracle, cfg, keys):
    """One key at a time gets a score 40 above the rest: a row's output is that key's V row if and only if
    the row sees the key (Eq. 1 / Eq. 2 with the mask of App. A), which moves the output by O(1) -- far outside
    the parity tolerance -- wherever the device and the oracle disagree on visibility."""
    st = W.make_step(cfg)
    layer = cfg.n_layers - 1
    dev = DeviceStep(st, layers=[layer])
    ly = st.layer(layer)
    L, T, g = int(st.kv_len[0]), cfg.n_nodes, cfg.gamma
    ly.q_main[..., 0] = ONE                                  # every query has component 0 equal to 1 ...
    ly.q_spec[..., 0] = ONE
    ly.k_cache[..., 0] = 0                                   # ... and no key has a component 0 ...
    ly.k_spec[..., 0] = 0
    dev.q_main[0].copy_(api.bf16_to_device(ly.q_main))
    dev.q_spec[0].copy_(api.bf16_to_device(ly.q_spec))
    for kind, idx in keys:
        k_cache, k_spec = ly.k_cache.copy(), ly.k_spec.copy()
        if kind == "prefix":
            k_cache[idx, :, 0] = FORTY                       # ... except the one under test
        elif kind == "node":
            k_cache[L + idx, :, 0] = FORTY
        else:
            node, j = idx
            k_spec[0, node, j - 1, :, 0] = FORTY
        dev.k_all[0].copy_(api.bf16_to_device(k_cache))
        dev.k_spec[0].copy_(api.bf16_to_device(k_spec))
        dev.run_attention()
        assert api.ss_status(dev.attn_ws) == 0
        probe = W.LayerInputs(layer, True, ly.q_main, ly.q_spec, k_spec, ly.v_spec, k_cache, ly.v_cache)
        assert_attention_close(oracle, st, probe, dev, 0)


@pytest.mark.parametrize("L", [2048, 0])
def test_key_visibility_three_row_blocks(cuda, oracle, L):
    """64 nodes x (1 + 4) rows = 320 rows per head: three blocks of 128 rows; the probed nodes sit on both
    sides of the block boundaries (rows 128 and 256 are stream rows of nodes 16 and 48)."""
    api, DeviceStep = cuda
    cfg = W.custom_config("vis3_%d" % L, n_layers=1, n_msa_layers=1, prefix_len=L, n_nodes=64, gamma=4, max_depth=5,
                          n_heads=2, head_dim=128, tree_kind="topk_growth", config_id=800)
    keys = [("node", n) for n in (0, 1, 15, 16, 31, 47, 48, 63)]
    keys += [("stream", (n, j)) for n in (0, 15, 16, 47, 48, 63) for j in (1, 4)]
    if L > 0:
        keys += [("prefix", 7), ("prefix", L - 1)]
    _membership_sweep(api, DeviceStep, oracle, cfg, keys)


@pytest.mark.parametrize("L,heads", [(300, 3), (0, 3), (1100, 40)])
def test_key_visibility_small_heads(cuda, oracle, L, heads):
    """12 nodes x (1 + 4) rows = 60 rows per head (the variant for at most 64 rows), every tree node and the
    streams of a few nodes; 3 heads split the keys 8 ways, 40 heads do not split at all."""
    api, DeviceStep = cuda
    cfg = W.custom_config("vis1_%d_%d" % (L, heads), n_layers=1, n_msa_layers=1, prefix_len=L, n_nodes=12, gamma=4,
                          max_depth=4, n_heads=heads, head_dim=128, tree_kind="topk_growth", config_id=801)
    keys = [("node", n) for n in range(12)] + [("stream", (n, j)) for n in (0, 5, 11) for j in (1, 2, 4)]
    if L > 0:
        keys += [("prefix", 0), ("prefix", L - 1)]
    if heads > 8:
        keys = keys[::3]
    _membership_sweep(api, DeviceStep, oracle, cfg, keys)


def test_verify_special_values(cuda, oracle):
    """NaN first, NaN in the middle, all NaN, -0 / +0, subnormals, -inf: the device takes the same arg-max as the
    oracle (a NaN is never selected while a comparable value exists; IEEE order otherwise)."""
    api, DeviceStep = cuda
    nan, inf = np.float32("nan"), np.float32("inf")
    V = 4100
    rows = np.zeros((7, V), dtype=np.float32)
    rows[0, :] = -1.0; rows[0, 0] = nan; rows[0, [900, 4097]] = 3.0
    rows[1, :] = nan
    rows[2, :] = -0.0; rows[2, 5] = 0.0
    rows[3, :] = 1e-45; rows[3, [77, 4099]] = 3e-45
    rows[4, :] = -inf; rows[4, 4098] = -3e38
    rows[5, :] = 0.5; rows[5, 1::2] = nan
    rows[6, :] = nan; rows[6, 4096] = -inf
    parent = np.array([-1, 0, 1, 2, 3, 4, 5], dtype=np.int32)
    am = [int(oracle.tree_verify(rows[t:t + 1], np.array([0]), np.array([-1]))["bonus_token"]) for t in range(7)]
    assert am == [900, 0, 0, 77, 4098, 0, 4096]
    tok = np.array([0] + am[:-1], dtype=np.int32)             # every draft equals its parent's arg-max: the chain is accepted
    trees = api.trees_to_device([api.ss_tree_build(parent, 0)])
    out = dict(accept_len=torch.zeros(1, dtype=torch.int32, device="cuda"),
               accept_path=torch.zeros((1, 64), dtype=torch.int32, device="cuda"),
               last_node=torch.zeros(1, dtype=torch.int32, device="cuda"),
               bonus_token=torch.zeros(1, dtype=torch.int32, device="cuda"),
               node_argmax=torch.zeros((1, 7), dtype=torch.int32, device="cuda"))
    ws = api.workspace(api.ss_tree_verify_workspace_bytes(1, 7, V))
    api.ss_tree_verify(torch.from_numpy(rows[None]).cuda(), torch.from_numpy(tok[None]).cuda(), trees, out["accept_len"],
                       out["accept_path"], out["last_node"], out["bonus_token"], out["node_argmax"], ws)
    assert api.ss_status(ws) == 0
    assert list(out["node_argmax"][0].cpu().numpy()) == am
    ref = oracle.tree_verify(rows, tok, parent, path_cap=64)
    assert int(out["accept_len"][0]) == ref["accept_len"] == 7
    assert int(out["bonus_token"][0]) == ref["bonus_token"]


def test_a_wait_that_runs_out_reports_a_timeout_and_the_stream_stays_usable(cuda, oracle):
    """The step in which a CTA of a split head combines partial rows is run with no second CTA launched
    (ss_wait_selftest): the rows it waits for cannot arrive.  With the bound shortened through the workspace
    header the wait gives up, the status word reads SS_ERR_DEVICE_TIMEOUT, nothing was written, and a split
    attention call on the same stream and workspace then matches the oracle."""
    api, DeviceStep = cuda
    cfg = W.custom_config("timeout", n_layers=1, n_msa_layers=0, prefix_len=600, n_nodes=12, gamma=0, max_depth=3,
                          n_heads=8, head_dim=128, config_id=810)       # 8 heads of 12 rows: 8 CTAs share a head's keys
    st = W.make_step(cfg)
    dev = DeviceStep(st)
    assert dev.attn_ws.numel() * dev.attn_ws.element_size() >= 65536
    words = dev.attn_ws.view(torch.int32)
    words[1] = 100                                             # bound of every wait: 100 x 1024 cycles
    api.ss_wait_selftest(dev.attn_ws)
    assert api.ss_status(dev.attn_ws) == api.SS_ERR_DEVICE_TIMEOUT
    torch.cuda.synchronize()                                   # nothing faulted: the context is healthy
    assert int(words[2:].abs().max()) == 0                     # the wait wrote nothing
    words[1] = 0
    dev.run_attention()
    assert api.ss_status(dev.attn_ws) == 0
    assert_attention_close(oracle, st, st.layer(0), dev, 0)
    assert int(words[2:].abs().max()) == 0                     # a call leaves the partial rows' area zero again


def test_no_wait_runs_out_over_many_replays(cuda):
    """The attention kernels' roles meet on phase-parity barriers; a waiter that falls two phases behind one of
    them would wait until its bound runs out (a one-second stall and SS_ERR_DEVICE_TIMEOUT).  Whether that can
    happen depends on timing, so the plain and the multi-stream layers of the 7B-class shape are replayed
    back to back a few thousand times, as graphs of their own and as the whole step, with the status word read
    after every batch of replays."""
    api, DeviceStep = cuda
    st = W.make_step(W.CONFIGS["7b"])
    dev = DeviceStep(st)
    stream = torch.cuda.Stream()
    nl = len(dev.layers)
    plain = [i for i in range(nl) if not dev.is_msa[i]]
    msa = [i for i in range(nl) if dev.is_msa[i]]

    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            fn(stream)
            stream.synchronize()
            with torch.cuda.graph(g, stream=stream):
                fn(stream)
        return g

    graphs = [capture(dev.run_step), capture(dev.run_attention), capture(lambda s: dev.run_attention(s, only=plain)),
              capture(lambda s: dev.run_attention(s, only=msa))]
    words = dev.attn_ws.view(torch.int32)
    for _ in range(40):
        for g in graphs:
            with torch.cuda.stream(stream):
                for _ in range(20):
                    g.replay()
            stream.synchronize()
            assert int(words[0]) == 0
