"""Pins for the oracle's attention (Eq. 1, Eq. 2) against things other than itself:
an independently coded dense-mask brute force, library routines on the special cases that
reduce to them, closed forms, the mask example printed in App. A, and causality invariants."""
import os

import numpy as np
import pytest

from paper_2402_11131_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_case(seed, T, L, gamma, H=2, d=16, kind="uniform_parent", max_depth=3):
    cfg = W.custom_config("small", n_heads=H, head_dim=d, prefix_len=L, n_nodes=T, max_depth=max_depth,
                          gamma=gamma, tree_kind=kind, config_id=1000 + seed)
    st = W.make_step(cfg)
    return st, st.layer(0)


def run_oracle(oracle, st, ly, b=0, parent=None, **kw):
    c = st.cfg
    s0 = int(st.kv_start[b])
    kc = ly.k_cache[s0:s0 + int(st.kv_capacity[b])]
    vc = ly.v_cache[s0:s0 + int(st.kv_capacity[b])]
    g = c.gamma if ly.is_msa else 0
    return oracle.msa_attention(
        st.parent[b] if parent is None else parent, int(st.kv_len[b]), g, st.sm_scale, ly.q_main[b], kc, vc,
        None if g == 0 else ly.q_spec[b], None if g == 0 else ly.k_spec[b], None if g == 0 else ly.v_spec[b], **kw)


def brute_force(st, ly, b=0):
    """Dense additive-mask attention over the concatenation of ALL keys of the step
    (prefix, tree, every stream key), mask built by walking parent pointers per query row."""
    c = st.cfg
    T, H, d, L = c.n_nodes, c.n_heads, c.head_dim, int(st.kv_len[b])
    g = c.gamma if ly.is_msa else 0
    par = st.parent[b]
    s0 = int(st.kv_start[b])
    f = W.bf16_bits_to_f64
    keys = [f(ly.k_cache[s0:s0 + L + T])]
    vals = [f(ly.v_cache[s0:s0 + L + T])]
    if g:
        keys.append(f(ly.k_spec[b]).reshape(T * g, H, d))
        vals.append(f(ly.v_spec[b]).reshape(T * g, H, d))
    K = np.concatenate(keys, 0)
    V = np.concatenate(vals, 0)
    nk = K.shape[0]
    rows, Q = [], []
    for t in range(T):
        rows.append((t, 0)); Q.append(f(ly.q_main[b, t]))
        for j in range(1, g + 1):
            rows.append((t, j)); Q.append(f(ly.q_spec[b, t, j - 1]))
    Q = np.stack(Q, 0)                       # [rows][H][d]
    mask = np.full((len(rows), nk), -np.inf)
    for r, (t, j) in enumerate(rows):
        mask[r, :L] = 0.0
        a = t
        while a >= 0:                        # the node and its chain of parents up to the root
            mask[r, L + a] = 0.0
            a = int(par[a])
        for i in range(1, j + 1):            # streams 1..j of the same node
            mask[r, L + T + t * g + (i - 1)] = 0.0
    out = np.zeros((len(rows), H, d))
    lse = np.zeros((len(rows), H))
    for h in range(H):
        s = st.sm_scale * (Q[:, h, :] @ K[:, h, :].T) + mask
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        out[:, h, :] = (p @ V[:, h, :]) / p.sum(axis=1, keepdims=True)
        lse[:, h] = (m + np.log(p.sum(axis=1, keepdims=True)))[:, 0]
    return rows, out, lse


@pytest.mark.parametrize("gamma", [0, 1, 2, 3])
@pytest.mark.parametrize("T,L", [(1, 0), (1, 5), (4, 0), (6, 16), (8, 9)])
def test_oracle_matches_dense_mask_brute_force(oracle, gamma, T, L):
    st, ly = small_case(7 * T + L + gamma, T, L, gamma)
    om, lm, os_, ls = run_oracle(oracle, st, ly)
    rows, ref, ref_lse = brute_force(st, ly)
    for r, (t, j) in enumerate(rows):
        got = om[t] if j == 0 else os_[t, j - 1]
        got_lse = lm[t] if j == 0 else ls[t, j - 1]
        np.testing.assert_allclose(got, ref[r], rtol=0, atol=1e-12)
        np.testing.assert_allclose(got_lse, ref_lse[r], rtol=0, atol=1e-12)


def test_chain_tree_gamma0_is_causal_decode_attention(oracle):
    """A chain tree with no streams is causal attention of T new tokens over L+T keys:
    compare with torch's scaled_dot_product_attention (is_causal) in fp64."""
    torch = pytest.importorskip("torch")
    T, L, H, d = 7, 13, 2, 16
    st, ly = small_case(3, T, L, 0, H=H, d=d, kind="chain", max_depth=T)
    assert list(st.parent[0]) == [-1] + list(range(T - 1))
    om, _, _, _ = run_oracle(oracle, st, ly)
    f = W.bf16_bits_to_f64
    n = L + T
    K = torch.from_numpy(f(ly.k_cache[:n])).permute(1, 0, 2)          # [H][n][d]
    V = torch.from_numpy(f(ly.v_cache[:n])).permute(1, 0, 2)
    Q = torch.zeros(H, n, d, dtype=torch.float64)
    Q[:, L:, :] = torch.from_numpy(f(ly.q_main[0])).permute(1, 0, 2)
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True, scale=st.sm_scale)
    np.testing.assert_allclose(om, ref[:, L:, :].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_single_node_is_single_query_softmax_attention(oracle):
    torch = pytest.importorskip("torch")
    st, ly = small_case(5, 1, 33, 0, H=3, d=32)
    om, lm, _, _ = run_oracle(oracle, st, ly)
    f = W.bf16_bits_to_f64
    for h in range(3):
        K = torch.from_numpy(f(ly.k_cache[:34, h]))
        V = torch.from_numpy(f(ly.v_cache[:34, h]))
        q = torch.from_numpy(f(ly.q_main[0, 0, h]))
        x = st.sm_scale * (K @ q)
        np.testing.assert_allclose(om[0, h], (torch.softmax(x, 0) @ V).numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(lm[0, h], torch.logsumexp(x, 0).item(), rtol=0, atol=1e-12)


def test_scale_argument_is_applied_to_scores(oracle):
    """Doubling sm_scale must equal doubling the queries (exact in bf16: exponent + 1)."""
    st, ly = small_case(11, 5, 12, 2)
    a = run_oracle(oracle, st, ly)
    ly.q_main = W.f32_to_bf16_bits((W.bf16_bits_to_f64(ly.q_main) * 2).astype(np.float32))
    ly.q_spec = W.f32_to_bf16_bits((W.bf16_bits_to_f64(ly.q_spec) * 2).astype(np.float32))
    st.sm_scale *= 0.5
    b = run_oracle(oracle, st, ly)
    for x, y in zip(a, b):
        np.testing.assert_allclose(x, y, rtol=0, atol=1e-13)


def test_zero_queries_count_visible_keys(oracle):
    """With q = 0 every score is 0, so exp(lse) is the number of visible keys and the output is
    the plain mean of the visible V rows: L + depth(t) + 1 keys for the main row, + j for stream j.
    The expected depths are written by hand for this tree."""
    parent = np.array([-1, 0, 0, 1, 1, 3, 2, 5], dtype=np.int32)
    depth = [0, 1, 1, 2, 2, 3, 2, 4]
    L, g = 10, 3
    st, ly = small_case(2, 8, L, g, max_depth=4)
    ly.q_main[:] = 0
    ly.q_spec[:] = 0
    # V[slot][h][0] = slot index, so the mean over visible keys identifies WHICH slots were seen
    ly.v_cache[:, :, 0] = W.f32_to_bf16_bits(np.arange(ly.v_cache.shape[0], dtype=np.float32))[:, None]
    ly.v_spec[..., 0] = W.f32_to_bf16_bits(np.full(ly.v_spec.shape[:-1], 100.0, dtype=np.float32))
    om, lm, os_, ls = run_oracle(oracle, st, ly, parent=parent)
    paths = {0: [0], 1: [0, 1], 2: [0, 2], 3: [0, 1, 3], 4: [0, 1, 4], 5: [0, 1, 3, 5], 6: [0, 2, 6],
             7: [0, 1, 3, 5, 7]}
    for t in range(8):
        n_main = L + depth[t] + 1
        np.testing.assert_allclose(np.exp(lm[t]), n_main, rtol=1e-12)
        slots = list(range(L)) + [L + a for a in paths[t]]
        np.testing.assert_allclose(om[t, :, 0], np.mean(slots), rtol=1e-12)
        for j in range(1, g + 1):
            np.testing.assert_allclose(np.exp(ls[t, j - 1]), n_main + j, rtol=1e-12)
            np.testing.assert_allclose(os_[t, j - 1, :, 0], (np.sum(slots) + 100.0 * j) / (n_main + j), rtol=1e-12)


def _read_mask_example():
    parent, vis = None, {}
    with open(os.path.join(GOLDEN, "mask_example.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":")
            if k == "parent":
                parent = np.array([int(x) for x in v.split()], dtype=np.int32)
            else:
                vis[int(k)] = {int(x) for x in v.split()}
    return parent, vis


def test_paper_mask_example_one_hot_membership(oracle):
    """For every (query row, key) pair of the App. A mask example: boost that key's score by +60;
    the output equals that key's V row iff the key is visible to the row."""
    parent, vis = _read_mask_example()
    T, L, g, H, d = 5, 3, 2, 1, 8
    st, ly = small_case(9, T, L, g, H=H, d=d)
    one = W.f32_to_bf16_bits(np.array([1.0], dtype=np.float32))[0]
    big = W.f32_to_bf16_bits(np.array([60.0], dtype=np.float32))[0]
    # q = e_0 for all rows; all keys have k[0] = 0 except the boosted one
    ly.q_main[:] = 0; ly.q_main[..., 0] = one
    ly.q_spec[:] = 0; ly.q_spec[..., 0] = one
    ly.k_cache[..., 0] = 0
    ly.k_spec[..., 0] = 0
    f = W.bf16_bits_to_f64
    n_rows = 0
    # cache keys: prefix 0..L-1 and tree nodes
    for slot in range(L + T):
        kc = ly.k_cache.copy(); kc[slot, :, 0] = big
        ly2 = W.LayerInputs(0, True, ly.q_main, ly.q_spec, ly.k_spec, ly.v_spec, kc, ly.v_cache)
        om, _, os_, _ = run_oracle(oracle, st, ly2, parent=parent)
        for t in range(T):
            visible = slot < L or (slot - L) in vis[t]
            for j in range(g + 1):
                got = om[t, 0] if j == 0 else os_[t, j - 1, 0]
                hit = np.allclose(got, f(ly.v_cache[slot, 0]), atol=1e-9)
                assert hit == visible, (slot, t, j)
                n_rows += 1
    # stream keys (t', i): visible only to streams j >= i of the same node
    for tp in range(T):
        for i in range(1, g + 1):
            ks = ly.k_spec.copy(); ks[0, tp, i - 1, :, 0] = big
            ly2 = W.LayerInputs(0, True, ly.q_main, ly.q_spec, ks, ly.v_spec, ly.k_cache, ly.v_cache)
            om, _, os_, _ = run_oracle(oracle, st, ly2, parent=parent)
            for t in range(T):
                for j in range(g + 1):
                    got = om[t, 0] if j == 0 else os_[t, j - 1, 0]
                    hit = np.allclose(got, f(ly.v_spec[0, tp, i - 1, 0]), atol=1e-9)
                    assert hit == (t == tp and 1 <= i <= j), (tp, i, t, j)
    assert n_rows == (L + T) * T * (g + 1)     # (1+gamma) rows per node (Sec. 3.2.3 row count)


def test_causality_invariants(oracle):
    T, L, g = 8, 11, 3
    st, ly = small_case(21, T, L, g, max_depth=3)
    base = run_oracle(oracle, st, ly)
    par = st.parent[0]
    rng = np.random.default_rng(0)

    def noise(shape):
        return W.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))

    # (1) streams > j do not affect stream j; no stream affects any main row
    for j in range(0, g):
        ks, vs = ly.k_spec.copy(), ly.v_spec.copy()
        ks[:, :, j:] = noise(ks[:, :, j:].shape)
        vs[:, :, j:] = noise(vs[:, :, j:].shape)
        ly2 = W.LayerInputs(0, True, ly.q_main, ly.q_spec, ks, vs, ly.k_cache, ly.v_cache)
        om, lm, os_, ls = run_oracle(oracle, st, ly2)
        assert np.array_equal(om, base[0]) and np.array_equal(lm, base[1])
        assert np.array_equal(os_[:, :j], base[2][:, :j])
        assert not np.allclose(os_[:, j:], base[2][:, j:])
    # (2) node t is unaffected by K/V of nodes off its root path (siblings, cousins, descendants)
    for victim in range(T):
        kc, vc = ly.k_cache.copy(), ly.v_cache.copy()
        kc[L + victim] = noise(kc[L + victim].shape)
        vc[L + victim] = noise(vc[L + victim].shape)
        ly2 = W.LayerInputs(0, True, ly.q_main, ly.q_spec, ly.k_spec, ly.v_spec, kc, vc)
        om, _, os_, _ = run_oracle(oracle, st, ly2)
        for t in range(T):
            on_path, a = False, t
            while a >= 0:
                on_path |= (a == victim)
                a = int(par[a])
            same = np.array_equal(om[t], base[0][t]) and np.array_equal(os_[t], base[2][t])
            assert same == (not on_path), (victim, t)
    # (3) slots past L+T-1 are never read
    kc = ly.k_cache.copy(); kc[L + T:] = noise(kc[L + T:].shape)
    ly2 = W.LayerInputs(0, True, ly.q_main, ly.q_spec, ly.k_spec, ly.v_spec, kc, ly.v_cache)
    assert np.array_equal(run_oracle(oracle, st, ly2)[0], base[0])
    # (4) permuting prefix slots (K and V together) changes nothing beyond rounding
    perm = rng.permutation(L)
    kc, vc = ly.k_cache.copy(), ly.v_cache.copy()
    kc[:L], vc[:L] = ly.k_cache[perm], ly.v_cache[perm]
    ly2 = W.LayerInputs(0, True, ly.q_main, ly.q_spec, ly.k_spec, ly.v_spec, kc, vc)
    for x, y in zip(run_oracle(oracle, st, ly2), base):
        np.testing.assert_allclose(x, y, rtol=0, atol=1e-13)
    # (5) swapping the roles of K and V is NOT a no-op (catches transposed operands)
    ly2 = W.LayerInputs(0, True, ly.q_main, ly.q_spec, ly.v_spec, ly.k_spec, ly.v_cache, ly.k_cache)
    assert not np.allclose(run_oracle(oracle, st, ly2)[0], base[0])


def test_node_and_head_selection_only_skips_rows(oracle):
    st, ly = small_case(4, 6, 8, 2, H=3)
    full = run_oracle(oracle, st, ly)
    sel = np.array([0, 1, 0, 0, 1, 0], dtype=np.uint8)
    part = run_oracle(oracle, st, ly, node_sel=sel, heads=(1, 3))
    assert np.array_equal(part[0][[1, 4]][:, 1:], full[0][[1, 4]][:, 1:])
    assert np.array_equal(part[2][[1, 4]][:, :, 1:], full[2][[1, 4]][:, :, 1:])
    assert np.isnan(part[0][0]).all() and np.isnan(part[0][1, 0]).all()


def test_tree_build_rejects_bad_parents(oracle):
    for bad in ([0, 0], [-1, 1], [-1, 0, 2], [-1, -1]):
        with pytest.raises(ValueError):
            oracle.tree_build(np.array(bad, dtype=np.int32))
    depth, anc, md = oracle.tree_build(np.array([-1, 0, 0, 1, 2], dtype=np.int32))
    parent, vis = _read_mask_example()
    assert md == 2 and list(depth) == [0, 1, 1, 2, 2]
    for t in range(5):
        assert set(np.nonzero(anc[t])[0]) == vis[t]
