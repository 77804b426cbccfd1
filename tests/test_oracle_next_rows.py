"""Pins for the oracle's next-draft construction (Sec. 3.2.2, App. A.1), tree pruning (Sec. 3.2.3),
soft / sampled verification (App. A.2, App. B), stream insertion (Eq. 3) and value rotation (Eq. 7).

Each function is checked against something other than itself: library routines (numpy's stable sort and
cumulative sums, scipy's softmax / log-sum-exp / entropy), closed forms (tree size of Sec. 3.2.3, the
k = 1 chain of App. D, norm and composition laws of a rotation), hand-built examples and brute force."""
import numpy as np
import pytest
from scipy.special import logsumexp, softmax
from scipy.stats import entropy

from paper_2402_11131_b200 import workloads as W


def _full_tree_size(k, gamma):
    return 1 + sum(k ** g for g in range(1, gamma + 1))


# ---- next draft ------------------------------------------------------------------------------------
@pytest.mark.parametrize("k,gamma", [(1, 4), (2, 3), (4, 2), (3, 3), (4, 3)])
def test_next_draft_size_levels_and_order(oracle, k, gamma):
    rng = np.random.default_rng(10 * k + gamma)
    V = 300
    lg = rng.standard_normal((gamma, V)).astype(np.float32)
    tokens, parent = oracle.next_draft(lg, k, bonus_token=17, max_nodes=1000)
    n = _full_tree_size(k, gamma)                       # 1 + sum_g k^g (Sec. 3.2.3)
    assert len(tokens) == n == len(parent)
    assert tokens[0] == 17 and parent[0] == -1          # the correction token is the root (App. A.1)
    assert all(parent[i] < i for i in range(1, n))
    depth = np.zeros(n, dtype=int)
    for i in range(1, n):
        depth[i] = depth[parent[i]] + 1
    assert depth.max() == gamma and np.all(np.diff(depth) >= 0)      # level by level
    for g in range(1, gamma + 1):
        top = np.argsort(-lg[g - 1], kind="stable")[:k]            # library: descending, equal values by index
        nodes = np.where(depth == g)[0]
        assert len(nodes) == k ** g
        for p in np.where(depth == g - 1)[0]:                         # every node of level g-1 has the k best of stream g
            kids = [i for i in nodes if parent[i] == p]
            assert list(tokens[kids]) == list(top)


def test_next_draft_k1_is_the_chain_of_the_qualitative_example(oracle):
    # gamma = 4, k = 1: a pass can advance at most 5 tokens (App. D): root + one token per stream, in a chain
    lg = np.random.default_rng(3).standard_normal((4, 64)).astype(np.float32)
    tokens, parent = oracle.next_draft(lg, 1, 5, 64)
    assert list(parent) == [-1, 0, 1, 2, 3]
    assert list(tokens[1:]) == list(np.argmax(lg, axis=1))


def test_next_draft_ties_take_lowest_indices_and_cut_at_max_nodes(oracle):
    lg = np.zeros((2, 40), dtype=np.float32)
    lg[0, [5, 9, 30]] = 2.0
    lg[1, [1, 2]] = 1.0
    tokens, parent = oracle.next_draft(lg, 3, 0, max_nodes=9)
    assert list(tokens[1:4]) == [5, 9, 30]
    assert len(tokens) == 9                                           # 1 + 3 + 9 = 13 nodes cut after 9
    assert list(tokens[4:9]) == [1, 2, 0, 1, 2] and list(parent[4:9]) == [1, 1, 1, 2, 2]
    # gamma = 0: the root alone
    t0, p0 = oracle.next_draft(np.zeros((0, 40), dtype=np.float32), 1, 3, 8)
    assert list(t0) == [3] and list(p0) == [-1]


def test_next_draft_tree_is_accepted_by_the_tree_builder_and_verifier(oracle):
    rng = np.random.default_rng(5)
    lg = rng.standard_normal((3, 97)).astype(np.float32)
    tokens, parent = oracle.next_draft(lg, 2, 11, 64)
    depth, anc, md = oracle.tree_build(parent)
    assert md == 3
    # a main stream that agrees with the first child at every level accepts the left-most deepest path
    am = np.zeros(len(tokens), dtype=int)
    node = 0
    for g in range(3):
        am[node] = tokens[[i for i in range(len(tokens)) if parent[i] == node][0]]
        node = [i for i in range(len(tokens)) if parent[i] == node][0]
    main = np.full((len(tokens), 97), -5.0, dtype=np.float32)
    main[np.arange(len(tokens)), am] = 5.0
    r = oracle.tree_verify(main, tokens, parent)
    assert r["accept_len"] == 4 and r["last_node"] == node


# ---- pruning -----------------------------------------------------------------------------------------
def test_prune_probabilities_are_the_library_softmax_and_threshold_drops_subtrees(oracle):
    rng = np.random.default_rng(7)
    parent = np.array([-1, 0, 0, 1, 1, 2, 2, 3, 5], dtype=np.int32)
    T, V = len(parent), 211
    lg = (2.0 * rng.standard_normal((T, V))).astype(np.float32)
    tok = rng.integers(0, V, T).astype(np.int32)
    sm = softmax(lg.astype(np.float64), axis=1)
    want = np.array([1.0] + [sm[parent[c], tok[c]] for c in range(1, T)])
    tau = float(np.median(want[1:]))
    r = oracle.tree_prune(lg, tok, parent, tau)
    np.testing.assert_allclose(r["edge_prob"], want, rtol=1e-12)
    # brute force: a node survives iff every edge on its root path is at or above the threshold
    keep = np.ones(T, dtype=bool)
    for c in range(1, T):
        a = c
        while a != 0:
            keep[c] &= want[a] >= tau
            a = parent[a]
    np.testing.assert_array_equal(r["keep"].astype(bool), keep)
    kept = np.where(keep)[0]
    np.testing.assert_array_equal(r["kept_nodes"], kept)
    remap = {int(o): i for i, o in enumerate(kept)}
    np.testing.assert_array_equal(r["new_parent"], [-1] + [remap[int(parent[o])] for o in kept[1:]])
    np.testing.assert_array_equal(r["new_index"], [remap.get(c, -1) for c in range(T)])
    assert 1 < len(kept) < T


def test_prune_example_of_the_tree_draft_figure(oracle):
    # the pruned-subtree example of App. A.1: nodes 2, 5, 6 go when the edge root -> node 2 is improbable
    parent = np.array([-1, 0, 0, 1, 1, 2, 2], dtype=np.int32)
    tok = np.array([0, 1, 2, 3, 4, 5, 6], dtype=np.int32)
    lg = np.zeros((7, 8), dtype=np.float32)
    lg[0, 1] = 6.0                                    # the root strongly prefers token 1 over token 2
    r = oracle.tree_prune(lg, tok, parent, threshold=0.05)
    assert list(r["kept_nodes"]) == [0, 1, 3, 4] and list(r["new_parent"]) == [-1, 0, 1, 1]
    # threshold 0 keeps everything, threshold above 1 keeps the root only
    assert len(oracle.tree_prune(lg, tok, parent, 0.0)["kept_nodes"]) == 7
    assert list(oracle.tree_prune(lg, tok, parent, 1.5)["kept_nodes"]) == [0]
    # decisions handed in replace the threshold
    r2 = oracle.tree_prune(lg, tok, parent, 0.0, decide=np.array([1, 0, 1, 1, 1, 1, 0], dtype=np.uint8))
    assert list(r2["kept_nodes"]) == [0, 2, 5]


# ---- soft and sampled verification ----------------------------------------------------------------------
def test_soft_matching_threshold_uses_the_library_entropy(oracle):
    rng = np.random.default_rng(11)
    parent = np.array([-1, 0, 0, 1, 2, 3], dtype=np.int32)
    T, V = len(parent), 150
    lg = (3.0 * rng.standard_normal((T, V))).astype(np.float32)
    tok = rng.integers(0, V, T).astype(np.int32)
    tok[1] = int(np.argmax(lg[0])); tok[3] = int(np.argmax(lg[1]))          # a likely path 0 -> 1 -> 3
    sm = softmax(lg.astype(np.float64), axis=1)
    ent = np.array([entropy(sm[t]) for t in range(T)])
    eps, delta = 0.3, 0.09
    r = oracle.tree_verify_soft(lg, tok, parent, eps, delta)
    np.testing.assert_allclose(r["node_entropy"], ent, rtol=1e-10)
    np.testing.assert_allclose(r["edge_prob"][1:], [sm[parent[c], tok[c]] for c in range(1, T)], rtol=1e-12)
    ok = [True] + [sm[parent[c], tok[c]] >= min(eps, delta * np.exp(-ent[parent[c]])) for c in range(1, T)]
    # brute force over root paths
    best, best_depth = 0, 0
    for c in range(T):
        path, a = [], c
        while a != -1:
            path.append(a); a = parent[a]
        if all(ok[x] for x in path) and len(path) - 1 > best_depth:
            best, best_depth = c, len(path) - 1
    assert r["last_node"] == best and r["accept_len"] == best_depth + 1
    assert r["bonus_token"] == int(np.argmax(lg[best]))
    assert r["accept_len"] >= 3                                                # the likely path is accepted


def test_soft_matching_with_a_vanishing_threshold_accepts_the_deepest_path_and_hard_limit(oracle):
    parent = np.array([-1, 0, 1, 2, 0], dtype=np.int32)
    lg = np.random.default_rng(2).standard_normal((5, 30)).astype(np.float32)
    tok = np.arange(5, dtype=np.int32)
    r = oracle.tree_verify_soft(lg, tok, parent, eps=1e-30, delta=1e-30)
    assert r["accept_len"] == 4 and r["last_node"] == 3
    r = oracle.tree_verify_soft(lg, tok, parent, eps=2.0, delta=1e9)            # bar = 2 > any probability
    assert r["accept_len"] == 1 and r["bonus_token"] == int(np.argmax(lg[0]))


def test_sampled_verification_draws_by_inversion_of_the_top_k_distribution(oracle):
    rng = np.random.default_rng(13)
    parent = np.array([-1, 0, 0, 1, 1, 3], dtype=np.int32)
    T, V, k = len(parent), 120, 5
    lg = (2.0 * rng.standard_normal((T, V))).astype(np.float32)
    u = rng.random(T).astype(np.float32)
    drawn = np.zeros(T, dtype=int)
    for t in range(T):
        idx = np.argsort(-lg[t], kind="stable")[:k]
        cdf = np.cumsum(softmax(lg[t, idx].astype(np.float64)))
        drawn[t] = idx[min(int(np.searchsorted(cdf, float(u[t]), side="right")), k - 1)]
    tok = rng.integers(0, V, T).astype(np.int32)
    tok[1] = drawn[0]; tok[3] = drawn[1]; tok[5] = drawn[3]                  # the path 0-1-3-5 matches the draws
    r = oracle.tree_verify_sampled(lg, tok, parent, k, u)
    np.testing.assert_array_equal(r["node_token"], drawn)
    assert r["accept_len"] == 4 and list(r["path"][:4]) == [0, 1, 3, 5] and r["bonus_token"] == drawn[5]
    # k = 1 is greedy verification; u = 0 always draws the arg-max
    g = oracle.tree_verify(lg, tok, parent)
    s = oracle.tree_verify_sampled(lg, tok, parent, 1, u)
    assert (s["accept_len"], s["last_node"], s["bonus_token"]) == (g["accept_len"], g["last_node"], g["bonus_token"])
    z = oracle.tree_verify_sampled(lg, tok, parent, k, np.zeros(T, dtype=np.float32))
    np.testing.assert_array_equal(z["node_token"], np.argmax(lg, axis=1))
    # empirical frequencies of the draw follow the top-k softmax
    row = np.array([[2.0, 1.0, 0.0, -1.0, 5.0 - 10.0]], dtype=np.float32)
    us = (np.arange(4000) + 0.5) / 4000
    cnt = np.zeros(5)
    for x in us:
        cnt[oracle.tree_verify_sampled(row, np.array([0]), np.array([-1]), 3, np.array([x], dtype=np.float32))["node_token"][0]] += 1
    np.testing.assert_allclose(cnt[:3] / 4000, softmax(np.array([2.0, 1.0, 0.0])), atol=2e-3)
    assert cnt[3:].sum() == 0


def test_argmax_rule_for_incomparable_and_special_values(oracle):
    """A NaN is never selected while a comparable value exists; -0 and +0 tie (lowest index); subnormals
    are ordinary values; -inf loses to everything finite; a row of NaNs reports index 0."""
    nan, inf = np.float32("nan"), np.float32("inf")
    rows = {
        "nan_first": ([nan, 1.0, 3.0, 3.0], 2),
        "all_nan": ([nan, nan, nan], 0),
        "zeros": ([-0.0, 0.0, -0.0], 0),
        "subnormals": ([1e-45, 3e-45, 2e-45, 3e-45], 1),
        "neg_inf": ([-inf, -inf, -3e38, -inf], 2),
        "nan_middle": ([0.5, nan, 0.5, 0.25], 0),
    }
    for name, (vals, want) in rows.items():
        lg = np.array([vals], dtype=np.float32)
        r = oracle.tree_verify(lg, np.array([0]), np.array([-1]))
        assert r["bonus_token"] == want, name


# ---- stream insertion and value rotation ------------------------------------------------------------------
def test_stream_insert_is_one_float32_addition(oracle):
    rng = np.random.default_rng(17)
    m = W.f32_to_bf16_bits(rng.standard_normal((9, 48)).astype(np.float32) * 3)
    p = W.f32_to_bf16_bits(rng.standard_normal((3, 48)).astype(np.float32) * 0.01)
    out = oracle.stream_insert(m, p)
    mf = W.bf16_bits_to_f64(m).astype(np.float32)
    pf = W.bf16_bits_to_f64(p).astype(np.float32)
    want = W.f32_to_bf16_bits(mf[:, None, :] + pf[None, :, :])              # numpy float32 add, then bf16 RNE
    np.testing.assert_array_equal(out, want)
    assert out.shape == (9, 3, 48)
    # a zero embedding reproduces the main stream in every stream
    z = oracle.stream_insert(m, np.zeros((2, 48), dtype=np.uint16))
    np.testing.assert_array_equal(z[:, 0], m); np.testing.assert_array_equal(z[:, 1], m)


def test_value_rotation_is_a_rotation(oracle):
    rng = np.random.default_rng(19)
    v = W.f32_to_bf16_bits(rng.standard_normal((7, 32)).astype(np.float32))
    eps, gamma = 0.05, 4
    out = W.bf16_bits_to_f64(oracle.value_rotate(v, gamma, eps))
    z = W.bf16_bits_to_f64(v)[:, 0::2] + 1j * W.bf16_bits_to_f64(v)[:, 1::2]
    for n in range(1, gamma + 1):
        want = z * np.exp(1j * eps * n)                                     # the closed form of Eq. 7
        got = out[:, n - 1, 0::2] + 1j * out[:, n - 1, 1::2]
        np.testing.assert_allclose(got, want, atol=2.0 ** -8 * 6)            # bf16 rounding of components up to ~4
        np.testing.assert_allclose(np.abs(got), np.abs(z), rtol=2.0 ** -7, atol=1e-3)   # a rotation keeps the modulus
    # angle 0 is the identity, exactly; pi / 2 maps (re, im) to (-im, re) up to the rounding of cos(pi/2) ~ 6e-17
    ident = oracle.value_rotate(v, 2, 0.0)
    np.testing.assert_array_equal(ident[:, 0], v); np.testing.assert_array_equal(ident[:, 1], v)
    q = W.bf16_bits_to_f64(oracle.value_rotate(v, 1, np.pi / 2))[:, 0]
    np.testing.assert_allclose(q[:, 0::2], -W.bf16_bits_to_f64(v)[:, 1::2], atol=1e-6)
    np.testing.assert_allclose(q[:, 1::2], W.bf16_bits_to_f64(v)[:, 0::2], atol=1e-6)
    # bit-level: numpy float32 products and sums with the same fp32 table
    cs = oracle.rotation_table(eps, gamma)
    vf = W.bf16_bits_to_f64(v).astype(np.float32)
    re, im = vf[:, 0::2], vf[:, 1::2]
    for n in range(gamma):
        c, s = cs[n]
        np.testing.assert_array_equal(oracle.value_rotate(v, gamma, eps)[:, n, 0::2], W.f32_to_bf16_bits(re * c - im * s))
        np.testing.assert_array_equal(oracle.value_rotate(v, gamma, eps)[:, n, 1::2], W.f32_to_bf16_bits(re * s + im * c))
