"""Pins for the oracle's greedy tree verification and KV compaction: the example of App. A.1,
closed forms, path enumeration, and a sequential-copy brute force."""
import os

import numpy as np
import pytest

from paper_2402_11131_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def logits_with_argmax(am, V, seed=0):
    rng = np.random.default_rng(seed)
    lg = rng.standard_normal((len(am), V)).astype(np.float32)
    for t, a in enumerate(am):
        lg[t, a] = 9.0
    return lg


def test_paper_accept_example(oracle):
    parent, tok, am, exp = [], [], [], {}
    with open(os.path.join(GOLDEN, "accept_example.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":")
            if k.startswith("expected_"):
                exp[k[len("expected_"):]] = [int(x) for x in v.split()]
            else:
                p, t, a = (int(x) for x in v.split())
                parent.append(p); tok.append(t); am.append(a)
    r = oracle.tree_verify(logits_with_argmax(am, 100), np.array(tok), np.array(parent), path_cap=5)
    assert r["accept_len"] == exp["accept_len"][0]
    assert list(r["path"][:r["accept_len"]]) == exp["path"]
    assert list(r["path"][r["accept_len"]:]) == [-1] * (5 - r["accept_len"])
    assert r["last_node"] == exp["last_node"][0]
    assert r["bonus_token"] == exp["bonus_token"][0]
    assert list(r["node_argmax"]) == am


def test_argmax_takes_lowest_index_on_ties(oracle):
    lg = np.zeros((1, 50), dtype=np.float32)
    lg[0, [7, 19, 33]] = 3.5
    r = oracle.tree_verify(lg, np.array([0]), np.array([-1]))
    assert r["bonus_token"] == 7 and r["accept_len"] == 1 and r["last_node"] == 0
    np.testing.assert_array_equal(r["node_argmax"], np.argmax(lg, axis=1))   # numpy: first maximum


def test_argmax_matches_library_on_random_rows(oracle):
    rng = np.random.default_rng(5)
    lg = rng.standard_normal((9, 777)).astype(np.float32)
    r = oracle.tree_verify(lg, np.zeros(9, dtype=np.int32), np.array([-1] + list(range(8))))
    np.testing.assert_array_equal(r["node_argmax"], np.argmax(lg, axis=1))


def test_chain_first_mismatch_gives_length(oracle):
    """gamma = 4, k = 1 draft (a chain of 5 nodes): at most 5 tokens advance per pass; a first
    mismatch at depth m accepts exactly m nodes."""
    T, V = 5, 64
    parent = np.array([-1, 0, 1, 2, 3])
    tok = np.array([3, 10, 11, 12, 13])
    for m in range(1, T + 1):
        am = [10, 11, 12, 13, 40]
        if m < T:
            am[m - 1] = 50                      # node m's token no longer matches its parent's argmax
        r = oracle.tree_verify(logits_with_argmax(am, V), tok, parent)
        assert r["accept_len"] == m and list(r["path"][:m]) == list(range(m))
        assert r["last_node"] == m - 1 and r["bonus_token"] == am[m - 1]
        assert r["accept_len"] <= 5


def test_all_correct_accepts_deepest_lowest_index_and_none_correct_accepts_root(oracle):
    parent = np.array([-1, 0, 0, 1, 1, 2, 3, 5])      # depths 0 1 1 2 2 2 3 3
    T, V = 8, 40
    tok = np.array([1, 5, 6, 7, 8, 9, 10, 10])
    # make every node valid: am[parent] must equal tok[child] for all children -> needs equal sibling
    # tokens, so use one token per parent instead
    tok = np.array([1, 5, 5, 7, 7, 9, 10, 11])
    am = [5, 7, 9, 10, 0, 11, 0, 0]
    r = oracle.tree_verify(logits_with_argmax(am, V), tok, parent)
    assert r["accept_len"] == 4 and r["last_node"] == 6 and list(r["path"][:4]) == [0, 1, 3, 6]
    am = [2, 2, 2, 2, 2, 2, 2, 2]
    r = oracle.tree_verify(logits_with_argmax(am, V), tok, parent)
    assert r["accept_len"] == 1 and r["last_node"] == 0 and r["bonus_token"] == 2 and r["path"][0] == 0


def test_duplicate_sibling_tokens_pick_lowest_node(oracle):
    parent = np.array([-1, 0, 0, 0])
    tok = np.array([0, 4, 4, 4])
    r = oracle.tree_verify(logits_with_argmax([4, 1, 2, 3], 16), tok, parent)
    assert r["accept_len"] == 2 and r["last_node"] == 1 and r["bonus_token"] == 1


def _enumerate_paths(parent, tok, am):
    """All root-to-node paths; a path is accepted iff every edge matches.  Returns the deepest
    accepted node, lowest index among equals."""
    best, best_len = 0, 1
    for t in range(len(parent)):
        path, a = [], t
        while a >= 0:
            path.append(a); a = parent[a]
        path.reverse()
        if all(tok[c] == am[p] for p, c in zip(path[:-1], path[1:])) and len(path) > best_len:
            best, best_len = t, len(path)
    return best, best_len


@pytest.mark.parametrize("name", ["tiny", "1.3b"])
def test_verify_matches_path_enumeration_on_generated_workloads(oracle, name):
    st = W.make_step(W.CONFIGS[name])
    lg = st.logits()
    for b in range(st.cfg.batch):
        r = oracle.tree_verify(lg[b], st.draft_tokens[b], st.parent[b])
        am = np.argmax(lg[b], axis=1)
        best, ln = _enumerate_paths(list(st.parent[b]), list(st.draft_tokens[b]), list(am))
        assert (r["last_node"], r["accept_len"]) == (best, ln)
        assert r["accept_len"] <= st.cfg.max_depth + 1


def test_random_trees_against_path_enumeration(oracle):
    rng = np.random.default_rng(11)
    for trial in range(200):
        T = int(rng.integers(1, 12))
        parent = W.draw_tree(rng, T, 4, "uniform_parent")
        tok = rng.integers(0, 3, size=T).astype(np.int32)       # tiny vocab -> many matches and ties
        lg = rng.integers(0, 3, size=(T, 3)).astype(np.float32)  # ties in the argmax too
        r = oracle.tree_verify(lg, tok, parent)
        am = np.argmax(lg, axis=1)
        best, ln = _enumerate_paths(list(parent), list(tok), list(am))
        assert (r["last_node"], r["accept_len"], r["bonus_token"]) == (best, ln, am[best])


def _cache(rng, n_layers, slots, H, d):
    return rng.integers(0, 65536, size=(n_layers, slots, H, d)).astype(np.uint16)


def test_compaction_matches_sequential_copy(oracle):
    rng = np.random.default_rng(3)
    n_layers, slots, H, d, L = 3, 24, 2, 8, 9
    k, v = _cache(rng, n_layers, slots, H, d), _cache(rng, n_layers, slots, H, d)
    path = np.array([0, 2, 5, 11, -1], dtype=np.int32)
    k2, v2, nl = oracle.kv_compact(k, v, L, 4, path)
    ke, ve = k.copy(), v.copy()
    for l in range(n_layers):                       # ascending in-place copy is safe: path[i] >= i
        for i in range(4):
            ke[l, L + i] = ke[l, L + path[i]]
            ve[l, L + i] = ve[l, L + path[i]]
    assert nl == L + 4
    assert np.array_equal(k2[:, :L + 4], ke[:, :L + 4]) and np.array_equal(v2[:, :L + 4], ve[:, :L + 4])
    assert np.array_equal(k2[:, :L], k[:, :L]) and np.array_equal(v2[:, :L], v[:, :L])   # prefix untouched
    assert not np.array_equal(k2[:, L + 1], v2[:, L + 1])                                 # K and V not mixed up
    for i, p in enumerate([0, 2, 5, 11]):
        assert np.array_equal(k2[:, L + i], k[:, L + p]) and np.array_equal(v2[:, L + i], v[:, L + p])


def test_compaction_identity_path_is_a_no_op(oracle):
    rng = np.random.default_rng(4)
    k, v = _cache(rng, 2, 16, 1, 4), _cache(rng, 2, 16, 1, 4)
    k2, v2, nl = oracle.kv_compact(k, v, 5, 3, np.array([0, 1, 2], dtype=np.int32))
    assert nl == 8 and np.array_equal(k2, k) and np.array_equal(v2, v)
