"""Parity of the draft-management entry points (through the C ABI) with the CPU oracle.

Integer results (tokens, trees, paths, indices) are bit-exact.  Where an fp32 probability decides an
integer (pruning, soft matching, sampling), the probabilities are compared within a tolerance, the decisions
are compared wherever the oracle's fp64 value is not within rounding of the threshold, and everything that
follows from the decisions the device took is checked bit-exactly by handing those decisions to the oracle."""
import ctypes as C

import numpy as np
import pytest

from paper_2402_11131_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

PROB_RTOL = 2e-5       # fp32 log-sum-exp over <= 51200 logits against the fp64 oracle
MARGIN = 1e-4          # decisions within this relative distance of their threshold may fall on either side


@pytest.fixture(scope="module")
def cuda():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2402_11131_b200 import api, build
    build.build()
    api.lib()
    return api


def _desc_fields(d, n_max=64):
    return (d.n_nodes, d.max_depth, list(d.parent[:n_max]), list(d.depth[:n_max]), [int(x) for x in d.anc_mask[:n_max]])


def _i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


# ---- next draft ------------------------------------------------------------------------------------
@pytest.mark.parametrize("B,gamma,V,k,max_nodes,ties", [(1, 4, 32000, 2, 64, False), (3, 3, 51200, 4, 64, False),
                                                         (2, 4, 4097, 8, 64, True), (2, 2, 37, 3, 9, True),
                                                         (1, 4, 32000, 1, 64, False), (16, 4, 32000, 2, 31, False)])
def test_next_draft_is_bit_exact(cuda, oracle, B, gamma, V, k, max_nodes, ties):
    api = cuda
    rng = np.random.default_rng(1000 + V + k)
    n_rows = 5
    lg = rng.standard_normal((B, n_rows, gamma, V)).astype(np.float32)
    if ties:
        lg = np.round(lg * 2) / 2                                        # heavy ties: lowest indices must win
    rows = rng.integers(0, n_rows, B).astype(np.int32)
    bonus = rng.integers(0, V, B).astype(np.int32)
    d_tokens = torch.full((B, max_nodes), -7, dtype=torch.int32, device="cuda")
    d_trees = api.empty_trees(B)
    ws = api.workspace(api.ss_next_draft_workspace_bytes(B, gamma, V))
    for rep in range(2):                                                 # the workspace is left ready for reuse
        api.ss_next_draft(torch.from_numpy(lg).cuda(), _i32(rows), _i32(bonus), k, max_nodes, d_tokens, d_trees, ws)
        assert api.ss_status(ws) == 0
        toks = d_tokens.cpu().numpy()
        descs = api.trees_from_device(d_trees)
        for b in range(B):
            want_tok, want_par = oracle.next_draft(lg[b, rows[b]], k, int(bonus[b]), max_nodes)
            n = len(want_tok)
            assert descs[b].n_nodes == n and descs[b].gamma == gamma
            np.testing.assert_array_equal(toks[b, :n], want_tok)
            assert (toks[b, n:] == -1).all()
            host = api.ss_tree_build(want_par, gamma)                    # the descriptor the host builder gives
            assert _desc_fields(descs[b]) == _desc_fields(host)


def test_next_draft_special_values_follow_the_order_of_the_verification(cuda, oracle):
    api = cuda
    V = 300
    lg = np.zeros((1, 1, 3, V), dtype=np.float32)
    lg[0, 0, 0, :] = np.nan; lg[0, 0, 0, [17, 5]] = [1.0, 1.0]            # NaNs rank below everything; ties by index
    lg[0, 0, 1, :] = -np.inf; lg[0, 0, 1, 250] = -3e38                    # -inf is an ordinary (lowest) value
    lg[0, 0, 2, :] = -0.0; lg[0, 0, 2, 9] = 0.0; lg[0, 0, 2, 100] = 1e-45   # -0 == +0; a subnormal is larger
    d_tokens = torch.zeros((1, 64), dtype=torch.int32, device="cuda")
    d_trees = api.empty_trees(1)
    ws = api.workspace(api.ss_next_draft_workspace_bytes(1, 3, V))
    api.ss_next_draft(torch.from_numpy(lg).cuda(), None, _i32([4]), 3, 64, d_tokens, d_trees, ws)
    want_tok, _ = oracle.next_draft(lg[0, 0], 3, 4, 64)
    np.testing.assert_array_equal(d_tokens.cpu().numpy()[0, :len(want_tok)], want_tok)
    assert list(want_tok[1:4]) == [5, 17, 0] and list(want_tok[4:7]) == [250, 0, 1] and list(want_tok[13:16]) == [100, 0, 1]


# ---- pruning -----------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["1.3b", "7b", "7b_ragged16"])
def test_tree_prune_matches_the_oracle(cuda, oracle, name):
    api = cuda
    st = W.make_step(W.CONFIGS[name])
    c = st.cfg
    B, T, V = c.batch, c.n_nodes, c.vocab
    lg = st.logits()                                                     # stands in for the early-exit logits
    tok = st.draft_tokens.astype(np.int32)
    descs = [api.ss_tree_build(st.parent[b][:st.nodes(b)], c.gamma) for b in range(B)]
    trees = api.trees_to_device(descs)
    # a threshold in the middle of the observed transition probabilities, so that both outcomes occur
    probs0 = oracle.tree_prune(lg[0], tok[0], st.parent[0], 0.0)["edge_prob"]
    tau = float(np.sort(probs0[1:])[len(probs0) // 2] * 1.5)
    out = dict(edge_prob=torch.zeros((B, T), device="cuda"), new_index=torch.zeros((B, T), dtype=torch.int32, device="cuda"),
               kept_nodes=torch.zeros((B, T), dtype=torch.int32, device="cuda"),
               kept_tokens=torch.zeros((B, T), dtype=torch.int32, device="cuda"))
    pruned = api.empty_trees(B)
    ws = api.workspace(api.ss_tree_prune_workspace_bytes(B, T, V))
    for rep in range(2):
        api.ss_tree_prune(torch.from_numpy(lg).cuda(), _i32(tok), trees, tau, out["edge_prob"], out["new_index"],
                          out["kept_nodes"], out["kept_tokens"], pruned, ws)
        assert api.ss_status(ws) == 0
        got = {k: v.cpu().numpy() for k, v in out.items()}
        pdesc = api.trees_from_device(pruned)
        n_dropped = 0
        for b in range(B):
            ref = oracle.tree_prune(lg[b], tok[b], st.parent[b], tau)
            np.testing.assert_allclose(got["edge_prob"][b], ref["edge_prob"], rtol=PROB_RTOL, atol=1e-30)
            dev_keep_edge = got["edge_prob"][b] >= np.float32(tau)      # the decision the device took, per edge
            clear = np.abs(ref["edge_prob"] - tau) > MARGIN * tau
            np.testing.assert_array_equal(dev_keep_edge[clear], (ref["edge_prob"] >= tau)[clear])
            follow = oracle.tree_prune(lg[b], tok[b], st.parent[b], tau, decide=dev_keep_edge.astype(np.uint8))
            n = len(follow["kept_nodes"])
            n_dropped += T - n
            np.testing.assert_array_equal(got["new_index"][b], follow["new_index"])
            np.testing.assert_array_equal(got["kept_nodes"][b, :n], follow["kept_nodes"])
            assert (got["kept_nodes"][b, n:] == -1).all()
            np.testing.assert_array_equal(got["kept_tokens"][b, :n], tok[b][follow["kept_nodes"]])
            assert _desc_fields(pdesc[b]) == _desc_fields(api.ss_tree_build(follow["new_parent"], c.gamma))
        assert 0 < n_dropped < B * T


# ---- soft and sampled verification ----------------------------------------------------------------------
def _verify_outputs(B):
    return dict(accept_len=torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                accept_path=torch.full((B, 64), -7, dtype=torch.int32, device="cuda"),
                last_node=torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                bonus_token=torch.full((B,), -7, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("name", ["tiny", "2.7b", "7b_ragged16"])
def test_soft_verification_matches_the_oracle(cuda, oracle, name):
    api = cuda
    st = W.make_step(W.CONFIGS[name])
    c = st.cfg
    B, T, V = c.batch, c.n_nodes, c.vocab
    lg = (st.logits() * 0.5).astype(np.float32)                          # flatter rows: the thresholds bite on some edges
    tok = st.draft_tokens.astype(np.int32)
    trees = api.trees_to_device([api.ss_tree_build(st.parent[b][:st.nodes(b)], c.gamma) for b in range(B)])
    eps, delta = 0.05, 0.3
    o = _verify_outputs(B)
    prob = torch.zeros((B, T), device="cuda")
    ent = torch.zeros((B, T), device="cuda")
    ws = api.workspace(api.ss_tree_prune_workspace_bytes(B, T, V))
    for rep in range(2):
        api.ss_tree_verify_soft(torch.from_numpy(lg).cuda(), _i32(tok), trees, eps, delta, o["accept_len"], o["accept_path"],
                                o["last_node"], o["bonus_token"], prob, ent, ws)
        assert api.ss_status(ws) == 0
        gp, ge = prob.cpu().numpy(), ent.cpu().numpy()
        lens = o["accept_len"].cpu().numpy()
        for b in range(B):
            ref = oracle.tree_verify_soft(lg[b], tok[b], st.parent[b], eps, delta, path_cap=64)
            np.testing.assert_allclose(gp[b], ref["edge_prob"], rtol=PROB_RTOL, atol=1e-30)
            np.testing.assert_allclose(ge[b], ref["node_entropy"], rtol=2e-5, atol=2e-5)
            par = st.parent[b]
            bar32 = np.minimum(np.float32(eps), np.float32(delta) * np.exp(-ge[b][np.maximum(par, 0)]).astype(np.float32))
            dev_ok = gp[b] >= bar32
            dev_ok[0] = True
            bar64 = np.minimum(eps, delta * np.exp(-ref["node_entropy"][np.maximum(par, 0)]))
            clear = np.abs(ref["edge_prob"] - bar64) > 10 * MARGIN * bar64
            clear[0] = False
            np.testing.assert_array_equal(dev_ok[clear], (ref["edge_prob"] >= bar64)[clear])
            follow = oracle.tree_verify_soft(lg[b], tok[b], par, eps, delta, decide=dev_ok.astype(np.uint8), path_cap=64)
            if clear[1:].all():
                assert int(lens[b]) == follow["accept_len"]
                np.testing.assert_array_equal(o["accept_path"][b].cpu().numpy(), follow["path"])
                assert int(o["last_node"][b]) == follow["last_node"]
                assert int(o["bonus_token"][b]) == follow["bonus_token"]
        assert lens.min() >= 1


@pytest.mark.parametrize("name,k", [("tiny", 3), ("1.3b", 8), ("7b", 4), ("7b_ragged16", 2)])
def test_sampled_verification_matches_the_oracle(cuda, oracle, name, k):
    api = cuda
    st = W.make_step(W.CONFIGS[name])
    c = st.cfg
    B, T, V = c.batch, c.n_nodes, c.vocab
    lg = st.logits()
    rng = np.random.default_rng(77 + k)
    u = rng.random((B, T)).astype(np.float32)
    # half of the children carry the token the oracle draws at their parent, so that paths get accepted
    tok = st.draft_tokens.astype(np.int32).copy()
    drawn_ref = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        drawn_ref[b] = oracle.tree_verify_sampled(lg[b], tok[b], st.parent[b], k, u[b], path_cap=64)["node_token"]
        for ch in range(1, T):
            if rng.random() < 0.5:
                tok[b, ch] = drawn_ref[b, st.parent[b][ch]]
    trees = api.trees_to_device([api.ss_tree_build(st.parent[b][:st.nodes(b)], c.gamma) for b in range(B)])
    o = _verify_outputs(B)
    node_token = torch.zeros((B, T), dtype=torch.int32, device="cuda")
    ws = api.workspace(api.ss_tree_verify_sampled_workspace_bytes(B, T, V))
    for rep in range(2):
        api.ss_tree_verify_sampled(torch.from_numpy(lg).cuda(), _i32(tok), trees, torch.from_numpy(u).cuda(), k,
                                   o["accept_len"], o["accept_path"], o["last_node"], o["bonus_token"], node_token, ws)
        assert api.ss_status(ws) == 0
        got_tok = node_token.cpu().numpy()
        n_same = 0
        for b in range(B):
            # the draw itself: equal to the oracle's unless u lies within rounding of a step of the distribution
            for t in range(T):
                idx = np.argsort(-lg[b, t], kind="stable")[:k]
                p = np.exp(lg[b, t, idx].astype(np.float64) - float(lg[b, t, idx[0]]))
                cdf = np.cumsum(p / p.sum())
                assert got_tok[b, t] in idx
                if np.min(np.abs(cdf - float(u[b, t]))) > 1e-5:
                    assert got_tok[b, t] == drawn_ref[b, t]
                    n_same += 1
            follow = oracle.tree_verify_sampled(lg[b], tok[b], st.parent[b], k, u[b], drawn=got_tok[b], path_cap=64)
            assert int(o["accept_len"][b]) == follow["accept_len"]
            np.testing.assert_array_equal(o["accept_path"][b].cpu().numpy(), follow["path"])
            assert int(o["last_node"][b]) == follow["last_node"]
            assert int(o["bonus_token"][b]) == follow["bonus_token"]
        assert n_same > 0.99 * B * T
        assert int(o["accept_len"].max()) >= 2


# ---- stream insertion and value rotation ------------------------------------------------------------------
@pytest.mark.parametrize("rows,gamma,hidden", [(64, 4, 4096), (1, 1, 8), (37, 3, 2560), (1024, 4, 4096), (0, 2, 64)])
def test_stream_insert_is_bit_exact(cuda, oracle, rows, gamma, hidden):
    api = cuda
    rng = np.random.default_rng(rows + hidden)
    m = W.f32_to_bf16_bits(rng.standard_normal((rows, hidden)).astype(np.float32) * 2)
    p = W.f32_to_bf16_bits(rng.standard_normal((gamma, hidden)).astype(np.float32) * 0.02)
    out = torch.zeros((rows, gamma, hidden), dtype=torch.bfloat16, device="cuda")
    api.ss_stream_insert(api.bf16_to_device(m) if rows else torch.zeros((0, hidden), dtype=torch.bfloat16, device="cuda"),
                         api.bf16_to_device(p), out)
    torch.cuda.synchronize()
    if rows:
        np.testing.assert_array_equal(api.bf16_to_host_bits(out), oracle.stream_insert(m, p))


@pytest.mark.parametrize("rows,gamma,width,eps", [(64 * 32, 4, 128, 0.01), (5, 1, 8, 0.3), (2048, 3, 80, 1.0 / 4100)])
def test_value_rotation_is_bit_exact(cuda, oracle, rows, gamma, width, eps):
    api = cuda
    rng = np.random.default_rng(rows + width)
    v = W.f32_to_bf16_bits(rng.standard_normal((rows, width)).astype(np.float32))
    out = torch.zeros((rows, gamma, width), dtype=torch.bfloat16, device="cuda")
    api.ss_value_rotate(api.bf16_to_device(v), out, eps)
    torch.cuda.synchronize()
    eps32 = float(np.float32(eps))                                       # the C ABI takes epsilon as fp32
    np.testing.assert_array_equal(api.bf16_to_host_bits(out), oracle.value_rotate(v, gamma, eps32))


def test_next_rows_reject_bad_arguments_before_launching(cuda):
    api = cuda
    lib, a = api.lib(), C.c_void_p(0x10000)
    assert lib.ss_next_draft(a, 1, None, a, 1, 5, 100, 2, 64, a, a, a, 1 << 20, None) == api.SS_ERR_UNSUPPORTED
    assert lib.ss_next_draft(a, 1, None, a, 1, 4, 100, 9, 64, a, a, a, 1 << 20, None) == api.SS_ERR_UNSUPPORTED
    assert lib.ss_next_draft(a, 1, None, a, 1, 4, 100, 2, 64, a, a, a, 16, None) == api.SS_ERR_WORKSPACE
    assert lib.ss_next_draft(None, 1, None, a, 1, 4, 100, 2, 64, a, a, a, 1 << 20, None) == api.SS_ERR_INVALID_ARG
    assert lib.ss_tree_prune(a, a, a, 1, 65, 100, 0.1, a, a, a, a, a, a, 1 << 20, None) == api.SS_ERR_UNSUPPORTED
    assert lib.ss_tree_verify_sampled(a, a, a, a, 1, 8, 100, 0, a, a, a, a, None, a, 1 << 20, None) == api.SS_ERR_INVALID_ARG
    assert lib.ss_stream_insert(a, a, a, 4, 2, 12, None) == api.SS_ERR_UNSUPPORTED
    assert lib.ss_value_rotate(a, a, 4, 5, 64, 0.1, None) == api.SS_ERR_UNSUPPORTED
