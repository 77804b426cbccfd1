"""The verification entry point that needs no caller-provided scratch (ss_tree_verify_static).

Callers that cannot allocate device memory where they call the library use it: its scratch is a
fixed array inside the library.  It must give exactly what ss_tree_verify gives (integer outputs,
bit-exact), also when called twice in a row, because the shared array keeps the previous call's
contents.  This file sorts last so that a failure here cannot hide another test's result."""
import ctypes as C

import numpy as np
import pytest

from paper_2402_11131_b200 import workloads as W

torch = pytest.importorskip("torch")


def _outputs(B, T):
    return dict(accept_len=torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                accept_path=torch.full((B, 64), -7, dtype=torch.int32, device="cuda"),
                last_node=torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                bonus_token=torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                node_argmax=torch.full((B, T), -7, dtype=torch.int32, device="cuda"))


@pytest.mark.gpu
def test_static_scratch_verify_matches_workspace_verify_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2402_11131_b200 import api, build
    build.build()
    names = ["7b", "1.3b"]                      # two different shapes share the one static array
    for call, name in enumerate(names + names):
        cfg = W.CONFIGS[name]
        st = W.make_step(cfg)
        B, T, V = cfg.batch, cfg.n_nodes, cfg.vocab
        logits = torch.from_numpy(st.logits()).cuda()
        tokens = torch.from_numpy(st.draft_tokens.astype(np.int32)).cuda()
        trees = api.trees_to_device([api.ss_tree_build(st.parent[b], cfg.gamma) for b in range(B)])
        ws = api.workspace(api.ss_tree_verify_workspace_bytes(B, T, V))
        ref, got = _outputs(B, T), _outputs(B, T)
        api.ss_tree_verify(logits, tokens, trees, ref["accept_len"], ref["accept_path"], ref["last_node"],
                           ref["bonus_token"], ref["node_argmax"], ws)
        assert api.ss_status(ws) == 0
        if call == 0:                           # the first call on a device looks up the array's address
            api.ss_tree_verify_static(logits, tokens, trees, got["accept_len"], got["accept_path"], got["last_node"],
                                      got["bonus_token"], got["node_argmax"])
            torch.cuda.synchronize()
        # neither the caching allocator nor the driver hands out memory during the call: free device memory
        # (as the driver reports it) and the allocator's count are the same before and after
        mem_before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
        api.ss_tree_verify_static(logits, tokens, trees, got["accept_len"], got["accept_path"], got["last_node"],
                                  got["bonus_token"], got["node_argmax"])
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == mem_before
        assert torch.cuda.mem_get_info()[0] == free_before
        for k in ref:
            assert torch.equal(ref[k], got[k]), (call, name, k)
        assert int(got["accept_len"].min()) >= 1
        # and both agree with the CPU oracle
        import oracle
        oracle.build()
        lg = st.logits()
        for b in range(B):
            r = oracle.tree_verify(lg[b], st.draft_tokens[b], st.parent[b], path_cap=api.SS_PATH_STRIDE)
            assert int(got["accept_len"][b]) == r["accept_len"] and int(got["bonus_token"][b]) == r["bonus_token"]
            assert np.array_equal(got["accept_path"][b].cpu().numpy(), r["path"])


@pytest.mark.gpu
def test_static_scratch_verify_rejects_sizes_beyond_its_array():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2402_11131_b200 import api
    B, T, V = 64, 64, 200000                   # 64 * 64 * 49 chunks * 8 B > 1 MiB
    assert api.ss_tree_verify_workspace_bytes(B, T, V) > api.SS_VERIFY_STATIC_SCRATCH_BYTES
    a = C.c_void_p(0x10000)
    rc = api.lib().ss_tree_verify_static(a, a, a, B, T, V, a, a, a, a, None, None)
    assert rc == api.SS_ERR_WORKSPACE


def test_static_scratch_verify_argument_checks_need_no_gpu():
    from paper_2402_11131_b200 import api, build
    build.build()
    a = C.c_void_p(0x10000)
    lib = api.lib()
    assert lib.ss_tree_verify_static(None, a, a, 1, 4, 100, a, a, a, a, None, None) == api.SS_ERR_INVALID_ARG
    assert lib.ss_tree_verify_static(a, a, a, 1, 65, 100, a, a, a, a, None, None) == api.SS_ERR_UNSUPPORTED
    assert lib.ss_tree_verify_static(a, a, a, 64, 64, 200000, a, a, a, a, None, None) == api.SS_ERR_WORKSPACE
