"""The no-allocation entry point, mtad_verify_chain_static.

Some users of the library cannot allocate device memory at the moment they need a verification step (they live
inside another engine's memory pool, or their allocator is frozen), so they cannot give mtad_create a workspace.
For them the library carries a fixed scratch array.  This test calls that entry point through the C ABI twice in
a row - the second call finds the first call's leftovers in the array - and checks every output against
mtad_verify_chain on an ordinary context with a caller-allocated workspace and against the CPU oracle, within the
tolerance of the parity tests.  A second test changes the chain length between two calls issued back to back on a
non-blocking stream, which makes the library lay the array out afresh while the first call may still be running.
It lives in its own file, collected last, so that a failure here cannot hide the other tests."""
import math

import pytest
import torch

import numpy as np

import mtad_synth as S
import paper_2407_09722_b200 as M
from oracle import mtad_oracle as O
from paper_2407_09722_b200 import binding as Bn
from paper_2407_09722_b200.runtime import DeviceModel
from tests.parity import GpuModel

pytestmark = pytest.mark.gpu
LP_TOL = 2e-3


def test_static_scratch_matches_workspace_path_twice_in_a_row():
    shape = S.WORKLOADS["tiny"].target
    gamma, L = 4, 48
    dm = GpuModel(shape, max_batch=1, max_nodes=gamma, capacity=128)
    V = shape.vocab
    for call, tau in enumerate([0.1, 0.6]):
        tree = S.chain_tree(gamma, V, stream=900 + call)
        tok = torch.tensor(tree.tok, dtype=torch.int32, device="cuda")
        lq = torch.tensor(tree.logq, dtype=torch.float32, device="cuda")
        u = S.bonus_uniforms(3, call, 1, V, "cuda")
        root = 5 + call
        dm.inject(0, L)
        want = M.ResultBuffers(1, gamma, gamma)
        dm.ctx.mtad_seq_set(0, L, root)
        dm.ctx.mtad_verify_chain([0], gamma, tok, lq, math.log(tau), u, want)
        torch.cuda.synchronize()
        w = want.host()
        got = M.ResultBuffers(1, gamma, gamma)
        rc = Bn.mtad_verify_chain_static(dm.desc, L, root, gamma, tok, lq, math.log(tau), u, got)
        assert rc == Bn.MTAD_OK, rc
        torch.cuda.synchronize()
        g = got.host()
        assert int(g["status"][0]) == 0
        for k in ("eta", "winner", "n_out", "row_cand"):
            assert torch.equal(g[k], w[k]), k
        eta = int(w["eta"][0])
        assert torch.equal(g["out_tok"][0, :eta + 1], w["out_tok"][0, :eta + 1])
        assert torch.equal(g["path"][0, :eta], w["path"][0, :eta])
        for k in ("node_lp", "node_LP", "row_lse", "row_cand_lp"):
            assert torch.max(torch.abs(g[k] - w[k])).item() <= LP_TOL, k
        assert torch.max(torch.abs(g["out_lp"][0, :eta + 1] - w["out_lp"][0, :eta + 1])).item() <= LP_TOL
        _against_oracle(dm, g, L, root, tree, tau, u)


def _against_oracle(gm, g, L, root, tree, tau, u):
    """The static call's outputs against the oracle's verify_chain on the cache as it was before the call."""
    cache = gm.cache_bits(0, L)
    r = O.verify_chain(gm.oracle(), cache, L, root, tree.tok, np.asarray(tree.logq, np.float32).astype(np.float64),
                       math.log(tau), u[0].cpu().numpy())
    n = len(tree.tok)
    assert np.max(np.abs(g["node_lp"][0, :n].numpy() - np.asarray(r.node_lp))) <= LP_TOL
    assert np.max(np.abs(g["node_LP"][0, :n].numpy() - np.asarray(r.node_LP))) <= LP_TOL
    if min(r.margin_accept, r.margin_tie, r.margin_bonus) >= 1e-3:
        assert int(g["eta"][0]) == r.eta
        assert g["out_tok"][0, :r.eta + 1].tolist() == r.out_tok


def test_static_scratch_relayout_on_a_non_blocking_stream():
    """Call 1 with gamma 4 and call 2 with gamma 3 on one non-blocking stream, no synchronisation in between: the
    second call re-carves and re-zeroes the array, which must not overlap the first call's kernels."""
    shape = S.WORKLOADS["tiny"].target
    L, V = 40, shape.vocab
    gm = GpuModel(shape, max_batch=1, max_nodes=4, capacity=128)
    gm.inject(0, L)
    before = gm.cache_bits(0, L)
    st = torch.cuda.Stream()
    calls = []
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        for call, gamma in enumerate([4, 3, 4]):
            tree = S.chain_tree(gamma, V, stream=930 + call)
            tok = torch.tensor(tree.tok, dtype=torch.int32, device="cuda")
            lq = torch.tensor(tree.logq, dtype=torch.float32, device="cuda")
            u = S.bonus_uniforms(4, call, 1, V, "cuda")
            got = M.ResultBuffers(1, gamma, gamma)
            calls.append((tree, tok, lq, u, got, gamma))
        st.synchronize()
        for call, (tree, tok, lq, u, got, gamma) in enumerate(calls):
            rc = Bn.mtad_verify_chain_static(gm.desc, L, 9, gamma, tok, lq, math.log(0.2), u, got, stream=st)
            assert rc == Bn.MTAD_OK, rc
    st.synchronize()
    for tree, tok, lq, u, got, gamma in calls:
        g = got.host()
        assert int(g["status"][0]) == 0
        r = O.verify_chain(gm.oracle(), before.copy(), L, 9, tree.tok,
                           np.asarray(tree.logq, np.float32).astype(np.float64), math.log(0.2), u[0].cpu().numpy())
        assert np.max(np.abs(g["node_lp"][0, :gamma].numpy() - np.asarray(r.node_lp))) <= LP_TOL
        if min(r.margin_accept, r.margin_tie, r.margin_bonus) >= 1e-3:
            assert int(g["eta"][0]) == r.eta and g["out_tok"][0, :r.eta + 1].tolist() == r.out_tok


def test_static_scratch_rejects_what_does_not_fit():
    shape = S.WORKLOADS["tiny"].target
    dm = DeviceModel(shape, max_batch=1, max_nodes=4, capacity=64)
    res = M.ResultBuffers(1, 255, 32)
    u = S.bonus_uniforms(3, 9, 1, shape.vocab, "cuda")
    tok = torch.zeros(255, dtype=torch.int32, device="cuda")
    lq = torch.zeros(255, dtype=torch.float32, device="cuda")
    # a huge shape needs more scratch than the built-in array: clear error, nothing launched
    big = S.WORKLOADS["70b_gqa_tree"].target
    d = Bn.ModelDesc(big.layers, big.d_model, big.n_q_heads, big.n_kv_heads, big.head_dim, big.d_ffn, big.vocab,
                     big.rope_base, big.rms_eps, dm.desc.embed, dm.desc.lm_head, dm.desc.final_norm,
                     dm.desc.layer_weights, dm.desc.kv_cache, 64)
    assert Bn.mtad_verify_chain_static(d, 0, 1, 32, tok, lq, -1.0, u, res) == Bn.MTAD_E_WORKSPACE
    assert Bn.mtad_verify_chain_static(dm.desc, 0, 1, -1, tok, lq, -1.0, u, res) == Bn.MTAD_E_INVALID
