"""GPU parity: the CUDA verification step (through the C ABI) against the CPU oracle on the same seeded inputs.
Tolerances: log-probs within 2e-3 absolute; eta / path / tokens exact except decisions whose oracle margin is
below 1e-3, which are counted."""
import math

import numpy as np
import pytest
import torch

import mtad_synth as S
import paper_2407_09722_b200 as M
from paper_2407_09722_b200 import binding as Bn
from tests.parity import GpuModel, SeqCase, ParityStats, compare, run_gpu, LP_TOL, gemm_eps

pytestmark = pytest.mark.gpu

TINY = S.WORKLOADS["tiny"].target
GQA = S.ModelShape(2, 128, 4, 2, 32, 200, 96)
GQA64 = S.ModelShape(3, 192, 6, 2, 64, 328, 500)


def _u(seed, it, B, V):
    return S.bonus_uniforms(seed, it, B, V, "cuda")


def _root(seed, k, V):
    return int(S.token_ids(seed, (21 << 40) | k, 1, V)[0])


@pytest.fixture(scope="module")
def tiny():
    return GpuModel(TINY, max_batch=4, max_nodes=40, capacity=256)


@pytest.mark.parametrize("gamma,L", [(4, 32), (0, 32), (1, 0), (7, 5), (9, 100), (12, 64), (4, 200)])
def test_tiny_chain_matches_oracle(tiny, gamma, L):
    tiny.inject(0, L)
    stats = ParityStats()
    for it, tau in enumerate([0.1, 0.5, 0.9, 0.0]):
        tree = S.chain_tree(gamma, TINY.vocab, stream=it * 16 + gamma)
        case = SeqCase(0, L, _root(0, it, TINY.vocab), tree)
        compare(tiny, [case], Bn.log_tau(tau), _u(0, it, 1, TINY.vocab), chain=True, stats=stats)
        tiny.inject(0, L)
    assert stats.ok(), stats
    assert stats.cache_ok(TINY.layers, gemm_eps(gamma + 1, TINY.d_ffn))


@pytest.mark.parametrize("depth,width,keep,L", [(4, 4, 4, 32), (3, 8, 2, 7), (4, 8, 4, 130), (2, 16, 4, 0)])
def test_tiny_tree_matches_oracle(tiny, depth, width, keep, L):
    stats = ParityStats()
    for it, tau in enumerate([0.1, 0.4, 0.8]):
        tiny.inject(1, L)
        tree = S.beam_tree(depth, width, keep, TINY.vocab, stream=it * 64 + width)
        case = SeqCase(1, L, _root(1, it, TINY.vocab), tree)
        compare(tiny, [case], Bn.log_tau(tau), _u(1, it, 1, TINY.vocab), chain=False, stats=stats)
    assert stats.ok(), stats
    assert stats.cache_ok(TINY.layers, gemm_eps(1 + depth * width, TINY.d_ffn))


@pytest.mark.parametrize("shape", [GQA, GQA64])
def test_gqa_and_odd_shapes(shape):
    gm = GpuModel(shape, max_batch=2, max_nodes=24, capacity=160)
    stats = ParityStats()
    for it, (L, tau) in enumerate([(3, 0.2), (77, 0.6), (128, 0.05)]):
        gm.inject(0, L)
        tree = S.beam_tree(3, 8, 4, shape.vocab, stream=it)
        compare(gm, [SeqCase(0, L, _root(2, it, shape.vocab), tree)], Bn.log_tau(tau), _u(2, it, 1, shape.vocab),
                chain=False, stats=stats)
    assert stats.ok(), stats


def test_ragged_batch_of_trees_and_chains(tiny):
    # three sequences, different committed lengths, different node counts
    Ls = [10, 97, 64]
    cases = []
    for b, L in enumerate(Ls):
        tiny.inject(b, L)
        tree = S.beam_tree(4, 8, 4, TINY.vocab, stream=100 + b)
        cases.append(SeqCase(b, L, _root(3, b, TINY.vocab), tree, n_nodes=[32, 19, 8][b]))
    stats = compare(tiny, cases, math.log(0.3), _u(3, 0, 3, TINY.vocab), chain=False)
    assert stats.ok() and stats.n_seq == 3, stats
    cases = []
    for b, L in enumerate(Ls):
        tiny.inject(b, L)
        cases.append(SeqCase(b, L, _root(4, b, TINY.vocab), S.chain_tree(6, TINY.vocab, stream=200 + b)))
    stats = compare(tiny, cases, math.log(0.2), _u(4, 0, 3, TINY.vocab), chain=True)
    assert stats.ok() and stats.n_seq == 3, stats


def test_chain_shaped_tree_equals_chain_call(tiny):
    L = 40
    tree = S.chain_tree(5, TINY.vocab, stream=7)
    u = _u(5, 0, 1, TINY.vocab)
    tiny.inject(0, L)
    a = run_gpu(tiny, [SeqCase(0, L, 11, tree)], math.log(0.3), u, chain=True, commit=False).host()
    tiny.inject(0, L)
    b = run_gpu(tiny, [SeqCase(0, L, 11, tree)], math.log(0.3), u, chain=False, commit=False).host()
    for k in ("eta", "winner", "n_out", "node_lp", "node_LP", "row_lse", "row_cand", "margin"):
        assert torch.equal(a[k], b[k]), k
    eta = int(a["eta"][0])
    assert torch.equal(a["out_tok"][0, :eta + 1], b["out_tok"][0, :eta + 1])


def test_runs_are_bit_reproducible(tiny):
    L = 90
    tree = S.beam_tree(4, 8, 4, TINY.vocab, stream=9)
    u = _u(6, 0, 1, TINY.vocab)
    outs = []
    for _ in range(2):
        tiny.inject(2, L)
        outs.append(run_gpu(tiny, [SeqCase(2, L, 5, tree)], math.log(0.3), u, chain=False, commit=False).host())
    for k in outs[0]:
        assert torch.equal(outs[0][k], outs[1][k]), k


def test_multi_iteration_decode_stays_on_the_oracle_trajectory(tiny):
    """16 teacher-free iterations from an empty cache: prefill as tau=0 chains, then verify+commit each step; the
    oracle replays the same drafts and must see the same tokens and lengths."""
    from oracle import mtad_oracle as O
    seq = 3
    prompt = S.token_ids(0, 77, 33, TINY.vocab).tolist()
    ctx = tiny.ctx
    ctx.mtad_seq_set(seq, 0, prompt[0])
    ocache = np.zeros((TINY.layers, 2, TINY.n_kv_heads, tiny.capacity, TINY.head_dim), np.uint16)
    model = tiny.oracle()
    # prefill: root = prompt[i], then up to 8 following prompt tokens as a chain that tau = 0 accepts whole
    L, i = 0, 0
    u = _u(7, 0, 1, TINY.vocab)
    while i < len(prompt):
        root = prompt[i]
        chunk = prompt[i + 1:i + 9]
        ctx.mtad_seq_set(seq, L, root)
        g = len(chunk)
        tok = torch.tensor(chunk, dtype=torch.int32, device="cuda") if g else None
        lq = torch.zeros(g, dtype=torch.float32, device="cuda") if g else None
        res = M.ResultBuffers(1, g, g)
        ctx.mtad_verify_chain([seq], g, tok, lq, -math.inf, u, res)
        ctx.kv_commit([seq], res)
        assert int(res.eta.cpu()[0]) == g
        r = O.verify_chain(model, ocache, L, root, chunk, np.zeros(g), -math.inf, u.cpu().numpy()[0])
        assert r.eta == g
        L = O.kv_commit(ocache, L, r.path)
        i = L
        root = r.out_tok[-1]               # after the last chunk: the first generated token
    assert L == len(prompt)
    ctx.mtad_seq_set(seq, L, root)
    near = 0
    for it in range(16):
        tree = S.chain_tree(4, TINY.vocab, stream=500 + it)
        u = _u(8, it, 1, TINY.vocab)
        tok = torch.tensor(tree.tok, dtype=torch.int32, device="cuda")
        lq = torch.tensor(tree.logq, dtype=torch.float32, device="cuda")
        res = M.ResultBuffers(1, 4, 4)
        ctx.mtad_verify_chain([seq], 4, tok, lq, math.log(0.1), u, res)
        ctx.kv_commit([seq], res)
        h = res.host()
        r = O.verify_chain(model, ocache, L, root, tree.tok, np.asarray(tree.logq, np.float32).astype(np.float64),
                           math.log(0.1), u.cpu().numpy()[0])
        L = O.kv_commit(ocache, L, r.path)
        root = r.out_tok[-1]
        if min(r.margin_accept, r.margin_bonus) < 1e-3:
            near += 1
            ctx.mtad_seq_set(seq, L, root)          # re-synchronise after a near tie
            continue
        eta = int(h["eta"][0])
        assert eta == r.eta and h["out_tok"][0, :eta + 1].tolist() == r.out_tok, it
        assert np.max(np.abs(h["out_lp"][0, :eta + 1].numpy() - np.asarray(r.out_lp))) < LP_TOL
        assert ctx.mtad_seq_get(seq) == (L, root)
    assert near <= 2


def test_device_side_rejections(tiny):
    L = 20
    tiny.inject(0, L)
    tiny.ctx.mtad_seq_set(0, L, 3)
    u = _u(9, 0, 1, TINY.vocab)
    N, D = 4, 4
    ref = torch.zeros(1, D, device="cuda")
    res = M.ResultBuffers(1, N, D)

    def call(tok, par, nn=None, D_=D):
        t = torch.tensor([tok], dtype=torch.int32, device="cuda")
        p = torch.tensor([par], dtype=torch.int32, device="cuda")
        n = None if nn is None else torch.tensor([nn], dtype=torch.int32, device="cuda")
        tiny.ctx.mtad_verify_tree([0], n, N, D_, t, p, ref, math.log(0.5), u, res)
        rc = tiny.ctx.kv_commit([0], res)
        torch.cuda.synchronize()
        return int(res.status.cpu()[0])

    assert call([1, 2, 3, 4], [-1, 0, 2, 1]) & Bn.ST_BAD_PARENT          # parent[2] = 2 is not < 2
    assert tiny.ctx.mtad_seq_get(0) == (L, 3)                              # commit left the sequence alone
    assert call([1, 2, 3, 4], [-1, -2, 0, 1]) & Bn.ST_BAD_PARENT
    assert call([1, 2, TINY.vocab, 4], [-1, 0, 1, 2]) & Bn.ST_BAD_TOKEN
    assert call([1, 2, 3, 4], [-1, 0, 1, 2], nn=5) & Bn.ST_BAD_COUNT
    assert call([1, 2, 3, 4], [-1, 0, 1, 2], D_=3) & Bn.ST_TOO_DEEP
    tiny.ctx.mtad_seq_set(0, tiny.capacity - 3, 3)
    assert call([1, 2, 3, 4], [-1, 0, 1, 2]) & Bn.ST_KV_OVERFLOW
    tiny.ctx.mtad_seq_set(0, L, 3)
    assert call([1, 2, 3, 4], [-1, 0, 1, 2]) == 0


def test_host_side_rejections(tiny):
    u = _u(9, 1, 1, TINY.vocab)
    res = M.ResultBuffers(1, 4, 4)
    tok = torch.zeros(1, 4, dtype=torch.int32, device="cuda")
    lq = torch.zeros(1, 4, device="cuda")
    c = tiny.ctx
    assert c.mtad_verify_chain([0], 4, tok, lq, 0.0, u, res, check=False) == Bn.MTAD_E_INVALID        # tau = 1
    assert c.mtad_verify_chain([0], 4, tok, lq, math.nan, u, res, check=False) == Bn.MTAD_E_INVALID
    assert c.mtad_verify_chain([0], 4, tok, lq, 0.5, u, res, check=False) == Bn.MTAD_E_INVALID        # tau > 1
    assert c.mtad_verify_chain([9], 4, tok, lq, -1.0, u, res, check=False) == Bn.MTAD_E_INVALID       # bad sequence
    assert c.mtad_verify_chain([0, 0], 4, tok, lq, -1.0, u, res, check=False) == Bn.MTAD_E_INVALID    # duplicate
    assert c.mtad_verify_chain([0], 41, tok, lq, -1.0, u, res, check=False) == Bn.MTAD_E_CAPACITY
    assert c.mtad_verify_chain([0], 4, None, lq, -1.0, u, res, check=False) == Bn.MTAD_E_INVALID
    assert c.kv_commit([0], res, check=False) == Bn.MTAD_E_INVALID                                    # nothing to commit
    with pytest.raises(M.MtadError):
        c.mtad_seq_set(0, tiny.capacity + 1, 0)


@pytest.mark.parametrize("path", ["tc", "simt", "warped"])
def test_non_finite_logits_set_a_status_bit(path, monkeypatch):
    """A NaN in the committed cache makes every logit of the sequence NaN: no arg-max candidate exists.  The call
    must report MTAD_ST_NONFINITE for that sequence (and leave the other one alone), not index with the missing
    candidate."""
    if path == "simt":
        monkeypatch.setenv("MTAD_PATH", "simt")
    gm = GpuModel(TINY, max_batch=2, max_nodes=8, capacity=96)
    for seq in range(2):
        gm.inject(seq, 40)
    gm.cache[0, 1, 0, 0, 3, 5] = float("nan")           # layer 0, sequence 1, K, head 0, position 3
    cases = [SeqCase(seq, 40, 3 + seq, S.chain_tree(4, TINY.vocab, stream=90 + seq)) for seq in range(2)]
    res = run_gpu(gm, cases, math.log(0.1), _u(6, 0, 2, TINY.vocab), chain=True,
                  warp=(10, 0.9) if path == "warped" else None)
    h = res.host()
    assert int(h["status"][0]) == 0 and int(h["n_out"][0]) >= 1
    assert int(h["status"][1]) & Bn.MTAD_ST_NONFINITE and int(h["n_out"][1]) == 0
    assert gm.ctx.mtad_seq_get(1) == (40, 4)              # nothing committed for the flagged sequence


def test_result_head_is_one_contiguous_copy(tiny):
    """The members a decode loop reads back every step (eta, n_out, status, out_tok, out_lp) lie in one block: a
    single device-to-host copy of `head` gives the same values as the member-by-member copies."""
    tiny.inject(0, 50)
    res = run_gpu(tiny, [SeqCase(0, 50, 8, S.chain_tree(5, TINY.vocab, stream=123))], math.log(0.1),
                  _u(7, 0, 1, TINY.vocab), chain=True)
    h = res.host()
    hv = res.head_views(res.head.cpu())
    assert set(hv) == {"eta", "n_out", "status", "out_tok", "out_lp"}
    for name, v in hv.items():
        assert torch.equal(v, h[name]), name


def test_empty_attention_splits_ignore_stale_partials():
    """A ragged batch in which the short sequence leaves whole key splits without keys: their partial outputs are
    never written, so whatever an earlier call (of another shape, for instance a draft) left in that scratch must not
    reach the result - here the scratch is filled with NaN beforehand."""
    gm = GpuModel(TINY, max_batch=2, max_nodes=8, capacity=256)
    stats = ParityStats()
    for it, (La, Lb) in enumerate([(200, 5), (3, 190)]):
        gm.inject(0, La)
        gm.inject(1, Lb)
        gm.ctx.region("attn_part", torch.float32).fill_(float("nan"))
        cases = [SeqCase(0, La, _root(3, it, TINY.vocab), S.chain_tree(4, TINY.vocab, stream=300 + it)),
                 SeqCase(1, Lb, _root(4, it, TINY.vocab), S.chain_tree(4, TINY.vocab, stream=310 + it))]
        compare(gm, cases, Bn.log_tau(0.2), _u(7, it, 2, TINY.vocab), chain=True, stats=stats)
    assert stats.ok() and stats.near_ties <= 1, stats
