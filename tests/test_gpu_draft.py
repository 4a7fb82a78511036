"""mtad_draft (beam sampling with the auxiliary model) and the auxiliary cache roll-forward against the oracle's
draft_beam / aux_commit, through whole draft -> verify -> commit iterations."""
import math

import numpy as np
import pytest
import torch

import mtad_synth as S
import paper_2407_09722_b200 as M
from oracle import mtad_oracle as O
from tests.parity import GpuModel, LP_TOL

pytestmark = pytest.mark.gpu
W = S.WORKLOADS["tiny"]


def draft_gap(keep_all: bool) -> float:
    """Smallest gap between two consecutive perturbed scores of the oracle's draft below which the device's order of
    them is not compared.  The plain tree orders b pairs a layer: 1e-3, the margin of every other decision.  With
    every candidate kept a layer orders b * b of them, and the k-th and (k+1)-th largest of V Gumbel-perturbed scores
    lie about 1/k apart, so some gap among gamma * b * b falls below 1e-3 in most drafts and that margin would skip
    nearly every case.  The device's error on one perturbed score is that of an fp32 logit of the auxiliary model
    (one narrow layer here: the node_logq comparison below measures at most 5e-6 against the fp64 oracle and asserts 2e-5
    on it), so 1e-4 still leaves a factor of five."""
    return 1e-4 if keep_all else 1e-3


# A draft on warped rows takes two more decisions per beam row (the top-k boundary in logits, the top-p cut in
# probability), 1 + (gamma - 1) b rows a draft.  On the random-init auxiliary model the rows are nearly flat (the 10th
# and 11th largest logit of 1024 lie 1e-3..3e-2 apart), so the closest of a draft's decisions is within 1e-3 in five
# drafts of six; as for the candidate order above, the comparison goes down to 1e-4, five times the asserted error of
# the device's logits.
DRAFT_WARP_MARGIN = 1e-4


def _draft_gpu(gm, seq, gamma, b, u, keep_all=False, warped=False):
    N = gamma * (b * b if keep_all else b)
    i32 = dict(dtype=torch.int32, device="cuda")
    f32 = dict(dtype=torch.float32, device="cuda")
    out = {"tok": torch.zeros(1, N, **i32), "parent": torch.zeros(1, N, **i32), "depth": torch.zeros(1, N, **i32),
           "node_logq": torch.zeros(1, N, **f32), "logq_ref": torch.zeros(1, gamma, **f32),
           "best_path": torch.zeros(1, gamma, **i32), "n_nodes": torch.full((1,), -7, **i32)}
    gm.ctx.mtad_draft([seq], gamma, b, u, out["tok"], out["parent"], out["depth"], out["node_logq"], out["logq_ref"],
                      out["best_path"], keep_all_candidates=keep_all, n_nodes=out["n_nodes"])
    torch.cuda.synchronize()
    assert warped or out["n_nodes"].tolist() == [N]
    return out


# the last four keep every candidate of the beam sampling: 64-, 12- and 128-node trees (Sec. 3.3 with the tree sizes
# of the full-size workloads), and the output sequence of such a draft verified as a chain
# the cases with a (top_k, top_p) pair draft from warped auxiliary rows (App. F): top-10 with top_p 0.85 (on a random-init
# model the ten kept tokens are almost equally likely, so a cut at 0.9 sits on the ninth partial sum and every draft
# would count as a near tie); two kept tokens a
# row, so that the first layers hold fewer nodes than the beam width; greedy rows (a single chain whatever the beam
# width); every candidate kept on warped rows; the output sequence of a warped draft verified as a chain
@pytest.mark.parametrize("gamma,b,chain,keep_all,warp", [
    (4, 4, False, False, None), (3, 2, True, False, None), (4, 1, True, False, None), (2, 8, False, False, None),
    (4, 4, False, True, None), (3, 2, False, True, None), (2, 8, False, True, None), (3, 3, True, True, None),
    (4, 4, False, False, (10, 0.85)), (3, 3, False, False, (2, 1.0)), (3, 3, False, False, (1, 1.0)),
    (3, 3, False, True, (5, 0.9)), (4, 4, True, False, (10, 0.85))])
def test_draft_verify_commit_iterations(gamma, b, chain, keep_all, warp):
    N = gamma * (b * b if keep_all else b)
    gm = GpuModel(W.target, max_batch=2, max_nodes=max(40, N), capacity=320, aux=W.aux, aux_capacity=320)
    seq, L = 1, 24
    gm.inject(seq, L)
    gm.inject_aux(seq, L)
    root = 5
    gm.ctx.mtad_seq_set(seq, L, root, aux_len=L)
    if warp:
        gm.ctx.mtad_set_draft_warp(*warp)
    tcache = gm.cache_bits(seq, L)
    acache = gm.aux_cache_bits(seq, L)
    La, pend = L, [root]
    V = W.target.vocab
    skipped = 0
    leaves = 0                  # accepted paths that end in a node the auxiliary model never ran
    lq_err = 0.0
    sizes = set()
    for it in range(6):
        u = S.uniforms(0, (31 << 40) | (it * 16 + gamma), gamma * b * V, "cuda").view(1, gamma, b, V)
        g = _draft_gpu(gm, seq, gamma, b, u, keep_all, warped=warp is not None)
        dr = O.draft_beam(gm.oracle_aux(), acache, La, pend, gamma, b, u[0].cpu().numpy(), keep_all=keep_all, warp=warp)
        n = len(dr.tok)                              # (on warped rows a layer may hold fewer nodes than it has room for)
        assert n == N or (warp and n < N)
        sizes.add(n)
        near = dr.min_gap < draft_gap(keep_all) or dr.margin_warp < DRAFT_WARP_MARGIN
        if not near:
            assert g["n_nodes"].tolist() == [n]
            assert g["tok"][0, :n].tolist() == dr.tok and g["parent"][0, :n].tolist() == dr.parent
            assert g["depth"][0, :n].tolist() == dr.depth and g["best_path"][0].tolist() == dr.best_path
            lq_err = max(lq_err, float(np.max(np.abs(g["node_logq"][0, :n].cpu().numpy() - np.asarray(dr.logq)))))
            assert np.max(np.abs(g["node_logq"][0, :n].cpu().numpy() - np.asarray(dr.logq))) < LP_TOL
            assert np.max(np.abs(g["logq_ref"][0].cpu().numpy() - np.asarray(dr.logq_ref))) < LP_TOL
        # The device verifies its own draft, straight from the arrays mtad_draft wrote; next to a tie of the draft
        # it gets the oracle's instead (and its caches are put back on the oracle's trajectory afterwards).
        bu = S.bonus_uniforms(9, it, 1, V, "cuda")
        log_tau = math.log(0.3)
        ref = np.asarray(dr.logq_ref, np.float32)
        d_ref = g["logq_ref"] if not near else torch.tensor(ref, device="cuda").view(1, -1)
        if chain:
            toks = [dr.tok[n] for n in dr.best_path]
            res = M.ResultBuffers(1, gamma, gamma)
            gm.ctx.mtad_verify_chain([seq], gamma, torch.tensor(toks, dtype=torch.int32, device="cuda"), d_ref,
                                     log_tau, bu, res)
            r = O.verify_chain(gm.oracle(), tcache, L, root, toks, ref.astype(np.float64), log_tau, bu[0].cpu().numpy())
            accepted = [dr.best_path[i] for i in r.path]
        else:
            res = M.ResultBuffers(1, N, gamma)
            pad = [0] * (N - n)
            d_tok = g["tok"] if not near else torch.tensor(dr.tok + pad, dtype=torch.int32, device="cuda")
            d_par = g["parent"] if not near else torch.tensor(dr.parent + pad, dtype=torch.int32, device="cuda")
            d_n = g["n_nodes"] if not near else torch.tensor([n], dtype=torch.int32, device="cuda")
            gm.ctx.mtad_verify_tree([seq], d_n, N, gamma, d_tok, d_par, d_ref, log_tau, bu, res)
            r = O.verify_tree(gm.oracle(), tcache, L, root, dr.tok, dr.parent, ref.astype(np.float64), log_tau,
                              bu[0].cpu().numpy())
            accepted = list(r.path)
        gm.ctx.kv_commit([seq], res)
        h = res.host()
        # (next to a tie of the draft the device rolls its auxiliary cache forward by its own tree, which the verified
        # one need not be: a range flag is possible there and the state is replaced below anyway)
        assert int(h["status"][0]) == 0 or near
        tie = min(r.margin_accept, r.margin_tie, r.margin_bonus) < 1e-3
        L = O.kv_commit(tcache, L, r.path)
        La, pend = O.aux_commit(acache, La, pend, dr, accepted, r.out_tok[-1], gamma)
        leaves += len(pend) == 2
        root = r.out_tok[-1]
        if near or tie:
            # a decision within 1e-3 of a tie may legitimately differ: put the device back on the oracle's trajectory
            skipped += 1
            gm.upload(seq, tcache, acache)
            gm.ctx.mtad_seq_set(seq, L, root, aux_len=La, pending_tok=pend[:-1])
            continue
        assert int(h["eta"][0]) == r.eta and h["out_tok"][0, :r.eta + 1].tolist() == r.out_tok
        assert gm.ctx.mtad_seq_get(seq) == (L, root)
    print(f"keep_all={keep_all} gamma={gamma} b={b} warp={warp}: skipped {skipped}, paths ending in a not-run node {leaves}, "
          f"largest node_logq error {lq_err:.2e}, tree sizes {sorted(sizes)}")
    assert skipped <= (4 if warp else 3) and lq_err < 2e-5
    assert gm.ctx.mtad_debug_check_canaries() == ""


def test_draft_wide_vocabulary():
    """Vocabulary 32000: the selection runs over 32 chunks per beam row, as at full size."""
    target = S.ModelShape(1, 128, 2, 2, 64, 344, 32000)
    aux = S.ModelShape(1, 128, 2, 2, 64, 512, 32000)
    gm = GpuModel(target, max_batch=1, max_nodes=16, capacity=128, aux=aux, aux_capacity=128)
    L, root, gamma, b = 20, 7, 3, 4
    gm.inject(0, L)
    gm.inject_aux(0, L)
    gm.ctx.mtad_seq_set(0, L, root, aux_len=L)
    acache = gm.aux_cache_bits(0, L)
    skipped = 0
    for it in range(3):
        u = S.uniforms(0, (33 << 40) | it, gamma * b * 32000, "cuda").view(1, gamma, b, 32000)
        g = _draft_gpu(gm, 0, gamma, b, u)
        dr = O.draft_beam(gm.oracle_aux(), acache, L, [root], gamma, b, u[0].cpu().numpy())
        if dr.min_gap < 1e-3:
            skipped += 1
        else:
            assert g["tok"][0].tolist() == dr.tok and g["parent"][0].tolist() == dr.parent
            assert g["best_path"][0].tolist() == dr.best_path
            assert np.max(np.abs(g["node_logq"][0].cpu().numpy() - np.asarray(dr.logq))) < LP_TOL
            assert np.max(np.abs(g["logq_ref"][0].cpu().numpy() - np.asarray(dr.logq_ref))) < LP_TOL
        gm.ctx.mtad_seq_set(0, L, root, aux_len=L)          # the same state again: only the noise changes
    assert skipped <= 1


def test_draft_rejects_bad_arguments():
    gm = GpuModel(W.target, max_batch=1, max_nodes=40, capacity=128, aux=W.aux, aux_capacity=128)
    V = W.target.vocab
    u = torch.full((1, 4, 4, V), 0.5, device="cuda")
    i32 = dict(dtype=torch.int32, device="cuda")
    t = torch.zeros(1, 64, **i32)
    f = torch.zeros(1, 64, device="cuda")
    c = gm.ctx
    assert c.mtad_draft([0], 0, 4, u, t, t, t, f, f, t, check=False) == M.binding.MTAD_E_INVALID
    assert c.mtad_draft([0], 4, 9, u, t, t, t, f, f, t, check=False) == M.binding.MTAD_E_CAPACITY
    assert c.mtad_draft([0], 33, 1, u, t, t, t, f, f, t, check=False) == M.binding.MTAD_E_CAPACITY
    assert c.mtad_draft([3], 4, 4, u, t, t, t, f, f, t, check=False) == M.binding.MTAD_E_INVALID
    # every candidate kept: gamma * b * b nodes must fit a verify call
    assert c.mtad_draft([0], 4, 8, u, t, t, t, f, f, t, check=False, keep_all_candidates=True) == M.binding.MTAD_E_CAPACITY
    # warped rows: limits as for the target's warping; the node count becomes a required output
    assert c.mtad_set_draft_warp(17, 0.9, check=False) == M.binding.MTAD_E_CAPACITY
    assert c.mtad_set_draft_warp(10, 0.0, check=False) == M.binding.MTAD_E_INVALID
    assert c.mtad_set_draft_warp(10, 0.9, check=False) == 0
    assert c.mtad_draft([0], 4, 4, u, t, t, t, f, f, t, check=False) == M.binding.MTAD_E_INVALID       # no n_nodes
    assert c.mtad_set_draft_warp(0, 1.0, check=False) == 0
    no_aux = GpuModel(W.target, max_batch=1, max_nodes=8, capacity=64)
    assert no_aux.ctx.mtad_set_draft_warp(10, 0.9, check=False) == M.binding.MTAD_E_INVALID
    assert no_aux.ctx.mtad_draft([0], 4, 4, u, t, t, t, f, f, t, check=False) == M.binding.MTAD_E_INVALID


def _draft_gpu_batch(gm, seqs, gamma, b, u, keep_all=False):
    B, N = len(seqs), gamma * (b * b if keep_all else b)
    i32 = dict(dtype=torch.int32, device="cuda")
    f32 = dict(dtype=torch.float32, device="cuda")
    out = {"tok": torch.zeros(B, N, **i32), "parent": torch.zeros(B, N, **i32), "depth": torch.zeros(B, N, **i32),
           "node_logq": torch.zeros(B, N, **f32), "logq_ref": torch.zeros(B, gamma, **f32),
           "best_path": torch.zeros(B, gamma, **i32), "n_nodes": torch.zeros(B, **i32)}
    gm.ctx.mtad_draft(seqs, gamma, b, u, out["tok"], out["parent"], out["depth"], out["node_logq"], out["logq_ref"],
                      out["best_path"], keep_all_candidates=keep_all, n_nodes=out["n_nodes"])
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("B,gamma,b", [(2, 4, 4), (3, 3, 2), (8, 4, 4), (8, 6, 4)])
def test_batched_draft_verify_commit_iterations(B, gamma, b):
    batched_iterations(W.target, W.aux, [10 + 7 * s for s in range(B)], gamma, b, 256, 256, 4)


@pytest.mark.parametrize("B,gamma,b,keep_all,warp", [(2, 3, 3, False, None), (3, 4, 4, True, None), (2, 3, 2, True, None),
                                                     (3, 3, 3, False, (5, 0.9)), (2, 3, 3, True, (2, 1.0))])
def test_batched_draft_tree_verify_commit_iterations(B, gamma, b, keep_all, warp):
    """MMTAD for a batch (Sec. 3.3): the tree that mtad_draft wrote goes to mtad_verify_tree as it lies on the device;
    with `warp` drafted from warped auxiliary rows (layers of different sizes from sequence to sequence)."""
    batched_iterations(W.target, W.aux, [10 + 7 * s for s in range(B)], gamma, b, 320, 320, 4, tree=True,
                       keep_all=keep_all, warp=warp)


def batched_iterations(target, aux, lens, gamma, b, capacity, aux_capacity, iters, tree=False, keep_all=False,
                       warp=None):
    """Several ragged sequences per mtad_draft call, each followed by a verification (of the output sequences as
    chains: Algorithm 1 for a batch; with `tree` of the whole draft trees, read from the arrays mtad_draft wrote) and
    a commit of all of them, teacher-forced on the oracle's draft_beam / verify / aux_commit per sequence; the guard
    bytes behind every workspace array must be intact afterwards."""
    B = len(lens)
    N = gamma * (b * b if keep_all else b)
    gm = GpuModel(target, max_batch=B, max_nodes=max(N, gamma), capacity=capacity, aux=aux,
                  aux_capacity=aux_capacity)
    V = target.vocab
    seqs = list(range(B))
    state = []
    for s in seqs:
        L = lens[s]
        gm.inject(s, L)
        gm.inject_aux(s, L)
        root = 5 + s
        gm.ctx.mtad_seq_set(s, L, root, aux_len=L)
        state.append({"L": L, "La": L, "pend": [root], "root": root, "tc": gm.cache_bits(s, L),
                      "ac": gm.aux_cache_bits(s, L)})
    if warp:
        gm.ctx.mtad_set_draft_warp(*warp)
    skipped = 0
    log_tau = math.log(0.3)
    for it in range(iters):
        u = S.uniforms(0, (35 << 40) | (it * 64 + B), B * gamma * b * V, "cuda").view(B, gamma, b, V)
        g = _draft_gpu_batch(gm, seqs, gamma, b, u, keep_all)
        bu = S.bonus_uniforms(11, it, B, V, "cuda")
        drafts, near = [], []
        for s in seqs:
            st = state[s]
            dr = O.draft_beam(gm.oracle_aux(), st["ac"], st["La"], st["pend"], gamma, b, u[s].cpu().numpy(),
                              keep_all=keep_all, warp=warp)
            drafts.append(dr)
            n = len(dr.tok)
            near.append(dr.min_gap < draft_gap(keep_all) or dr.margin_warp < DRAFT_WARP_MARGIN)
            if not near[-1]:
                assert int(g["n_nodes"][s]) == n
                assert g["tok"][s, :n].tolist() == dr.tok and g["parent"][s, :n].tolist() == dr.parent, (it, s)
                assert g["best_path"][s].tolist() == dr.best_path
                assert np.max(np.abs(g["node_logq"][s, :n].cpu().numpy() - np.asarray(dr.logq))) < LP_TOL
                assert np.max(np.abs(g["logq_ref"][s].cpu().numpy() - np.asarray(dr.logq_ref))) < LP_TOL
        ref = torch.tensor([dr.logq_ref for dr in drafts], dtype=torch.float32, device="cuda")
        if tree:
            # sequences next to a tie of the draft get the oracle's tree (they are put back on its trajectory below)
            for s in seqs:
                if near[s]:
                    n = len(drafts[s].tok)
                    g["tok"][s, :n] = torch.tensor(drafts[s].tok, dtype=torch.int32, device="cuda")
                    g["parent"][s, :n] = torch.tensor(drafts[s].parent, dtype=torch.int32, device="cuda")
                    g["n_nodes"][s] = n
            res = M.ResultBuffers(B, N, gamma)
            gm.ctx.mtad_verify_tree(seqs, g["n_nodes"], N, gamma, g["tok"], g["parent"], ref, log_tau, bu, res)
        else:
            toks = torch.tensor([[dr.tok[n] for n in dr.best_path] for dr in drafts], dtype=torch.int32, device="cuda")
            res = M.ResultBuffers(B, gamma, gamma)
            gm.ctx.mtad_verify_chain(seqs, gamma, toks, ref, log_tau, bu, res)
        gm.ctx.kv_commit(seqs, res)
        h = res.host()
        for s in seqs:
            st, dr = state[s], drafts[s]
            assert int(h["status"][s]) == 0 or near[s]
            ref64 = np.asarray(dr.logq_ref, np.float32).astype(np.float64)
            if tree:
                r = O.verify_tree(gm.oracle(), st["tc"], st["L"], st["root"], dr.tok, dr.parent, ref64, log_tau,
                                  bu[s].cpu().numpy())
                accepted = list(r.path)
            else:
                r = O.verify_chain(gm.oracle(), st["tc"], st["L"], st["root"], [dr.tok[n] for n in dr.best_path],
                                   ref64, log_tau, bu[s].cpu().numpy())
                accepted = [dr.best_path[i] for i in r.path]
            tie = min(r.margin_accept, r.margin_tie, r.margin_bonus) < 1e-3
            st["L"] = O.kv_commit(st["tc"], st["L"], r.path)
            st["La"], st["pend"] = O.aux_commit(st["ac"], st["La"], st["pend"], dr, accepted, r.out_tok[-1], gamma)
            st["root"] = r.out_tok[-1]
            if near[s] or tie:
                skipped += 1
                gm.upload(s, st["tc"], st["ac"])
                gm.ctx.mtad_seq_set(s, st["L"], st["root"], aux_len=st["La"], pending_tok=st["pend"][:-1])
                continue
            assert int(h["eta"][s]) == r.eta and h["out_tok"][s, :r.eta + 1].tolist() == r.out_tok, (it, s)
            assert gm.ctx.mtad_seq_get(s) == (st["L"], st["root"])
    assert skipped <= B
    assert gm.ctx.mtad_debug_check_canaries() == ""
