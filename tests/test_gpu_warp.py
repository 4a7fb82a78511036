"""GPU parity of the warped verification (top-k, renormalise, top-p on every target row: mtad_set_warp) against the
oracle's warp_row.  The drafts are built from the oracle's own likely tokens, so that accepted paths, dropped tokens
and extra tokens from truncated rows all occur; decisions the oracle reports as near ties are counted, not compared."""
import math

import numpy as np
import pytest
import torch

import mtad_synth as S
from oracle import mtad_oracle as O
from tests.parity import GpuModel, SeqCase, ParityStats, compare

pytestmark = pytest.mark.gpu

TINY = S.WORKLOADS["tiny"].target
GQA64 = S.ModelShape(3, 192, 6, 2, 64, 328, 500)
WIDE_VOCAB = S.ModelShape(1, 128, 2, 2, 64, 344, 32000)     # 32 chunks of the vocabulary per row, as at full size


def _likely_tree(gm, seq, L, root, parent, ranks, dq):
    """Tokens for a tree of the given shape: node n takes the ranks[n]-th most likely token of the oracle's row of
    its parent (one oracle forward per depth).  Draft likelihoods: the oracle's own path likelihoods shifted by
    dq per token, so that some prefixes pass the threshold and some do not."""
    model, cache = gm.oracle(), gm.cache_bits(seq, L)
    depth = O.node_depths(parent)
    tok = [0] * len(parent)
    logp = None
    for d in range(1, max(depth, default=0) + 1):
        logits = O.decoder_rows(model, cache, L, *O.tree_rows(L, root, tok, parent))
        logp = O.log_softmax(logits)
        for n, p in enumerate(parent):
            if depth[n] == d:
                order = sorted(range(logp.shape[1]), key=lambda v: (-logp[p + 1, v], v))
                tok[n] = order[ranks[n]]
    logits = O.decoder_rows(model, cache, L, *O.tree_rows(L, root, tok, parent))
    logp = O.log_softmax(logits)
    lq = [0.0] * len(parent)
    for n, p in enumerate(parent):
        lq[n] = (lq[p] if p >= 0 else 0.0) + float(logp[p + 1, tok[n]]) + dq[n]
    # x**: the deepest node with the largest draft likelihood, and its ancestors
    D = max(depth, default=0)
    last = [n for n in range(len(parent)) if depth[n] == D]
    best, path = (max(last, key=lambda n: lq[n]) if last else -1), []
    while best >= 0:
        path.append(best)
        best = parent[best]
    path.reverse()
    return S.DraftTree(tok, list(parent), depth, lq, path, [lq[n] for n in path])


@pytest.mark.parametrize("shape,warp", [(TINY, (10, 0.9)), (TINY, (4, 0.6)), (GQA64, (16, 0.95)), (TINY, (1, 0.9)),
                                        (WIDE_VOCAB, (10, 0.9))])
def test_warped_chain_matches_oracle(shape, warp):
    gm = GpuModel(shape, max_batch=2, max_nodes=16, capacity=160)
    rng = np.random.default_rng(warp[0])
    stats = ParityStats()
    for it, (L, g) in enumerate([(40, 4), (96, 6), (7, 3), (64, 5)]):
        cases = []
        for seq in range(2):
            gm.inject(seq, L + seq)
            parent = list(range(-1, g - 1))
            # mostly the likeliest tokens, now and then one far down the list (dropped by the warping)
            ranks = [int(r) for r in rng.choice([0, 0, 1, 2, 3, 40], size=g)]
            dq = [float(x) for x in rng.normal(0.3, 0.8, size=g)]
            tree = _likely_tree(gm, seq, L + seq, 5 + seq, parent, ranks, dq)
            cases.append(SeqCase(seq, L + seq, 5 + seq, tree))
        u = S.bonus_uniforms(3, it, 2, shape.vocab, "cuda")
        compare(gm, cases, math.log(0.3), u, chain=True, stats=stats, warp=warp)
    assert stats.ok(tie_cap=stats.n_seq // 2), stats
    assert max(stats.etas) > 0


def test_warped_tree_matches_oracle():
    gm = GpuModel(TINY, max_batch=1, max_nodes=24, capacity=160)
    rng = np.random.default_rng(9)
    stats = ParityStats()
    for it in range(4):
        L = 30 + 17 * it
        gm.inject(0, L)
        # three layers of four nodes: every node of a layer hangs off one of the first two nodes of the layer before
        parent = [-1, -1, -1, -1] + [int(p) for p in rng.integers(0, 2, size=4)] + \
                 [int(p) for p in rng.integers(4, 6, size=4)]
        ranks, seen = [], {}
        for n, p in enumerate(parent):              # distinct tokens among siblings
            seen[p] = seen.get(p, -1) + 1
            ranks.append(seen[p] if rng.uniform() < 0.8 else 30 + seen[p])
        dq = [float(x) for x in rng.normal(0.2, 0.6, size=len(parent))]
        tree = _likely_tree(gm, 0, L, 9, parent, ranks, dq)
        u = S.bonus_uniforms(4, it, 1, TINY.vocab, "cuda")
        compare(gm, [SeqCase(0, L, 9, tree)], math.log(0.2), u, chain=False, stats=stats, warp=(10, 0.9))
    assert stats.ok(), stats
    assert max(stats.etas) > 0


def test_warp_off_again_and_bad_arguments():
    gm = GpuModel(TINY, max_batch=1, max_nodes=8, capacity=96)
    from paper_2407_09722_b200 import binding as Bn
    assert gm.ctx.mtad_set_warp(17, 0.9, check=False) == Bn.MTAD_E_CAPACITY
    assert gm.ctx.mtad_set_warp(10, 0.0, check=False) == Bn.MTAD_E_INVALID
    assert gm.ctx.mtad_set_warp(10, 1.5, check=False) == Bn.MTAD_E_INVALID
    assert gm.ctx.mtad_set_warp(-1, 0.9, check=False) == Bn.MTAD_E_INVALID
    # a warped call, then an unwarped one on the same context: the second must equal the plain path
    stats = ParityStats()
    for it, warp in enumerate([(10, 0.9), None]):
        gm.inject(0, 48)
        tree = S.chain_tree(4, TINY.vocab, stream=77 + it)
        compare(gm, [SeqCase(0, 48, 3, tree)], math.log(0.1), S.bonus_uniforms(5, it, 1, TINY.vocab, "cuda"),
                chain=True, stats=stats, warp=warp)
    assert stats.ok(), stats
