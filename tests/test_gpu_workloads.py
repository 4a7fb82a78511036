"""Parity at the shapes of the benchmark workloads (same launch configuration as bench.py): the 7B chain, the 7B
tree and the 13B ragged batch at full depth, the 70B GQA tree at reduced depth (the oracle widens every weight to
fp64 on the host, so depth is what bounds its run time; width, row count, cache length and tree shape are the
workload's own)."""
import dataclasses
import math

import pytest
import torch

import mtad_synth as S
from tests.parity import GpuModel, SeqCase, ParityStats, compare, gemm_eps

pytestmark = pytest.mark.gpu


def _cases(w, lens, it=0):
    return [SeqCase(b, lens[b], 1 + b, S.workload_tree(w, seq=b, iteration=it)) for b in range(w.batch)]


def _run(w, shape, capacity, taus, check_cache=True):
    lens = S.kv_lengths(w)
    gm = GpuModel(shape, max_batch=w.batch, max_nodes=w.n_nodes, capacity=capacity)
    stats = ParityStats()
    for it, tau in enumerate(taus):
        for b, L in enumerate(lens):
            gm.inject(b, L)
        u = S.bonus_uniforms(0, it, w.batch, shape.vocab, "cuda")
        compare(gm, _cases(w, lens, it), math.log(tau), u, chain=(w.kind == "chain"), stats=stats,
                check_cache=check_cache)
    assert stats.ok(), stats
    return stats


def test_7b_chain_full_depth():
    w = S.WORKLOADS["7b_chain"]
    st = _run(w, w.target, 2048 + 64, [0.1, 0.5])
    assert st.max_lp_err < 2e-3 and st.cache_ok(w.target.layers, gemm_eps(w.gamma + 1, w.target.d_ffn))


def test_7b_tree_full_depth():
    w = S.WORKLOADS["7b_tree"]
    st = _run(w, w.target, 2048 + 128, [0.1])
    assert st.max_lp_err < 2e-3


def test_13b_ragged_batch_four_layers():
    w = S.WORKLOADS["13b_batched_chain"]
    shape = dataclasses.replace(w.target, layers=4)
    st = _run(w, shape, 4096 + 16, [0.1])
    assert st.n_seq == 8


def test_70b_shape_chain_two_layers():
    """The 8192-wide GQA model itself is inside the bound: same weights and cache length as the 70B tree case, with a
    5-row chain instead of the 129-row tree."""
    w = S.WORKLOADS["70b_gqa_tree"]
    c = dataclasses.replace(S.WORKLOADS["7b_chain"], target=w.target, kv_len=w.kv_len)
    shape = dataclasses.replace(w.target, layers=2)
    st = _run(c, shape, max(w.kv_len) + 256, [0.1])
    assert st.max_lp_err < 5e-4


@pytest.mark.parametrize("layers", [2, 8])
def test_70b_gqa_tree(layers):
    """129 rows at width 8192.  K and V are rounded to bf16 for the cache; an element that rounds the other way than
    the exact value shifts the scores of the rows that attend to it, and the peaked attention over draft rows at this
    width amplifies that by two orders of magnitude into the next layer.  The Q/K/V projection therefore keeps its
    relative error near 5e-7 (three operand terms, accumulation chains of at most eight k-blocks), which holds the
    log-probabilities inside the bound with room to spare at two and at eight layers."""
    w = S.WORKLOADS["70b_gqa_tree"]
    shape = dataclasses.replace(w.target, layers=layers)
    st = _run(w, shape, 1024 + 256, [0.1])
    assert st.max_lp_err < 1.5e-3 and st.near_ties <= 1, st


def test_13b_ragged_batch_full_depth():
    """All 40 layers of the 13B-shaped batch (eight ragged sequences, seven rows each) on the device; the oracle, which
    widens every weight to fp64 on the host, follows two of the eight sequences (the longest and the shortest)."""
    w = S.WORKLOADS["13b_batched_chain"]
    lens = S.kv_lengths(w)
    gm = GpuModel(w.target, max_batch=w.batch, max_nodes=w.n_nodes, capacity=4096 + 16)
    for b, L in enumerate(lens):
        gm.inject(b, L)
    u = S.bonus_uniforms(0, 0, w.batch, w.target.vocab, "cuda")
    pick = [max(range(w.batch), key=lambda b: lens[b]), min(range(w.batch), key=lambda b: lens[b])]
    st = compare(gm, _cases(w, lens, 0), math.log(0.1), u, chain=True, only=pick)
    assert st.n_seq == 2 and st.ok() and st.near_ties <= 1, st
    assert st.max_lp_err < 2e-3


def test_13b_pair_batched_draft_two_layers():
    """The batched iteration of Algorithm 1 at the 13B-shaped pair: eight ragged sequences of 1024..4096 committed
    tokens, the full-size auxiliary model (2 layers, 1024 wide, 16 heads of 64), gamma 6, beam width 4, the target cut
    to two layers so that the oracle stays affordable: mtad_draft of all eight, mtad_verify_chain of the eight output
    sequences, kv_commit of both caches, twice, against the oracle sequence by sequence."""
    from tests.test_gpu_draft import batched_iterations
    w = S.WORKLOADS["13b_batched_chain"]
    shape = dataclasses.replace(w.target, layers=2)
    batched_iterations(shape, w.aux, S.kv_lengths(w), w.gamma, 4, 4160, 4160, 2)


def test_7b_pair_drafted_tree_two_layers():
    """MMTAD end to end at the 7B-shaped pair (Sec. 3.3): the full-size auxiliary model (2 layers, 768 wide) drafts
    with beam width 4 for gamma 4 and keeps every candidate - the 64-node tree of the tree workload -, the target (cut
    to two layers so that the oracle stays affordable) verifies that tree from the arrays mtad_draft wrote, kv_commit
    rolls both caches forward; two iterations at 2048 committed tokens, against the oracle."""
    from tests.test_gpu_draft import batched_iterations
    w = S.WORKLOADS["7b_tree"]
    shape = dataclasses.replace(w.target, layers=2)
    batched_iterations(shape, w.aux, [2048], w.gamma, 4, 2048 + 160, 2048 + 160, 2, tree=True, keep_all=True)


def test_7b_pair_chain_eight_iterations_two_layers():
    """Algorithm 1 for eight consecutive iterations at the 7B-shaped pair (target cut to two layers so that the oracle
    stays affordable, the full-size auxiliary model): draft, verification of the output sequence as a chain, commit of
    both caches, each iteration starting from the state the one before left on the device, against the oracle."""
    from tests.test_gpu_draft import batched_iterations
    w = S.WORKLOADS["7b_chain"]
    shape = dataclasses.replace(w.target, layers=2)
    batched_iterations(shape, w.aux, [2048], w.gamma, 4, 2048 + 96, 2048 + 96, 8)
