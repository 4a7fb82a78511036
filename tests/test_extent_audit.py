"""Host-side extent audit (mtad_audit_extents): for the benchmark configurations with their auxiliary models, and for
the shapes of a batched draft -> verify -> commit iteration, every index that the kernels of a call form stays inside
the array it goes into.  Pure host arithmetic through the C ABI: no GPU."""
import pytest

import mtad_synth as S
from paper_2407_09722_b200 import binding as Bn

BEAM = 4


def _check(records, where):
    assert records, where
    bad = [(w, r, e) for (w, r, e) in records if not (0 < r <= e)]
    assert not bad, (where, bad[:5])


def _cap(w, extra=0):
    return (w.kv_len[1] + 200 + extra + 63) // 64 * 64


@pytest.mark.parametrize("name", ["tiny", "7b_chain", "7b_tree", "13b_batched_chain", "70b_gqa_tree"])
def test_verify_and_commit_extents_of_every_config(name):
    w = S.WORKLOADS[name]
    cap = _cap(w)
    t = Bn.shape_desc(w.target, cap)
    for aux in (None, Bn.shape_desc(w.aux, cap + w.gamma * BEAM + 8)):
        for max_nodes in (w.n_nodes, max(w.n_nodes, w.gamma * BEAM)):
            for L in (0, w.kv_len[0], w.kv_len[1]):
                where = (name, aux is not None, max_nodes, L)
                _check(Bn.mtad_audit_extents(t, aux, w.batch, max_nodes, Bn.AUDIT_VERIFY, w.batch, w.n_nodes, w.gamma,
                                             BEAM, L), where)
                _check(Bn.mtad_audit_extents(t, aux, w.batch, max_nodes, Bn.AUDIT_COMMIT, w.batch, w.n_nodes, w.gamma,
                                             BEAM, L), where)


@pytest.mark.parametrize("name,B", [("tiny", 1), ("tiny", 3), ("tiny", 8), ("7b_chain", 1), ("7b_chain", 4),
                                    ("13b_batched_chain", 8), ("70b_gqa_tree", 1), ("70b_gqa_tree", 2)])
def test_draft_extents(name, B):
    """mtad_draft with gamma steps of `BEAM` beams for B sequences, then the chain verify and the commit that follow
    it on the same context - the shapes of the batched iteration of Algorithm 1 (13B pair: eight ragged sequences of
    1024..4096 tokens, gamma 6, auxiliary capacity 4160)."""
    w = S.WORKLOADS[name]
    g = w.gamma
    cap = 4160 if name == "13b_batched_chain" else _cap(w)
    t = Bn.shape_desc(w.target, cap)
    a = Bn.shape_desc(w.aux, cap)
    max_nodes = max(w.n_nodes, g * BEAM)
    for L in (w.kv_len[0], w.kv_len[1]):
        for pending in (0, 1, g):           # rows replayed by step 0, less the root
            _check(Bn.mtad_audit_extents(t, a, B, max_nodes, Bn.AUDIT_DRAFT, B, pending, g, BEAM, L), (name, B, L, pending))
        _check(Bn.mtad_audit_extents(t, a, B, max_nodes, Bn.AUDIT_VERIFY, B, g, g, BEAM, L), (name, B, L))
        _check(Bn.mtad_audit_extents(t, a, B, max_nodes, Bn.AUDIT_COMMIT, B, g, g, BEAM, L), (name, B, L))


def test_audit_sees_an_undersized_region():
    """The audit is not vacuous: asked about more draft nodes than the context was created for, it is refused, and a
    cache too short for the rows of the call shows up as a reach beyond the extent."""
    w = S.WORKLOADS["tiny"]
    t = Bn.shape_desc(w.target, 64)
    with pytest.raises(Bn.MtadError):
        Bn.mtad_audit_extents(t, None, 1, 4, Bn.AUDIT_VERIFY, 1, 5, 5, BEAM, 10)
    a = Bn.shape_desc(w.aux, 40)
    rec = Bn.mtad_audit_extents(t, a, 1, 16, Bn.AUDIT_DRAFT, 1, 0, 4, BEAM, 30)
    assert any(r > e for (_, r, e) in rec if _ == "aux cache slots")
