"""The time-out path of the GEMM kernels: a bounded wait that runs out must end in MTAD_ST_TIMEOUT for every
sequence of the call, the kernels must return normally, kv_commit must leave those sequences alone, and the next call
on the same context must match the oracle again.  The wait is made to run out on the host's request (the operand-row
copies are left out, so the barrier they would complete is never completed); nothing faults and nothing hangs."""
import math

import pytest
import torch

import mtad_synth as S
import paper_2407_09722_b200 as M
from paper_2407_09722_b200 import binding as Bn
from tests.parity import GpuModel, SeqCase, ParityStats, compare

pytestmark = pytest.mark.gpu
TINY = S.WORKLOADS["tiny"].target


@pytest.mark.parametrize("gamma", [4, 11])      # 5 rows: the few-row cluster kernel and (gate / up) the stream-K kernel; 12 rows x 3 sequences = 36: the many-row cluster kernel
def test_wait_runs_out_then_context_recovers(gamma):
    gm = GpuModel(TINY, max_batch=3, max_nodes=16, capacity=128)
    V = TINY.vocab
    seqs, L = [0, 1, 2], 20
    for s in seqs:
        gm.inject(s, L)
        gm.ctx.mtad_seq_set(s, L, 3 + s)
    trees = [S.chain_tree(gamma, V, stream=70 + s) for s in seqs]
    tok = torch.tensor([t.tok for t in trees], dtype=torch.int32, device="cuda")
    lq = torch.tensor([t.logq for t in trees], dtype=torch.float32, device="cuda")
    u = S.bonus_uniforms(5, 0, 3, V, "cuda")
    res = M.ResultBuffers(3, gamma, gamma)
    gm.ctx.mtad_debug_set_wait(2000, True)
    gm.ctx.mtad_verify_chain(seqs, gamma, tok, lq, math.log(0.1), u, res)
    gm.ctx.kv_commit(seqs, res)
    torch.cuda.synchronize()                      # the kernels came back: no fault, no hang
    h = res.host()
    assert all(int(x) & Bn.MTAD_ST_TIMEOUT for x in h["status"].tolist()), h["status"]
    assert h["n_out"].tolist() == [0, 0, 0]
    for s in seqs:
        assert gm.ctx.mtad_seq_get(s) == (L, 3 + s)        # nothing was committed
    # hook off: the same context verifies correctly again (counters and tensor memory were left clean)
    gm.ctx.mtad_debug_set_wait(0, False)
    stats = ParityStats()
    for it in range(2):
        for s in seqs:
            gm.inject(s, L)
        cases = [SeqCase(s, L, 3 + s, S.chain_tree(gamma, V, stream=80 + 8 * it + s)) for s in seqs]
        compare(gm, cases, math.log(0.3), S.bonus_uniforms(6, it, 3, V, "cuda"), chain=True, stats=stats)
    assert stats.ok() and stats.near_ties <= 2, stats
