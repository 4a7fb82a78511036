"""GPU parity of the speculative-decoding accept mode (mtad_verify_chain_spd, Sec. 2.2) against the oracle's
spd_from_logits: accepted length and tokens exact unless the oracle reports a decision within the margin (the accept
test within 1e-3 in log u; the final draw not robust to a 2e-3 error in log p), log-probabilities within 2e-3."""
import numpy as np
import pytest
import torch

import mtad_synth as S
import paper_2407_09722_b200 as M
from oracle import mtad_oracle as O
from tests.parity import GpuModel, LP_TOL, MARGIN

pytestmark = pytest.mark.gpu

TINY = S.WORKLOADS["tiny"].target
GQA64 = S.ModelShape(3, 192, 6, 2, 64, 328, 500)


def _draft(rng, g, V, scale):
    """Synthetic auxiliary distributions (log-softmax of random logits) and a chain drawn from them."""
    rows = O.log_softmax(rng.normal(scale=scale, size=(g, V)))
    tok = [int(rng.choice(V, p=np.exp(rows[i]))) for i in range(g)]
    return rows, tok


@pytest.mark.parametrize("shape,scale", [(TINY, 0.6), (TINY, 0.02), (GQA64, 1.0)])
def test_spd_chain_matches_oracle(shape, scale):
    B, V = 2, shape.vocab
    gm = GpuModel(shape, max_batch=B, max_nodes=8, capacity=160)
    rng = np.random.default_rng(int(scale * 100))
    skipped, n, etas = 0, 0, []
    L = [33, 70]
    root = [4, 9]
    cache = []
    for b in range(B):
        gm.inject(b, L[b])
        gm.ctx.mtad_seq_set(b, L[b], root[b])
        cache.append(gm.cache_bits(b, L[b]))
    for it in range(5):
        g = 3 + it % 3
        rows, toks = zip(*(_draft(rng, g, V, scale) for _ in range(B)))
        u_acc = rng.uniform(0.02, 0.98, size=(B, g)).astype(np.float32)
        u_res = S.bonus_uniforms(13, it, B, V, "cuda")
        res = M.ResultBuffers(B, g, g)
        rows32 = np.asarray(rows, np.float32)
        gm.ctx.mtad_verify_chain_spd(list(range(B)), g, torch.tensor(toks, dtype=torch.int32, device="cuda"),
                                     torch.tensor(rows32, device="cuda"), torch.tensor(u_acc, device="cuda"), u_res, res)
        gm.ctx.kv_commit(list(range(B)), res)
        h = res.host()
        for b in range(B):
            r = O.verify_chain_spd(gm.oracle(), cache[b], L[b], root[b], list(toks[b]), rows32[b].astype(np.float64),
                                   u_acc[b].astype(np.float64), u_res[b].cpu().numpy())
            assert int(h["status"][b]) == 0
            L[b] = O.kv_commit(cache[b], L[b], r.path)
            root[b] = r.out_tok[-1]
            n += 1
            etas.append(r.eta)
            if r.margin_accept < MARGIN or r.margin_bonus_robust <= 0:
                skipped += 1
                gm.upload(b, cache[b])
                gm.ctx.mtad_seq_set(b, L[b], root[b])
                continue
            assert int(h["eta"][b]) == r.eta and int(h["n_out"][b]) == r.eta + 1
            assert h["out_tok"][b, :r.eta + 1].tolist() == r.out_tok
            assert h["path"][b, :r.eta].tolist() == r.path
            assert np.max(np.abs(h["out_lp"][b, :r.eta + 1].numpy() - np.asarray(r.out_lp))) < LP_TOL
            assert gm.ctx.mtad_seq_get(b) == (L[b], root[b])
    assert skipped <= n // 2
    assert min(etas) < max(etas)            # both rejections and longer acceptances occurred


def test_spd_non_finite_logits_set_a_status_bit():
    gm = GpuModel(TINY, max_batch=2, max_nodes=8, capacity=96)
    V, g = TINY.vocab, 4
    for seq in range(2):
        gm.inject(seq, 40)
        gm.ctx.mtad_seq_set(seq, 40, 3 + seq)
    gm.cache[0, 1, 0, 0, 3, 5] = float("nan")           # layer 0, sequence 1, K, head 0, position 3
    rng = np.random.default_rng(2)
    rows, toks = zip(*(_draft(rng, g, V, 0.5) for _ in range(2)))
    res = M.ResultBuffers(2, g, g)
    gm.ctx.mtad_verify_chain_spd([0, 1], g, torch.tensor(toks, dtype=torch.int32, device="cuda"),
                                 torch.tensor(np.asarray(rows, np.float32), device="cuda"),
                                 torch.full((2, g), 0.5, device="cuda"), S.bonus_uniforms(1, 0, 2, V, "cuda"), res)
    gm.ctx.kv_commit([0, 1], res)
    h = res.host()
    assert int(h["status"][0]) == 0 and int(h["n_out"][0]) >= 1
    assert int(h["status"][1]) & M.binding.MTAD_ST_NONFINITE and int(h["n_out"][1]) == 0
    assert gm.ctx.mtad_seq_get(1) == (40, 4)


def test_spd_rejects_bad_arguments():
    gm = GpuModel(TINY, max_batch=1, max_nodes=8, capacity=96)
    V = TINY.vocab
    res = M.ResultBuffers(1, 4, 4)
    t = torch.zeros(1, 4, dtype=torch.int32, device="cuda")
    rows = torch.zeros(1, 4, V, device="cuda")
    u = torch.full((1, 4), 0.5, device="cuda")
    ur = torch.full((1, V), 0.5, device="cuda")
    c = gm.ctx
    assert c.mtad_verify_chain_spd([0], 0, t, rows, u, ur, res, check=False) == M.binding.MTAD_E_INVALID
    assert c.mtad_verify_chain_spd([0], 4, t, None, u, ur, res, check=False) == M.binding.MTAD_E_INVALID
    assert c.mtad_verify_chain_spd([0], 4, t, rows, None, ur, res, check=False) == M.binding.MTAD_E_INVALID
    assert c.mtad_verify_chain_spd([0], 9, t, rows, u, ur, res, check=False) == M.binding.MTAD_E_CAPACITY
