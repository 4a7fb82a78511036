"""Pins for the oracle's decoder forward: things the mathematics fixes, independent of the oracle's own code."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import mtad_synth as S
from oracle import mtad_oracle as O
from oracle.adapters import oracle_model, bits

TINY = S.WORKLOADS["tiny"].target
GQA = S.ModelShape(2, 128, 4, 2, 32, 200, 96)          # grouped-query shape, odd FFN width


def _empty_cache(shape, cap):
    return np.zeros((shape.layers, 2, shape.n_kv_heads, cap, shape.head_dim), dtype=np.uint16)


def _prefill(model, cache, toks):
    """token-by-token causal decoding: the textbook KV-cache loop"""
    out = []
    for i, t in enumerate(toks):
        out.append(O.decoder_rows(model, cache, i, [t], [i], [i], [[i]])[0])
    return np.stack(out)


def test_bf16_round_trip_and_rounding():
    b = np.arange(0, 0x7F80, 37, dtype=np.uint16)                        # finite positive bf16 patterns
    x = O.bf16_bits_to_f64(b)
    assert np.array_equal(O.f64_to_bf16_bits(x), b)
    # exact ties round to even; 1 + 2^-8 lies midway between 1.0 (even) and 1 + 2^-7
    assert O.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80
    assert O.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82
    t = torch.randn(1000, dtype=torch.float32)
    assert np.array_equal(O.f64_to_bf16_bits(t.double().numpy()), bits(t.to(torch.bfloat16)))


def test_rope_closed_forms():
    rng = np.random.default_rng(0)
    q = rng.standard_normal((3, 2, 64)); k = rng.standard_normal((3, 2, 64))
    assert np.allclose(O.rope(q, np.zeros(3, dtype=np.int64), 10000.0), q, atol=0)
    pos = np.array([5, 77, 1234])
    rq = O.rope(q, pos, 10000.0)
    assert np.allclose(np.linalg.norm(rq, axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-13)
    # scores depend on the relative position only
    a = np.einsum("rhd,rhd->rh", O.rope(q, pos, 1e4), O.rope(k, pos - 3, 1e4))
    b = np.einsum("rhd,rhd->rh", O.rope(q, pos + 400, 1e4), O.rope(k, pos + 397, 1e4))
    assert np.allclose(a, b, atol=1e-9)
    # first pair rotates by exactly `pos` radians (inverse frequency 1), last pair by pos * base^(-(hd-2)/hd)
    e = np.zeros((1, 1, 64)); e[0, 0, 0] = 1.0
    r = O.rope(e, np.array([2]), 10000.0)[0, 0]
    assert abs(r[0] - math.cos(2.0)) < 1e-15 and abs(r[32] - math.sin(2.0)) < 1e-15
    e = np.zeros((1, 1, 64)); e[0, 0, 31] = 1.0
    r = O.rope(e, np.array([9]), 10000.0)[0, 0]
    th = 9 * 10000.0 ** (-62 / 64)
    assert abs(r[31] - math.cos(th)) < 1e-15 and abs(r[63] - math.sin(th)) < 1e-15


def test_small_closed_forms():
    x = np.array([[3.0, 4.0]])
    assert np.allclose(O.rmsnorm(x, np.array([1.0, 2.0]), 0.0), [[3 / math.sqrt(12.5), 8 / math.sqrt(12.5)]])
    assert O.silu(np.array([0.0]))[0] == 0.0
    z = np.linspace(-5, 5, 11)
    assert np.allclose(O.silu(z) - O.silu(-z), z)
    lz = np.random.default_rng(1).standard_normal((4, 1000)) * 3
    assert np.allclose(np.exp(O.log_softmax(lz)).sum(-1), 1.0, atol=1e-12)
    assert np.allclose(O.log_softmax(lz), torch.log_softmax(torch.from_numpy(lz), -1).numpy(), atol=1e-12)
    assert np.allclose(O.log_softmax(lz + 1e4), O.log_softmax(lz), atol=1e-9)   # shift invariance at large offsets


@pytest.mark.parametrize("shape", [TINY, GQA])
def test_chain_tree_equals_token_by_token_decoding(shape):
    model = oracle_model(S.make_model(shape, 0))
    toks = S.token_ids(0, 99, 13, shape.vocab).tolist()
    c1 = _empty_cache(shape, 32)
    step = _prefill(model, c1, toks)
    c2 = _empty_cache(shape, 32)
    _prefill(model, c2, toks[:8])
    rows = O.tree_rows(8, toks[8], toks[9:], list(range(-1, 3)))
    block = O.decoder_rows(model, c2, 8, *rows)
    assert np.max(np.abs(block - step[8:])) < 1e-10
    assert np.array_equal(c1[:, :, :, :13], c2[:, :, :, :13])


@pytest.mark.parametrize("shape", [TINY, GQA])
def test_every_tree_node_equals_its_own_path_chain(shape):
    model = oracle_model(S.make_model(shape, 0))
    ctx = S.token_ids(0, 5, 7, shape.vocab).tolist()
    tr = S.beam_tree(3, 4, 2, shape.vocab, stream=3)
    base = _empty_cache(shape, 40)
    _prefill(model, base, ctx[:6])
    c = base.copy()
    logits = O.decoder_rows(model, c, 6, *O.tree_rows(6, ctx[6], tr.tok, tr.parent))
    for n in range(len(tr.tok)):
        path, m = [], n
        while m >= 0:
            path.append(m); m = tr.parent[m]
        path.reverse()
        cc = base.copy()
        chain = O.decoder_rows(model, cc, 6, *O.tree_rows(6, ctx[6], [tr.tok[i] for i in path],
                                                          list(range(-1, len(path) - 1))))
        assert np.max(np.abs(chain[-1] - logits[n + 1])) < 1e-10


def _torch_reference(model_t, shape, cache_t, L, row_tok, row_pos, vis_mask):
    """Same decoder from stock torch fp64 ops (sdpa with a boolean mask, complex-number rotary)."""
    f64 = torch.float64
    R = len(row_tok)
    Hq, Hkv, hd = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    h = model_t["embed"].to(f64)[torch.tensor(row_tok)]
    inv = 1.0 / (shape.rope_base ** (torch.arange(0, hd, 2, dtype=f64) / hd))
    ang = torch.tensor(row_pos, dtype=f64)[:, None] * inv[None]
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]                 # [R,1,hd/2]

    def rotary(x):                                                           # x [R,H,hd]; pair (i, i+hd/2)
        z = torch.complex(x[..., :hd // 2], x[..., hd // 2:]) * rot
        return torch.cat([z.real, z.imag], -1)

    S_tot = vis_mask.shape[1]
    for l, w in enumerate(model_t["layers"]):
        a = F.rms_norm(h, (shape.d_model,), w["attn_norm"].to(f64), shape.rms_eps)
        q = rotary(F.linear(a, w["wq"].to(f64)).view(R, Hq, hd))
        k = rotary(F.linear(a, w["wk"].to(f64)).view(R, Hkv, hd))
        v = F.linear(a, w["wv"].to(f64)).view(R, Hkv, hd)
        cache_t[l, 0, :, L:L + R] = k.transpose(0, 1).float().to(torch.bfloat16)
        cache_t[l, 1, :, L:L + R] = v.transpose(0, 1).float().to(torch.bfloat16)
        K = cache_t[l, 0, :, :S_tot].to(f64).repeat_interleave(Hq // Hkv, 0)      # [Hq,S,hd]
        V = cache_t[l, 1, :, :S_tot].to(f64).repeat_interleave(Hq // Hkv, 0)
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], K[None], V[None],
                                           attn_mask=torch.from_numpy(vis_mask)[None, None])[0]
        h = h + F.linear(o.transpose(0, 1).reshape(R, Hq * hd), w["wo"].to(f64))
        f = F.rms_norm(h, (shape.d_model,), w["ffn_norm"].to(f64), shape.rms_eps)
        h = h + F.linear(F.silu(F.linear(f, w["w_gate"].to(f64))) * F.linear(f, w["w_up"].to(f64)),
                         w["w_down"].to(f64))
    hn = F.rms_norm(h, (shape.d_model,), model_t["final_norm"].to(f64), shape.rms_eps)
    return F.linear(hn, model_t["lm_head"].to(f64)).numpy()


@pytest.mark.parametrize("shape", [TINY, GQA])
def test_tree_forward_against_stock_torch_ops(shape):
    mt = S.make_model(shape, 0)
    model = oracle_model(mt)
    L, cap = 21, 48
    cache_t = torch.zeros(S.kv_cache_shape(shape, 1, cap), dtype=torch.bfloat16)
    S.fill_kv_cache(cache_t, 0, 0, L)
    from oracle.adapters import cache_bits
    c = cache_bits(cache_t, 0)
    tr = S.beam_tree(3, 4, 2, shape.vocab, stream=8)
    rows = O.tree_rows(L, 17, tr.tok, tr.parent)
    logits = O.decoder_rows(model, c, L, *rows)
    R = len(rows[0])
    mask = np.zeros((R, L + R), dtype=bool)
    mask[:, :L] = True
    for r in range(R):
        for s in rows[3][r]:
            mask[r, s] = True
    ref = _torch_reference(mt, shape, cache_t[:, 0].clone(), L, rows[0], rows[1], mask)
    assert np.max(np.abs(ref - logits)) < 1e-9
    # the mask itself: ancestors-or-self only (hand check on the known topology)
    for n, p in enumerate(tr.parent):
        anc = {0, n + 1}
        m = p
        while m >= 0:
            anc.add(m + 1); m = tr.parent[m]
        assert set(np.nonzero(mask[n + 1, L:])[0].tolist()) == anc


def test_kv_commit_equals_rerunning_the_accepted_tokens():
    shape = TINY
    model = oracle_model(S.make_model(shape, 0))
    ctx = S.token_ids(0, 6, 9, shape.vocab).tolist()
    tr = S.beam_tree(3, 4, 2, shape.vocab, stream=5)
    c = _empty_cache(shape, 40)
    _prefill(model, c, ctx[:8])
    O.decoder_rows(model, c, 8, *O.tree_rows(8, ctx[8], tr.tok, tr.parent))
    leaf = max(range(len(tr.tok)), key=lambda n: (tr.depth[n], n))
    path, m = [], leaf
    while m >= 0:
        path.append(m); m = tr.parent[m]
    path.reverse()
    newL = O.kv_commit(c, 8, path)
    assert newL == 8 + len(path) + 1
    nxt = O.decoder_rows(model, c, newL, [123], [newL], [newL], [[newL]])[0]
    c2 = _empty_cache(shape, 40)
    full = ctx + [tr.tok[n] for n in path] + [123]
    ref = _prefill(model, c2, full)[-1]
    assert np.max(np.abs(ref - nxt)) < 1e-10
    assert np.array_equal(c[:, :, :, :newL + 1], c2[:, :, :, :newL + 1])
