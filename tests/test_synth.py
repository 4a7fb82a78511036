"""The seeded generators: determinism, ranges, tree well-formedness."""
import math

import torch

import mtad_synth as S


def test_hash_matches_python_reference():
    # the tensor path must equal the plain-int splitmix64 finaliser
    seed, stream = 3, (5 << 32) | 17
    key = S.stream_key(seed, stream)
    h = S.hash_u64(seed, stream, 10, 4).tolist()
    for i, got in enumerate(h):
        want = S._mix_int((10 + i) * S._GOLDEN + key)
        assert got & S._M64 == want


def test_chunking_is_invisible():
    a = S.normal_bf16(0, 9, 1000, 0.02, chunk=1 << 24)
    b = S.normal_bf16(0, 9, 1000, 0.02, chunk=77)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_weight_statistics():
    x = S.normal_bf16(0, 21, 1 << 18, 0.02).double()
    assert abs(x.mean().item()) < 3e-4
    assert abs(x.std().item() - 0.02) < 3e-4
    g = S.make_tensor(S.WORKLOADS["tiny"].target, 0, "attn_norm", 0).double()
    assert abs(g.mean().item() - 1.0) < 0.03 and g.min().item() > 0.5


def test_uniforms_open_interval_and_tokens_in_range():
    u = S.uniforms(0, 4, 100000)
    assert u.dtype == torch.float32 and u.min().item() > 0.0 and u.max().item() < 1.0
    assert abs(u.double().mean().item() - 0.5) < 0.01
    t = S.token_ids(0, 4, 10000, 1000)
    assert t.min().item() >= 0 and t.max().item() < 1000


def test_trees_well_formed():
    for (depth, width, keep) in [(4, 16, 4), (4, 32, 8), (4, 4, 4), (3, 8, 2)]:
        tr = S.beam_tree(depth, width, keep, 32000, stream=depth * 100 + width)
        n = depth * width
        assert len(tr.tok) == len(tr.parent) == len(tr.depth) == len(tr.logq) == n
        for i, p in enumerate(tr.parent):
            assert -1 <= p < i
            assert tr.depth[i] == (1 if p < 0 else tr.depth[p] + 1)
            assert tr.logq[i] < (0.0 if p < 0 else tr.logq[p])
        # siblings carry distinct tokens
        seen = set()
        for i, p in enumerate(tr.parent):
            assert (p, tr.tok[i]) not in seen
            seen.add((p, tr.tok[i]))
        assert [tr.depth[i] for i in tr.best_path] == list(range(1, depth + 1))
        deepest = [i for i in range(n) if tr.depth[i] == depth]
        assert tr.logq[tr.best_path[-1]] == max(tr.logq[i] for i in deepest)
    ch = S.chain_tree(6, 32000)
    assert ch.parent == [-1, 0, 1, 2, 3, 4] and ch.logq_ref == ch.logq


def test_workload_byte_counts():
    w = S.WORKLOADS["7b_chain"].target
    assert w.layer_params() == 202_375_168
    assert abs(w.streamed_weight_bytes() / 1e9 - 13.214) < 1e-3
    assert w.kv_bytes_per_token() == 524288
    assert S.WORKLOADS["70b_gqa_tree"].target.kv_bytes_per_token() == 327680
    lens = S.kv_lengths(S.WORKLOADS["13b_batched_chain"])
    assert len(lens) == 8 and all(1024 <= x <= 4096 for x in lens)
