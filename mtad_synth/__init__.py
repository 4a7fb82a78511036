"""Seeded synthetic inputs for the MTAD / MMTAD verification step.

Everything here is an *input generator*: model shapes, hashed bf16 weights,
hashed token ids, uniforms, draft trees and draft log-likelihoods.  None of
the method's arithmetic (decoder forward, log-softmax, prefix sums, accept
rule, sampling) lives in this module; both the CPU oracle's tests and the
CUDA path's tests consume what it returns.

All values are pure functions of (seed, stream id, flat element index) built
from 64-bit integer mixing only, so the same call gives the same bits on the
CPU and on a CUDA device.

The paper evaluates on trained Llama / OPT pairs and public suites that are
not available offline; these generators stand in for them with random-init
models of the same shapes, uniform-random token ids, draft chains of gamma =
3..6 and beam trees of width 4..8 (the paper's hyper-parameter grid, App. F).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, asdict
from typing import Dict, List, Optional

import torch

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _s64(c: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant (torch has no uint64 math)."""
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


def _mix_int(x: int) -> int:
    """splitmix64 finaliser on a Python int."""
    x &= _M64
    x ^= x >> 30
    x = (x * _C1) & _M64
    x ^= x >> 27
    x = (x * _C2) & _M64
    x ^= x >> 31
    return x


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix_t(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on an int64 tensor (wrap-around multiply)."""
    x = x ^ _lsr(x, 30)
    x = x * _s64(_C1)
    x = x ^ _lsr(x, 27)
    x = x * _s64(_C2)
    x = x ^ _lsr(x, 31)
    return x


def stream_key(seed: int, stream: int) -> int:
    return _mix_int((seed * _GOLDEN + stream * _C1 + 0x1234567) & _M64)


def hash_u64(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """int64 tensor of `count` hashed words for flat indices start..start+count-1."""
    key = stream_key(seed, stream)
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _mix_t(idx * _s64(_GOLDEN) + _s64(key))


_TABLES: Dict[float, torch.Tensor] = {}


def normal_table(scale: float) -> torch.Tensor:
    """65536-entry bf16 table: entry k = bf16(scale * Phi^-1((k + 0.5) / 65536)), built in fp64 on the host."""
    t = _TABLES.get(scale)
    if t is None:
        k = torch.arange(65536, dtype=torch.float64)
        t = (scale * torch.special.ndtri((k + 0.5) / 65536.0)).to(torch.bfloat16)
        _TABLES[scale] = t
    return t


def normal_bf16(seed: int, stream: int, numel: int, scale: float, device="cpu",
                offset: float = 0.0, chunk: int = 1 << 24) -> torch.Tensor:
    """bf16 tensor of `numel` values ~ offset + N(0, scale^2), quantised through the 65536-entry table."""
    table = normal_table(scale)
    if offset != 0.0:
        table = (table.to(torch.float64) + offset).to(torch.bfloat16)
    table = table.to(device)
    out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    for s in range(0, numel, chunk):
        n = min(chunk, numel - s)
        h = hash_u64(seed, stream, s, n, device)
        out[s:s + n] = table[h & 0xFFFF]
    return out


def token_ids(seed: int, stream: int, n: int, vocab: int, device="cpu") -> torch.Tensor:
    h = hash_u64(seed, stream, 0, n, device)
    return (_lsr(h, 16) % vocab).to(torch.int32)


def uniforms(seed: int, stream: int, n: int, device="cpu") -> torch.Tensor:
    """fp32 uniforms strictly inside (0, 1): (23 hashed bits + 0.5) / 2^23, every value exact in fp32
    (smallest 2^-24, largest 1 - 2^-24)."""
    h = hash_u64(seed, stream, 0, n, device)
    return ((_lsr(h, 41).to(torch.float64) + 0.5) / float(1 << 23)).to(torch.float32)


# ----------------------------------------------------------------------------
# model shapes
# ----------------------------------------------------------------------------

@dataclass(frozen=True)
class ModelShape:
    layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5

    @property
    def q_dim(self):
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self):
        return self.n_kv_heads * self.head_dim

    def layer_params(self) -> int:
        d = self.d_model
        return d * self.q_dim + 2 * d * self.kv_dim + self.q_dim * d + 3 * d * self.d_ffn

    def streamed_weight_bytes(self) -> int:
        """bf16 bytes every verify step must read once: all layer matrices + the LM head."""
        return 2 * (self.layers * self.layer_params() + self.vocab * self.d_model)

    def kv_bytes_per_token(self) -> int:
        return self.layers * 2 * self.kv_dim * 2


LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def layer_tensor_shapes(s: ModelShape) -> Dict[str, tuple]:
    return {
        "attn_norm": (s.d_model,),
        "wq": (s.q_dim, s.d_model),
        "wk": (s.kv_dim, s.d_model),
        "wv": (s.kv_dim, s.d_model),
        "wo": (s.d_model, s.q_dim),
        "ffn_norm": (s.d_model,),
        "w_gate": (s.d_ffn, s.d_model),
        "w_up": (s.d_ffn, s.d_model),
        "w_down": (s.d_model, s.d_ffn),
    }


@dataclass(frozen=True)
class Workload:
    name: str
    target: ModelShape
    aux: ModelShape
    batch: int
    kind: str                 # "chain" or "tree"
    gamma: int                # chain length or tree depth
    n_nodes: int              # draft nodes per sequence (chain: gamma)
    kv_len: tuple             # committed KV length(s): (lo, hi) -> uniform in [lo, hi] per sequence
    tree_width: int = 0       # nodes per tree layer
    tree_keep: int = 0        # nodes per layer that get children
    prompt_len: int = 0
    decode_iters: int = 0


def _llama(layers, d, hq, hkv, hd, f, v=32000):
    return ModelShape(layers, d, hq, hkv, hd, f, v)


WORKLOADS: Dict[str, Workload] = {
    # tiny reference pair; aux FFN width is not given by the config list -> 4 * d
    "tiny": Workload("tiny", ModelShape(2, 256, 4, 4, 64, 688, 1024), ModelShape(1, 128, 2, 2, 64, 512, 1024),
                     batch=1, kind="chain", gamma=4, n_nodes=4, kv_len=(32, 32), prompt_len=32, decode_iters=16),
    "7b_chain": Workload("7b_chain", _llama(32, 4096, 32, 32, 128, 11008), _llama(2, 768, 12, 12, 64, 3072),
                         batch=1, kind="chain", gamma=4, n_nodes=4, kv_len=(2048, 2048), prompt_len=512,
                         decode_iters=128),
    "7b_chain_l512": Workload("7b_chain_l512", _llama(32, 4096, 32, 32, 128, 11008),
                              _llama(2, 768, 12, 12, 64, 3072),
                              batch=1, kind="chain", gamma=4, n_nodes=4, kv_len=(512, 512), prompt_len=512,
                              decode_iters=128),
    # four layers of the 7B shape: small enough (about 2 GB on the device) for multi-pass profiler captures
    "7b_chain_4l": Workload("7b_chain_4l", _llama(4, 4096, 32, 32, 128, 11008), _llama(2, 768, 12, 12, 64, 3072),
                            batch=1, kind="chain", gamma=4, n_nodes=4, kv_len=(2048, 2048), prompt_len=512,
                            decode_iters=128),
    "7b_tree_4l": Workload("7b_tree_4l", _llama(4, 4096, 32, 32, 128, 11008), _llama(2, 768, 12, 12, 64, 3072),
                           batch=1, kind="tree", gamma=4, n_nodes=64, kv_len=(2048, 2048), tree_width=16, tree_keep=4),
    "7b_tree": Workload("7b_tree", _llama(32, 4096, 32, 32, 128, 11008), _llama(2, 768, 12, 12, 64, 3072),
                        batch=1, kind="tree", gamma=4, n_nodes=64, kv_len=(2048, 2048), tree_width=16, tree_keep=4),
    "13b_batched_chain": Workload("13b_batched_chain", _llama(40, 5120, 40, 40, 128, 13824),
                                  _llama(2, 1024, 16, 16, 64, 4096),
                                  batch=8, kind="chain", gamma=6, n_nodes=6, kv_len=(1024, 4096)),
    "70b_gqa_tree": Workload("70b_gqa_tree", _llama(80, 8192, 64, 8, 128, 28672), _llama(4, 1024, 16, 16, 64, 4096),
                             batch=1, kind="tree", gamma=4, n_nodes=128, kv_len=(1024, 1024), tree_width=32,
                             tree_keep=8),
}


# ----------------------------------------------------------------------------
# weights, caches
# ----------------------------------------------------------------------------

_TID = {"embed": 1, "lm_head": 2, "final_norm": 3}


def _tensor_stream(model_id: int, name: str, layer: int = -1) -> int:
    if layer < 0:
        t = _TID[name]
    else:
        t = 16 + layer * 16 + LAYER_TENSORS.index(name)
    return (model_id << 32) | t


def make_tensor(shape: ModelShape, model_id: int, name: str, layer: int = -1, seed: int = 0,
                device="cpu") -> torch.Tensor:
    """One named weight tensor, bf16, row-major [out, in].  Matrices ~ N(0, 0.02^2); norm gains ~ 1 + N(0, 0.1^2)."""
    if name in ("embed", "lm_head"):
        dims = (shape.vocab, shape.d_model)
    elif name == "final_norm":
        dims = (shape.d_model,)
    else:
        dims = layer_tensor_shapes(shape)[name]
    numel = math.prod(dims)
    st = _tensor_stream(model_id, name, layer)
    if name.endswith("norm"):
        t = normal_bf16(seed, st, numel, 0.1, device, offset=1.0)
    else:
        t = normal_bf16(seed, st, numel, 0.02, device)
    return t.view(*dims)


def make_layer(shape: ModelShape, model_id: int, layer: int, seed: int = 0, device="cpu") -> Dict[str, torch.Tensor]:
    return {n: make_tensor(shape, model_id, n, layer, seed, device) for n in LAYER_TENSORS}


def make_model(shape: ModelShape, model_id: int, seed: int = 0, device="cpu") -> dict:
    """{'shape', 'embed', 'lm_head', 'final_norm', 'layers': [dict per layer]} of bf16 tensors."""
    return {
        "shape": shape,
        "embed": make_tensor(shape, model_id, "embed", seed=seed, device=device),
        "lm_head": make_tensor(shape, model_id, "lm_head", seed=seed, device=device),
        "final_norm": make_tensor(shape, model_id, "final_norm", seed=seed, device=device),
        "layers": [make_layer(shape, model_id, l, seed, device) for l in range(shape.layers)],
    }


def kv_cache_shape(shape: ModelShape, batch: int, capacity: int) -> tuple:
    """Cache layout [layer][sequence][K|V][kv head][position][head_dim], bf16."""
    return (shape.layers, batch, 2, shape.n_kv_heads, capacity, shape.head_dim)


def fill_kv_cache(cache: torch.Tensor, model_id: int, seq: int, length: int, seed: int = 0) -> None:
    """Inject `length` committed positions of unit-variance hashed bf16 K and V into sequence `seq` (in place)."""
    layers, _, _, hkv, cap, hd = cache.shape
    for l in range(layers):
        st = (7 << 40) | (model_id << 32) | (seq << 16) | l
        vals = normal_bf16(seed, st, 2 * hkv * length * hd, 1.0, cache.device).view(2, hkv, length, hd)
        cache[l, seq, :, :, :length, :] = vals


def kv_lengths(w: Workload, seed: int = 0) -> List[int]:
    lo, hi = w.kv_len
    if lo == hi:
        return [lo] * w.batch
    h = hash_u64(seed, (9 << 40), 0, w.batch)
    return [int(lo + (int(x) & 0x7FFFFFFF) % (hi - lo + 1)) for x in h.tolist()]


# ----------------------------------------------------------------------------
# draft trees and draft log-likelihoods
# ----------------------------------------------------------------------------

@dataclass
class DraftTree:
    tok: List[int]            # token of node n
    parent: List[int]         # parent node of n, -1 = child of the root row; parent[n] < n
    depth: List[int]          # 1-based depth of node n
    logq: List[float]         # joint draft log-likelihood of the path ending at n
    best_path: List[int]      # node ids of the draft's output sequence x** (one per depth)
    logq_ref: List[float]     # logq of best_path[i] for depth i+1


def _distinct_tokens(seed, stream, n, vocab) -> List[int]:
    raw = token_ids(seed, stream, 4 * n + 8, vocab).tolist()
    out: List[int] = []
    for t in raw:
        if t not in out:
            out.append(t)
        if len(out) == n:
            return out
    k = 0
    while len(out) < n:          # vocab smaller than the request window: fill deterministically
        if k not in out:
            out.append(k)
        k += 1
    return out


def chain_tree(gamma: int, vocab: int, seed: int = 0, stream: int = 0, logq_mean: Optional[float] = None,
               logq_std: float = 1.0) -> DraftTree:
    """A draft chain x_1..x_gamma with synthetic per-token draft log-probs ~ N(mean, std^2) accumulated along it."""
    if logq_mean is None:
        logq_mean = -math.log(vocab) - 0.3
    tok = token_ids(seed, (11 << 40) | stream, gamma, vocab).tolist()
    z = normal_bf16(seed, (12 << 40) | stream, gamma, 1.0).to(torch.float64).tolist()
    logq, acc = [], 0.0
    for i in range(gamma):
        acc += min(-1e-3, logq_mean + logq_std * z[i])
        logq.append(acc)
    return DraftTree(tok, list(range(-1, gamma - 1)), list(range(1, gamma + 1)), logq,
                     list(range(gamma)), list(logq))


def beam_tree(depth: int, width: int, keep: int, vocab: int, seed: int = 0, stream: int = 0,
              logq_mean: Optional[float] = None, logq_std: float = 1.0) -> DraftTree:
    """Layered candidate tree: every layer has `width` nodes; `keep` hashed nodes of a layer each get
    width/keep children with distinct tokens in the next layer (layer 1 hangs off the root row).
    x** is the deepest-layer node with the largest synthetic joint log q."""
    assert width % keep == 0
    if logq_mean is None:
        logq_mean = -math.log(vocab) - 0.3
    per = width // keep
    tok, parent, dep, logq = [], [], [], []
    prev_layer: List[int] = []
    zs = normal_bf16(seed, (13 << 40) | stream, depth * width, 1.0).to(torch.float64).tolist()
    for layer in range(depth):
        if layer == 0:
            parents = [-1] * width
            toks = _distinct_tokens(seed, (14 << 40) | (stream << 8) | layer, width, vocab)
        else:
            order = hash_u64(seed, (15 << 40) | (stream << 8) | layer, 0, width).tolist()
            ranked = sorted(range(width), key=lambda i: (order[i], i))
            kept = sorted(prev_layer[i] for i in ranked[:keep])
            parents, toks = [], []
            for j, p in enumerate(kept):
                parents += [p] * per
                toks += _distinct_tokens(seed, (14 << 40) | (stream << 8) | (layer * 64 + j + 1), per, vocab)
        cur = []
        for i in range(width):
            n = len(tok)
            tok.append(toks[i]); parent.append(parents[i]); dep.append(layer + 1)
            base = 0.0 if parents[i] < 0 else logq[parents[i]]
            logq.append(base + min(-1e-3, logq_mean + logq_std * zs[layer * width + i]))
            cur.append(n)
        prev_layer = cur
    best = max(prev_layer, key=lambda n: (logq[n], -n))
    path = []
    n = best
    while n >= 0:
        path.append(n)
        n = parent[n]
    path.reverse()
    return DraftTree(tok, parent, dep, logq, path, [logq[n] for n in path])


def workload_tree(w: Workload, seq: int = 0, seed: int = 0, iteration: int = 0) -> DraftTree:
    stream = (iteration << 8) | seq
    if w.kind == "chain":
        return chain_tree(w.gamma, w.target.vocab, seed, stream)
    return beam_tree(w.gamma, w.tree_width, w.tree_keep, w.target.vocab, seed, stream)


def bonus_uniforms(seed: int, iteration: int, batch: int, vocab: int, device="cpu") -> torch.Tensor:
    """[batch, vocab] fp32 uniforms in (0,1) for the bonus-token draw of one iteration."""
    return uniforms(seed, (17 << 40) | iteration, batch * vocab, device).view(batch, vocab)
