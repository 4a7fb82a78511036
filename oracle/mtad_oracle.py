"""CPU oracle for one MTAD / MMTAD iteration (arxiv 2407.09722).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain fp64 statement of what
the verification hot path computes.  It is imported by the tests, by the smoke
check and by the benchmark's CPU-baseline leg, never by the product path, and
it shares no code with the CUDA kernels.

What follows the paper, and where:
  * target forward over the draft rows, giving P[i, :] = p(. | x_{1:i-1}, input)
    (Algorithm 1, the line "P <- M_p(input, X)"; Sec. 3.3 for the tree form
    with tree attention);
  * joint likelihood of every draft prefix as a running product along the
    path (Sec. 3.2 "Draft Tokens Verification"; Algorithm 1 loop), kept in
    the log domain here;
  * chain rule: prefix j passes iff min(1, p/q) > tau, the longest passing
    prefix is accepted, every prefix is tested (Sec. 3.2);
  * tree rule: candidate passes iff p(candidate) / q(x**_{1:i}) clears tau,
    longest accepted candidate wins, ties by target likelihood (Sec. 3.3,
    the displayed acceptance equation and the paragraph after it);
  * one extra token sampled from the target row after the accepted prefix
    (Algorithm 1, "t ~ p'"), drawn with the Gumbel-max identity from caller
    supplied uniforms so that the draw is a pure function of its inputs;
  * beam sampling draft with the auxiliary model (Sec. 2.1, the p_beam
    equation), sampled without replacement with Gumbel-top-b;
  * optionally, the warping of the paper's experiments on every target row
    before the rule (App. F: top-k, renormalise, top-p);
  * the rule of vanilla speculative decoding as a second accept mode
    (Sec. 2.2: per-token ratio test against a uniform, stop at the first
    rejection, resample from the normalised positive part of p - q).

The decoder itself is only named by the paper (Llama / OPT families); the
definition used is the Llama one: pre-RMSNorm, rotary embedding with
half-split pairing, grouped-query softmax attention, SwiGLU FFN, untied LM
head.  The KV cache stores bf16 (round-to-nearest-even), a storage decision
both sides of the parity tests take; every other quantity is fp64.

Parity pins (tests/test_oracle_*.py): chain-shaped tree == token-by-token
causal decoding; every tree node == the chain of its own path; cross-check
against stock torch fp64 ops; log-softmax normalisation; prefix sums vs
products of probabilities; hand-built accept cases incl. the non-monotone
one; exhaustive enumeration at vocab 8, gamma 3; sampler frequencies;
hand-computed warped rows, and brute-force subset search for top-p;
for speculative decoding the closed form "accept + residual == target
distribution" at vocab 8, its threshold in u, and p == q accepting all.
The *distribution* of the beam-sampling draft is pinned only through the
Gumbel-top-b inclusion probabilities at vocab 8: beyond that it is
"parity unpinned".
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

NEG_INF = float("-inf")


# ----------------------------------------------------------------------------
# bf16 <-> fp64
# ----------------------------------------------------------------------------

def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp64 exactly."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round to bf16, nearest-even, through fp32 (the value first becomes an fp32, as it is on the device)."""
    u = np.ascontiguousarray(x, dtype=np.float64).astype(np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


# ----------------------------------------------------------------------------
# model container
# ----------------------------------------------------------------------------

@dataclass
class OracleModel:
    """A decoder given as bf16 bit patterns (uint16 arrays), matrices row-major [out, in].

    `layers` is any indexable of per-layer dicts with keys attn_norm, wq, wk, wv, wo, ffn_norm,
    w_gate, w_up, w_down (it may build a layer on demand so that large shapes stream through memory).
    """
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float
    rms_eps: float
    embed: np.ndarray
    lm_head: np.ndarray
    final_norm: np.ndarray
    layers: Sequence[dict]


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain, row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotary embedding, half-split pairing: element i pairs with i + hd/2, angle pos * base^(-2i/hd).

    x: [R, H, hd]; pos: [R]."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = base ** (-2.0 * np.arange(half, dtype=np.float64) / hd)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]          # [R, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def log_softmax(z: np.ndarray) -> np.ndarray:
    """log P[r, j] = z[r, j] - log sum_k exp z[r, k], with the row maximum subtracted first."""
    m = np.max(z, axis=-1, keepdims=True)
    return z - (m + np.log(np.sum(np.exp(z - m), axis=-1, keepdims=True)))


def decoder_rows(model: OracleModel, cache: np.ndarray, L: int, row_tok: Sequence[int], row_pos: Sequence[int],
                 row_slot: Sequence[int], row_visible: Sequence[Sequence[int]]) -> np.ndarray:
    """Run R new rows through the decoder against one sequence's KV cache.

    cache: uint16 [layers, 2, Hkv, capacity, hd] (bf16 bits), positions [0, L) committed.  Row r has token
    row_tok[r], rotary position row_pos[r]; its K and V are rounded to bf16 and written at cache slot
    row_slot[r] (>= L); it attends to every committed position and to the slots listed in row_visible[r]
    (which must include its own slot).  Returns the fp64 logits [R, vocab].
    """
    R = len(row_tok)
    Hq, Hkv, hd = model.n_q_heads, model.n_kv_heads, model.head_dim
    group = Hq // Hkv
    pos = np.asarray(row_pos, dtype=np.int64)
    h = bf16_bits_to_f64(model.embed[np.asarray(row_tok, dtype=np.int64)])        # [R, d]
    hi_slot = max(row_slot) + 1
    # visibility mask over cache slots [0, hi_slot): committed prefix + listed speculative slots
    vis = np.zeros((R, hi_slot), dtype=bool)
    vis[:, :L] = True
    for r in range(R):
        assert row_slot[r] in row_visible[r]
        for s in row_visible[r]:
            assert s >= L
            vis[r, s] = True
    for l in range(model.n_layers):
        w = model.layers[l]
        a = rmsnorm(h, bf16_bits_to_f64(w["attn_norm"]), model.rms_eps)
        q = (a @ bf16_bits_to_f64(w["wq"]).T).reshape(R, Hq, hd)
        k = (a @ bf16_bits_to_f64(w["wk"]).T).reshape(R, Hkv, hd)
        v = (a @ bf16_bits_to_f64(w["wv"]).T).reshape(R, Hkv, hd)
        q = rope(q, pos, model.rope_base)
        k = rope(k, pos, model.rope_base)
        for r in range(R):
            cache[l, 0, :, row_slot[r], :] = f64_to_bf16_bits(k[r])
            cache[l, 1, :, row_slot[r], :] = f64_to_bf16_bits(v[r])
        o = np.zeros((R, Hq, hd), dtype=np.float64)
        for g in range(Hkv):
            Kc = bf16_bits_to_f64(cache[l, 0, g, :hi_slot, :])                    # [S, hd]
            Vc = bf16_bits_to_f64(cache[l, 1, g, :hi_slot, :])
            for hq in range(g * group, (g + 1) * group):
                s = (q[:, hq, :] @ Kc.T) / math.sqrt(hd)                          # [R, S]
                s = np.where(vis, s, NEG_INF)
                s = s - np.max(s, axis=-1, keepdims=True)
                p = np.exp(s)
                p = p / np.sum(p, axis=-1, keepdims=True)
                o[:, hq, :] = p @ Vc
        h = h + o.reshape(R, Hq * hd) @ bf16_bits_to_f64(w["wo"]).T
        f = rmsnorm(h, bf16_bits_to_f64(w["ffn_norm"]), model.rms_eps)
        gate = f @ bf16_bits_to_f64(w["w_gate"]).T
        up = f @ bf16_bits_to_f64(w["w_up"]).T
        h = h + (silu(gate) * up) @ bf16_bits_to_f64(w["w_down"]).T
    hn = rmsnorm(h, bf16_bits_to_f64(model.final_norm), model.rms_eps)
    return hn @ bf16_bits_to_f64(model.lm_head).T


# ----------------------------------------------------------------------------
# tree bookkeeping
# ----------------------------------------------------------------------------

def node_depths(parent: Sequence[int]) -> List[int]:
    """1-based depth of every node; parent[n] = -1 means the node follows the root row directly."""
    d: List[int] = []
    for n, p in enumerate(parent):
        assert -1 <= p < n, "nodes must be topologically sorted (parent[n] < n)"
        d.append(1 if p < 0 else d[p] + 1)
    return d


def tree_rows(L: int, root_tok: int, tok: Sequence[int], parent: Sequence[int]):
    """Rows of the verify forward: row 0 = root (last emitted token, position L), row n+1 = node n at
    position L + depth(n); a row sees the committed context, its ancestors and itself."""
    depth = node_depths(parent)
    row_tok = [root_tok] + list(tok)
    row_pos = [L] + [L + d for d in depth]
    row_slot = [L + r for r in range(len(row_tok))]
    visible = [[L]]
    for n, p in enumerate(parent):
        visible.append(visible[p + 1] + [L + n + 1])
    return row_tok, row_pos, row_slot, visible


def node_logprobs(logits: np.ndarray, tok: Sequence[int], parent: Sequence[int]):
    """lp[n] = log P[row(parent(n)), tok[n]]: the target's conditional log-probability of node n's token given
    its path (row i of P predicts the token after x_{1:i-1}; Algorithm 1's comment on P).  Also the log-sum-exp
    of each row."""
    logp = log_softmax(logits)
    lp = np.array([logp[parent[n] + 1, tok[n]] for n in range(len(tok))], dtype=np.float64)
    m = np.max(logits, axis=-1)
    lse = m + np.log(np.sum(np.exp(logits - m[:, None]), axis=-1))
    return lp, lse


def path_prefix_sums(lp: Sequence[float], parent: Sequence[int]) -> np.ndarray:
    """LP[n] = LP[parent(n)] + lp[n], LP[root] = 0: log of the running product p <- p * P[i, x_i]."""
    LP = np.zeros(len(lp), dtype=np.float64)
    for n, p in enumerate(parent):
        LP[n] = (0.0 if p < 0 else LP[p]) + lp[n]
    return LP


# ----------------------------------------------------------------------------
# accept rules
# ----------------------------------------------------------------------------

def accept_chain(LP: Sequence[float], logq: Sequence[float], log_tau: float):
    """Longest prefix j with log p(x_{1:j}) - log q(x_{1:j}) > log tau; every j is tested, a failure does not
    stop the scan.  min(1, p/q) > tau is the same test because tau < 1.  Returns (eta, margin) with margin the
    smallest distance of any tested prefix from the threshold."""
    eta, margin = 0, float("inf")
    for j in range(len(LP)):
        gap = (LP[j] - logq[j]) - log_tau
        if gap > 0:
            eta = j + 1
        if math.isfinite(gap):
            margin = min(margin, abs(gap))
    return eta, margin


def accept_tree(LP: Sequence[float], parent: Sequence[int], logq_ref: Sequence[float], log_tau: float):
    """Candidate n (depth i) passes iff LP[n] - log q(x**_{1:i}) > log tau.  Winner: deepest passing node, then
    highest LP, then lowest index; no passing node -> the root (-1).  Returns (winner, eta, path, margin_accept,
    margin_tie) where margin_tie is the LP gap between the winner and the best other passing node of its depth."""
    depth = node_depths(parent)
    winner, best = -1, (0, NEG_INF)
    margin = float("inf")
    for n in range(len(LP)):
        gap = (LP[n] - logq_ref[depth[n] - 1]) - log_tau
        if math.isfinite(gap):
            margin = min(margin, abs(gap))
        if gap > 0 and (depth[n], LP[n]) > best:          # strict: ties keep the lower index
            winner, best = n, (depth[n], LP[n])
    path: List[int] = []
    n = winner
    while n >= 0:
        path.append(n)
        n = parent[n]
    path.reverse()
    tie = float("inf")
    if winner >= 0:
        for n in range(len(LP)):
            if n != winner and depth[n] == depth[winner] and \
                    (LP[n] - logq_ref[depth[n] - 1]) - log_tau > 0:
                tie = min(tie, LP[winner] - LP[n])
    return winner, len(path), path, margin, tie


def gumbel_argmax(z: np.ndarray, u: np.ndarray):
    """A draw from softmax(z): argmax_j (z_j + g_j), g_j = -log(-log u_j), lowest index on ties.
    Returns (token, gap between the best and second-best perturbed value)."""
    y = np.asarray(z, dtype=np.float64) - np.log(-np.log(np.asarray(u, dtype=np.float64)))
    t = int(np.argmax(y))
    second = np.max(np.delete(y, t)) if y.size > 1 else NEG_INF
    return t, float(y[t] - second)


def inverse_cdf_sample(p: np.ndarray, u: float) -> int:
    """The other exact sampler (used only in the small enumeration tests): t = min{k : C_k > u}."""
    c = np.cumsum(np.asarray(p, dtype=np.float64))
    return int(min(np.searchsorted(c, u, side="right"), len(c) - 1))


# ----------------------------------------------------------------------------
# warped distributions (App. F: top-k, renormalise, then top-p)
# ----------------------------------------------------------------------------

def warp_row(z: np.ndarray, top_k: int, top_p: float):
    """The warping of the paper's experiments applied to one row of logits (App. F): keep the top_k most likely
    tokens and renormalise; sort them by probability, descending (lower token id first among equals), and keep the
    first K whose cumulative probability is larger than top_p (all of them if it never is); the rest get
    probability 0.  The kept tokens are renormalised so that the row is a distribution to sample from (Sec. 2.1:
    tokens are sampled from that smallest subset).  Returns (log-probabilities with -inf for dropped tokens,
    margin), margin = how close any of the decisions was to going the other way: the logit gap across the top_k
    boundary and the distance of every partial cumulative sum from top_p."""
    z = np.asarray(z, dtype=np.float64)
    V = z.size
    order = sorted(range(V), key=lambda i: (-z[i], i))
    k = min(top_k, V)
    top = order[:k]
    margin = float(z[order[k - 1]] - z[order[k]]) if k < V else float("inf")
    zt = z[top]
    pt = np.exp(zt - zt[0])
    pt = pt / pt.sum()
    keep = k
    c = 0.0
    for i in range(k):
        c += pt[i]
        if i + 1 < k or c > top_p:
            margin = min(margin, abs(c - top_p))
        if c > top_p:
            keep = i + 1
            break
    kept = top[:keep]
    out = np.full(V, NEG_INF, dtype=np.float64)
    zk = z[kept]
    out[kept] = zk - (zk[0] + np.log(np.sum(np.exp(zk - zk[0]))))
    return out, margin


def warp_rows(logits: np.ndarray, top_k: int, top_p: float):
    rows, margins = zip(*(warp_row(r, top_k, top_p) for r in logits))
    return np.stack(rows), float(min(margins))


# ----------------------------------------------------------------------------
# one verification step and the cache commit
# ----------------------------------------------------------------------------

@dataclass
class VerifyResult:
    eta: int
    winner: int                 # node index of the accepted candidate, -1 = none (root)
    path: List[int]             # node ids root-to-winner
    out_tok: List[int]          # [tok[path_1..eta], bonus]
    out_lp: List[float]         # their target log-probs
    node_lp: np.ndarray
    node_LP: np.ndarray
    row_lse: np.ndarray
    row_cand: np.ndarray        # Gumbel-argmax token of every row
    row_cand_lp: np.ndarray
    margin_accept: float
    margin_tie: float
    margin_bonus: float
    logits: Optional[np.ndarray] = None
    margin_warp: float = float("inf")   # closest warping decision (warp_row) over all rows; inf without warping


def verify_from_logits(logits: np.ndarray, tok, parent, logq_or_ref, log_tau: float, u: np.ndarray,
                       chain: bool, warp=None) -> VerifyResult:
    """warp = (top_k, top_p): every row of P is warped first (the paper's footnote to Sec. 3.2: the method is
    equally valid on warped distributions); a drafted token outside a row's kept set has probability 0."""
    m_warp = float("inf")
    if warp is not None:
        logits, m_warp = warp_rows(logits, warp[0], warp[1])
    lp, lse = node_logprobs(logits, tok, parent)
    LP = path_prefix_sums(lp, parent)
    if chain:
        eta, m_acc = accept_chain(LP, logq_or_ref, log_tau)
        winner, path, m_tie = eta - 1, list(range(eta)), float("inf")
    else:
        winner, eta, path, m_acc, m_tie = accept_tree(LP, parent, logq_or_ref, log_tau)
    R = logits.shape[0]
    cand = np.zeros(R, dtype=np.int64)
    cand_lp = np.zeros(R, dtype=np.float64)
    gaps = np.zeros(R, dtype=np.float64)
    for r in range(R):
        cand[r], gaps[r] = gumbel_argmax(logits[r], u)
        cand_lp[r] = logits[r, cand[r]] - lse[r]
    wrow = winner + 1
    out_tok = [int(tok[n]) for n in path] + [int(cand[wrow])]
    out_lp = [float(lp[n]) for n in path] + [float(cand_lp[wrow])]
    return VerifyResult(eta, winner, path, out_tok, out_lp, lp, LP, lse, cand, cand_lp, m_acc, m_tie,
                        float(gaps[wrow]), logits, m_warp)


def verify_chain(model: OracleModel, cache: np.ndarray, L: int, root_tok: int, draft_tok, draft_logq,
                 log_tau: float, u: np.ndarray, warp=None) -> VerifyResult:
    """Algorithm 1 from "P <- M_p(input, X)" to the return: draft_logq[i] = log q(x_{1:i+1} | input)."""
    parent = list(range(-1, len(draft_tok) - 1))
    rows = tree_rows(L, root_tok, draft_tok, parent)
    logits = decoder_rows(model, cache, L, *rows)
    return verify_from_logits(logits, draft_tok, parent, draft_logq, log_tau, u, chain=True, warp=warp)


def verify_tree(model: OracleModel, cache: np.ndarray, L: int, root_tok: int, tok, parent, logq_ref,
                log_tau: float, u: np.ndarray, warp=None) -> VerifyResult:
    """Sec. 3.3: all candidates in one forward under the tree mask, normalised by the output beam's likelihood."""
    assert max(node_depths(parent), default=0) <= len(logq_ref)
    rows = tree_rows(L, root_tok, tok, parent)
    logits = decoder_rows(model, cache, L, *rows)
    return verify_from_logits(logits, tok, parent, logq_ref, log_tau, u, chain=False, warp=warp)


# ----------------------------------------------------------------------------
# vanilla speculative decoding (Sec. 2.2), the rule MTAD is measured against
# ----------------------------------------------------------------------------

def spd_residual(logp_row: np.ndarray, logq_row: np.ndarray) -> np.ndarray:
    """Unnormalised residual weights max(0, p - q) of Sec. 2.2, step 4 (the distribution a rejected position is
    resampled from, norm(max(0, p - q)))."""
    return np.maximum(0.0, np.exp(np.asarray(logp_row, np.float64)) - np.exp(np.asarray(logq_row, np.float64)))


@dataclass
class SpdResult:
    eta: int
    path: List[int]
    out_tok: List[int]
    out_lp: List[float]             # target log-probabilities of the emitted tokens
    margin_accept: float            # smallest |log u_i - min(0, log p_i - log q_i)| over the tested positions
    margin_bonus: float             # gap between the two largest perturbed values of the last draw
    margin_bonus_robust: float      # the same gap when every log p may be off by +-tol against the winner
    logits: Optional[np.ndarray] = None


def spd_from_logits(logits: np.ndarray, tok: Sequence[int], logq_rows: np.ndarray, u_acc: Sequence[float],
                    u_res: np.ndarray, tol: float = 2e-3) -> SpdResult:
    """Sec. 2.2, steps 2-4: draft token i (drawn from q_i) is accepted with probability min(1, p_i(x_i) / q_i(x_i)),
    i.e. iff u_i < that ratio; verification stops at the first rejection, whose position is resampled from
    norm(max(0, p_i - q_i)); with every token accepted one more is drawn from the target's next row.
    logits: [gamma + 1, V] target rows; logq_rows: [gamma, V] the auxiliary model's normalised log-distributions
    at the draft positions; u_acc: [gamma] uniforms of the accept tests; u_res: [V] uniforms of the final draw
    (Gumbel-argmax, as for the extra token of Algorithm 1)."""
    logp = log_softmax(logits)
    g = len(tok)
    eta, margin = g, float("inf")
    for i in range(g):
        ratio = min(0.0, float(logp[i, tok[i]] - logq_rows[i, tok[i]]))
        lu = math.log(u_acc[i])
        margin = min(margin, abs(lu - ratio))
        if not lu < ratio:
            eta = i
            break
    if eta == g:
        z = logp[g]
        z_lo, z_hi = z - tol, z + tol
    else:
        p_row, q_row = np.exp(logp[eta]), np.exp(np.asarray(logq_rows[eta], np.float64))
        with np.errstate(divide="ignore"):
            z = np.log(np.maximum(0.0, p_row - q_row))
            z_lo = np.log(np.maximum(0.0, p_row * math.exp(-tol) - q_row))
            z_hi = np.log(np.maximum(0.0, p_row * math.exp(tol) - q_row))
    t, gap = gumbel_argmax(z, u_res)
    noise = -np.log(-np.log(np.asarray(u_res, dtype=np.float64)))
    others = np.delete(z_hi + noise, t)
    robust = float(z_lo[t] + noise[t] - (np.max(others) if others.size else NEG_INF))
    path = list(range(eta))
    out_tok = [int(tok[i]) for i in path] + [t]
    out_lp = [float(logp[i, tok[i]]) for i in path] + [float(logp[eta, t])]
    return SpdResult(eta, path, out_tok, out_lp, margin, gap, robust, logits)


def verify_chain_spd(model: OracleModel, cache: np.ndarray, L: int, root_tok: int, draft_tok, logq_rows,
                     u_acc, u_res) -> SpdResult:
    parent = list(range(-1, len(draft_tok) - 1))
    rows = tree_rows(L, root_tok, draft_tok, parent)
    logits = decoder_rows(model, cache, L, *rows)
    return spd_from_logits(logits, draft_tok, logq_rows, u_acc, u_res)


def kv_commit(cache: np.ndarray, L: int, path: Sequence[int]) -> int:
    """Keep the root row and the accepted path: node path[i] (slot L + 1 + path[i]) moves to position L + 1 + i.
    Everything after is dropped (the "rollback").  Returns the new committed length L + eta + 1."""
    for i, n in enumerate(path):
        src, dst = L + 1 + n, L + 1 + i
        assert src >= dst
        if src != dst:
            cache[:, :, :, dst, :] = cache[:, :, :, src, :]
    return L + len(path) + 1


# ----------------------------------------------------------------------------
# beam-sampling draft with the auxiliary model
# ----------------------------------------------------------------------------

@dataclass
class DraftResult:
    tok: List[int]
    parent: List[int]
    depth: List[int]
    logq: List[float]           # joint log q of the path ending at each node
    best_path: List[int]        # node ids of x** (the final beam with the highest draft likelihood)
    logq_ref: List[float]       # log q(x**_{1:i})
    min_gap: float = float("inf")   # smallest gap between neighbouring perturbed scores among the b kept and the
                                    # first one dropped, over all steps (how close any pick was to a tie)
    slot: List[int] = field(default_factory=list)   # per node: its row in the auxiliary cache is base + slot (the
                                                    # k-th beam of layer s has slot s * b + k); -1 for a candidate
                                                    # that was recorded but not kept as a beam (never run)
    margin_warp: float = float("inf")   # closest warping decision over all beam rows (warp_row); inf without warping


def gumbel_top_b(scores: np.ndarray, u: np.ndarray, b: int, with_gap: bool = False):
    """Sample b distinct flat indices without replacement, successive draws proportional to exp(scores):
    the b largest of scores + Gumbel noise, in decreasing order (lowest index first on ties)."""
    y = np.asarray(scores, dtype=np.float64).ravel() - np.log(-np.log(np.asarray(u, dtype=np.float64).ravel()))
    # an index of probability 0 (score -inf: a token dropped by the warping) cannot be drawn, so fewer than b may come back
    order = sorted((i for i in range(y.size) if y[i] > NEG_INF), key=lambda i: (-y[i], i))
    if with_gap:
        top = [y[i] for i in order[:b + 1]]
        gap = min((top[k] - top[k + 1] for k in range(len(top) - 1)), default=float("inf"))
        return order[:b], float(gap)
    return order[:b]


def draft_beam(model: OracleModel, cache: np.ndarray, L: int, pending_tok: Sequence[int], gamma: int, b: int,
               u: np.ndarray, keep_all: bool = False, warp: Optional[Tuple[int, float]] = None) -> DraftResult:
    """Beam sampling of width b for gamma steps (Sec. 2.1): at each step the b kept sequences are drawn without
    replacement from p_beam over (beam, token) pairs, i.e. proportionally to the joint likelihood
    q(beam) * q(token | beam).  Every intermediate beam becomes a tree node (Sec. 3.3).

    pending_tok: tokens not yet in the auxiliary cache, oldest first, ending with the root (last emitted token);
    they occupy positions L .. L+len-1 and are run causally in the first step.  u: [gamma, b, vocab] uniforms.
    The k-th beam of layer s uses cache slot L + len(pending) + s * b + k (DraftResult.slot).

    keep_all: the tree also records the candidates that the sampling looked at but did not keep - every layer
    holds b * b nodes: the b * b best perturbed tokens of the context in the first layer, the b best perturbed tokens
    of each of the b beams afterwards, beam by beam, best first.  The beams kept for the next step are, as before,
    the b best of all (beam, token) pairs, which are among those; the others are leaves (slot -1).  Without keep_all a
    layer holds just its b beams, best first (the paper's tree).

    warp = (top_k, top_p): every beam row q(. | beam) is warped as in the paper's experiments (App. F, warp_row) before
    the sampling, so the draft samples from, and reports the likelihoods of, the warped auxiliary distribution.  Dropped
    tokens have probability 0 and are never drafted; a step whose rows keep fewer than b (beam, token) pairs in all
    keeps that many beams, so layers may hold fewer nodes (node ids stay consecutive).
    """
    P = len(pending_tok)
    base = L + P
    tok: List[int] = []
    parent: List[int] = []
    depth: List[int] = []
    logq: List[float] = []
    # step 1: the context is the only beam
    vis = [[L + i for i in range(r + 1)] for r in range(P)]
    logits = decoder_rows(model, cache, L, list(pending_tok), [L + i for i in range(P)],
                          [L + i for i in range(P)], vis)
    beams = [-1]                                   # node ids of the current beams (-1 = context)
    beam_logq = np.array([0.0])
    margin_warp = float("inf")

    def row_logp(z):                               # [n_beams, V] log q(token | beam), warped if asked for
        nonlocal margin_warp
        if warp is None:
            return log_softmax(z)
        lp, m = warp_rows(z, warp[0], warp[1])
        margin_warp = min(margin_warp, m)
        return lp

    beam_logp = row_logp(logits[P - 1:P])
    root_vis = vis[P - 1]
    node_vis = {-1: root_vis}
    min_gap = float("inf")
    slot: List[int] = []
    for step in range(gamma):
        scores = beam_logq[:, None] + beam_logp    # joint log-likelihood of every (beam, token) pair
        picks, gap = gumbel_top_b(scores, u[step, :len(beams), :], b, with_gap=True)
        min_gap = min(min_gap, gap)
        V = scores.shape[1]
        if keep_all:
            # the layer's nodes: per beam its best perturbed tokens (b * b of the single beam of the first step)
            per_beam = b * b if step == 0 else b
            layer = []
            for j in range(len(beams)):
                own, gap_j = gumbel_top_b(scores[j:j + 1], u[step, j:j + 1, :], per_beam, with_gap=True)
                min_gap = min(min_gap, gap_j)
                layer += [j * V + int(v) for v in own]
        else:
            layer = list(picks)
        new_nodes = [None] * len(picks)
        for flat in layer:
            j, v = divmod(flat, V)
            n = len(tok)
            tok.append(int(v)); parent.append(beams[j]); depth.append(step + 1)
            logq.append(float(scores[j, v]))
            if flat in picks:                      # kept as the k-th beam of this layer: gets a row of the cache
                k = list(picks).index(flat)
                slot.append(step * b + k)
                node_vis[n] = node_vis[beams[j]] + [base + step * b + k]
                new_nodes[k] = n
            else:
                slot.append(-1)
        beams = new_nodes
        beam_logq = np.array([logq[n] for n in beams])
        if step + 1 < gamma:
            logits = decoder_rows(model, cache, L, [tok[n] for n in beams], [base - 1 + depth[n] for n in beams],
                                  [base + slot[n] for n in beams], [node_vis[n] for n in beams])
            beam_logp = row_logp(logits)
    best = max(beams, key=lambda n: (logq[n], -n))
    path = []
    n = best
    while n >= 0:
        path.append(n)
        n = parent[n]
    path.reverse()
    return DraftResult(tok, parent, depth, logq, path, [logq[n] for n in path], min_gap, slot, margin_warp)


def aux_commit(cache: np.ndarray, L: int, pending_tok: Sequence[int], draft: DraftResult, accepted: Sequence[int],
               bonus_tok: int, gamma: int):
    """Roll the auxiliary cache forward after a verification: the pending rows (slots L ..) are already in place;
    accepted draft node accepted[i] (tree id, depth i + 1, row L + P + slot) moves to position L + P + i if the draft
    ran it (a beam of a layer before the last).  A node of the last layer, or a recorded candidate that was not kept
    as a beam, was never run by the auxiliary model: it stays pending, ahead of the new root (it can only be the last
    node of the path: neither has children).  Returns (new committed length, new pending tokens ending with the new
    root)."""
    P = len(pending_tok)
    base = L + P
    slot = draft.slot if draft.slot else list(range(len(draft.tok)))
    ran = lambda n: draft.depth[n] < gamma and slot[n] >= 0
    kept = [n for n in accepted if ran(n)]
    assert kept == list(accepted[:len(kept)])
    for i, n in enumerate(kept):
        src, dst = base + slot[n], base + i
        assert src >= dst
        if src != dst:
            cache[:, :, :, dst, :] = cache[:, :, :, src, :]
    pend = [draft.tok[n] for n in accepted if not ran(n)] + [bonus_tok]
    return base + len(kept), pend
