"""Parity harness: runs one verification step through the C-ABI on the GPU and through the CPU oracle on the same
seeded inputs and compares them.  Test infrastructure (imports the oracle)."""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

import mtad_synth as S
import paper_2407_09722_b200 as M
from paper_2407_09722_b200.runtime import DeviceModel
from oracle import mtad_oracle as O
from oracle.adapters import oracle_model, bits

LP_TOL = 2e-3          # absolute tolerance on log-probabilities (per token and joint)
MARGIN = 1e-3          # decisions closer than this to a boundary are counted, not compared
# Error of one projection relative to its largest output; test_gpu_gemm.py holds the GEMM kernels alone to these (about
# twice what they show).  Up to 32 rows the activations enter as three bf16 terms, i.e. exactly, and what is left is the
# tensor cores' fp32 accumulation, which grows with the k-blocks summed in one accumulator; beyond 32 rows they enter
# as two terms (2^-17 relative per element).
GEMM_EPS_FEW = 1e-6    # up to 32 rows, K <= 2048
GEMM_EPS_WIDE = 8e-6   # up to 32 rows, K > 2048 (the 7B / 13B / 70B matrices)
GEMM_EPS_MANY = 6e-6   # more than 32 rows, K <= 2048


def gemm_eps(rows: int, k: int) -> float:
    return GEMM_EPS_WIDE if k > 2048 else (GEMM_EPS_FEW if rows <= 32 else GEMM_EPS_MANY)


class GpuModel(DeviceModel):
    """Seeded weights + KV cache on the device, the library context, and a lazily built oracle twin."""

    def __init__(self, *a, **k):
        super().__init__(*a, **k)
        self._oracle = None

    def oracle(self) -> O.OracleModel:
        if self._oracle is None:
            s = self.shape
            w = self.weights
            self._oracle = oracle_model(
                {"shape": s, "embed": w["embed"], "lm_head": w["lm_head"], "final_norm": w["final_norm"]},
                layer_maker=lambda l: w["layers"][l])
        return self._oracle

    def oracle_aux(self) -> O.OracleModel:
        if getattr(self, "_oracle_aux", None) is None:
            self._oracle_aux = oracle_model(self.aux_weights)
        return self._oracle_aux

    def inject_aux(self, seq: int, length: int):
        S.fill_kv_cache(self.aux_cache, 1, seq, length, self.seed)

    def aux_cache_bits(self, seq: int, upto: int) -> np.ndarray:
        s = self.aux_shape
        cap = self.aux_cache.shape[4]
        out = np.zeros((s.layers, 2, s.n_kv_heads, cap, s.head_dim), np.uint16)
        out[:, :, :, :upto] = bits(self.aux_cache[:, seq, :, :, :upto].contiguous())
        return out

    def upload(self, seq: int, target_bits: np.ndarray = None, aux_bits: np.ndarray = None):
        """Overwrite one sequence's device caches with host bit arrays [layers, 2, Hkv, cap, hd]."""
        if target_bits is not None:
            t = torch.from_numpy(target_bits.view(np.int16)).view(torch.bfloat16).cuda()
            self.cache[:, seq] = t
        if aux_bits is not None:
            t = torch.from_numpy(aux_bits.view(np.int16)).view(torch.bfloat16).cuda()
            self.aux_cache[:, seq] = t

    def cache_bits(self, seq: int, upto: int) -> np.ndarray:
        """Host copy of one sequence's cache [layers, 2, Hkv, capacity, hd] as bf16 bits (only [0, upto) filled)."""
        out = np.zeros((self.shape.layers, 2, self.shape.n_kv_heads, self.capacity, self.shape.head_dim), np.uint16)
        out[:, :, :, :upto] = bits(self.cache[:, seq, :, :, :upto].contiguous())
        return out


@dataclass
class SeqCase:
    seq: int
    L: int
    root: int
    tree: S.DraftTree
    n_nodes: Optional[int] = None      # use only the first n nodes (ragged batches)


@dataclass
class ParityStats:
    max_lp_err: float = 0.0
    max_LP_err: float = 0.0
    max_lse_err: float = 0.0
    n_seq: int = 0
    eta_match: int = 0
    path_match: int = 0
    tok_match: int = 0
    near_ties: int = 0
    cache_rows: int = 0
    cache_exact: int = 0
    cache_max_excess: float = -1.0
    cache_scale: float = 0.0
    etas: List[int] = field(default_factory=list)

    def cache_ok(self, layers: int, gemm_error: float) -> bool:
        """The K/V rows a call appends, against the oracle's (fp64, rounded to bf16 once).

        The device rounds its fp32 value y to bf16, the oracle its fp64 value y*.  |y - y*| <= eps * s with s the
        largest |K/V| value of the call and eps = gemm_error per layer: gemm_error (gemm_eps above) is the bound
        test_gpu_gemm.py holds the projection alone to, and every layer adds one projection's worth to the residual
        stream the next one reads.  Two things follow.
        (1) Where both sides round the same way the elements are equal; where they do not they are one bf16 step of
        the value apart, at most 2^-7 |y*|; only next to zero can the difference exceed that, and then by no more than
        |y - y*|.  So excess = |got - want| - 2^-7 |want| <= eps * s everywhere.
        (2) A value rounds the other way when y* lies within eps * s of a rounding boundary; boundaries are
        2^-8 |y*| apart (at least), so that happens with probability min(1, 2 eps s / (2^-8 |y*|)).  For values spread
        like a normal distribution of standard deviation s / 4 (s is a four-sigma maximum) the mean of that is below
        q (1 + ln(1 / q)) * 0.8 with q = 2048 eps - the bound on the share of unequal elements."""
        eps = gemm_error * layers
        q = 2048.0 * eps
        flips = 0.8 * q * (1.0 + math.log(1.0 / q))
        rate = 1.0 - self.cache_exact / max(self.cache_rows, 1)
        print(f"cache: {self.cache_rows} elements, unequal share {rate:.2e} (bound {flips:.2e}), excess "
              f"{self.cache_max_excess:.2e} (bound {eps * self.cache_scale:.2e})")
        return self.cache_rows > 0 and self.cache_max_excess <= eps * self.cache_scale and rate <= flips

    def ok(self, tie_cap: Optional[int] = None) -> bool:
        """Log-probabilities within LP_TOL everywhere; every decision equal except in sequences that have one within
        MARGIN of going the other way, and those are few: at most a third of the sequences (rounded up) unless the
        test states another cap (warped rows add a top-k and a top-p boundary to every row).  The margins of a
        random-init model are spread over several nats, so a share like that already means something is off."""
        clean = self.n_seq - self.near_ties
        cap = (self.n_seq + 2) // 3 if tie_cap is None else tie_cap
        print(f"parity: {self.n_seq} sequences, {self.near_ties} near a tie (cap {cap}), eta/path/token equal in "
              f"{self.eta_match}/{self.path_match}/{self.tok_match}, largest error lp {self.max_lp_err:.2e} "
              f"LP {self.max_LP_err:.2e} lse {self.max_lse_err:.2e}")
        return (self.max_lp_err <= LP_TOL and self.max_LP_err <= LP_TOL and self.eta_match >= clean
                and self.path_match >= clean and self.tok_match >= clean and self.near_ties <= cap)


def _trim(tree: S.DraftTree, n: Optional[int]) -> S.DraftTree:
    if n is None or n >= len(tree.tok):
        return tree
    return S.DraftTree(tree.tok[:n], tree.parent[:n], tree.depth[:n], tree.logq[:n], tree.best_path, tree.logq_ref)


def run_gpu(gm: GpuModel, cases: Sequence[SeqCase], log_tau: float, u: torch.Tensor, chain: bool,
            commit: bool = True, warp=None) -> M.ResultBuffers:
    """One verify call (+ kv_commit) through the C-ABI. u: [B, vocab] device uniforms."""
    gm.ctx.mtad_set_warp(*(warp if warp is not None else (0, 1.0)))
    B = len(cases)
    seqs = [c.seq for c in cases]
    for c in cases:
        gm.ctx.mtad_seq_set(c.seq, c.L, c.root)
    if chain:
        g = len(cases[0].tree.tok)
        assert all(len(c.tree.tok) == g and c.n_nodes is None for c in cases)
        tok = torch.tensor([c.tree.tok for c in cases], dtype=torch.int32, device="cuda").view(B, g)
        lq = torch.tensor([c.tree.logq_ref for c in cases], dtype=torch.float32, device="cuda").view(B, g)
        res = M.ResultBuffers(B, g, g)
        gm.ctx.mtad_verify_chain(seqs, g, tok if g else None, lq if g else None, log_tau, u, res)
    else:
        N = max(len(c.tree.tok) for c in cases)
        D = max(max(c.tree.depth, default=1) for c in cases)
        tok = torch.zeros(B, N, dtype=torch.int32)
        par = torch.full((B, N), -1, dtype=torch.int32)
        ref = torch.zeros(B, D, dtype=torch.float32)
        nn = torch.zeros(B, dtype=torch.int32)
        for i, c in enumerate(cases):
            t = _trim(c.tree, c.n_nodes)
            n = len(t.tok)
            tok[i, :n] = torch.tensor(t.tok, dtype=torch.int32)
            par[i, :n] = torch.tensor(t.parent, dtype=torch.int32)
            ref[i, :len(t.logq_ref)] = torch.tensor(t.logq_ref, dtype=torch.float32)
            nn[i] = n
        res = M.ResultBuffers(B, N, D)
        gm.ctx.mtad_verify_tree(seqs, nn.cuda(), N, D, tok.cuda(), par.cuda(), ref.cuda(), log_tau, u, res)
    if commit:
        gm.ctx.kv_commit(seqs, res)
    torch.cuda.synchronize()
    return res


def run_oracle(gm: GpuModel, case: SeqCase, cache_before: np.ndarray, log_tau: float, u_row: np.ndarray,
               chain: bool, warp=None):
    t = _trim(case.tree, case.n_nodes)
    model = gm.oracle()
    cache = cache_before
    if chain:
        # the device receives fp32 draft log-likelihoods; the oracle gets the same values
        lq = np.asarray(t.logq_ref, dtype=np.float32).astype(np.float64)
        r = O.verify_chain(model, cache, case.L, case.root, t.tok, lq, log_tau, u_row, warp=warp)
    else:
        ref = np.asarray(t.logq_ref, dtype=np.float32).astype(np.float64)
        r = O.verify_tree(model, cache, case.L, case.root, t.tok, t.parent, ref, log_tau, u_row, warp=warp)
    newL = O.kv_commit(cache, case.L, r.path)
    return r, cache, newL


WARP_MARGIN = 1e-3     # a warping decision (top-k boundary in logits, top-p cut in probability) closer than this is a tie


def _max_abs_diff(got: np.ndarray, want: np.ndarray) -> float:
    """Largest |got - want| over finite entries; an entry that is -inf on one side only counts as inf."""
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    if got.size == 0:
        return 0.0
    fin = np.isfinite(got) & np.isfinite(want)
    if np.any(np.isfinite(got) != np.isfinite(want)):
        return float("inf")
    return float(np.max(np.abs(got[fin] - want[fin]))) if np.any(fin) else 0.0


def compare(gm: GpuModel, cases: Sequence[SeqCase], log_tau: float, u: torch.Tensor, chain: bool,
            stats: Optional[ParityStats] = None, check_cache: bool = True, warp=None,
            only: Optional[Sequence[int]] = None) -> ParityStats:
    """Run both sides on the same inputs and accumulate the comparison.  warp = (top_k, top_p): warped target rows on
    both sides; a sequence with a warping decision within WARP_MARGIN of going the other way counts as a near tie
    and only its decisions-independent outputs are skipped."""
    stats = stats or ParityStats()
    before = [gm.cache_bits(c.seq, c.L) if (only is None or i in only) else None for i, c in enumerate(cases)]
    res = run_gpu(gm, cases, log_tau, u, chain, warp=warp)
    h = res.host()
    u_host = u.cpu().numpy()
    for i, c in enumerate(cases):
        assert int(h["status"][i]) == 0, f"device status {int(h['status'][i])}"
        if only is not None and i not in only:      # the device ran the whole batch; the oracle follows a part of it
            continue
        r, ocache, newL = run_oracle(gm, c, before[i], log_tau, u_host[i], chain, warp=warp)
        n = len(r.node_lp)
        warp_tie = r.margin_warp < WARP_MARGIN
        if n and not warp_tie:
            stats.max_lp_err = max(stats.max_lp_err, _max_abs_diff(h["node_lp"][i, :n].numpy(), r.node_lp))
            stats.max_LP_err = max(stats.max_LP_err, _max_abs_diff(h["node_LP"][i, :n].numpy(), r.node_LP))
        if warp is None:
            stats.max_lse_err = max(stats.max_lse_err,
                                    float(np.max(np.abs(h["row_lse"][i, :n + 1].numpy() - r.row_lse))))
        stats.n_seq += 1
        stats.etas.append(r.eta)
        near = min(r.margin_accept, r.margin_tie, r.margin_bonus) < MARGIN or warp_tie
        stats.near_ties += int(near)
        g_eta = int(h["eta"][i])
        g_path = h["path"][i, :g_eta].tolist()
        g_tok = h["out_tok"][i, :g_eta + 1].tolist()
        e_ok = g_eta == r.eta
        p_ok = e_ok and g_path == r.path and int(h["winner"][i]) == r.winner
        t_ok = p_ok and g_tok == r.out_tok and int(h["n_out"][i]) == r.eta + 1
        stats.eta_match += int(e_ok)
        stats.path_match += int(p_ok)
        stats.tok_match += int(t_ok)
        if t_ok:
            lp_err = np.max(np.abs(h["out_lp"][i, :g_eta + 1].numpy() - np.asarray(r.out_lp)))
            stats.max_lp_err = max(stats.max_lp_err, float(lp_err))
        if check_cache and p_ok:
            gL, groot = gm.ctx.mtad_seq_get(c.seq)
            assert gL == newL and groot == r.out_tok[-1] or not t_ok, (gL, newL)
            got = O.bf16_bits_to_f64(bits(gm.cache[:, c.seq, :, :, c.L:newL].contiguous()))
            want = O.bf16_bits_to_f64(ocache[:, :, :, c.L:newL])
            stats.cache_rows += got.size
            stats.cache_exact += int(np.sum(got == want))
            # a differing element is one bf16 rounding step apart (2^-8 relative at most) or, near zero, within the
            # fp32 accumulation error: report the excess over one step
            excess = np.abs(got - want) - 2.0 ** -7 * np.abs(want)
            stats.cache_max_excess = max(stats.cache_max_excess, float(np.max(excess)))
            stats.cache_scale = max(stats.cache_scale, float(np.max(np.abs(want))))
    damaged = gm.ctx.mtad_debug_check_canaries()
    assert damaged == "", f"write past the end of workspace array {damaged}"
    return stats
