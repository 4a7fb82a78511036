#!/usr/bin/env python
"""Benchmark of the MTAD verification hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 7b_chain] [--impl ours|reference]

A step is one pass of the whole hot path over one batch of synthetic drafts: mtad_verify_chain / mtad_verify_tree
followed by kv_commit.  Consecutive steps are consecutive decode iterations (the committed length grows).  Prints
one JSON line (rank 0).  With N > 1 every rank runs an independent replica (the path does not shard).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import mtad_synth as S  # noqa: E402

TAU = 0.1
SEED = 0
# (DRAM read + write) / algorithmic bytes of the GEMM launches of one layer, ncu on the 4-layer workloads of the same
# shape (profiles/tc_gemm_7b_chain_4l.md, profiles/tc_gemm_7b_tree_4l.md); no figure for the other workloads
NCU_TRAFFIC_RATIO = {"7b_chain": 1.011, "7b_chain_4l": 1.011, "7b_chain_l512": 1.011, "7b_tree": 1.033, "7b_tree_4l": 1.033}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def step_trees(w: S.Workload, it: int):
    return [S.workload_tree(w, seq=b, seed=SEED, iteration=it) for b in range(w.batch)]


def algorithmic_bytes(w: S.Workload, lens) -> float:
    """bf16 weight bytes streamed once per step + committed K/V bytes of every sequence read once."""
    return w.target.streamed_weight_bytes() + w.target.kv_bytes_per_token() * float(sum(lens))


class ClockSampler:
    def __init__(self, index: int):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
        self.proc = None
        self.first = ""
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            # nvidia-smi stalls the driver for some milliseconds while it starts: let that pass before timing
            self.first = self.proc.stdout.readline()
        except OSError:
            pass

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, watts, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in (self.first + out).strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            try:
                watts.append(float(f[2]))
            except ValueError:
                pass
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons),
                "power_w_mean": sum(watts) / len(watts) if watts else None}


# ---------------------------------------------------------------------------------------------------------------
# reference arm and CPU baseline: the oracle, as it stands, on the host cores
# ---------------------------------------------------------------------------------------------------------------

def _blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


class OracleSampler:
    """Times the oracle's verify step on a model truncated to `n_layers` layers (same shapes and inputs) and on the
    same model with no layers (embedding, final norm, LM head, accept rule); the full-depth time is extrapolated
    as t0 + layers * (tn - t0) / n.  Accepted tokens are always those decided by the model truncated to ONE layer,
    whatever n_layers is, so that two samples of the same step count the same tokens."""

    def __init__(self, w: S.Workload, n_layers: int):
        from oracle import mtad_oracle as O
        from oracle.adapters import oracle_model, bits
        import numpy as np
        self.O, self.np, self.w, self.n = O, np, w, n_layers
        s = w.target
        dev = "cuda" if torch.cuda.is_available() else "cpu"
        head = {"shape": s, "embed": S.make_tensor(s, 0, "embed", seed=SEED, device=dev),
                "lm_head": S.make_tensor(s, 0, "lm_head", seed=SEED, device=dev),
                "final_norm": S.make_tensor(s, 0, "final_norm", seed=SEED, device=dev)}
        layers = [{k: bits(v) for k, v in S.make_layer(s, 0, l, SEED, dev).items()} for l in range(n_layers)]
        self.models = {}
        for n in sorted({0, 1, n_layers}):
            m = oracle_model(head, layer_maker=lambda l: None)
            m.layers = layers
            m.n_layers = n
            self.models[n] = m
        self.lens = S.kv_lengths(w, SEED)
        cap = max(self.lens) + w.n_nodes + 8
        cache = torch.zeros(S.kv_cache_shape(S.ModelShape(n_layers, s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim,
                                                          s.d_ffn, s.vocab), 1, cap), dtype=torch.bfloat16)
        S.fill_kv_cache(cache, 0, 0, self.lens[0], SEED)
        self.cache = bits(cache[:, 0]).copy()
        self.t0_last = None
        self.step(0)                      # untimed first touch (page faults, BLAS start-up)
        self.t0_last = None

    def step(self, it: int):
        """One sampled step for sequence 0 of the workload. Returns (estimated full-depth seconds for the whole
        batch, accepted tokens for the whole batch)."""
        O, np, w = self.O, self.np, self.w
        tree = S.workload_tree(w, seq=0, seed=SEED, iteration=it)
        u = S.bonus_uniforms(SEED, it, w.batch, w.target.vocab)[0].numpy()
        ref = np.asarray(tree.logq_ref, np.float32).astype(np.float64)
        ts = {}
        acc = 0
        for n in sorted({0, 1, self.n}):
            # the zero-layer run (embedding, final norm, LM head, accept rule) costs the same every step: it is timed on
            # every 16th step and its time reused in between, which keeps a long run of sampled steps within minutes
            if n == 0 and self.t0_last is not None and it % 16 != 0:
                ts[0] = self.t0_last
                continue
            cache = self.cache.copy()
            t0 = time.perf_counter()
            if w.kind == "chain":
                r = O.verify_chain(self.models[n], cache, self.lens[0], 1, tree.tok, ref, math.log(TAU), u)
            else:
                r = O.verify_tree(self.models[n], cache, self.lens[0], 1, tree.tok, tree.parent, ref, math.log(TAU), u)
            ts[n] = time.perf_counter() - t0
            if n == 0:
                self.t0_last = ts[0]
            if n == 1:
                acc = r.eta + 1
        per_layer = max(ts[self.n] - ts[0], 0.0) / self.n
        est = (ts[0] + w.target.layers * per_layer) * w.batch
        return est, acc * w.batch, ts


def run_reference(args, w: S.Workload):
    n_layers = 1
    smp = OracleSampler(w, n_layers)
    for i in range(args.warmup):
        smp.step(i)
    tot_t, tot_a = 0.0, 0
    for i in range(args.steps):
        est, acc, _ = smp.step(args.warmup + i)
        tot_t += est
        tot_a += acc
    value = tot_a / tot_t
    sample = (f"each step: oracle verify step of sequence 0 on the {w.name} shapes truncated to {n_layers} layer(s) "
              f"and to 0 layers (the latter timed every 16th step); full depth extrapolated as t0 + {w.target.layers} * (t{n_layers} - t0) / {n_layers}, "
              f"times batch {w.batch}")
    cores = _blas_threads()
    line = {"impl": "reference", "metric": "accepted_tokens_per_s", "value": value, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * tot_t / max(args.steps, 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "tau": TAU, "batch": w.batch, "rows_per_seq": w.n_nodes + 1,
                       "kv_len_start": smp.lens, "replicas": 1,
                       "l2": "inputs larger than L2 (weights streamed once per step)",
                       "block_efficiency": tot_a / max(args.steps * w.batch, 1), "warp": None},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def cpu_baseline(w: S.Workload, it: int = 0):
    n_layers = min(8, w.target.layers)
    smp = OracleSampler(w, n_layers)
    est, acc, ts = smp.step(it)
    return {"value": acc / est, "unit": "tokens/s", "cores": _blas_threads(), "kind": "oracle",
            "sample": (f"one oracle verify step of sequence 0 truncated to {n_layers} of {w.target.layers} layers "
                       f"({ts[n_layers]:.1f} s) and to 0 layers ({ts[0]:.1f} s); full depth extrapolated linearly, "
                       f"times batch {w.batch}: {est:.1f} s per step; tokens: the decision of the 1-layer model on "
                       f"step {it}, as in the --impl reference arm"),
            "est_step_s": est}


# ---------------------------------------------------------------------------------------------------------------
# replicas: every rank runs the whole path on its own sequences; only the timing and the token count are combined
# ---------------------------------------------------------------------------------------------------------------

def combine_ranks(local_ms: float, local_tokens: float, world: int, device="cuda"):
    """(max over ranks of the timed milliseconds, sum over ranks of the accepted tokens)."""
    if world <= 1:
        return local_ms, local_tokens
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    n = torch.tensor([local_tokens], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    torch.distributed.all_reduce(n, op=torch.distributed.ReduceOp.SUM)
    return float(t.item()), float(n.item())


def throughput(total_ms: float, tokens: float) -> float:
    return tokens / (total_ms * 1e-3)


# ---------------------------------------------------------------------------------------------------------------
# the whole iteration of Algorithm 1 with the library's own draft (chain workloads): mtad_draft -> verify -> commit
# ---------------------------------------------------------------------------------------------------------------

DRAFT_BEAM = 4          # the paper's smaller beam width


def draft_loop(w: S.Workload, steps: int, warmup: int, cap: int, warp=None):
    """Decode iterations in which the auxiliary model drafts by beam sampling, the target verifies and both caches are
    rolled forward.  Chain workloads verify the best beam (Algorithm 1); tree workloads keep every candidate of the
    beam sampling (beam * beam nodes a layer, the workload's tree size) and verify that tree as mtad_draft left it on
    the device (Sec. 3.3).  Returns tokens/s including the draft and the draft's share; a reported extra, not the
    headline (the headline times the verification path on synthetic drafts).  warp = (top_k, top_p): both models'
    rows warped as in the paper's experiments (App. F)."""
    import paper_2407_09722_b200 as M
    from paper_2407_09722_b200.runtime import DeviceModel
    lens = S.kv_lengths(w, SEED)
    tree = w.kind == "tree"
    g, B, V = w.gamma, w.batch, w.target.vocab
    b = DRAFT_BEAM
    if tree:                                   # the beam width whose candidates fill the workload's tree
        b = max(1, int(round(math.sqrt(w.n_nodes / g))))
    N = g * b * b if tree else g * b
    dm = DeviceModel(w.target, B, max(w.n_nodes, N), cap, SEED, aux=w.aux, aux_capacity=cap + g * b + 8)
    ctx = dm.ctx
    if warp:
        ctx.mtad_set_warp(*warp)
        ctx.mtad_set_draft_warp(*warp)
    seqs = list(range(B))
    for s_, L in enumerate(lens):
        dm.inject(s_, L)
        S.fill_kv_cache(dm.aux_cache, 1, s_, L, SEED)
        ctx.mtad_seq_set(s_, L, 1, aux_len=L)
    i32 = dict(dtype=torch.int32, device="cuda")
    f32 = dict(dtype=torch.float32, device="cuda")
    tok, parent, depth = (torch.zeros(B, N, **i32) for _ in range(3))
    node_logq, logq_ref, best = torch.zeros(B, N, **f32), torch.zeros(B, g, **f32), torch.zeros(B, g, **i32)
    n_nodes = torch.zeros(B, **i32)
    n_u = 4
    u_draft = [S.uniforms(SEED, (41 << 40) | i, B * g * b * V, "cuda").view(B, g, b, V) for i in range(n_u)]
    u_bonus = [S.bonus_uniforms(SEED, 1000 + i, B, V, "cuda") for i in range(n_u)]
    res = M.ResultBuffers(B, N, g) if tree else M.ResultBuffers(B, g, g)
    acc = torch.zeros((), dtype=torch.int64, device="cuda")
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    log_tau = math.log(TAU)
    for i in range(-warmup, steps):
        if i >= 0:
            ev[i][0].record()
        ctx.mtad_draft(seqs, g, b, u_draft[i % n_u], tok, parent, depth, node_logq, logq_ref, best,
                       keep_all_candidates=tree, n_nodes=n_nodes)
        if i >= 0:
            ev[i][1].record()
        if tree:
            ctx.mtad_verify_tree(seqs, n_nodes, N, g, tok, parent, logq_ref, log_tau, u_bonus[i % n_u], res)
        else:
            chain_tok = tok.gather(1, best.long())              # tokens of the best beam, in depth order
            ctx.mtad_verify_chain(seqs, g, chain_tok, logq_ref, log_tau, u_bonus[i % n_u], res)
        ctx.kv_commit(seqs, res)
        if i >= 0:
            acc += res.n_out.sum()
            ev[i][2].record()
        elif i == -1:
            acc.zero_()
    torch.cuda.synchronize()
    status = int(res.status.max().item())
    d_us = [1e3 * e[0].elapsed_time(e[1]) for e in ev]
    it_ms = [e[0].elapsed_time(e[2]) for e in ev]
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    accepted = float(acc.item())
    return {"value": accepted / (total_ms * 1e-3), "unit": "tokens/s", "steps": steps, "gamma": g, "beam": b,
            "nodes": N, "verified_as": "tree" if tree else "chain", "warp": list(warp) if warp else None,
            "block_efficiency": accepted / (steps * B), "iteration_ms": total_ms / steps,
            "draft_us_median": statistics.median(d_us), "verify_commit_us_median": 1e3 * statistics.median(it_ms)
            - statistics.median(d_us), "device_status": status}


# ---------------------------------------------------------------------------------------------------------------
# extra records of the default run: the other configuration the 70 % target is stated on, the rows sweep, the
# read-only streaming rate
# ---------------------------------------------------------------------------------------------------------------

def quantiles(xs):
    s = sorted(xs)
    q = lambda f: s[min(len(s) - 1, max(0, int(round(f * (len(s) - 1)))))]
    return {"median": statistics.median(s), "p10": q(0.1), "p90": q(0.9), "min": s[0], "max": s[-1]}


def quick_time(w: S.Workload, steps: int, warmup: int, profile: bool = True, dm=None):
    """Device-timed verify + commit steps of one workload (synthetic drafts, inputs resident): step-time quantiles,
    achieved share of the HBM roofline on the step's algorithmic bytes and, optionally, per-class event times."""
    import paper_2407_09722_b200 as M
    from paper_2407_09722_b200.runtime import DeviceModel, StepInputs
    lens = S.kv_lengths(w, SEED)
    chain = w.kind == "chain"
    total = warmup + steps
    cap = (max(lens) + (total + 2) * (w.gamma + 1) + w.n_nodes + 9 + 63) // 64 * 64
    own = dm is None
    if own:
        dm = DeviceModel(w.target, w.batch, w.n_nodes, cap, SEED)
    for b_, L in enumerate(lens):
        dm.inject(b_, L)
    ctx = dm.ctx
    seqs = list(range(w.batch))
    inputs = [StepInputs(step_trees(w, i), chain) for i in range(total)]
    unis = [S.bonus_uniforms(SEED, i, w.batch, w.target.vocab, "cuda") for i in range(min(total, 4))]
    res = M.ResultBuffers(w.batch, inputs[0].N, inputs[0].D)
    log_tau = math.log(TAU)

    def reset():
        for b_, L in enumerate(lens):
            ctx.mtad_seq_set(b_, L, 1)

    reset()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    acc = torch.zeros((), dtype=torch.int64, device="cuda")
    bad = torch.zeros((), dtype=torch.int32, device="cuda")
    for i in range(total):
        if i == warmup:
            torch.cuda.synchronize()
            acc.zero_()
            ev[0].record()
        inputs[i].verify(ctx, seqs, log_tau, unis[i % len(unis)], res)
        ctx.kv_commit(seqs, res)
        acc += res.n_out.sum()
        if i >= warmup:
            ev[i - warmup + 1].record()
    bad |= res.status.max()
    torch.cuda.synchronize()
    step_ms = [ev[k].elapsed_time(ev[k + 1]) for k in range(steps)]
    final = [ctx.mtad_seq_get(b_)[0] for b_ in seqs]
    peak, _ = measured_peaks()
    step_bytes = algorithmic_bytes(w, [(a + c) / 2 for a, c in zip(lens, final)])
    med = statistics.median(step_ms)
    out = {"workload": w.name, "batch": w.batch, "rows_per_seq": w.n_nodes + 1, "steps": steps,
           "step_us": {k: 1e3 * v for k, v in quantiles(step_ms).items()},
           "accepted_tokens_per_s": float(acc.item()) / (sum(step_ms) * 1e-3),
           "algorithmic_gb": step_bytes / 1e9, "achieved_gbs": step_bytes / (med * 1e-3) / 1e9,
           "frac_of_measured_copy": step_bytes / (med * 1e-3) / 1e9 / peak,
           "frac_of_8000": step_bytes / (med * 1e-3) / 1e9 / 8000.0, "device_status": int(bad.item())}
    if profile:
        reset()
        n = min(steps, 4)
        ctx.mtad_profile_grouped(True)
        ctx.mtad_profile_begin(n * (w.target.layers * 16 + 32))
        for i in range(n):
            inputs[i].verify(ctx, seqs, log_tau, unis[i % len(unis)], res)
            ctx.kv_commit(seqs, res)
        prof = ctx.mtad_profile_end()
        ctx.mtad_profile_grouped(False)
        out["per_class_ms_per_step"] = {k: v["ms"] / n for k, v in prof.items()}
        g = prof["gemm"]
        out["gemm_gbs"] = g["bytes"] / (g["ms"] * 1e-3) / 1e9 if g["ms"] > 0 else None
    if own:
        del dm, ctx
        torch.cuda.empty_cache()
    return out


def rows_sweep(steps: int, warmup: int):
    """Rows per forward R in {1, 2, 4, 8, 16} at the 13B shape on one set of weights: what the paper's batch-size
    table (Sec. 4) varies - the step time is nearly flat while the weights dominate the bytes."""
    from paper_2407_09722_b200.runtime import DeviceModel
    base = S.WORKLOADS["13b_batched_chain"]
    dm = DeviceModel(base.target, 1, 16, 2048 + 64 * 17, SEED)
    out = []
    for rows in (1, 2, 4, 8, 16):
        w = S.Workload(f"13b_rows{rows}", base.target, base.aux, batch=1, kind="chain", gamma=rows - 1, n_nodes=rows - 1,
                       kv_len=(2048, 2048))
        r = quick_time(w, steps, warmup, profile=False, dm=dm)
        out.append({"rows": rows, "step_us_median": r["step_us"]["median"], "frac_of_measured_copy": r["frac_of_measured_copy"]})
    del dm
    torch.cuda.empty_cache()
    return out


def read_only_peak(gb: float = 8.0):
    """Read-only streaming rate of this GPU: a sum over `gb` GB of fp32 (the path is read-dominated; the copy figure
    of MEASURED_PEAKS.json counts read + write)."""
    n = int(gb * 1e9 / 4)
    x = torch.ones(n, dtype=torch.float32, device="cuda")
    best = 0.0
    for _ in range(4):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        x.sum()
        e1.record()
        torch.cuda.synchronize()
        best = max(best, n * 4 / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    del x
    torch.cuda.empty_cache()
    return best


# ---------------------------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------------------------

def run_ours(args, w: S.Workload, rank: int, world: int, local_rank: int):
    import paper_2407_09722_b200 as M
    from paper_2407_09722_b200.runtime import DeviceModel, StepInputs

    torch.cuda.set_device(local_rank)
    lens = S.kv_lengths(w, SEED)
    chain = w.kind == "chain"
    rows = w.n_nodes + 1
    total_steps = args.warmup + args.steps
    cap = max(lens) + (total_steps + 2) * (w.gamma + 1) + rows + 8
    cap = (cap + 63) // 64 * 64
    dm = DeviceModel(w.target, w.batch, w.n_nodes, cap, SEED)
    for b, L in enumerate(lens):
        dm.inject(b, L)
    ctx = dm.ctx
    if args.top_k > 0:
        ctx.mtad_set_warp(args.top_k, args.top_p)      # the warping of the paper's experiments (App. F) on the target rows
    seqs = list(range(w.batch))
    V = w.target.vocab
    log_tau = math.log(TAU)

    inputs = [StepInputs(step_trees(w, i), chain, pin=True) for i in range(total_steps)]
    unis_host = [S.bonus_uniforms(SEED, i, w.batch, V).pin_memory() for i in range(total_steps)]
    unis = [u.cuda() for u in unis_host]
    res = M.ResultBuffers(w.batch, inputs[0].N, inputs[0].D)

    def reset():
        for b, L in enumerate(lens):
            ctx.mtad_seq_set(b, L, 1)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ---------------------------------------------------------------------------------
    reset()
    sampler = ClockSampler(local_rank)       # started before the warm-up: nvidia-smi needs a moment to come up
    acc_dev = torch.zeros((), dtype=torch.int64, device="cuda")
    bad_dev = torch.zeros((), dtype=torch.int32, device="cuda")      # OR of the per-sequence device status words
    for i in range(args.warmup):
        inputs[i].verify(ctx, seqs, log_tau, unis[i], res)
        ctx.kv_commit(seqs, res)
        acc_dev += res.n_out.sum()           # also warms up torch's own reduction kernel
    acc_dev.zero_()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    launches0 = M.mtad_kernel_launches()
    ev[0].record()
    for k in range(args.steps):
        i = args.warmup + k
        inputs[i].verify(ctx, seqs, log_tau, unis[i], res)
        ctx.kv_commit(seqs, res)
        acc_dev += res.n_out.sum()
        ev[k + 1].record()
        if k % 16 == 15 or k == args.steps - 1:      # outside the per-step events' critical path most of the time
            bad_dev |= res.status.max()
    barrier()
    device_status = int(bad_dev.item())
    if device_status != 0:
        raise RuntimeError(f"device status {device_status:#x} during the timed steps (see MTAD_ST_* in mtad.h)")
    launches = M.mtad_kernel_launches() - launches0
    clocks = sampler.stop()
    total_ms, accepted = combine_ranks(ev[0].elapsed_time(ev[-1]), float(acc_dev.item()), world)
    step_ms = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
    value = throughput(total_ms, accepted)
    final_lens = [ctx.mtad_seq_get(b)[0] for b in seqs]

    # ---- per-kernel passes: the same steps again under the library's event brackets -------------------------------
    # grouped: one event pair around every run of consecutive launches of a class (the four projections between two
    # attention passes keep their programmatic overlap, as in the timed steps); isolated: one pair per launch (an
    # event between two launches serialises them, so every kernel is timed as if it stood alone)
    prof_steps = min(args.steps, 4)

    def profile_pass(grouped: bool):
        reset()
        for i in range(min(args.warmup, 1)):
            inputs[i].verify(ctx, seqs, log_tau, unis[i], res)
            ctx.kv_commit(seqs, res)
        ctx.mtad_profile_grouped(grouped)
        ctx.mtad_profile_begin(prof_steps * (w.target.layers * 16 + 32))
        for k in range(prof_steps):
            i = args.warmup + k
            inputs[i].verify(ctx, seqs, log_tau, unis[i], res)
            ctx.kv_commit(seqs, res)
        out = ctx.mtad_profile_end()
        ctx.mtad_profile_grouped(False)
        return out

    prof_iso = profile_pass(False)
    prof = profile_pass(True)
    gemm, gemm_iso = prof["gemm"], prof_iso["gemm"]
    peak, peak_kind = measured_peaks()
    achieved = gemm["bytes"] / (gemm["ms"] * 1e-3) / 1e9 if gemm["ms"] > 0 else 0.0
    achieved_iso = gemm_iso["bytes"] / (gemm_iso["ms"] * 1e-3) / 1e9 if gemm_iso["ms"] > 0 else 0.0
    prof_total = sum(v["ms"] for v in prof.values())
    alg_per_launch = gemm["bytes"] / max(gemm["launches"], 1)
    ratio = NCU_TRAFFIC_RATIO.get(w.name)
    roofline = {"bound": "hbm",
                "kernel": "the weight-streaming GEMMs (tc_gemm_cluster_kernel / tc_gemm_cluster_big_kernel / tc_gemm_kernel: "
                          "all weight matrices + LM head)", "achieved": achieved,
                "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                "timing": "CUDA events on the launching stream around every run of consecutive GEMM launches "
                          "(O, gate/up, down, next QKV or LM head), summed and divided by the launches",
                "algorithmic_bytes_per_launch": alg_per_launch,
                # DRAM read + write bytes per launch: the ratio to the algorithmic bytes was taken with ncu on the
                # 4-layer workload of the same shape and scales with the weights streamed
                "traffic": alg_per_launch * ratio if ratio else None,
                "launches_per_step": gemm["launches"] / prof_steps,
                "avg_launch_us": 1e3 * gemm["ms"] / max(gemm["launches"], 1),
                "share_of_step": gemm["ms"] / prof_total if prof_total else None,
                "per_class_ms_per_step": {k: v["ms"] / prof_steps for k, v in prof.items()},
                "isolated": {"achieved": achieved_iso, "frac": achieved_iso / peak,
                             "avg_launch_us": 1e3 * gemm_iso["ms"] / max(gemm_iso["launches"], 1),
                             "per_class_ms_per_step": {k: v["ms"] / prof_steps for k, v in prof_iso.items()},
                             "timing": "one event pair per launch"}}

    # ---- end to end: host buffers in, host results out, every step --------------------------------------------------
    reset()
    # per step: ONE host-to-device copy of a pinned block (uniforms, then the draft arrays) and ONE device-to-host
    # copy of the result head (eta, n_out, status, out_tok, out_lp)
    names = list(inputs[0].host.keys())

    def pack(i):
        parts = [unis_host[i].view(torch.int32).flatten()]
        parts += [inputs[i].host[k].view(torch.int32).flatten() for k in names]
        return torch.cat(parts).pin_memory()

    packed = [pack(i) for i in range(total_steps)]
    stage_buf = torch.empty_like(packed[0], device="cuda")
    off = unis_host[0].numel()
    u_stage = stage_buf[:off].view(torch.float32).view_as(unis[0])
    stage = {}
    for k in names:
        v = inputs[0].host[k]
        piece = stage_buf[off:off + v.numel()]
        stage[k] = (piece if v.dtype == torch.int32 else piece.view(v.dtype)).view_as(v)
        off += v.numel()
    head_host = torch.empty_like(res.head, device="cpu").pin_memory()
    out_host = res.head_views(head_host)
    h2d = packed[0].numel() * 4
    d2h = head_host.numel() * 4

    def e2e_step(i):
        stage_buf.copy_(packed[i], non_blocking=True)
        inputs[i].verify(ctx, seqs, log_tau, u_stage, res, dev=stage)
        ctx.kv_commit(seqs, res)
        head_host.copy_(res.head, non_blocking=True)
        torch.cuda.synchronize()
        # log-likelihood of the emitted tokens under the target, for the output perplexity (Eq. 1)
        n = out_host["n_out"].long()
        emitted = torch.arange(out_host["out_lp"].shape[1])[None, :] < n[:, None]
        lp_sum[0] += float(out_host["out_lp"].double()[emitted].sum())
        return int(n.sum())

    lp_sum = [0.0]
    for i in range(args.warmup):
        e2e_step(i)
    lp_sum[0] = 0.0
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    acc_e2e = 0
    for k in range(args.steps):
        acc_e2e += e2e_step(args.warmup + k)
    e1.record()
    barrier()
    wall = time.perf_counter() - t0
    e2e_ms, e2e_tokens = combine_ranks(max(e0.elapsed_time(e1), wall * 1e3), float(acc_e2e), world)
    e2e_value = throughput(e2e_ms, e2e_tokens)

    if rank != 0:
        return
    mid_lens = [(a + b) / 2 for a, b in zip(lens, final_lens)]
    step_bytes = algorithmic_bytes(w, mid_lens)
    ms_per_step = total_ms / args.steps
    line = {
        "metric": "accepted_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "tau": TAU, "batch": w.batch, "rows_per_seq": rows, "kv_len_start": lens,
                   "replicas": world, "l2": "inputs larger than L2 (weights streamed once per step)",
                   "block_efficiency": accepted / (args.steps * w.batch * world),
                   "warp": {"top_k": args.top_k, "top_p": args.top_p} if args.top_k > 0 else None},
        "verify_step_us": {k: 1e3 * v for k, v in quantiles(step_ms).items()},
        "value_note": "verify + commit steps on synthetic drafts with synthetic draft likelihoods (no auxiliary model in "
                      "the timed region); draft_loop.value is accepted tokens/s of whole iterations with mtad_draft",
        "step_hbm": {"algorithmic_gb": step_bytes / 1e9, "achieved_gbs": step_bytes / (ms_per_step * 1e-3) / 1e9,
                     "frac_of_measured_copy": step_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
                     "frac_of_8000": step_bytes / (ms_per_step * 1e-3) / 1e9 / 8000.0},
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / args.steps},
        "gpu_launches": int(launches), "device_status": device_status,
        "clocks": clocks,
        # what the paper reports around the path (Eq. 1; Sec. 5 and App. D), on synthetic random-init models:
        # perplexity of the emitted tokens under the target, tokens per iteration, energy per token from the
        # sampled board power over the device-timed steps
        "metrics": {"output_ppl": math.exp(-lp_sum[0] / acc_e2e) if acc_e2e else None,
                    "tokens_per_iteration": accepted / (args.steps * w.batch * world),
                    "power_w_mean": clocks.get("power_w_mean"),
                    "joules_per_token": (clocks["power_w_mean"] * total_ms * 1e-3 * world / accepted
                                         if clocks.get("power_w_mean") and accepted else None)},
    }
    del dm, ctx
    torch.cuda.empty_cache()
    if world == 1 and not args.no_draft_loop:
        line["draft_loop"] = draft_loop(w, min(args.steps, 32), 3, cap,
                                        warp=(args.top_k, args.top_p) if args.top_k > 0 else None)
        torch.cuda.empty_cache()
    if world == 1 and not args.no_extras:
        line["read_only_peak_gbs"] = read_only_peak()
        if w.name != "7b_tree":
            wt = S.WORKLOADS["7b_tree"]
            line["tree"] = quick_time(wt, min(args.steps, 16), 3)
            if not args.no_draft_loop:
                n_it = min(args.steps, 16)
                line["tree"]["draft_loop"] = draft_loop(wt, n_it, 3, max(S.kv_lengths(wt, SEED)) + (n_it + 5) *
                                                        (wt.gamma + 1) + wt.n_nodes + 64)
            torch.cuda.empty_cache()
        line["rows_sweep_13b"] = rows_sweep(8, 3)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, args.warmup)
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--workload", default="7b_chain", choices=sorted(S.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-draft-loop", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the tree record, the rows sweep and the read-only rate")
    ap.add_argument("--top-k", type=int, default=0, help="warp the target rows: top-k (0 = off, the default)")
    ap.add_argument("--top-p", type=float, default=0.9)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = S.WORKLOADS[args.workload]
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if rank == 0:
            run_reference(args, w)
        return
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, w, rank, world, local_rank)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
