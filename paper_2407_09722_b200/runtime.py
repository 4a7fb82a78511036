"""Device-side set-up shared by the tests, the benchmark and the smoke check: seeded weights and KV cache on the
GPU, the descriptors, and the library context.  No arithmetic of the method lives here."""
from __future__ import annotations

from typing import List, Optional

import torch

import mtad_synth as S
from . import binding as B


class DeviceModel:
    def __init__(self, target: S.ModelShape, max_batch: int, max_nodes: int, capacity: int, seed: int = 0,
                 aux: Optional[S.ModelShape] = None, aux_capacity: Optional[int] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: the verification path has no CPU fallback")
        B.load_library()
        dev = "cuda"
        self.shape, self.aux_shape, self.seed = target, aux, seed
        self.max_batch, self.max_nodes, self.capacity = max_batch, max_nodes, capacity
        self.weights = S.make_model(target, 0, seed, dev)
        self.cache = torch.zeros(S.kv_cache_shape(target, max_batch, capacity), dtype=torch.bfloat16, device=dev)
        self._keep: list = []
        self.desc = B.make_desc(target, self.weights, self.cache, self._keep)
        self.aux_desc = None
        if aux is not None:
            self.aux_weights = S.make_model(aux, 1, seed, dev)
            self.aux_cache = torch.zeros(S.kv_cache_shape(aux, max_batch, aux_capacity or capacity),
                                         dtype=torch.bfloat16, device=dev)
            self.aux_desc = B.make_desc(aux, self.aux_weights, self.aux_cache, self._keep)
        self.ctx = B.Context(self.desc, self.aux_desc, max_batch, max_nodes, keep=self._keep)

    def inject(self, seq: int, length: int):
        """Fill positions [0, length) of one sequence's target cache with seeded unit-variance bf16 K/V."""
        S.fill_kv_cache(self.cache, 0, seq, length, self.seed)


class StepInputs:
    """Device tensors of one verify call for a batch of draft trees (or chains)."""

    def __init__(self, trees: List[S.DraftTree], chain: bool, device="cuda", pin: bool = False):
        Bn = len(trees)
        self.chain = chain
        N = max(len(t.tok) for t in trees)
        D = max(max(t.depth, default=0) for t in trees)
        self.N, self.D = N, D
        tok = torch.zeros(Bn, max(N, 1), dtype=torch.int32)
        par = torch.full((Bn, max(N, 1)), -1, dtype=torch.int32)
        ref = torch.zeros(Bn, max(D, 1), dtype=torch.float32)
        nn = torch.zeros(Bn, dtype=torch.int32)
        for i, t in enumerate(trees):
            n = len(t.tok)
            tok[i, :n] = torch.tensor(t.tok, dtype=torch.int32)
            par[i, :n] = torch.tensor(t.parent, dtype=torch.int32)
            ref[i, :len(t.logq_ref)] = torch.tensor(t.logq_ref, dtype=torch.float32)
            nn[i] = n
        self.host = {"tok": tok, "parent": par, "logq_ref": ref, "n_nodes": nn}
        if pin:
            self.host = {k: v.pin_memory() for k, v in self.host.items()}
        self.dev = {k: v.to(device) for k, v in self.host.items()}

    def verify(self, ctx: B.Context, seqs, log_tau: float, u: torch.Tensor, res: B.ResultBuffers, dev=None):
        d = dev or self.dev
        if self.chain:
            ctx.mtad_verify_chain(seqs, self.N, d["tok"] if self.N else None, d["logq_ref"] if self.N else None,
                                  log_tau, u, res)
        else:
            ctx.mtad_verify_tree(seqs, d["n_nodes"], self.N, self.D, d["tok"], d["parent"], d["logq_ref"], log_tau,
                                 u, res)
