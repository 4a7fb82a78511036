"""ctypes binding of libmtad.so: the same entry points as include/mtad.h, argument marshalling only.

Every step of the verification path runs inside the library's CUDA kernels; this module only turns torch
tensors into pointers.  There is no fallback: if the library is missing or cannot be loaded, importing a
function from here raises.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Dict, List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmtad.so")

MTAD_OK = 0
MTAD_E_INVALID, MTAD_E_CAPACITY, MTAD_E_CUDA, MTAD_E_TIMEOUT, MTAD_E_UNIMPLEMENTED, MTAD_E_WORKSPACE = \
    -1, -2, -3, -4, -5, -6
MTAD_MAX_BATCH, MTAD_MAX_NODES, MTAD_MAX_DEPTH, MTAD_LAYER_TENSORS = 64, 255, 32, 9
ST_BAD_PARENT, ST_BAD_TOKEN, ST_KV_OVERFLOW, ST_TOO_DEEP, ST_BAD_COUNT, ST_TIMEOUT = 1, 2, 4, 8, 16, 32
LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


class ModelDesc(C.Structure):
    _fields_ = [("layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("rope_base", C.c_float), ("rms_eps", C.c_float),
                ("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("layer_weights", C.POINTER(C.c_void_p)), ("kv_cache", C.c_void_p), ("kv_capacity", C.c_int64)]


class Result(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("eta", "winner", "path", "n_out", "out_tok", "out_lp", "node_lp",
                                           "node_LP", "row_lse", "row_cand", "row_cand_lp", "margin", "status")]


class Extent(C.Structure):
    _fields_ = [("what", C.c_char_p), ("reach", C.c_int64), ("extent", C.c_int64)]


AUDIT_VERIFY, AUDIT_DRAFT, AUDIT_COMMIT = 0, 1, 2

EXPORTS = ("mtad_workspace_bytes", "mtad_create", "mtad_destroy", "mtad_seq_set", "mtad_seq_get", "mtad_draft",
           "mtad_verify_chain", "mtad_verify_tree", "kv_commit", "mtad_status_str", "mtad_last_cuda_error",
           "mtad_profile_begin", "mtad_profile_end", "mtad_kernel_launches", "mtad_verify_chain_static",
           "mtad_debug_gemm", "mtad_set_warp", "mtad_set_draft_warp", "mtad_profile_grouped",
           "mtad_verify_chain_spd", "mtad_seq_hint", "mtad_debug_set_wait", "mtad_audit_extents",
           "mtad_debug_check_canaries", "mtad_debug_region")
MTAD_STATIC_SCRATCH_BYTES = 16 << 20
MTAD_ST_TIMEOUT, MTAD_ST_AUX_PENDING, MTAD_ST_NONFINITE, MTAD_ST_RANGE = 32, 64, 128, 256      # device status bits (mtad.h)
KERNEL_CLASSES = ("prepare", "norm", "gemm", "rope_append", "attention", "lm_reduce", "accept", "commit")

_lib = None


def load_library() -> C.CDLL:
    """Load libmtad.so (built in-tree by paper_2407_09722_b200.build).  Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2407_09722_b200.build` first "
                           "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    P, I, F = C.c_void_p, C.c_int, C.c_float
    MD, RS = C.POINTER(ModelDesc), C.POINTER(Result)
    I32P = C.POINTER(C.c_int32)
    lib.mtad_workspace_bytes.argtypes = [MD, MD, I, I, C.POINTER(C.c_size_t)]
    lib.mtad_create.argtypes = [MD, MD, I, I, P, C.c_size_t, C.POINTER(P)]
    lib.mtad_destroy.argtypes = [P]
    lib.mtad_seq_set.argtypes = [P, I, C.c_int32, C.c_int32, C.c_int32, I32P, P]
    lib.mtad_seq_get.argtypes = [P, I, I32P, I32P, P]
    lib.mtad_set_warp.argtypes = [P, I, C.c_float]
    lib.mtad_set_draft_warp.argtypes = [P, I, C.c_float]
    lib.mtad_seq_hint.argtypes = [P, I, C.c_int32]
    lib.mtad_audit_extents.argtypes = [MD, MD, I, I, I, I, I, I, I, C.c_int64, C.POINTER(Extent), I, C.POINTER(I)]
    lib.mtad_debug_set_wait.argtypes = [P, C.c_uint, I]
    lib.mtad_debug_region.argtypes = [P, C.c_char_p, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.mtad_debug_check_canaries.argtypes = [P, P, C.POINTER(C.c_char_p)]
    lib.mtad_profile_grouped.argtypes = [P, I]
    lib.mtad_draft.argtypes = [P, I, I32P, I, I, I, P, P, P, P, P, P, P, P, P]
    lib.mtad_verify_chain.argtypes = [P, I, I32P, I, P, P, F, P, RS, P]
    lib.mtad_verify_tree.argtypes = [P, I, I32P, P, I, I, P, P, P, F, P, RS, P]
    lib.mtad_verify_chain_spd.argtypes = [P, I, I32P, I, P, P, P, P, RS, P]
    lib.kv_commit.argtypes = [P, I, I32P, RS, P]
    lib.mtad_status_str.argtypes = [I]
    lib.mtad_status_str.restype = C.c_char_p
    lib.mtad_last_cuda_error.argtypes = [P]
    lib.mtad_profile_begin.argtypes = [P, I]
    lib.mtad_profile_end.argtypes = [P, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    lib.mtad_kernel_launches.argtypes = []
    lib.mtad_debug_gemm.argtypes = [P, P, I, I, P, I, P, I, P]
    lib.mtad_verify_chain_static.argtypes = [MD, C.c_int32, C.c_int32, I, P, P, F, P, RS, P]
    for n in EXPORTS:
        if n not in ("mtad_status_str", "mtad_kernel_launches"):
            getattr(lib, n).restype = I
    lib.mtad_kernel_launches.restype = C.c_uint64
    _lib = lib
    return lib


class MtadError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0):
        self.code, self.cuda = code, cuda
        msg = load_library().mtad_status_str(code).decode()
        super().__init__(f"{where}: {msg} ({code})" + (f", cudaError {cuda}" if cuda else ""))


def _ptr(t: Optional[torch.Tensor], dtype=None) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device pointers must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return t.data_ptr()


def _seqs(seqs: Sequence[int]):
    return (C.c_int32 * len(seqs))(*seqs)


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def make_desc(shape, weights: dict, kv_cache: torch.Tensor, keep: list) -> ModelDesc:
    """Descriptor from a model dict {'embed','lm_head','final_norm','layers':[{...}]} of CUDA bf16 tensors and a
    cache tensor [layers, max_batch, 2, Hkv, capacity, head_dim].  `keep` receives the objects that must outlive
    the descriptor."""
    arr = (C.c_void_p * (shape.layers * MTAD_LAYER_TENSORS))()
    for l, lw in enumerate(weights["layers"]):
        for i, n in enumerate(LAYER_TENSORS):
            arr[l * MTAD_LAYER_TENSORS + i] = _ptr(lw[n], torch.bfloat16)
    keep.append(arr)
    keep.append(weights)
    keep.append(kv_cache)
    assert kv_cache.dtype == torch.bfloat16 and kv_cache.dim() == 6
    return ModelDesc(shape.layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                     shape.vocab, shape.rope_base, shape.rms_eps,
                     _ptr(weights["embed"], torch.bfloat16), _ptr(weights["lm_head"], torch.bfloat16),
                     _ptr(weights["final_norm"], torch.bfloat16), C.cast(arr, C.POINTER(C.c_void_p)),
                     _ptr(kv_cache), kv_cache.shape[4])


def mtad_workspace_bytes(target: ModelDesc, aux: Optional[ModelDesc], max_batch: int, max_nodes: int) -> int:
    out = C.c_size_t(0)
    rc = load_library().mtad_workspace_bytes(C.byref(target), C.byref(aux) if aux is not None else None,
                                             max_batch, max_nodes, C.byref(out))
    if rc != MTAD_OK:
        raise MtadError(rc, "mtad_workspace_bytes")
    return out.value


class ResultBuffers:
    """Caller-owned device arrays of one verify call, plus the struct that points at them."""

    def __init__(self, B: int, N: int, D: int, device="cuda"):
        i32 = dict(dtype=torch.int32, device=device)
        self.B, self.N, self.D = B, N, D
        # one allocation, the members are views: `head` (eta, n_out, status, out_tok, out_lp - what a decode loop reads
        # back every step) is contiguous, so that a caller can fetch it with a single device-to-host copy
        shapes = [("eta", (B,), torch.int32), ("n_out", (B,), torch.int32), ("status", (B,), torch.int32),
                  ("out_tok", (B, D + 1), torch.int32), ("out_lp", (B, D + 1), torch.float32),
                  ("winner", (B,), torch.int32), ("path", (B, max(D, 1)), torch.int32),
                  ("node_lp", (B, max(N, 1)), torch.float32), ("node_LP", (B, max(N, 1)), torch.float32),
                  ("row_lse", (B, N + 1), torch.float32), ("row_cand", (B, N + 1), torch.int32),
                  ("row_cand_lp", (B, N + 1), torch.float32), ("margin", (B, 2), torch.float32)]
        words = [int(math.prod(sh)) for _, sh, _ in shapes]
        self.buf = torch.zeros(sum(words), **i32)
        self.head_fields, off = {}, 0
        for (name, sh, dt), n in zip(shapes, words):
            v = self.buf[off:off + n]
            setattr(self, name, (v if dt == torch.int32 else v.view(torch.float32)).view(*sh))
            if name in ("eta", "n_out", "status", "out_tok", "out_lp"):
                self.head_fields[name] = (off, sh, dt)
            off += n
        self.head = self.buf[:sum(words[:5])]
        self.struct = Result(*[getattr(self, n).data_ptr() for n, _ in Result._fields_])

    def host(self) -> Dict[str, torch.Tensor]:
        return {n: getattr(self, n).cpu() for n, _ in Result._fields_}

    def head_views(self, host_head: torch.Tensor) -> Dict[str, torch.Tensor]:
        """Views of a host copy of `head` (an int32 tensor of the same length) under the members' names."""
        out = {}
        for name, (off, sh, dt) in self.head_fields.items():
            v = host_head[off:off + int(math.prod(sh))]
            out[name] = (v if dt == torch.int32 else v.view(torch.float32)).view(*sh)
        return out


class Context:
    """Owns the workspace tensor and the opaque mtad_ctx handle; methods are the C entry points by name."""

    def __init__(self, target: ModelDesc, aux: Optional[ModelDesc], max_batch: int, max_nodes: int, keep=None):
        self._lib = load_library()
        self._keep = [target, aux, keep]
        nbytes = mtad_workspace_bytes(target, aux, max_batch, max_nodes)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        base = (self.workspace.data_ptr() + 255) & ~255
        h = C.c_void_p()
        rc = self._lib.mtad_create(C.byref(target), C.byref(aux) if aux is not None else None, max_batch, max_nodes,
                                   base, nbytes, C.byref(h))
        if rc != MTAD_OK:
            raise MtadError(rc, "mtad_create")
        self.handle = h
        self.workspace_bytes = nbytes

    def _check(self, rc: int, where: str):
        if rc != MTAD_OK:
            raise MtadError(rc, where, self._lib.mtad_last_cuda_error(self.handle))

    def close(self):
        if self.handle:
            self._lib.mtad_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def mtad_seq_set(self, seq: int, kv_len: int, root_token: int, aux_len: Optional[int] = None,
                     pending_tok: Optional[Sequence[int]] = None, stream=None):
        aux_len = kv_len if aux_len is None else aux_len
        pend = (C.c_int32 * len(pending_tok))(*pending_tok) if pending_tok else None
        self._check(self._lib.mtad_seq_set(self.handle, seq, kv_len, root_token, aux_len, pend, _stream(stream)),
                    "mtad_seq_set")

    def mtad_set_warp(self, top_k: int, top_p: float = 1.0, check=True) -> int:
        rc = self._lib.mtad_set_warp(self.handle, top_k, top_p)
        if check:
            self._check(rc, "mtad_set_warp")
        return rc

    def mtad_set_draft_warp(self, top_k: int, top_p: float = 1.0, check=True) -> int:
        rc = self._lib.mtad_set_draft_warp(self.handle, top_k, top_p)
        if check:
            self._check(rc, "mtad_set_draft_warp")
        return rc

    def mtad_seq_hint(self, seq: int, kv_len: int):
        self._check(self._lib.mtad_seq_hint(self.handle, seq, kv_len), "mtad_seq_hint")

    def mtad_debug_set_wait(self, wait_limit: int, no_operands: bool):
        self._check(self._lib.mtad_debug_set_wait(self.handle, wait_limit, 1 if no_operands else 0),
                    "mtad_debug_set_wait")

    def region(self, name: str, dtype) -> torch.Tensor:
        """View of the workspace array `name` (a live view of device memory, for tests)."""
        off, cnt, el = C.c_size_t(0), C.c_size_t(0), C.c_size_t(0)
        self._check(self._lib.mtad_debug_region(self.handle, name.encode(), C.byref(off), C.byref(cnt), C.byref(el)),
                    "mtad_debug_region")
        base = ((self.workspace.data_ptr() + 255) & ~255) - self.workspace.data_ptr()
        raw = self.workspace[base + off.value: base + off.value + cnt.value * el.value]
        return raw.view(dtype)

    def mtad_debug_check_canaries(self, stream=None) -> str:
        """Name of the first workspace array whose guard bytes are damaged, '' if all are intact."""
        name = C.c_char_p(None)
        n = self._lib.mtad_debug_check_canaries(self.handle, _stream(stream), C.byref(name))
        if n < 0:
            raise MtadError(n, "mtad_debug_check_canaries", self._lib.mtad_last_cuda_error(self.handle))
        return name.value.decode() if n > 0 and name.value else ""

    def mtad_seq_get(self, seq: int, stream=None):
        a, b = C.c_int32(), C.c_int32()
        self._check(self._lib.mtad_seq_get(self.handle, seq, C.byref(a), C.byref(b), _stream(stream)), "mtad_seq_get")
        return a.value, b.value

    def mtad_verify_chain(self, seqs, gamma: int, draft_tok, draft_logq, log_tau: float, bonus_uniform,
                          out: ResultBuffers, stream=None, check=True) -> int:
        rc = self._lib.mtad_verify_chain(self.handle, len(seqs), _seqs(seqs), gamma, _ptr(draft_tok, torch.int32),
                                         _ptr(draft_logq, torch.float32), log_tau,
                                         _ptr(bonus_uniform, torch.float32), C.byref(out.struct), _stream(stream))
        if check:
            self._check(rc, "mtad_verify_chain")
        return rc

    def mtad_verify_chain_spd(self, seqs, gamma: int, draft_tok, draft_logq_rows, accept_uniform, resample_uniform,
                              out: ResultBuffers, stream=None, check=True) -> int:
        rc = self._lib.mtad_verify_chain_spd(self.handle, len(seqs), _seqs(seqs), gamma,
                                             _ptr(draft_tok, torch.int32), _ptr(draft_logq_rows, torch.float32),
                                             _ptr(accept_uniform, torch.float32),
                                             _ptr(resample_uniform, torch.float32), C.byref(out.struct),
                                             _stream(stream))
        if check:
            self._check(rc, "mtad_verify_chain_spd")
        return rc

    def mtad_verify_tree(self, seqs, n_nodes, max_nodes: int, max_depth: int, tok, parent, logq_ref, log_tau: float,
                         bonus_uniform, out: ResultBuffers, stream=None, check=True) -> int:
        rc = self._lib.mtad_verify_tree(self.handle, len(seqs), _seqs(seqs), _ptr(n_nodes, torch.int32), max_nodes,
                                        max_depth, _ptr(tok, torch.int32), _ptr(parent, torch.int32),
                                        _ptr(logq_ref, torch.float32), log_tau, _ptr(bonus_uniform, torch.float32),
                                        C.byref(out.struct), _stream(stream))
        if check:
            self._check(rc, "mtad_verify_tree")
        return rc

    def kv_commit(self, seqs, res: ResultBuffers, stream=None, check=True) -> int:
        rc = self._lib.kv_commit(self.handle, len(seqs), _seqs(seqs), C.byref(res.struct), _stream(stream))
        if check:
            self._check(rc, "kv_commit")
        return rc

    def mtad_debug_gemm(self, W: torch.Tensor, x: torch.Tensor, y: torch.Tensor, stream=None, check=True,
                        variant: int = 0) -> int:
        N, K = W.shape
        T = x.shape[0]
        rc = self._lib.mtad_debug_gemm(self.handle, _ptr(W, torch.bfloat16), N, K, _ptr(x, torch.float32), T,
                                       _ptr(y, torch.float32), variant, _stream(stream))
        if check:
            self._check(rc, "mtad_debug_gemm")
        return rc

    def mtad_profile_begin(self, max_launches: int = 8192):
        self._check(self._lib.mtad_profile_begin(self.handle, max_launches), "mtad_profile_begin")

    def mtad_profile_grouped(self, on: bool):
        self._check(self._lib.mtad_profile_grouped(self.handle, 1 if on else 0), "mtad_profile_grouped")

    def mtad_profile_end(self) -> Dict[str, dict]:
        n = len(KERNEL_CLASSES)
        ms, by, cnt = (C.c_double * n)(), (C.c_double * n)(), (C.c_int64 * n)()
        self._check(self._lib.mtad_profile_end(self.handle, ms, by, cnt), "mtad_profile_end")
        return {k: {"ms": ms[i], "bytes": by[i], "launches": cnt[i]} for i, k in enumerate(KERNEL_CLASSES)}

    def mtad_draft(self, seqs, gamma: int, beam_width: int, uniforms, tok, parent, depth, node_logq, logq_ref,
                   best_path, stream=None, check=True, keep_all_candidates=False, n_nodes=None) -> int:
        """Node arrays hold gamma * beam_width entries per sequence, gamma * beam_width**2 with keep_all_candidates."""
        rc = self._lib.mtad_draft(self.handle, len(seqs), _seqs(seqs), gamma, beam_width,
                                  1 if keep_all_candidates else 0, _ptr(uniforms, torch.float32),
                                  None if n_nodes is None else _ptr(n_nodes, torch.int32),
                                  _ptr(tok, torch.int32), _ptr(parent, torch.int32),
                                  _ptr(depth, torch.int32), _ptr(node_logq, torch.float32),
                                  _ptr(logq_ref, torch.float32), _ptr(best_path, torch.int32), _stream(stream))
        if check:
            self._check(rc, "mtad_draft")
        return rc


def mtad_verify_chain_static(target: ModelDesc, kv_len: int, root_token: int, gamma: int, draft_tok, draft_logq,
                             log_tau: float, bonus_uniform, out: "ResultBuffers", stream=None) -> int:
    """Chain verification for one sequence with the library's built-in scratch array instead of a workspace:
    for callers that are not allowed to allocate device memory.  Returns the status code (no exception)."""
    return load_library().mtad_verify_chain_static(
        C.byref(target), kv_len, root_token, gamma, _ptr(draft_tok, torch.int32), _ptr(draft_logq, torch.float32),
        log_tau, _ptr(bonus_uniform, torch.float32), C.byref(out.struct), _stream(stream))


def shape_desc(shape, capacity: int) -> ModelDesc:
    """Descriptor of a model shape without any memory behind it (for the host-only extent audit)."""
    return ModelDesc(shape.layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                     shape.vocab, shape.rope_base, shape.rms_eps, None, None, None, None, None, capacity)


def mtad_audit_extents(target: ModelDesc, aux: Optional[ModelDesc], max_batch: int, max_nodes: int, call: int, B: int,
                       nodes: int, gamma: int, beam: int, len_ub: int):
    """[(what, reach, extent)] of one call shape: see mtad_audit_extents in mtad.h.  Host arithmetic only."""
    out = (Extent * 4096)()
    n = C.c_int(0)
    rc = load_library().mtad_audit_extents(C.byref(target), C.byref(aux) if aux is not None else None, max_batch,
                                           max_nodes, call, B, nodes, gamma, beam, len_ub, out, 4096, C.byref(n))
    if rc != MTAD_OK:
        raise MtadError(rc, "mtad_audit_extents")
    return [(out[i].what.decode(), out[i].reach, out[i].extent) for i in range(min(n.value, 4096))]


def mtad_kernel_launches() -> int:
    return int(load_library().mtad_kernel_launches())


def log_tau(tau: float) -> float:
    return -math.inf if tau == 0.0 else math.log(tau)
