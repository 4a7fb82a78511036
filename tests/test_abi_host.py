"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared symbol, sizes the
workspace, and refuses malformed arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

import mtad_synth as S
import paper_2407_09722_b200 as M
from paper_2407_09722_b200 import binding as Bn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2407_09722_b200.build import build
    build()
    return M.load_library()


def _desc(shape, ptrs=False):
    d = Bn.ModelDesc(shape.layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                     shape.vocab, shape.rope_base, shape.rms_eps, None, None, None, None, None, 128)
    return d


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "mtad.h")).read()
    declared = set(re.findall(r"^(?:int|uint64_t|const char\*)\s+(\w+)\(", header, flags=re.M))
    assert declared == set(M.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert lib.mtad_status_str(0) == b"ok"
    for code in range(-6, 0):
        assert lib.mtad_status_str(code) not in (b"ok", b"unknown status")
    assert lib.mtad_status_str(-99) == b"unknown status"


def test_workspace_bytes_scales_and_validates(lib):
    t = _desc(S.WORKLOADS["tiny"].target)
    a = _desc(S.WORKLOADS["tiny"].aux)
    small = M.mtad_workspace_bytes(t, None, 1, 4)
    big = M.mtad_workspace_bytes(t, None, 8, 64)
    assert 0 < small < big and small % 256 == 0
    assert M.mtad_workspace_bytes(t, a, 1, 4) >= small
    seven = _desc(S.WORKLOADS["7b_tree"].target)
    assert M.mtad_workspace_bytes(seven, None, 1, 64) < 1 << 30
    out = C.c_size_t()
    assert lib.mtad_workspace_bytes(None, None, 1, 4, C.byref(out)) == Bn.MTAD_E_INVALID
    assert lib.mtad_workspace_bytes(C.byref(t), None, 0, 4, C.byref(out)) == Bn.MTAD_E_INVALID
    assert lib.mtad_workspace_bytes(C.byref(t), None, 65, 4, C.byref(out)) == Bn.MTAD_E_CAPACITY
    assert lib.mtad_workspace_bytes(C.byref(t), None, 1, 256, C.byref(out)) == Bn.MTAD_E_CAPACITY
    bad = _desc(S.ModelShape(2, 256, 4, 3, 64, 688, 1024))          # heads not divisible
    assert lib.mtad_workspace_bytes(C.byref(bad), None, 1, 4, C.byref(out)) == Bn.MTAD_E_INVALID
    bad = _desc(S.ModelShape(2, 256, 4, 4, 48, 688, 1024))          # unsupported head_dim
    assert lib.mtad_workspace_bytes(C.byref(bad), None, 1, 4, C.byref(out)) == Bn.MTAD_E_INVALID


def test_create_refuses_bad_arguments_without_touching_the_device(lib):
    t = _desc(S.WORKLOADS["tiny"].target)
    h = C.c_void_p()
    # null weights
    assert lib.mtad_create(C.byref(t), None, 1, 4, 256, 1 << 30, C.byref(h)) == Bn.MTAD_E_INVALID
    assert not h.value
    assert lib.mtad_create(C.byref(t), None, 1, 4, 256, 1 << 30, None) == Bn.MTAD_E_INVALID


def test_null_context_calls_are_rejected(lib):
    seqs = (C.c_int32 * 1)(0)
    r = Bn.Result()
    assert lib.mtad_verify_chain(None, 1, seqs, 4, None, None, -1.0, None, C.byref(r), None) == Bn.MTAD_E_INVALID
    assert lib.mtad_verify_tree(None, 1, seqs, None, 4, 4, None, None, None, -1.0, None, C.byref(r), None) \
        == Bn.MTAD_E_INVALID
    assert lib.kv_commit(None, 1, seqs, C.byref(r), None) == Bn.MTAD_E_INVALID
    assert lib.mtad_seq_set(None, 0, 0, 0, 0, None, None) == Bn.MTAD_E_INVALID
    assert lib.mtad_last_cuda_error(None) == 0
    assert lib.mtad_destroy(None) == 0
