"""The tensor-core weight-streaming GEMMs alone (mtad_debug_gemm: the stream-K kernel and the two cluster kernels)
against an fp64 matmul of the same bf16 weights."""
import pytest
import torch

import mtad_synth as S
from paper_2407_09722_b200 import binding as Bn
from tests.parity import gemm_eps
from paper_2407_09722_b200.runtime import DeviceModel

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def small_ctx():
    # F = 1408 bounds K, vocab 4096 bounds the tile count of the workspace
    return DeviceModel(S.ModelShape(1, 256, 4, 4, 64, 1408, 4096), max_batch=1, max_nodes=255, capacity=320)


def _check(dm, N, K, T, seed, variant=0, allow_small_workspace=False):
    W = S.normal_bf16(seed, 1000 + N + K, N * K, 0.02, "cuda").view(N, K)
    x = S.normal_bf16(seed, 2000 + T + K, T * K, 1.0, "cuda").float().view(T, K)
    x = x * (1.0 + 1e-3 * torch.arange(T * K, device="cuda").view(T, K).remainder(7))     # not bf16-representable
    y = torch.full((T, N), float("nan"), device="cuda")
    rc = dm.ctx.mtad_debug_gemm(W, x, y, variant=variant, check=False)
    if variant == 1 and rc == Bn.MTAD_E_UNIMPLEMENTED:
        return False                                 # the shape does not suit the cluster kernels
    if allow_small_workspace and rc == Bn.MTAD_E_WORKSPACE:
        return False                                 # the context's split-K workspace (sized for its model) is too small
    assert rc == 0, rc
    torch.cuda.synchronize()
    ref = x.double() @ W.double().t()
    err = (y.double() - ref).abs().max().item()
    scale = ref.abs().max().item()
    tol = gemm_eps(T, K)            # the classes and what they rest on: tests/parity.py
    print(f"gemm variant {variant} N={N} K={K} T={T}: error / scale {err / max(scale, 1.0):.2e} (bound {tol:.1e})")
    assert err <= tol * max(scale, 1.0), (N, K, T, err, scale)
    return True


@pytest.mark.parametrize("N,K,T", [(128, 64, 1), (128, 256, 5), (256, 256, 16), (384, 688, 17), (200, 136, 3),
                                   (1024, 1408, 65), (4096, 256, 129), (640, 1024, 256), (4096, 1408, 5)])
def test_debug_gemm_shapes(small_ctx, N, K, T):
    _check(small_ctx, N, K, T, 0)


# cluster kernels: up to 32 rows the small one (clusters of up to eight CTAs over a 128-feature tile), beyond the big one
# (two halves per tile, bulk copies between the CTAs); ragged N, K and T, one k-block per CTA, a single-CTA cluster
@pytest.mark.parametrize("N,K,T,runs", [(128, 64, 1, True), (128, 256, 5, True), (384, 688, 17, True), (200, 136, 3, True),
                                        (4096, 1408, 5, True), (4096, 256, 32, True),
                                        (1024, 1408, 65, True), (1024, 1408, 33, True), (640, 1024, 128, None),
                                        (200, 136, 40, True), (4096, 256, 100, None), (4096, 512, 65, True),
                                        (4096, 256, 129, False), (640, 1024, 256, False)])
def test_debug_gemm_cluster_shapes(small_ctx, N, K, T, runs):
    ran = _check(small_ctx, N, K, T, 3, variant=1)         # (runs = None: either way, as the shared-memory plan has it)
    assert runs is None or ran == runs


def test_debug_gemm_cluster_twice_is_bit_identical(small_ctx):
    N, K, T = 1024, 1408, 65
    W = S.normal_bf16(1, 7, N * K, 0.02, "cuda").view(N, K)
    x = torch.randn(T, K, device="cuda")
    a = torch.empty(T, N, device="cuda"); b = torch.empty(T, N, device="cuda")
    small_ctx.ctx.mtad_debug_gemm(W, x, a, variant=1)
    small_ctx.ctx.mtad_debug_gemm(W, x, b, variant=1)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_debug_gemm_twice_is_bit_identical(small_ctx):
    N, K, T = 1024, 1408, 33
    W = S.normal_bf16(1, 7, N * K, 0.02, "cuda").view(N, K)
    x = torch.randn(T, K, device="cuda")
    a = torch.empty(T, N, device="cuda"); b = torch.empty(T, N, device="cuda")
    small_ctx.ctx.mtad_debug_gemm(W, x, a)
    small_ctx.ctx.mtad_debug_gemm(W, x, b)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_debug_gemm_7b_shapes():
    dm = DeviceModel(S.ModelShape(1, 4096, 32, 32, 128, 11008, 32000), max_batch=1, max_nodes=8, capacity=64)
    for (N, K, T) in [(4096, 4096, 5), (4096, 11008, 5), (32000, 4096, 9)]:
        _check(dm, N, K, T, 2)
        assert _check(dm, N, K, T, 2, variant=1)


def test_debug_gemm_seeded_shape_sweep(small_ctx):
    """Ragged shapes drawn from a seeded generator, through the stream-K kernel and - where the plan takes them - the
    cluster kernels: row counts on both sides of the 32-row boundary between the two cluster kernels, feature counts
    that are no multiple of a tile, k that is no multiple of a k-block."""
    import random
    rng = random.Random(2407)
    ran_cluster = ran_stream = 0
    for i in range(24):
        T = rng.choice([rng.randint(1, 32), rng.randint(33, 128)])
        N = rng.randint(1, 32) * 128 - rng.choice([0, 0, 8, 56, 120])
        K = rng.randint(2, 176) * 8
        ran = _check(small_ctx, N, K, T, 100 + i, variant=0, allow_small_workspace=True)
        ran_stream += bool(ran)
        ran_cluster += bool(_check(small_ctx, N, K, T, 100 + i, variant=1, allow_small_workspace=True))
    print(f"sweep: {ran_stream} shapes through the stream-K kernel, {ran_cluster} through the cluster kernels")
    assert ran_stream >= 16 and ran_cluster >= 12
