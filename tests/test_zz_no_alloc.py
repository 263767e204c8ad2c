"""specvla_gemm_static: the GEMM entry point for callers that may not allocate device memory
(stream captures, real-time loops, plug-ins that are handed only their buffers). Its scratch is
a fixed array inside the library, so this checks that it gives what specvla_gemm gives with
caller-allocated scratch, twice in a row on the shared array, and that it refuses shapes the
array cannot hold. Collected last on purpose: a failure here cannot hide another test."""
import pytest
import torch

from synth_inputs import rng

pytestmark = pytest.mark.gpu


def _case(seed, T, N, K):
    x = rng.normal(seed, 1, (T, K), 1.0, "cuda", dtype=torch.float32)
    w = rng.normal_bf16(seed, 2, (N, K), 0.02, "cuda")
    return x, w


def test_static_scratch_gemm_matches_allocating_gemm_twice():
    from paper_2507_22424_b200 import binding as B
    # the second call is smaller and of another row-tile size, so planes and limbs left behind by
    # the first call would show up in its result if they were not rewritten
    for seed, (T, N, K) in enumerate([(27, 4096, 4096), (9, 1000, 520)]):
        x, w = _case(31 + seed, T, N, K)
        assert B.lib.specvla_gemm_scratch_bytes(T, N, K) <= B.STATIC_SCRATCH_BYTES
        y = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
        got = B.gemm_static(x, w, y).cpu().double()
        want = B.gemm(x, w).cpu().double()
        ref = x.cpu().double() @ w.cpu().double().T
        tol = 1e-4 * 0.02 * (K ** 0.5) + 1e-6          # the tolerance of the GEMM parity tests
        assert torch.isfinite(got).all()
        assert (got - want).abs().max() < tol, float((got - want).abs().max())
        assert (got - ref).abs().max() < tol, float((got - ref).abs().max())


def test_static_scratch_gemm_rejects_oversize():
    from paper_2507_22424_b200 import binding as B
    T, N, K = 1024, 256, 8192          # the two limbs of X alone need 32 MiB
    assert B.lib.specvla_gemm_scratch_bytes(T, N, K) > B.STATIC_SCRATCH_BYTES
    x = torch.zeros(T, K, dtype=torch.float32, device="cuda")
    w = torch.zeros(N, K, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(T, N, dtype=torch.float32, device="cuda")
    with pytest.raises(B.SpecVLAError) as e:
        B.gemm_static(x, w, y)
    assert e.value.code == -2


def test_static_scratch_gemm_asynchronous_then_status():
    """wait = 0 (the form a stream capture needs): the call returns at once; the status of the
    built-in scratch is asked for afterwards."""
    import ctypes as C
    from paper_2507_22424_b200 import binding as B
    T, N, K = 27, 1024, 1024
    x, w = _case(41, T, N, K)
    y = torch.full((T, N), float("nan"), dtype=torch.float32, device="cuda")
    rc = B.lib.specvla_gemm_static(C.c_void_p(x.data_ptr()), C.c_void_p(w.data_ptr()), C.c_void_p(y.data_ptr()),
                                   T, N, K, 0, B._stream())
    assert rc == 0
    assert B.lib.specvla_gemm_static_status(B._stream()) == 0
    want = B.gemm(x, w).cpu().double()
    assert (y.cpu().double() - want).abs().max() < 1e-4 * 0.02 * (K ** 0.5) + 1e-6
