"""hbfp_gemm_static: the GEMM for callers that cannot allocate device memory (a plug-in inside a
framework that owns the whole device, a loop where allocation is forbidden). It must give exactly
what hbfp_gemm gives, call after call, on the scratch built into the library.

Collected last on purpose: a run that stops at the first failure has then already run everything else."""
import numpy as np
import pytest

import oracle
from paper_1804_01526_b200 import workloads as wl
from tests.helpers import ofmt, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hb():
    from paper_1804_01526_b200 import binding
    binding.lib()
    return binding


CASES = [
    # (transA, transB, M, N, K, format kwargs): an ordinary tile grid, and a small output with a
    # long contraction, which splits K and therefore also keeps partial tiles in the scratch
    (0, 0, 256, 384, 512, dict(mant_bits=8, block=64, rounding=1, seed=5)),
    (1, 0, 200, 72, 4096, dict(mant_bits=8, block=32)),
    (0, 1, 96, 160, 320, dict(mant_bits=12, block=64, rounding=1, seed=7)),
]


def _allocation_state():
    """(requests torch's allocator has served so far, bytes it holds from the driver, bytes the driver has free)."""
    import gc
    import torch
    gc.collect()                              # tensors of earlier tests that only a cycle keeps alive
    torch.cuda.synchronize()
    stats = torch.cuda.memory_stats()
    return (stats["allocation.all.allocated"], stats["segment.all.allocated"], torch.cuda.memory_reserved(),
            torch.cuda.mem_get_info()[0])


@pytest.mark.parametrize("transA,transB,M,N,K,fd", CASES)
def test_static_scratch_matches_workspace_entry_point_twice(hb, transA, transB, M, N, K, fd):
    import torch
    A_host = wl.draw("lognormal", (K, M) if transA else (M, K), seed=41)
    B_host = wl.draw("lognormal", (N, K) if transB else (K, N), seed=42)
    A, B = to_dev(A_host), to_dev(B_host)
    fa, fb = hb.Format(**fd), hb.Format(**{**fd, "stream_id": 1})
    want = hb.gemm(transA, transB, A, B, fa, fb).cpu().numpy()
    ref = oracle.hbfp_gemm(transA, transB, A_host, B_host, ofmt(fd), ofmt(fd, stream_id=1))
    out = torch.empty((M, N), dtype=torch.float32, device="cuda")
    for call in range(2):                    # the second call finds the first call's bytes in the scratch
        out.fill_(float("nan"))
        if call == 1:                        # nothing is allocated: not through torch, not behind its back
            before = _allocation_state()
        got = hb.gemm_static(transA, transB, A, B, fa, fb, out=out)
        if call == 1:
            assert _allocation_state() == before
        got = got.cpu().numpy()
        # same kernels in the same order on the same inputs: the tolerance of the GEMM tests
        # (1e-6 of accumulator magnitude) tightens to bit equality here
        assert np.array_equal(got, want)
        # and against the oracle itself, within the tolerance the GEMM tests use
        err = np.abs(got.astype(np.float64) - ref["c_ref"].astype(np.float64))
        assert (err <= 1e-6 * ref["a_mag"]).all()
    assert hb.device_status() == 0


def test_static_scratch_rejects_what_does_not_fit(hb):
    import torch
    n = 4096                                  # packed operands alone need 2 x 16 MiB
    A = torch.zeros((n, n), device="cuda")
    f = hb.Format(8, 64)
    assert hb.gemm_workspace(0, 0, n, n, n, f, f) > hb.STATIC_WORKSPACE_BYTES
    with pytest.raises(hb.HbfpError) as e:
        hb.gemm_static(0, 0, A, A, f, f)
    assert e.value.code == hb.ERR_STATIC_LIMIT
    assert "built-in scratch" in str(e.value)
