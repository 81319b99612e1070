"""The projection entry point that allocates nothing, checked against the ordinary one.

Some users of this library cannot call cudaMalloc where they need the projection: a serving loop whose
device memory was planned at start-up, or a plugin that only works on buffers handed to it.  For them
jot_gemm_bf16_noalloc keeps the split-K scratch in a fixed array inside the library.  This file is
collected last on purpose, so a failure here cannot hide the result of any other test.
"""
import pytest
import torch

from helpers import bf16_matmul_oracle
from paper_2602_11133_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def jot():
    from paper_2602_11133_b200 import jot as binding
    binding._lib()
    return binding


def test_noalloc_projection_matches_ordinary_entry_point_twice(jot):
    """Two calls in a row (different inputs, the second with a residual) through the C ABI; the shared
    scratch still holds the first call's partial sums when the second one starts."""
    M, N, K = 200, 1024, 4096          # few output tiles, long K: the split-K path, which is what uses scratch
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for call, seed in enumerate((11, 12)):
        a = inputs.normal(seed, "a", (M, K), 1.0).cuda()
        w = inputs.normal(seed, "w", (N, K), 0.03).cuda()
        res = inputs.normal(seed, "r", (M, N), 1.0).cuda() if call == 1 else None
        want = jot.gemm_bf16(a, w, res, scratch=torch.empty(4 * M * N, dtype=torch.float32, device="cuda"))
        out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        n0 = jot.launch_count()
        jot.gemm_bf16_noalloc(a, w, res, out, status)
        assert jot.launch_count() - n0 == 2       # partial sums + reduction: the built-in scratch was used
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got, ref = out.float().cpu(), want.float().cpu()
        assert torch.isfinite(got).all()
        # the tolerance the projection tests use: one bf16 ulp of the value plus accumulation noise
        tol = 2.0 ** -8 * ref.abs() + 1e-3 * ref.abs().max()
        assert ((got - ref).abs() <= tol).all()
        assert ref.abs().max().item() > 0.1
        # ... and against the float64 definition of the projection, with the same tolerance
        exact = bf16_matmul_oracle(a.cpu(), w.cpu(), None if res is None else res.cpu())
        assert ((got.double() - exact).abs() <= 2.0 ** -8 * exact.abs() + 1e-3 * exact.abs().max()).all()


def test_noalloc_projection_rejects_what_does_not_fit(jot):
    M, N, K = 1024, 1032, 64           # 4 * M * N * 4 bytes = 16.1 MiB > 16 MiB
    assert 4 * M * N * 4 > jot.NOALLOC_SCRATCH_BYTES
    a = torch.zeros(M, K, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(N, K, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(M, N, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    n0 = jot.launch_count()
    with pytest.raises(jot.JotError) as e:
        jot.gemm_bf16_noalloc(a, w, None, out, status)
    assert e.value.status == -7 and "scratch" in str(e.value)
    assert jot.launch_count() == n0    # refused before anything was launched
    # the largest size that fits is accepted
    M2 = (jot.NOALLOC_SCRATCH_BYTES // 16) // N
    jot.gemm_bf16_noalloc(a[:M2].contiguous(), w, None, out[:M2].contiguous(), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
