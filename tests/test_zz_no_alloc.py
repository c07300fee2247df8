"""The allocation-free GEMM entry point against the allocating one.

gala_gemm_bf16_static is for processes that cannot call cudaMalloc while the library runs: the
device memory already belongs to a framework's allocator, or a device-wide stall is not
affordable.  It must give what gala_gemm_bf16 gives, call after call, although all calls share
one built-in scratch array that still holds the previous call's partial sums.

Collected last on purpose (file name): a failure here cannot hide the other tests in a run that
stops at the first failure.
"""
import numpy as np
import pytest

from tests.helpers import assert_close

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

# (groups, M, N, K, a_mn, b_mn, split_k): second call is smaller than the first and uses other
# layouts, so stale partial sums of the first call lie all over its scratch region; the last call has more
# splits than K tiles, i.e. a split with nothing to add, which must still overwrite what lies in its region
CALLS = [(2, 576, 64, 3920, 1, 1, 4), (1, 256, 40, 200, 1, 0, 2), (3, 300, 72, 136, 0, 0, 1), (1, 130, 130, 72, 0, 0, 3)]


def _operands(case, seed):
    groups, M, N, K, a_mn, b_mn, split = case
    g = torch.Generator(device="cpu").manual_seed(seed)
    a = torch.randn((groups, M, K), generator=g).cuda().to(torch.bfloat16)
    b = torch.randn((groups, N, K), generator=g).cuda().to(torch.bfloat16)
    if a_mn:
        a = a.transpose(1, 2).contiguous()
    if b_mn:
        b = b.transpose(1, 2).contiguous()
    return a, b


def test_static_scratch_gemm_matches_allocating_gemm_twice_in_a_row():
    from paper_1906_04585_b200 import binding as B
    st = torch.cuda.current_stream().cuda_stream
    for rep in range(2):                       # two passes: every call also follows a different call
        for idx, case in enumerate(CALLS):
            groups, M, N, K, a_mn, b_mn, split = case
            a, b = _operands(case, 100 * rep + idx)
            want = torch.full((groups, M, N), float("nan"), device="cuda")
            got = torch.full((groups, M, N), float("nan"), device="cuda")
            B.gala_gemm_bf16(a, b, want, groups, M, N, K, a_mn, b_mn, split, st)
            B.gala_gemm_bf16_static(a, b, got, groups, M, N, K, a_mn, b_mn, split, st)
            torch.cuda.synchronize()
            assert_close("D%s" % (case,), got.cpu().numpy(), want.cpu().numpy(), 1e-4)
            # same kernels, same summation order: in fact identical
            assert torch.equal(got, want)


def test_static_scratch_gemm_refuses_oversized_requests():
    from paper_1906_04585_b200 import binding as B
    a = torch.zeros((1, 2048, 64), device="cuda", dtype=torch.bfloat16)
    b = torch.zeros((1, 2048, 64), device="cuda", dtype=torch.bfloat16)
    d = torch.zeros((1, 2048, 2048), device="cuda")
    with pytest.raises(B.GalaError) as ei:    # 1 * 1 * 2048 * 2048 * split 1 is fine, split 2 is not (8 Mi floats)
        B.gala_gemm_bf16_static(a, b, d, 1, 2048, 2048, 64, 0, 0, 2, torch.cuda.current_stream().cuda_stream)
    assert ei.value.status == B.GALA_EINVAL and "8 MiB" in str(ei.value)
    B.gala_gemm_bf16_static(a, b, d, 1, 2048, 2048, 64, 0, 0, 1, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert float(d.abs().max()) == 0.0
