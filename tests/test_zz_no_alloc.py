"""GPU test of hgemm_run_splitk_static, the split-K GEMM whose scratch memory is a static array
inside the library (for callers that may not allocate device memory: a memory-frozen server, a
callback inside another library).  Collected last on purpose (the file name sorts after every other
test file), so that a run that stops at the first failure has already run everything else.

It calls the new entry point through the C ABI twice in a row -- the second call meets the scratch
contents the first one left -- and compares with the plan-based entry point running the same
configuration: bit for bit on integer-valued inputs, and within the library's contract tolerance
against the CPU oracle on random ones.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2512_02551_b200 import hgemm, inputs  # noqa: E402

CASES = [
    # M, N, K, block_n, split_k
    (64, 64, 8192, 64, 8),
    (300, 200, 1000, 96, 3),
    (512, 512, 12288, 128, 6),
    (256, 256, 256, 128, 1),        # no split: the scratch is not used at all
]


def _reference_through_plan(ctx, A, B, block_n, split_k):
    M, K = A.shape
    N = B.shape[0]
    plan = ctx.plan(M, N, K)
    stages = min(6, max(s for s in range(1, 13)
                        if hgemm.config_smem_bytes(hgemm.Config.make(block_n=block_n, stages=s)) <= 232448))
    plan.set_config(hgemm.Config.make(family=hgemm.FAMILY_UMMA_1CTA, block_n=block_n, stages=stages, split_k=split_k,
                                      raster_group=1, epilogue=hgemm.EPILOGUE_DIRECT, block_k=64,
                                      split_mode=hgemm.SPLIT_WORKSPACE))
    C = torch.empty(M, N, dtype=torch.float16, device="cuda")
    plan.run(A, B, C)
    torch.cuda.synchronize()
    plan.close()
    return C


@pytest.mark.parametrize("M,N,K,block_n,split_k", CASES)
def test_static_scratch_matches_plan_based_run(M, N, K, block_n, split_k):
    import oracle
    assert torch.cuda.is_available(), "this test needs a B200"
    stream = torch.cuda.current_stream().cuda_stream
    with hgemm.Context(0) as ctx:
        for dist in ("int5", "uniform"):
            A, B = inputs.make_ab(M, N, K, dist, "cuda")
            want = _reference_through_plan(ctx, A, B, block_n, split_k)
            for call in range(2):                      # two calls in a row share the static scratch
                C = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
                torch.cuda.synchronize()
                free_before, _ = torch.cuda.mem_get_info()
                st = hgemm.run_splitk_static(M, N, K, block_n, split_k, A.data_ptr(), B.data_ptr(), C.data_ptr(), stream)
                assert st == hgemm.OK, hgemm.status_string(st)
                torch.cuda.synchronize()
                if call == 1:                          # the first call on a device may load the module; later ones allocate nothing
                    assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the amount of free device memory"
                assert torch.equal(C.view(torch.int16), want.view(torch.int16)), (dist, call)
            # and the result itself is right, not merely equal to the other entry point's
            ref = oracle.hgemm_full(inputs.bits(A), inputs.bits(B))
            if dist == "int5":                         # exact sums: bit for bit the correctly rounded oracle value
                want_bits = oracle.f64_to_f16_bits(ref.ravel()).reshape(M, N)
                assert np.array_equal(oracle.canonical_bits(inputs.bits(C)), oracle.canonical_bits(want_bits))
            else:
                got = inputs.bits(C).view(np.float16).astype(np.float64)
                assert oracle.check_contract(got, ref, K)["ok"]
                assert oracle.check_scale_aware(got, ref, K)["ok"]


def test_static_scratch_rejects_what_does_not_fit():
    A = torch.zeros(16, dtype=torch.float16, device="cuda")
    a = A.data_ptr()
    # 8 x 8 tiles x 4 slices x 128 x 256 x 4 bytes = 32 MiB of partial sums: more than the 8 MiB built in
    assert hgemm.run_splitk_static(1024, 2048, 4096, 256, 4, a, a, a, 0) == hgemm.ERR_SCRATCH_LIMIT
    assert hgemm.run_splitk_static(64, 64, 8192, 48, 2, a, a, a, 0) == hgemm.ERR_UNSUPPORTED      # illegal tile width
    assert hgemm.run_splitk_static(64, 64, 128, 64, 3, a, a, a, 0) == hgemm.ERR_UNSUPPORTED       # more slices than k-blocks
    assert hgemm.run_splitk_static(64, 64, 8192, 64, 2, a + 2, a, a, 0) == hgemm.ERR_INVALID_ARG  # misaligned pointer
    assert hgemm.run_splitk_static(64, 64, 8192, 64, 2, 0, a, a, 0) == hgemm.ERR_INVALID_ARG
