"""GPU tests of the C-ABI's error behaviour, the bounded-wait status path, and the full 729-shape grid."""
import ctypes
import os
import time

import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2512_02551_b200 import hgemm, inputs  # noqa: E402

GRID = [64, 128, 256, 512, 1024, 2048, 4096, 8192, 12288]


@pytest.fixture(scope="module")
def ctx():
    assert torch.cuda.is_available(), "these tests need a B200"
    c = hgemm.Context(0)
    yield c
    c.close()


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


def test_library_is_loaded_from_the_tree():
    path = hgemm.LIB_PATH
    assert os.path.exists(path)
    with open("/proc/self/maps") as f:
        hgemm.lib()
        assert any(os.path.basename(path) in line for line in f.read().splitlines())


def test_argument_errors(ctx):
    L = hgemm.lib()
    plan = ctx.plan(256, 256, 256)
    A, B = inputs.make_ab(256, 256, 256, device="cuda")
    C = torch.empty(256, 256, dtype=torch.float16, device="cuda")
    a, b, c = A.data_ptr(), B.data_ptr(), C.data_ptr()
    assert L.hgemm_run(None, a, b, c, None) == hgemm.ERR_INVALID_ARG
    assert L.hgemm_run(plan._h, None, b, c, None) == hgemm.ERR_INVALID_ARG
    assert L.hgemm_run(plan._h, a + 2, b, c, None) == hgemm.ERR_INVALID_ARG       # not 16-byte aligned
    assert L.hgemm_run(plan._h, a, b, c + 8, None) == hgemm.ERR_INVALID_ARG
    out = ctypes.c_void_p()
    assert L.hgemm_plan(ctx._h, 64, 64, 1 << 23, ctypes.byref(out)) == hgemm.ERR_UNSUPPORTED and not out.value
    assert L.hgemm_plan(ctx._h, 0, 64, 64, ctypes.byref(out)) == hgemm.ERR_INVALID_ARG
    assert L.hgemm_plan(None, 64, 64, 64, ctypes.byref(out)) == hgemm.ERR_INVALID_ARG
    assert L.hgemm_create(ctypes.byref(out), 99) == hgemm.ERR_INVALID_ARG
    bad = hgemm.Config.make(block_n=48)
    before = plan.config.as_dict()
    assert plan.try_set_config(bad) == hgemm.ERR_UNSUPPORTED
    assert plan.config.as_dict() == before                                         # plan unchanged
    plan.run(A, B, C)                                                              # still usable
    assert ctx.last_device_status() == (hgemm.OK, 0)
    plan.close()


RAGGED = [(1, 1, 1), (64, 63, 8), (100, 135, 77), (257, 1000, 1003), (129, 9, 4099), (512, 520, 12), (33, 4100, 250)]


@pytest.mark.parametrize("M,N,K", RAGGED)
def test_ragged_k_and_n(ctx, gu, M, N, K):
    """K % 8 != 0 runs on zero-padded copies of A and B, N % 8 != 0 stores C element by element: same
    results as any other shape, for the library's own plan and for split-K in both modes."""
    import oracle
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    ref_i = oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi))
    cfgs = [None]
    kp = (K + 7) // 8 * 8
    if kp >= 128:
        cfgs += [hgemm.Config.make(block_n=64, stages=4, split_k=2, raster_group=1, split_mode=m) for m in (0, 1)]
        cfgs += [hgemm.Config.make(family=hgemm.FAMILY_UMMA_2CTA, block_n=96, stages=3, raster_group=2, epilogue=hgemm.EPILOGUE_TMA)]
    for cfg in cfgs:
        C, _, plan = gu.run_gemm(ctx, A, B, cfg)
        gu.assert_close_full(C, A, B, f"{(M, N, K)} {plan.config.as_dict()}")
        Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
        gu.assert_exact(Ci, ref_i, f"{(M, N, K)} integers")
        plan.close()


@pytest.mark.parametrize("M,N,K", [(16384, 256, 16384), (64, 16384, 4096), (16384, 16384, 1024), (512, 512, 16384)])
def test_paper_grid_value_16384(ctx, gu, M, N, K):
    """The paper's grid has a tenth value, 16384 (four of its shapes, one per regime; all 271 are run further down)."""
    gu.check_shape(ctx, M, N, K, "uniform")


def test_plan_tracks_new_pointers(ctx, gu):
    """Tensor maps are cached per (A, B, C); a call with other buffers must re-encode them."""
    M, N, K = 384, 256, 512
    plan = ctx.plan(M, N, K)
    for seed in (1, 2, 3):
        A, B = inputs.make_ab(M, N, K, "int5", "cuda", seed=seed)
        C, _, _ = gu.run_gemm(ctx, A, B, plan=plan)
        assert torch.equal(C.float(), A.float() @ B.float().T)
    plan.close()


def test_run_on_a_side_stream(ctx, gu):
    M, N, K = 512, 512, 1024
    A, B = inputs.make_ab(M, N, K, "int5", "cuda")
    C = torch.zeros(M, N, dtype=torch.float16, device="cuda")
    plan = ctx.plan(M, N, K)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        plan.run(A, B, C)              # picks up the current (side) stream
    s.synchronize()
    assert torch.equal(C.float(), A.float() @ B.float().T)
    plan.close()


def test_bounded_wait_reports_timeout_and_context_survives(ctx, gu):
    """A wait on a barrier that nothing signals runs out, the kernel returns, the host reads a
    status, and the context keeps working (no fault, no hang)."""
    ctx.set_wait_budget(2_000_000)                 # about a millisecond
    t0 = time.time()
    ctx.debug_timeout_probe()
    st, code = ctx.last_device_status()
    assert st == hgemm.ERR_TIMEOUT and (code >> 24) == 4
    assert time.time() - t0 < 5.0
    assert ctx.last_device_status() == (hgemm.OK, 0)          # the word is cleared by the read
    ctx.set_wait_budget(2_000_000_000)
    gu.check_shape(ctx, 256, 256, 256, "uniform")


def test_status_words_are_per_plan(ctx, gu):
    """Each plan has its own status word: an event recorded in the context's word (the probe kernel's) is not
    reported by a plan's query, and the context-wide query finds and clears it."""
    p1, p2 = ctx.plan(256, 256, 256), ctx.plan(512, 256, 1024)
    ctx.set_wait_budget(2_000_000)
    ctx.debug_timeout_probe()
    assert p1.last_device_status() == (hgemm.OK, 0)
    assert p2.last_device_status() == (hgemm.OK, 0)
    st, code = ctx.last_device_status()
    assert st == hgemm.ERR_TIMEOUT and (code >> 24) == 4
    assert ctx.last_device_status() == (hgemm.OK, 0)
    ctx.set_wait_budget(2_000_000_000)
    L = hgemm.lib()
    code = ctypes.c_uint32(7)
    assert L.hgemm_last_device_status(None, ctypes.byref(code)) == hgemm.ERR_INVALID_ARG and code.value == 7
    assert L.hgemm_last_device_status(p1._h, None) == hgemm.ERR_INVALID_ARG
    p1.close()
    p2.close()


def test_failed_allocation_leaves_the_plan_as_it_was(ctx, gu):
    """hgemm_plan_set_config that cannot get its larger workspace (the failure is injected: an error code from
    a stand-in for cudaMalloc) returns HGEMM_ERR_ALLOC and the plan keeps its configuration, its buffers and its
    results."""
    import oracle
    M, N, K = 512, 512, 4096
    A, B = inputs.make_ab(M, N, K, "int5", "cuda")
    want = oracle.hgemm_full(inputs.bits(A), inputs.bits(B))
    small = hgemm.Config.make(block_n=128, stages=4, split_k=2, raster_group=1, split_mode=hgemm.SPLIT_WORKSPACE)
    # more tiles and more slices: both the workspace and the arrival counters have to grow
    large = hgemm.Config.make(block_n=64, stages=4, split_k=8, raster_group=1, split_mode=hgemm.SPLIT_WORKSPACE)
    C, _, plan = gu.run_gemm(ctx, A, B, small)
    gu.assert_exact(C, want, "before the failed call")
    before = plan.config.as_dict()
    for after in (0, 1):                                # the workspace allocation fails; then the counters' one
        ctx.debug_fail_allocs(after, 1)
        assert plan.try_set_config(large) == hgemm.ERR_ALLOC
        ctx.debug_fail_allocs(0, 0)
        assert plan.config.as_dict() == before
        C2, _, _ = gu.run_gemm(ctx, A, B, plan=plan)
        gu.assert_exact(C2, want, "after the failed call")
    plan.set_config(large)                              # and without the injected failure the larger one goes in
    C3, _, _ = gu.run_gemm(ctx, A, B, plan=plan)
    gu.assert_exact(C3, want, "larger configuration")
    # a plan that cannot get its buffers at creation is not created
    ctx.debug_fail_allocs(0, 1)
    out = ctypes.c_void_p()
    assert hgemm.lib().hgemm_plan(ctx._h, 200, 136, 77, ctypes.byref(out)) == hgemm.ERR_ALLOC and not out.value   # K % 8 != 0: padded copies
    ctx.debug_fail_allocs(0, 0)
    plan.close()


def test_full_grid_default_plans(ctx, gu):
    """All 729 grid shapes with the plan the library picks: full-output oracle check up to 2048^3
    by volume, 4096 samples + one row + one column above."""
    worst = 0.0
    for M in GRID:
        for N in GRID:
            for K in GRID:
                rep = gu.check_shape(ctx, M, N, K, "uniform")
                worst = max(worst, rep["max_err_over_bound"])
    assert worst < 1.0


def test_paper_grid_with_16384_default_plans(ctx, gu):
    """The 271 shapes that the paper's tenth grid value adds (every (M, N, K) over {64 .. 12288, 16384} with at least one
    16384), each with the plan the library picks: full-output oracle check up to 2048^3 by volume, 4096 samples + one row
    + one column above."""
    g10 = GRID + [16384]
    worst, count = 0.0, 0
    for M in g10:
        for N in g10:
            for K in g10:
                if 16384 not in (M, N, K):
                    continue
                rep = gu.check_shape(ctx, M, N, K, "uniform")
                worst = max(worst, rep["max_err_over_bound"])
                count += 1
    assert count == 271 and worst < 1.0


# ---- the checked build: the same tests under a library that verifies its own invariants on the device ---------------

def _run_under_checked_build(args, timeout):
    import subprocess
    import sys
    from paper_2512_02551_b200 import build as hbuild
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, HGEMM_LIB=hbuild.build(checked=True), PYTHONPATH=root)
    return subprocess.run([sys.executable] + args, env=env, cwd=root, capture_output=True, text=True, timeout=timeout)


def test_checked_build_reports_a_violated_invariant(ctx):
    """The reporting path, exercised by a probe whose invariant is false by construction (no bad access anywhere): the
    checked build records (role 7, site 99) and the status calls return HGEMM_ERR_CHECK; the ordinary build records nothing."""
    ctx.debug_check_probe()
    assert ctx.last_device_status() == (hgemm.OK, 0) and not hgemm.build_is_checked()
    code = ("from paper_2512_02551_b200 import hgemm\n"
            "assert hgemm.build_is_checked()\n"
            "with hgemm.Context(0) as ctx:\n"
            "    ctx.debug_check_probe()\n"
            "    st, code = ctx.last_device_status()\n"
            "    again = ctx.last_device_status()\n"
            "    print(st, code, again[0], again[1])\n")
    r = _run_under_checked_build(["-c", code], 300)
    assert r.returncode == 0, r.stderr[-2000:]
    st, code, st2, code2 = (int(v) for v in r.stdout.split())
    assert st == hgemm.ERR_CHECK and code == (7 << 24) | (99 << 8)
    assert (st2, code2) == (hgemm.OK, 0)                     # reading the status clears it


def test_checked_build_finds_nothing_in_the_parity_cases():
    """Every kernel family, reduction and tail mode of the parity suite under the checked build: same results, and no
    invariant violated (each of those tests asserts a clean status word after every call)."""
    r = _run_under_checked_build(["-m", "pytest", "tests/test_gpu_parity.py", "-x", "-q", "-m", "gpu", "-k",
                                  "unit_shapes or stream_k or tail_split or swapped_operands or small_family or light_family or "
                                  "double_accumulator or split_k_is_deterministic or nn_layout or scaled_form or serpentine"], 1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-1000:]
    assert " passed" in r.stdout and "failed" not in r.stdout


# ---- hgemm_run_host: host buffers, copies on the context's own streams ------------------------------------------------

def test_run_host_sequences(ctx, gu):
    """hgemm_run_host over sequences of calls: several plans in a row on one stream, the same plan twice without a
    synchronisation in between (its staging is reused: the calls must stay ordered), a side stream, new host data after
    a synchronisation, pageable memory -- every result equal to the device-resident run, bit for bit."""
    import oracle
    shapes = [(512, 384, 256), (1024, 1024, 512), (96, 200, 72), (2048, 512, 1024)]
    plans, host, want = [], [], []
    for i, (M, N, K) in enumerate(shapes):
        A, B = inputs.make_ab(M, N, K, "int5" if i % 2 == 0 else "uniform", "cuda")
        plan = ctx.plan(M, N, K)
        C = torch.empty(M, N, dtype=torch.float16, device="cuda")
        plan.run(A, B, C)
        torch.cuda.synchronize()
        plans.append(plan)
        want.append(C.cpu())
        host.append((A.cpu().pin_memory(), B.cpu().pin_memory(), torch.zeros(M, N, dtype=torch.float16).pin_memory()))
    s = torch.cuda.current_stream().cuda_stream
    for rep in range(3):                                           # the second and third pass reuse every plan's staging
        for hA, hB, hC in host:
            hC.zero_()
        for plan, (hA, hB, hC) in zip(plans, host):
            plan.run_host(hA, hB, hC, s)
        torch.cuda.synchronize()
        for (hA, hB, hC), w in zip(host, want):
            assert torch.equal(hC, w), f"pass {rep}"
    gu.assert_exact(host[0][2].cuda(), oracle.hgemm_full(inputs.bits(host[0][0].cuda()), inputs.bits(host[0][1].cuda())), "run_host, integers")
    # the same plan twice in a row with different host buffers, no synchronisation in between
    M, N, K = shapes[1]
    A2, B2 = inputs.make_ab(M, N, K, "int5", "cuda")
    C2 = torch.empty(M, N, dtype=torch.float16, device="cuda")
    plans[1].run(A2, B2, C2)
    torch.cuda.synchronize()
    hA2, hB2, hC2 = A2.cpu().pin_memory(), B2.cpu().pin_memory(), torch.zeros(M, N, dtype=torch.float16).pin_memory()
    host[1][2].zero_()
    plans[1].run_host(host[1][0], host[1][1], host[1][2], s)
    plans[1].run_host(hA2, hB2, hC2, s)
    plans[1].run_host(host[1][0], host[1][1], host[1][2], s)
    torch.cuda.synchronize()
    assert torch.equal(hC2, C2.cpu()) and torch.equal(host[1][2], want[1])
    # a side stream; work enqueued on it after the call sees the finished result copy
    side = torch.cuda.Stream()
    host[3][2].zero_()
    with torch.cuda.stream(side):
        plans[3].run_host(host[3][0], host[3][1], host[3][2], side.cuda_stream)
    side.synchronize()
    assert torch.equal(host[3][2], want[3])
    # new host data after a synchronisation; pageable memory (blocking copies)
    hA, hB, hC = host[2]
    A3, B3 = inputs.make_ab(*shapes[2], "int5", "cuda")
    hA.copy_(A3.cpu())
    hB.copy_(B3.cpu())
    plans[2].run_host(hA, hB, hC, s)
    torch.cuda.synchronize()
    assert torch.equal(hC.float(), (A3.float() @ B3.float().T).cpu())
    pA, pB, pC = A3.cpu(), B3.cpu(), torch.zeros(shapes[2][0], shapes[2][1], dtype=torch.float16)
    plans[2].run_host(pA, pB, pC, s)
    torch.cuda.synchronize()
    assert torch.equal(pC, hC)
    assert ctx.last_device_status() == (hgemm.OK, 0)
    for plan in plans:
        plan.close()
