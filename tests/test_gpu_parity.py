"""GPU parity tests: the CUDA library, called through its C ABI, against the fp64 CPU oracle.

Bar: bit-exact on inputs whose sums are exactly representable (paper section 2.3, "Exact
Match", generalised to signed small integers because this library accumulates in fp32);
|C - C_ref| <= 2^-10 |C_ref| + 1e-3 sqrt(K) elementwise on random inputs, plus the
scale-aware checks of oracle/acceptance.py.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2512_02551_b200 import hgemm, inputs  # noqa: E402

F1, F2 = hgemm.FAMILY_UMMA_1CTA, hgemm.FAMILY_UMMA_2CTA
DIRECT, TMA = hgemm.EPILOGUE_DIRECT, hgemm.EPILOGUE_TMA
WIDE = hgemm.EPILOGUE_TMA_WIDE


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


WORKSPACE, CLUSTER = hgemm.SPLIT_WORKSPACE, hgemm.SPLIT_CLUSTER


def _cfg(family=F1, bn=128, stages=4, split=1, raster=8, epi=DIRECT, bk=64, mode=WORKSPACE):
    return hgemm.Config.make(family=family, block_n=bn, stages=stages, split_k=split, raster_group=raster, epilogue=epi,
                             block_k=bk, split_mode=mode)


VARIANTS = [(F1, DIRECT), (F1, TMA), (F2, DIRECT), (F2, TMA)]


# ---- configuration 1: single 128^3 GEMM, random and integer-valued -------------------------------

@pytest.mark.parametrize("family,epi", VARIANTS)
def test_config1_128_cubed(ctx, gu, family, epi):
    import oracle
    M = N = K = 128
    cfg = _cfg(family, 128, 4, 1, 1, epi)
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C, _, plan = gu.run_gemm(ctx, A, B, cfg)
    rep = gu.assert_close_full(C, A, B, "128^3 uniform")
    assert rep["rel_frobenius"] < 3e-4
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
    gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), "128^3 integers")
    plan.close()


def test_default_plan_128_cubed(ctx, gu):
    gu.check_shape(ctx, 128, 128, 128, "uniform")


# ---- closed forms, bit for bit, every family and split factor ---------------------------------------

@pytest.mark.parametrize("family,epi", VARIANTS)
@pytest.mark.parametrize("split", [1, 3])
def test_exact_closed_forms(ctx, gu, family, epi, split):
    import oracle
    M, N, K = 200, 136, 320          # ragged in M and N, 5 k-blocks
    cfg = _cfg(family, 64, 3, split, 2, epi)
    rng = np.random.default_rng(7)
    # permutation: C[i][j] = B[j][pi(i)]
    pi = rng.permutation(K)[:M]
    A = torch.zeros(M, K, dtype=torch.float16)
    A[torch.arange(M), torch.from_numpy(pi)] = 1.0
    B = inputs.draw(3, inputs.TAG_B, N, K, "uniform")
    C, _, plan = gu.run_gemm(ctx, A.cuda(), B.cuda(), cfg)
    gu.assert_exact(C, B.double().numpy()[:, pi].T, "permutation")
    # rank-1, one-hot k: C[i][j] = fp16(u_i v_j)
    u = inputs.draw(5, 1, M, 1, "uniform")[:, 0]
    v = inputs.draw(5, 2, N, 1, "uniform")[:, 0]
    A = torch.zeros(M, K, dtype=torch.float16)
    B = torch.zeros(N, K, dtype=torch.float16)
    A[:, 77] = u
    B[:, 77] = v
    C, _, _ = gu.run_gemm(ctx, A.cuda(), B.cuda(), plan=plan)
    gu.assert_exact(C, np.outer(u.double().numpy(), v.double().numpy()), "rank-1 one-hot")
    # rank-1 constant along k with power-of-two entries: C[i][j] = K u_i v_j, all partial sums exact
    vals = np.array([0.5, 1.0, 2.0, -0.5, -1.0, -2.0])
    uu, vv = rng.choice(vals, M), rng.choice(vals, N)
    A = torch.from_numpy(np.repeat(uu[:, None], K, 1)).to(torch.float16)
    B = torch.from_numpy(np.repeat(vv[:, None], K, 1)).to(torch.float16)
    C, _, _ = gu.run_gemm(ctx, A.cuda(), B.cuda(), plan=plan)
    gu.assert_exact(C, K * np.outer(uu, vv), "rank-1 constant")
    # integers in {-2..2}
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    C, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
    gu.assert_exact(C, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), "integers")
    plan.close()


def test_identity_returns_b_transposed(ctx, gu):
    M = K = 256
    N = 96
    B = inputs.draw(9, inputs.TAG_B, N, K, "uniform", "cuda")
    A = torch.eye(M, K, dtype=torch.float16, device="cuda")
    C, _, plan = gu.run_gemm(ctx, A, B)
    assert torch.equal(C, B.T.contiguous())
    plan.close()


def test_paper_style_binary_exact_match(ctx, gu):
    """Section 2.3: {0,1} inputs, exact equality required wherever the reference is below 2048."""
    import oracle
    M, N, K = 256, 192, 8192
    for seed in (1, 2, 3):
        A, B = inputs.make_ab(M, N, K, "binary", "cuda", seed=seed, p=inputs.binary_p(K))
        C, _, plan = gu.run_gemm(ctx, A, B)
        ref = oracle.hgemm_full(inputs.bits(A), inputs.bits(B))
        got = gu.bits_to_f64(gu.c_bits(C))
        small = ref < 2048
        assert small.mean() > 0.9 and np.array_equal(got[small], ref[small])
        plan.close()


# ---- unit shapes: one tile, ring wrap-around, tails, many tiles per CTA, tile widths -------------------

UNIT_CASES = [
    # M, N, K, bn, stages, split, raster
    (128, 128, 64, 128, 4, 1, 1),       # one tile, one k-block
    (128, 128, 1024, 128, 3, 1, 1),     # ring wraps five times
    (128, 32, 64, 32, 1, 1, 1),         # narrowest tile, single stage
    (8, 8, 8, 32, 2, 1, 1),             # smallest legal shape: tails in all three dimensions
    (100, 136, 72, 64, 4, 1, 1),        # ragged M, N and K
    (130, 264, 200, 256, 4, 1, 1),      # one row / one column group past a tile edge
    (384, 416, 192, 96, 4, 1, 2),       # tile width that is not a power of two
    (640, 480, 256, 160, 2, 1, 3),
    (1024, 2048, 128, 32, 9, 1, 4),     # 512 tiles on 148 SMs: several tiles per CTA, accumulators alternate
    (2048, 2048, 64, 64, 2, 1, 16),
    (64, 64, 2048, 64, 4, 4, 1),        # split-K
    (300, 200, 1000, 96, 4, 16, 1),     # one k-block per slice
    (512, 384, 640, 128, 4, 3, 2),      # uneven slices (10 k-blocks over 3)
]

# M, N, K, bn, stages, split, raster, block_k, split mode: 128-wide K stages and cluster split-K
UNIT_CASES_WIDE = [
    (128, 128, 64, 128, 2, 1, 1, 128, WORKSPACE),     # K shorter than one stage: second sub-tile all zero-fill
    (256, 256, 1024, 256, 2, 1, 1, 128, WORKSPACE),   # ring wraps
    (100, 136, 200, 64, 4, 1, 1, 128, WORKSPACE),     # ragged everywhere, K = 1.56 stages
    (640, 480, 1152, 160, 2, 1, 3, 128, WORKSPACE),
    (300, 200, 1000, 96, 3, 4, 1, 128, WORKSPACE),    # split-K over 128-wide stages (8 stages over 4 slices)
    (64, 64, 4096, 64, 4, 8, 1, 64, CLUSTER),         # one tile, eight slices in one cluster
    (100, 136, 520, 32, 4, 9, 1, 64, CLUSTER),        # more slices than a portable cluster (non-portable size 9)
    (512, 384, 640, 128, 4, 3, 2, 64, CLUSTER),       # uneven slices
    (300, 200, 1000, 96, 3, 4, 1, 128, CLUSTER),
    (256, 512, 12288, 256, 4, 4, 1, 64, CLUSTER),     # widest tile: its 128 KB partial plus three received shares fill shared memory
    (256, 512, 12288, 192, 4, 16, 1, 64, CLUSTER),    # largest cluster
    (64, 640, 2048, 160, 2, 7, 1, 128, CLUSTER),      # shares of 732 float4 units: they cut the staged tile inside its rows
]


@pytest.mark.parametrize("family", [F1, F2])
@pytest.mark.parametrize("case", UNIT_CASES, ids=lambda c: "x".join(map(str, c[:3])) + f"-bn{c[3]}s{c[4]}k{c[5]}")
def test_unit_shapes(ctx, gu, family, case):
    import oracle
    M, N, K, bn, stages, split, raster = case
    for epi in (DIRECT, TMA):
        cfg = _cfg(family, bn, stages, split, raster, epi)
        A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
        C, _, plan = gu.run_gemm(ctx, A, B, cfg)
        gu.assert_close_full(C, A, B, f"{case} family={family} epi={epi}")
        Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
        Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
        gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"{case} integers")
        plan.close()
        if split > 1:
            break                         # split-K always finishes with direct stores


@pytest.mark.parametrize("case", UNIT_CASES_WIDE, ids=lambda c: "x".join(map(str, c[:3])) + f"-bn{c[3]}s{c[4]}k{c[5]}bk{c[7]}m{c[8]}")
def test_unit_shapes_wide_stages_and_cluster_split(ctx, gu, case):
    import oracle
    M, N, K, bn, stages, split, raster, bk, mode = case
    for family in (F1, F2):
        cfg = _cfg(family, bn, stages, split, raster, TMA if split == 1 else DIRECT, bk, mode)
        if hgemm.validate_config(M, N, K, cfg) == hgemm.ERR_UNSUPPORTED and family == F2 and mode == CLUSTER:
            continue                      # more than 8 pairs per cluster, or a stage count only the 1-CTA family fits
        A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
        C, _, plan = gu.run_gemm(ctx, A, B, cfg)
        gu.assert_close_full(C, A, B, f"{case} family={family}")
        Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
        Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
        gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"{case} integers")
        plan.close()


# ---- swapped operands: the rows of B on the MMA's 128-row side, the tile stored transposed ----------------------

SWAP_CASES = [
    # M, N, K, family, bn (covers rows of A), stages, split, block_k, split mode, epilogue
    (64, 128, 64, F1, 64, 2, 1, 64, WORKSPACE, TMA),          # one tile
    (64, 256, 256, F2, 64, 4, 1, 64, WORKSPACE, TMA),         # one pair tile: each CTA stages 32 rows of A
    (64, 4096, 1024, F2, 64, 4, 1, 128, WORKSPACE, TMA),      # the skinny projection case, 16 pair tiles
    (128, 2048, 512, F2, 128, 4, 1, 64, WORKSPACE, DIRECT),   # 2-byte transposed stores
    (256, 1536, 384, F2, 256, 3, 1, 128, WORKSPACE, TMA),
    (200, 1000, 328, F1, 224, 3, 1, 64, WORKSPACE, TMA),      # ragged M, N (a multiple of 8) and K
    (37, 520, 200, F2, 64, 4, 1, 64, WORKSPACE, TMA),         # fewer rows than one box; the last pair tile is mostly empty
    (37, 520, 200, F1, 32, 4, 1, 64, WORKSPACE, DIRECT),      # two column tiles of the kernel's problem
    (96, 2048, 4096, F1, 96, 4, 4, 64, CLUSTER, DIRECT),      # K slices summed inside a cluster, stored transposed
    (64, 1024, 8192, F2, 64, 4, 4, 64, CLUSTER, DIRECT),      # clusters of four pairs
    (128, 512, 2048, F1, 128, 4, 3, 64, WORKSPACE, DIRECT),   # K slices through the workspace
    (256, 768, 1152, F2, 128, 4, 2, 128, WORKSPACE, DIRECT),  # two column tiles per pair row, uneven slices
    (1000, 136, 320, F1, 128, 4, 1, 64, WORKSPACE, TMA),      # many rows of A after all: eight column tiles, raster groups
]


@pytest.mark.parametrize("case", SWAP_CASES, ids=lambda c: "x".join(map(str, c[:3])) + f"-f{c[3]}bn{c[4]}k{c[6]}m{c[8]}e{c[9]}")
def test_swapped_operands(ctx, gu, case):
    """swap_ab = 1 computes the same C: exact on integer inputs, the contract on random ones, nothing written
    outside C (guard bands), every element written (sentinel)."""
    import oracle
    M, N, K, family, bn, stages, split, bk, mode, epi = case
    cfg = hgemm.Config.make(family=family, block_n=bn, stages=stages, split_k=split, raster_group=3, epilogue=epi, block_k=bk,
                            split_mode=mode, swap_ab=1, raster_mode=hgemm.RASTER_SERPENTINE if M > 256 else hgemm.RASTER_SWEEP)
    assert hgemm.validate_config(M, N, K, cfg) == hgemm.OK
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C, _, plan = gu.run_gemm(ctx, A, B, cfg)
    assert plan.config.swap_ab == 1
    gu.assert_close_full(C, A, B, f"swapped {case}")
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
    gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"swapped {case} integers")
    # the general form through the same configuration (exact: 0/1 operands, small integers in C)
    Ab, Bb = inputs.make_ab(M, N, K, "binary", "cuda")
    C0 = inputs.draw(33, inputs.TAG_A, M, N, "int5", "cuda")
    buf, Cs = gu.alloc_c_with_guards(M, N)
    Cs.copy_(C0)
    plan.run_scaled(2.0, -3.0, Ab, Bb, Cs)
    assert ctx.last_device_status() == (hgemm.OK, 0)
    assert gu.guards_intact(buf, M, N)
    gu.assert_exact(Cs, oracle.hgemm_scaled_full(inputs.bits(Ab), inputs.bits(Bb), inputs.bits(C0), 2.0, -3.0), f"swapped {case} scaled")
    plan.close()


def test_swapped_operands_rules(ctx):
    ok = hgemm.Config.make(family=F2, block_n=64, stages=4, epilogue=TMA, swap_ab=1)
    assert hgemm.validate_config(64, 4096, 4096, ok) == hgemm.OK
    assert hgemm.validate_config(64, 4100, 4096, ok) == hgemm.ERR_UNSUPPORTED            # rows of C must be multiples of 16 bytes
    for kw in (dict(epilogue=WIDE), dict(accumulate=hgemm.ACC_F16), dict(tail_split=2), dict(swap_ab=2)):
        c = hgemm.Config.make(**{**dict(family=F2, block_n=64, stages=4, epilogue=TMA, swap_ab=1), **kw})
        assert hgemm.validate_config(64, 4096, 4096, c) == hgemm.ERR_UNSUPPORTED, kw
    # K that needs padded copies works too: the copies trade places with the operands
    plan = ctx.plan(48, 264, 100)
    plan.set_config(hgemm.Config.make(family=F1, block_n=64, stages=3, epilogue=TMA, swap_ab=1))
    A, B = inputs.make_ab(48, 264, 100, "int5", "cuda")
    C = torch.zeros(48, 264, dtype=torch.float16, device="cuda")
    plan.run(A, B, C)
    torch.cuda.synchronize()
    assert torch.equal(C.float(), A.float() @ B.float().T)
    # the NN layout has no swapped form
    nn = ctx.plan(64, 512, 256, layout=hgemm.LAYOUT_NN)
    assert nn.try_set_config(hgemm.Config.make(family=F1, block_n=64, stages=3, epilogue=TMA, swap_ab=1)) == hgemm.ERR_UNSUPPORTED
    nn.close()
    plan.close()


@pytest.mark.parametrize("family", [F1, F2])
@pytest.mark.parametrize("shape,bn,raster", [((1024, 2048, 128), 32, 3), ((2048, 1536, 256), 128, 4), ((1300, 1000, 192), 96, 2),
                                              ((4096, 4096, 512), 256, 5)])
def test_serpentine_raster(ctx, gu, family, shape, bn, raster):
    """The serpentine tile order visits every tile exactly once: same results as the plain sweep, bit for bit, with
    full and ragged last raster groups and more tiles than SMs."""
    import oracle
    M, N, K = shape
    A, B = inputs.make_ab(M, N, K, "int5", "cuda")
    want = oracle.hgemm_full(inputs.bits(A), inputs.bits(B))
    for epi in (TMA, DIRECT):
        cfg = hgemm.Config.make(family=family, block_n=bn, stages=3, raster_group=raster, epilogue=epi, raster_mode=hgemm.RASTER_SERPENTINE)
        C, _, plan = gu.run_gemm(ctx, A, B, cfg)
        gu.assert_exact(C, want, f"serpentine {shape} family={family} epi={epi}")
        plan.close()
    assert hgemm.validate_config(M, N, K, hgemm.Config.make(block_n=bn, stages=3, raster_mode=2)) == hgemm.ERR_UNSUPPORTED


# ---- the 256 x 512 pair tile that fills both accumulators ---------------------------------------------------------

DUAL_CASES = [
    # M, N, K, block_k, stages, epilogue, raster
    (256, 512, 64, 64, 2, TMA, 1),          # one tile, one k-block
    (256, 512, 1024, 64, 4, TMA, 1),        # ring wraps
    (300, 1024, 200, 64, 3, DIRECT, 1),     # ragged M and K: dead rows, zero-filled k tail
    (512, 1536, 384, 128, 2, TMA, 2),       # 128-wide stages (two of them fill shared memory)
    (4096, 8192, 128, 64, 4, TMA, 4),       # 256 tiles on 74 pairs: up to four tiles per pair, the accumulators' phase alternates
    (2048, 4096, 256, 64, 3, WIDE, 3),      # 64-column store boxes
    (100, 512, 72, 64, 4, TMA, 1),          # fewer rows than one CTA's 128
]


@pytest.mark.parametrize("case", DUAL_CASES, ids=lambda c: "x".join(map(str, c[:3])) + f"-bk{c[3]}s{c[4]}e{c[5]}")
def test_double_accumulator_tile(ctx, gu, case):
    """block_n = 512: each accumulator column must land in the column of C that the two-MMA layout assigns it --
    a wrong permutation fails the integer case on nearly every element."""
    import oracle
    M, N, K, bk, stages, epi, raster = case
    cfg = hgemm.Config.make(family=F2, block_n=512, stages=stages, raster_group=raster, epilogue=epi, block_k=bk,
                            raster_mode=hgemm.RASTER_SERPENTINE if raster > 1 else hgemm.RASTER_SWEEP)
    assert hgemm.validate_config(M, N, K, cfg) == hgemm.OK
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    Ci, _, plan = gu.run_gemm(ctx, Ai, Bi, cfg)
    assert plan.config.block_n == 512
    if M * N * K <= gu.FULL_CHECK_VOLUME // 4:
        gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"double tile {case} integers")
        A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
        C, _, _ = gu.run_gemm(ctx, A, B, plan=plan)
        gu.assert_close_full(C, A, B, f"double tile {case}")
    else:
        # sampled: 4096 seeded entries, one full row, one full column -- exact values on integer inputs
        ii, jj, row, col = inputs.sample_indices(11, M, N, 4096)
        ii = np.concatenate([ii, np.full(N, row, dtype=np.int64), np.arange(M, dtype=np.int64)])
        jj = np.concatenate([jj, np.arange(N, dtype=np.int64), np.full(M, col, dtype=np.int64)])
        ref = oracle.hgemm_sampled(inputs.bits(Ai), inputs.bits(Bi), ii, jj)
        got = gu.bits_to_f64(inputs.bits(Ci[torch.from_numpy(ii).cuda(), torch.from_numpy(jj).cuda()]))
        assert np.array_equal(got, ref), f"double tile {case}: sampled integer entries differ"
        # and every entry against the library's own 256-wide pair tile (bit for bit: the same fp32 sums in the same order)
        C2, _, _ = gu.run_gemm(ctx, Ai, Bi, hgemm.Config.make(family=F2, block_n=256, stages=3, raster_group=4, epilogue=TMA), plan=plan)
        assert torch.equal(Ci.view(torch.int16), C2.view(torch.int16))
    plan.close()


def test_double_accumulator_tile_other_forms(ctx, gu):
    import oracle
    M, N, K = 384, 1024, 320
    cfg = hgemm.Config.make(family=F2, block_n=512, stages=4, raster_group=1, epilogue=TMA, block_k=64)
    plan = ctx.plan(M, N, K)
    plan.set_config(cfg)
    # alpha / beta (exact: 0/1 operands, small integers in C)
    Ab, Bb = inputs.make_ab(M, N, K, "binary", "cuda")
    C0 = inputs.draw(35, inputs.TAG_A, M, N, "int5", "cuda")
    buf, Cs = gu.alloc_c_with_guards(M, N)
    Cs.copy_(C0)
    plan.run_scaled(-1.0, 2.0, Ab, Bb, Cs)
    assert ctx.last_device_status() == (hgemm.OK, 0) and gu.guards_intact(buf, M, N)
    gu.assert_exact(Cs, oracle.hgemm_scaled_full(inputs.bits(Ab), inputs.bits(Bb), inputs.bits(C0), -1.0, 2.0), "double tile scaled")
    # fp16 accumulators
    cfg.accumulate = hgemm.ACC_F16
    plan.set_config(cfg)
    C, _, _ = gu.run_gemm(ctx, Ab, Bb, plan=plan)
    gu.assert_exact(C, oracle.hgemm_full(inputs.bits(Ab), inputs.bits(Bb)), "double tile, fp16 accumulators, 0/1 operands")
    plan.close()
    # rules
    ok = hgemm.Config.make(family=F2, block_n=512, stages=4, epilogue=TMA)
    assert hgemm.validate_config(512, 1024, 512, ok) == hgemm.OK
    assert hgemm.validate_config(512, 1000, 512, ok) == hgemm.ERR_UNSUPPORTED                       # N must be a multiple of 512
    for kw in (dict(family=F1), dict(split_k=2), dict(tail_split=2), dict(swap_ab=1), dict(stages=5)):
        c = hgemm.Config.make(**{**dict(family=F2, block_n=512, stages=4, epilogue=TMA), **kw})
        assert hgemm.validate_config(512, 1024, 4096, c) == hgemm.ERR_UNSUPPORTED, kw
    nn = ctx.plan(512, 1024, 512, layout=hgemm.LAYOUT_NN)
    assert nn.try_set_config(ok) == hgemm.ERR_UNSUPPORTED
    nn.close()


# ---- the light family: one tile per CTA, for the latency-bound shapes ----------------------------------------------

LIGHT = hgemm.FAMILY_LIGHT
LIGHT_CASES = [
    # M, N, K, bn, block_k, stages
    (128, 128, 64, 128, 64, 1),         # one tile, one k-block, one stage
    (128, 128, 1024, 128, 64, 3),       # the ring wraps five times
    (64, 64, 64, 32, 64, 1),            # half-empty tile rows, two column tiles
    (8, 8, 8, 32, 64, 1),               # smallest legal shape: tails in all three dimensions
    (100, 136, 72, 64, 64, 2),          # ragged M, N and K (multiples of 8)
    (512, 512, 512, 32, 64, 8),         # every k-block has its own stage: no stage is ever freed
    (512, 512, 512, 64, 128, 4),        # 128-wide stages
    (256, 256, 4096, 256, 128, 2),      # widest tile, long K through two stages
    (1024, 2048, 128, 32, 64, 2),       # 512 CTAs on 148 SMs: several waves
    (384, 416, 192, 96, 64, 3),         # tile width that is not a power of two
    (130, 264, 200, 256, 64, 4),        # one row group / a few columns past a tile edge
]


@pytest.mark.parametrize("case", LIGHT_CASES, ids=lambda c: "x".join(map(str, c[:3])) + f"-bn{c[3]}bk{c[4]}s{c[5]}")
def test_light_family(ctx, gu, case):
    import oracle
    M, N, K, bn, bk, stages = case
    plan = None
    for epi in (DIRECT, TMA):
        cfg = hgemm.Config.make(family=LIGHT, block_n=bn, stages=stages, raster_group=1, epilogue=epi, block_k=bk)
        if epi == TMA and hgemm.validate_config(M, N, K, cfg) != hgemm.OK:
            cfg.stages = stages - 1                      # the store staging takes the room of a stage
        assert hgemm.validate_config(M, N, K, cfg) == hgemm.OK
        A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
        C, _, plan = gu.run_gemm(ctx, A, B, cfg, plan=plan)
        assert plan.config.family == LIGHT
        gu.assert_close_full(C, A, B, f"light {case} epilogue {epi}")
        Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
        Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
        gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"light {case} epilogue {epi} integers")
    # the general form (exact: 0/1 operands, small integers in C)
    Ab, Bb = inputs.make_ab(M, N, K, "binary", "cuda")
    C0 = inputs.draw(37, inputs.TAG_A, M, N, "int5", "cuda")
    buf, Cs = gu.alloc_c_with_guards(M, N)
    Cs.copy_(C0)
    plan.run_scaled(2.0, -1.0, Ab, Bb, Cs)
    assert ctx.last_device_status() == (hgemm.OK, 0) and gu.guards_intact(buf, M, N)
    gu.assert_exact(Cs, oracle.hgemm_scaled_full(inputs.bits(Ab), inputs.bits(Bb), inputs.bits(C0), 2.0, -1.0), f"light {case} scaled")
    plan.close()


def test_light_family_rules_and_stream_order(ctx, gu):
    import oracle
    ok = hgemm.Config.make(family=LIGHT, block_n=64, stages=4, epilogue=TMA)
    assert hgemm.validate_config(512, 512, 512, ok) == hgemm.OK
    assert hgemm.validate_config(512, 516, 512, ok) == hgemm.ERR_UNSUPPORTED            # rows of C: multiples of 16 bytes
    assert hgemm.validate_config(512, 512, 516, ok) == hgemm.ERR_UNSUPPORTED            # rows of A and B too (no padded copies here)
    for kw in (dict(split_k=2), dict(epilogue=WIDE), dict(accumulate=hgemm.ACC_F16), dict(tail_split=2),
               dict(swap_ab=1), dict(block_n=512), dict(raster_mode=1)):
        c = hgemm.Config.make(**{**dict(family=LIGHT, block_n=64, stages=4, epilogue=TMA), **kw})
        assert hgemm.validate_config(512, 512, 4096, c) == hgemm.ERR_UNSUPPORTED, kw
    nn = ctx.plan(256, 512, 256, layout=hgemm.LAYOUT_NN)
    assert nn.try_set_config(ok) == hgemm.ERR_UNSUPPORTED
    nn.close()
    # a chain of dependent launches through light plans: C1 = A B1^T, C2 = C1 B2^T, stream order kept
    M, K1, N1, N2 = 512, 64, 64, 384
    A = inputs.draw(1, inputs.TAG_A, M, K1, "int5", "cuda")
    B1 = inputs.draw(2, inputs.TAG_B, N1, K1, "int5", "cuda")
    B2 = inputs.draw(3, inputs.TAG_B, N2, N1, "int5", "cuda")
    c1_ref = oracle.hgemm_full(inputs.bits(A), inputs.bits(B1))
    c2_ref = oracle.hgemm_full(oracle.f64_to_f16_bits(c1_ref.ravel()).reshape(M, N1), inputs.bits(B2))
    p1, p2 = ctx.plan(M, N1, K1), ctx.plan(M, N2, N1)
    p1.set_config(hgemm.Config.make(family=LIGHT, block_n=64, stages=1, epilogue=TMA))
    p2.set_config(hgemm.Config.make(family=LIGHT, block_n=96, stages=1, epilogue=TMA))
    for rep in range(25):
        C1 = torch.zeros(M, N1, dtype=torch.float16, device="cuda")
        C2 = torch.zeros(M, N2, dtype=torch.float16, device="cuda")
        p1.run(A, B1, C1)
        p2.run(C1, B2, C2)
        p1.run(A, B1, C1)
        torch.cuda.synchronize()
        gu.assert_exact(C2, c2_ref, f"light chain, repetition {rep}")
    assert ctx.last_device_status() == (hgemm.OK, 0)
    p1.close()
    p2.close()


# ---- the small family: register accumulators, for the smallest problems -------------------------------------------

SMALL_CASES = [
    (64, 64, 64), (8, 8, 8), (64, 64, 8), (128, 128, 128), (100, 136, 72), (64, 64, 4096), (256, 256, 256), (200, 328, 200),
    (512, 512, 512), (1000, 64, 136), (64, 2048, 64), (320, 192, 1000),
]


@pytest.mark.parametrize("tile", [64, 32])
@pytest.mark.parametrize("shape", SMALL_CASES, ids=lambda c: "x".join(map(str, c)))
def test_small_family(ctx, gu, shape, tile):
    """mma.sync with register accumulators: the same arithmetic as the tcgen05 kernels (exact on integers, the contract
    on random inputs), tails in every dimension, K shorter and much longer than the cp.async ring."""
    import oracle
    M, N, K = shape
    cfg = hgemm.Config.small(tile)
    assert hgemm.validate_config(M, N, K, cfg) == hgemm.OK
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C, _, plan = gu.run_gemm(ctx, A, B, cfg)
    assert plan.config.family == hgemm.FAMILY_SMALL and plan.config.block_n == tile
    gu.assert_close_full(C, A, B, f"small {shape}")
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
    gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"small {shape} integers")
    Ab, Bb = inputs.make_ab(M, N, K, "binary", "cuda")
    C0 = inputs.draw(39, inputs.TAG_A, M, N, "int5", "cuda")
    for alpha, beta in ((2.0, -1.0), (0.5, 0.0)):
        buf, Cs = gu.alloc_c_with_guards(M, N)                 # pre-filled with a NaN pattern
        if beta != 0.0:
            Cs.copy_(C0)
        plan.run_scaled(alpha, beta, Ab, Bb, Cs)
        assert ctx.last_device_status() == (hgemm.OK, 0) and gu.guards_intact(buf, M, N)
        gu.assert_exact(Cs, oracle.hgemm_scaled_full(inputs.bits(Ab), inputs.bits(Bb), inputs.bits(C0), alpha, beta), f"small {shape} scaled")
    plan.close()


SMALL_SPLIT_CASES = [
    # M, N, K, tile, K slices
    (64, 64, 1024, 32, 8), (64, 64, 1024, 64, 16), (256, 64, 1024, 32, 4), (128, 128, 2048, 64, 2), (100, 136, 1000, 32, 16),
    (200, 72, 328, 64, 4), (1024, 64, 1024, 32, 2), (64, 64, 128, 32, 2), (96, 40, 200, 64, 3), (512, 512, 2048, 64, 8),
]


@pytest.mark.parametrize("case", SMALL_SPLIT_CASES, ids=lambda c: f"{c[0]}x{c[1]}x{c[2]}-t{c[3]}s{c[4]}")
def test_small_family_split_k(ctx, gu, case):
    """The register-accumulator kernel with the K loop cut into the CTAs of a cluster: exact on integers, the contract on
    random inputs, the scaled form, ragged edges, uneven slices (K blocks not a multiple of the slices), and the same
    bits run after run with other work in flight."""
    import oracle
    M, N, K, tile, split = case
    cfg = hgemm.Config.small(tile, split)
    assert hgemm.validate_config(M, N, K, cfg) == hgemm.OK
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C, _, plan = gu.run_gemm(ctx, A, B, cfg)
    assert plan.config.family == hgemm.FAMILY_SMALL and plan.config.split_k == split
    gu.assert_close_full(C, A, B, f"small split {case}")
    bits0 = C.view(torch.int16).clone()
    noise = torch.empty(1 << 22, device="cuda")
    side = torch.cuda.Stream()
    for it in range(4):
        C2 = torch.empty_like(C)
        with torch.cuda.stream(side):
            for _ in range(it % 3 + 1):
                noise.normal_()
        plan.run(A, B, C2)
        torch.cuda.synchronize()
        assert torch.equal(C2.view(torch.int16), bits0), f"run {it} differs"
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
    gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"small split {case} integers")
    Ab, Bb = inputs.make_ab(M, N, K, "binary", "cuda")
    C0 = inputs.draw(39, inputs.TAG_A, M, N, "int5", "cuda")
    for alpha, beta in ((2.0, -1.0), (0.5, 0.0)):
        buf, Cs = gu.alloc_c_with_guards(M, N)
        if beta != 0.0:
            Cs.copy_(C0)
        plan.run_scaled(alpha, beta, Ab, Bb, Cs)
        assert ctx.last_device_status() == (hgemm.OK, 0) and gu.guards_intact(buf, M, N)
        gu.assert_exact(Cs, oracle.hgemm_scaled_full(inputs.bits(Ab), inputs.bits(Bb), inputs.bits(C0), alpha, beta), f"small split {case} scaled")
    plan.close()


def test_small_family_rules(ctx, gu):
    ok = hgemm.Config.small()
    assert hgemm.validate_config(256, 256, 256, ok) == hgemm.OK
    assert hgemm.validate_config(256, 260, 256, ok) == hgemm.ERR_UNSUPPORTED and hgemm.validate_config(256, 256, 260, ok) == hgemm.ERR_UNSUPPORTED
    # K slices: at most 16, at most one per 64-wide k-block, and only inside a cluster
    assert hgemm.validate_config(256, 256, 256, hgemm.Config.small(32, 4)) == hgemm.OK
    assert hgemm.validate_config(256, 256, 256, hgemm.Config.small(32, 8)) == hgemm.ERR_UNSUPPORTED
    assert hgemm.validate_config(256, 256, 4096, hgemm.Config.small(32, 32)) == hgemm.ERR_UNSUPPORTED
    for field, value in (("block_n", 128), ("stages", 4), ("split_k", 2), ("epilogue", TMA), ("swap_ab", 1), ("block_m", 128), ("accumulate", 1)):
        c = hgemm.Config.small()
        setattr(c, field, value)
        assert hgemm.validate_config(256, 256, 256, c) == hgemm.ERR_UNSUPPORTED, field
    # K that needs padded copies: the plan pads, the kernel sees a multiple of 8
    plan = ctx.plan(48, 64, 100)
    plan.set_config(hgemm.Config.small())
    A, B = inputs.make_ab(48, 64, 100, "int5", "cuda")
    C = torch.zeros(48, 64, dtype=torch.float16, device="cuda")
    plan.run(A, B, C)
    torch.cuda.synchronize()
    assert torch.equal(C.float(), A.float() @ B.float().T)
    plan.close()
    nn = ctx.plan(64, 512, 256, layout=hgemm.LAYOUT_NN)
    assert nn.try_set_config(hgemm.Config.small()) == hgemm.ERR_UNSUPPORTED
    nn.close()


def test_dependent_launch_keeps_stream_order(ctx, gu):
    """Launches may become resident before the kernel ahead of them has finished.  A chain in which each
    GEMM consumes the previous GEMM's output must still see stream order: C1 = A B1^T, C2 = C1 B2^T."""
    import oracle
    M, K1, N1, N2 = 512, 64, 64, 384
    A = inputs.draw(1, inputs.TAG_A, M, K1, "int5", "cuda")
    B1 = inputs.draw(2, inputs.TAG_B, N1, K1, "int5", "cuda")
    B2 = inputs.draw(3, inputs.TAG_B, N2, N1, "int5", "cuda")
    c1_ref = oracle.hgemm_full(inputs.bits(A), inputs.bits(B1))                 # |c| <= 256: exact in fp16
    c1_bits = oracle.f64_to_f16_bits(c1_ref.ravel()).reshape(M, N1)
    c2_ref = oracle.hgemm_full(c1_bits, inputs.bits(B2))                        # sums < 2^24: exact in fp32
    p1, p2 = ctx.plan(M, N1, K1), ctx.plan(M, N2, N1)
    for enabled in (True, False):
        ctx.set_dependent_launch(enabled)
        for rep in range(25):
            C1 = torch.zeros(M, N1, dtype=torch.float16, device="cuda")
            C2 = torch.zeros(M, N2, dtype=torch.float16, device="cuda")
            p1.run(A, B1, C1)
            p2.run(C1, B2, C2)
            p1.run(A, B1, C1)                                                   # overwrites what p2 is reading from? no: same values
            torch.cuda.synchronize()
            gu.assert_exact(C2, c2_ref, f"chain, dependent launch {enabled}, repetition {rep}")
    ctx.set_dependent_launch(True)
    assert ctx.last_device_status() == (hgemm.OK, 0)
    p1.close()
    p2.close()


def test_static_operand_promise_keeps_the_other_operand_ordered(ctx, gu):
    """With HGEMM_STATIC_B the weights' first loads leave before the stream dependency is resolved; the activations,
    which the kernel ahead produces, must still be read after it: C1 = A B1^T, C2 = C1 B2^T through every persistent
    path that takes early loads (both families, 64- and 128-wide stages, split-K in a cluster, swapped operands)."""
    import oracle
    M, K1, N1, N2 = 256, 512, 1024, 2048
    A = inputs.draw(1, inputs.TAG_A, M, K1, "binary", "cuda")
    B1 = inputs.draw(2, inputs.TAG_B, N1, K1, "binary", "cuda")
    B2 = inputs.draw(3, inputs.TAG_B, N2, N1, "binary", "cuda")
    c1_ref = oracle.hgemm_full(inputs.bits(A), inputs.bits(B1))                 # <= 512: exact in fp16
    c2_ref = oracle.hgemm_full(oracle.f64_to_f16_bits(c1_ref.ravel()).reshape(M, N1), inputs.bits(B2))   # < 2^24: exact in fp32
    p1, p2 = ctx.plan(M, N1, K1), ctx.plan(M, N2, N1)
    configs = [
        hgemm.Config.make(family=F1, block_n=128, stages=4, raster_group=1, epilogue=TMA, block_k=64),
        hgemm.Config.make(family=F2, block_n=256, stages=3, raster_group=1, epilogue=TMA, block_k=128),
        hgemm.Config.make(family=F1, block_n=128, stages=6, split_k=4, raster_group=1, epilogue=DIRECT, block_k=64, split_mode=CLUSTER),
        hgemm.Config.make(family=F2, block_n=256, stages=4, raster_group=1, epilogue=TMA, block_k=64, swap_ab=1),
        hgemm.Config.make(family=F2, block_n=512, stages=4, raster_group=1, epilogue=TMA, block_k=64),          # the double tile
    ]
    for cfg in configs:
        for plan in (p1, p2):
            plan.set_config(cfg)
            plan.set_static_operands(b=True)
        for rep in range(15):
            C1 = torch.zeros(M, N1, dtype=torch.float16, device="cuda")
            C2 = torch.zeros(M, N2, dtype=torch.float16, device="cuda")
            p1.run(A, B1, C1)
            p2.run(C1, B2, C2)                                                  # reads C1 as its A: not static
            p1.run(A, B1, C1)
            torch.cuda.synchronize()
            gu.assert_exact(C2, c2_ref, f"static B, {cfg.as_dict()}, repetition {rep}")
            gu.assert_exact(C1, c1_ref, f"static B, first product, repetition {rep}")
    assert ctx.last_device_status() == (hgemm.OK, 0)
    assert hgemm.lib().hgemm_plan_set_static_operands(p1._h, 4) == hgemm.ERR_INVALID_ARG
    p1.set_static_operands()
    p1.close()
    p2.close()


# ---- tail split: only the tiles of the last, partly filled wave are cut along K ------------------------------

@pytest.mark.parametrize("family,bn,bk,stages,tail", [(F2, 256, 64, 6, 2), (F1, 256, 64, 4, 2), (F1, 128, 128, 3, 2), (F2, 128, 128, 4, 3)])
@pytest.mark.parametrize("M,N,K", [(4096, 4096, 512), (2000, 4104, 520), (12288, 4096, 256)])
def test_tail_split(ctx, gu, family, bn, bk, stages, tail, M, N, K):
    import oracle
    cfg = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=9, epilogue=TMA, block_k=bk, tail_split=tail)
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C, _, plan = gu.run_gemm(ctx, A, B, cfg)
    gu.assert_close_full(C, A, B, f"tail split {cfg.as_dict()}") if M * N * K <= gu.FULL_CHECK_VOLUME else \
        gu.assert_close_sampled(C, A, B, "uniform", inputs.shape_seed(M, N, K), f"tail split {cfg.as_dict()}")
    bits0 = C.view(torch.int16).clone()
    for _ in range(3):                                   # the split tiles reproduce their bits
        C2, _, _ = gu.run_gemm(ctx, A, B, plan=plan)
        assert torch.equal(C2.view(torch.int16), bits0)
    plan.close()


# ---- wave pacing: the CTAs of the persistent grid start their r-th tile together -------------------------------

PACE_CASES = [
    # family, block_n, block_k, stages, epilogue, raster group, raster mode, M, N, K
    (F2, 256, 64, 6, TMA, 4, 0, 4096, 4096, 512),        # 256 pair tiles on 74 pairs: four rounds, the last one partly filled
    (F1, 128, 128, 3, DIRECT, 8, 1, 4096, 4096, 256),    # 1024 tiles on 148 SMs: seven rounds, serpentine sweep
    (F2, 512, 64, 4, TMA, 8, 1, 4096, 4096, 256),        # the 256 x 512 tile: 128 tiles, two rounds
    (F1, 96, 64, 6, TMA, 3, 0, 3000, 2008, 520),         # ragged in every dimension
    (F2, 192, 64, 5, WIDE, 2, 0, 2048, 6144, 128),       # the wide epilogue
    (F1, 256, 64, 4, TMA, 1, 0, 512, 512, 1024),         # fewer tiles than SMs: one round, nothing to pace
]


@pytest.mark.parametrize("case", PACE_CASES, ids=lambda c: f"f{c[0]}bn{c[1]}bk{c[2]}e{c[4]}-{c[7]}x{c[8]}x{c[9]}")
def test_wave_pacing(ctx, gu, case):
    """wave_pace = 1 changes when tiles start, not what they compute: the same bits as without it, launch after launch
    (the arrival counter counts on from one launch to the next), also with other plans and other work in between."""
    family, bn, bk, stages, epi, rg, rm, M, N, K = case
    base = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=rg, epilogue=epi, block_k=bk, raster_mode=rm)
    paced = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=rg, epilogue=epi, block_k=bk, raster_mode=rm, wave_pace=1)
    assert hgemm.validate_config(M, N, K, paced) == hgemm.OK
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C0, _, plan = gu.run_gemm(ctx, A, B, base)
    gu.assert_close_full(C0, A, B, f"{base.as_dict()}") if M * N * K <= gu.FULL_CHECK_VOLUME else \
        gu.assert_close_sampled(C0, A, B, "uniform", inputs.shape_seed(M, N, K), f"{base.as_dict()}")
    ref_bits = C0.view(torch.int16).clone()
    C1, _, _ = gu.run_gemm(ctx, A, B, paced, plan=plan)
    assert plan.config.wave_pace == 1
    assert torch.equal(C1.view(torch.int16), ref_bits)
    other = ctx.plan(256, 256, 256)
    Ao, Bo = inputs.make_ab(256, 256, 256, "int5", "cuda")
    Co = torch.empty(256, 256, dtype=torch.float16, device="cuda")
    noise = torch.empty(1 << 22, device="cuda")
    side = torch.cuda.Stream()
    for it in range(12):                                 # back to back: a launch starts while the one before it drains
        C = torch.empty_like(C0)
        if it % 3 == 0:
            other.run(Ao, Bo, Co)
        if it % 4 == 1:
            with torch.cuda.stream(side):
                noise.normal_()
        plan.run(A, B, C)
        plan.run(A, B, C)
        torch.cuda.synchronize()
        assert torch.equal(C.view(torch.int16), ref_bits), f"launch {it} differs"
    assert ctx.last_device_status() == (hgemm.OK, 0)
    other.close()
    plan.close()


# ---- stream-K tail: the tiles beyond the full waves as one sequence of k-blocks, dealt out in equal shares ------

STREAM_CASES = [
    # family, block_n, block_k, stages, tail_split, epilogue, M, N, K
    (F1, 256, 64, 4, 2, TMA, 12288, 256, 2048),        # 96 tiles on 148 SMs: no full wave, every tile in two or three pieces
    (F2, 256, 64, 6, 2, TMA, 12288, 256, 2048),        # the same as 48 pair tiles on 74 pairs
    (F1, 128, 128, 3, 4, DIRECT, 128, 12288, 4096),    # 96 tiles of a skinny problem, 128-wide stages
    (F1, 128, 64, 6, 16, TMA, 512, 512, 4096),         # 16 tiles cut into up to 16 pieces each
    (F2, 128, 64, 8, 3, TMA, 4096, 4096, 512),         # full waves first, then a stream-K tail of 68 tiles
    (F1, 256, 64, 4, 2, DIRECT, 4096, 4096, 512),      # ... with direct stores
    (F1, 96, 64, 6, 5, DIRECT, 2000, 4104, 520),       # ragged M, N and K
    (F2, 192, 128, 3, 2, TMA, 2100, 3000, 300),        # ragged, K not a multiple of the stage width, pairs
    (F1, 64, 64, 8, 2, TMA, 100, 1000, 1000),          # fewer positions than SMs
]


@pytest.mark.parametrize("case", STREAM_CASES, ids=lambda c: f"f{c[0]}bn{c[1]}bk{c[2]}t{c[4]}e{c[5]}-{c[6]}x{c[7]}x{c[8]}")
def test_stream_k_tail(ctx, gu, case):
    """HGEMM_TAIL_STREAM against the oracle: uniform inputs at the contract tolerance, small integers exactly, the same
    bits run after run with other work in flight, and the same bits as the configuration without the tail cut
    wherever a tile was left whole."""
    import oracle
    family, bn, bk, stages, tail, epi, M, N, K = case
    cfg = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=4, epilogue=epi, block_k=bk, tail_split=tail,
                            tail_mode=hgemm.TAIL_STREAM)
    assert hgemm.validate_config(M, N, K, cfg) == hgemm.OK
    first = hgemm.stream_item(M, N, K, cfg, 0, 0, torch.cuda.get_device_properties(0).multi_processor_count)
    assert first is not None and first[4] >= 2, "the case is meant to cut tiles"
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C, _, plan = gu.run_gemm(ctx, A, B, cfg)
    gu.assert_close_full(C, A, B, f"stream-K {cfg.as_dict()}") if M * N * K <= gu.FULL_CHECK_VOLUME else \
        gu.assert_close_sampled(C, A, B, "uniform", inputs.shape_seed(M, N, K), f"stream-K {cfg.as_dict()}")
    bits0 = C.view(torch.int16).clone()
    noise = torch.empty(1 << 24, device="cuda")
    side = torch.cuda.Stream()
    for it in range(4):                                  # the cut tiles reproduce their bits
        C2 = torch.empty_like(C)
        with torch.cuda.stream(side):
            for _ in range(it % 3 + 1):
                noise.normal_()
        plan.run(A, B, C2)
        torch.cuda.synchronize()
        assert torch.equal(C2.view(torch.int16), bits0), f"run {it} differs"
    st, code = plan.last_device_status()
    assert st == hgemm.OK, hex(code)
    # whole tiles (the full waves) are computed exactly as without the tail cut
    plain = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=4, epilogue=epi, block_k=bk)
    C_plain, _, _ = gu.run_gemm(ctx, A, B, plain, plan=plan)
    cg = 2 if family == F2 else 1
    tiles_m, tiles_n = -(-M // (128 * cg)), -(-N // bn)
    whole = first[0]                                     # index of the first cut tile = number of whole tiles
    if whole > 0:
        # tiles are numbered along the raster: compare the rows of the first raster group that is entirely whole
        group_tiles = min(4, tiles_m) * tiles_n
        whole_groups = whole // group_tiles
        rows = min(M, whole_groups * min(4, tiles_m) * 128 * cg)
        if rows > 0:
            assert torch.equal(C[:rows].view(torch.int16), C_plain[:rows].view(torch.int16))
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    if M * N * K <= gu.FULL_CHECK_VOLUME:
        plan.set_config(cfg)
        Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
        gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"stream-K, integers {cfg.as_dict()}")
    plan.close()


def test_stream_k_tail_with_other_features(ctx, gu):
    """The stream-K tail under the scaled form, the NN layout and a K that needs padding."""
    import oracle
    M, N, K = 384, 1024, 2056
    cfg = hgemm.Config.make(family=F1, block_n=128, stages=4, raster_group=2, epilogue=TMA, block_k=64, tail_split=4, tail_mode=hgemm.TAIL_STREAM)
    A, B = inputs.make_ab(M, N, K, "int5", "cuda")
    with ctx.plan(M, N, K) as plan:
        plan.set_config(cfg)
        assert hgemm.stream_item(M, N, K, cfg, 0, 0, torch.cuda.get_device_properties(0).multi_processor_count)[4] >= 2
        C0 = inputs.draw(11, 0xC, M, N, "int5", "cuda")
        C = C0.clone()
        plan.run_scaled(0.5, 2.0, A, B, C)
        torch.cuda.synchronize()
        ref = oracle.hgemm_scaled_full(inputs.bits(A), inputs.bits(B), inputs.bits(C0), 0.5, 2.0)
        gu.assert_exact(C, ref, "stream-K, scaled form")
    Bt = B.T.contiguous()                                # K x N row-major
    with ctx.plan(M, N, K, layout=hgemm.LAYOUT_NN) as plan:
        plan.set_config(cfg)
        C = torch.empty(M, N, dtype=torch.float16, device="cuda")
        plan.run(A, Bt, C)
        torch.cuda.synchronize()
        gu.assert_exact(C, oracle.hgemm_full(inputs.bits(A), inputs.bits(B)), "stream-K, NN layout")
    # rules: no transposed stores, no double tile, no light kernel, no fp16 accumulators
    bad = [hgemm.Config.make(family=F1, block_n=128, stages=4, tail_split=4, tail_mode=hgemm.TAIL_STREAM, swap_ab=1),
           hgemm.Config.make(family=F2, block_n=512, stages=3, tail_split=4, tail_mode=hgemm.TAIL_STREAM, epilogue=TMA),
           hgemm.Config.make(family=F1, block_n=128, stages=3, tail_split=4, tail_mode=hgemm.TAIL_STREAM, epilogue=WIDE),
           hgemm.Config.make(family=hgemm.FAMILY_LIGHT, block_n=128, stages=4, tail_split=4, tail_mode=hgemm.TAIL_STREAM),
           hgemm.Config.make(family=F1, block_n=128, stages=4, tail_split=4, tail_mode=hgemm.TAIL_STREAM, accumulate=hgemm.ACC_F16)]
    for c in bad:
        assert hgemm.validate_config(1024, 1024, 1024, c) == hgemm.ERR_UNSUPPORTED, c.as_dict()


# ---- tail split along N: the last wave's tiles as independent narrower tiles ---------------------------------

@pytest.mark.parametrize("family,bn,bk,stages,pieces", [(F2, 256, 128, 3, 2), (F2, 256, 64, 6, 4), (F1, 256, 64, 4, 2), (F1, 128, 128, 3, 4),
                                                        (F2, 192, 128, 3, 2), (F1, 64, 64, 8, 2)])
@pytest.mark.parametrize("M,N,K", [(4096, 4096, 512), (2000, 4104, 520), (12288, 4096, 256), (2100, 3000, 300), (4096, 1280, 384)])
def test_tail_split_along_n(ctx, gu, family, bn, bk, stages, pieces, M, N, K):
    import oracle
    for epi in (TMA, DIRECT):
        cfg = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=9, epilogue=epi, block_k=bk,
                                tail_split=pieces, tail_mode=hgemm.TAIL_N)
        A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
        C, _, plan = gu.run_gemm(ctx, A, B, cfg)
        gu.assert_close_full(C, A, B, f"tail pieces {cfg.as_dict()}") if M * N * K <= gu.FULL_CHECK_VOLUME else \
            gu.assert_close_sampled(C, A, B, "uniform", inputs.shape_seed(M, N, K), f"tail pieces {cfg.as_dict()}")
        # the pieces compute the same dot products in the same order as whole tiles do: bit-identical results
        plain = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=9, epilogue=epi, block_k=bk)
        C_plain, _, _ = gu.run_gemm(ctx, A, B, plain, plan=plan)
        assert torch.equal(C.view(torch.int16), C_plain.view(torch.int16))
        Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
        if M * N * K <= gu.FULL_CHECK_VOLUME:
            plan.set_config(cfg)
            Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
            gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"tail pieces, integers {cfg.as_dict()}")
        plan.close()


# ---- wide TMA-store epilogue: 32-row x 64-column boxes --------------------------------------------------------

WIDE_CASES = [
    # family, bn, bk, stages, tail_split, tail_mode, M, N, K
    (F1, 64, 64, 4, 0, 0, 128, 64, 64),                 # one box per warp pair
    (F1, 128, 64, 4, 0, 0, 100, 136, 72),               # ragged M, N and K; the last box of a row is clipped inside its first half
    (F1, 256, 64, 3, 0, 0, 130, 264, 200),              # one row / one column group past a tile edge
    (F2, 256, 128, 2, 0, 0, 520, 552, 1024),            # CTA pairs, 128-wide stages; N leaves a 40-column edge (second half box empty)
    (F1, 192, 128, 1, 0, 0, 384, 416, 192),             # three boxes per tile: the warps of a quarter get two and one
    (F2, 64, 64, 8, 0, 0, 1024, 2048, 128),             # several tiles per CTA: accumulators and store buffers alternate
    (F1, 256, 64, 3, 0, 0, 4096, 4096, 64),             # epilogue-bound: one k-block per tile
    (F2, 256, 64, 5, 2, 0, 4096, 4096, 512),            # last wave cut along K: whole tiles leave through wide boxes, cut ones through the workspace
    (F2, 256, 64, 5, 2, 1, 2100, 3000, 300),            # last wave cut into two 128-column pieces
    (F1, 256, 64, 3, 4, 1, 4096, 1280, 384),            # ... into four 64-column pieces
    (F1, 128, 64, 4, 0, 0, 77, 204, 333),               # N % 8 != 0: falls back to element stores
]


@pytest.mark.parametrize("case", WIDE_CASES, ids=lambda c: f"f{c[0]}bn{c[1]}bk{c[2]}s{c[3]}t{c[4]}m{c[5]}-{c[6]}x{c[7]}x{c[8]}")
def test_wide_store_epilogue(ctx, gu, case):
    import oracle
    family, bn, bk, stages, tail, tmode, M, N, K = case
    wide = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=4, epilogue=WIDE, block_k=bk,
                             tail_split=tail, tail_mode=tmode)
    narrow = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=4, epilogue=TMA, block_k=bk,
                               tail_split=tail, tail_mode=tmode)
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C, _, plan = gu.run_gemm(ctx, A, B, wide)
    gu.assert_close_full(C, A, B, f"wide {wide.as_dict()}") if M * N * K <= gu.FULL_CHECK_VOLUME else \
        gu.assert_close_sampled(C, A, B, "uniform", inputs.shape_seed(M, N, K), f"wide {wide.as_dict()}")
    # the box width changes nothing in the arithmetic: the same bits as through 32-column boxes
    C_narrow, _, _ = gu.run_gemm(ctx, A, B, narrow, plan=plan)
    assert torch.equal(C.view(torch.int16), C_narrow.view(torch.int16))
    if M * N * K <= gu.FULL_CHECK_VOLUME:
        Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
        plan.set_config(wide)
        Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
        gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), f"wide, integers {wide.as_dict()}")
    plan.close()


def test_wide_store_epilogue_limits(ctx):
    ok = hgemm.Config.make(family=F1, block_n=128, stages=2, epilogue=WIDE, block_k=64)
    assert hgemm.validate_config(512, 512, 512, ok) == hgemm.OK
    for bad in (dict(block_n=96), dict(split_k=2), dict(block_n=128, tail_split=4, tail_mode=hgemm.TAIL_N), dict(block_n=256, stages=4)):
        kw = dict(family=F1, block_n=128, stages=2, epilogue=WIDE, block_k=64)
        kw.update(bad)
        assert hgemm.validate_config(512, 512, 512, hgemm.Config.make(**kw)) == hgemm.ERR_UNSUPPORTED, bad
    # 32 KB more staging: one stage fewer fits than with 32-column boxes
    assert hgemm.validate_config(512, 512, 512, hgemm.Config.make(family=F1, block_n=256, stages=4, epilogue=TMA, block_k=64)) == hgemm.OK


# ---- the NN layout: B given as the K x N operand, row-major ----------------------------------------------

@pytest.mark.parametrize("M,N,K", [(128, 64, 64), (100, 136, 72), (300, 520, 200), (1024, 1024, 1024), (64, 64, 8192),
                                    (512, 384, 640), (256, 4096, 4096), (2048, 2048, 2048)])
def test_nn_layout(ctx, gu, M, N, K):
    """All three matrices row-major (the paper's "NN" layout, section 2.2): same product, B indexed [k][j]."""
    import oracle
    for dist in ("uniform", "int5"):
        A, B_nk = inputs.make_ab(M, N, K, dist, "cuda")
        B_kn = B_nk.T.contiguous()                       # the same operand, stored K x N
        plan = ctx.plan(M, N, K, hgemm.LAYOUT_NN)
        buf, C = gu.alloc_c_with_guards(M, N)
        plan.run(A, B_kn, C)
        assert ctx.last_device_status() == (hgemm.OK, 0)
        assert gu.guards_intact(buf, M, N)
        if dist == "int5":
            gu.assert_exact(C, oracle.hgemm_full(inputs.bits(A), inputs.bits(B_nk)), f"NN {M}x{N}x{K} integers")
        else:
            gu.assert_close_full(C, A, B_nk, f"NN {M}x{N}x{K} {plan.config.as_dict()}")
        plan.close()
    with pytest.raises(hgemm.HgemmError):
        ctx.plan(64, 60, 64, hgemm.LAYOUT_NN)             # ragged rows of B cannot be fetched by TMA in this layout


NN_FEATURE_CASES = [
    # M, N, K, configuration keywords, what it combines with the NN layout
    (4096, 1280, 384, dict(family=F2, block_n=256, stages=6, block_k=64, epilogue=TMA, tail_split=2, tail_mode=hgemm.TAIL_N), "tail tiles cut into column pieces"),
    (4096, 2560, 512, dict(family=F1, block_n=256, stages=4, block_k=64, epilogue=DIRECT, tail_split=2, tail_mode=hgemm.TAIL_N), "column pieces, 1-CTA family"),
    (300, 520, 4096, dict(family=F2, block_n=128, stages=4, block_k=64, epilogue=DIRECT, split_k=4, split_mode=CLUSTER), "cluster split-K of CTA pairs"),
    (256, 384, 4096, dict(family=F1, block_n=128, stages=4, block_k=64, epilogue=DIRECT, split_k=3, split_mode=WORKSPACE), "workspace split-K"),
    (520, 392, 1024, dict(family=F1, block_n=128, stages=3, block_k=128, epilogue=TMA, accumulate=hgemm.ACC_F16), "fp16 accumulators"),
]


@pytest.mark.parametrize("case", NN_FEATURE_CASES, ids=lambda c: f"{c[0]}x{c[1]}x{c[2]}-{c[4].replace(' ', '_').replace(',', '')}")
def test_nn_layout_with_other_features(ctx, gu, case):
    """The row-major-B layout combined with the tail pieces, both split-K exchanges, the scaled form and fp16
    accumulators: the same results as the TN layout gives for the same operands, bit for bit."""
    import oracle
    M, N, K, kw, what = case
    cfg = hgemm.Config.make(raster_group=4, **kw)
    A, B_nk = inputs.make_ab(M, N, K, "binary", "cuda")      # 0/1 operands: every sum exact in either accumulator
    B_kn = B_nk.T.contiguous()
    plan_nn = ctx.plan(M, N, K, hgemm.LAYOUT_NN)
    plan_nn.set_config(cfg)
    plan_tn = ctx.plan(M, N, K)
    plan_tn.set_config(cfg)
    buf, C_nn = gu.alloc_c_with_guards(M, N)
    plan_nn.run(A, B_kn, C_nn)
    assert ctx.last_device_status() == (hgemm.OK, 0)
    assert gu.guards_intact(buf, M, N)
    gu.assert_exact(C_nn, oracle.hgemm_full(inputs.bits(A), inputs.bits(B_nk)), f"NN with {what}")
    Au, Bu_nk = inputs.make_ab(M, N, K, "uniform", "cuda")
    Bu_kn = Bu_nk.T.contiguous()
    C0 = inputs.draw(31, inputs.TAG_A, M, N, "uniform", "cuda")
    C_nn = C0.clone()
    C_tn = C0.clone()
    plan_nn.run_scaled(1.5, -0.5, Au, Bu_kn, C_nn)
    plan_tn.run_scaled(1.5, -0.5, Au, Bu_nk, C_tn)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == (hgemm.OK, 0)
    assert torch.equal(C_nn.view(torch.int16), C_tn.view(torch.int16)), f"NN and TN differ with {what}"
    if kw.get("accumulate", 0) == 0:
        ref = oracle.hgemm_scaled_full(inputs.bits(Au), inputs.bits(Bu_nk), inputs.bits(C0), 1.5, -0.5)
        assert oracle.check_contract(gu.bits_to_f64(gu.c_bits(C_nn)), ref, K, abs_scale=1.5)["ok"]
    plan_nn.close()
    plan_tn.close()


# ---- configuration 2: square sweep ---------------------------------------------------------------------

@pytest.mark.parametrize("S", [1024, 2048, 4096, 8192])
def test_config2_square(ctx, gu, S):
    rep = gu.check_shape(ctx, S, S, S, "uniform")
    assert rep["rel_frobenius"] < 3e-4


@pytest.mark.parametrize("family,bn,stages,epi", [(F1, 256, 4, TMA), (F1, 256, 4, DIRECT), (F2, 256, 6, TMA),
                                                   (F2, 256, 4, DIRECT), (F2, 224, 4, TMA)])
def test_config2_bench_configurations_4096(ctx, gu, family, bn, stages, epi):
    """The launch configurations the benchmark times on 4096^3, checked on samples + one row + one column."""
    gu.check_shape(ctx, 4096, 4096, 4096, "uniform", _cfg(family, bn, stages, 1, 4, epi))


# ---- configuration 3: skinny LLM projections, N(0,1)/sqrt(K) ----------------------------------------------

@pytest.mark.parametrize("NK", [(4096, 4096), (12288, 4096), (4096, 12288)])
@pytest.mark.parametrize("M", [64, 128, 256])
def test_config3_skinny(ctx, gu, M, NK):
    N, K = NK
    rep = gu.check_shape(ctx, M, N, K, "normal")
    assert rep["rel_frobenius"] < 3e-4


# ---- configuration 4: small M, N with large K; split-K determinism ------------------------------------------

@pytest.mark.parametrize("K", [8192, 12288])
@pytest.mark.parametrize("MN", [64, 256, 512])
def test_config4_small_mn_large_k(ctx, gu, MN, K):
    gu.check_shape(ctx, MN, MN, K, "uniform")


@pytest.mark.parametrize("family,mode", [(F1, WORKSPACE), (F2, WORKSPACE), (F1, CLUSTER), (F2, CLUSTER)])
@pytest.mark.parametrize("MN,K,bn,split", [(64, 8192, 64, 8), (64, 12288, 32, 48), (256, 12288, 128, 12),
                                            (512, 8192, 128, 6), (512, 12288, 256, 16), (512, 12288, 256, 4),
                                            (512, 12288, 192, 16)])
def test_split_k_is_deterministic(ctx, gu, family, mode, MN, K, bn, split):
    """Every split-K configuration reproduces its own bits run after run, with other work in flight
    to perturb the order in which slices finish."""
    if mode == CLUSTER and split * (2 if family == F2 else 1) > 16:
        pytest.skip("a cluster holds at most 16 CTAs")
    cfg = _cfg(family, bn, 4, split, 1, DIRECT, 64, mode)
    if mode == CLUSTER and hgemm.validate_config(MN, MN, K, cfg) == hgemm.ERR_UNSUPPORTED:
        pytest.skip("this tile's partial sums and received shares do not fit in shared memory")
    A, B = inputs.make_ab(MN, MN, K, "uniform", "cuda")
    C0, _, plan = gu.run_gemm(ctx, A, B, cfg)
    gu.assert_close_full(C0, A, B, f"split-K {cfg.as_dict()}")
    ref_bits = C0.view(torch.int16).clone()
    noise = torch.empty(1 << 24, device="cuda")
    side = torch.cuda.Stream()
    for it in range(10):
        C = torch.empty_like(C0)
        with torch.cuda.stream(side):
            for _ in range(it % 3 + 1):
                noise.normal_()
        plan.run(A, B, C)
        torch.cuda.synchronize()
        assert torch.equal(C.view(torch.int16), ref_bits), f"run {it} differs"
    plan.close()


# ---- the input generator draws the same bits on both devices --------------------------------------------------

def test_generator_matches_across_devices():
    for dist in ("uniform", "int5", "binary"):
        a = inputs.draw(77, inputs.TAG_A, 513, 264, dist, "cpu")
        b = inputs.draw(77, inputs.TAG_A, 513, 264, dist, "cuda")
        assert torch.equal(a, b.cpu()), dist


# ---- the general form C = alpha A B^T + beta C (paper section 2.1) ------------------------------------------

SCALED_CASES = [
    # M, N, K, config (None: the planner's), why
    (128, 128, 128, None, "one tile"),
    (300, 264, 520, ("f1", 96, 4, 1, 64, WORKSPACE, TMA), "ragged tiles, TMA-store epilogue"),
    (300, 264, 520, ("f1", 96, 4, 1, 64, WORKSPACE, DIRECT), "direct stores"),
    (520, 392, 1024, ("f2", 128, 3, 1, 128, WORKSPACE, TMA), "CTA pairs"),
    (77, 203, 333, None, "N and K not multiples of 8: element-wise reads of the old C"),
    (256, 384, 4096, ("f1", 128, 4, 4, 64, WORKSPACE, DIRECT), "split-K through the workspace"),
    (256, 384, 4096, ("f2", 128, 4, 3, 64, WORKSPACE, DIRECT), "split-K, CTA pairs"),
    (64, 640, 2048, ("f1", 160, 2, 7, 128, CLUSTER, DIRECT), "split-K inside a cluster"),
    (300, 520, 4096, ("f2", 128, 4, 4, 64, CLUSTER, DIRECT), "split-K inside a cluster of CTA pairs"),
]


@pytest.mark.parametrize("case", SCALED_CASES, ids=lambda c: f"{c[0]}x{c[1]}x{c[2]}-{c[4].split(':')[0].replace(' ', '_')}")
def test_scaled_form_matches_oracle(ctx, gu, case):
    import oracle
    M, N, K, cfg_t, why = case
    plan = ctx.plan(M, N, K)
    if cfg_t is not None:
        fam, bn, stages, split, bk, mode, epi = cfg_t
        plan.set_config(_cfg(F1 if fam == "f1" else F2, bn, stages, split, 1, epi, bk, mode))
    # exact case: 0/1 operands, small integers in C and factors that keep every fp32 intermediate exact
    Ai, Bi = inputs.make_ab(M, N, K, "binary", "cuda")
    C0 = inputs.draw(21, inputs.TAG_A, M, N, "int5", "cuda")
    for alpha, beta in [(1.0, 1.0), (2.0, -3.0), (-1.0, 0.5), (0.0, 2.0), (0.5, 0.0)]:
        buf, C = gu.alloc_c_with_guards(M, N)
        C.copy_(C0)
        plan.run_scaled(alpha, beta, Ai, Bi, C)
        st, code = ctx.last_device_status()
        assert st == hgemm.OK, f"device status {st} code {code:#x}"
        assert gu.guards_intact(buf, M, N), f"{why}: the kernel wrote outside C"
        ref = oracle.hgemm_scaled_full(inputs.bits(Ai), inputs.bits(Bi), inputs.bits(C0), alpha, beta)
        assert np.abs(ref).max() < 2 ** 24          # every fp32 intermediate is exact: both sides round the same number once
        gu.assert_exact(C, ref, f"{why}: alpha={alpha} beta={beta}")
    # beta == 0 never reads the old C: NaN there must not reach the result
    buf, C = gu.alloc_c_with_guards(M, N)               # pre-filled with a NaN pattern
    plan.run_scaled(2.0, 0.0, Ai, Bi, C)
    gu.assert_exact(C, oracle.hgemm_scaled_full(inputs.bits(Ai), inputs.bits(Bi), None, 2.0, 0.0), f"{why}: beta=0 over NaN")
    # random inputs: the contract's bound with its absolute term scaled by |alpha|
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    Cu = inputs.draw(22, inputs.TAG_B, M, N, "uniform", "cuda")
    for alpha, beta in [(0.75, -1.5), (-2.5, 0.3)]:
        buf, C = gu.alloc_c_with_guards(M, N)
        C.copy_(Cu)
        plan.run_scaled(alpha, beta, A, B, C)
        ref = oracle.hgemm_scaled_full(inputs.bits(A), inputs.bits(B), inputs.bits(Cu), alpha, beta)
        rep = oracle.check_contract(gu.bits_to_f64(gu.c_bits(C)), ref, K, abs_scale=abs(alpha))
        assert rep["ok"], f"{why}: alpha={alpha} beta={beta}: {rep}"
    # hgemm_run is the case alpha = 1, beta = 0, bit for bit
    C1, _, _ = gu.run_gemm(ctx, A, B, plan=plan)
    buf, C2 = gu.alloc_c_with_guards(M, N)
    plan.run_scaled(1.0, 0.0, A, B, C2)
    assert torch.equal(C1.view(torch.int16), C2.view(torch.int16))
    assert hgemm.lib().hgemm_run_scaled(plan._h, float("nan"), 0.0, A.data_ptr(), B.data_ptr(), C2.data_ptr(), 0) == hgemm.ERR_INVALID_ARG
    plan.close()


# ---- fp16 accumulators (the paper's other setting for fp16 inputs, section 1) ----------------------------------

F16ACC_CASES = [
    # family, bn, bk, stages, epilogue, tail pieces, M, N, K
    (F1, 128, 64, 4, TMA, 0, 128, 128, 128),
    (F1, 64, 128, 4, DIRECT, 0, 200, 136, 520),
    (F2, 256, 64, 4, TMA, 0, 512, 520, 1024),
    (F2, 128, 128, 4, DIRECT, 0, 300, 264, 2048),
    (F1, 96, 64, 4, TMA, 0, 77, 203, 333),              # ragged N and K
    (F2, 256, 64, 6, TMA, 2, 2100, 3000, 300),          # with the last wave cut into column pieces
    (F1, 256, 64, 4, TMA, 0, 256, 256, 4096),
]


@pytest.mark.parametrize("case", F16ACC_CASES, ids=lambda c: f"f{c[0]}bn{c[1]}bk{c[2]}e{c[4]}t{c[5]}-{c[6]}x{c[7]}x{c[8]}")
def test_fp16_accumulation(ctx, gu, case):
    import oracle
    family, bn, bk, stages, epi, pieces, M, N, K = case
    cfg = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=4, epilogue=epi, block_k=bk,
                            tail_split=pieces, tail_mode=hgemm.TAIL_N if pieces else hgemm.TAIL_K, accumulate=hgemm.ACC_F16)
    # exact case: every partial sum, in any order, is an integer of magnitude <= 2048
    Ab, Bb = inputs.make_ab(M, N, K, "binary", "cuda")
    bound = float((Ab.float() @ Bb.float().T).max())
    assert bound <= 2048
    C, _, plan = gu.run_gemm(ctx, Ab, Bb, cfg)
    gu.assert_exact(C, oracle.hgemm_full(inputs.bits(Ab), inputs.bits(Bb)), f"fp16 accumulation, 0/1 operands {cfg.as_dict()}")
    # Random inputs.  What is asserted is what holds for every schedule that rounds the running sum at most once
    # per 16-wide K step (one MMA instruction) to one of its two fp16 neighbours: the envelope computed from the
    # fp64 oracle's prefix sums.  No hardware-fitted model takes part in the verdict.
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C, _, _ = gu.run_gemm(ctx, A, B, plan=plan)
    exact, bound = oracle.f16acc_envelope(inputs.bits(A), inputs.bits(B))
    got = gu.bits_to_f64(gu.c_bits(C))
    err = np.abs(got - exact)
    assert np.isfinite(got).all()
    assert (err <= bound).all(), f"outside the fp16-accumulation envelope: worst {float((err / bound).max()):.3f} of it"
    # Reported, never asserted: how much of the result equals the schedule "one round-to-nearest per MMA step"
    model = oracle.f16_bits_to_f64(oracle.hgemm_f16acc_full(inputs.bits(A), inputs.bits(B)).ravel()).reshape(M, N)
    print(f"fp16 accumulation {M}x{N}x{K}: {float(np.mean(got == model)):.4f} of the entries equal the per-step "
          f"round-to-nearest model; worst error {float((err / bound).max()):.3f} of the envelope")
    # and it is a different arithmetic from fp32 accumulation: once K is large its relative Frobenius error is
    # above the 2^-11 that fp32 accumulators must stay under (they leave one final rounding, about 2^-12.2; K / 16
    # roundings of the running sum leave about 2^-9 at K = 1024); the same plan with fp32 accumulators meets the contract
    if K >= 1024:
        assert np.sqrt((err ** 2).sum() / (exact ** 2).sum()) > 2.0 ** -11
    cfg32 = hgemm.Config.make(family=family, block_n=bn, stages=stages, raster_group=4, epilogue=epi, block_k=bk,
                              tail_split=pieces, tail_mode=hgemm.TAIL_N if pieces else hgemm.TAIL_K)
    C32, _, _ = gu.run_gemm(ctx, A, B, cfg32, plan=plan)
    assert oracle.check_contract(gu.bits_to_f64(gu.c_bits(C32)), exact, K)["ok"]
    plan.close()


def test_fp16_accumulation_rejects_splits_along_k(ctx):
    bad = hgemm.Config.make(block_n=128, stages=4, split_k=2, accumulate=hgemm.ACC_F16)
    assert hgemm.validate_config(256, 256, 4096, bad) == hgemm.ERR_UNSUPPORTED
    bad = hgemm.Config.make(block_n=128, stages=4, tail_split=2, accumulate=hgemm.ACC_F16)
    assert hgemm.validate_config(256, 256, 4096, bad) == hgemm.ERR_UNSUPPORTED


# ---- special values: infinities, NaN, overflow of the fp16 result -------------------------------------------

def test_infinities_nan_and_overflow(ctx, gu):
    """IEEE behaviour the paper does not discuss but a drop-in GEMM must have: inf and NaN operands propagate
    as the exact arithmetic of the oracle says, and sums beyond 65504 round to infinity."""
    import oracle
    M, N, K = 128, 96, 128
    A, B = inputs.make_ab(M, N, K, "int5", "cuda")
    A = A.clone(); B = B.clone()
    A[23, :] = 60000.0; B[5, :] = 1.0; B[6, :] = -1.0             # overflow: about +-7.7e6 -> +-inf after rounding to fp16
    A[3, 5] = float("inf"); B[:, 5] = B[:, 5].abs() + 1           # row 3: +inf times positive values -> +inf everywhere
    A[7, 9] = float("-inf"); B[0:48, 9] = 2.0; B[48:, 9] = -2.0   # row 7: -inf and +inf halves
    A[11, 20] = float("inf"); B[17, 20] = 0.0                     # inf * 0 -> NaN in one element (row 11, column 17)
    A[19, 33] = float("nan")                                      # row 19: NaN everywhere
    C, _, plan = gu.run_gemm(ctx, A, B, _cfg(F1, 96, 4, 1, 1, TMA))
    ref = oracle.hgemm_full(inputs.bits(A), inputs.bits(B))       # fp64 arithmetic: inf, NaN as IEEE defines them
    want = oracle.f64_to_f16_bits(ref.ravel()).reshape(M, N)
    got = gu.c_bits(C)
    want_nan = np.isnan(ref)
    got_nan = np.isnan(gu.bits_to_f64(got))
    assert np.array_equal(got_nan, want_nan), "NaN pattern differs"
    assert want_nan[19].all() and want_nan[11, 17] and not want_nan[3].any()
    ok = ~want_nan
    assert np.array_equal(oracle.canonical_bits(got)[ok], oracle.canonical_bits(want)[ok])
    assert np.isposinf(ref[3]).all() and np.isneginf(ref[7, :48]).all() and np.isposinf(ref[7, 48:]).all()
    assert gu.bits_to_f64(got)[23, 5] == np.inf and gu.bits_to_f64(got)[23, 6] == -np.inf       # 7.68e6 does not fit fp16
    # the same through the CTA-pair kernel and a split-K reduction (partial sums carry inf / NaN through fp32)
    for cfg in (_cfg(F2, 96, 4, 1, 1, DIRECT), _cfg(F1, 96, 4, 2, 1, DIRECT, 64, CLUSTER), _cfg(F1, 96, 4, 2, 1, DIRECT, 64, WORKSPACE)):
        C2, _, _ = gu.run_gemm(ctx, A, B, cfg, plan=plan)
        g2 = gu.c_bits(C2)
        assert np.array_equal(np.isnan(gu.bits_to_f64(g2)), want_nan), cfg.as_dict()
        assert np.array_equal(oracle.canonical_bits(g2)[ok], oracle.canonical_bits(want)[ok]), cfg.as_dict()
    plan.close()


# ---- run-time tuning of a plan --------------------------------------------------------------------------------

@pytest.mark.parametrize("M,N,K", [(3584, 896, 1024), (320, 5000, 512), (100, 136, 77), (64, 640, 4096)])
def test_plan_autotune(ctx, gu, M, N, K):
    """hgemm_plan_autotune leaves a legal configuration that is at least as fast as the one it started from,
    C holding the product, and the plan usable as before."""
    import oracle
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    C = torch.zeros(M, N, dtype=torch.float16, device="cuda")
    plan = ctx.plan(M, N, K)
    before = plan.config

    def per_call_us(n=50):
        for _ in range(5):
            plan.run(A, B, C)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            plan.run(A, B, C)
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) / n * 1e3

    t_before = min(per_call_us() for _ in range(3))
    C.zero_()
    us = plan.autotune(A, B, C, max_candidates=24)
    assert us > 0.0
    after = plan.config
    assert hgemm.validate_config(M, N, (K + 7) // 8 * 8, after) == hgemm.OK
    gu.assert_close_full(C, A, B, f"autotuned {after.as_dict()}")          # C is the product on return
    t_after = min(per_call_us() for _ in range(3))
    # (margin for timing noise: the small shapes are bound by the host's launch rate)
    assert t_after <= 1.25 * t_before + 1.0, (t_before, t_after, before.as_dict(), after.as_dict())
    Ai, Bi = inputs.make_ab(M, N, K, "int5", "cuda")
    Ci, _, _ = gu.run_gemm(ctx, Ai, Bi, plan=plan)
    gu.assert_exact(Ci, oracle.hgemm_full(inputs.bits(Ai), inputs.bits(Bi)), "autotuned plan, integers")
    assert ctx.last_device_status() == (hgemm.OK, 0)
    plan.close()


def test_plan_autotune_on_nn_layout_skips_unsupported_candidates(ctx, gu):
    M, N, K = 520, 392, 1024
    A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
    Bt = B.T.contiguous()                                                  # the K x N operand
    C = torch.empty(M, N, dtype=torch.float16, device="cuda")
    plan = ctx.plan(M, N, K, hgemm.LAYOUT_NN)
    us = plan.autotune(A, Bt, C, max_candidates=16)
    assert us > 0.0
    gu.assert_close_full(C, A, B, f"autotuned NN {plan.config.as_dict()}")
    plan.close()


def test_every_grid_shape_plans_in_both_layouts(ctx):
    """hgemm_plan / hgemm_plan_layout accept all 729 grid shapes: the NN layout adapts the tabulated configuration
    (whole 64-column blocks per CTA, fewer stages with the planned epilogue's staging) and must end up legal."""
    grid = [64, 128, 256, 512, 1024, 2048, 4096, 8192, 12288]
    for M in grid:
        for N in grid:
            for K in grid:
                for layout in (hgemm.LAYOUT_TN, hgemm.LAYOUT_NN):
                    plan = ctx.plan(M, N, K, layout)
                    c = plan.config
                    assert hgemm.validate_config(M, N, K, c) == hgemm.OK, (M, N, K, layout, c.as_dict())
                    if layout == hgemm.LAYOUT_NN:
                        assert c.block_n % (64 * (c.family + 1)) == 0
                    plan.close()
