"""Pins for the oracle's triple loop (CPU only).

Each test fixes the loop against something the mathematics decides, chosen so that
a dropped term, a wrong index or a transposed operand fails at least one:
exact int64 arithmetic on integer inputs, identity / permutation / rank-1 closed
forms on non-square shapes, a library fp64 matmul, exact rationals on tiny shapes.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from paper_2512_02551_b200 import inputs


def _f16_exact(bits):
    """Independent decode: numpy float16 -> python float (exact)."""
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (64, 192, 320), (37, 53, 1000), (8, 16, 12288)])
def test_integer_inputs_match_int64(oracle_lib, M, N, K):
    a, b = inputs.make_ab(M, N, K, dist="int5")
    ai = a.to(torch.int64).numpy()
    bi = b.to(torch.int64).numpy()
    want = ai @ bi.T                                       # exact integer arithmetic
    got = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    assert got.shape == (M, N)
    assert np.array_equal(got, want.astype(np.float64))
    assert np.abs(want).max() > 0
    # the rounded result is the integer itself wherever it is representable
    small = np.abs(want) <= 2048
    assert np.array_equal(_f16_exact(oracle_lib.f64_to_f16_bits(got.ravel()))[small.ravel()],
                          want.astype(np.float64).ravel()[small.ravel()])


def test_identity_returns_b_transposed(oracle_lib):
    K = M = 96
    N = 40
    b = inputs.draw(7, inputs.TAG_B, N, K, "uniform")
    eye = torch.eye(M, K, dtype=torch.float16)
    got = oracle_lib.hgemm_full(inputs.bits(eye), inputs.bits(b))
    assert np.array_equal(got, b.double().numpy().T)


def test_permutation_selects_columns(oracle_lib):
    M, N, K = 50, 70, 90
    rng = np.random.default_rng(3)
    pi = rng.permutation(K)[:M]
    a = torch.zeros(M, K, dtype=torch.float16)
    a[torch.arange(M), torch.from_numpy(pi)] = 1.0
    b = inputs.draw(11, inputs.TAG_B, N, K, "uniform")
    got = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    want = b.double().numpy()[:, pi].T                     # C[i][j] = B[j][pi(i)]
    assert np.array_equal(got, want)


def test_rank1_one_hot_k(oracle_lib):
    M, N, K, k0 = 33, 65, 128, 77
    u = inputs.draw(5, 1, M, 1, "uniform")[:, 0]
    v = inputs.draw(5, 2, N, 1, "uniform")[:, 0]
    a = torch.zeros(M, K, dtype=torch.float16)
    b = torch.zeros(N, K, dtype=torch.float16)
    a[:, k0] = u
    b[:, k0] = v
    got = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    want = np.outer(u.double().numpy(), v.double().numpy())  # exact: 22-bit products
    assert np.array_equal(got, want)
    got16 = oracle_lib.f64_to_f16_bits(got.ravel())
    want16 = want.astype(np.float16).view(np.uint16).ravel()
    assert np.array_equal(got16, want16)


@pytest.mark.parametrize("K", [64, 4096, 12288])
def test_rank1_constant_along_k(oracle_lib, K):
    M, N = 24, 40
    vals = np.array([0.5, 1.0, 2.0, -0.5, -1.0, -2.0])
    rng = np.random.default_rng(K)
    u = rng.choice(vals, M)
    v = rng.choice(vals, N)
    a = torch.from_numpy(np.repeat(u[:, None], K, 1)).to(torch.float16)
    b = torch.from_numpy(np.repeat(v[:, None], K, 1)).to(torch.float16)
    got = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    assert np.array_equal(got, K * np.outer(u, v))         # every partial sum is exact


@pytest.mark.parametrize("dist", ["uniform", "normal"])
def test_library_fp64_matmul(oracle_lib, dist):
    M, N, K = 70, 90, 2048
    a, b = inputs.make_ab(M, N, K, dist=dist)
    got = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    want = torch.matmul(a.double(), b.double().T).numpy()  # other summation order, fp64
    scale = (a.double().abs() @ b.double().abs().T).numpy()
    assert np.all(np.abs(got - want) <= 1e-12 * scale + 1e-300)


def test_tiny_shapes_exact_rationals(oracle_lib):
    for (M, N, K) in [(1, 1, 1), (2, 3, 5), (4, 7, 8), (8, 8, 8), (3, 2, 17)]:
        a, b = inputs.make_ab(M, N, K, dist="uniform", seed=100 + M + N + K)
        af = [[Fraction(float(x)) for x in row] for row in a.tolist()]
        bf = [[Fraction(float(x)) for x in row] for row in b.tolist()]
        got = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
        for i in range(M):
            for j in range(N):
                exact = sum(af[i][k] * bf[j][k] for k in range(K))
                # K <= 17 terms of <= 22 bits each: the fp64 sum is exact
                assert Fraction(float(got[i, j])) == exact, (M, N, K, i, j)


def test_sampled_equals_full_and_handles_gathered_rows(oracle_lib):
    M, N, K = 45, 77, 256
    a, b = inputs.make_ab(M, N, K)
    full = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    ii, jj, row, col = inputs.sample_indices(99, M, N, n=500)
    got = oracle_lib.hgemm_sampled(inputs.bits(a), inputs.bits(b), ii, jj)
    assert np.array_equal(got, full[ii, jj])
    # gathered form: only the needed rows are drawn
    ui, inv_i = np.unique(ii, return_inverse=True)
    uj, inv_j = np.unique(jj, return_inverse=True)
    s = inputs.shape_seed(M, N, K)
    ag = inputs.draw(s, inputs.TAG_A, M, K, row_index=ui)
    bg = inputs.draw(s, inputs.TAG_B, N, K, row_index=uj)
    assert torch.equal(ag, a[torch.from_numpy(ui)])
    got2 = oracle_lib.hgemm_sampled(inputs.bits(ag), inputs.bits(bg), inv_i, inv_j)
    assert np.array_equal(got2, got)
    with pytest.raises(IndexError):
        oracle_lib.hgemm_sampled(inputs.bits(a), inputs.bits(b), [M], [0])


def test_empty_and_degenerate(oracle_lib):
    z = oracle_lib.hgemm_full(np.zeros((0, 8), np.uint16), np.zeros((5, 8), np.uint16))
    assert z.shape == (0, 5)
    z = oracle_lib.hgemm_full(np.zeros((3, 0), np.uint16), np.zeros((5, 0), np.uint16))
    assert z.shape == (3, 5) and not z.any()               # empty sum = 0
    with pytest.raises(ValueError):
        oracle_lib.hgemm_full(np.zeros((3, 4), np.uint16), np.zeros((5, 6), np.uint16))
    with pytest.raises(TypeError):
        oracle_lib.hgemm_full(np.zeros((3, 4), np.float32), np.zeros((5, 4), np.float32))


def test_paper_style_binary_exact_match(oracle_lib):
    """Section 2.3 "Exact Match with binary Inputs": {0,1} inputs give non-negative integer
    sums; every entry below 2048 is exactly representable in fp16."""
    M, N, K = 64, 64, 8192
    p = inputs.binary_p(K)
    a, b = inputs.make_ab(M, N, K, dist="binary", p=p)
    got = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    want = (a.to(torch.int64) @ b.to(torch.int64).T).numpy()
    assert np.array_equal(got, want)
    frac_checkable = np.mean((want > 0) & (want < 2048))
    assert frac_checkable > 0.9
    r16 = _f16_exact(oracle_lib.f64_to_f16_bits(got.ravel())).reshape(M, N)
    assert np.array_equal(r16[want < 2048], want[want < 2048].astype(np.float64))


# ---- the general form C = alpha A B^T + beta C (paper section 2.1) ------------------------------------------

def test_scaled_form_exact_rationals(oracle_lib):
    """Brute force on tiny shapes: alpha, beta and every element as exact rationals."""
    for (M, N, K, alpha, beta) in [(2, 3, 5, 0.5, -2.0), (4, 7, 8, -1.25, 0.75), (3, 2, 9, 3.0, 1.0)]:
        a, b = inputs.make_ab(M, N, K, dist="uniform", seed=7 + M + N + K)
        c = inputs.draw(11, inputs.TAG_A, M, N, "uniform")
        af = [[Fraction(float(x)) for x in row] for row in a.tolist()]
        bf = [[Fraction(float(x)) for x in row] for row in b.tolist()]
        cf = [[Fraction(float(x)) for x in row] for row in c.tolist()]
        got = oracle_lib.hgemm_scaled_full(inputs.bits(a), inputs.bits(b), inputs.bits(c), alpha, beta)
        for i in range(M):
            for j in range(N):
                exact = Fraction(alpha) * sum(af[i][k] * bf[j][k] for k in range(K)) + Fraction(beta) * cf[i][j]
                # a few dozen bits in all: every fp64 operation above is exact
                assert Fraction(float(got[i, j])) == exact, (M, N, K, i, j)


def test_scaled_form_special_cases(oracle_lib):
    M, N, K = 33, 65, 96
    a, b = inputs.make_ab(M, N, K, dist="int5")
    c = inputs.draw(5, inputs.TAG_A, M, N, "int5")
    ab = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    cb = inputs.bits(c)
    # alpha = 1, beta = 0 is the plain product, whatever C holds (NaN included)
    nan_c = np.full((M, N), 0x7E00, dtype=np.uint16)
    assert np.array_equal(oracle_lib.hgemm_scaled_full(inputs.bits(a), inputs.bits(b), nan_c, 1.0, 0.0), ab)
    # alpha = 0 leaves beta C; integers keep everything exact
    assert np.array_equal(oracle_lib.hgemm_scaled_full(inputs.bits(a), inputs.bits(b), cb, 0.0, 3.0),
                          3.0 * c.to(torch.float64).numpy())
    # linear in (alpha, beta): int64 arithmetic decides
    want = 2 * (a.to(torch.int64).numpy() @ b.to(torch.int64).numpy().T) - 3 * c.to(torch.int64).numpy()
    assert np.array_equal(oracle_lib.hgemm_scaled_full(inputs.bits(a), inputs.bits(b), cb, 2.0, -3.0), want.astype(np.float64))
    # the factors are the fp32 values the library receives
    third = oracle_lib.hgemm_scaled_full(inputs.bits(a), inputs.bits(b), cb, 1.0 / 3.0, 0.0)
    assert np.array_equal(third, float(np.float32(1.0 / 3.0)) * ab)
    with pytest.raises(ValueError):
        oracle_lib.hgemm_scaled_full(inputs.bits(a), inputs.bits(b), cb[:, :-1], 1.0, 1.0)


# ---- fp16 accumulation: the running sum is rounded once per 16-wide K step -------------------------------------

def test_f16_accumulation_rounding_points(oracle_lib):
    """Hand-made rows that show where the model rounds: 2048 + 1 + 1 in three K steps stays 2048
    (each +1 is a tie that goes to the even neighbour), while the exact sum is 2050; the same
    numbers inside ONE step are added exactly and give 2050."""
    one = np.float16(1.0).view(np.uint16)
    def row(vals, K):
        r = np.zeros(K, dtype=np.float16); r[:len(vals)] = vals; return r.view(np.uint16)
    K = 48
    a = np.zeros((1, K), dtype=np.float16); b = np.zeros((1, K), dtype=np.float16)
    a[0, :16] = 32.0; b[0, :16] = 4.0          # first step: 16 * 128 = 2048
    a[0, 16] = 1.0; b[0, 16] = 1.0             # second step: +1
    a[0, 32] = 1.0; b[0, 32] = 1.0             # third step: +1
    got = oracle_lib.hgemm_f16acc_full(a.view(np.uint16), b.view(np.uint16))
    assert oracle_lib.f16_bits_to_f64(got.ravel())[0] == 2048.0
    assert oracle_lib.hgemm_full(a.view(np.uint16), b.view(np.uint16))[0, 0] == 2050.0
    # the same three contributions inside one 16-wide step: exact inner sum, one rounding
    a2 = np.zeros((1, 16), dtype=np.float16); b2 = np.zeros((1, 16), dtype=np.float16)
    a2[0, :14] = 32.0; b2[0, :14] = 4.0; a2[0, 14] = 16.0; b2[0, 14] = 16.0   # 14 * 128 + 256 = 2048
    a2[0, 15] = 2.0; b2[0, 15] = 1.0                                          # + 2
    got2 = oracle_lib.hgemm_f16acc_full(a2.view(np.uint16), b2.view(np.uint16))
    assert oracle_lib.f16_bits_to_f64(got2.ravel())[0] == 2050.0
    # a step size of the whole K is one rounding of the exact product
    a3, b3 = inputs.make_ab(9, 11, 64, dist="uniform")
    whole = oracle_lib.hgemm_f16acc_full(inputs.bits(a3), inputs.bits(b3), k_step=64)
    assert np.array_equal(whole, oracle_lib.f64_to_f16_bits(oracle_lib.hgemm_full(inputs.bits(a3), inputs.bits(b3)).ravel()).reshape(9, 11))


def test_f16_accumulation_exact_when_sums_are_representable(oracle_lib):
    """Integer operands whose absolute products sum to at most 2048 per element: every partial sum,
    in any order, is an integer fp16 holds exactly, so the model must return the exact product."""
    M, N, K = 40, 56, 640
    a, b = inputs.make_ab(M, N, K, dist="int5")
    bound = np.abs(a.to(torch.int64).numpy()) @ np.abs(b.to(torch.int64).numpy()).T
    assert bound.max() <= 2048
    want = (a.to(torch.int64).numpy() @ b.to(torch.int64).numpy().T).astype(np.float64)
    got = oracle_lib.f16_bits_to_f64(oracle_lib.hgemm_f16acc_full(inputs.bits(a), inputs.bits(b)).ravel()).reshape(M, N)
    assert np.array_equal(got, want)


def test_f16_accumulation_error_grows_with_k(oracle_lib):
    """On random inputs the model differs from the exact product by roughly sqrt(K / 16) roundings of the
    running magnitude -- more than fp32 accumulation would, less than the worst case."""
    M, N, K = 32, 48, 2048
    a, b = inputs.make_ab(M, N, K, dist="uniform")
    exact = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    got = oracle_lib.f16_bits_to_f64(oracle_lib.hgemm_f16acc_full(inputs.bits(a), inputs.bits(b)).ravel()).reshape(M, N)
    err = np.abs(got - exact)
    half_ulp = 2.0 ** -7                       # half the fp16 spacing at the largest running magnitudes (32..64)
    assert err.max() > 2.0 ** -11 * np.abs(exact).max()          # worse than one final rounding
    assert err.max() < (K / 16) * half_ulp                       # far inside the worst case


# ---- the envelope that fp16 accumulation is held to: valid for every faithful rounding schedule -----------------

def test_f16_spacing_is_the_ieee_spacing(oracle_lib):
    """Against numpy's own float16 spacing on every finite non-negative fp16 value."""
    bits = np.arange(0, 0x7C00, dtype=np.uint16)
    vals = bits.view(np.float16)
    with np.errstate(over="ignore"):
        want = np.spacing(vals).astype(np.float64)
    # np.spacing at the largest finite value overflows to inf in float16: the spacing there is 32
    want[-1] = 32.0
    assert np.array_equal(oracle_lib.f16_spacing(vals.astype(np.float64)), want)


def _neighbours16(x):
    """The two fp16 values that enclose the real number x (equal when x is representable)."""
    h = np.float16(x)
    if float(h) == x:
        return float(h), float(h)
    other = np.nextafter(h, np.float16(np.inf) if float(h) < x else np.float16(-np.inf))
    lo, hi = sorted((float(h), float(other)))
    assert lo < x < hi
    return lo, hi


@pytest.mark.parametrize("dist,K", [("uniform", 64), ("uniform", 512), ("int5", 2048), ("normal", 256)])
def test_f16acc_envelope_holds_for_every_faithful_schedule(oracle_lib, dist, K):
    """Brute force on small problems: run the accumulation in python floats under adversarial roundings --
    always up, always down, away from the exact prefix, to nearest, random -- and with rounding every 16, 32
    or 64 columns or once at the end; every result must lie inside the envelope computed for steps of 16."""
    M, N = 3, 4
    a, b = inputs.make_ab(M, N, K, dist=dist)
    af, bf = _f16_exact(inputs.bits(a)), _f16_exact(inputs.bits(b))
    exact, bound = oracle_lib.f16acc_envelope(inputs.bits(a), inputs.bits(b))
    assert np.allclose(exact, af @ bf.T, rtol=1e-13, atol=0)
    rng = np.random.default_rng(7)
    worst = 0.0
    for every in (16, 32, 64, K):
        for policy in ("up", "down", "away", "nearest", "random"):
            for i in range(M):
                for j in range(N):
                    d, prefix = 0.0, 0.0
                    for k0 in range(0, K, every):
                        s = float(np.dot(af[i, k0:k0 + every], bf[j, k0:k0 + every]))   # exact: few short products
                        prefix += s
                        lo, hi = _neighbours16(d + s)
                        if policy == "up":
                            d = hi
                        elif policy == "down":
                            d = lo
                        elif policy == "away":
                            d = hi if hi - prefix >= prefix - lo else lo
                        elif policy == "nearest":
                            d = float(np.float16(d + s))
                        else:
                            d = hi if rng.random() < 0.5 else lo
                    e = abs(d - exact[i, j])
                    assert e <= bound[i, j], (every, policy, i, j, e, bound[i, j])
                    worst = max(worst, e / bound[i, j])
    if dist == "int5":
        assert worst == 0.0      # every partial sum is a small integer: nothing is ever rounded
    else:
        assert worst > 0.05      # the envelope is not vacuous: adversarial schedules come within sight of it


def test_f16acc_envelope_on_the_hand_made_row(oracle_lib):
    """2048 + 1 + 1 over three steps: round-to-nearest-even loses both ones (error 2), rounding up gains
    two (2052); the envelope must admit both and is a handful of spacings wide, not more."""
    K = 48
    a = np.zeros((1, K), dtype=np.float16); b = np.zeros((1, K), dtype=np.float16)
    a[0, :16] = 32.0; b[0, :16] = 4.0
    a[0, 16] = 1.0; b[0, 16] = 1.0
    a[0, 32] = 1.0; b[0, 32] = 1.0
    exact, bound = oracle_lib.f16acc_envelope(a.view(np.uint16), b.view(np.uint16))
    assert exact[0, 0] == 2050.0
    assert 2.0 <= bound[0, 0] <= 6.0          # spacing 1 below 2048 once, then spacing 2 twice: 1 + 2 + 2 = 5


# ---- IEEE special values through the loop ------------------------------------------------------------------------

def test_infinities_and_nan_propagate_as_ieee_says(oracle_lib):
    """Three hand-written rows of A against three of B (K = 4); the expected values are IEEE 754's own:
    inf * finite = inf with the product's sign, inf * 0 = NaN, inf - inf = NaN, NaN absorbs everything,
    and finite sums beyond 65504 + 16 round to infinity only in the fp16 encoding, not in the fp64 result."""
    inf, nan = np.inf, np.nan
    A = np.array([[inf, 1.0, 2.0, 0.0],
                  [-inf, 0.0, 0.0, 3.0],
                  [nan, 1.0, 1.0, 1.0]], dtype=np.float16)
    B = np.array([[1.0, 1.0, 1.0, 1.0],        # row 0: +inf, row 1: -inf, row 2: NaN
                  [0.0, 5.0, 5.0, 5.0],        # inf * 0 = NaN for rows 0 and 1, NaN for row 2
                  [-2.0, 60000.0, 60000.0, 0.0]],  # row 0: -inf + finite = -inf; row 1: +inf; row 2: NaN
                 dtype=np.float16)
    got = oracle_lib.hgemm_full(A.view(np.uint16), B.view(np.uint16))
    want = np.array([[inf, nan, -inf],
                     [-inf, nan, inf],
                     [nan, nan, nan]])
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])
    # inf - inf inside one dot product
    A2 = np.array([[inf, -inf, 1.0, 1.0], [inf, inf, 1.0, 1.0]], dtype=np.float16)
    B2 = np.array([[1.0, 1.0, 1.0, 1.0]], dtype=np.float16)
    got2 = oracle_lib.hgemm_full(A2.view(np.uint16), B2.view(np.uint16))
    assert np.isnan(got2[0, 0]) and got2[1, 0] == inf
    # overflow belongs to the fp16 encoding: the fp64 sum is finite, its fp16 image is infinite
    A3 = np.array([[60000.0, 60000.0, 0.0, 0.0]], dtype=np.float16)
    B3 = np.array([[1.0, 1.0, 0.0, 0.0], [-1.0, -1.0, 0.0, 0.0], [1.0, 0.09, 0.0, 0.0]], dtype=np.float16)
    got3 = oracle_lib.hgemm_full(A3.view(np.uint16), B3.view(np.uint16))
    assert got3[0, 0] == 2.0 * float(np.float16(60000.0)) and np.isfinite(got3).all()
    enc = oracle_lib.f64_to_f16_bits(got3.ravel())
    assert enc[0] == 0x7C00 and enc[1] == 0xFC00                  # +inf, -inf
    assert enc[2] == np.float16(got3[0, 2]).view(np.uint16) and enc[2] < 0x7C00   # about 65400: still finite
