"""Host-side checks of the seeded input generator and of the acceptance rules (CPU only)."""
import numpy as np
import torch

from paper_2512_02551_b200 import inputs


def test_splitmix64_reference_vector():
    # First outputs of SplitMix64 seeded with 0 (the published reference sequence of the
    # generator: state += golden gamma, then the two multiply-xorshift rounds).
    want = [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    state = 0
    for w in want:
        assert inputs._splitmix64_int(state) == w
        state = (state + inputs._GOLDEN) & inputs._MASK64
    t = torch.tensor([inputs._s64(i * inputs._GOLDEN) for i in range(3)], dtype=torch.int64)
    got = [int(v) & inputs._MASK64 for v in inputs._splitmix64(t)]
    assert got == want


def test_draw_is_stateless_and_row_addressable():
    a = inputs.draw(42, inputs.TAG_A, 300, 200, "uniform")
    again = inputs.draw(42, inputs.TAG_A, 300, 200, "uniform", chunk_rows=7)
    assert torch.equal(a, again)
    rows = [299, 0, 17, 17]
    sub = inputs.draw(42, inputs.TAG_A, 300, 200, "uniform", row_index=rows)
    assert torch.equal(sub, a[rows])
    assert not torch.equal(a, inputs.draw(43, inputs.TAG_A, 300, 200, "uniform"))
    assert not torch.equal(a[:200], inputs.draw(42, inputs.TAG_B, 200, 200, "uniform"))


def test_distributions():
    u = inputs.draw(1, 1, 512, 512, "uniform").double()
    assert u.min() >= -1 and u.max() <= 1
    assert abs(u.mean()) < 0.01 and abs(u.var() - 1 / 3) < 0.01
    i5 = inputs.draw(1, 1, 512, 512, "int5").double()
    assert set(np.unique(i5.numpy())) == {-2.0, -1.0, 0.0, 1.0, 2.0}
    nb = inputs.draw(1, 1, 256, 4096, "normal").double()
    assert abs(nb.mean()) < 1e-3 and abs(nb.std() * 64 - 1) < 0.02
    bn = inputs.draw(1, 1, 256, 4096, "binary", p=0.25).double()
    assert abs(bn.mean() - 0.25) < 0.01
    assert inputs.shape_seed(64, 128, 256) != inputs.shape_seed(128, 64, 256)


def test_contract_rejects_wrong_results(oracle_lib):
    M, N, K = 64, 96, 512
    a, b = inputs.make_ab(M, N, K)
    ref = oracle_lib.hgemm_full(inputs.bits(a), inputs.bits(b))
    good = oracle_lib.f16_bits_to_f64(oracle_lib.f64_to_f16_bits(ref.ravel())).reshape(M, N)
    an = a.double().norm(dim=1).numpy()
    bn = b.double().norm(dim=1).numpy()
    assert oracle_lib.check_contract(good, ref, K)["ok"]
    rep = oracle_lib.check_scale_aware(good, ref, K, an, bn)
    assert rep["ok"] and rep["rel_frobenius"] < 3e-4
    # a transposed result, a dropped k-block and a NaN all fail
    a2, b2 = inputs.make_ab(N, M, K)
    assert not oracle_lib.check_contract(good, oracle_lib.hgemm_full(inputs.bits(b), inputs.bits(a)).T + 1.0, K)["ok"]
    dropped = oracle_lib.hgemm_full(inputs.bits(a[:, :K - 64]), inputs.bits(b[:, :K - 64]))
    assert not oracle_lib.check_contract(dropped, ref, K)["ok"]
    bad = good.copy()
    bad[3, 5] = np.nan
    assert not oracle_lib.check_contract(bad, ref, K)["ok"]
    # the loose absolute term alone would accept zeros for small-valued outputs; the
    # scale-aware check does not
    an_, bn_ = inputs.make_ab(M, N, 4096, dist="normal")
    refn = oracle_lib.hgemm_full(inputs.bits(an_), inputs.bits(bn_))
    assert oracle_lib.check_contract(np.zeros_like(refn), refn, 4096)["ok"]
    assert not oracle_lib.check_scale_aware(np.zeros_like(refn), refn, 4096)["ok"]


def test_canonical_bits(oracle_lib):
    x = np.array([0x8000, 0x0000, 0x3c00, 0xbc00], dtype=np.uint16)
    assert list(oracle_lib.canonical_bits(x)) == [0, 0, 0x3c00, 0xbc00]
