"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and its planner returns legal configurations."""
import os
import re

import pytest

from paper_2512_02551_b200 import build as hbuild
from paper_2512_02551_b200 import hgemm

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GRID = [64, 128, 256, 512, 1024, 2048, 4096, 8192, 12288]


@pytest.fixture(scope="module")
def lib():
    hbuild.build()
    return hgemm.lib()


def test_header_symbols_are_exported(lib):
    text = open(os.path.join(ROOT, "include", "hgemm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(hgemm_[a-z_]+)\s*\(", text))
    assert declared == set(hgemm.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    seen = {hgemm.status_string(s) for s in range(8)}
    assert len(seen) == 8 and "ok" in seen


def test_shape_rules(lib):
    for bad in [(0, 64, 64), (64, 0, 64), (64, 64, 0), (-1, 64, 64)]:
        with pytest.raises(hgemm.HgemmError) as e:
            hgemm.heuristic_config(*bad)
        assert e.value.status == hgemm.ERR_INVALID_ARG
    for unsup in [(64, 64, 1 << 23), (1 << 23, 64, 64)]:
        with pytest.raises(hgemm.HgemmError) as e:
            hgemm.heuristic_config(*unsup)
        assert e.value.status == hgemm.ERR_UNSUPPORTED
    for odd in [(1, 1, 1), (64, 60, 64), (64, 64, 60), (7, 13, 1001)]:   # ragged rows are handled by the plan
        hgemm.heuristic_config(*odd)


def test_heuristic_is_legal_over_the_grid(lib):
    for M in GRID:
        for N in GRID:
            for K in GRID:
                c = hgemm.heuristic_config(M, N, K)
                assert hgemm.validate_config(M, N, K, c) == hgemm.OK, (M, N, K, c.as_dict())
                assert hgemm.config_smem_bytes(c) <= 232448
                assert c.split_k <= (K + 63) // 64
                if c.split_k > 1 and c.split_mode == hgemm.SPLIT_WORKSPACE:
                    assert hgemm.config_workspace_bytes(M, N, K, c) > 0
                else:
                    assert hgemm.config_workspace_bytes(M, N, K, c) == 0


def test_validate_rejects_illegal_configs(lib):
    M = N = K = 1024
    ok = hgemm.Config.make(block_n=128, stages=4)
    assert hgemm.validate_config(M, N, K, ok) == hgemm.OK
    for kw in [dict(block_n=48), dict(block_n=288), dict(block_n=0), dict(stages=0), dict(stages=13),
               dict(block_n=256, stages=5), dict(split_k=0), dict(split_k=17), dict(block_k=32), dict(block_k=256), dict(raster_group=0),
               dict(epilogue=3), dict(family=4)]:
        c = hgemm.Config.make(**{**dict(block_n=128, stages=4), **kw})
        assert hgemm.validate_config(M, N, K, c) == hgemm.ERR_UNSUPPORTED, kw
    c = hgemm.Config.make(block_n=128, stages=4)
    c.block_m = 256                           # wrong for the 1-CTA family
    assert hgemm.validate_config(M, N, K, c) == hgemm.ERR_UNSUPPORTED
    c = hgemm.Config.make(block_n=128, stages=4)
    c.reserved[0] = 1
    assert hgemm.validate_config(M, N, K, c) == hgemm.ERR_UNSUPPORTED
    # wave pacing: 0 or 1, whole equal tiles of the persistent kernel only
    assert hgemm.validate_config(M, N, K, hgemm.Config.make(block_n=128, stages=4, wave_pace=1)) == hgemm.OK
    assert hgemm.validate_config(M, N, K, hgemm.Config.make(family=1, block_n=512, stages=4, epilogue=hgemm.EPILOGUE_TMA, wave_pace=1)) == hgemm.OK
    for kw in [dict(wave_pace=2), dict(wave_pace=1, split_k=2), dict(wave_pace=1, tail_split=2), dict(wave_pace=1, tail_split=2, tail_mode=hgemm.TAIL_STREAM),
               dict(wave_pace=1, family=hgemm.FAMILY_LIGHT)]:
        c = hgemm.Config.make(**{**dict(block_n=128, stages=4), **kw})
        assert hgemm.validate_config(M, N, K, c) == hgemm.ERR_UNSUPPORTED, kw
    small = hgemm.Config.small()
    small.wave_pace = 1
    assert hgemm.validate_config(M, N, K, small) == hgemm.ERR_UNSUPPORTED
    # cluster split-K: at most 16 CTAs per cluster (16 slices, 8 for CTA pairs), the ring must hold the fp32 partial
    assert hgemm.validate_config(M, N, 4096, hgemm.Config.make(block_n=128, stages=4, split_k=8, split_mode=1)) == hgemm.OK
    assert hgemm.validate_config(M, N, 4096, hgemm.Config.make(family=1, block_n=128, stages=4, split_k=8, split_mode=1)) == hgemm.OK
    for kw in [dict(family=1, split_k=12), dict(split_k=32), dict(block_n=256, stages=2, split_k=4)]:
        c = hgemm.Config.make(**{**dict(block_n=128, stages=4, split_mode=1), **kw})
        assert hgemm.validate_config(M, N, 4096, c) == hgemm.ERR_UNSUPPORTED, kw
    # wide TMA-store epilogue: 64-column boxes need block_n (and column pieces) in multiples of 64, no split along K,
    # and 32 KB more store staging
    wide = hgemm.Config.make(block_n=128, stages=4, epilogue=hgemm.EPILOGUE_TMA_WIDE)
    assert hgemm.validate_config(M, N, K, wide) == hgemm.OK
    assert hgemm.config_smem_bytes(wide) == hgemm.config_smem_bytes(ok) + 32768
    for kw in [dict(block_n=96), dict(block_n=160), dict(split_k=2), dict(block_n=256, stages=4), dict(tail_split=4, tail_mode=hgemm.TAIL_N)]:
        c = hgemm.Config.make(**{**dict(block_n=128, stages=4, epilogue=hgemm.EPILOGUE_TMA_WIDE), **kw})
        assert hgemm.validate_config(M, N, K, c) == hgemm.ERR_UNSUPPORTED, kw
    assert hgemm.validate_config(M, N, K, hgemm.Config.make(block_n=256, stages=3, epilogue=hgemm.EPILOGUE_TMA_WIDE,
                                                            tail_split=4, tail_mode=hgemm.TAIL_N)) == hgemm.OK
    pair = hgemm.Config.make(family=hgemm.FAMILY_UMMA_2CTA, block_n=256, stages=6)
    assert hgemm.validate_config(M, N, K, pair) == hgemm.OK
    assert hgemm.config_smem_bytes(pair) == 1024 + 6 * (16384 + 128 * 128) + 32768 + 512


def test_workspace_size(lib):
    c = hgemm.Config.make(block_n=64, stages=4, split_k=8)
    # one 128 x 64 fp32 partial per slice + 2 counters of 4 bytes for the single tile
    assert hgemm.config_workspace_bytes(64, 64, 8192, c) == 8 * 128 * 64 * 4 + 8


def test_no_gpu_create_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(hgemm.HgemmError):
        hgemm.Context(0)


def test_planned_config_for_tabulated_and_other_shapes(lib):
    """hgemm_planned_config: the table's entry on a tabulated shape; elsewhere a legal configuration that the
    cost model does not rank behind the pure heuristic's choice by more than the neighbours' calibration allows."""
    c = hgemm.planned_config(4096, 4096, 4096)
    assert hgemm.validate_config(4096, 4096, 4096, c) == hgemm.OK
    assert (c.family, c.block_n) == (hgemm.FAMILY_UMMA_2CTA, 256)          # the tuned entry of the flagship square
    shapes = [(1, 1, 1), (7, 9, 11), (1536, 1536, 1536), (96, 11008, 4096), (3000, 5000, 7000), (200, 200, 20000),
              (16384, 16384, 16384), (4194304, 64, 64), (64, 64, 4194304), (77, 203, 333)]
    for (M, N, K) in shapes:
        c = hgemm.planned_config(M, N, K)
        Kp = (K + 7) // 8 * 8                                               # plans run on K padded to a multiple of 8
        assert hgemm.validate_config(M, N, Kp, c) == hgemm.OK, (M, N, K, c.as_dict())
        assert 1 <= c.split_k <= -(-Kp // c.block_k)
        assert c.accumulate == hgemm.ACC_F32                                # fp16 accumulators are never chosen
        h = hgemm.heuristic_config(M, N, Kp)
        # a re-fitted neighbour only replaces the heuristic's choice when the model, scaled by what was measured
        # around the shape, prefers it; the raw estimates therefore stay within the spread of those scales
        assert hgemm.estimate_config(M, N, Kp, c) <= 3.0 * hgemm.estimate_config(M, N, Kp, h)
    with pytest.raises(hgemm.HgemmError):
        hgemm.planned_config(0, 64, 64)


def test_every_grid_shape_plans_to_a_legal_configuration(lib):
    """The tuned table covers the 9 x 9 x 9 grid: every entry must validate against its own shape (a stale
    entry would silently fall back to the neighbours' configurations)."""
    grid = [64, 128, 256, 512, 1024, 2048, 4096, 8192, 12288]
    families = set()
    for M in grid:
        for N in grid:
            for K in grid:
                c = hgemm.planned_config(M, N, K)
                assert hgemm.validate_config(M, N, K, c) == hgemm.OK, (M, N, K, c.as_dict())
                assert hgemm.config_smem_bytes(c) <= 232448
                families.add(c.family)
    assert {hgemm.FAMILY_UMMA_1CTA, hgemm.FAMILY_UMMA_2CTA} <= families <= {hgemm.FAMILY_UMMA_1CTA, hgemm.FAMILY_UMMA_2CTA, hgemm.FAMILY_LIGHT, hgemm.FAMILY_SMALL}


def test_candidate_configs_are_legal_ranked_and_distinct(lib):
    for (M, N, K) in [(64, 64, 64), (8, 8, 8), (3584, 896, 1024), (13824, 512, 16384), (4096, 4096, 4096), (100, 136, 77)]:
        Kp = (K + 7) // 8 * 8                                        # the library pads K to a multiple of 8
        cands = hgemm.candidate_configs(M, N, K, max_count=48)
        assert 1 <= len(cands) <= 48
        est = [hgemm.estimate_config(M, N, Kp, c) for c in cands]
        assert est == sorted(est)                                    # best estimate first
        assert all(hgemm.validate_config(M, N, Kp, c) == hgemm.OK for c in cands)
        keys = {tuple(sorted(c.as_dict().items())) for c in cands}
        assert len(keys) == len(cands)
    # all three families, both stage widths, split-K and the wide epilogue all occur among the candidates of a shape that admits them
    pool = hgemm.candidate_configs(512, 512, 4096, max_count=256)
    assert {c.family for c in pool} == {0, 1, 2, 3} and {c.block_k for c in pool} == {64, 128}
    small = [c for c in pool if c.family == hgemm.FAMILY_SMALL]                               # its two tiles, whole or in 2..16 K slices
    assert {c.block_n for c in small} <= {32, 64} and 1 <= len(small) <= 10
    assert all(c.split_mode == hgemm.SPLIT_CLUSTER for c in small if c.split_k > 1) and {c.split_k for c in small} <= {1, 2, 4, 8, 16}
    tiny = hgemm.candidate_configs(128, 128, 128, max_count=256)
    assert {c.block_n for c in tiny if c.family == hgemm.FAMILY_SMALL} == {32, 64}
    assert all(c.split_k == 1 and c.epilogue != hgemm.EPILOGUE_TMA_WIDE for c in pool if c.family == hgemm.FAMILY_LIGHT)
    big = hgemm.candidate_configs(8192, 8192, 8192, max_count=256)
    assert any(c.block_n == 512 and c.family == hgemm.FAMILY_UMMA_2CTA for c in big)          # the double-accumulator tile
    skinny = hgemm.candidate_configs(64, 12288, 4096, max_count=256)
    assert any(c.swap_ab == 1 for c in skinny) and not any(c.swap_ab for c in big)            # swapped operands: few rows only
    assert any(c.split_k > 1 and c.split_mode == 1 for c in pool) and any(c.split_k > 1 and c.split_mode == 0 for c in pool)
    assert any(c.epilogue == hgemm.EPILOGUE_TMA_WIDE for c in pool)
    assert hgemm.candidate_configs(0, 64, 64) == [] and hgemm.candidate_configs(64, 64, 1 << 30) == []



def test_table_file_overrides_the_built_in_table(lib, tmp_path):
    """HGEMM_TABLE names a file of tuner rows that take precedence over the compiled-in table (read once per process,
    so the check runs in a child process)."""
    import subprocess
    import sys
    table = tmp_path / "table.inc"
    table.write_text("// a comment line\n"
                     "{4096, 4096, 4096, 0, 96, 64, 5, 1, 0, 0, 7, 0, 0, 123.00f, 0, 1, 1},\n"   # a tabulated shape, overridden (newest row format)
                     "{1000, 2000, 3000, 1, 128, 128, 3, 1, 0, 0, 4, 1, 0, 50.00f},\n"            # an off-grid shape, old row format
                     "{64, 64, 64, 0, 48, 64, 2, 1, 0, 0, 1, 0, 0, 1.00f, 0, 0},\n")              # an illegal row: ignored
    code = ("from paper_2512_02551_b200 import hgemm\n"
            "a = hgemm.planned_config(4096, 4096, 4096); b = hgemm.planned_config(1000, 2000, 3000); c = hgemm.planned_config(64, 64, 64)\n"
            "print(a.family, a.block_n, a.stages, a.raster_group, a.raster_mode, b.family, b.block_n, b.block_k, c.block_n, a.wave_pace, b.wave_pace)")
    env = dict(os.environ, HGEMM_TABLE=str(table), PYTHONPATH=ROOT)
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, check=True).stdout.split()
    assert out[:8] == ["0", "96", "5", "7", "1", "1", "128", "128"]
    assert out[8] != "48"
    assert out[9:11] == ["1", "0"]


def test_every_table_row_is_what_the_planner_returns(lib):
    """A row of the tuned table that failed validation would silently be replaced by its neighbours' configurations:
    every row of the compiled-in table must come back from the planner field by field."""
    path = os.path.join(ROOT, "paper_2512_02551_b200", "csrc", "hgemm_table.inc")
    rows = 0
    families = set()
    for line in open(path):
        if not line.startswith("{"):
            continue
        v = [x.strip().rstrip("f") for x in line.strip().rstrip(",").strip("{}").split(",")]
        M, N, K, family, bn, bk, stages, split, mode, tail, rg, epi, tail_mode = (int(x) for x in v[:13])
        swap, raster_mode = (int(v[14]), int(v[15])) if len(v) >= 16 else (0, 0)
        pace = int(v[16]) if len(v) >= 17 else 0
        c = hgemm.planned_config(M, N, K)
        got = (c.family, c.block_n, c.block_k, c.stages, c.split_k, c.split_mode, c.tail_split, c.raster_group, c.epilogue, c.tail_mode,
               c.swap_ab, c.raster_mode, c.wave_pace)
        assert got == (family, bn, bk, stages, split, mode, tail, rg, epi, tail_mode, swap, raster_mode, pace), (M, N, K, got, line)
        rows += 1
        families.add(family)
    assert rows >= 1000 and families == {0, 1, 2, 3}


def _stream_partition(M, N, K, family, bn, bk, tail, sms):
    """Brute-force check of one stream-K tail: returns None where the configuration has none on this shape."""
    cfg = hgemm.Config.make(family=family, block_n=bn, stages=3, block_k=bk, tail_split=tail, tail_mode=hgemm.TAIL_STREAM,
                            epilogue=hgemm.EPILOGUE_TMA)
    if hgemm.validate_config(M, N, K, cfg) != hgemm.OK or hgemm.stream_item(M, N, K, cfg, 0, 0, sms) is None:
        return None
    cg = 2 if family == hgemm.FAMILY_UMMA_2CTA else 1
    units = sms // cg
    tiles = -(-M // (128 * cg)) * -(-N // bn)
    kb = -(-K // bk)
    rem = tiles % units
    cover, per_tile, positions = {}, {}, None
    for j in range(units):
        for h in (0, 1):
            t, k0, n, sl, sls, gs = hgemm.stream_item(M, N, K, cfg, j, h, sms)
            positions = gs
            if n == 0:
                continue
            assert j < gs and tiles - rem <= t < tiles and 0 <= k0 and k0 + n <= kb
            for k in range(k0, k0 + n):
                assert (t, k) not in cover, "a k-block is computed twice"
                cover[(t, k)] = j
            per_tile.setdefault(t, []).append((sl, sls, k0, j, h))
    assert len(cover) == rem * kb, "a k-block of the tail is computed by no one"
    for t, frags in per_tile.items():
        frags.sort()
        sls = frags[0][1]
        assert [f[0] for f in frags] == list(range(sls)) and all(f[1] == sls for f in frags), "slices 0..S-1, once each"
        assert [f[2] for f in frags] == sorted(f[2] for f in frags), "slices are in K order"
        assert [f[3] for f in frags] == list(range(frags[0][3], frags[0][3] + sls)), "consecutive positions"
        assert all(f[4] == 0 for f in frags[1:]), "only a tile's first piece can be a position's second item"
    shares = [sum(1 for v in cover.values() if v == j) for j in range(positions)]
    assert max(shares) - min(shares) <= 1, "equal shares"
    most = max(len(v) for v in per_tile.values())
    # the workspace holds `most` slots per cut tile
    assert hgemm.config_workspace_bytes(M, N, K, cfg) >= 0
    return positions, most


def test_stream_k_tail_partition(lib):
    """The arithmetic that deals the tail's k-blocks out (the kernel decodes its work items with the same function):
    every k-block of every cut tile exactly once, equal shares, a tile's pieces on consecutive positions in K order."""
    import itertools
    checked = 0
    shapes = [(12288, 256, 12288), (128, 12288, 12288), (512, 4096, 8192), (4096, 4096, 4096), (640, 640, 640), (100, 1000, 1000),
              (2048, 2048, 256), (256, 256, 12288), (64, 64, 16384), (12288, 12288, 128)]
    for (M, N, K) in shapes:
        for family, bn, bk, tail in itertools.product((0, 1), (32, 128, 192, 256), (64, 128), (2, 3, 8, 16)):
            checked += _stream_partition(M, N, K, family, bn, bk, tail, 148) is not None
    for sms in (2, 4, 7, 16, 132):                       # other SM counts (the layout is a function of the device)
        for family, bn, tail in itertools.product((0, 1), (64, 256), (2, 5, 16)):
            checked += _stream_partition(3000, 1000, 2000, family, bn, 64, tail, sms) is not None
    assert checked > 300
    # 96 tiles of 128 x 256 on 148 SMs: all 148 positions, each tile in two or three pieces
    assert _stream_partition(12288, 256, 12288, 0, 256, 64, 2, 148) == (148, 3)
    # a whole number of waves, or too few k-blocks to share: no tail, the configuration runs as if tail_split were off
    cfg = hgemm.Config.make(family=0, block_n=128, stages=3, tail_split=2, tail_mode=hgemm.TAIL_STREAM, epilogue=hgemm.EPILOGUE_TMA)
    assert hgemm.stream_item(148 * 128, 128, 4096, cfg, 0, 0, 148) is None
    assert hgemm.stream_item(4096, 4096, 64, cfg, 0, 0, 148) is None
    assert hgemm.config_workspace_bytes(4096, 4096, 64, cfg) == 0


def test_checked_build_exports_the_same_abi(lib):
    """The checked build (-DHGEMM_CHECKED=1) is a second library with the same exports; which one is loaded is the
    environment's choice (HGEMM_LIB), and each says which it is."""
    import ctypes
    import subprocess
    import sys
    path = hbuild.build(checked=True)
    assert os.path.basename(path) == "libhgemm_checked.so" and os.path.exists(path)
    L = ctypes.CDLL(path)
    for name in hgemm.EXPORTS:
        assert hasattr(L, name), name
    L.hgemm_build_is_checked.restype = ctypes.c_int32
    assert L.hgemm_build_is_checked() == 1 and lib.hgemm_build_is_checked() == 0
    code = "from paper_2512_02551_b200 import hgemm; print(int(hgemm.build_is_checked()), hgemm.LIB_PATH)"
    out = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, HGEMM_LIB=path, PYTHONPATH=ROOT), capture_output=True, text=True,
                         check=True).stdout.split()
    assert out == ["1", path]
    assert hgemm.status_string(hgemm.ERR_CHECK) == "the checked build found an invariant violated"


def test_tuner_candidates_and_table_round_trip(lib, tmp_path):
    """The tuner's host side: every candidate it would time is legal, every kernel family and mode is among them where the
    shape admits it, and a row it writes reads back as the same configuration (through the HGEMM_TABLE file path)."""
    import subprocess
    import sys
    from paper_2512_02551_b200 import tune
    for (M, N, K) in [(64, 64, 64), (256, 64, 1024), (128, 12288, 4096), (4096, 4096, 4096), (12288, 256, 12288), (8192, 8192, 8192)]:
        cands = tune.candidates(M, N, K)
        assert cands and all(hgemm.validate_config(M, N, K, c) == hgemm.OK for c in cands), (M, N, K)
        assert len({tune.key(c) for c in cands}) == len(cands), "duplicates"
    small = tune.candidates(256, 64, 1024)
    assert {c.split_k for c in small if c.family == hgemm.FAMILY_SMALL} >= {1, 2, 4, 8, 16}
    skinny = tune.candidates(128, 12288, 4096)
    assert any(c.swap_ab for c in skinny) and any(c.family == hgemm.FAMILY_LIGHT for c in skinny)
    big = tune.candidates(8192, 8192, 8192)
    assert any(c.block_n == 512 for c in big) and any(c.epilogue == hgemm.EPILOGUE_TMA_WIDE for c in big)
    odd = tune.candidates(12288, 256, 12288)
    assert any(c.tail_mode == hgemm.TAIL_STREAM and c.tail_split >= 2 for c in odd)
    # a row written by the tuner, read back by the library in a child process
    cfg = hgemm.Config.make(family=1, block_n=256, stages=6, raster_group=9, epilogue=hgemm.EPILOGUE_TMA, tail_split=2, tail_mode=hgemm.TAIL_STREAM)
    cfg2 = hgemm.Config.make(family=1, block_n=512, stages=4, raster_group=12, epilogue=hgemm.EPILOGUE_TMA, raster_mode=1, wave_pace=1)
    cfg3 = hgemm.Config.small(32, 8)
    rows = [{"M": 12288, "N": 256, "K": 12288, "best": cfg.as_dict(), "us": 75.9, "ok": True},
            {"M": 8192, "N": 8192, "K": 8192, "best": cfg2.as_dict(), "us": 700.0, "ok": True},
            {"M": 256, "N": 64, "K": 1024, "best": cfg3.as_dict(), "us": 3.3, "ok": True},
            {"M": 64, "N": 64, "K": 64, "best": cfg3.as_dict(), "us": 1.0, "ok": False}]          # a failed check is not written
    path = tmp_path / "table.inc"
    tune.write_table(rows, str(path))
    text = path.read_text()
    assert text.count("\n{") == 3 and "{64, 64, 64," not in text
    tune.merge_table([{"M": 256, "N": 64, "K": 1024, "best": hgemm.Config.small(64, 4).as_dict(), "us": 3.0, "ok": True}], str(path))
    code = ("from paper_2512_02551_b200 import hgemm\n"
            "for s in ((12288, 256, 12288), (8192, 8192, 8192), (256, 64, 1024)):\n"
            "    c = hgemm.planned_config(*s)\n"
            "    print(c.family, c.block_n, c.stages, c.split_k, c.split_mode, c.tail_split, c.tail_mode, c.raster_group, c.raster_mode, c.wave_pace)")
    out = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, HGEMM_TABLE=str(path), PYTHONPATH=ROOT), capture_output=True, text=True,
                         check=True).stdout.strip().split("\n")
    assert out[0].split() == ["1", "256", "6", "1", "0", "2", "2", "9", "0", "0"]
    assert out[1].split() == ["1", "512", "4", "1", "0", "0", "0", "12", "1", "1"]
    assert out[2].split() == ["3", "64", "3", "4", "1", "0", "0", "1", "0", "0"]             # the merged row replaced the first one
