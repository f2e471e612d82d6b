"""Per-shape tuner: times candidate configurations on the GPU and writes the planner's table.

    python -m paper_2512_02551_b200.tune [--out DIR] [--shapes MxNxK ...] [--grid10] [--top 20] [--resume]
                                         [--time-limit SECONDS] [--merge-into csrc/hgemm_table.inc]

For every shape of the 9 x 9 x 9 grid (with --grid10: the 271 shapes that the paper's tenth grid value,
16384, adds; or the shapes given) it ranks the legal configurations with
the planner's cost model, times the best `--top` of them plus the heuristic's own choice, checks
the winner against torch.matmul, and writes
  DIR/tune.jsonl        one line per shape (resumable with --resume)
  DIR/hgemm_table.inc   the table to copy over csrc/hgemm_table.inc before rebuilding the library.
The protocol follows the library auto-tuning baseline the paper compares against (appendix
Listing 8): warm-up, then timed rounds in shuffled order, median per candidate.
"""
from __future__ import annotations

import argparse
import functools
import json
import os
import random
import statistics

import torch

from . import hgemm, inputs

GRID = [64, 128, 256, 512, 1024, 2048, 4096, 8192, 12288]
SPLITS = [1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64]
NUM_SMS = 148


@functools.lru_cache(maxsize=None)
def max_stages(family: int, bn: int, bk: int, epilogue: int = hgemm.EPILOGUE_TMA) -> int:
    best = 0
    for st in range(1, 13):
        c = hgemm.Config.make(family=family, block_n=bn, stages=st, block_k=bk, epilogue=epilogue)
        if hgemm.config_smem_bytes(c) <= 232448:
            best = st
    return best


def candidates(M: int, N: int, K: int):
    out = []
    for tile in (64, 32):                                         # the register-accumulator kernel: two tiles, K slices in a cluster
        for split in (1, 2, 4, 8, 16):
            small = hgemm.Config.small(tile, split)
            if hgemm.validate_config(M, N, K, small) == hgemm.OK and M * N * K <= (1 << 31) and \
                    -(-M // tile) * -(-N // tile) * split <= 8 * NUM_SMS:
                out.append(small)
    for swap in (0, 1):
        if swap and not (M <= 256 and N >= 512 and N % 8 == 0):
            continue
        out += _candidates(M, N, K, swap)
    return out


def _candidates(M: int, N: int, K: int, swap: int):
    """The configurations of one orientation; with swap = 1 the kernel tiles the transposed problem."""
    out = []
    Mk, Nk = (N, M) if swap else (M, N)
    for family in (0, 1, 2):
        light = family == hgemm.FAMILY_LIGHT
        if light and (swap or K % 8 or N % 8):
            continue
        cg = 2 if family == 1 else 1
        units = NUM_SMS // cg
        widths = list(range(32, 257, 32)) + ([512] if family == 1 and not swap and Nk % 512 == 0 else [])   # 512: the double tile
        for bn in widths:
            if bn > 32 and bn - 32 >= Nk:
                break
            tiles = -(-Mk // (128 * cg)) * -(-Nk // bn)
            for bk in (64, 128):
                if bk == 128 and (K < 128 or bn == 512):
                    continue
                st = min(max_stages(family, bn, bk), 8)
                if st < 1:
                    continue
                for split in SPLITS:
                    if split > -(-K // bk):
                        break
                    if split > 1 and (light or tiles * split > 2 * units):
                        continue
                    rg = max(1, min(-(-Mk // (128 * cg)), round((units * bn / (128.0 * cg)) ** 0.5)))
                    modes = (0,) if split == 1 else ((0, 1) if split * cg <= 16 else (0,))
                    for mode in modes:
                        epis = (hgemm.EPILOGUE_DIRECT,)
                        if split == 1:
                            epis = (hgemm.EPILOGUE_TMA, hgemm.EPILOGUE_DIRECT) + ((hgemm.EPILOGUE_TMA_WIDE,) if bn % 64 == 0 and not swap else ())
                        if light:
                            epis = (hgemm.EPILOGUE_DIRECT, hgemm.EPILOGUE_TMA)
                        for epi in epis:
                            st = min(max_stages(family, bn, bk, epi), 8)      # the wide epilogue's staging leaves fewer stages
                            if light:
                                st = min(max_stages(family, bn, bk, epi), -(-K // bk))      # no more stages than k-blocks
                            if st < 1:
                                continue
                            c = hgemm.Config.make(family=family, block_n=bn, stages=st, split_k=split, raster_group=rg,
                                                  epilogue=epi, block_k=bk, split_mode=mode, swap_ab=swap)
                            if hgemm.validate_config(M, N, K, c) == hgemm.OK:
                                out.append(c)
                            if swap or light:
                                continue                      # no tail cuts in the swapped orientation or the light kernel
                            if split == 1 and epi != hgemm.EPILOGUE_TMA_WIDE and tiles % units:
                                # stream-K: the tiles beyond the full waves (all of them when there are fewer tiles than SMs)
                                # as one sequence of k-blocks in equal shares, each tile cut into about `pieces` pieces
                                seen_units = set()
                                for pieces in (2, 4, 8):
                                    c4 = hgemm.Config.make(family=family, block_n=bn, stages=st, split_k=1, raster_group=rg, epilogue=epi,
                                                           block_k=bk, tail_split=pieces, tail_mode=hgemm.TAIL_STREAM)
                                    if hgemm.validate_config(M, N, K, c4) != hgemm.OK:
                                        continue
                                    item = hgemm.stream_item(M, N, K, c4, 0, 0, NUM_SMS)
                                    if item is not None and item[5] not in seen_units:      # (more pieces, same number of positions: the same schedule)
                                        seen_units.add(item[5])
                                        out.append(c4)
                            tail = tiles % units
                            if split == 1 and tiles > units and 0 < tail <= units // 2:
                                ts = min(units // tail, 8, -(-K // bk))
                                if ts >= 2:
                                    c2 = hgemm.Config.make(family=family, block_n=bn, stages=st, split_k=1, raster_group=rg,
                                                           epilogue=epi, block_k=bk, split_mode=0, tail_split=ts)
                                    if hgemm.validate_config(M, N, K, c2) == hgemm.OK:
                                        out.append(c2)
                            if split == 1 and tiles > units and 0 < tail <= units // 2:
                                # the last wave's tiles as 2 or 4 independent column pieces
                                for pieces in (2, 4):
                                    if tail * pieces <= units and bn % (32 * pieces) == 0:
                                        c3 = hgemm.Config.make(family=family, block_n=bn, stages=st, split_k=1, raster_group=rg,
                                                               epilogue=epi, block_k=bk, split_mode=0, tail_split=pieces,
                                                               tail_mode=hgemm.TAIL_N)
                                        if hgemm.validate_config(M, N, K, c3) == hgemm.OK:
                                            out.append(c3)
    return out


def batch_ms(fn, n: int, stream) -> float:
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(n):
        fn()
    e1.record(stream)
    e1.synchronize()
    return e0.elapsed_time(e1) / n


def ctypes_copy(dst: hgemm.Config, src: hgemm.Config) -> None:
    import ctypes
    ctypes.memmove(ctypes.byref(dst), ctypes.byref(src), ctypes.sizeof(hgemm.Config))


def key(c: hgemm.Config):
    d = c.as_dict()
    return tuple(d[k] for k in ("family", "block_n", "block_k", "stages", "split_k", "split_mode", "tail_split", "tail_mode", "raster_group", "epilogue",
                                "swap_ab", "raster_mode", "wave_pace"))


def device_times(plan, configs, run, reps: int = 5) -> dict:
    """GPU-side duration (microseconds, median of `reps` isolated calls) of each configuration, from the profiler's
    kernel records: what a call costs on the device when nothing overlaps it, without the host path."""
    from torch.profiler import ProfilerActivity, profile, record_function
    usable = []
    for c in configs:
        if plan.try_set_config(c) == hgemm.OK:
            run()
            usable.append(c)
    torch.cuda.synchronize()
    with profile(activities=[ProfilerActivity.CPU, ProfilerActivity.CUDA]) as prof:
        for i, c in enumerate(usable):
            plan.set_config(c)
            run()
            torch.cuda.synchronize()
            for r in range(reps):
                with record_function(f"hgemm_tune_{i}_{r}"):
                    run()
                torch.cuda.synchronize()
    samples = {}
    for ev in prof.events():
        if ev.name.startswith("hgemm_tune_") and ev.device_type == torch.autograd.DeviceType.CUDA:
            i = int(ev.name.split("_")[2])
            samples.setdefault(i, []).append(ev.time_range.end - ev.time_range.start)
    return {key(usable[i]): statistics.median(v) for i, v in samples.items() if v}


def tune_shape(ctx, M, N, K, A_all, B_all, C_all, top: int, rng: random.Random, stream, explore: int = 0,
               device_metric: bool = False, only_specials: bool = False) -> dict:
    A = A_all.view(-1)[:M * K].view(M, K)
    B = B_all.view(-1)[:N * K].view(N, K)
    C = C_all[:M * N].view(M, N)
    plan = ctx.plan(M, N, K)
    default = plan.config
    cands = candidates(M, N, K)
    cands.sort(key=lambda c: hgemm.estimate_config(M, N, K, c))
    # the wide-store candidates are ranked on their own (8 of them), so that they take no place among the `top`
    wide = [c for c in cands if c.epilogue == hgemm.EPILOGUE_TMA_WIDE][:8]
    # so are the double-accumulator tiles and the light kernel's configurations, which the cost model was not fitted on
    wide += [c for c in cands if c.block_n == 512 and c.epilogue != hgemm.EPILOGUE_TMA_WIDE][:4]
    wide += [c for c in cands if c.family == hgemm.FAMILY_LIGHT][:8]
    wide += [c for c in cands if c.family == hgemm.FAMILY_SMALL]
    is_stream = lambda c: c.tail_mode == hgemm.TAIL_STREAM and c.tail_split >= 2   # noqa: E731
    wide += [c for c in cands if is_stream(c)][:12]
    cands = [c for c in cands if c.epilogue != hgemm.EPILOGUE_TMA_WIDE and c.block_n != 512 and c.family not in (hgemm.FAMILY_LIGHT, hgemm.FAMILY_SMALL)
             and not is_stream(c)]
    if only_specials:                          # a challenge run: the plan's current configuration against the separately ranked groups
        if not any(is_stream(c) for c in wide):
            plan.close()
            return None
        wide = [c for c in wide if is_stream(c)]
        cands = []
    chosen, seen = [], set()
    extra = rng.sample(cands[top:], min(explore, max(0, len(cands) - top))) if explore > 0 else []   # for refitting the cost model
    for c in [default] + cands[:top] + wide + extra:
        if key(c) not in seen:
            seen.add(key(c))
            chosen.append(c)
    a, b, cptr, s = A.data_ptr(), B.data_ptr(), C.data_ptr(), stream.cuda_stream
    run = lambda: plan.run_ptr(a, b, cptr, s)   # noqa: E731
    results = []
    for c in chosen:
        if plan.try_set_config(c) != hgemm.OK:
            continue
        for _ in range(3):
            run()
        est = max(batch_ms(run, 3, stream), 1e-3)
        n = max(3, min(100, int(0.6 / est)))
        times = [batch_ms(run, n, stream) for _ in range(3)]
        results.append((statistics.median(times), hgemm.estimate_config(M, N, K, c), c))
    st, code = ctx.last_device_status()
    if st != hgemm.OK:
        raise RuntimeError(f"device status {st} code {code:#x} while tuning {M}x{N}x{K}")
    # re-time the five fastest in shuffled order and keep the median of medians
    results.sort(key=lambda r: (round(r[0] * 1e3 / 0.25), r[1]))   # ties within 0.25 us: lower estimate first
    finalists = results[:5]
    if only_specials and not any(key(c) == key(default) for _, _, c in finalists):
        finalists += [r for r in results if key(r[2]) == key(default)]      # a challenge run always re-times the configuration in use
    again = {key(c): [t] for t, _, c in finalists}
    for _ in range(2):
        order = list(finalists)
        rng.shuffle(order)
        for t, _, c in order:
            plan.set_config(c)
            run()
            n = max(3, min(100, int(0.6 / max(t, 1e-3))))
            again[key(c)].append(batch_ms(run, n, stream))
    final = sorted(((statistics.median(again[key(c)]), e, c) for _, e, c in finalists),
                   key=lambda r: (round(r[0] * 1e3 / 0.25), r[1]))
    if final[0][0] > 0.08:
        # long kernels run under the power cap when called back to back: rank the finalists by a
        # sustained run (about a quarter of a second each, shuffled order) instead of by short bursts
        sustained = {}
        order = list(final)
        rng.shuffle(order)
        for t, e, c in order:
            plan.set_config(c)
            n = max(5, min(2000, int(0.25 / (t * 1e-3))))      # calls that fill about 0.25 s
            for _ in range(3):
                run()
            sustained[key(c)] = batch_ms(run, n, stream)
        final = sorted(((sustained[key(c)], e, c) for _, e, c in final), key=lambda r: r[0])
    best_t, _, best = final[0]
    default_final = next((t for t, _, c in final if key(c) == key(default)), None)   # timed like the winner (None: not a finalist)
    cold_us = None
    L2 = 126 << 20
    foot = 2 * (M * K + N * K + M * N)
    sets = min(-(-2 * L2 // foot), A_all.numel() // max(M * K, 1), B_all.numel() // max(N * K, 1), C_all.numel() // max(M * N, 1))
    if 0.008 <= best_t <= 0.08 and sets >= 2 and sets * foot >= 2 * L2:
        # Mid-size kernels whose operands fit in L2 run in two regimes: back to back on the same buffers (everything
        # above was timed like that), or with operands that come from HBM -- a call between other work.  Among the
        # finalists within 3 % of the best warm time, take the one with the best geometric mean of the warm time and the
        # cold time (buffer sets rotating through more than twice the L2): deeper rings win there at no warm cost.
        ptrs = [(A_all[r * M * K:].data_ptr(), B_all[r * N * K:].data_ptr(), C_all[r * M * N:].data_ptr()) for r in range(sets)]

        def cold_ms(n):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(n):
                pa, pb, pc = ptrs[i % sets]
                plan.run_ptr(pa, pb, pc, s)
            e1.record(stream)
            e1.synchronize()
            return e0.elapsed_time(e1) / n
        scored = []
        for t, e, c in final:
            if t > 1.03 * best_t:
                continue
            plan.set_config(c)
            cold_ms(sets)                                           # tensor maps of every set encoded
            n = max(sets, min(200, int(0.6 / max(t, 1e-3))))
            tc = statistics.median(cold_ms(n) for _ in range(3))
            scored.append(((t * tc) ** 0.5, t, tc, e, c))
        if scored:
            scored.sort(key=lambda r: r[0])
            _, best_t, tc, _, best = scored[0]
            cold_us = tc * 1e3
    dev_us = None
    if device_metric and best_t < 0.008:
        # Short kernels: back-to-back calls overlap one call's start with the previous call's end and are bounded by
        # the host's launch rate, so many configurations tie.  Among those that tie (within 3 % + 0.1 us of the best),
        # take the one whose kernel is shortest on the device when it runs alone -- what a single call after an idle
        # gap, or a call between other kernels, pays.
        b2b = {key(c): t for t, _, c in results}
        for t, _, c in final:
            b2b[key(c)] = min(b2b.get(key(c), t), t)
        ranked = sorted(results, key=lambda r: r[0])
        pool, seen_k = [], set()
        for t, _, c in ranked[:10] + [r for r in ranked if r[2].family == hgemm.FAMILY_LIGHT][:6] + [r for r in ranked if r[2].family == hgemm.FAMILY_SMALL]:
            if key(c) not in seen_k:
                seen_k.add(key(c))
                pool.append(c)
        try:
            dev = device_times(plan, pool, run)
        except Exception:                                     # no profiler: keep the back-to-back winner
            dev = {}
        allowed = [c for c in pool if key(c) in dev and b2b[key(c)] <= 1.03 * best_t + 1e-4]
        if allowed:
            pick = min(allowed, key=lambda c: dev[key(c)])
            if key(best) not in dev or dev[key(pick)] < 0.98 * dev[key(best)]:
                best, best_t = pick, b2b[key(pick)]
            dev_us = dev.get(key(best))
    # The tile order of the winner: the candidates above all carry the raster group of a square-ish wave; with more
    # tiles than SMs other groups, and the serpentine sweep, change what stays in L2 between waves.  Timed the same
    # way as the finalists (sustained for long kernels), the winner's own order included again.
    cg = best.family + 1
    tiles_m = -(-(N if best.swap_ab else M) // (128 * cg))
    tiles_n = -(-(M if best.swap_ab else N) // best.block_n)
    if tiles_m > 1 and tiles_n > 1 and tiles_m * tiles_n > NUM_SMS // cg and best.split_k == 1:
        sustained = best_t > 0.08
        orders = {(best.raster_group, best.raster_mode)}
        for rg in (1, 2, 4, 8, 16, tiles_m):
            for rm in (hgemm.RASTER_SWEEP, hgemm.RASTER_SERPENTINE):
                orders.add((min(rg, tiles_m), rm))
        timed = []
        order_list = sorted(orders)
        rng.shuffle(order_list)
        for rg, rm in order_list:
            c = hgemm.Config()
            ctypes_copy(c, best)
            c.raster_group, c.raster_mode = rg, rm
            if plan.try_set_config(c) != hgemm.OK:
                continue
            for _ in range(3):
                run()
            n = max(5, min(2000, int(0.25 / (best_t * 1e-3)))) if sustained else max(3, min(100, int(0.6 / max(best_t, 1e-3))))
            t = batch_ms(run, n, stream) if sustained else statistics.median(batch_ms(run, n, stream) for _ in range(3))
            timed.append((t, c))
        timed.sort(key=lambda r: r[0])
        if timed and timed[0][0] < 0.995 * min(t for t, c in timed if (c.raster_group, c.raster_mode) == (best.raster_group, best.raster_mode)):
            best_t, best = timed[0]
    plan.set_config(best)
    C.zero_()
    run()
    # the winner must meet the library's own acceptance formula, |C - C_ref| <= 2^-10 |C_ref| + 1e-3 sqrt(K), here
    # against an fp32 product of the same operands (the tuner is product code and may not use the test oracle)
    ref32 = torch.matmul(A.float(), B.float().T) if M * N <= (1 << 26) else None
    if ref32 is not None:
        ok = bool(((C.float() - ref32).abs() <= 2.0 ** -10 * ref32.abs() + 1e-3 * K ** 0.5).all())
    else:                                                   # large outputs: the first and last 2048 rows
        ok = True
        rows = max(1, min(M, (1 << 26) // N))
        for r0 in (0, M - rows):
            r32 = torch.matmul(A[r0:r0 + rows].float(), B.float().T)
            ok = ok and bool(((C[r0:r0 + rows].float() - r32).abs() <= 2.0 ** -10 * r32.abs() + 1e-3 * K ** 0.5).all())
    ref = torch.empty_like(C)
    n_ref = max(5, min(2000, int(0.25 / (best_t * 1e-3)))) if best_t > 0.08 else max(3, min(100, int(0.6 / max(best_t, 1e-3))))
    t_torch = statistics.median(batch_ms(lambda: torch.matmul(A, B.T, out=ref), n_ref, stream)
                                for _ in range(1 if best_t > 0.08 else 3))
    default_t = next((t for t, _, c in results if key(c) == key(default)), None)
    plan.close()
    return {"M": M, "N": N, "K": K, "best": best.as_dict(), "us": best_t * 1e3, "default_us": None if default_t is None else default_t * 1e3,
            "torch_us": t_torch * 1e3, "ok": ok, "tried": len(results), "dev_us": dev_us, "cold_us": cold_us,
            "default_final_us": None if default_final is None else default_final * 1e3,
            "all": [list(key(c)) + [round(t * 1e3, 3)] for t, _, c in results]}   # every first-pass timing: key fields, us


def challenge_pace(ctx, M, N, K, A_all, B_all, C_all, rng: random.Random, stream):
    """The plan's configuration with and without wave pacing, timed alternately in sustained runs (about a quarter of a second
    each, three rounds); returns a row like tune_shape's with pacing switched on if it is at least 0.5 % faster, else None."""
    A = A_all.view(-1)[:M * K].view(M, K)
    B = B_all.view(-1)[:N * K].view(N, K)
    C = C_all[:M * N].view(M, N)
    plan = ctx.plan(M, N, K)
    base = plan.config
    paced = hgemm.Config()
    ctypes_copy(paced, base)
    paced.wave_pace = 1
    if base.wave_pace or hgemm.validate_config(M, N, K, paced) != hgemm.OK:
        plan.close()
        return None
    cg = 2 if base.family == hgemm.FAMILY_UMMA_2CTA else 1
    tiles = -(-M // (128 * cg)) * -(-N // base.block_n)
    if tiles <= NUM_SMS // cg:                               # one tile per CTA: nothing to pace
        plan.close()
        return None
    a, b, cptr, s = A.data_ptr(), B.data_ptr(), C.data_ptr(), stream.cuda_stream
    run = lambda: plan.run_ptr(a, b, cptr, s)   # noqa: E731
    times = {0: [], 1: []}
    plan.set_config(base)
    for _ in range(3):
        run()
    est = max(batch_ms(run, 3, stream), 1e-3)
    n = max(5, min(2000, int(250.0 / est)))
    for _ in range(3):
        order = [(0, base), (1, paced)]
        rng.shuffle(order)
        for which, cfg in order:
            plan.set_config(cfg)
            run()
            times[which].append(batch_ms(run, n, stream))
    st, code = ctx.last_device_status()
    plan.close()
    if st != hgemm.OK:
        raise RuntimeError(f"device status {st} code {code:#x} while timing {M}x{N}x{K}")
    t0, t1 = statistics.median(times[0]), statistics.median(times[1])
    if t1 > 0.995 * t0:
        return None
    return {"M": M, "N": N, "K": K, "best": paced.as_dict(), "us": t1 * 1e3, "default_us": t0 * 1e3, "default_final_us": t0 * 1e3, "torch_us": t0 * 1e3,
            "ok": True, "tried": 2, "dev_us": None, "cold_us": None, "all": []}


def write_table(rows, path):
    with open(path, "w") as f:
        f.write("// Tuned per-shape configurations for B200, written by tune.py on the GPU box.\n")
        f.write("// {M, N, K, family, block_n, block_k, stages, split_k, split_mode, tail_split, raster_group, epilogue, tail_mode, measured us, swap_ab, raster_mode, wave_pace}\n")
        for r in rows:
            if not r["ok"]:
                continue
            b = r["best"]
            f.write(f"{{{r['M']}, {r['N']}, {r['K']}, {b['family']}, {b['block_n']}, {b['block_k']}, {b['stages']}, "
                    f"{b['split_k']}, {b['split_mode']}, {b.get('tail_split', 0)}, {b['raster_group']}, {b['epilogue']}, {b.get('tail_mode', 0)}, {r['us']:.2f}f, "
                    f"{b.get('swap_ab', 0)}, {b.get('raster_mode', 0)}, {b.get('wave_pace', 0)}}},\n")


def merge_table(new_rows, path):
    """Rewrites the table at `path`: rows of shapes in `new_rows` are replaced, every other row is kept."""
    import re
    fresh = {(r["M"], r["N"], r["K"]): r for r in new_rows if r["ok"]}
    kept, header = [], []
    if os.path.exists(path):
        for line in open(path):
            m = re.match(r"\{(\d+), (\d+), (\d+),", line)
            if m is None:
                if line.startswith("//"):
                    header.append(line)
                continue
            if tuple(int(v) for v in m.groups()) not in fresh:
                kept.append(line)
    tmp = path + ".new"
    write_table(list(fresh.values()), tmp)
    body = [line for line in open(tmp) if not line.startswith("//")]
    head = [line for line in open(tmp) if line.startswith("//")]
    os.remove(tmp)

    def shape_key(line):
        return tuple(int(v) for v in re.match(r"\{(\d+), (\d+), (\d+),", line).groups())
    with open(path, "w") as f:
        f.writelines(head)
        f.writelines(sorted(kept + body, key=shape_key))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="tune_out", help="directory for tune.jsonl and hgemm_table.inc")
    ap.add_argument("--shapes", nargs="*")
    ap.add_argument("--top", type=int, default=20)
    ap.add_argument("--resume", action="store_true")
    ap.add_argument("--explore", type=int, default=0, help="also time this many randomly drawn candidates per shape")
    ap.add_argument("--device-metric", action="store_true",
                    help="for kernels under 8 us: among the configurations that tie back to back, pick the shortest on the device")
    ap.add_argument("--max-us", type=float, default=0.0, help="with --resume-from: only shapes whose recorded time is below this")
    ap.add_argument("--from-log", metavar="JSONL", help="take the shape list (and --max-us times) from an earlier tune.jsonl")
    ap.add_argument("--challenge-stream", action="store_true",
                    help="time only the plan's current configuration against the stream-K candidates (shapes without any are skipped)")
    ap.add_argument("--challenge-pace", action="store_true",
                    help="time only the plan's current configuration with and without wave pacing; rows only where pacing wins")
    ap.add_argument("--min-us", type=float, default=0.0, help="with --from-log: only shapes whose recorded time is at least this")
    ap.add_argument("--grid10", action="store_true", help="the 271 shapes of the ten-value grid that contain 16384")
    ap.add_argument("--time-limit", type=float, default=0.0, help="stop starting new shapes after this many seconds (resume later)")
    ap.add_argument("--merge-into", metavar="TABLE", help="replace these shapes' rows in an existing table file, keep its other rows")
    args = ap.parse_args()
    os.makedirs(args.out, exist_ok=True)
    if args.shapes:
        shapes = [tuple(int(v) for v in s.lower().split("x")) for s in args.shapes]
    elif args.grid10:
        g10 = GRID + [16384]
        shapes = [(M, N, K) for M in g10 for N in g10 for K in g10 if 16384 in (M, N, K)]
    else:
        shapes = [(M, N, K) for M in GRID for N in GRID for K in GRID]
    if args.from_log:
        earlier = [json.loads(line) for line in open(args.from_log)]
        shapes = [(r["M"], r["N"], r["K"]) for r in earlier if (args.max_us <= 0 or r["us"] < args.max_us) and r["us"] >= args.min_us]
    log_path = os.path.join(args.out, "tune.jsonl")
    done = {}
    if args.resume and os.path.exists(log_path):
        for line in open(log_path):
            r = json.loads(line)
            done[(r["M"], r["N"], r["K"])] = r
    mx_mk = max(max(M * K, N * K) for M, N, K in shapes)
    mx_mn = max(M * N for M, N, K in shapes)
    stream = torch.cuda.current_stream()
    # pools: the largest operand of the run, plus room for the rotating buffer sets of the cold-regime timing (> 2x L2)
    room = 132 << 20
    cols = 4096
    A_all = inputs.draw(1, inputs.TAG_A, -(-(mx_mk + room) // cols), cols, "uniform", "cuda").view(-1)
    B_all = inputs.draw(1, inputs.TAG_B, -(-(mx_mk + room) // cols), cols, "uniform", "cuda").view(-1)
    C_all = torch.empty(mx_mn + room, dtype=torch.float16, device="cuda")
    rng = random.Random(2512)
    rows = []
    import time
    started = time.time()
    with hgemm.Context(0) as ctx, open(log_path, "a" if args.resume else "w") as log:
        for (M, N, K) in shapes:
            r = done.get((M, N, K))
            if r is None:
                if args.time_limit > 0 and time.time() - started > args.time_limit:
                    continue                                   # out of time: left for a later --resume run
                if args.challenge_pace:
                    r = challenge_pace(ctx, M, N, K, A_all, B_all, C_all, rng, stream)
                else:
                    r = tune_shape(ctx, M, N, K, A_all, B_all, C_all, args.top, rng, stream, args.explore, args.device_metric, args.challenge_stream)
                if r is None:                                  # a challenge run on a shape without challengers
                    continue
                log.write(json.dumps(r) + "\n")
                log.flush()
            rows.append(r)
    write_table(rows, os.path.join(args.out, "hgemm_table.inc"))
    if args.merge_into:
        merge_table(rows, args.merge_into)
    import math
    g = math.exp(sum(math.log(r["torch_us"] / r["us"]) for r in rows) / len(rows)) if rows else float("nan")
    bad = [r for r in rows if not r["ok"]]
    what = "geomean time without / with pacing" if args.challenge_pace else "geomean torch/ours"
    print(f"tuned {len(rows)} shapes; {what} = {g:.3f}; failed checks: {len(bad)}")


if __name__ == "__main__":
    main()
