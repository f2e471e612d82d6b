"""Run one HGEMM shape a few times through the C ABI and print its device time.

    python -m paper_2512_02551_b200.run_case 8192x8192x8192 [--iters 3] [--warmup 2]
        [--family 0|1|2|3 --block-n 256 --block-k 64|128 --stages 4 --split-k 1 --split-mode 0|1 --raster 8
         --raster-mode 0|1 --epilogue 0|1|2 --swap-ab 0|1 --tail-split 2 --tail-mode 0|1|2]

Small enough to sit under a profiler: it draws the inputs, plans, warms up and launches
`iters` times.  Without the configuration flags the library's own plan is used; with --family the
configuration starts from a plain one of that family and the other flags refine it.
"""
from __future__ import annotations

import argparse

import torch

from . import hgemm, inputs


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("shape", help="MxNxK")
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=2)
    ap.add_argument("--family", type=int)
    ap.add_argument("--block-n", type=int)
    ap.add_argument("--stages", type=int)
    ap.add_argument("--split-k", type=int)
    ap.add_argument("--raster", type=int)
    ap.add_argument("--epilogue", type=int)
    ap.add_argument("--block-k", type=int)
    ap.add_argument("--split-mode", type=int)
    ap.add_argument("--raster-mode", type=int)
    ap.add_argument("--swap-ab", type=int)
    ap.add_argument("--tail-split", type=int)
    ap.add_argument("--tail-mode", type=int)
    args = ap.parse_args()
    M, N, K = (int(v) for v in args.shape.lower().split("x"))
    with hgemm.Context(0) as ctx:
        A, B = inputs.make_ab(M, N, K, "uniform", "cuda")
        C = torch.empty(M, N, dtype=torch.float16, device="cuda")
        plan = ctx.plan(M, N, K)
        cfg = plan.config
        if args.family is not None:
            # an explicit family starts from a clean configuration instead of the plan's own (whose other fields may not apply)
            cfg = hgemm.Config.small(split_k=args.split_k or 1) if args.family == hgemm.FAMILY_SMALL else hgemm.Config.make(
                family=args.family, block_n=128, stages=4, raster_group=1, epilogue=hgemm.EPILOGUE_TMA)
        for name, attr in (("family", "family"), ("block_n", "block_n"), ("stages", "stages"), ("split_k", "split_k"),
                           ("raster", "raster_group"), ("epilogue", "epilogue"), ("block_k", "block_k"), ("split_mode", "split_mode"),
                           ("raster_mode", "raster_mode"), ("swap_ab", "swap_ab"), ("tail_split", "tail_split"), ("tail_mode", "tail_mode")):
            v = getattr(args, name)
            if v is not None:
                setattr(cfg, attr, v)
        cfg.block_m = 256 if cfg.family == hgemm.FAMILY_UMMA_2CTA else cfg.block_n if cfg.family == hgemm.FAMILY_SMALL else 128
        plan.set_config(cfg)
        for _ in range(args.warmup):
            plan.run(A, B, C)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.iters):
            plan.run(A, B, C)
        e1.record()
        torch.cuda.synchronize()
        st, code = ctx.last_device_status()
        ms = e0.elapsed_time(e1) / max(args.iters, 1)
        print(f"{M}x{N}x{K} {plan.config.as_dict()} status={st} {ms * 1e3:.1f} us/call "
              f"{2.0 * M * N * K / (ms * 1e-3) / 1e12:.1f} TFLOP/s")
        plan.close()


if __name__ == "__main__":
    main()
