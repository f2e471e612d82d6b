"""Thin ctypes binding of ``libhgemm.so`` (the C ABI declared in ``include/hgemm.h``).

Argument marshalling only: every step of the GEMM runs in the library's CUDA
kernels.  PyTorch appears here only as the owner of device memory and streams
(``tensor.data_ptr()``, ``torch.cuda.current_stream().cuda_stream``).  There is no
fallback: if the library is missing or a call fails, this module raises.
"""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("HGEMM_LIB") or os.path.join(HERE, "libhgemm.so")      # HGEMM_LIB: another build of the library (the checked one)

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALLOC, ERR_CUDA, ERR_ARCH, ERR_TIMEOUT, ERR_SCRATCH_LIMIT, ERR_CHECK = range(9)
FAMILY_UMMA_1CTA, FAMILY_UMMA_2CTA, FAMILY_LIGHT, FAMILY_SMALL = 0, 1, 2, 3
EPILOGUE_DIRECT, EPILOGUE_TMA, EPILOGUE_TMA_WIDE = 0, 1, 2
SPLIT_WORKSPACE, SPLIT_CLUSTER = 0, 1
TAIL_K, TAIL_N, TAIL_STREAM = 0, 1, 2
ACC_F32, ACC_F16 = 0, 1
LAYOUT_TN, LAYOUT_NN = 0, 1
RASTER_SWEEP, RASTER_SERPENTINE = 0, 1
STATIC_A, STATIC_B = 1, 2

# every symbol include/hgemm.h declares
EXPORTS = [
    "hgemm_create", "hgemm_destroy", "hgemm_plan", "hgemm_plan_layout", "hgemm_run", "hgemm_run_host", "hgemm_run_scaled", "hgemm_run_splitk_static", "hgemm_plan_destroy",
    "hgemm_plan_get_config", "hgemm_plan_set_config", "hgemm_plan_set_static_operands", "hgemm_plan_autotune", "hgemm_candidate_configs", "hgemm_heuristic_config", "hgemm_planned_config", "hgemm_validate_config", "hgemm_estimate_config",
    "hgemm_config_smem_bytes", "hgemm_config_workspace_bytes", "hgemm_plan_launches_per_run",
    "hgemm_last_device_status", "hgemm_ctx_last_device_status", "hgemm_debug_fail_allocs", "hgemm_set_wait_budget", "hgemm_set_dependent_launch", "hgemm_debug_timeout_probe", "hgemm_debug_check_probe", "hgemm_build_is_checked", "hgemm_debug_stream_item", "hgemm_debug_set_trace", "hgemm_debug_set_skip",
    "hgemm_last_cuda_error", "hgemm_status_string",
]


class HgemmError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (status {status})")


class Config(ctypes.Structure):
    """Mirror of ``hgemm_config_t``."""
    _fields_ = [("family", ctypes.c_int32), ("block_m", ctypes.c_int32), ("block_n", ctypes.c_int32),
                ("block_k", ctypes.c_int32), ("stages", ctypes.c_int32), ("split_k", ctypes.c_int32),
                ("raster_group", ctypes.c_int32), ("epilogue", ctypes.c_int32), ("split_mode", ctypes.c_int32),
                ("tail_split", ctypes.c_int32), ("tail_mode", ctypes.c_int32), ("accumulate", ctypes.c_int32),
                ("swap_ab", ctypes.c_int32), ("raster_mode", ctypes.c_int32), ("wave_pace", ctypes.c_int32),
                ("reserved", ctypes.c_int32 * 1)]

    @classmethod
    def small(cls, tile: int = 64, split_k: int = 1) -> "Config":
        """A configuration of the register-accumulator kernel for the smallest problems (tile = 64 or 32; split_k > 1:
        that many K slices per tile, summed inside a cluster)."""
        c = cls.make(family=FAMILY_SMALL, block_n=tile, stages=3, split_k=split_k, raster_group=1, epilogue=EPILOGUE_DIRECT, block_k=64,
                     split_mode=SPLIT_CLUSTER if split_k > 1 else SPLIT_WORKSPACE)
        c.block_m = tile
        return c

    def as_dict(self) -> dict:
        return {k: int(getattr(self, k)) for k, _ in self._fields_ if k != "reserved"}

    @classmethod
    def make(cls, family=FAMILY_UMMA_1CTA, block_n=128, stages=4, split_k=1, raster_group=8,
             epilogue=EPILOGUE_DIRECT, block_k=64, split_mode=0, tail_split=0, tail_mode=0, accumulate=0, swap_ab=0,
             raster_mode=0, wave_pace=0) -> "Config":
        c = cls()
        c.family = family
        c.block_m = 256 if family == FAMILY_UMMA_2CTA else 64 if family == FAMILY_SMALL else 128
        c.block_n = block_n
        c.block_k = block_k
        c.stages = stages
        c.split_k = split_k
        c.raster_group = raster_group
        c.epilogue = epilogue
        c.split_mode = split_mode
        c.tail_split = tail_split
        c.tail_mode = tail_mode
        c.accumulate = accumulate
        c.swap_ab = swap_ab
        c.raster_mode = raster_mode
        c.wave_pace = wave_pace
        return c


_lib = None


def lib() -> ctypes.CDLL:
    """Load the library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2512_02551_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        i32, i64, p = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
        cfgp = ctypes.POINTER(Config)
        sig = {
            "hgemm_create": (i32, [ctypes.POINTER(p), ctypes.c_int]),
            "hgemm_destroy": (i32, [p]),
            "hgemm_plan": (i32, [p, i64, i64, i64, ctypes.POINTER(p)]),
            "hgemm_plan_layout": (i32, [p, i64, i64, i64, i32, ctypes.POINTER(p)]),
            "hgemm_run": (i32, [p, p, p, p, p]),
            "hgemm_run_host": (i32, [p, p, p, p, p]),
            "hgemm_run_scaled": (i32, [p, ctypes.c_float, ctypes.c_float, p, p, p, p]),
            "hgemm_run_splitk_static": (i32, [i64, i64, i64, i32, i32, p, p, p, p]),
            "hgemm_plan_destroy": (i32, [p]),
            "hgemm_plan_get_config": (i32, [p, cfgp]),
            "hgemm_plan_set_config": (i32, [p, cfgp]),
            "hgemm_plan_set_static_operands": (i32, [p, ctypes.c_uint32]),
            "hgemm_plan_autotune": (i32, [p, p, p, p, p, i32, ctypes.POINTER(ctypes.c_float)]),
            "hgemm_heuristic_config": (i32, [i64, i64, i64, i32, cfgp]),
            "hgemm_candidate_configs": (i32, [i64, i64, i64, i32, cfgp, i32]),
            "hgemm_planned_config": (i32, [i64, i64, i64, i32, cfgp]),
            "hgemm_validate_config": (i32, [i64, i64, i64, cfgp]),
            "hgemm_estimate_config": (ctypes.c_double, [i64, i64, i64, i32, cfgp]),
            "hgemm_config_smem_bytes": (i64, [cfgp]),
            "hgemm_config_workspace_bytes": (i64, [i64, i64, i64, cfgp]),
            "hgemm_plan_launches_per_run": (i32, [p]),
            "hgemm_last_device_status": (i32, [p, ctypes.POINTER(ctypes.c_uint32)]),
            "hgemm_ctx_last_device_status": (i32, [p, ctypes.POINTER(ctypes.c_uint32)]),
            "hgemm_debug_fail_allocs": (i32, [p, i32, i32]),
            "hgemm_set_wait_budget": (i32, [p, i64]),
            "hgemm_set_dependent_launch": (i32, [p, i32]),
            "hgemm_debug_timeout_probe": (i32, [p, p]),
            "hgemm_debug_check_probe": (i32, [p, p]),
            "hgemm_build_is_checked": (i32, []),
            "hgemm_debug_stream_item": (i32, [i64, i64, i64, cfgp, i32, i32, i32, ctypes.POINTER(ctypes.c_int32)]),
            "hgemm_debug_set_trace": (i32, [p, p]),
            "hgemm_debug_set_skip": (i32, [p, ctypes.c_uint32]),
            "hgemm_last_cuda_error": (i32, [p]),
            "hgemm_status_string": (ctypes.c_char_p, [i32]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().hgemm_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != OK:
        raise HgemmError(status, what)


def heuristic_config(M: int, N: int, K: int, num_sms: int = 148) -> Config:
    c = Config()
    _check(lib().hgemm_heuristic_config(M, N, K, num_sms, ctypes.byref(c)), f"hgemm_heuristic_config({M},{N},{K})")
    return c


def planned_config(M: int, N: int, K: int, num_sms: int = 148) -> Config:
    c = Config()
    _check(lib().hgemm_planned_config(M, N, K, num_sms, ctypes.byref(c)), f"hgemm_planned_config({M},{N},{K})")
    return c


def candidate_configs(M: int, N: int, K: int, max_count: int = 64, num_sms: int = 148) -> list:
    """The configurations ``Plan.autotune`` draws from, best estimate first."""
    arr = (Config * max_count)()
    n = int(lib().hgemm_candidate_configs(M, N, K, num_sms, arr, max_count))
    out = []
    for i in range(n):
        c = Config()
        ctypes.memmove(ctypes.byref(c), ctypes.byref(arr[i]), ctypes.sizeof(Config))
        out.append(c)
    return out


def validate_config(M: int, N: int, K: int, cfg: Config) -> int:
    return int(lib().hgemm_validate_config(M, N, K, ctypes.byref(cfg)))


def build_is_checked() -> bool:
    """True when the loaded library is the checked build (``HGEMM_LIB`` names it)."""
    return bool(lib().hgemm_build_is_checked())


def stream_item(M: int, N: int, K: int, cfg: "Config", position: int, h: int, num_sms: int = 148):
    """Work item `h` of CTA position `position` of a stream-K tail, as the kernel decodes it:
    (tile, kb_begin, kb_count, slice, slices, positions), or None when the configuration has no such tail here."""
    out = (ctypes.c_int32 * 6)()
    st = lib().hgemm_debug_stream_item(M, N, K, ctypes.byref(cfg), num_sms, position, h, out)
    if st == ERR_UNSUPPORTED:
        return None
    _check(st, "hgemm_debug_stream_item")
    return tuple(out)


def estimate_config(M: int, N: int, K: int, cfg: Config, num_sms: int = 148) -> float:
    return float(lib().hgemm_estimate_config(M, N, K, num_sms, ctypes.byref(cfg)))


def config_smem_bytes(cfg: Config) -> int:
    return int(lib().hgemm_config_smem_bytes(ctypes.byref(cfg)))


def config_workspace_bytes(M: int, N: int, K: int, cfg: Config) -> int:
    return int(lib().hgemm_config_workspace_bytes(M, N, K, ctypes.byref(cfg)))


def run_splitk_static(M: int, N: int, K: int, block_n: int, split_k: int, a_ptr: int, b_ptr: int, c_ptr: int,
                      stream: int = 0) -> int:
    """``hgemm_run_splitk_static`` on raw device pointers: the split-K GEMM whose scratch memory is a
    static array inside the library, for callers that may not allocate.  Returns the status."""
    return int(lib().hgemm_run_splitk_static(M, N, K, block_n, split_k, a_ptr, b_ptr, c_ptr, stream))


class Context:
    """``hgemm_create`` / ``hgemm_destroy``."""

    def __init__(self, device: int = 0):
        self._h = ctypes.c_void_p()
        _check(lib().hgemm_create(ctypes.byref(self._h), int(device)), f"hgemm_create(device={device})")
        self.device = int(device)

    def plan(self, M: int, N: int, K: int, layout: int = LAYOUT_TN) -> "Plan":
        return Plan(self, M, N, K, layout)

    def set_wait_budget(self, cycles: int) -> None:
        _check(lib().hgemm_set_wait_budget(self._h, int(cycles)), "hgemm_set_wait_budget")

    def set_dependent_launch(self, enabled: bool) -> None:
        _check(lib().hgemm_set_dependent_launch(self._h, 1 if enabled else 0), "hgemm_set_dependent_launch")

    def last_device_status(self) -> tuple[int, int]:
        """``hgemm_ctx_last_device_status``: (status, code) over the context's own status word and those of
        all its live plans; synchronises the device."""
        code = ctypes.c_uint32(0)
        st = lib().hgemm_ctx_last_device_status(self._h, ctypes.byref(code))
        return int(st), int(code.value)

    def debug_fail_allocs(self, after: int, count: int) -> None:
        _check(lib().hgemm_debug_fail_allocs(self._h, int(after), int(count)), "hgemm_debug_fail_allocs")

    def debug_timeout_probe(self, stream: int = 0) -> None:
        _check(lib().hgemm_debug_timeout_probe(self._h, ctypes.c_void_p(stream)), "hgemm_debug_timeout_probe")

    def debug_check_probe(self, stream: int = 0) -> None:
        _check(lib().hgemm_debug_check_probe(self._h, ctypes.c_void_p(stream)), "hgemm_debug_check_probe")

    def last_cuda_error(self) -> int:
        return int(lib().hgemm_last_cuda_error(self._h))

    def close(self) -> None:
        if self._h:
            lib().hgemm_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


class Plan:
    """``hgemm_plan`` / ``hgemm_run`` / ``hgemm_plan_destroy``."""

    def __init__(self, ctx: Context, M: int, N: int, K: int, layout: int = LAYOUT_TN):
        self.ctx = ctx
        self.shape = (int(M), int(N), int(K))
        self.layout = int(layout)
        self._h = ctypes.c_void_p()
        _check(lib().hgemm_plan_layout(ctx._h, int(M), int(N), int(K), int(layout), ctypes.byref(self._h)),
               f"hgemm_plan_layout({M},{N},{K},layout={layout})")
        self._run = lib().hgemm_run

    @property
    def config(self) -> Config:
        c = Config()
        _check(lib().hgemm_plan_get_config(self._h, ctypes.byref(c)), "hgemm_plan_get_config")
        return c

    def set_config(self, cfg: Config) -> None:
        _check(lib().hgemm_plan_set_config(self._h, ctypes.byref(cfg)), f"hgemm_plan_set_config({cfg.as_dict()})")

    def set_static_operands(self, a: bool = False, b: bool = False) -> None:
        """``hgemm_plan_set_static_operands``: promise that no kernel ahead of a call in its stream writes A and/or B."""
        _check(lib().hgemm_plan_set_static_operands(self._h, (1 if a else 0) | (2 if b else 0)), "hgemm_plan_set_static_operands")

    def try_set_config(self, cfg: Config) -> int:
        return int(lib().hgemm_plan_set_config(self._h, ctypes.byref(cfg)))

    def last_device_status(self) -> tuple[int, int]:
        """``hgemm_last_device_status``: (status, code) of this plan's own status word; synchronises the device."""
        code = ctypes.c_uint32(0)
        st = lib().hgemm_last_device_status(self._h, ctypes.byref(code))
        return int(st), int(code.value)

    @property
    def launches_per_run(self) -> int:
        return int(lib().hgemm_plan_launches_per_run(self._h))

    def run_ptr(self, a_ptr: int, b_ptr: int, c_ptr: int, stream: int = 0) -> None:
        """``hgemm_run`` on raw device pointers and a raw ``cudaStream_t``."""
        st = self._run(self._h, a_ptr, b_ptr, c_ptr, stream)
        if st != OK:
            raise HgemmError(st, f"hgemm_run{self.shape}")

    def run(self, A, B, C, stream=None) -> None:
        """``hgemm_run`` on torch CUDA tensors: A (M,K), B (N,K) -- or (K,N) for an NN plan --, C (M,N),
        fp16, contiguous."""
        import torch
        M, N, K = self.shape
        b_shape = (K, N) if self.layout == LAYOUT_NN else (N, K)
        for t, shp, name in ((A, (M, K), "A"), (B, b_shape, "B"), (C, (M, N), "C")):
            if t.dtype != torch.float16 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != shp:
                raise ValueError(f"{name} must be a contiguous CUDA fp16 tensor of shape {shp}")
        s = torch.cuda.current_stream().cuda_stream if stream is None else int(stream)
        self.run_ptr(A.data_ptr(), B.data_ptr(), C.data_ptr(), s)

    def autotune(self, A, B, C, max_candidates: int = 24, stream=None) -> float:
        """``hgemm_plan_autotune``: times the plan's configuration and up to ``max_candidates`` others on these
        tensors, installs the fastest (C then holds A B^T) and returns its time per call in microseconds."""
        import torch
        M, N, K = self.shape
        b_shape = (K, N) if self.layout == LAYOUT_NN else (N, K)
        for t, shp, name in ((A, (M, K), "A"), (B, b_shape, "B"), (C, (M, N), "C")):
            if t.dtype != torch.float16 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != shp:
                raise ValueError(f"{name} must be a contiguous CUDA fp16 tensor of shape {shp}")
        s = torch.cuda.current_stream().cuda_stream if stream is None else int(stream)
        us = ctypes.c_float(0.0)
        _check(lib().hgemm_plan_autotune(self._h, A.data_ptr(), B.data_ptr(), C.data_ptr(), s, int(max_candidates), ctypes.byref(us)),
               f"hgemm_plan_autotune{self.shape}")
        return float(us.value)

    def run_scaled(self, alpha: float, beta: float, A, B, C, stream=None) -> None:
        """``hgemm_run_scaled``: C = alpha * A B^T + beta * C in place, on torch CUDA tensors as for ``run``."""
        import torch
        M, N, K = self.shape
        b_shape = (K, N) if self.layout == LAYOUT_NN else (N, K)
        for t, shp, name in ((A, (M, K), "A"), (B, b_shape, "B"), (C, (M, N), "C")):
            if t.dtype != torch.float16 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != shp:
                raise ValueError(f"{name} must be a contiguous CUDA fp16 tensor of shape {shp}")
        s = torch.cuda.current_stream().cuda_stream if stream is None else int(stream)
        st = lib().hgemm_run_scaled(self._h, float(alpha), float(beta), A.data_ptr(), B.data_ptr(), C.data_ptr(), s)
        if st != OK:
            raise HgemmError(st, f"hgemm_run_scaled{self.shape}")

    def set_trace(self, device_ptr: int) -> None:
        _check(lib().hgemm_debug_set_trace(self._h, ctypes.c_void_p(device_ptr)), "hgemm_debug_set_trace")

    def set_skip(self, mask: int) -> None:
        _check(lib().hgemm_debug_set_skip(self._h, int(mask)), "hgemm_debug_set_skip")

    def run_host(self, A, B, C, stream=None) -> None:
        """``hgemm_run_host`` on torch CPU tensors (pinned for an asynchronous call)."""
        import torch
        M, N, K = self.shape
        for t, shp, name in ((A, (M, K), "A"), (B, (N, K), "B"), (C, (M, N), "C")):
            if t.dtype != torch.float16 or t.is_cuda or not t.is_contiguous() or tuple(t.shape) != shp:
                raise ValueError(f"{name} must be a contiguous host fp16 tensor of shape {shp}")
        s = torch.cuda.current_stream().cuda_stream if stream is None else int(stream)
        st = lib().hgemm_run_host(self._h, A.data_ptr(), B.data_ptr(), C.data_ptr(), s)
        if st != OK:
            raise HgemmError(st, f"hgemm_run_host{self.shape}")

    def close(self) -> None:
        if self._h and self.ctx._h:
            lib().hgemm_plan_destroy(self._h)
        self._h = ctypes.c_void_p()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
