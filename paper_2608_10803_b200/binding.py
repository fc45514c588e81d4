"""ctypes binding of ``libadaptmm.so``: the same names as ``include/adapt_matmul.h``.

Argument marshalling only.  Every step of the GEMM path runs inside the CUDA
library; there is no fallback.  If the shared object is missing, ``load()``
raises and nothing else in this module works.
"""
from __future__ import annotations

import ctypes
import os

F16, BF16 = 0, 1
ROW_MAJOR, COL_MAJOR = 0, 1
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NOMEM, ERR_CUDA, ERR_TIMEOUT, ERR_NOT_INIT = range(7)
CLASS_NAMES = ["Common", "SingleCoreSplitK", "MultiCoreSplitK", "HybridSplitK"]
FAMILY_NAMES = ["umma_1cta", "umma_2cta", "skinny", "simt", "cluster"]
FAM_UMMA_1CTA, FAM_UMMA_2CTA, FAM_SKINNY, FAM_SIMT, FAM_CLUSTER = range(5)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libadaptmm.so")

EXPORTS = [
    "adapt_init", "adapt_shutdown", "adapt_matmul_plan", "adapt_matmul", "adapt_matmul_host", "adapt_last_error",
    "adapt_last_error_message", "adapt_status_string", "adapt_plan_info", "adapt_plan_candidates",
    "adapt_matmul_plan_forced", "adapt_classify", "adapt_model_read_volume", "adapt_model_write_volume",
    "adapt_model_pipeline", "adapt_poll_device_status", "adapt_plan_cache_size", "adapt_launch_count",
    "adapt_matmul_noalloc", "adapt_matmul_batch", "adapt_matmul_repeat", "adapt_measure_dispatch",
    "adapt_measure_empty_launch", "adapt_map_encode_count", "adapt_set_map_cache", "adapt_selftest_wait_expiry",
    "adapt_measure_store_rate", "adapt_plan_many", "adapt_plan_table_save", "adapt_plan_table_load",
    "adapt_addmm", "adapt_matmul_strided_batch", "adapt_set_option",
    "adapt_set_calibration", "adapt_get_calibration", "adapt_calibration_names",
]


class PlanInfo(ctypes.Structure):
    _fields_ = [
        ("tiling_key", ctypes.c_uint64),
        ("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
        ("dtype", ctypes.c_int32), ("layoutA", ctypes.c_int32), ("layoutB", ctypes.c_int32),
        ("taxonomy_class", ctypes.c_int32), ("family", ctypes.c_int32),
        ("BM", ctypes.c_int32), ("BN", ctypes.c_int32), ("BK", ctypes.c_int32),
        ("stages", ctypes.c_int32),
        ("P_m", ctypes.c_int32), ("P_n", ctypes.c_int32), ("P_k", ctypes.c_int32),
        ("cluster", ctypes.c_int32), ("srcA", ctypes.c_int32), ("srcB", ctypes.c_int32),
        ("grid", ctypes.c_int32), ("fused", ctypes.c_int32),
        ("streamk", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("workspace_bytes", ctypes.c_int64),
        ("flops", ctypes.c_double), ("hbm_bytes", ctypes.c_double),
        ("t_pro_us", ctypes.c_double), ("t_main_us", ctypes.c_double), ("t_epi_us", ctypes.c_double),
        ("predicted_us", ctypes.c_double),
    ]

    def as_dict(self):
        d = {k: getattr(self, k) for k, _ in self._fields_}
        d["class_name"] = CLASS_NAMES[self.taxonomy_class]
        d["family_name"] = FAMILY_NAMES[self.family] if 0 <= self.family < len(FAMILY_NAMES) else "?"
        return d


class DispatchCost(ctypes.Structure):
    _fields_ = [
        ("host_us_call", ctypes.c_double), ("host_us_call_map_miss", ctypes.c_double),
        ("host_us_bare_launches", ctypes.c_double),
        ("device_us_call", ctypes.c_double), ("device_us_call_map_miss", ctypes.c_double),
        ("device_us_bare_launches", ctypes.c_double),
        ("launches_per_call", ctypes.c_int32), ("maps_per_call", ctypes.c_int32),
    ]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class AdaptError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"adapt_matmul status {status}: {message}")
        self.status = status


_lib = None


def load():
    """Load the C-ABI library (built in-tree by ``paper_2608_10803_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_10803_b200.build`; there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    i64, i32, u64, vp, dbl = ctypes.c_int64, ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_double
    lib.adapt_init.restype = i32
    lib.adapt_init.argtypes = [i32]
    lib.adapt_shutdown.restype = None
    lib.adapt_matmul_plan.restype = vp
    lib.adapt_matmul_plan.argtypes = [i64, i64, i64, i32, i32, i32]
    lib.adapt_matmul_plan_forced.restype = vp
    lib.adapt_matmul_plan_forced.argtypes = [i64, i64, i64, i32, i32, i32, u64]
    lib.adapt_matmul.restype = i32
    lib.adapt_matmul.argtypes = [vp, vp, vp, vp, vp]
    lib.adapt_matmul_host.restype = i32
    lib.adapt_matmul_host.argtypes = [vp, vp, vp, vp, vp]
    lib.adapt_matmul_noalloc.restype = i32
    lib.adapt_matmul_noalloc.argtypes = [i64, i64, i64, i32, i32, i32, vp, vp, vp, vp]
    lib.adapt_last_error.restype = i32
    lib.adapt_last_error_message.restype = ctypes.c_char_p
    lib.adapt_status_string.restype = ctypes.c_char_p
    lib.adapt_status_string.argtypes = [i32]
    lib.adapt_plan_info.restype = i32
    lib.adapt_plan_info.argtypes = [vp, ctypes.POINTER(PlanInfo)]
    lib.adapt_plan_candidates.restype = i32
    lib.adapt_plan_candidates.argtypes = [i64, i64, i64, i32, i32, i32, ctypes.POINTER(PlanInfo), i32]
    lib.adapt_classify.restype = i32
    lib.adapt_classify.argtypes = [i64] * 8
    lib.adapt_model_read_volume.restype = dbl
    lib.adapt_model_read_volume.argtypes = [i64] * 5
    lib.adapt_model_write_volume.restype = dbl
    lib.adapt_model_write_volume.argtypes = [i32] + [i64] * 5
    lib.adapt_model_pipeline.restype = dbl
    lib.adapt_model_pipeline.argtypes = [i32, i64, i64, dbl, dbl, dbl]
    lib.adapt_poll_device_status.restype = i32
    lib.adapt_poll_device_status.argtypes = [vp]
    lib.adapt_plan_cache_size.restype = i64
    lib.adapt_launch_count.restype = i64
    lib.adapt_map_encode_count.restype = i64
    lib.adapt_set_option.restype = i32
    lib.adapt_set_option.argtypes = [ctypes.c_char_p, i32]
    lib.adapt_set_calibration.restype = i32
    lib.adapt_set_calibration.argtypes = [ctypes.c_char_p, ctypes.c_double]
    lib.adapt_get_calibration.restype = i32
    lib.adapt_get_calibration.argtypes = [ctypes.c_char_p, ctypes.POINTER(ctypes.c_double)]
    lib.adapt_calibration_names.restype = i32
    lib.adapt_calibration_names.argtypes = [ctypes.c_char_p, i32]
    lib.adapt_set_map_cache.restype = None
    lib.adapt_set_map_cache.argtypes = [i32]
    lib.adapt_matmul_batch.restype = i32
    lib.adapt_matmul_batch.argtypes = [i64, vp, vp, vp, vp, vp]
    lib.adapt_matmul_repeat.restype = i32
    lib.adapt_matmul_repeat.argtypes = [vp, i32, vp, vp, vp, i32, vp]
    lib.adapt_measure_dispatch.restype = i32
    lib.adapt_measure_dispatch.argtypes = [vp, vp, vp, vp, vp, i32, ctypes.POINTER(DispatchCost)]
    lib.adapt_measure_empty_launch.restype = i32
    lib.adapt_measure_empty_launch.argtypes = [i32, i32, vp, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
    lib.adapt_measure_store_rate.restype = i32
    lib.adapt_measure_store_rate.argtypes = [vp, i64, i64, i32, i32, i32, i32, i32, vp, ctypes.POINTER(dbl)]
    lib.adapt_addmm.restype = i32
    lib.adapt_addmm.argtypes = [vp, vp, vp, vp, i32, ctypes.c_float, ctypes.c_float, vp, vp]
    lib.adapt_matmul_strided_batch.restype = i32
    lib.adapt_matmul_strided_batch.argtypes = [vp, vp, i64, vp, i64, vp, i64, i64, vp]
    lib.adapt_plan_many.restype = i64
    lib.adapt_plan_many.argtypes = [i64, vp, vp, vp]
    lib.adapt_plan_table_save.restype = i64
    lib.adapt_plan_table_save.argtypes = [ctypes.c_char_p]
    lib.adapt_plan_table_load.restype = i64
    lib.adapt_plan_table_load.argtypes = [ctypes.c_char_p]
    lib.adapt_selftest_wait_expiry.restype = i32
    lib.adapt_selftest_wait_expiry.argtypes = [u64, vp]
    _lib = lib
    return lib


def _check(status):
    if status != OK:
        raise AdaptError(status, load().adapt_last_error_message().decode())


def adapt_init(device: int = 0):
    _check(load().adapt_init(device))


def adapt_shutdown():
    load().adapt_shutdown()


def adapt_matmul_plan(M, N, K, dtype, layoutA=ROW_MAJOR, layoutB=ROW_MAJOR):
    h = load().adapt_matmul_plan(M, N, K, dtype, layoutA, layoutB)
    if not h:
        lib = load()
        raise AdaptError(lib.adapt_last_error(), lib.adapt_last_error_message().decode())
    return h


def adapt_matmul_plan_forced(M, N, K, dtype, layoutA, layoutB, tiling_key):
    h = load().adapt_matmul_plan_forced(M, N, K, dtype, layoutA, layoutB, tiling_key)
    if not h:
        lib = load()
        raise AdaptError(lib.adapt_last_error(), lib.adapt_last_error_message().decode())
    return h


def adapt_matmul(plan, A_ptr: int, B_ptr: int, C_ptr: int, stream: int = 0):
    """Enqueue C = A*B.  Pointers are raw device addresses (``tensor.data_ptr()``)."""
    _check(load().adapt_matmul(plan, A_ptr, B_ptr, C_ptr, stream))


def adapt_addmm(plan, A_ptr: int, B_ptr: int, D_ptr: int, d_is_vector: bool, alpha: float, beta: float, C_ptr: int, stream: int = 0):
    """Enqueue C = alpha * (A*B) + beta * D (D: M x N, or a row of N values when d_is_vector)."""
    _check(load().adapt_addmm(plan, A_ptr, B_ptr, D_ptr, 1 if d_is_vector else 0, alpha, beta, C_ptr, stream))


def adapt_matmul_strided_batch(plan, A_ptr: int, stride_a: int, B_ptr: int, stride_b: int, C_ptr: int, stride_c: int, batch: int,
                               stream: int = 0):
    """Enqueue `batch` GEMMs of the plan's shape on operands the given numbers of elements apart."""
    _check(load().adapt_matmul_strided_batch(plan, A_ptr, stride_a, B_ptr, stride_b, C_ptr, stride_c, batch, stream))


def adapt_matmul_host(plan, A_host_ptr: int, B_host_ptr: int, C_host_ptr: int, stream: int = 0):
    """Enqueue H2D(A, B), the GEMM and D2H(C) for host buffers (raw host addresses)."""
    _check(load().adapt_matmul_host(plan, A_host_ptr, B_host_ptr, C_host_ptr, stream))


def adapt_matmul_noalloc(M, N, K, dtype, layoutA, layoutB, A_ptr: int, B_ptr: int, C_ptr: int, stream: int = 0):
    """C = A*B without any device allocation: split-K partials go to the library's fixed 4 MiB
    scratch.  For callers that may not call cudaMalloc; the output must satisfy
    2 * M * roundup(N, 8) * 4 bytes <= 4 MiB.  Calls that overlap on the GPU race on the scratch."""
    _check(load().adapt_matmul_noalloc(M, N, K, dtype, layoutA, layoutB, A_ptr, B_ptr, C_ptr, stream))


def pointer_array(values):
    """A host array of pointers (plans or device addresses) for the batched entry points."""
    return (ctypes.c_void_p * len(values))(*values)


def adapt_matmul_batch(plans, A_ptrs, B_ptrs, C_ptrs, stream: int = 0, count=None):
    """adapt_matmul(plans[i], A[i], B[i], C[i]) for every i, one foreign call.  The arguments are
    ``pointer_array`` objects (or sequences, converted here)."""
    arrs = [a if isinstance(a, ctypes.Array) else pointer_array(list(a)) for a in (plans, A_ptrs, B_ptrs, C_ptrs)]
    _check(load().adapt_matmul_batch(len(arrs[0]) if count is None else count, *arrs, stream))


def adapt_matmul_repeat(plan, A_ptrs, B_ptrs, C_ptrs, calls: int, stream: int = 0):
    arrs = [a if isinstance(a, ctypes.Array) else pointer_array(list(a)) for a in (A_ptrs, B_ptrs, C_ptrs)]
    _check(load().adapt_matmul_repeat(plan, len(arrs[0]), *arrs, calls, stream))


def adapt_measure_dispatch(plan, A_ptr: int, B_ptr: int, C_ptr: int, stream: int = 0, calls: int = 100000) -> DispatchCost:
    out = DispatchCost()
    _check(load().adapt_measure_dispatch(plan, A_ptr, B_ptr, C_ptr, stream, calls, ctypes.byref(out)))
    return out


def adapt_measure_empty_launch(launches: int, programmatic: bool, stream: int = 0):
    """(host us, device us) per launch of an empty kernel issued back to back."""
    h, d = ctypes.c_double(), ctypes.c_double()
    _check(load().adapt_measure_empty_launch(launches, 1 if programmatic else 0, stream, ctypes.byref(h), ctypes.byref(d)))
    return h.value, d.value


def adapt_measure_store_rate(buf_ptr: int, rows: int, cols: int, mode: int, tile_cols: int = 192, order: int = 0,
                             hint: bool = False, passes: int = 3, stream: int = 0) -> float:
    """Device microseconds of one write-only pass over a [rows][cols] 16-bit matrix (see the header)."""
    us = ctypes.c_double()
    _check(load().adapt_measure_store_rate(buf_ptr, rows, cols, mode, tile_cols, order, 1 if hint else 0, passes, stream,
                                           ctypes.byref(us)))
    return us.value


def adapt_plan_many(shapes):
    """Plan a list of (M, N, K, dtype[, layoutA, layoutB]) in one call; returns the handles."""
    n = len(shapes)
    dims = (ctypes.c_int64 * (3 * n))()
    flags = (ctypes.c_int32 * (3 * n))()
    for i, sh in enumerate(shapes):
        dims[3 * i], dims[3 * i + 1], dims[3 * i + 2] = sh[0], sh[1], sh[2]
        flags[3 * i] = sh[3]
        flags[3 * i + 1] = sh[4] if len(sh) > 4 else ROW_MAJOR
        flags[3 * i + 2] = sh[5] if len(sh) > 5 else ROW_MAJOR
    handles = (ctypes.c_void_p * n)()
    planned = load().adapt_plan_many(n, dims, flags, handles)
    if planned < 0:
        lib = load()
        raise AdaptError(lib.adapt_last_error(), lib.adapt_last_error_message().decode())
    return list(handles)


def adapt_plan_table_save(path: str) -> int:
    n = load().adapt_plan_table_save(path.encode())
    if n < 0:
        lib = load()
        raise AdaptError(lib.adapt_last_error(), lib.adapt_last_error_message().decode())
    return n


def adapt_plan_table_load(path: str) -> int:
    n = load().adapt_plan_table_load(path.encode())
    if n < 0:
        lib = load()
        raise AdaptError(lib.adapt_last_error(), lib.adapt_last_error_message().decode())
    return n


def adapt_map_encode_count() -> int:
    return load().adapt_map_encode_count()


def adapt_set_option(name: str, value: int):
    _check(load().adapt_set_option(name.encode(), int(value)))


def adapt_set_calibration(name: str, value: float):
    _check(load().adapt_set_calibration(name.encode(), float(value)))


def adapt_get_calibration(name: str) -> float:
    v = ctypes.c_double(0.0)
    _check(load().adapt_get_calibration(name.encode(), ctypes.byref(v)))
    return float(v.value)


def adapt_calibration_names():
    lib = load()
    need = lib.adapt_calibration_names(None, 0)
    buf = ctypes.create_string_buffer(need + 1)
    lib.adapt_calibration_names(buf, need + 1)
    return buf.value.decode().split(",")


def adapt_set_map_cache(enabled: bool):
    load().adapt_set_map_cache(1 if enabled else 0)


def adapt_selftest_wait_expiry(limit_ns: int, stream: int = 0):
    _check(load().adapt_selftest_wait_expiry(limit_ns, stream))


def adapt_plan_info(plan) -> PlanInfo:
    info = PlanInfo()
    _check(load().adapt_plan_info(plan, ctypes.byref(info)))
    return info


def adapt_plan_candidates(M, N, K, dtype, layoutA=ROW_MAJOR, layoutB=ROW_MAJOR, cap: int = 512):
    buf = (PlanInfo * cap)()
    n = load().adapt_plan_candidates(M, N, K, dtype, layoutA, layoutB, buf, cap)
    if n < 0:
        lib = load()
        raise AdaptError(lib.adapt_last_error(), lib.adapt_last_error_message().decode())
    return [buf[i] for i in range(min(n, cap))]


def adapt_classify(M, N, m, n, m1, n1, n_core, acc_bytes) -> int:
    return load().adapt_classify(M, N, m, n, m1, n1, n_core, acc_bytes)


def adapt_model_read_volume(M, N, K, m1, n1) -> float:
    return load().adapt_model_read_volume(M, N, K, m1, n1)


def adapt_model_write_volume(cls, M, N, K, k, k1) -> float:
    return load().adapt_model_write_volume(cls, M, N, K, k, k1)


def adapt_model_pipeline(schedule, Q, L, t_M, t_P, T_drain) -> float:
    return load().adapt_model_pipeline(schedule, Q, L, t_M, t_P, T_drain)


def adapt_poll_device_status(stream: int = 0):
    _check(load().adapt_poll_device_status(stream))


def adapt_plan_cache_size() -> int:
    return load().adapt_plan_cache_size()


def adapt_launch_count() -> int:
    return load().adapt_launch_count()


# ---- convenience for torch callers (memory and streams only) -------------------------------------

def matmul(A, B, out=None, layoutA=ROW_MAJOR, layoutB=ROW_MAJOR, plan=None):
    """C = A @ B for CUDA fp16/bf16 torch tensors through the library (row-major storage by default).

    ``A`` holds M*K elements and ``B`` K*N elements in the stated layouts; shapes are read
    as (M, K) and (K, N).  torch is used for the output allocation and the current stream.
    """
    import torch

    assert A.is_cuda and B.is_cuda and A.dtype == B.dtype and A.is_contiguous() and B.is_contiguous()
    dtype = F16 if A.dtype == torch.float16 else BF16
    M, K = (A.shape if layoutA == ROW_MAJOR else (A.shape[1], A.shape[0]))
    K2, N = (B.shape if layoutB == ROW_MAJOR else (B.shape[1], B.shape[0]))
    assert K == K2
    if out is None:
        out = torch.empty((M, N), dtype=A.dtype, device=A.device)
    if plan is None:
        plan = adapt_matmul_plan(M, N, K, dtype, layoutA, layoutB)
    adapt_matmul(plan, A.data_ptr(), B.data_ptr(), out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    return out
