"""ctypes binding of libgmagnus.so.  Names mirror the C ABI (gm_spgemm_plan -> spgemm_plan ...).

Argument marshalling only: device arrays are torch tensors, their data_ptr() values go straight
into the gm_csr structs, and the library's device allocations are served by torch's caching
allocator through the gm_set_allocator hook, so results come back as torch tensors without a copy.
There is no fallback: if the library cannot be loaded, importing this module fails.
"""
from __future__ import annotations

import ctypes
import os
import threading
from dataclasses import dataclass

import numpy as np
import torch

from . import build as _build

GM_MAX_LEVELS = 8
EXPORTED_SYMBOLS = [
    "gm_set_allocator", "gm_planner_params", "gm_planner_batches", "gm_spgemm_plan", "gm_spgemm_plan_ex", "gm_spgemm_execute",
    "gm_spgemm_host", "gm_plan_get_info", "gm_exec_get_stats", "gm_plan_set_timing",
    "gm_plan_get_row_products", "gm_row_products_noalloc", "gm_csr_free", "gm_plan_destroy", "gm_status_string", "gm_last_error",
]


class GmError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str):
        super().__init__(f"{where} failed: {status_string(status)} ({status}): {detail}")
        self.status = status


class _CSR(ctypes.Structure):
    _fields_ = [("n_rows", ctypes.c_int64), ("n_cols", ctypes.c_int64), ("nnz", ctypes.c_int64),
                ("row_ptr", ctypes.c_void_p), ("col_idx", ctypes.c_void_p), ("vals", ctypes.c_void_p),
                ("dtype", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class PlanOpts(ctypes.Structure):
    """gm_plan_opts: zero means "derive it"."""
    _fields_ = [("tau", ctypes.c_int64), ("chunk_width", ctypes.c_int32), ("max_fanout", ctypes.c_int32),
                ("acc_ctas_per_sm", ctypes.c_int32), ("stage_elems", ctypes.c_int64),
                ("c_capacity", ctypes.c_int64), ("separate_histogram", ctypes.c_int32),
                ("validate_inputs", ctypes.c_int32), ("single_stream", ctypes.c_int32),
                ("level0_multisplit", ctypes.c_int32), ("small_chunk_max", ctypes.c_int32),
                ("mid_chunk_max", ctypes.c_int32), ("expand_staging", ctypes.c_int32),
                ("debug_spin_limit", ctypes.c_int32), ("expand_order", ctypes.c_int32), ("early_exit", ctypes.c_int32)]


class Params(ctypes.Structure):
    _fields_ = [("tau", ctypes.c_int64), ("light_slots", ctypes.c_int32), ("chunk_width", ctypes.c_int32),
                ("chunks_required", ctypes.c_int32), ("max_fanout", ctypes.c_int32), ("n_levels", ctypes.c_int32),
                ("fanout", ctypes.c_int32 * GM_MAX_LEVELS), ("shift", ctypes.c_int32 * GM_MAX_LEVELS),
                ("acc_ctas_per_sm", ctypes.c_int32), ("acc_block_threads", ctypes.c_int32)]

    def levels(self):
        return [int(self.fanout[i]) for i in range(self.n_levels)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("params", Params), ("n_rows", ctypes.c_int64), ("n_cols_c", ctypes.c_int64),
                ("products_total", ctypes.c_int64), ("products_heavy", ctypes.c_int64),
                ("products_max_row", ctypes.c_int64), ("rows_heavy", ctypes.c_int64),
                ("rows_light", ctypes.c_int64), ("rows_empty", ctypes.c_int64), ("nnz_a_heavy", ctypes.c_int64),
                ("c_nnz_upper", ctypes.c_int64), ("n_batches", ctypes.c_int64), ("stage_elems", ctypes.c_int64),
                ("workspace_bytes", ctypes.c_int64), ("light_bin_rows", ctypes.c_int64 * 8),
                ("launches", ctypes.c_int64), ("level0_direct", ctypes.c_int64)]


class ExecStats(ctypes.Structure):
    _fields_ = [("c_nnz", ctypes.c_int64), ("c_nnz_heavy", ctypes.c_int64), ("c_capacity", ctypes.c_int64), ("staged_products", ctypes.c_int64),
                ("final_chunks", ctypes.c_int64), ("launches", ctypes.c_int64),
                ("small_chunk_products", ctypes.c_int64), ("small_chunk_entries", ctypes.c_int64),
                ("ms_light_symbolic", ctypes.c_float), ("ms_light_numeric", ctypes.c_float),
                ("ms_expand", ctypes.c_float), ("ms_histogram", ctypes.c_float), ("ms_multisplit", ctypes.c_float),
                ("ms_accumulate", ctypes.c_float), ("ms_gather", ctypes.c_float), ("ms_scan", ctypes.c_float),
                ("ms_total", ctypes.c_float), ("ms_small_chunks", ctypes.c_float), ("ms_mid_chunks", ctypes.c_float),
                ("reserved", ctypes.c_float * 3), ("mid_chunk_products", ctypes.c_int64), ("mid_chunk_entries", ctypes.c_int64),
                ("early_exit_products", ctypes.c_int64), ("early_exit_chunks", ctypes.c_int64),
                ("split_products", ctypes.c_int64)]


_ALLOC_FN = ctypes.CFUNCTYPE(ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p)
_FREE_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p)

_lib = None
_lock = threading.Lock()
_live: dict[int, torch.Tensor] = {}   # device blocks handed to the library, by address
_alloc_cb = None
_free_cb = None


def _torch_alloc(nbytes, stream, user):
    try:
        t = torch.empty(max(int(nbytes), 16), dtype=torch.uint8, device="cuda")
    except Exception:  # out of memory: the library turns NULL into GM_ERR_OOM
        return None
    _live[t.data_ptr()] = t
    return t.data_ptr()


def _torch_free(ptr, stream, user):
    _live.pop(ptr, None)


def load_library(install_torch_allocator: bool = True):
    """Loads (building it first if needed) libgmagnus.so and declares the C signatures."""
    global _lib, _alloc_cb, _free_cb
    with _lock:
        if _lib is not None:
            return _lib
        path = _build.build()
        lib = ctypes.CDLL(path)
        vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
        P = ctypes.POINTER
        lib.gm_set_allocator.argtypes = [_ALLOC_FN, _FREE_FN, vp]
        lib.gm_planner_params.argtypes = [i64, i32, sz, P(PlanOpts), P(Params)]
        lib.gm_planner_batches.argtypes = [vp, i64, i64, vp, i64]
        lib.gm_planner_batches.restype = i64
        lib.gm_spgemm_plan.argtypes = [P(_CSR), P(_CSR), sz, P(vp)]
        lib.gm_spgemm_plan_ex.argtypes = [P(_CSR), P(_CSR), sz, P(PlanOpts), vp, P(vp)]
        lib.gm_spgemm_execute.argtypes = [vp, vp, P(_CSR)]
        lib.gm_spgemm_host.argtypes = [P(_CSR), P(_CSR), sz, P(PlanOpts), P(_CSR), i64]
        lib.gm_plan_get_info.argtypes = [vp, P(PlanInfo)]
        lib.gm_exec_get_stats.argtypes = [vp, P(ExecStats)]
        lib.gm_plan_set_timing.argtypes = [vp, ctypes.c_int]
        lib.gm_plan_get_row_products.argtypes = [vp, vp, vp]
        lib.gm_row_products_noalloc.argtypes = [P(_CSR), P(_CSR), vp, vp]
        lib.gm_csr_free.argtypes = [P(_CSR)]
        lib.gm_csr_free.restype = None
        lib.gm_plan_destroy.argtypes = [vp]
        lib.gm_plan_destroy.restype = None
        lib.gm_status_string.argtypes = [ctypes.c_int]
        lib.gm_status_string.restype = ctypes.c_char_p
        lib.gm_last_error.argtypes = []
        lib.gm_last_error.restype = ctypes.c_char_p
        if install_torch_allocator and torch.cuda.is_available():
            _alloc_cb, _free_cb = _ALLOC_FN(_torch_alloc), _FREE_FN(_torch_free)
            lib.gm_set_allocator(_alloc_cb, _free_cb, None)
        _lib = lib
        return lib


def status_string(status: int) -> str:
    return load_library().gm_status_string(status).decode()


def _check(status: int, where: str):
    if status != 0:
        raise GmError(status, where, load_library().gm_last_error().decode())


@dataclass
class DeviceCSR:
    """CSR matrix in device memory: int64 row_ptr, int32 col, float32/float64 val (torch tensors)."""
    n_rows: int
    n_cols: int
    row_ptr: torch.Tensor
    col: torch.Tensor
    val: torch.Tensor
    nnz: int | None = None

    def __post_init__(self):
        if self.nnz is None:
            self.nnz = int(self.col.numel())

    @staticmethod
    def from_host(M, device="cuda") -> "DeviceCSR":
        """M: any object with n_rows, n_cols, row_ptr, col, val numpy arrays."""
        return DeviceCSR(M.n_rows, M.n_cols, torch.from_numpy(M.row_ptr).to(device),
                         torch.from_numpy(M.col).to(device), torch.from_numpy(M.val).to(device), int(M.row_ptr[-1]))

    def _struct(self) -> _CSR:
        assert self.row_ptr.dtype == torch.int64 and self.col.dtype == torch.int32
        assert self.val.dtype in (torch.float32, torch.float64)
        assert self.row_ptr.is_contiguous() and self.col.is_contiguous() and self.val.is_contiguous()
        return _CSR(self.n_rows, self.n_cols, self.nnz, self.row_ptr.data_ptr(), self.col.data_ptr(),
                    self.val.data_ptr(), 0 if self.val.dtype == torch.float32 else 1, 0)


def planner_params(c_cols: int, dtype, smem_bytes: int, opts: PlanOpts | None = None) -> Params:
    """gm_planner_params: host-only parameter selection (Section III-D)."""
    out = Params()
    code = 0 if np.dtype(dtype) == np.float32 else 1
    _check(load_library().gm_planner_params(c_cols, code, smem_bytes, ctypes.byref(opts) if opts else None,
                                            ctypes.byref(out)), "gm_planner_params")
    return out


def planner_batches(heavy_prefix: np.ndarray, stage_elems: int) -> list[int]:
    """gm_planner_batches: boundaries (heavy-row positions) of the staging-buffer batches."""
    hp = np.ascontiguousarray(heavy_prefix, dtype=np.int64)
    n = hp.size - 1
    out = np.zeros(n + 2, dtype=np.int64)
    rc = load_library().gm_planner_batches(hp.ctypes.data, n, stage_elems, out.ctypes.data, out.size)
    if rc < 0:
        raise GmError(int(rc), "gm_planner_batches", "a row exceeds stage_elems")
    return out[: rc + 1].tolist()


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


class Plan:
    """Owner of a gm_plan*.  Keeps A and B alive, since the plan borrows their arrays."""

    def __init__(self, handle, A: DeviceCSR, B: DeviceCSR):
        self._h, self.A, self.B = handle, A, B

    def info(self) -> PlanInfo:
        out = PlanInfo()
        _check(load_library().gm_plan_get_info(self._h, ctypes.byref(out)), "gm_plan_get_info")
        return out

    def stats(self) -> ExecStats:
        out = ExecStats()
        _check(load_library().gm_exec_get_stats(self._h, ctypes.byref(out)), "gm_exec_get_stats")
        return out

    def set_timing(self, enable: bool):
        _check(load_library().gm_plan_set_timing(self._h, int(enable)), "gm_plan_set_timing")

    def row_products(self, stream=None) -> torch.Tensor:
        out = torch.empty(self.A.n_rows, dtype=torch.int64, device=self.A.row_ptr.device)
        _check(load_library().gm_plan_get_row_products(self._h, out.data_ptr(), _stream_ptr(stream)),
               "gm_plan_get_row_products")
        return out

    def destroy(self):
        if self._h:
            load_library().gm_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


NOALLOC_MAX_NNZ_A = 1048576


def row_products_noalloc(A: DeviceCSR, B: DeviceCSR, out: torch.Tensor, stream=None) -> torch.Tensor:
    """gm_row_products_noalloc: IP_i for every row of A, written into the caller's int64 device tensor
    `out` (A.n_rows entries).  The library allocates nothing: its scratch is a fixed array in the library
    image, so nnz(A) is limited to NOALLOC_MAX_NNZ_A and calls that overlap on the GPU race on it."""
    assert out.dtype == torch.int64 and out.is_contiguous() and out.numel() >= A.n_rows
    a, b = A._struct(), B._struct()
    _check(load_library().gm_row_products_noalloc(ctypes.byref(a), ctypes.byref(b), out.data_ptr(),
                                                  _stream_ptr(stream)), "gm_row_products_noalloc")
    return out


def spgemm_plan(A: DeviceCSR, B: DeviceCSR, smem_bytes: int = 232448, opts: PlanOpts | None = None,
                stream=None) -> Plan:
    """gm_spgemm_plan_ex on the current (or given) torch stream."""
    lib = load_library()
    h = ctypes.c_void_p()
    a, b = A._struct(), B._struct()
    _check(lib.gm_spgemm_plan_ex(ctypes.byref(a), ctypes.byref(b), smem_bytes,
                                 ctypes.byref(opts) if opts else None, _stream_ptr(stream), ctypes.byref(h)),
           "gm_spgemm_plan")
    return Plan(h, A, B)


def _wrap(ptr: int, numel: int, dtype) -> torch.Tensor:
    block = _live.pop(ptr)
    return block.view(dtype)[:numel] if numel else block.view(dtype)[:0]


def spgemm_execute(plan: Plan, stream=None) -> DeviceCSR:
    """gm_spgemm_execute; the result's arrays are torch tensors over the library's allocations."""
    lib = load_library()
    c = _CSR()
    _check(lib.gm_spgemm_execute(plan._h, _stream_ptr(stream), ctypes.byref(c)), "gm_spgemm_execute")
    vdt = torch.float32 if c.dtype == 0 else torch.float64
    return DeviceCSR(c.n_rows, c.n_cols, _wrap(c.row_ptr, c.n_rows + 1, torch.int64),
                     _wrap(c.col_idx, c.nnz, torch.int32), _wrap(c.vals, c.nnz, vdt), int(c.nnz))


def spgemm(A: DeviceCSR, B: DeviceCSR, smem_bytes: int = 232448, opts: PlanOpts | None = None, stream=None):
    """plan + execute + destroy; returns (C, PlanInfo, ExecStats)."""
    plan = spgemm_plan(A, B, smem_bytes, opts, stream)
    try:
        C = spgemm_execute(plan, stream)
        return C, plan.info(), plan.stats()
    finally:
        plan.destroy()


def _host_struct(M, keep: list) -> _CSR:
    rp = np.ascontiguousarray(M.row_ptr, dtype=np.int64)
    ci = np.ascontiguousarray(M.col, dtype=np.int32)
    va = np.ascontiguousarray(M.val)
    keep += [rp, ci, va]
    return _CSR(M.n_rows, M.n_cols, int(rp[-1]), rp.ctypes.data, ci.ctypes.data, va.ctypes.data,
                0 if va.dtype == np.float32 else 1, 0)


def spgemm_host(A, B, out_row_ptr: np.ndarray, out_col: np.ndarray, out_val: np.ndarray,
                smem_bytes: int = 232448, opts: PlanOpts | None = None) -> int:
    """gm_spgemm_host: A, B and the output buffers are HOST arrays (numpy; pinned if they wrap pinned
    torch tensors).  Returns nnz(C); raises GmError(GM_ERR_CAPACITY) if the buffers are too small."""
    keep: list = []
    a, b = _host_struct(A, keep), _host_struct(B, keep)
    c = _CSR(0, 0, 0, out_row_ptr.ctypes.data, out_col.ctypes.data, out_val.ctypes.data, a.dtype, 0)
    cap = min(out_col.size, out_val.size)
    _check(load_library().gm_spgemm_host(ctypes.byref(a), ctypes.byref(b), smem_bytes,
                                         ctypes.byref(opts) if opts else None, ctypes.byref(c), cap),
           "gm_spgemm_host")
    return int(c.nnz)
