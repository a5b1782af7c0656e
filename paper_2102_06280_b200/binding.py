"""ctypes binding with the names of include/dbw.h.

Argument marshalling only: every step of the round runs in the CUDA library.  Torch supplies
device memory and the current stream.  If libdbw.so is missing or fails to load, importing any
entry point raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

WEIGHT_METROPOLIS, WEIGHT_UNIFORM = 0, 1
ORDER_LOCAL_THEN_MIX, ORDER_MIX_THEN_CORRECT = 0, 2
GEMM_FP32, GEMM_BF16 = 0, 4
STATUS_BAD_B, STATUS_NAN_TIME, STATUS_WAIT_TIMEOUT, STATUS_BAD_INDEX, STATUS_INTERNAL, STATUS_BOUNDS = 1, 2, 4, 8, 16, 32
MAX_LAYERS = 8

_ERR = {-1: "DBW_ERR_NULL", -2: "DBW_ERR_BAD_GRAPH", -3: "DBW_ERR_BAD_SHAPE", -4: "DBW_ERR_BAD_B",
        -5: "DBW_ERR_BAD_MODEL", -6: "DBW_ERR_CUDA", -7: "DBW_ERR_STATE", -8: "DBW_ERR_TOO_LARGE"}
SELECT_STATIC_MAX_N = 16384


class DbwError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        extra = ""
        if code == -6 and _lib is not None:
            extra = " (cudaError %d)" % _lib.dbw_last_cuda_error()
        super().__init__("%s failed: %s%s" % (where, _ERR.get(code, str(code)), extra))


class _ModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("dims", C.c_int32 * (MAX_LAYERS + 1)),
                ("w_off", C.c_int64 * MAX_LAYERS), ("b_off", C.c_int64 * MAX_LAYERS), ("batch", C.c_int32)]


# DBW_LIBRARY=debug selects the bounds-checked build (libdbw_dbg.so, see build.py)
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                         "libdbw_dbg.so" if os.environ.get("DBW_LIBRARY", "") == "debug" else "libdbw.so")
_lib = None

_P = C.c_void_p
_SIGNATURES = {
    "dbw_model_layout": (C.c_int, [_P, C.c_int32, C.c_int32, C.POINTER(_ModelDesc), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "dbw_init": (C.c_int, [C.POINTER(_P), C.c_int32, C.c_int64, C.c_int64, _P, _P, C.POINTER(_ModelDesc), C.c_uint32, C.c_int]),
    "dbw_destroy": (C.c_int, [_P]),
    "dbw_set_dataset": (C.c_int, [_P, _P, _P, C.c_int32]),
    "dbw_set_edge_times": (C.c_int, [_P, _P]),
    "dbw_select": (C.c_int, [_P, _P, _P, _P, _P, _P, _P, _P]),
    "dbw_select_static": (C.c_int, [C.c_int32, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P]),
    "dbw_grad": (C.c_int, [_P, _P, _P, _P, _P, _P]),
    "dbw_mix": (C.c_int, [_P, _P, _P, _P, _P, C.c_float, _P, _P, _P]),
    "dbw_mix_in_place_ok": (C.c_int, [_P]),
    "dbw_set_mix_panel": (C.c_int, [_P, C.c_int32]),
    "dbw_mix_kernel": (C.c_int, [_P]),
    "dbw_set_param_tracking": (C.c_int, [_P, C.c_int]),
    "dbw_set_fused_round": (C.c_int, [_P, C.c_int]),
    "dbw_round_is_fused": (C.c_int, [_P]),
    "dbw_round": (C.c_int, [_P, _P, _P, _P, _P, _P, C.c_float, _P, _P, _P, _P, _P, _P, _P, _P]),
    "dbw_round_host": (C.c_int, [_P, _P, _P, _P, _P, _P, C.c_float, _P, _P, _P, _P, _P, _P, _P]),
    "dbw_update_backups": (C.c_int, [_P, _P, _P, _P, _P]),
    "dbw_reset_backups": (C.c_int, [_P, _P]),
    "dbw_state_export": (C.c_int, [_P, _P, C.POINTER(C.c_size_t), _P]),
    "dbw_state_import": (C.c_int, [_P, _P, C.c_size_t, _P]),
    "dbw_status": (C.c_int, [_P]),
    "dbw_get_links": (C.c_int, [_P, _P]),
    "dbw_profile": (C.c_int, [_P, C.c_int]),
    "dbw_profile_read": (C.c_int, [_P, C.POINTER(C.c_double), C.POINTER(C.c_int32)]),
    "dbw_debug_wait_probe": (C.c_int, [_P, C.c_uint32, _P, _P]),
    "dbw_graph_order_2of4": (C.c_int, [C.c_int32, _P, _P, _P, C.c_int32]),
    "dbw_launch_count": (C.c_int64, []),
    "dbw_last_cuda_error": (C.c_int, []),
}


def lib() -> C.CDLL:
    """The loaded C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError("%s is missing: build it with `python -m paper_2102_06280_b200.build` "
                              "(there is no CPU fallback)" % _LIB_PATH)
        handle = C.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def exported_symbols() -> List[str]:
    return list(_SIGNATURES)


def _check(code: int, where: str) -> int:
    if code < 0:
        raise DbwError(code, where)
    return code


@dataclass
class ModelLayout:
    dims: List[int]
    batch: int
    w_off: List[int]
    b_off: List[int]
    d: int
    ld: int
    desc: _ModelDesc

    def pack(self, rows: np.ndarray) -> np.ndarray:
        """Logical rows (n, d) -> padded rows (n, ld), padding zero.  Pure re-indexing."""
        rows = np.asarray(rows)
        out = np.zeros((rows.shape[0], self.ld), dtype=rows.dtype)
        off = 0
        for l in range(len(self.dims) - 1):
            wsz = self.dims[l] * self.dims[l + 1]
            out[:, self.w_off[l]: self.w_off[l] + wsz] = rows[:, off: off + wsz]
            off += wsz
            out[:, self.b_off[l]: self.b_off[l] + self.dims[l + 1]] = rows[:, off: off + self.dims[l + 1]]
            off += self.dims[l + 1]
        return out

    def unpack(self, rows: np.ndarray) -> np.ndarray:
        """Padded rows (n, ld) -> logical rows (n, d)."""
        rows = np.asarray(rows)
        parts = []
        for l in range(len(self.dims) - 1):
            wsz = self.dims[l] * self.dims[l + 1]
            parts.append(rows[:, self.w_off[l]: self.w_off[l] + wsz])
            parts.append(rows[:, self.b_off[l]: self.b_off[l] + self.dims[l + 1]])
        return np.concatenate(parts, axis=1)


def model_layout(dims: Sequence[int], batch: int) -> ModelLayout:
    dims = [int(v) for v in dims]
    arr = (C.c_int32 * len(dims))(*dims)
    desc = _ModelDesc()
    d, ld = C.c_int64(), C.c_int64()
    _check(lib().dbw_model_layout(arr, len(dims) - 1, int(batch), C.byref(desc), C.byref(d), C.byref(ld)),
           "dbw_model_layout")
    L = len(dims) - 1
    return ModelLayout(dims, int(batch), [int(desc.w_off[l]) for l in range(L)],
                       [int(desc.b_off[l]) for l in range(L)], int(d.value), int(ld.value), desc)


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array (None stays NULL)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


class Dbw:
    """Handle of one simulated network (dbw_init ... dbw_destroy)."""

    def __init__(self, rowptr, col, d: int, ld: Optional[int] = None, model: Optional[ModelLayout] = None,
                 flags: int = 0, device: int = 0):
        rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
        col = np.ascontiguousarray(col, dtype=np.int32)
        self.N = len(rowptr) - 1
        self.nnz = len(col)
        self.model = model
        self.d = int(d)
        self.ld = int(ld if ld is not None else (model.ld if model else (d + 3) // 4 * 4))
        self.flags = flags
        self.device = device
        self._h = _P()
        self._keep = None
        _check(lib().dbw_init(C.byref(self._h), self.N, self.d, self.ld, rowptr.ctypes.data, col.ctypes.data,
                              C.byref(model.desc) if model else None, flags, device), "dbw_init")

    def close(self):
        if self._h:
            lib().dbw_destroy(self._h)
            self._h = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_dataset(self, feat, labels, S: int):
        self._keep = (feat, labels)
        _check(lib().dbw_set_dataset(self._h, _ptr(feat), _ptr(labels), int(S)), "dbw_set_dataset")

    def set_edge_times(self, t_edge):
        self._keep_edge = t_edge
        _check(lib().dbw_set_edge_times(self._h, _ptr(t_edge)), "dbw_set_edge_times")

    def select(self, t, b, kept, T_worker=None, T_nbr=None, T_round=None):
        _check(lib().dbw_select(self._h, _ptr(t), _ptr(b), _ptr(kept), _ptr(T_worker), _ptr(T_nbr), _ptr(T_round),
                                _stream()), "dbw_select")

    def grad(self, X, batch_idx, G, loss=None):
        _check(lib().dbw_grad(self._h, _ptr(X), _ptr(batch_idx), _ptr(G), _ptr(loss), _stream()), "dbw_grad")

    def mix(self, X, G, kept, b, lr: float, X_out, lr_per_worker=None):
        _check(lib().dbw_mix(self._h, _ptr(X), _ptr(G), _ptr(kept), _ptr(b), float(lr), _ptr(lr_per_worker),
                             _ptr(X_out), _stream()), "dbw_mix")

    def mix_in_place_ok(self) -> bool:
        return bool(lib().dbw_mix_in_place_ok(self._h))

    def set_param_tracking(self, enable: bool):
        _check(lib().dbw_set_param_tracking(self._h, int(bool(enable))), "dbw_set_param_tracking")

    def set_fused_round(self, enable):
        """True / False, or None for the library's own choice."""
        _check(lib().dbw_set_fused_round(self._h, -1 if enable is None else int(bool(enable))), "dbw_set_fused_round")

    def round_is_fused(self) -> bool:
        return bool(_check(lib().dbw_round_is_fused(self._h), "dbw_round_is_fused"))

    def mix_kernel(self) -> str:
        return ("mix_direct_kernel", "mix_panel_kernel", "mix_staged_kernel", "mix_tc_kernel", "mix_sp_kernel")[_check(lib().dbw_mix_kernel(self._h), "dbw_mix_kernel")]

    def set_mix_panel(self, cols: int):
        _check(lib().dbw_set_mix_panel(self._h, int(cols)), "dbw_set_mix_panel")

    def round(self, X, t, b, lr: float, X_out, kept, batch_idx=None, G_ext=None, lr_per_worker=None,
              T_worker=None, T_nbr=None, T_round=None, loss=None):
        _check(lib().dbw_round(self._h, _ptr(X), _ptr(t), _ptr(b), _ptr(batch_idx), _ptr(G_ext), float(lr),
                               _ptr(lr_per_worker), _ptr(X_out), _ptr(kept), _ptr(T_worker), _ptr(T_nbr),
                               _ptr(T_round), _ptr(loss), _stream()), "dbw_round")

    def round_host(self, X, h_t, h_b, lr: float, X_out, h_batch_idx=None, G_ext=None, h_kept=None,
                   h_T_worker=None, h_T_round=None, h_loss=None, h_b_out=None):
        _check(lib().dbw_round_host(self._h, _ptr(X), _ptr(h_t), _ptr(h_b), _ptr(h_batch_idx), _ptr(G_ext),
                                    float(lr), _ptr(X_out), _ptr(h_kept), _ptr(h_T_worker), _ptr(h_T_round),
                                    _ptr(h_loss), _ptr(h_b_out), _stream()), "dbw_round_host")

    def update_backups(self, t_next, b_out, theta_out=None):
        _check(lib().dbw_update_backups(self._h, _ptr(t_next), _ptr(b_out), _ptr(theta_out), _stream()),
               "dbw_update_backups")

    def reset_backups(self):
        _check(lib().dbw_reset_backups(self._h, _stream()), "dbw_reset_backups")

    def state_export(self) -> bytes:
        size = C.c_size_t(0)
        _check(lib().dbw_state_export(self._h, None, C.byref(size), _stream()), "dbw_state_export")
        buf = C.create_string_buffer(size.value)
        _check(lib().dbw_state_export(self._h, buf, C.byref(size), _stream()), "dbw_state_export")
        return buf.raw[: size.value]

    def state_import(self, blob: bytes):
        _check(lib().dbw_state_import(self._h, blob, len(blob), _stream()), "dbw_state_import")

    def profile(self, enable: bool):
        _check(lib().dbw_profile(self._h, int(bool(enable))), "dbw_profile")

    def profile_read(self):
        """({'grad': ms, 'select': ms, 'mix': ms, 'gemm': ms}, rounds) accumulated since the last read
        ('gemm' = the tensor-core GEMM launches inside the gradient stage)."""
        ms = (C.c_double * 4)(0.0, 0.0, 0.0, 0.0)
        n = C.c_int32(0)
        _check(lib().dbw_profile_read(self._h, ms, C.byref(n)), "dbw_profile_read")
        return {"grad": ms[0], "select": ms[1], "mix": ms[2], "gemm": ms[3]}, int(n.value)

    def debug_wait_probe(self, polls: int, out):
        _check(lib().dbw_debug_wait_probe(self._h, int(polls), _ptr(out), _stream()), "dbw_debug_wait_probe")

    def status(self) -> int:
        return _check(lib().dbw_status(self._h), "dbw_status")

    def links(self) -> np.ndarray:
        out = np.zeros((max(self.N - 1, 0), 2), dtype=np.int32)
        _check(lib().dbw_get_links(self._h, out.ctypes.data), "dbw_get_links")
        return out


def select_static(rowptr, col, t, b, kept, T_worker=None, T_nbr=None, T_round=None, status_out=None):
    """dbw_select_static: selection on the current device without a handle and without allocating.

    rowptr / col are device tensors here (int32); the other arguments are as in Dbw.select."""
    n = int(rowptr.numel()) - 1
    _check(lib().dbw_select_static(n, _ptr(rowptr), _ptr(col), _ptr(t), _ptr(b), _ptr(kept), _ptr(T_worker),
                                   _ptr(T_nbr), _ptr(T_round), _ptr(status_out), _stream()), "dbw_select_static")


def graph_order_2of4(rowptr, col) -> Optional[np.ndarray]:
    """dbw_graph_order_2of4: the worker order of the structured-sparse mix (host only); None if there is none."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    col = np.ascontiguousarray(col, dtype=np.int32)
    order = np.full(1024, -1, dtype=np.int32)
    n = _check(lib().dbw_graph_order_2of4(len(rowptr) - 1, rowptr.ctypes.data, col.ctypes.data, order.ctypes.data, 1024),
               "dbw_graph_order_2of4")
    return order[:n].copy() if n > 0 else None


def launch_count() -> int:
    return int(lib().dbw_launch_count())
