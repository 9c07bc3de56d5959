"""ctypes front end of the CPU oracle (test infrastructure only).

RefEFCP mirrors the product's handle (create / step / getters) but runs the
plain fp64 CPU restatement in efcp_oracle.cpp on numpy arrays.
"""
import ctypes as C

import numpy as np

from . import build as _build

RHS_COMPRESSED = 0
RHS_ACCUMULATOR = 1
VALUES_BF16 = 2

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        vp, i32, i64, f32, u32, f64 = (C.c_void_p, C.c_int32, C.c_int64, C.c_float,
                                       C.c_uint32, C.c_double)
        L.efcp_ref_create.argtypes = [C.POINTER(vp), i64, i32, i64, f32, u32]
        L.efcp_ref_create_blockwise.argtypes = [C.POINTER(vp), i64, i32, i64, f32, u32, i64]
        L.efcp_ref_row_length.argtypes = [vp]
        L.efcp_ref_row_length.restype = i64
        L.efcp_ref_destroy.argtypes = [vp]
        L.efcp_ref_destroy.restype = None
        L.efcp_ref_step.argtypes = [vp, vp, vp]
        L.efcp_ref_update_rowform.argtypes = [vp, vp]
        L.efcp_ref_gram_full.argtypes = [vp, vp]
        L.efcp_ref_step_count.argtypes = [vp]
        L.efcp_ref_step_count.restype = i64
        for n in ("error", "accumulator", "gram", "p", "coef"):
            getattr(L, "efcp_ref_get_" + n).argtypes = [vp, vp]
        L.efcp_ref_get_row.argtypes = [vp, i32, vp, vp]
        L.efcp_ref_topk.argtypes = [vp, i64, i64, vp, vp]
        L.efcp_ref_topk_fullsort.argtypes = [vp, i64, i64, vp, vp]
        L.efcp_ref_woodbury_coef.argtypes = [vp, vp, i32, f64, vp]
        L.efcp_ref_wsm_coef.argtypes = [vp, vp, i32, f64, vp]
        L.efcp_ref_round_bf16.argtypes = [vp, vp, i64]
        L.efcp_ref_round_bf16.restype = None
        L.efcp_ref_num_threads.argtypes = []
        L.efcp_ref_set_num_threads.argtypes = [i32]
        L.efcp_ref_set_num_threads.restype = None
        _lib = L
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(lib().efcp_ref_num_threads())


def set_num_threads(n: int) -> None:
    """Size of the OpenMP team of the following calls (results do not depend on it)."""
    lib().efcp_ref_set_num_threads(int(n))


def topk(a: np.ndarray, k: int, fullsort: bool = False):
    a = np.ascontiguousarray(a, dtype=np.float32)
    idx = np.empty(k, np.int32)
    val = np.empty(k, np.float32)
    fn = lib().efcp_ref_topk_fullsort if fullsort else lib().efcp_ref_topk
    rc = fn(_ptr(a), a.size, k, _ptr(idx), _ptr(val))
    if rc != 0:
        raise ValueError(f"efcp_ref_topk rc={rc}")
    return idx, val


def round_bf16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty_like(a)
    lib().efcp_ref_round_bf16(_ptr(a), _ptr(out), a.size)
    return out


def woodbury_coef(S, p, lam):
    S = np.ascontiguousarray(S, np.float64)
    p = np.ascontiguousarray(p, np.float64)
    out = np.empty(p.size, np.float64)
    rc = lib().efcp_ref_woodbury_coef(_ptr(S), _ptr(p), p.size, float(lam), _ptr(out))
    if rc != 0:
        raise ArithmeticError(f"woodbury rc={rc}")
    return out


def wsm_coef(S, p, lam):
    S = np.ascontiguousarray(S, np.float64)
    p = np.ascontiguousarray(p, np.float64)
    out = np.empty(p.size, np.float64)
    rc = lib().efcp_ref_wsm_coef(_ptr(S), _ptr(p), p.size, float(lam), _ptr(out))
    if rc != 0:
        raise ArithmeticError(f"wsm rc={rc}")
    return out


class RefEFCP:
    def __init__(self, d, m, k, lam, flags=RHS_COMPRESSED, block=0):
        """block > 0: Top-k in blocks of `block` coordinates; self.k then becomes the row
        length (the sum of the per-block counts), self.k_req keeps the requested k."""
        self._h = None
        self.d, self.m, self.k, self.lam, self.flags = int(d), int(m), int(k), float(lam), flags
        self.k_req, self.block = int(k), int(block)
        h = C.c_void_p()
        rc = lib().efcp_ref_create_blockwise(C.byref(h), self.d, self.m, self.k, self.lam, flags,
                                             self.block)
        if rc != 0:
            raise ValueError(f"efcp_ref_create rc={rc}")
        self._h = h
        self.k = int(lib().efcp_ref_row_length(h))

    def close(self):
        if self._h:
            lib().efcp_ref_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def step(self, grad: np.ndarray) -> np.ndarray:
        g = np.ascontiguousarray(grad, dtype=np.float32)
        assert g.size == self.d
        u = np.empty(self.d, np.float32)
        rc = lib().efcp_ref_step(self._h, _ptr(g), _ptr(u))
        if rc != 0:
            raise ArithmeticError(f"efcp_ref_step rc={rc}")
        return u

    def update_rowform(self) -> np.ndarray:
        u = np.empty(self.d, np.float32)
        rc = lib().efcp_ref_update_rowform(self._h, _ptr(u))
        if rc != 0:
            raise ArithmeticError(f"rowform rc={rc}")
        return u

    @property
    def step_count(self):
        return int(lib().efcp_ref_step_count(self._h))

    def _get(self, name, shape, dtype):
        out = np.empty(shape, dtype)
        rc = getattr(lib(), "efcp_ref_get_" + name)(self._h, _ptr(out))
        assert rc == 0
        return out

    def error(self):
        return self._get("error", self.d, np.float32)

    def accumulator(self):
        return self._get("accumulator", self.d, np.float32)

    def gram(self):
        return self._get("gram", (self.m, self.m), np.float64)

    def gram_full(self):
        out = np.empty((self.m, self.m), np.float64)
        assert lib().efcp_ref_gram_full(self._h, _ptr(out)) == 0
        return out

    def p(self):
        return self._get("p", self.m, np.float64)

    def coef(self):
        return self._get("coef", self.m, np.float64)

    def row(self, slot):
        idx = np.empty(self.k, np.int32)
        val = np.empty(self.k, np.float32)
        assert lib().efcp_ref_get_row(self._h, slot, _ptr(idx), _ptr(val)) == 0
        return idx, val
