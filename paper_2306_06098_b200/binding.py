"""Thin ctypes binding over libefcp.so (argument marshalling only).

The names mirror include/efcp.h.  PyTorch is used for device memory and streams; every
step of the method runs inside the CUDA library.  Importing this module fails loudly
when the library has not been built (there is no fallback path).
"""
import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libefcp.so")

OK, EINVAL, ENOMEM, ECUDA, ENUMERIC, ETIMEOUT, EINTERNAL, ETOOBIG = 0, -1, -2, -3, -4, -5, -6, -7
TOPK_STATIC_MAX_D = 1 << 20
RHS_COMPRESSED, RHS_ACCUMULATOR, VALUES_BF16, PRECOND_GGT, LCG_FP32, DEBUG_CHECKS = 0, 1, 2, 4, 8, 16
HOOK_DROP_BLOCK_LOADS = 1
GGT_MAX_M = 160

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2306_06098_b200.build` "
        "(nvcc, sm_100a). There is no CPU fallback.")

_lib = C.CDLL(LIB_PATH)
_vp, _i32, _i64, _f32, _u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_uint32

EXPORTS = {
    "efcp_create": ([C.POINTER(_vp), _i64, _i32, _i64, _f32], C.c_int),
    "efcp_create_ex": ([C.POINTER(_vp), _i64, _i32, _i64, _f32, _u32], C.c_int),
    "efcp_create_blockwise": ([C.POINTER(_vp), _i64, _i32, _i64, _f32, _u32, _i32], C.c_int),
    "efcp_workspace_bytes": ([_i64, _i32, _i64, _u32, _i32], _i64),
    "efcp_create_in": ([C.POINTER(_vp), _i64, _i32, _i64, _f32, _u32, _i32, _vp, _i64], C.c_int),
    "efcp_test_hook": ([_vp, _i32, _i32], C.c_int),
    "efcp_create_shard": ([C.POINTER(_vp), _i64, _i64, _i64, _i32, _i64, _i64, _f32, _u32, _i32,
                           _i32], C.c_int),
    "efcp_shard_phase": ([_vp, _i32, _vp, _vp, _vp], C.c_int),
    "efcp_shard_buffer": ([_vp, _i32, C.POINTER(_vp), C.POINTER(_i64), C.POINTER(_i32)], C.c_int),
    "efcp_row_count": ([_vp, _i32], _i64),
    "efcp_row_length": ([_vp], _i64),
    "efcp_step": ([_vp, _vp, _vp, _vp], C.c_int),
    "efcp_step_host": ([_vp, _vp, _vp, _vp], C.c_int),
    "efcp_destroy": ([_vp], C.c_int),
    "efcp_get_error": ([_vp, _vp], C.c_int),
    "efcp_get_row": ([_vp, _i32, _vp, _vp], C.c_int),
    "efcp_get_gram": ([_vp, _vp], C.c_int),
    "efcp_get_weights": ([_vp, _vp], C.c_int),
    "efcp_get_window": ([_vp, _vp, _vp], C.c_int),
    "efcp_state_size": ([_vp], _i64),
    "efcp_state_export": ([_vp, _vp, _i64], C.c_int),
    "efcp_state_import": ([_vp, _vp, _i64], C.c_int),
    "efcp_error_norm": ([_vp, _vp], C.c_int),
    "efcp_update_norm": ([_vp, _vp, _vp, _vp], C.c_int),
    "efcp_apply_update": ([_vp, _vp, _vp, _i64, _f32, _f32, _f32, _vp], C.c_int),
    "efcp_step_apply": ([_vp, _vp, _vp, _vp, _f32, _f32, _f32, _vp], C.c_int),
    "efcp_validate": ([_vp, _vp], C.c_int),
    "efcp_step_count": ([_vp], _i64),
    "efcp_status": ([_vp], C.c_int),
    "efcp_last_cuda_error": ([_vp], C.c_int),
    "efcp_last_residual": ([_vp], C.c_double),
    "efcp_state_bytes": ([_i64, _i32, _i64], _i64),
    "efcp_launches_per_step": ([_vp], _i32),
    "efcp_fixed_point_fallbacks": ([_vp], _i64),
    "efcp_profile_begin": ([_vp, _i32], C.c_int),
    "efcp_profile_end": ([_vp, _vp, _vp], C.c_int),
    "efcp_topk_static": ([_vp, _i64, _i64, _vp, _vp, _vp], C.c_int),
    "efcp_strerror": ([C.c_int], C.c_char_p),
}
for _name, (_args, _res) in EXPORTS.items():
    _fn = getattr(_lib, _name)  # AttributeError here = header and library out of sync
    _fn.argtypes = _args
    _fn.restype = _res


class EfcpError(RuntimeError):
    def __init__(self, code, where, cuda=0):
        self.code = code
        msg = _lib.efcp_strerror(code).decode()
        super().__init__(f"{where}: {msg} (code {code}" + (f", cudaError {cuda})" if cuda else ")"))


def strerror(code: int) -> str:
    return _lib.efcp_strerror(code).decode()


def state_bytes(d: int, m: int, k: int) -> int:
    return int(_lib.efcp_state_bytes(d, m, k))


def workspace_bytes(d: int, m: int, k: int, flags: int = 0, block: int = 0) -> int:
    return int(_lib.efcp_workspace_bytes(d, m, k, flags, block))


def paper_state_bytes(d: int, m: int, k: int, value_bytes: int = 4) -> int:
    """Footprint of Sparse M-FAC as the paper's appendix "Memory savings" counts it:
    indices 4mk, values value_bytes*mk, error feedback 4d, SP result 4m, LCG result 4d."""
    return 4 * m * k + value_bytes * m * k + 4 * d + 4 * m + 4 * d


def topk_static(a: torch.Tensor, k: int, idx: torch.Tensor, val: torch.Tensor, stream=None):
    """efcp_topk_static: exact Top-k of the device vector `a` into the device tensors `idx`
    (int32, k) and `val` (fp32, k), ascending indices, using no allocation at all (the
    scratch memory is a fixed array inside the library; at most TOPK_STATIC_MAX_D elements).
    For callers that must not allocate device memory; asynchronous on `stream`.  `a` must start
    on a 16-byte boundary (the library refuses other pointers with EINVAL)."""
    assert a.is_cuda and idx.is_cuda and val.is_cuda
    assert a.dtype == torch.float32 and val.dtype == torch.float32 and idx.dtype == torch.int32
    assert a.is_contiguous() and idx.is_contiguous() and val.is_contiguous()
    assert idx.numel() >= k and val.numel() >= k
    s = torch.cuda.current_stream() if stream is None else stream
    rc = _lib.efcp_topk_static(a.data_ptr(), a.numel(), int(k), idx.data_ptr(), val.data_ptr(),
                               s.cuda_stream)
    if rc != OK:
        raise EfcpError(rc, "efcp_topk_static")


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


class Efcp:
    """One optimizer state (efcp_ctx) on the current CUDA device."""

    def __init__(self, d: int, m: int, k: int, lam: float, flags: int = RHS_COMPRESSED,
                 block: int = 0, workspace: torch.Tensor = None, shard=None):
        """block > 0: Top-k in blocks of `block` coordinates (efcp_create_blockwise); self.k is
        then the row length efcp_row_length reports, self.k_req the requested k.
        workspace: a contiguous device tensor the handle takes all its memory from
        (efcp_create_in; workspace_bytes() gives the size); it must outlive the handle.
        shard: (d_global, d_lo, d_hi, k_global, index, count) makes the handle one coordinate
        shard of a larger state (efcp_create_shard); d is then d_hi - d_lo and k the row
        capacity (<= 0: the worst case)."""
        self._h = None
        self.d, self.m, self.k, self.lam, self.flags = int(d), int(m), int(k), float(lam), flags
        self.k_req, self.block = int(k), int(block)
        self._workspace = workspace
        h = _vp()
        if shard is not None:
            d_global, d_lo, d_hi, k_global, index, count = shard
            assert d_hi - d_lo == self.d and workspace is None and not block
            rc = _lib.efcp_create_shard(C.byref(h), d_global, d_lo, d_hi, self.m, k_global,
                                        self.k, self.lam, flags, index, count)
        elif workspace is None:
            rc = _lib.efcp_create_blockwise(C.byref(h), self.d, self.m, self.k, self.lam, flags,
                                            self.block)
        else:
            assert workspace.is_cuda and workspace.is_contiguous()
            rc = _lib.efcp_create_in(C.byref(h), self.d, self.m, self.k, self.lam, flags,
                                     self.block, workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size())
        if rc != OK:
            raise EfcpError(rc, "efcp_create_blockwise" if workspace is None else "efcp_create_in")
        self._h = h
        self.k = int(_lib.efcp_row_length(h))

    def close(self):
        if self._h and _lib is not None:  # (_lib is gone while the interpreter shuts down)
            _lib.efcp_destroy(self._h)
        self._h = None

    def __del__(self):
        self.close()

    def _check(self, rc, where):
        if rc != OK:
            raise EfcpError(rc, where, _lib.efcp_last_cuda_error(self._h))

    def step(self, grad: torch.Tensor, update: torch.Tensor, stream=None):
        """efcp_step on device tensors (fp32, contiguous, d elements); asynchronous."""
        assert grad.is_cuda and update.is_cuda and grad.dtype == update.dtype == torch.float32
        assert grad.is_contiguous() and update.is_contiguous()
        assert grad.numel() == self.d and update.numel() == self.d
        s = torch.cuda.current_stream() if stream is None else stream
        self._check(_lib.efcp_step(self._h, grad.data_ptr(), update.data_ptr(), s.cuda_stream),
                    "efcp_step")
        return update

    def step_ptr(self, grad_ptr: int, update_ptr: int, stream_ptr: int = 0):
        self._check(_lib.efcp_step(self._h, grad_ptr, update_ptr, stream_ptr), "efcp_step")

    def step_host(self, grad: torch.Tensor, update: torch.Tensor, stream=None):
        """efcp_step_host on host tensors (pinned preferred); returns when update is ready."""
        assert not grad.is_cuda and not update.is_cuda
        assert grad.dtype == update.dtype == torch.float32
        assert grad.is_contiguous() and update.is_contiguous()
        assert grad.numel() == self.d and update.numel() == self.d
        s = torch.cuda.current_stream() if stream is None else stream
        self._check(_lib.efcp_step_host(self._h, grad.data_ptr(), update.data_ptr(),
                                        s.cuda_stream), "efcp_step_host")
        return update

    @property
    def step_count(self) -> int:
        return int(_lib.efcp_step_count(self._h))

    @property
    def launches_per_step(self) -> int:
        return int(_lib.efcp_launches_per_step(self._h))

    def status(self) -> int:
        return int(_lib.efcp_status(self._h))

    def shard_phase(self, phase: int, grad=None, update=None, stream=None):
        """efcp_shard_phase: phase 0 takes the shard's gradient, phase 5 its update tensor."""
        s = torch.cuda.current_stream() if stream is None else stream
        self._check(_lib.efcp_shard_phase(self._h, phase,
                                          None if grad is None else grad.data_ptr(),
                                          None if update is None else update.data_ptr(),
                                          s.cuda_stream), "efcp_shard_phase")

    def shard_buffer(self, phase: int) -> torch.Tensor:
        """The device buffer to be summed over the shards after `phase`, as a tensor aliasing
        the library's memory (int32 for the counts - same bits as uint32 - or float64)."""
        p, n, f = _vp(), _i64(), _i32()
        self._check(_lib.efcp_shard_buffer(self._h, phase, C.byref(p), C.byref(n), C.byref(f)),
                    "efcp_shard_buffer")

        class _Alias:
            def __init__(self, ptr, typestr, count):
                self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr,
                                                 "data": (ptr, False), "version": 3}

        dev = torch.device("cuda", torch.cuda.current_device())
        return torch.as_tensor(_Alias(p.value, "<f8" if f.value else "<i4", int(n.value)),
                               device=dev)

    def row_count(self, slot: int) -> int:
        return int(_lib.efcp_row_count(self._h, slot))

    def test_hook(self, hook: int, value: int):
        self._check(_lib.efcp_test_hook(self._h, hook, value), "efcp_test_hook")

    def last_residual(self) -> float:
        return float(_lib.efcp_last_residual(self._h))

    def profile_begin(self, max_steps: int):
        self._check(_lib.efcp_profile_begin(self._h, max_steps), "efcp_profile_begin")

    def profile_end(self):
        """Returns ({stage: total ms}, steps recorded)."""
        ms = (C.c_double * 4)()
        n = C.c_int32()
        self._check(_lib.efcp_profile_end(self._h, C.cast(ms, C.c_void_p),
                                          C.cast(C.byref(n), C.c_void_p)), "efcp_profile_end")
        return dict(zip(("ef_topk", "sp", "mxm", "lcg"), list(ms))), int(n.value)

    def error(self) -> np.ndarray:
        out = np.empty(self.d, np.float32)
        self._check(_lib.efcp_get_error(self._h, _np_ptr(out)), "efcp_get_error")
        return out

    def row(self, slot: int):
        idx = np.empty(self.k, np.int32)
        val = np.empty(self.k, np.float32)
        self._check(_lib.efcp_get_row(self._h, slot, _np_ptr(idx), _np_ptr(val)), "efcp_get_row")
        return idx, val

    def gram(self) -> np.ndarray:
        out = np.empty((self.m, self.m), np.float64)
        self._check(_lib.efcp_get_gram(self._h, _np_ptr(out)), "efcp_get_gram")
        return out

    def window(self):
        """(I, V): the ring buffer as read-only (m, k) device tensors that alias the library's
        memory (efcp_get_window); valid until close()."""
        pi, pv = _vp(), _vp()
        self._check(_lib.efcp_get_window(self._h, C.cast(C.byref(pi), _vp),
                                         C.cast(C.byref(pv), _vp)), "efcp_get_window")

        class _Alias:
            def __init__(self, ptr, typestr, shape):
                self.__cuda_array_interface__ = {"shape": shape, "typestr": typestr,
                                                 "data": (ptr, False), "version": 3}

        shape = (self.m, self.k)
        dev = torch.device("cuda", torch.cuda.current_device())
        return (torch.as_tensor(_Alias(pi.value, "<i4", shape), device=dev),
                torch.as_tensor(_Alias(pv.value, "<f4", shape), device=dev))

    def state_export(self) -> np.ndarray:
        """The whole optimizer state as one host byte array (efcp_state_export)."""
        n = int(_lib.efcp_state_size(self._h))
        buf = np.empty(n, np.uint8)
        self._check(_lib.efcp_state_export(self._h, _np_ptr(buf), n), "efcp_state_export")
        return buf

    def state_import(self, buf: np.ndarray):
        buf = np.ascontiguousarray(buf, np.uint8)
        self._check(_lib.efcp_state_import(self._h, _np_ptr(buf), buf.size), "efcp_state_import")

    def error_norm(self) -> float:
        out = C.c_double()
        self._check(_lib.efcp_error_norm(self._h, C.cast(C.byref(out), C.c_void_p)),
                    "efcp_error_norm")
        return float(out.value)

    def update_norm(self, update: torch.Tensor, sync: bool = True, stream=None):
        """efcp_update_norm: |u|_2, kept on the device for apply_update; returned when sync."""
        assert update.is_cuda and update.dtype == torch.float32 and update.is_contiguous()
        assert update.numel() == self.d
        s = torch.cuda.current_stream() if stream is None else stream
        out = C.c_double()
        self._check(_lib.efcp_update_norm(self._h, update.data_ptr(),
                                          C.cast(C.byref(out), C.c_void_p) if sync else None,
                                          s.cuda_stream), "efcp_update_norm")
        return float(out.value) if sync else None

    def apply_update(self, theta: torch.Tensor, update: torch.Tensor, eta: float,
                     gamma: float = 0.0, clip_norm: float = 0.0, stream=None):
        """efcp_apply_update on the same sub-range of the parameters and of u (device, fp32,
        contiguous, equal lengths <= d); asynchronous."""
        assert theta.is_cuda and update.is_cuda and theta.dtype == update.dtype == torch.float32
        assert theta.is_contiguous() and update.is_contiguous()
        assert theta.numel() == update.numel()
        s = torch.cuda.current_stream() if stream is None else stream
        self._check(_lib.efcp_apply_update(self._h, theta.data_ptr(), update.data_ptr(),
                                           theta.numel(), eta, gamma, clip_norm, s.cuda_stream),
                    "efcp_apply_update")
        return theta

    def step_apply(self, grad: torch.Tensor, theta: torch.Tensor, update, eta: float,
                   gamma: float = 0.0, clip_norm: float = 0.0, stream=None):
        """efcp_step_apply: one optimizer step including the parameter update; asynchronous.
        update=None (only without clipping): u is not materialised, the linear combination
        updates theta directly."""
        for t in (grad, theta) + (() if update is None else (update,)):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
            assert t.numel() == self.d
        s = torch.cuda.current_stream() if stream is None else stream
        self._check(_lib.efcp_step_apply(self._h, grad.data_ptr(), theta.data_ptr(),
                                         None if update is None else update.data_ptr(), eta,
                                         gamma, clip_norm, s.cuda_stream), "efcp_step_apply")
        return theta

    def fixed_point_fallbacks(self) -> int:
        return int(_lib.efcp_fixed_point_fallbacks(self._h))

    def validate(self) -> int:
        """efcp_validate: raises EfcpError when the window's derived structures are
        inconsistent; returns 0 otherwise."""
        bad = C.c_int64()
        self._check(_lib.efcp_validate(self._h, C.cast(C.byref(bad), C.c_void_p)), "efcp_validate")
        return int(bad.value)

    def weights(self) -> np.ndarray:
        out = np.empty(self.m, np.float64)
        self._check(_lib.efcp_get_weights(self._h, _np_ptr(out)), "efcp_get_weights")
        return out
