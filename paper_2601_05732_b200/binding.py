"""Thin ctypes binding over libmhclite.so (argument marshalling only).

Every method of :class:`MhcLite` has the name of the C entry point it calls
(``include/mhclite.h``) and passes the tensors' device pointers straight through;
no step of the path runs in Python or on the CPU.  PyTorch supplies device memory
and the CUDA stream.  Without the compiled library or without a CUDA device the
calls raise.
"""
from __future__ import annotations

import ctypes as C
import math
import os

_LIB = None
_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libmhclite.so")

OK, ERR_BAD_ARG, ERR_CUDA, ERR_WORKSPACE, ERR_TIMEOUT = 0, -1, -2, -3, -4


class MhcLiteError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)}) {detail}".rstrip())


_p, _i, _i64, _f, _sz = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_size_t

# name -> (restype, argtypes); mirrors include/mhclite.h
SIGNATURES = {
    "mhclite_create": (_i, [C.POINTER(_p), _i, _i, _i]),
    "mhclite_destroy": (_i, [_p]),
    "mhclite_status_string": (C.c_char_p, [_i]),
    "mhclite_last_error": (C.c_char_p, [_p]),
    "mhclite_perm_table": (_i, [_i, _p]),
    "mhclite_perm_table_device": (_i, [_p, _p]),
    "mhclite_workspace_bytes": (_sz, [_i, _i, _i64, _i]),
    "mhclite_set_workspace": (_i, [_p, _p, _sz]),
    "mhclite_set_perm_subset": (_i, [_p, _i, _p]),
    "mhclite_workspace_bytes_subset": (_sz, [_i, _i, _i64, _i]),
    "mhclite_coeffs_fwd": (_i, [_p, _i64, _p, _p, _p, _p, _p, _f, _p, _p, _p, _p, _p, _p, _p]),
    "mhclite_premix_fwd": (_i, [_p, _i64, _p, _p, _p, _p]),
    "mhclite_postres_fwd": (_i, [_p, _i64, _p, _p, _p, _p, _p, _p]),
    "mhclite_pre_fwd_fused": (_i, [_p, _i64, _p, _p, _p, _p, _p, _f, _p, _p, _p, _p, _p, _p, _p, _p]),
    "mhclite_pre_fwd_fused_ustat": (_i, [_p, _i64, _p, _p, _p, _p, _p, _f, _p, _p, _p, _p, _p, _p, _p, _p, _f, _p]),
    "mhclite_postres_fwd_next_proj": (_i, [_p, _i64, _p, _p, _p, _p, _p, _p, _p, _p]),
    "mhclite_pre_fwd_resume": (_i, [_p, _i64, _p, _p, _p, _f, _p, _p, _p, _p, _p, _p, _p, _p]),
    "mhclite_postres_bwd": (_i, [_p, _i64, _p, _p, _p, _p, _p, _p, _p, _p, _p, _i, _p]),
    "mhclite_premix_bwd": (_i, [_p, _i64, _p, _p, _p, _p, _p, _i, _p]),
    "mhclite_coeffs_bwd": (_i, [_p, _i64, _p, _p, _p, _p, _f, _p, _p, _p, _p, _p, _p, _p, _p, _p, _i,
                                _p, _p, _p, _p, _i, _p]),
    "mhclite_static_scratch_bytes": (_sz, []),
    "mhclite_coeffs_bwd_static": (_i, [_p, _i64, _p, _p, _p, _p, _f, _p, _p, _p, _p, _p, _p, _p, _p, _p, _i,
                                       _p, _p, _p, _p, _i, _p]),
    "mhclite_tail_bwd_fused": (_i, [_p, _i64, _p, _p, _p, _p, _f, _p, _p, _p, _p, _p, _p, _p, _p, _p, _p,
                                    _p, _p, _p, _p, _p, _i, _p]),
    "mhc_sk20_coeffs_fwd": (_i, [_p, _i64, _p, _p, _p, _p, _p, _f, _i, _p, _p, _p, _p, _p, _p]),
    "mhc_sk20_pre_fwd_fused": (_i, [_p, _i64, _p, _p, _p, _p, _p, _f, _i, _p, _p, _p, _p, _p, _p, _p]),
    "mhc_sk20_coeffs_bwd": (_i, [_p, _i64, _p, _p, _p, _p, _p, _f, _i, _p, _p, _p, _p, _p, _p, _p, _p, _i,
                                 _p, _p, _p, _p, _i, _p]),
    "mhc_sk20_tail_bwd_fused": (_i, [_p, _i64, _p, _p, _p, _p, _p, _f, _i, _p, _p, _p, _p, _p, _p, _p, _p, _p,
                                     _p, _p, _p, _p, _p, _i, _p]),
    "mhclite_ds_gap": (_i, [_p, _i64, _p, _p, _p, _p]),
    "mhclite_ds_gap_stats": (_i, [_p, _i64, _p, _p, _p]),
    "mhclite_log_inv_nu_histogram": (_i, [_p, _i64, _p, _i, _f, _f, _p, _p]),
    "mhclite_depth_product": (_i, [_p, _i64, _p, _p, _i, _p]),
    "mhclite_relative_range": (_i, [_p, _i64, _p, _p, _p]),
    "mhclite_step_host_bytes": (_sz, [_i, _i, _i64]),
    "mhclite_step_host": (_i, [_p, _i64, _p, _p, _p, _p, _p, _p, _p, _p, _f, _p, _p, _p, _p, _p, _p, _p, _p, _i,
                               _p, _sz, _p]),
    "mhclite_kernel_launches": (_i64, [_p]),
    "mhclite_device_status": (_i, [_p]),
    "mhclite_set_kernel_timing": (_i, [_p, _i]),
    "mhclite_kernel_time_ms": (_i, [_p, _i, C.POINTER(_f)]),
}


def load(path: str | None = None):
    """Loads libmhclite.so (building it with nvcc if it is absent). Raises if that fails."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    path = path or LIB_PATH
    if not os.path.exists(path):
        from . import build as _build
        _build.build()
    lib = C.CDLL(path)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _LIB = lib
    return lib


def status_string(status: int) -> str:
    return load().mhclite_status_string(int(status)).decode()


def perm_table(n: int):
    """sigma[k, i] of the lexicographically ordered permutations, from the library's host generator."""
    import numpy as np
    buf = np.zeros((math.factorial(n), n), dtype=np.uint8)
    rc = load().mhclite_perm_table(n, buf.ctypes.data)
    if rc:
        raise MhcLiteError(rc, "mhclite_perm_table")
    return buf


def workspace_bytes(n: int, Cc: int, T: int, kind: int = 0) -> int:
    return int(load().mhclite_workspace_bytes(n, Cc, T, kind))


class MhcLite:
    """One library context: n residual streams of C channels on one CUDA device."""

    def __init__(self, n: int, C_: int, device: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("mHC-lite needs a CUDA device; there is no CPU path")
        self._torch = torch
        self.lib = load()
        self.n, self.C, self.device = n, C_, device
        self.nfact = math.factorial(n)          # residual weights per token (K once a subset is attached)
        self._table = None
        h = _p()
        rc = self.lib.mhclite_create(C.byref(h), n, C_, device)
        if rc:
            raise MhcLiteError(rc, "mhclite_create")
        self._h = h
        self._ws = None

    def close(self):
        if getattr(self, "_h", None):
            self.lib.mhclite_destroy(self._h)
            self._h = None

    __del__ = close

    # -- helpers ---------------------------------------------------------------------------------
    def _check(self, rc: int, where: str):
        if rc:
            raise MhcLiteError(rc, where, self.lib.mhclite_last_error(self._h).decode())

    def _ptr(self, t, dtype=None):
        if t is None:
            return None
        torch = self._torch
        if not t.is_cuda or t.device.index != self.device or not t.is_contiguous():
            raise ValueError("expected a contiguous tensor on cuda:%d" % self.device)
        if dtype is not None and t.dtype != dtype:
            raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
        return t.data_ptr()

    def _stream(self):
        return self._torch.cuda.current_stream(self.device).cuda_stream

    def n_cols(self, kind: int = 0) -> int:
        return (self.nfact if kind == 0 else self.n * self.n) + 2 * self.n

    def set_perm_subset(self, table):
        """Attaches a table [K, n] (uint8 tensor on the device, or None) of K distinct permutations:
        Eq. (5) then runs over those K matrices only (paper Section 5)."""
        if table is None:
            self._check(self.lib.mhclite_set_perm_subset(self._h, 0, None), "mhclite_set_perm_subset")
            self._table, self.nfact = None, math.factorial(self.n)
            return
        if table.dtype != self._torch.uint8 or table.dim() != 2 or table.shape[1] != self.n:
            raise ValueError("expected a uint8 tensor of shape [K, n]")
        self._check(self.lib.mhclite_set_perm_subset(self._h, table.shape[0], self._ptr(table)), "mhclite_set_perm_subset")
        self._table, self.nfact = table, int(table.shape[0])

    def ensure_workspace(self, T: int, kind: int = 0):
        """Allocates (with torch) and attaches scratch large enough for T tokens."""
        lite = (workspace_bytes(self.n, self.C, T, 0) if self._table is None else
                int(self.lib.mhclite_workspace_bytes_subset(self.n, self.C, T, self.nfact)))
        need = max(lite, workspace_bytes(self.n, self.C, T, kind) if kind else 0)
        if self._ws is None or self._ws.numel() < need:
            self._ws = self._torch.empty(need + 256, dtype=self._torch.uint8, device=f"cuda:{self.device}")
            base = self._ws.data_ptr()
            self._ws_off = (-base) % 256
            self._check(self.lib.mhclite_set_workspace(self._h, base + self._ws_off, need), "mhclite_set_workspace")
        return need

    def perm_table_device(self):
        import numpy as np
        buf = np.zeros((self.nfact, self.n), dtype=np.uint8)
        self._check(self.lib.mhclite_perm_table_device(self._h, buf.ctypes.data), "mhclite_perm_table_device")
        return buf

    # -- forward ---------------------------------------------------------------------------------
    def coeffs_fwd(self, x, W, b, alpha, gain, eps, H_res, H_pre, H_post, a_saved, p_saved, rstd):
        t, f, h = self._torch, self._torch.float32, self._torch.bfloat16
        self.ensure_workspace(x.shape[0], 0)
        self._check(self.lib.mhclite_coeffs_fwd(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W, f), self._ptr(b, f), self._ptr(alpha, f),
            self._ptr(gain, f), float(eps), self._ptr(H_res, f), self._ptr(H_pre, f), self._ptr(H_post, f),
            self._ptr(a_saved, f), self._ptr(p_saved, f), self._ptr(rstd, f), self._stream()), "mhclite_coeffs_fwd")

    def premix_fwd(self, x, H_pre, u):
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhclite_premix_fwd(self._h, x.shape[0], self._ptr(x, h), self._ptr(H_pre, f),
                                                self._ptr(u, h), self._stream()), "mhclite_premix_fwd")

    def postres_fwd(self, x, y, H_res, H_post, x_next):
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhclite_postres_fwd(self._h, x.shape[0], self._ptr(x, h), self._ptr(y, h),
                                                 self._ptr(H_res, f), self._ptr(H_post, f), self._ptr(x_next, h),
                                                 self._stream()), "mhclite_postres_fwd")

    def pre_fwd_fused(self, x, W, b, alpha, gain, eps, H_res, H_pre, H_post, a_saved, p_saved, rstd, u):
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhclite_pre_fwd_fused(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W, f), self._ptr(b, f), self._ptr(alpha, f),
            self._ptr(gain, f), float(eps), self._ptr(H_res, f), self._ptr(H_pre, f), self._ptr(H_post, f),
            self._ptr(a_saved, f), self._ptr(p_saved, f), self._ptr(rstd, f), self._ptr(u, h), self._stream()),
            "mhclite_pre_fwd_fused")

    def pre_fwd_fused_ustat(self, x, W, b, alpha, gain, eps, H_res, H_pre, H_post, a_saved, p_saved, rstd, u, u_rstd,
                            eps_u):
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhclite_pre_fwd_fused_ustat(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W, f), self._ptr(b, f), self._ptr(alpha, f),
            self._ptr(gain, f), float(eps), self._ptr(H_res, f), self._ptr(H_pre, f), self._ptr(H_post, f),
            self._ptr(a_saved, f), self._ptr(p_saved, f), self._ptr(rstd, f), self._ptr(u, h), self._ptr(u_rstd, f),
            float(eps_u), self._stream()), "mhclite_pre_fwd_fused_ustat")

    def postres_fwd_next_proj(self, x, y, H_res, H_post, x_next, W_next, gain_next):
        f, h = self._torch.float32, self._torch.bfloat16
        self.ensure_workspace(x.shape[0], 0)
        self._check(self.lib.mhclite_postres_fwd_next_proj(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(y, h), self._ptr(H_res, f), self._ptr(H_post, f),
            self._ptr(x_next, h), self._ptr(W_next, f), self._ptr(gain_next, f), self._stream()),
            "mhclite_postres_fwd_next_proj")

    def pre_fwd_resume(self, x, b, alpha, eps, H_res, H_pre, H_post, a_saved, p_saved, rstd, u):
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhclite_pre_fwd_resume(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(b, f), self._ptr(alpha, f), float(eps),
            self._ptr(H_res, f), self._ptr(H_pre, f), self._ptr(H_post, f), self._ptr(a_saved, f), self._ptr(p_saved, f),
            self._ptr(rstd, f), self._ptr(u, h), self._stream()), "mhclite_pre_fwd_resume")

    # -- backward --------------------------------------------------------------------------------
    def postres_bwd(self, x, y, H_res, H_post, g, dy, dH_res, dH_post, dx=None, accumulate_dx=False):
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhclite_postres_bwd(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(y, h), self._ptr(H_res, f), self._ptr(H_post, f),
            self._ptr(g, h), self._ptr(dy, h), self._ptr(dH_res, f), self._ptr(dH_post, f), self._ptr(dx, h),
            int(accumulate_dx), self._stream()), "mhclite_postres_bwd")

    def premix_bwd(self, x, H_pre, du, dH_pre, dx=None, accumulate_dx=False):
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhclite_premix_bwd(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(H_pre, f), self._ptr(du, h), self._ptr(dH_pre, f),
            self._ptr(dx, h), int(accumulate_dx), self._stream()), "mhclite_premix_bwd")

    def coeffs_bwd(self, x, W, alpha, gain, eps, a_saved, p_saved, rstd, H_pre, H_post, dH_res, dH_pre, dH_post,
                   dx, accumulate_dx, dW, db, dalpha, dgain, accumulate_params=False):
        f, h = self._torch.float32, self._torch.bfloat16
        self.ensure_workspace(x.shape[0], 0)
        self._check(self.lib.mhclite_coeffs_bwd(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W, f), self._ptr(alpha, f), self._ptr(gain, f), float(eps),
            self._ptr(a_saved, f), self._ptr(p_saved, f), self._ptr(rstd, f), self._ptr(H_pre, f), self._ptr(H_post, f),
            self._ptr(dH_res, f), self._ptr(dH_pre, f), self._ptr(dH_post, f), self._ptr(dx, h), int(accumulate_dx),
            self._ptr(dW, f), self._ptr(db, f), self._ptr(dalpha, f), self._ptr(dgain, f), int(accumulate_params),
            self._stream()), "mhclite_coeffs_bwd")

    def coeffs_bwd_static(self, x, W, alpha, gain, eps, a_saved, p_saved, rstd, H_pre, H_post, dH_res, dH_pre,
                          dH_post, dx, accumulate_dx, dW, db, dalpha, dgain, accumulate_params=False):
        """coeffs_bwd for callers that cannot allocate: scratch is the library's built-in device array
        (no workspace is attached or touched; sizes beyond the array raise)."""
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhclite_coeffs_bwd_static(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W, f), self._ptr(alpha, f), self._ptr(gain, f), float(eps),
            self._ptr(a_saved, f), self._ptr(p_saved, f), self._ptr(rstd, f), self._ptr(H_pre, f), self._ptr(H_post, f),
            self._ptr(dH_res, f), self._ptr(dH_pre, f), self._ptr(dH_post, f), self._ptr(dx, h), int(accumulate_dx),
            self._ptr(dW, f), self._ptr(db, f), self._ptr(dalpha, f), self._ptr(dgain, f), int(accumulate_params),
            self._stream()), "mhclite_coeffs_bwd_static")

    def tail_bwd_fused(self, x, W, alpha, gain, eps, a_saved, p_saved, rstd, H_res, H_pre, H_post, g, du,
                       dH_res, dH_post, dx, dW, db, dalpha, dgain, accumulate_params=False):
        f, h = self._torch.float32, self._torch.bfloat16
        self.ensure_workspace(x.shape[0], 0)
        self._check(self.lib.mhclite_tail_bwd_fused(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W, f), self._ptr(alpha, f), self._ptr(gain, f), float(eps),
            self._ptr(a_saved, f), self._ptr(p_saved, f), self._ptr(rstd, f), self._ptr(H_res, f), self._ptr(H_pre, f),
            self._ptr(H_post, f), self._ptr(g, h), self._ptr(du, h), self._ptr(dH_res, f), self._ptr(dH_post, f),
            self._ptr(dx, h), self._ptr(dW, f), self._ptr(db, f), self._ptr(dalpha, f), self._ptr(dgain, f),
            int(accumulate_params), self._stream()), "mhclite_tail_bwd_fused")

    # -- SK comparison path ----------------------------------------------------------------------
    def sk20_coeffs_fwd(self, x, W_sk, b_sk, alpha, gain, eps, iters, H_res, H_pre, H_post, p_saved, rstd):
        f, h = self._torch.float32, self._torch.bfloat16
        self._check(self.lib.mhc_sk20_coeffs_fwd(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W_sk, f), self._ptr(b_sk, f), self._ptr(alpha, f),
            self._ptr(gain, f), float(eps), int(iters), self._ptr(H_res, f), self._ptr(H_pre, f), self._ptr(H_post, f),
            self._ptr(p_saved, f), self._ptr(rstd, f), self._stream()), "mhc_sk20_coeffs_fwd")

    def sk20_pre_fwd_fused(self, x, W_sk, b_sk, alpha, gain, eps, iters, H_res, H_pre, H_post, p_saved, rstd, u):
        f, h = self._torch.float32, self._torch.bfloat16
        self.ensure_workspace(x.shape[0], 1)
        self._check(self.lib.mhc_sk20_pre_fwd_fused(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W_sk, f), self._ptr(b_sk, f), self._ptr(alpha, f),
            self._ptr(gain, f), float(eps), int(iters), self._ptr(H_res, f), self._ptr(H_pre, f), self._ptr(H_post, f),
            self._ptr(p_saved, f), self._ptr(rstd, f), self._ptr(u, h), self._stream()), "mhc_sk20_pre_fwd_fused")

    def sk20_coeffs_bwd(self, x, W_sk, b_sk, alpha, gain, eps, iters, p_saved, rstd, H_pre, H_post, dH_res, dH_pre,
                        dH_post, dx, accumulate_dx, dW, db, dalpha, dgain, accumulate_params=False):
        f, h = self._torch.float32, self._torch.bfloat16
        self.ensure_workspace(x.shape[0], 1)
        self._check(self.lib.mhc_sk20_coeffs_bwd(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W_sk, f), self._ptr(b_sk, f), self._ptr(alpha, f),
            self._ptr(gain, f), float(eps), int(iters), self._ptr(p_saved, f), self._ptr(rstd, f), self._ptr(H_pre, f),
            self._ptr(H_post, f), self._ptr(dH_res, f), self._ptr(dH_pre, f), self._ptr(dH_post, f), self._ptr(dx, h),
            int(accumulate_dx), self._ptr(dW, f), self._ptr(db, f), self._ptr(dalpha, f), self._ptr(dgain, f),
            int(accumulate_params), self._stream()), "mhc_sk20_coeffs_bwd")

    def sk20_tail_bwd_fused(self, x, W_sk, b_sk, alpha, gain, eps, iters, p_saved, rstd, H_res, H_pre, H_post, g, du,
                            dH_res, dH_post, dx, dW, db, dalpha, dgain, accumulate_params=False):
        f, h = self._torch.float32, self._torch.bfloat16
        self.ensure_workspace(x.shape[0], 1)
        self._check(self.lib.mhc_sk20_tail_bwd_fused(
            self._h, x.shape[0], self._ptr(x, h), self._ptr(W_sk, f), self._ptr(b_sk, f), self._ptr(alpha, f),
            self._ptr(gain, f), float(eps), int(iters), self._ptr(p_saved, f), self._ptr(rstd, f), self._ptr(H_res, f),
            self._ptr(H_pre, f), self._ptr(H_post, f), self._ptr(g, h), self._ptr(du, h), self._ptr(dH_res, f),
            self._ptr(dH_post, f), self._ptr(dx, h), self._ptr(dW, f), self._ptr(db, f), self._ptr(dalpha, f),
            self._ptr(dgain, f), int(accumulate_params), self._stream()), "mhc_sk20_tail_bwd_fused")

    KERNELS = ("proj_fwd", "act_premix", "postres_fwd", "postres_bwd", "tail_pre", "tail_dx")

    def set_kernel_timing(self, on: bool):
        self._check(self.lib.mhclite_set_kernel_timing(self._h, int(on)), "mhclite_set_kernel_timing")

    def kernel_time_ms(self, kernel: int) -> float:
        ms = _f()
        self._check(self.lib.mhclite_kernel_time_ms(self._h, kernel, C.byref(ms)), "mhclite_kernel_time_ms")
        return float(ms.value)

    def device_status(self):
        """Raises if a kernel recorded a timed-out wait (synchronises the device)."""
        self._check(self.lib.mhclite_device_status(self._h), "mhclite_device_status")

    def kernel_launches(self) -> int:
        return int(self.lib.mhclite_kernel_launches(self._h))

    def step_host(self, x_host, y_host, g_host, du_host, W, b, alpha, gain, eps, u_host, x_next_host, dy_host,
                  dx_host, dW, db, dalpha, dgain, accumulate_params=False):
        """One fwd+bwd pass from (pinned) HOST activation tensors; device staging is kept on the context."""
        torch, f = self._torch, self._torch.float32
        T = x_host.shape[0]
        for t in (x_host, y_host, g_host, du_host, u_host, x_next_host, dy_host, dx_host):
            if t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous():
                raise ValueError("expected contiguous bf16 host tensors")
        self.ensure_workspace(T, 0)
        need = int(self.lib.mhclite_step_host_bytes(self.n, self.C, T))
        if getattr(self, "_staging", None) is None or self._staging.numel() < need + 256:
            self._staging = torch.empty(need + 256, dtype=torch.uint8, device=f"cuda:{self.device}")
        base = self._staging.data_ptr()
        base += (-base) % 256
        self._check(self.lib.mhclite_step_host(
            self._h, T, x_host.data_ptr(), y_host.data_ptr(), g_host.data_ptr(), du_host.data_ptr(),
            self._ptr(W, f), self._ptr(b, f), self._ptr(alpha, f), self._ptr(gain, f), float(eps),
            u_host.data_ptr(), x_next_host.data_ptr(), dy_host.data_ptr(), dx_host.data_ptr(),
            self._ptr(dW, f), self._ptr(db, f), self._ptr(dalpha, f), self._ptr(dgain, f), int(accumulate_params),
            base, need, self._stream()), "mhclite_step_host")

    def ds_gap_stats(self, H_res, stats):
        """stats [4] f32 <- (max l1, sum l1, max column deviation, sum column deviation) over the tokens."""
        f = self._torch.float32
        self._check(self.lib.mhclite_ds_gap_stats(self._h, H_res.shape[0], self._ptr(H_res, f), self._ptr(stats, f),
                                                  self._stream()), "mhclite_ds_gap_stats")

    def log_inv_nu_histogram(self, X, bins, lo, hi, hist):
        """hist [bins + 1] int64 <- histogram of log10(1/nu) of the matrices X[t]; hist[bins] counts nu == 0."""
        self._check(self.lib.mhclite_log_inv_nu_histogram(self._h, X.shape[0], self._ptr(X, self._torch.float32), int(bins),
                                                          float(lo), float(hi), self._ptr(hist, self._torch.int64),
                                                          self._stream()), "mhclite_log_inv_nu_histogram")

    def depth_product(self, H_res, P, first=False):
        """P[t] <- H_res[t] P[t] in place (P[t] <- H_res[t] when first)."""
        f = self._torch.float32
        self._check(self.lib.mhclite_depth_product(self._h, H_res.shape[0], self._ptr(H_res, f), self._ptr(P, f),
                                                   int(first), self._stream()), "mhclite_depth_product")

    def relative_range(self, X, nu):
        f = self._torch.float32
        self._check(self.lib.mhclite_relative_range(self._h, X.shape[0], self._ptr(X, f), self._ptr(nu, f),
                                                    self._stream()), "mhclite_relative_range")

    def ds_gap(self, H_res, l1_err=None, colsum_dev=None):
        f = self._torch.float32
        self._check(self.lib.mhclite_ds_gap(self._h, H_res.shape[0], self._ptr(H_res, f), self._ptr(l1_err, f),
                                            self._ptr(colsum_dev, f), self._stream()), "mhclite_ds_gap")
