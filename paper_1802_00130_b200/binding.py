"""ctypes binding for include/gn.h.  Names mirror the C entry points (gn_Gv -> GnContext.Gv, ...)."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

GN_TF32 = 0
GN_FP32_ACCURATE = 1
_STATUS = {0: "GN_OK", 1: "GN_EINVAL", 2: "GN_ENOMEM", 3: "GN_ECUDA", 4: "GN_ESTATE", 5: "GN_ETIMEOUT"}

_vp, _i32, _i64, _dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_double
_SIGNATURES = {
    "gn_create": (_i32, [C.POINTER(_vp), _i32, C.POINTER(_i32), _dbl, _i64, _vp, _vp, _i32, _vp]),
    "gn_destroy": (_i32, [_vp]),
    "gn_num_params": (_i64, [_vp]),
    "gn_last_error": (C.c_char_p, [_vp]),
    "gn_workspace_bytes": (_i64, [_vp]),
    "gn_kernel_launches": (_i64, [_vp]),
    "gn_graph_replays": (_i64, [_vp]),
    "gn_set_batch_rows": (_i32, [_vp, _i64]),
    "gn_set_blockdiag_method": (_i32, [_vp, _i32]),
    "gn_set_accurate_method": (_i32, [_vp, _i32]),
    "gn_set_split": (_i32, [_vp, C.POINTER(_i32)]),
    "gn_num_partitions": (_i32, [_vp]),
    "gn_set_cg_termination": (_i32, [_vp, _i32, _dbl]),
    "gn_set_theta": (_i32, [_vp, _vp]),
    "gn_set_theta_host": (_i32, [_vp, _vp]),
    "gn_set_subsample": (_i32, [_vp, _vp, _i64]),
    "gn_set_subsample_host": (_i32, [_vp, _vp, _i64]),
    "gn_fun": (_i32, [_vp, C.POINTER(_dbl)]),
    "gn_grad": (_i32, [_vp, _vp, C.POINTER(_dbl)]),
    "gn_grad_host": (_i32, [_vp, _vp, C.POINTER(_dbl)]),
    "gn_Gv": (_i32, [_vp, _vp, _vp]),
    "gn_Gv_host": (_i32, [_vp, _vp, _vp]),
    "gn_Gv_blockdiag": (_i32, [_vp, _vp, _vp]),
    "gn_Gv_blockdiag_host": (_i32, [_vp, _vp, _vp]),
    "gn_cg_solve": (_i32, [_vp, _vp, _dbl, _i32, _i32, _dbl, _vp, C.POINTER(_i32), _vp, C.POINTER(_dbl)]),
    "gn_cg_solve_host": (_i32, [_vp, _vp, _dbl, _i32, _i32, _dbl, _vp, C.POINTER(_i32), C.POINTER(_dbl)]),
    "gn_debug_activations": (_i32, [_vp, _i32, _vp]),
    "gn_newton_iter": (_i32, [_vp, _vp, _vp, _i64, _vp, _vp, _vp]),
    "gn_debug_timeout_probe": (_i32, [_vp, _dbl]),
    "gn_debug_option": (_i32, [_vp, _i32, _i32]),
    "gn_debug_check_canaries": (_i32, [_vp, C.POINTER(_i64)]),
    "gn_debug_plan_group": (_i32, [_i32, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32), _i32, _i32, C.POINTER(_i32),
                                   C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32)]),
    "gn_profile": (_i32, [_vp, _i32]),
    "gn_profile_read": (_i32, [_vp, C.POINTER(_dbl), C.POINTER(_dbl), C.POINTER(_i64)]),
    "gn_thin_m_gemm_noalloc": (_i32, [_i32, _i32, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _vp, C.c_char_p, _i64]),
    "gn_debug_gemm": (_i32, [_vp, _i32, _i32, _i32, _i32, _vp, _i64, _i32, _vp, _i64, _i32, _vp, _i64]),
    "gn_debug_gemm_epilogue": (_i32, [_vp, _i32, _i32, _i32, _i32, _vp, _i64, _i32, _vp, _i64, _i32, _vp, _i64,
                                      _vp, _i32, _vp, _i64, C.c_float, _vp, _i64, C.c_float]),
}


class NewtonParams(C.Structure):
    """gn_newton_params; defaults are the paper's constants (eta is left open there)."""
    _fields_ = [("lam", _dbl), ("sigma", _dbl), ("eta", _dbl), ("eps", _dbl), ("drop", _dbl), ("boost", _dbl),
                ("cg_max", _i32), ("blockdiag", _i32), ("max_backtrack", _i32), ("reserved", _i32)]

    def __init__(self, lam=1.0, sigma=1e-3, eta=1e-4, eps=1e-5, drop=2.0 / 3.0, boost=1.5, cg_max=250, blockdiag=1,
                 max_backtrack=30):
        super().__init__(lam, sigma, eta, eps, drop, boost, cg_max, blockdiag, max_backtrack, 0)


class NewtonReport(C.Structure):
    _fields_ = [("f_before", _dbl), ("f_after", _dbl), ("alpha", _dbl), ("beta1", _dbl), ("beta2", _dbl), ("rho", _dbl),
                ("gTd", _dbl), ("dGd", _dbl), ("lambda_next", _dbl), ("cg_iters", _i32), ("backtracks", _i32)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class GnError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"{_STATUS.get(status, status)}: {message}")
        self.status = status


_lib = None


def lib_path():
    return _build.LIB


def exported_symbols():
    return sorted(_SIGNATURES)


def lib():
    """Load libgn_b200.so (building it if the sources are newer).  Fails loudly if it cannot."""
    global _lib
    if _lib is None:
        path = _build.build()
        handle = C.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)          # AttributeError if the symbol is missing
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _dev_ptr(t, dtype, count=None):
    import torch
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("expected a CUDA tensor")
    if t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"expected a contiguous {dtype} tensor")
    if count is not None and t.numel() != count:
        raise ValueError(f"expected {count} elements, got {t.numel()}")
    return _vp(t.data_ptr())


def _host_ptr(a, dtype, count=None):
    if not isinstance(a, np.ndarray) or a.dtype != dtype or not a.flags.c_contiguous:
        raise TypeError(f"expected a C-contiguous numpy array of {dtype}")
    if count is not None and a.size != count:
        raise ValueError(f"expected {count} elements, got {a.size}")
    return _vp(a.ctypes.data)


def plan_group(shapes, pairs=74, keep_order=False):
    """Work list of a grouped launch for [(M, N, K), ...] (host arithmetic of the library, no device needed):
    returns (pairs_used, order, tiles, waves, counts) with counts[k][q] = tiles of the k-th problem in launch order
    that pair q runs."""
    n = len(shapes)
    arr = lambda xs: (C.c_int32 * len(xs))(*[int(x) for x in xs])
    M, N, K = arr([s[0] for s in shapes]), arr([s[1] for s in shapes]), arr([s[2] for s in shapes])
    counts, waves, order, tiles = (C.c_int32 * (n * pairs))(), (C.c_int32 * n)(), (C.c_int32 * n)(), (C.c_int32 * n)()
    used = lib().gn_debug_plan_group(n, M, N, K, int(pairs), int(bool(keep_order)), counts, waves, order, tiles)
    if used < 0:
        raise ValueError("bad shapes / pair count")
    return used, list(order), list(tiles), list(waves), [list(counts[k * pairs:(k + 1) * pairs]) for k in range(n)]


def thin_m_gemm_noalloc(A, B, out, stream=None):
    """out[M][N] = sum_r A[r][m] B[r][n], M <= 16, through gn_thin_m_gemm_noalloc.

    For callers that cannot allocate device memory: the library call itself allocates nothing (its
    scratch is a fixed array inside the library), and this wrapper allocates nothing either - the
    caller brings `out`.  A [rows][M], B [rows][N], out [M][N]: CUDA float32, rows may be strided
    (stride(0) is the leading dimension).  Raises GnError with the library's message on failure.
    """
    import torch
    for t in (A, B, out):
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.dim() == 2 and t.stride(1) == 1):
            raise TypeError("expected 2-D CUDA float32 tensors with unit inner stride")
    rows, M = A.shape
    N = B.shape[1]
    if B.shape[0] != rows or tuple(out.shape) != (M, N):
        raise ValueError("shapes must be A [rows][M], B [rows][N], out [M][N]")
    st = stream if stream is not None else torch.cuda.current_stream(A.device)
    msg = C.create_string_buffer(256)
    rc = lib().gn_thin_m_gemm_noalloc(M, N, rows, _vp(A.data_ptr()), A.stride(0), _vp(B.data_ptr()), B.stride(0),
                                      _vp(out.data_ptr()), out.stride(0), _vp(st.cuda_stream), msg, 256)
    if rc != 0:
        raise GnError(rc, msg.value.decode())
    return out


class GnContext:
    """One problem (widths, C, X, Y) on the current CUDA device; wraps a gn_ctx."""

    def __init__(self, widths, C_reg, X, Y, precision=GN_FP32_ACCURATE, stream=None):
        import torch
        self._lib = lib()
        self.widths = [int(w) for w in widths]
        L = len(self.widths) - 1
        l = X.shape[0]
        if X.dim() != 2 or Y.dim() != 2 or X.shape[1] != self.widths[0] or Y.shape != (l, self.widths[-1]):
            raise ValueError("X must be [l][n_0] and Y [l][n_L]")
        self._X, self._Y = X, Y                 # borrowed by the library: keep them alive
        self._stream = stream if stream is not None else torch.cuda.current_stream(X.device)
        arr = (_i32 * (L + 1))(*self.widths)
        handle = _vp()
        st = self._lib.gn_create(C.byref(handle), L, arr, float(C_reg), l, _dev_ptr(X, torch.float32),
                                 _dev_ptr(Y, torch.float32), int(precision), _vp(self._stream.cuda_stream))
        if st != 0:
            raise GnError(st, "gn_create failed (needs an sm_100 device and valid arguments)")
        self._h = handle
        self.precision = int(precision)
        self.n = int(self._lib.gn_num_params(self._h))
        self.device = X.device

    # ------------------------------------------------------------------ helpers
    def _check(self, st):
        if st != 0:
            raise GnError(st, self._lib.gn_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            self._lib.gn_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _new(self, count=None):
        import torch
        return torch.empty(self.n if count is None else count, dtype=torch.float32, device=self.device)

    @property
    def workspace_bytes(self):
        return int(self._lib.gn_workspace_bytes(self._h))

    @property
    def kernel_launches(self):
        return int(self._lib.gn_kernel_launches(self._h))

    @property
    def graph_replays(self):
        return int(self._lib.gn_graph_replays(self._h))

    # ------------------------------------------------------------------ entry points
    def set_batch_rows(self, rows):
        self._check(self._lib.gn_set_batch_rows(self._h, int(rows)))

    def set_blockdiag_method(self, method):
        """0 choose, 1 propagate stacked streams, 2 stored Jacobian factors (Section 3.3.1)."""
        self._check(self._lib.gn_set_blockdiag_method(self._h, int(method)))

    def set_accurate_method(self, method):
        """0 choose, 1 FP32 FMA GEMM only, 2 error-compensated tensor-core form where the shape allows."""
        self._check(self._lib.gn_set_accurate_method(self._h, int(method)))

    def set_split(self, split):
        """Variable partition of Section 3.1: split[m] contiguous neuron groups in layer m (L+1 counts)."""
        split = [int(x) for x in split]
        if len(split) != len(self.widths):
            raise ValueError("split needs one count per layer, input layer included")
        arr = (C.c_int32 * len(split))(*split)
        self._check(self._lib.gn_set_split(self._h, arr))

    @property
    def num_partitions(self):
        return int(self._lib.gn_num_partitions(self._h))

    def set_cg_termination(self, cg_min=0, finished_share=1.0):
        """Termination rule of Section 4.4 for block-diagonal solves."""
        self._check(self._lib.gn_set_cg_termination(self._h, int(cg_min), float(finished_share)))

    def set_theta(self, theta):
        import torch
        self._check(self._lib.gn_set_theta(self._h, _dev_ptr(theta, torch.float32, self.n)))

    def set_theta_host(self, theta):
        self._check(self._lib.gn_set_theta_host(self._h, _host_ptr(theta, np.float32, self.n)))

    def set_subsample(self, idx):
        import torch
        self._check(self._lib.gn_set_subsample(self._h, _dev_ptr(idx, torch.int32), idx.numel()))
        self.nS = idx.numel()

    def set_subsample_host(self, idx):
        self._check(self._lib.gn_set_subsample_host(self._h, _host_ptr(idx, np.int32), idx.size))
        self.nS = idx.size

    def fun(self):
        f = _dbl()
        self._check(self._lib.gn_fun(self._h, C.byref(f)))
        return f.value

    def grad(self, out=None, with_f=False):
        import torch
        out = self._new() if out is None else out
        f = _dbl()
        self._check(self._lib.gn_grad(self._h, _dev_ptr(out, torch.float32, self.n), C.byref(f) if with_f else None))
        return (out, f.value) if with_f else out

    def grad_host(self, out=None, with_f=False):
        out = np.empty(self.n, dtype=np.float32) if out is None else out
        f = _dbl()
        self._check(self._lib.gn_grad_host(self._h, _host_ptr(out, np.float32, self.n), C.byref(f) if with_f else None))
        return (out, f.value) if with_f else out

    def Gv(self, v, out=None):
        import torch
        out = self._new() if out is None else out
        self._check(self._lib.gn_Gv(self._h, _dev_ptr(v, torch.float32, self.n), _dev_ptr(out, torch.float32, self.n)))
        return out

    def Gv_blockdiag(self, v, out=None):
        import torch
        out = self._new() if out is None else out
        self._check(self._lib.gn_Gv_blockdiag(self._h, _dev_ptr(v, torch.float32, self.n),
                                              _dev_ptr(out, torch.float32, self.n)))
        return out

    def Gv_host(self, v, out=None, blockdiag=False):
        out = np.empty(self.n, dtype=np.float32) if out is None else out
        fn = self._lib.gn_Gv_blockdiag_host if blockdiag else self._lib.gn_Gv_host
        self._check(fn(self._h, _host_ptr(v, np.float32, self.n), _host_ptr(out, np.float32, self.n)))
        return out

    def cg_solve(self, g, lam, blockdiag=False, max_iter=250, tol=1e-3, out=None, keep_iterates=False):
        """Returns (d, iters, resnorms[, iterates])."""
        import torch
        out = self._new() if out is None else out
        its = _i32()
        res = (_dbl * (max_iter + 1))()
        iterates = self._new(max_iter * self.n) if keep_iterates else None
        self._check(self._lib.gn_cg_solve(
            self._h, _dev_ptr(g, torch.float32, self.n), float(lam), int(bool(blockdiag)), int(max_iter), float(tol),
            _dev_ptr(out, torch.float32, self.n), C.byref(its),
            _dev_ptr(iterates, torch.float32) if keep_iterates else None, res))
        resn = np.array(res[: its.value + 1])
        if keep_iterates:
            return out, its.value, resn, iterates.view(max_iter, self.n)[: its.value]
        return out, its.value, resn

    def cg_solve_host(self, g, lam, blockdiag=False, max_iter=250, tol=1e-3, out=None):
        out = np.empty(self.n, dtype=np.float32) if out is None else out
        its = _i32()
        res = (_dbl * (max_iter + 1))()
        self._check(self._lib.gn_cg_solve_host(
            self._h, _host_ptr(g, np.float32, self.n), float(lam), int(bool(blockdiag)), int(max_iter), float(tol),
            _host_ptr(out, np.float32, self.n), C.byref(its), res))
        return out, its.value, np.array(res[: its.value + 1])

    def profile(self, enable):
        self._check(self._lib.gn_profile(self._h, int(bool(enable))))

    def profile_read(self):
        """Per-kernel GEMM timing since the last read: {"tensor": {...}, "ffma": {...}, "thin": {...}, "tensor_x3": {...},
        "tensor_1cta": {...}} ("tensor" = the CTA-pair kernel)."""
        ms, flop, cnt = (_dbl * 5)(), (_dbl * 5)(), (_i64 * 5)()
        self._check(self._lib.gn_profile_read(self._h, ms, flop, cnt))
        return {name: {"ms": ms[k], "flop": flop[k], "launches": cnt[k]}
                for k, name in enumerate(("tensor", "ffma", "thin", "tensor_x3", "tensor_1cta"))}

    def debug_gemm(self, kind, A, B, a_kmajor=True, b_kmajor=True):
        """Test hook: D[M][N] from A ([M][K] or [K][M]) and B ([N][K] or [K][N]); kind 0 tensor-core, 1 FMA."""
        import torch
        M, K = (A.shape if a_kmajor else A.shape[::-1])
        N = B.shape[0] if b_kmajor else B.shape[1]
        D = torch.empty((M, N), dtype=torch.float32, device=A.device)
        self._check(self._lib.gn_debug_gemm(self._h, int(kind), M, N, K, _dev_ptr(A, torch.float32), A.stride(0),
                                            int(a_kmajor), _dev_ptr(B, torch.float32), B.stride(0), int(b_kmajor),
                                            _dev_ptr(D, torch.float32), D.stride(0)))
        return D

    def debug_gemm_epilogue(self, kind, A, B, a_kmajor=True, b_kmajor=True, bias=None, sigmoid=False, dsig=None,
                            alpha=1.0, cin=None, beta=0.0):
        """Test hook: debug_gemm with the epilogue options of the path's contraction kernels (see gn.h)."""
        import torch
        M, K = (A.shape if a_kmajor else A.shape[::-1])
        N = B.shape[0] if b_kmajor else B.shape[1]
        D = torch.empty((M, N), dtype=torch.float32, device=A.device)
        ptr = lambda t: None if t is None else _dev_ptr(t, torch.float32)
        self._check(self._lib.gn_debug_gemm_epilogue(
            self._h, int(kind), M, N, K, _dev_ptr(A, torch.float32), A.stride(0), int(a_kmajor),
            _dev_ptr(B, torch.float32), B.stride(0), int(b_kmajor), _dev_ptr(D, torch.float32), D.stride(0),
            ptr(bias), int(bool(sigmoid)), ptr(dsig), 0 if dsig is None else dsig.stride(0), float(alpha),
            ptr(cin), 0 if cin is None else cin.stride(0), float(beta)))
        return D

    def newton_iter(self, theta, idx, direction, params):
        """One iteration of Algorithm 3 on this GPU; theta and direction are updated in place.  Returns the report."""
        import torch
        rep = NewtonReport()
        self._check(self._lib.gn_newton_iter(self._h, _dev_ptr(theta, torch.float32, self.n), _dev_ptr(idx, torch.int32),
                                             idx.numel(), _dev_ptr(direction, torch.float32, self.n), C.byref(params),
                                             C.byref(rep)))
        return rep.as_dict()

    def debug_timeout_probe(self, limit_ms=1.0):
        """Test hook: raises GnError(GN_ETIMEOUT) after a bounded device wait has run out."""
        self._check(self._lib.gn_debug_timeout_probe(self._h, float(limit_ms)))

    def debug_option(self, option, value):
        """Test hook: switch a launch strategy (0 = grouped launches, 1 = K slices of left-over tiles)."""
        self._check(self._lib.gn_debug_option(self._h, int(option), int(value)))

    def debug_check_canaries(self):
        """Test hook: raises GnError if a kernel wrote past the end of a workspace; returns the allocations checked."""
        n = _i64()
        self._check(self._lib.gn_debug_check_canaries(self._h, C.byref(n)))
        return int(n.value)

    def debug_activations(self, m):
        import torch
        out = torch.empty(self.nS * self.widths[m], dtype=torch.float32, device=self.device)
        self._check(self._lib.gn_debug_activations(self._h, int(m), _dev_ptr(out, torch.float32)))
        return out.view(self.nS, self.widths[m])
