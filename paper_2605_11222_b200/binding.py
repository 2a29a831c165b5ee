"""ctypes binding over libadmmq.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every numerical step runs in the CUDA
kernels of the library.  If the library is missing the first call raises -- there is no
CPU path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libadmmq.so")

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_STATE, ERR_WORKSPACE, ERR_NOT_SPD, ERR_NONFINITE, ERR_TIMEOUT, \
    ERR_CUDA, ERR_UNSUPPORTED, WARN_MOVE_CAP = range(11)
F32, BF16 = 0, 1
FACTOR_TRIDIAG = 0
GEMM_TENSOR, GEMM_SIMT = 0, 1

EXPORTS = [
    "admmq_status_string", "admmq_workspace_bytes", "admmq_create", "admmq_destroy",
    "admmq_set_gemm_kind", "admmq_last_device_status", "admmq_hessian_reset",
    "admmq_hessian_accumulate", "admmq_hessian_set", "admmq_factor", "admmq_quantize_layer",
    "admmq_w_update", "admmq_local_search", "admmq_objective", "admmq_get_hessian",
    "admmq_launch_count", "admmq_set_timing", "admmq_reset_timing", "admmq_get_timing",
    "admmq_objective_static", "admmq_get_factor", "admmq_pair_swap", "admmq_test_set_wait",
    "admmq_hessian_export", "admmq_hessian_import", "admmq_test_w_update_correction",
    "admmq_test_w_update_series",
]
T_HESSIAN_PRODUCT, T_TRANSPOSE, T_FACTOR, T_WUPDATE_PRODUCT1, T_TRIDIAG_SOLVE, T_WUPDATE_PRODUCT2, \
    T_GRADIENT_PRODUCT, T_LOCAL_SEARCH, T_ROW_SPLIT, T_WUPDATE_ONE_PLANE = range(10)
TIMING_NAMES = ["hessian_product", "transpose", "factor", "wupdate_product1", "tridiag_solve",
                "wupdate_product2", "gradient_product", "local_search", "row_split", "wupdate_one_plane"]


class FactorCfg(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("damp_frac", C.c_double), ("precondition", C.c_int),
                ("kind", C.c_int), ("T", C.c_int), ("h_rho", C.POINTER(C.c_double)),
                ("rho0", C.c_double), ("gamma", C.c_double)]


class QuantCfg(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("bits", C.c_int), ("group_size", C.c_int),
                ("symmetric", C.c_int), ("use_caller_grid", C.c_int), ("n_refresh", C.c_int),
                ("h_refresh_iters", C.POINTER(C.c_int)), ("clip_points", C.c_int),
                ("clip_min_ratio", C.c_double), ("fused_epilogue", C.c_int), ("wupdate_route", C.c_int),
                ("product_planes", C.c_int), ("wupdate_series", C.c_int)]


class LsCfg(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("bits", C.c_int), ("group_size", C.c_int),
                ("max_moves_per_col", C.c_longlong), ("accept_tol", C.c_double)]


class PairSwapCfg(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("bits", C.c_int), ("group_size", C.c_int), ("rounds", C.c_int),
                ("batch", C.c_int), ("d_pairs", C.c_void_p), ("accept_tol", C.c_double)]


class Report(C.Structure):
    _fields_ = [("err_before", C.c_double), ("err_after", C.c_double), ("moves", C.c_longlong),
                ("iters_run", C.c_int), ("capped_columns", C.c_int), ("ms", C.c_float),
                ("refreshed_iter", C.c_int), ("one_plane_iters", C.c_int), ("series_iters", C.c_int),
                ("series2_iters", C.c_int), ("series0_iters", C.c_int)]


class AdmmqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def load_library(path: Optional[str] = None):
    """Loads libadmmq.so (once).  Raises if it is missing: there is no fallback path."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(
            f"{p} not found: build it with `python -m paper_2605_11222_b200.build` "
            "(the solver has no CPU or library fallback)")
    lib = C.CDLL(p)
    vp, ci, cll, cd = C.c_void_p, C.c_int, C.c_longlong, C.c_double
    lib.admmq_status_string.restype = C.c_char_p
    lib.admmq_status_string.argtypes = [ci]
    lib.admmq_workspace_bytes.restype = C.c_size_t
    lib.admmq_workspace_bytes.argtypes = [ci, ci, ci]
    lib.admmq_create.argtypes = [C.POINTER(vp), ci, ci, ci, vp, C.c_size_t, vp]
    lib.admmq_destroy.argtypes = [vp]
    lib.admmq_set_gemm_kind.argtypes = [vp, ci]
    lib.admmq_last_device_status.argtypes = [vp]
    lib.admmq_hessian_reset.argtypes = [vp]
    lib.admmq_hessian_accumulate.argtypes = [vp, vp, ci, cll, cll]
    lib.admmq_hessian_set.argtypes = [vp, vp]
    lib.admmq_hessian_export.argtypes = [vp, vp, C.POINTER(cll)]
    lib.admmq_hessian_import.argtypes = [vp, vp, cll]
    lib.admmq_factor.argtypes = [vp, C.POINTER(FactorCfg)]
    lib.admmq_quantize_layer.argtypes = [vp, vp, ci, C.POINTER(QuantCfg), vp, vp, vp, vp, vp,
                                         C.POINTER(Report)]
    lib.admmq_w_update.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp, cd, vp]
    lib.admmq_test_w_update_correction.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp, cd, vp]
    lib.admmq_test_w_update_series.argtypes = [vp, vp, ci, ci, vp, vp, vp, vp, cd, ci, vp]
    lib.admmq_local_search.argtypes = [vp, vp, ci, C.POINTER(LsCfg), vp, vp, vp, vp, C.POINTER(Report)]
    lib.admmq_objective.argtypes = [vp, vp, ci, ci, vp, vp, vp, C.POINTER(cd)]
    lib.admmq_pair_swap.argtypes = [vp, vp, ci, C.POINTER(PairSwapCfg), vp, vp, vp, vp, C.POINTER(Report)]
    lib.admmq_get_hessian.argtypes = [vp, vp, vp]
    lib.admmq_get_factor.argtypes = [vp, vp, vp, vp]
    lib.admmq_set_timing.argtypes = [vp, ci]
    lib.admmq_reset_timing.argtypes = [vp]
    lib.admmq_get_timing.argtypes = [vp, ci, C.POINTER(cd), C.POINTER(cll)]
    lib.admmq_objective_static.argtypes = [vp, ci, vp, ci, ci, vp, vp, vp, vp, vp]
    lib.admmq_test_set_wait.argtypes = [vp, cll, ci]
    lib.admmq_launch_count.restype = cll
    lib.admmq_launch_count.argtypes = [vp]
    for name in EXPORTS:
        if name not in ("admmq_status_string", "admmq_workspace_bytes", "admmq_launch_count"):
            getattr(lib, name).restype = ci
    if path is None:
        _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().admmq_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return C.c_void_p(t.data_ptr())


def _check(st: int, where: str, allow=(OK,)):
    if st not in allow:
        raise AdmmqError(st, where)
    return st


class Solver:
    """One context of the C ABI (fixed d_in), with its workspace held in a torch buffer."""

    def __init__(self, d_in: int, d_out_max: int, T_max: int = 500, device="cuda:0",
                 stream: Optional[torch.cuda.Stream] = None):
        self.lib = load_library()
        self.device = torch.device(device)
        self.d_in, self.d_out_max, self.T_max = d_in, d_out_max, T_max
        nbytes = self.lib.admmq_workspace_bytes(d_in, d_out_max, T_max)
        if nbytes == 0:
            raise AdmmqError(ERR_SHAPE, "admmq_workspace_bytes")
        torch.cuda.set_device(self.device)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.stream = stream
        sp = C.c_void_p(stream.cuda_stream if stream is not None else
                        torch.cuda.current_stream(self.device).cuda_stream)
        h = C.c_void_p()
        _check(self.lib.admmq_create(C.byref(h), d_in, d_out_max, T_max, C.c_void_p(base), nbytes, sp),
               "admmq_create")
        self.h = h
        self._rho_keepalive = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.admmq_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- thin wrappers, one per ABI call ----
    def set_gemm_kind(self, kind: int):
        _check(self.lib.admmq_set_gemm_kind(self.h, kind), "admmq_set_gemm_kind")

    def last_device_status(self) -> int:
        return self.lib.admmq_last_device_status(self.h)

    def hessian_reset(self):
        _check(self.lib.admmq_hessian_reset(self.h), "admmq_hessian_reset")

    def hessian_accumulate(self, X: torch.Tensor):
        assert X.dim() == 2 and X.is_cuda and X.stride(1) == 1
        dt = {torch.float32: F32, torch.bfloat16: BF16}[X.dtype]
        _check(self.lib.admmq_hessian_accumulate(self.h, C.c_void_p(X.data_ptr()), dt, X.shape[0],
                                                 X.stride(0)), "admmq_hessian_accumulate")

    def hessian_set(self, H: torch.Tensor):
        _check(self.lib.admmq_hessian_set(self.h, _ptr(H)), "admmq_hessian_set")

    def hessian_export(self):
        """(sum_t x_t x_t^T as a full symmetric fp32 matrix, rows accumulated so far)."""
        H = torch.empty(self.d_in, self.d_in, dtype=torch.float32, device=self.device)
        ntok = C.c_longlong(0)
        _check(self.lib.admmq_hessian_export(self.h, _ptr(H), C.byref(ntok)), "admmq_hessian_export")
        return H, int(ntok.value)

    def hessian_import(self, H_raw: torch.Tensor, n_tokens: int):
        _check(self.lib.admmq_hessian_import(self.h, _ptr(H_raw), int(n_tokens)), "admmq_hessian_import")

    def factor(self, rho: Optional[Sequence[float]] = None, T: int = 0, rho0: float = 0.1,
               gamma: float = 1.1, damp_frac: float = 0.01, precondition: bool = True,
               kind: int = FACTOR_TRIDIAG):
        cfg = FactorCfg()
        cfg.struct_size = C.sizeof(FactorCfg)
        cfg.damp_frac = damp_frac
        cfg.precondition = int(precondition)
        cfg.kind = kind
        if rho is not None:
            arr = (C.c_double * len(rho))(*[float(r) for r in rho])
            cfg.h_rho = C.cast(arr, C.POINTER(C.c_double))
            cfg.T = len(rho)
            self._rho_keepalive = arr
        else:
            cfg.h_rho = None
            cfg.T = T
            cfg.rho0, cfg.gamma = rho0, gamma
        _check(self.lib.admmq_factor(self.h, C.byref(cfg)), "admmq_factor")
        self.T = cfg.T

    def quantize_layer(self, W0: torch.Tensor, bits: int, group_size: int = 0, symmetric: bool = False,
                       codes=None, scale=None, zero=None, Wq=None, resid=None, use_caller_grid=False,
                       report: bool = True, refresh_at: Sequence[int] = (), clip_points: int = 0,
                       clip_min_ratio: float = 0.8, fused_epilogue: bool = False, wupdate_route: int = 0,
                       product_planes: int = 0, wupdate_series: int = 0):
        p, n = W0.shape
        gs = n if group_size in (0, n) else group_size
        dev = W0.device
        codes = codes if codes is not None else torch.empty(p, n, dtype=torch.uint8, device=dev)
        scale = scale if scale is not None else torch.empty(p, n // gs, dtype=torch.float32, device=dev)
        zero = zero if zero is not None else torch.empty(p, n // gs, dtype=torch.float32, device=dev)
        iters = (C.c_int * max(1, len(refresh_at)))(*[int(t) for t in refresh_at])
        cfg = QuantCfg(C.sizeof(QuantCfg), bits, group_size, int(symmetric), int(use_caller_grid),
                       len(refresh_at), C.cast(iters, C.POINTER(C.c_int)) if len(refresh_at) else None,
                       int(clip_points), float(clip_min_ratio), int(fused_epilogue), int(wupdate_route),
                       int(product_planes), int(wupdate_series))
        rep = Report()
        st = self.lib.admmq_quantize_layer(self.h, _ptr(W0), p, C.byref(cfg), _ptr(codes), _ptr(scale),
                                           _ptr(zero), _ptr(Wq), _ptr(resid),
                                           C.byref(rep) if report else None)
        _check(st, "admmq_quantize_layer")
        return codes, scale, zero, (rep if report else None)

    def w_update(self, W0, group_size, codes, scale, zero, V, rho: float, W_out=None):
        W_out = W_out if W_out is not None else torch.empty_like(W0)
        _check(self.lib.admmq_w_update(self.h, _ptr(W0), W0.shape[0], group_size, _ptr(codes), _ptr(scale),
                                       _ptr(zero), _ptr(V), float(rho), _ptr(W_out)), "admmq_w_update")
        return W_out

    def w_update_correction(self, W0, group_size, codes, scale, zero, V, rho: float, Z_out=None):
        """W^(t+1) - W_hat' of one W-update (admmq_testing.h): the same call as w_update without the weight-sized
        term, for accuracy checks at the scale of a grid step."""
        Z_out = Z_out if Z_out is not None else torch.empty_like(W0)
        _check(self.lib.admmq_test_w_update_correction(self.h, _ptr(W0), W0.shape[0], group_size, _ptr(codes),
                                                       _ptr(scale), _ptr(zero), _ptr(V), float(rho), _ptr(Z_out)),
               "admmq_test_w_update_correction")
        return Z_out

    def w_update_series(self, W0, group_size, codes, scale, zero, V, rho: float, terms: int = 1, Z_out=None):
        """The same correction evaluated as the truncated series of the later iterations, `terms` terms of E kept
        (admmq_testing.h)."""
        Z_out = Z_out if Z_out is not None else torch.empty_like(W0)
        _check(self.lib.admmq_test_w_update_series(self.h, _ptr(W0), W0.shape[0], group_size, _ptr(codes),
                                                   _ptr(scale), _ptr(zero), _ptr(V), float(rho), int(terms),
                                                   _ptr(Z_out)),
               "admmq_test_w_update_series")
        return Z_out

    def local_search(self, W0, bits, group_size, codes, scale, zero, Wq=None, max_moves_per_col: int = 0,
                     accept_tol: float = 1e-6, report: bool = True):
        cfg = LsCfg(C.sizeof(LsCfg), bits, group_size, max_moves_per_col, accept_tol)
        rep = Report()
        st = self.lib.admmq_local_search(self.h, _ptr(W0), W0.shape[0], C.byref(cfg), _ptr(codes),
                                         _ptr(scale), _ptr(zero), _ptr(Wq), C.byref(rep) if report else None)
        _check(st, "admmq_local_search", allow=(OK, WARN_MOVE_CAP))
        return (rep if report else None), st

    def pair_swap(self, W0, bits, group_size, codes, scale, zero, pairs, Wq=None, accept_tol: float = 1e-6,
                  report: bool = True):
        """pairs: int32 device tensor [rounds, batch, 2] of candidate row pairs (the caller's random draws)."""
        assert pairs.dtype == torch.int32 and pairs.dim() == 3 and pairs.shape[2] == 2
        cfg = PairSwapCfg(C.sizeof(PairSwapCfg), bits, group_size, pairs.shape[0], pairs.shape[1],
                          pairs.data_ptr() if pairs.numel() else None, accept_tol)
        rep = Report()
        st = self.lib.admmq_pair_swap(self.h, _ptr(W0), W0.shape[0], C.byref(cfg), _ptr(codes), _ptr(scale),
                                      _ptr(zero), _ptr(Wq), C.byref(rep) if report else None)
        _check(st, "admmq_pair_swap")
        return (rep if report else None), st

    def objective(self, W0, group_size, codes, scale, zero) -> float:
        out = C.c_double(0.0)
        _check(self.lib.admmq_objective(self.h, _ptr(W0), W0.shape[0], group_size, _ptr(codes), _ptr(scale),
                                        _ptr(zero), C.byref(out)), "admmq_objective")
        return out.value

    def get_hessian(self):
        H = torch.empty(self.d_in, self.d_in, dtype=torch.float32, device=self.device)
        s = torch.empty(self.d_in, dtype=torch.float32, device=self.device)
        _check(self.lib.admmq_get_hessian(self.h, _ptr(H), _ptr(s)), "admmq_get_hessian")
        return H, s

    def get_factor(self):
        """(Q^T [n, n], diag(T) [n], offdiag(T) [n]) in fp64, copies of the factorisation H~ = Q T Q^T."""
        n = self.d_in
        QT = torch.empty(n, n, dtype=torch.float64, device=self.device)
        td = torch.empty(n, dtype=torch.float64, device=self.device)
        te = torch.empty(n, dtype=torch.float64, device=self.device)
        _check(self.lib.admmq_get_factor(self.h, _ptr(QT), _ptr(td), _ptr(te)), "admmq_get_factor")
        return QT, td, te

    def set_timing(self, on: bool):
        _check(self.lib.admmq_set_timing(self.h, int(on)), "admmq_set_timing")

    def reset_timing(self):
        _check(self.lib.admmq_reset_timing(self.h), "admmq_reset_timing")

    def get_timing(self) -> dict:
        """{kind name: (total ms, launches)} since the last reset (synchronises)."""
        out = {}
        for k, name in enumerate(TIMING_NAMES):
            ms, cnt = C.c_double(0.0), C.c_longlong(0)
            _check(self.lib.admmq_get_timing(self.h, k, C.byref(ms), C.byref(cnt)), "admmq_get_timing")
            out[name] = (ms.value, cnt.value)
        return out

    def launch_count(self) -> int:
        return int(self.lib.admmq_launch_count(self.h))

    def test_set_wait(self, wait_limit_cycles: int = 2_000_000_000, hold_loads: bool = False):
        """Failure-handling tests only: bound of the product kernel's device-side waits, and whether its
        producer withholds every load (admmq_testing.h)."""
        _check(self.lib.admmq_test_set_wait(self.h, int(wait_limit_cycles), int(hold_loads)),
               "admmq_test_set_wait")


def objective_static(H: torch.Tensor, W0: torch.Tensor, group_size: int, codes: torch.Tensor,
                     scale: torch.Tensor, zero: torch.Tensor, out: torch.Tensor,
                     stream: Optional[torch.cuda.Stream] = None) -> int:
    """admmq_objective_static: the layer error into `out` (one device double) without any context,
    workspace or allocation inside the library -- for callers whose device memory is all spoken for.
    Returns the status; asynchronous on `stream` (default: the current stream).  The call is made with the
    tensors' device current, as the entry point requires."""
    lib = load_library()
    assert out.dtype == torch.float64 and out.is_cuda and out.numel() == 1
    with torch.cuda.device(W0.device):
        sp = C.c_void_p(stream.cuda_stream if stream is not None else
                        torch.cuda.current_stream(W0.device).cuda_stream)
        return lib.admmq_objective_static(_ptr(H), H.shape[0], _ptr(W0), W0.shape[0], group_size, _ptr(codes),
                                          _ptr(scale), _ptr(zero), _ptr(out), sp)
