"""Thin ctypes binding over libfd.so: same names as include/fd.h, argument marshalling only.

PyTorch is used for device memory and streams, nothing else: every step of the path runs in
the library's own CUDA kernels.  There is no CPU fallback; if the library cannot be loaded the
import fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_int32, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfd.so")

FD_OK, FD_ERR_INVALID, FD_ERR_WORKSPACE, FD_ERR_CUDA, FD_ERR_NOT_CONVERGED = 0, 1, 2, 3, 4
FD_ERR_PERRON_WALL, FD_ERR_UNSUPPORTED, FD_ERR_TIMEOUT, FD_ERR_NONFINITE, FD_ERR_COMM = 5, 6, 7, 8, 9
FD_PREC_FP32, FD_PREC_FAST = 0, 1
FD_PATH_AUTO, FD_PATH_SIMT, FD_PATH_TC = 0, 1, 2
FD_FLOW_VERTEX, FD_FLOW_PERRON_WALL, FD_FLOW_LEFT_EDGE, FD_FLOW_RIGHT_EDGE = 0, 1, 2, 3
FLOW_OUTCOMES = {0: "VERTEX", 1: "PERRON_WALL", 2: "LEFT_EDGE", 3: "RIGHT_EDGE"}

# Every symbol include/fd.h declares (checked by the CPU test-suite against the header).
EXPORTS = [
    "fd_workspace_bytes", "fd_create", "fd_destroy", "fd_set_option", "fd_get_option", "fd_beta0", "fd_degree",
    "fd_apply", "fd_apply_general", "fd_synchronize", "fd_eigs", "fd_beta_flow", "fd_beta_flow_cascade", "fd_nystrom", "fd_ladder_start", "fd_scale_by_degree",
    "fd_apply_general_static", "fd_unit_peaks", "fd_shard_rows", "fd_shard_exchange_bytes", "fd_set_shard", "fd_status_string", "fd_last_error", "fd_version", "fd_launch_count",
]


class fd_eigs_info(Structure):
    _fields_ = [("applies", c_int32), ("restarts", c_int32), ("converged", c_int32), ("basis_cols", c_int32),
                ("max_residual", c_double), ("seconds_apply", c_double), ("seconds_total", c_double)]


class fd_unit_rates(Structure):
    _fields_ = [("sm_count", c_int32)] + [(n, c_double) for n in (
        "ex2_per_clk_sm", "ffma_per_clk_sm", "cvt_f16x2_per_clk_sm", "lop_per_clk_sm", "fadd_per_clk_sm",
        "clk_mma_ts_n64", "clk_mma_ts_n128", "clk_mma_ss_n64", "clk_mma_ss_n128")]


class fd_probe(Structure):
    _fields_ = [(n, c_double) for n in ("beta", "S_off", "S_off_2beta", "n_eff", "d_hat", "V_bias", "V_stat", "V_mach",
                                        "V", "g_P", "lambda1")] + [("applies", c_int32), ("flags", c_int32)]


class fd_flow_opts(Structure):
    _fields_ = [("beta_start", c_double), ("beta_max", c_double), ("ratio", c_double), ("alpha", c_double),
                ("eta", c_double), ("tol", c_double), ("k", c_int32), ("b", c_int32), ("max_applies", c_int32),
                ("warm_start", c_int32)]


class fd_cascade_stage(Structure):
    _fields_ = [("prec", c_int32), ("eta", c_double), ("tol", c_double)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                          "(the CUDA library is the product; there is no fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.fd_workspace_bytes.argtypes = [c_int64, c_int32, c_int32, c_int32]
    lib.fd_workspace_bytes.restype = c_size_t
    lib.fd_create.argtypes = [POINTER(c_void_p), c_void_p, c_int64, c_int32, c_int64, c_int32, c_int32, c_int32,
                              c_void_p, c_size_t, c_void_p]
    lib.fd_destroy.argtypes = [c_void_p]
    lib.fd_set_option.argtypes = [c_void_p, c_char_p, c_double]
    lib.fd_get_option.argtypes = [c_void_p, c_char_p, POINTER(c_double)]
    lib.fd_beta0.argtypes = [c_void_p, POINTER(c_double)]
    lib.fd_degree.argtypes = [c_void_p, c_double, c_double, c_int32, c_void_p, c_void_p, c_void_p,
                              POINTER(c_double), POINTER(c_double)]
    lib.fd_synchronize.argtypes = [c_void_p]
    lib.fd_apply.argtypes = [c_void_p, c_void_p, c_int64, c_int32, c_void_p, c_int64, c_int32]
    lib.fd_apply_general.argtypes = [c_void_p, c_double, c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_void_p,
                                     c_int64, c_int32, c_void_p, c_int64, c_int32]
    lib.fd_eigs.argtypes = [c_void_p, c_int32, c_int32, c_double, c_int32, c_void_p, c_int64, c_int32,
                            POINTER(c_double), c_void_p, c_int64, POINTER(fd_eigs_info)]
    lib.fd_beta_flow.argtypes = [c_void_p, POINTER(fd_flow_opts), c_void_p, c_int64, c_int32, POINTER(fd_probe),
                                 POINTER(c_int32), POINTER(c_int32), POINTER(c_double), POINTER(c_double), c_void_p,
                                 c_int64]
    lib.fd_beta_flow_cascade.argtypes = [c_void_p, POINTER(fd_flow_opts), POINTER(fd_cascade_stage), c_int32, c_void_p,
                                         c_int64, c_int32, POINTER(fd_probe), POINTER(c_int32), POINTER(c_int32),
                                         POINTER(c_int32), POINTER(c_double), POINTER(c_double), c_void_p, c_int64]
    lib.fd_nystrom.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_int64, c_int32, POINTER(c_double),
                               c_void_p, c_int64]
    lib.fd_ladder_start.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_int64, c_int32, POINTER(c_double),
                                    c_void_p, c_int64]
    lib.fd_ladder_start.restype = c_int32
    lib.fd_scale_by_degree.argtypes = [c_void_p, c_void_p, c_int64, c_int32, c_double, c_void_p, c_int64]
    for name in ("fd_synchronize", "fd_create", "fd_destroy", "fd_set_option", "fd_get_option", "fd_beta0", "fd_degree", "fd_apply",
                 "fd_apply_general", "fd_eigs", "fd_beta_flow", "fd_beta_flow_cascade", "fd_nystrom", "fd_scale_by_degree"):
        getattr(lib, name).restype = c_int32
    lib.fd_apply_general_static.argtypes = [c_void_p, c_int64, c_int32, c_int64, c_double, c_void_p, c_void_p, c_void_p,
                                            c_int64, c_int32, c_void_p, c_int64, c_void_p, ctypes.c_char_p, c_size_t]
    lib.fd_apply_general_static.restype = c_int32
    lib.fd_unit_peaks.argtypes = [c_void_p, c_size_t, c_void_p, POINTER(fd_unit_rates)]
    lib.fd_unit_peaks.restype = c_int32
    lib.fd_status_string.argtypes = [c_int32]
    lib.fd_status_string.restype = c_char_p
    lib.fd_last_error.argtypes = [c_void_p]
    lib.fd_last_error.restype = c_char_p
    lib.fd_version.restype = c_int32
    lib.fd_launch_count.restype = c_int64
    return lib


lib = _load()


class FdError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        msg = lib.fd_status_string(status).decode()
        super().__init__(f"fd status {status} ({msg})" + (f": {detail}" if detail else ""))


def fd_workspace_bytes(N: int, D: int, b_max: int, m_max: int) -> int:
    return int(lib.fd_workspace_bytes(N, D, b_max, m_max))


def fd_launch_count() -> int:
    return int(lib.fd_launch_count())


def fd_version() -> int:
    return int(lib.fd_version())


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _colmajor(rows: int, cols: int, device) -> torch.Tensor:
    """(rows x cols) float32 tensor whose storage is column-major (ld = rows)."""
    return torch.empty((cols, rows), dtype=torch.float32, device=device).t()


def _ld(t: torch.Tensor) -> int:
    """Leading dimension of a column-major 2-D (or 1-D) float32 tensor."""
    if t.dim() == 1:
        return t.shape[0]
    assert t.dim() == 2 and t.stride(0) == 1, "blocks must be column-major (use .t() of a contiguous (cols, rows) tensor)"
    return t.stride(1) if t.shape[1] > 1 else max(t.shape[0], t.stride(1))


class Context:
    """One data set on one GPU.  Methods mirror the C entry points one to one."""

    def __init__(self, X: torch.Tensor, b_max: int = 64, m_max: int = 0, center: bool = True, stream=None):
        assert X.is_cuda and X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1
        self.N, self.D = int(X.shape[0]), int(X.shape[1])
        self.device = X.device
        self.b_max, self.m_max = int(b_max), int(m_max)
        nbytes = fd_workspace_bytes(self.N, self.D, b_max, m_max)
        if nbytes == 0:
            raise FdError(FD_ERR_INVALID, "fd_workspace_bytes rejected the shape")
        self.workspace_bytes = nbytes
        with torch.cuda.device(self.device):
            self._ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            off = (-self._ws.data_ptr()) % 256
            self._stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            h = c_void_p()
            st = lib.fd_create(byref(h), _ptr(X), self.N, self.D, X.stride(0), 1 if center else 0, b_max, m_max,
                               c_void_p(self._ws.data_ptr() + off), nbytes, c_void_p(self._stream.cuda_stream))
        if st != FD_OK:
            raise FdError(st)
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib.fd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, ok=(FD_OK,)):
        if st not in ok:
            shard = getattr(self, "_shard", None)
            if st == FD_ERR_COMM and shard is not None and shard.error is not None:
                err, shard.error = shard.error, None
                raise FdError(st, lib.fd_last_error(self._h).decode()) from err
            raise FdError(st, lib.fd_last_error(self._h).decode())
        return st

    def set_shard(self, shard):
        """Row-sharded operation (fd_set_shard): `shard` is a shard.Shard built for this context's (N, b_max), or
        None to return to unsharded operation.  The context keeps the shard (buffer and callbacks) alive."""
        if shard is not None:
            assert shard.N == self.N and shard.b_max >= self.b_max
        self._check(lib.fd_set_shard(self._h, ctypes.byref(shard.struct) if shard is not None else None))
        self._shard = shard

    def set_option(self, name: str, value: float):
        self._check(lib.fd_set_option(self._h, name.encode(), float(value)))

    def get_option(self, name: str) -> float:
        v = c_double()
        self._check(lib.fd_get_option(self._h, name.encode(), byref(v)))
        return v.value

    def beta0(self) -> float:
        v = c_double()
        self._check(lib.fd_beta0(self._h, byref(v)))
        return v.value

    def degree(self, beta: float, alpha: float, prec: int = FD_PREC_FP32):
        """Returns (q, d, s, S_off(beta), S_off(2 beta))."""
        q, d, s = (torch.empty(self.N, dtype=torch.float32, device=self.device) for _ in range(3))
        so, so2 = c_double(), c_double()
        with torch.cuda.device(self.device):
            self._check(lib.fd_degree(self._h, beta, alpha, prec, _ptr(q), _ptr(d), _ptr(s), byref(so), byref(so2)))
        return q, d, s, so.value, so2.value

    def synchronize(self):
        with torch.cuda.device(self.device):
            self._check(lib.fd_synchronize(self._h))

    def apply(self, V: torch.Tensor, out: torch.Tensor | None = None, prec: int = FD_PREC_FP32) -> torch.Tensor:
        if V.dim() == 1:
            V = V[:, None]
        b = V.shape[1]
        Y = out if out is not None else _colmajor(self.N, b, self.device)
        with torch.cuda.device(self.device):
            self._check(lib.fd_apply(self._h, _ptr(V), _ld(V), b, _ptr(Y), _ld(Y), prec))
        return Y

    def apply_general(self, beta: float, V: torch.Tensor | None, left=None, right=None, Xrow=None,
                      out: torch.Tensor | None = None, prec: int = FD_PREC_FP32) -> torch.Tensor:
        if V is not None and V.dim() == 1:
            V = V[:, None]
        b = 1 if V is None else V.shape[1]
        nrow = self.N if Xrow is None else int(Xrow.shape[0])
        Y = out if out is not None else _colmajor(nrow, b, self.device)
        with torch.cuda.device(self.device):
            self._check(lib.fd_apply_general(self._h, beta, _ptr(left), _ptr(right), _ptr(Xrow), nrow,
                                             0 if Xrow is None else Xrow.stride(0), _ptr(V),
                                             self.N if V is None else _ld(V), b, _ptr(Y), _ld(Y), prec))
        return Y

    def eigs(self, k: int, b: int, tol: float = 1e-6, max_applies: int = 1000, Q0: torch.Tensor | None = None,
             allow_not_converged: bool = False):
        """Returns (evals[k+1] float64 numpy, evecs N x (k+1) column-major tensor, info)."""
        import numpy as np
        ev = (c_double * (k + 1))()
        U = _colmajor(self.N, k + 1, self.device)
        info = fd_eigs_info()
        with torch.cuda.device(self.device):
            st = lib.fd_eigs(self._h, k, b, tol, max_applies, _ptr(Q0), 0 if Q0 is None else _ld(Q0),
                             0 if Q0 is None else Q0.shape[1], ev, _ptr(U), _ld(U), byref(info))
        self._check(st, ok=(FD_OK, FD_ERR_NOT_CONVERGED) if allow_not_converged else (FD_OK,))
        return np.array(ev[:], dtype=np.float64), U, info

    def beta_flow(self, k: int, b: int, alpha: float, beta_start: float = 0.0, beta_max: float = 1000.0,
                  tol: float = 1e-6, max_applies: int = 2000, warm_start: bool = True, eta: float = 0.0,
                  Q0: torch.Tensor | None = None, max_probes: int = 64):
        """Returns (beta_x, outcome name, evals, evecs, list of probe dicts)."""
        import numpy as np
        opts = fd_flow_opts(beta_start, beta_max, 2.0, alpha, eta, tol, k, b, max_applies, 1 if warm_start else 0)
        log = (fd_probe * max_probes)()
        n = c_int32(max_probes)
        outcome = c_int32()
        bx = c_double()
        ev = (c_double * (k + 1))()
        U = _colmajor(self.N, k + 1, self.device)
        with torch.cuda.device(self.device):
            st = lib.fd_beta_flow(self._h, byref(opts), _ptr(Q0), 0 if Q0 is None else _ld(Q0),
                                  0 if Q0 is None else Q0.shape[1], log, byref(n), byref(outcome), byref(bx), ev,
                                  _ptr(U), _ld(U))
        self._check(st)
        recs = [{f[0]: getattr(log[i], f[0]) for f in fd_probe._fields_} for i in range(n.value)]
        return bx.value, FLOW_OUTCOMES[outcome.value], np.array(ev[:], dtype=np.float64), U, recs

    def beta_flow_cascade(self, k: int, b: int, alpha: float, stages, beta_start: float = 0.0, beta_max: float = 1000.0,
                          max_applies: int = 2000, warm_start: bool = True, Q0: torch.Tensor | None = None,
                          max_probes: int = 64):
        """stages: sequence of (precision, eta, tol) with eta / tol <= 0 for the mode's defaults.
        Returns (beta_x, outcome name, evals, evecs, [list of probe dicts per stage])."""
        import numpy as np
        opts = fd_flow_opts(beta_start, beta_max, 2.0, alpha, 0.0, 0.0, k, b, max_applies, 1 if warm_start else 0)
        ns = len(stages)
        st_arr = (fd_cascade_stage * ns)(*[fd_cascade_stage(int(p), float(e), float(t)) for p, e, t in stages])
        cap = max_probes * ns
        log = (fd_probe * cap)()
        n = c_int32(cap)
        first = (c_int32 * (ns + 1))()
        outcome = c_int32()
        bx = c_double()
        ev = (c_double * (k + 1))()
        U = _colmajor(self.N, k + 1, self.device)
        with torch.cuda.device(self.device):
            st = lib.fd_beta_flow_cascade(self._h, byref(opts), st_arr, ns, _ptr(Q0), 0 if Q0 is None else _ld(Q0),
                                          0 if Q0 is None else Q0.shape[1], log, byref(n), first, byref(outcome), byref(bx),
                                          ev, _ptr(U), _ld(U))
        self._check(st)
        recs = [[{f[0]: getattr(log[i], f[0]) for f in fd_probe._fields_} for i in range(first[s], first[s + 1])]
                for s in range(ns)]
        return bx.value, FLOW_OUTCOMES[outcome.value], np.array(ev[:], dtype=np.float64), U, recs

    def nystrom(self, Xnew: torch.Tensor, psi: torch.Tensor, evals) -> torch.Tensor:
        m = psi.shape[1]
        lam = (c_double * m)(*[float(v) for v in evals])
        out = _colmajor(int(Xnew.shape[0]), m, self.device)
        with torch.cuda.device(self.device):
            self._check(lib.fd_nystrom(self._h, _ptr(Xnew), Xnew.shape[0], Xnew.stride(0), _ptr(psi), _ld(psi), m, lam,
                                       _ptr(out), _ld(out)))
        return out

    def ladder_start(self, old: "Context", Xnew: torch.Tensor, evecs_old: torch.Tensor, evals) -> torch.Tensor:
        """Warm-start basis for this (new, larger) level from the eigenpairs of `old` (the level over its first rows)."""
        m = evecs_old.shape[1]
        lam = (c_double * m)(*[float(v) for v in evals])
        Q0 = _colmajor(self.N, m, self.device)
        with torch.cuda.device(self.device):
            self._check(lib.fd_ladder_start(old._h, self._h, _ptr(Xnew), Xnew.stride(0), _ptr(evecs_old), _ld(evecs_old), m,
                                            lam, _ptr(Q0), _ld(Q0)))
        return Q0

    def scale_by_degree(self, v: torch.Tensor, power: float) -> torch.Tensor:
        out = _colmajor(self.N, v.shape[1], self.device)
        with torch.cuda.device(self.device):
            self._check(lib.fd_scale_by_degree(self._h, _ptr(v), _ld(v), v.shape[1], power, _ptr(out), _ld(out)))
        return out


FD_STATIC_MAX_N, FD_STATIC_MAX_D, FD_STATIC_MAX_B = 8192, 32, 32


def fd_apply_general_static(X: torch.Tensor, beta: float, V: torch.Tensor, left=None, right=None,
                            out: torch.Tensor | None = None) -> torch.Tensor:
    """Y = diag(left) K(X, X) diag(right) V through the entry point that allocates nothing on the device: its
    scratch is the library's own fixed device array.  For callers that cannot allocate; sizes are limited to
    FD_STATIC_MAX_N / _D / _B, and calls must not overlap on the GPU.  `out` must be given by such a caller; when it
    is omitted here the binding allocates it for convenience (that allocation is the binding's, not the library's)."""
    assert X.is_cuda and X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1
    if V.dim() == 1:
        V = V[:, None]
    N, D, b = int(X.shape[0]), int(X.shape[1]), int(V.shape[1])
    Y = out if out is not None else _colmajor(N, b, X.device)
    err = ctypes.create_string_buffer(256)
    with torch.cuda.device(X.device):
        st = lib.fd_apply_general_static(_ptr(X), N, D, X.stride(0), float(beta), _ptr(left), _ptr(right), _ptr(V), _ld(V), b,
                                         _ptr(Y), _ld(Y), c_void_p(torch.cuda.current_stream(X.device).cuda_stream), err, 256)
    if st != FD_OK:
        raise FdError(st, err.value.decode())
    return Y


def fd_unit_peaks(device) -> dict:
    """Measured unit throughput of `device` (fd.h: fd_unit_peaks): rates per clock per SM and SM cycles per tcgen05.mma."""
    scratch = torch.empty(1 << 20, dtype=torch.uint8, device=device)
    out = fd_unit_rates()
    with torch.cuda.device(device):
        st = lib.fd_unit_peaks(_ptr(scratch), scratch.numel(), c_void_p(torch.cuda.current_stream(device).cuda_stream),
                               ctypes.byref(out))
    if st != FD_OK:
        raise FdError(st)
    return {n: getattr(out, n) for n, _ in fd_unit_rates._fields_}


def to_colmajor(a, device) -> torch.Tensor:
    """numpy (rows x cols) array -> column-major float32 device tensor."""
    import numpy as np
    a = np.asarray(a, dtype=np.float32)
    if a.ndim == 1:
        a = a[:, None]
    t = torch.from_numpy(np.ascontiguousarray(a.T)).to(device)
    return t.t()
