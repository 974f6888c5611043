"""Float64 CPU oracle for the plasticity-evaluation path (test infrastructure only).

This package wraps ``egeria_oracle.c`` (plain C, float64) with ctypes.  It is the
slow, obviously-correct definition that the CUDA library is compared against.
It shares no code with the CUDA path and must only be imported by the tests,
the smoke check and the benchmark's CPU-baseline leg -- never by the product.

Paper passages followed: Sec. 4.2.1 / Eq. 1 (SP loss = plasticity), Sec. 4.2.2 /
Eq. 2 (moving average), Sec. 4.2.2 + Algorithm 1 (window linear fit, stale
counter, freezing decision, frontmost-active module, learning-rate-based
unfreezing), Sec. 3 (end of the bootstrapping stage).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "egeria_oracle.c"
_LIB = _HERE / "libegeria_oracle.so"

EPS = 1e-12  # clamp on a row norm of the similarity matrix (all-zero sample)


def build(force: bool = False) -> Path:
    """Compile the oracle's C file with gcc (OpenMP on) if it is missing or stale."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_LIB))
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        i64 = ctypes.c_int64
        L.egeria_oracle_num_threads.restype = ctypes.c_int
        L.egeria_oracle_set_num_threads.argtypes = [ctypes.c_int]
        L.egeria_oracle_gram.argtypes = [u16p, i64, i64, f64p]
        L.egeria_oracle_gram.restype = ctypes.c_int
        L.egeria_oracle_gram_row.argtypes = [u16p, i64, i64, i64, f64p]
        L.egeria_oracle_gram_row.restype = ctypes.c_int
        L.egeria_oracle_row_normalise.argtypes = [f64p, i64, ctypes.c_double, f64p]
        L.egeria_oracle_frobenius_loss.argtypes = [f64p, f64p, i64]
        L.egeria_oracle_frobenius_loss.restype = ctypes.c_double
        L.egeria_oracle_sp_loss.argtypes = [u16p, u16p, i64, i64, ctypes.c_double,
                                            f64p, f64p, f64p]
        L.egeria_oracle_sp_loss.restype = ctypes.c_int
        L.egeria_oracle_smooth.argtypes = [f64p, i64, i64]
        L.egeria_oracle_smooth.restype = ctypes.c_double
        L.egeria_oracle_ols_slope.argtypes = [f64p, i64]
        L.egeria_oracle_ols_slope.restype = ctypes.c_double
        L.egeria_oracle_plasticity_replay.argtypes = [
            ctypes.POINTER(ctypes.c_float), i64, i64, ctypes.c_double, ctypes.c_int,
            f64p, f64p, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
        L.egeria_oracle_plasticity_replay.restype = ctypes.c_int
        i32p = ctypes.POINTER(ctypes.c_int32)
        L.egeria_oracle_plasticity_replay_auto.argtypes = [
            ctypes.POINTER(ctypes.c_float), i64, i64, ctypes.c_int, f64p, i32p, f64p]
        L.egeria_oracle_plasticity_replay_auto.restype = ctypes.c_int
        L.egeria_oracle_frontmost_replay.argtypes = [
            ctypes.POINTER(ctypes.c_float), i64, i64, i64, f64p, ctypes.c_int, ctypes.c_int, i32p, i32p, f64p]
        L.egeria_oracle_frontmost_replay.restype = ctypes.c_int
        L.egeria_oracle_bootstrap_replay.argtypes = [ctypes.POINTER(ctypes.c_float), i64, i64, ctypes.c_double, f64p]
        L.egeria_oracle_bootstrap_replay.restype = ctypes.c_int64
        u8p = ctypes.POINTER(ctypes.c_uint8)
        L.egeria_oracle_unfreeze_replay.argtypes = [
            ctypes.POINTER(ctypes.c_float), f64p, i64, i64, i64, f64p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            f64p, u8p, i32p, i32p]
        L.egeria_oracle_unfreeze_replay.restype = ctypes.c_int
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().egeria_oracle_num_threads())


def set_num_threads(n: int) -> None:
    lib().egeria_oracle_set_num_threads(int(n))


def _bits(a) -> np.ndarray:
    """A b x d array of bfloat16 bit patterns (uint16), C-contiguous."""
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16 or a.ndim != 2:
        raise TypeError("oracle inputs are 2-D uint16 arrays holding bfloat16 bits")
    return a


def _p(a: np.ndarray, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def gram(a_bits) -> np.ndarray:
    """Pair-wise similarity matrix G = A A^T of one b x d activation (Sec. 4.2.1)."""
    a = _bits(a_bits)
    b, d = a.shape
    g = np.empty((b, b), dtype=np.float64)
    if lib().egeria_oracle_gram(_p(a, ctypes.c_uint16), b, d, _p(g, ctypes.c_double)):
        raise MemoryError("oracle gram")
    return g


def gram_row(a_bits, i: int) -> np.ndarray:
    """Row i of G only (sampled checks at full workload sizes)."""
    a = _bits(a_bits)
    b, d = a.shape
    g = np.empty(b, dtype=np.float64)
    if lib().egeria_oracle_gram_row(_p(a, ctypes.c_uint16), b, d, int(i), _p(g, ctypes.c_double)):
        raise ValueError("oracle gram_row")
    return g


def row_normalise(g: np.ndarray, eps: float = EPS) -> np.ndarray:
    g = np.ascontiguousarray(g, dtype=np.float64)
    b = g.shape[0]
    out = np.empty_like(g)
    lib().egeria_oracle_row_normalise(_p(g, ctypes.c_double), b, eps, _p(out, ctypes.c_double))
    return out


def sp_loss(at_bits, ar_bits, eps: float = EPS, return_grams: bool = False):
    """Plasticity of one module: SP loss of (A_T, A_R) (Eq. 1)."""
    at, ar = _bits(at_bits), _bits(ar_bits)
    if at.shape != ar.shape:
        raise ValueError("A_T and A_R differ in shape")
    b, d = at.shape
    loss = ctypes.c_double()
    if return_grams:
        gt = np.empty((b, b), dtype=np.float64)
        gr = np.empty((b, b), dtype=np.float64)
        pt, pr = _p(gt, ctypes.c_double), _p(gr, ctypes.c_double)
    else:
        gt = gr = None
        pt = pr = None
    rc = lib().egeria_oracle_sp_loss(_p(at, ctypes.c_uint16), _p(ar, ctypes.c_uint16), b, d,
                                     eps, ctypes.byref(loss), pt, pr)
    if rc:
        raise RuntimeError(f"oracle sp_loss failed ({rc})")
    return (loss.value, gt, gr) if return_grams else loss.value


def sp_loss_batch(at_list, ar_list, eps: float = EPS) -> np.ndarray:
    """Plasticity of every monitored module of one evaluation."""
    return np.array([sp_loss(a, r, eps) for a, r in zip(at_list, ar_list)], dtype=np.float64)


def smooth(p, i: int, W: int) -> float:
    """Moving average of the last min(i+1, W) raw readings (Eq. 2)."""
    p = np.ascontiguousarray(p, dtype=np.float64)
    return float(lib().egeria_oracle_smooth(_p(p, ctypes.c_double), int(i), int(W)))


def ols_slope(y) -> float:
    """Least-squares slope of y against 0..n-1 (Sec. 4.2.2)."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    return float(lib().egeria_oracle_ols_slope(_p(y, ctypes.c_double), y.shape[0]))


def plasticity_replay(hist, W: int, T: float, signed_test: bool = False):
    """Algorithm 1 over one module's whole raw-loss history (float32 readings).

    Returns dict(smoothed[H], slopes[H], counter, freeze_eval, converged)."""
    h = np.ascontiguousarray(hist, dtype=np.float32)
    H = h.shape[0]
    sm = np.empty(max(H, 1), dtype=np.float64)
    sl = np.empty(max(H, 1), dtype=np.float64)
    cnt = ctypes.c_int32()
    fe = ctypes.c_int32()
    rc = lib().egeria_oracle_plasticity_replay(
        _p(h, ctypes.c_float), H, int(W), float(T), int(bool(signed_test)),
        _p(sm, ctypes.c_double), _p(sl, ctypes.c_double), ctypes.byref(cnt), ctypes.byref(fe))
    if rc < 0:
        raise RuntimeError(f"oracle replay failed ({rc})")
    return dict(smoothed=sm[:H], slopes=sl[:H], counter=cnt.value, freeze_eval=fe.value,
                converged=bool(rc))


def plasticity_replay_auto(hist, W: int, signed_test: bool = False):
    """Algorithm 1 with the per-module tolerance of Sec. 4.2.2: 20 % of the largest |slope| in
    the module's initial 3 readings.  Returns dict(slopes[H], freeze_eval, converged, T)."""
    h = np.ascontiguousarray(hist, dtype=np.float32)
    H = h.shape[0]
    sl = np.empty(max(H, 1), dtype=np.float64)
    fe = ctypes.c_int32()
    T = ctypes.c_double()
    rc = lib().egeria_oracle_plasticity_replay_auto(_p(h, ctypes.c_float), H, int(W), int(bool(signed_test)),
                                                    _p(sl, ctypes.c_double), ctypes.byref(fe), ctypes.byref(T))
    if rc < 0:
        raise RuntimeError(f"oracle replay_auto failed ({rc})")
    return dict(slopes=sl[:H], freeze_eval=fe.value, converged=bool(rc), T=T.value)


def frontmost_replay(hist, W: int, T=None, signed_test: bool = False):
    """Frontmost-active policy (Sec. 4.2.2, Algorithm 1 `l <- l + 1`) over [M, H] raw readings.
    T: per-module tolerances, or None for the automatic one.
    Returns dict(freeze_eval[M], monitored[H], slopes[H], frozen)."""
    h = np.ascontiguousarray(hist, dtype=np.float32)
    M, H = h.shape
    auto = T is None
    Tarr = np.zeros(M, dtype=np.float64) if auto else np.ascontiguousarray(np.broadcast_to(T, (M,)), dtype=np.float64)
    fe = np.empty(M, dtype=np.int32)
    mon = np.empty(max(H, 1), dtype=np.int32)
    sl = np.empty(max(H, 1), dtype=np.float64)
    rc = lib().egeria_oracle_frontmost_replay(_p(h, ctypes.c_float), M, H, int(W), _p(Tarr, ctypes.c_double),
                                              int(bool(signed_test)), int(auto), _p(fe, ctypes.c_int32),
                                              _p(mon, ctypes.c_int32), _p(sl, ctypes.c_double))
    if rc < 0:
        raise RuntimeError(f"oracle frontmost_replay failed ({rc})")
    return dict(freeze_eval=fe, monitored=mon[:H], slopes=sl[:H], frozen=int(rc))


def bootstrap_replay(loss_hist, W: int, rate_tol: float = 0.1):
    """End of the bootstrapping stage (Sec. 3, Sec. 4.2.2): first evaluation with a full window
    whose changing rate |slope| (W - 1) / |window mean| of the smoothed training loss is below
    rate_tol.  Returns dict(end, rates[H])."""
    h = np.ascontiguousarray(loss_hist, dtype=np.float32)
    H = h.shape[0]
    rates = np.empty(max(H, 1), dtype=np.float64)
    end = lib().egeria_oracle_bootstrap_replay(_p(h, ctypes.c_float), H, int(W), float(rate_tol),
                                               _p(rates, ctypes.c_double))
    if end < -1:
        raise RuntimeError("oracle bootstrap_replay: bad sizes")
    return dict(end=int(end), rates=rates[:H])


def unfreeze_replay(hist, lr, W: int, T=None, frontmost: bool = False, signed_test: bool = False):
    """Algorithm 1 with its learning-rate-based unfreezing (Sec. 4.2.2 "Unfreezing") over [M, H]
    raw readings and the learning rate lr[H] at each evaluation: once the learning rate is a
    tenth (or less) of what it was at the first freeze, all modules restart and W is halved
    (never below 2).  T: per-module tolerances, or None for the automatic one.
    Returns dict(slopes[M, H], frozen[H, M], window[H], restarted[H], restarts)."""
    h = np.ascontiguousarray(hist, dtype=np.float32)
    M, H = h.shape
    lr = np.ascontiguousarray(np.broadcast_to(lr, (H,)), dtype=np.float64)
    auto = T is None
    Tarr = np.zeros(M, dtype=np.float64) if auto else np.ascontiguousarray(np.broadcast_to(T, (M,)), dtype=np.float64)
    fz = np.zeros((max(H, 1), M), dtype=np.uint8)
    win = np.empty(max(H, 1), dtype=np.int32)
    rs = np.zeros(max(H, 1), dtype=np.int32)
    sl_c = np.empty(M * max(H, 1), dtype=np.float64)
    rc = lib().egeria_oracle_unfreeze_replay(_p(h, ctypes.c_float), _p(lr, ctypes.c_double), M, H, int(W),
                                             _p(Tarr, ctypes.c_double), int(bool(signed_test)), int(auto),
                                             int(bool(frontmost)), _p(sl_c, ctypes.c_double),
                                             _p(fz, ctypes.c_uint8), _p(win, ctypes.c_int32), _p(rs, ctypes.c_int32))
    if rc < 0:
        raise RuntimeError(f"oracle unfreeze_replay failed ({rc})")
    sl = sl_c[:M * H].reshape(M, H)
    return dict(slopes=sl, frozen=fz[:H], window=win[:H], restarted=rs[:H], restarts=int(rc))
