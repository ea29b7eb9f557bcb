"""ctypes front end of the DES-LOC CPU oracle (``desloc_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the test-suite, the smoke check and
the benchmark's CPU-baseline leg import this package.  It builds the C file
with gcc on first use and forwards numpy arrays to it; all of the method's
arithmetic lives in the C file (Algorithms 1-3 of the paper, plus the
post-average ordering of Algorithms 4-5).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

ADAM, ADOPT, SGDM = 0, 1, 2
SYNC_X, SYNC_U, SYNC_V = 1, 2, 4
FLAG_ADOPT_NORM_CLIP = 1
FLAG_POST_AVERAGE = 2
FLAG_ADOPT_AVG_NORMALISER = 4

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "desloc_oracle.c")
_LIB = os.path.join(_HERE, "libdesloc_oracle.so")
_lock = threading.Lock()
_lib = None


class OracleCfg(ctypes.Structure):
    _fields_ = [
        ("M", ctypes.c_int32),
        ("opt", ctypes.c_int32),
        ("beta1", ctypes.c_double),
        ("beta2", ctypes.c_double),
        ("eps", ctypes.c_double),
        ("weight_decay", ctypes.c_double),
        ("clip_rho", ctypes.c_double),
        ("Kx", ctypes.c_int32),
        ("Ku", ctypes.c_int32),
        ("Kv", ctypes.c_int32),
        ("flags", ctypes.c_uint32),
    ]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no fast-math) if it is stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-Wall", "-Wextra", "-shared",
                 "-fPIC", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def configure(L: ctypes.CDLL) -> ctypes.CDLL:
    """Declare the argument and result types of every oracle entry point on a loaded library."""
    L.desloc_oracle_sync_mask.restype = ctypes.c_uint32
    L.desloc_oracle_sync_mask.argtypes = [ctypes.c_int32] * 4 + [ctypes.c_int64]
    L.desloc_oracle_step.restype = ctypes.c_uint32
    L.desloc_oracle_step.argtypes = [
        ctypes.POINTER(OracleCfg), ctypes.c_int64, ctypes.c_double, ctypes.c_double,
        ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
        ctypes.c_void_p]
    L.desloc_oracle_step_scaled.restype = ctypes.c_uint32
    L.desloc_oracle_step_scaled.argtypes = L.desloc_oracle_step.argtypes + [ctypes.c_void_p]
    L.desloc_oracle_step_full.restype = ctypes.c_uint32
    L.desloc_oracle_step_full.argtypes = L.desloc_oracle_step_scaled.argtypes + [ctypes.c_void_p]
    L.desloc_oracle_tensor_norms.restype = None
    L.desloc_oracle_tensor_norms.argtypes = [ctypes.c_int32, ctypes.c_int64, ctypes.c_int32,
                                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                             ctypes.c_void_p, ctypes.c_void_p]
    L.desloc_oracle_norm_scales.restype = None
    L.desloc_oracle_norm_scales.argtypes = [ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                            ctypes.c_void_p, ctypes.c_double, ctypes.c_void_p,
                                            ctypes.c_void_p]
    L.desloc_oracle_worker_mean.restype = None
    L.desloc_oracle_worker_mean.argtypes = [ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                            ctypes.c_void_p, ctypes.c_void_p]
    L.desloc_oracle_rel_change.restype = None
    L.desloc_oracle_rel_change.argtypes = [ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    L.desloc_oracle_run.restype = None
    L.desloc_oracle_run.argtypes = [
        ctypes.POINTER(OracleCfg), ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
        ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    return L


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = configure(ctypes.CDLL(build()))
    return _lib


def make_cfg(M, opt, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, clip_rho=0.0,
             Kx=1, Ku=1, Kv=1, flags=0) -> OracleCfg:
    return OracleCfg(int(M), int(opt), float(beta1), float(beta2), float(eps),
                     float(weight_decay), float(clip_rho), int(Kx), int(Ku), int(Kv), int(flags))


def sync_mask(opt, Kx, Ku, Kv, t) -> int:
    return int(lib().desloc_oracle_sync_mask(int(opt), int(Kx), int(Ku), int(Kv), int(t)))


def _check(a, M, name, allow_none=False):
    if a is None:
        if allow_none:
            return None
        raise ValueError(f"{name} is required")
    if not (isinstance(a, np.ndarray) and a.dtype == np.float32 and a.ndim == 2
            and a.shape[0] == M and a.flags["C_CONTIGUOUS"]):
        raise ValueError(f"{name} must be a C-contiguous float32 array of shape [M, n]")
    return a.ctypes.data


def norm_scales(g, max_norm: float):
    """Per-worker gradient norms and norm-clip factors min(1, max_norm/||g^m||) for g of shape [M, n]."""
    M = g.shape[0]
    pg = _check(g, M, "g")
    norms = np.zeros(M, dtype=np.float64)
    scales = np.zeros(M, dtype=np.float64)
    lib().desloc_oracle_norm_scales(M, g.shape[1], g.shape[1], pg, float(max_norm),
                                    norms.ctypes.data, scales.ctypes.data)
    return norms, scales


def worker_mean(s):
    """E_m[s^m]: the fp32-rounded mean over workers of a float32 array of shape [M, n]."""
    M = s.shape[0]
    ps = _check(s, M, "s")
    out = np.zeros(s.shape[1], dtype=np.float32)
    lib().desloc_oracle_worker_mean(M, s.shape[1], s.shape[1], ps, out.ctypes.data)
    return out


def rel_change(now, then):
    """Per-worker ||now - then||_2 / ||then||_2 for float32 arrays of shape [M, n]."""
    M = now.shape[0]
    pn, pt = _check(now, M, "now"), _check(then, M, "then")
    out = np.zeros(M, dtype=np.float64)
    lib().desloc_oracle_rel_change(M, now.shape[1], now.shape[1], pn, pt, out.ctypes.data)
    return out


def tensor_norms(a, offs, numel):
    """L2 norms per (worker, tensor) and per worker of an [M, n] array (any float dtype, widened
    to fp64 exactly); tensor k is a[:, offs[k] : offs[k] + numel[k]].  Returns ([M, nt], [M])."""
    a64 = np.ascontiguousarray(a, dtype=np.float64)
    if a64.ndim != 2:
        raise ValueError("a must have shape [M, n]")
    M, n = a64.shape
    o = np.ascontiguousarray(offs, dtype=np.int64)
    c = np.ascontiguousarray(numel, dtype=np.int64)
    if o.shape != c.shape or o.ndim != 1 or np.any(o < 0) or np.any(o + c > n):
        raise ValueError("offs / numel do not fit the array")
    out = np.zeros((M, len(o)), dtype=np.float64)
    tot = np.zeros(M, dtype=np.float64)
    lib().desloc_oracle_tensor_norms(M, n, len(o), o.ctypes.data, c.ctypes.data, a64.ctypes.data,
                                     out.ctypes.data, tot.ctypes.data)
    return out, tot


def step(cfg: OracleCfg, t: int, lr: float, x, u, v, g, clip_bound: float = 0.0,
         gscale=None, d_out=None) -> int:
    """One step in place on float32 arrays of shape [M, n]; returns the sync mask.
    gscale: optional per-worker factors applied to g before the coordinate clip.
    d_out: optional float64 array [M, n] that receives every worker's update d_t."""
    M = cfg.M
    px, pu, pg = _check(x, M, "x"), _check(u, M, "u"), _check(g, M, "g")
    pv = _check(v, M, "v", allow_none=(cfg.opt == SGDM))
    n = x.shape[1]
    if u.shape != x.shape or g.shape != x.shape or (v is not None and v.shape != x.shape):
        raise ValueError("x, u, v, g must share one shape")
    if gscale is not None or d_out is not None:
        gs = None
        if gscale is not None:
            gs = np.ascontiguousarray(gscale, dtype=np.float64)
            assert gs.shape == (M,)
        if d_out is not None and not (isinstance(d_out, np.ndarray) and d_out.dtype == np.float64
                                      and d_out.shape == x.shape and d_out.flags["C_CONTIGUOUS"]):
            raise ValueError("d_out must be a C-contiguous float64 array shaped like x")
        return int(lib().desloc_oracle_step_full(
            ctypes.byref(cfg), int(t), float(lr), float(clip_bound), n, n, px, pu, pv, pg,
            gs.ctypes.data if gs is not None else None,
            d_out.ctypes.data if d_out is not None else None))
    return int(lib().desloc_oracle_step(ctypes.byref(cfg), int(t), float(lr), float(clip_bound),
                                        n, n, px, pu, pv, pg))


def run(cfg: OracleCfg, t0: int, lrs, x, u, v, g, clip_bounds=None):
    """T = len(lrs) steps in place; g has shape [T, M, n].  Returns the mask of every step."""
    M = cfg.M
    lrs = np.ascontiguousarray(lrs, dtype=np.float64)
    T = lrs.shape[0]
    if not (g.dtype == np.float32 and g.ndim == 3 and g.shape[0] == T and g.shape[1] == M
            and g.flags["C_CONTIGUOUS"] and g.shape[2] == x.shape[1]):
        raise ValueError("g must be a C-contiguous float32 array of shape [T, M, n]")
    px, pu = _check(x, M, "x"), _check(u, M, "u")
    pv = _check(v, M, "v", allow_none=(cfg.opt == SGDM))
    cb = None
    if clip_bounds is not None:
        cb = np.ascontiguousarray(clip_bounds, dtype=np.float64)
        assert cb.shape[0] == T
    masks = np.zeros(T, dtype=np.uint32)
    n = x.shape[1]
    lib().desloc_oracle_run(ctypes.byref(cfg), int(t0), T, lrs.ctypes.data,
                            cb.ctypes.data if cb is not None else None, n, n, px, pu, pv,
                            g.ctypes.data, masks.ctypes.data)
    return masks
