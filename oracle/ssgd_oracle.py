"""ctypes/numpy wrapper around the plain C++ oracle (ssgd_oracle.cpp) -- TEST INFRASTRUCTURE ONLY.

Argument marshalling only: every number comes out of the C++ functions, which follow Algorithm 3
(lines 5-13) and Algorithm 4 of the paper step by step.  Arrays are numpy, C-contiguous, on the host.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ssgd_oracle.cpp")
_HDR = os.path.join(_HERE, "ssgd_oracle.h")
_LIB = os.path.join(_HERE, "libssgd_oracle.so")
_lock = threading.Lock()
_lib = None

MAX_R = 15


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA).  -ffp-contract=off: nothing fuses but the explicit fmaf."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC", "-shared", "-Wall",
             "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = C.CDLL(build())
            vp, i64, i32, u64, f32 = C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_float
            sig = {
                "ssgd_oracle_derive_params": [u64, i32, vp],
                "ssgd_oracle_create": [C.POINTER(vp), i64, i32, i64, i64, i32, u64],
                "ssgd_oracle_get_params": [vp, vp],
                "ssgd_oracle_set_params": [vp, vp],
                "ssgd_oracle_hashes": [vp, i64, vp, vp, vp],
                "ssgd_oracle_accumulate": [vp, vp, i64, f32, vp, vp, i64],
                "ssgd_oracle_sketch_f32": [vp, vp, vp, vp],
                "ssgd_oracle_sketch_f64": [vp, vp, vp, vp],
                "ssgd_oracle_sketch_workers": [vp, vp, i64, vp, vp, vp],
                "ssgd_oracle_estimate": [vp, vp, vp],
                "ssgd_oracle_select": [i64, vp, vp, i64, vp],
                "ssgd_oracle_second_round": [vp, vp, i64, vp, i64, vp],
                "ssgd_oracle_zero": [vp, vp, vp, i64, vp, i64],
                "ssgd_oracle_step": [vp, vp, i64, f32, vp, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, i32],
                "ssgd_oracle_fill_priority": [u64, i64, vp, vp],
                "ssgd_oracle_l2_estimate": [vp, vp, vp],
                "ssgd_oracle_heavymix": [vp, vp, vp, i64, u64, vp, vp, vp, vp],
                "ssgd_oracle_quantize16": [i64, vp, i32, vp],
                "ssgd_oracle_merge16": [i32, i64, vp, i32, vp],
            }
            for name, args in sig.items():
                fn = getattr(lib, name)
                fn.argtypes = args
                fn.restype = C.c_int
            lib.ssgd_oracle_destroy.argtypes = [vp]
            lib.ssgd_oracle_destroy.restype = None
            _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a, dtype, name):
    if not isinstance(a, np.ndarray) or a.dtype != dtype or not a.flags["C_CONTIGUOUS"]:
        raise TypeError(f"{name}: need a C-contiguous numpy array of {np.dtype(dtype)}")
    return a


def _ok(code, what):
    if code != 0:
        raise ValueError(f"oracle: {what} failed with code {code}")


def derive_params(seed: int, r: int) -> np.ndarray:
    """[r][4] uint32: a_j, b_j, a'_j, b'_j from the seed."""
    out = np.zeros((r, 4), np.uint32)
    _ok(_load().ssgd_oracle_derive_params(seed, r, _ptr(out)), "derive_params")
    return out


def select(val: np.ndarray, m: int, ids: np.ndarray | None = None) -> np.ndarray:
    """Positions of the m best items under (|val| descending on fp32 bits, id ascending), best first."""
    val = _chk(np.ascontiguousarray(val, np.float32), np.float32, "val")
    if ids is not None:
        ids = _chk(np.ascontiguousarray(ids, np.int32), np.int32, "ids")
    out = np.zeros(m, np.int32)
    _ok(_load().ssgd_oracle_select(val.size, _ptr(val), _ptr(ids), m, _ptr(out)), "select")
    return out


def fill_priority(seed: int, idx) -> np.ndarray:
    """Random-fill priorities of HEAVYMIX (Algorithm 1 line 4) for the listed coordinates."""
    idx = np.ascontiguousarray(idx, np.int64)
    out = np.zeros(idx.size, np.uint32)
    _ok(_load().ssgd_oracle_fill_priority(seed, idx.size, _ptr(idx), _ptr(out)), "fill_priority")
    return out


FMT_F16, FMT_BF16 = 0, 1


def quantize16(x, fmt: int) -> np.ndarray:
    """fp32 -> 16-bit encodings (uint16), round to nearest even; fmt 0 = binary16 (saturating), 1 = bfloat16."""
    x = np.ascontiguousarray(x, np.float32)
    q = np.zeros(x.shape, np.uint16)
    _ok(_load().ssgd_oracle_quantize16(x.size, _ptr(x), fmt, _ptr(q)), "quantize16")
    return q


def merge16(q16, fmt: int) -> np.ndarray:
    """[W][...] uint16 encodings -> fp32 sum over the first axis, in worker order."""
    q16 = np.ascontiguousarray(q16, np.uint16)
    W = q16.shape[0]
    out = np.zeros(q16.shape[1:], np.float32)
    _ok(_load().ssgd_oracle_merge16(W, out.size, _ptr(q16), fmt, _ptr(out)), "merge16")
    return out


class Oracle:
    """One problem shape (d, r, c, k, W, seed) of Algorithm 3 with the Count Sketch of Algorithm 4."""

    def __init__(self, d, r, c, k, W, seed):
        self._lib = _load()
        h = C.c_void_p()
        _ok(self._lib.ssgd_oracle_create(C.byref(h), d, r, c, k, W, seed), "create")
        self._h = h
        self.d, self.r, self.c, self.k, self.W, self.seed = d, r, c, k, W, seed

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            self._lib.ssgd_oracle_destroy(h)

    # ---- hash functions (Algorithm 4 line 2) -------------------------------------------------
    def params(self) -> np.ndarray:
        out = np.zeros((self.r, 4), np.uint32)
        _ok(self._lib.ssgd_oracle_get_params(self._h, _ptr(out)), "get_params")
        return out

    def set_params(self, p) -> None:
        p = np.ascontiguousarray(p, np.uint32).reshape(self.r, 4)
        _ok(self._lib.ssgd_oracle_set_params(self._h, _ptr(p)), "set_params")

    def hashes(self, idx):
        """(h, s): int32 [r][n] bucket and sign (+1/-1) of each listed coordinate."""
        idx = np.ascontiguousarray(idx, np.int64)
        h = np.zeros((self.r, idx.size), np.int32)
        s = np.zeros((self.r, idx.size), np.int32)
        _ok(self._lib.ssgd_oracle_hashes(self._h, idx.size, _ptr(idx), _ptr(h), _ptr(s)), "hashes")
        return h, s

    # ---- stages ------------------------------------------------------------------------------
    def _state(self, a, name):
        _chk(a, np.float32, name)
        if a.ndim != 2 or a.shape[0] != self.W or a.shape[1] < self.d:
            raise ValueError(f"{name}: need shape [W][ld>=d]")
        return a

    def accumulate(self, g, rho, u, v) -> None:
        """Algorithm 3 lines 5-6, in place on u and v."""
        self._state(g, "g"); self._state(u, "u"); self._state(v, "v")
        if u.shape != v.shape:
            raise ValueError("u and v must have one shape")
        _ok(self._lib.ssgd_oracle_accumulate(self._h, _ptr(g), g.shape[1], rho, _ptr(u), _ptr(v),
                                             u.shape[1]), "accumulate")

    def sketch(self, x, with_mass=False):
        """Algorithm 4 update() over one vector x[d] (fp32 or fp64): fp64 table [r][c] (and L1 mass)."""
        x = np.ascontiguousarray(x)
        if x.shape != (self.d,):
            raise ValueError("x: need shape [d]")
        T = np.zeros((self.r, self.c), np.float64)
        M = np.zeros((self.r, self.c), np.float64) if with_mass else None
        if x.dtype == np.float32:
            _ok(self._lib.ssgd_oracle_sketch_f32(self._h, _ptr(x), _ptr(T), _ptr(M)), "sketch")
        elif x.dtype == np.float64:
            _ok(self._lib.ssgd_oracle_sketch_f64(self._h, _ptr(x), _ptr(T), _ptr(M)), "sketch")
        else:
            raise TypeError("x: float32 or float64")
        return (T, M) if with_mass else T

    def sketch_workers(self, v, per_worker=False):
        """Algorithm 3 lines 7-8: (T, M[, Tw]) -- summed fp64 table, bucket L1 mass, per-worker tables."""
        self._state(v, "v")
        T = np.zeros((self.r, self.c), np.float64)
        M = np.zeros((self.r, self.c), np.float64)
        Tw = np.zeros((self.W, self.r, self.c), np.float64) if per_worker else None
        _ok(self._lib.ssgd_oracle_sketch_workers(self._h, _ptr(v), v.shape[1], _ptr(T), _ptr(M),
                                                 _ptr(Tw)), "sketch_workers")
        return (T, M, Tw) if per_worker else (T, M)

    def estimate(self, Tf) -> np.ndarray:
        """Algorithm 4 estimate() for every coordinate, from an fp32 [r][c] table."""
        Tf = _chk(np.ascontiguousarray(Tf, np.float32), np.float32, "Tf")
        if Tf.shape != (self.r, self.c):
            raise ValueError("Tf: need shape [r][c]")
        est = np.zeros(self.d, np.float32)
        _ok(self._lib.ssgd_oracle_estimate(self._h, _ptr(Tf), _ptr(est)), "estimate")
        return est

    def second_round(self, v, cand) -> np.ndarray:
        """Algorithm 3 line 10: fp64 sums over workers of v at the candidates."""
        self._state(v, "v")
        cand = np.ascontiguousarray(cand, np.int32)
        xs = np.zeros(cand.size, np.float64)
        _ok(self._lib.ssgd_oracle_second_round(self._h, _ptr(v), v.shape[1], _ptr(cand), cand.size,
                                               _ptr(xs)), "second_round")
        return xs

    def final_topk(self, cand, xs):
        """Algorithm 3 line 11 on given candidates and their exact sums: (out_idx[k], out_val[k])."""
        cand = np.ascontiguousarray(cand, np.int32)
        xsf = np.asarray(xs).astype(np.float32)
        best = select(xsf, self.k, cand)
        return cand[best].copy(), xsf[best].copy()

    def zero(self, u, v, idx) -> None:
        """Algorithm 3 line 13, in place."""
        self._state(u, "u"); self._state(v, "v")
        idx = np.ascontiguousarray(idx, np.int32)
        _ok(self._lib.ssgd_oracle_zero(self._h, _ptr(u), _ptr(v), u.shape[1], _ptr(idx), idx.size),
            "zero")

    def step(self, g, rho, u, v, ncand, zero_state=True, full=False):
        """Algorithm 3 lines 5-13.  Returns a dict with out_idx, out_val (best first) and, if full,
        T, M (fp64 [r][c]), est (fp32 [d]), cand (best first) and xs (fp64, aligned with cand)."""
        self._state(g, "g"); self._state(u, "u"); self._state(v, "v")
        out_idx = np.zeros(self.k, np.int32)
        out_val = np.zeros(self.k, np.float32)
        T = M = est = cand = xs = None
        if full:
            T = np.zeros((self.r, self.c), np.float64)
            M = np.zeros((self.r, self.c), np.float64)
            est = np.zeros(self.d, np.float32)
            cand = np.zeros(ncand, np.int32)
            xs = np.zeros(ncand, np.float64)
        _ok(self._lib.ssgd_oracle_step(self._h, _ptr(g), g.shape[1], rho, _ptr(u), _ptr(v), u.shape[1],
                                       ncand, _ptr(out_idx), _ptr(out_val), _ptr(T), _ptr(M), _ptr(est),
                                       _ptr(cand), _ptr(xs), 1 if zero_state else 0), "step")
        return dict(out_idx=out_idx, out_val=out_val, T=T, M=M, est=est, cand=cand, xs=xs)

    # ---- Algorithm 1 (HEAVYMIX) --------------------------------------------------------------------
    def l2_estimate(self, Tf) -> float:
        """Line 1: median over rows of the row's sum of squares."""
        Tf = _chk(np.ascontiguousarray(Tf, np.float32), np.float32, "Tf")
        out = C.c_double()
        _ok(self._lib.ssgd_oracle_l2_estimate(self._h, _ptr(Tf), C.byref(out)), "l2_estimate")
        return out.value

    def heavymix(self, Tf, v, fill_seed):
        """Lines 1-5: dict(out_idx ascending, out_val, l2, nheavy)."""
        Tf = _chk(np.ascontiguousarray(Tf, np.float32), np.float32, "Tf")
        self._state(v, "v")
        out_idx = np.zeros(self.k, np.int32)
        out_val = np.zeros(self.k, np.float32)
        l2 = C.c_double()
        nh = C.c_int64()
        _ok(self._lib.ssgd_oracle_heavymix(self._h, _ptr(Tf), _ptr(v), v.shape[1], fill_seed, _ptr(out_idx),
                                           _ptr(out_val), C.byref(l2), C.byref(nh)), "heavymix")
        return dict(out_idx=out_idx, out_val=out_val, l2=l2.value, nheavy=nh.value)
