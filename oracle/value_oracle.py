"""Loader for the C value oracle (value_oracle.c).  TEST INFRASTRUCTURE ONLY:
imported by tests, the smoke check and the benchmark's CPU-baseline leg, never
by the product path.  Compiles the C file with gcc on first use."""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "value_oracle.c")
_LIB = os.path.join(_HERE, "libvalue_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.moe_oracle_tokens.restype = ctypes.c_int
        _lib.moe_oracle_tokens_single.restype = ctypes.c_int
        _lib.moe_oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_load().moe_oracle_threads())


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def forward_tokens(x: np.ndarray, expert: np.ndarray, gate: np.ndarray, w1: np.ndarray, w2: np.ndarray,
                   El: int, first_local: int, sel: np.ndarray, nthreads: int = 0
                   ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """x [R,T,d] bf16 bits; expert/gate [R,T,k]; w1 [El,2F,d]; w2 [El,d,F]; sel: flat token ids r*T+t.

    Returns (out [n,d] bf16 bits, y [n,kmax,d] bf16 bits, y_expert [n,kmax] int32)."""
    R, T, d = x.shape
    k = expert.shape[-1]
    F = w2.shape[-1]
    assert w1.shape == (El, 2 * F, d) and w2.shape == (El, d, F)
    kmax = min(k, El)
    x = np.ascontiguousarray(x, np.uint16)
    expert = np.ascontiguousarray(expert, np.int32)
    gate = np.ascontiguousarray(gate, np.float32)
    w1 = np.ascontiguousarray(w1, np.uint16)
    w2 = np.ascontiguousarray(w2, np.uint16)
    sel = np.ascontiguousarray(sel, np.int32)
    n = int(sel.shape[0])
    out = np.zeros((n, d), np.uint16)
    y = np.zeros((n, kmax, d), np.uint16)
    y_exp = np.full((n, kmax), -1, np.int32)
    rc = _load().moe_oracle_tokens(
        ctypes.c_int(T), ctypes.c_int(k), ctypes.c_int(d), ctypes.c_int(F), ctypes.c_int(El),
        ctypes.c_int(first_local), _p(x), _p(expert), _p(gate), _p(w1), _p(w2),
        ctypes.c_int(n), _p(sel), ctypes.c_int(kmax), _p(out), _p(y), _p(y_exp), ctypes.c_int(nthreads))
    if rc != 0:
        raise ValueError("a token selects more local experts than min(k, El)")
    return out, y, y_exp


def forward_tokens_single(x: np.ndarray, expert: np.ndarray, gate: np.ndarray, w: np.ndarray, El: int,
                          first_local: int, sel: np.ndarray, nthreads: int = 0
                          ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Single-projection experts: x [R,T,d]; w [El,N,d].  Returns (out [n,N], y [n,kmax,N], y_expert [n,kmax])."""
    R, T, d = x.shape
    k = expert.shape[-1]
    N = w.shape[1]
    assert w.shape == (El, N, d)
    kmax = min(k, El)
    x = np.ascontiguousarray(x, np.uint16)
    expert = np.ascontiguousarray(expert, np.int32)
    gate = np.ascontiguousarray(gate, np.float32)
    w = np.ascontiguousarray(w, np.uint16)
    sel = np.ascontiguousarray(sel, np.int32)
    n = int(sel.shape[0])
    out = np.zeros((n, N), np.uint16)
    y = np.zeros((n, kmax, N), np.uint16)
    y_exp = np.full((n, kmax), -1, np.int32)
    rc = _load().moe_oracle_tokens_single(
        ctypes.c_int(T), ctypes.c_int(k), ctypes.c_int(d), ctypes.c_int(N), ctypes.c_int(El),
        ctypes.c_int(first_local), _p(x), _p(expert), _p(gate), _p(w),
        ctypes.c_int(n), _p(sel), ctypes.c_int(kmax), _p(out), _p(y), _p(y_exp), ctypes.c_int(nthreads))
    if rc != 0:
        raise ValueError("a token selects more local experts than min(k, El)")
    return out, y, y_exp
