"""NumPy-facing wrapper of the fp64 C++ oracle (oracle/gdn_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the benchmark's
CPU-baseline leg; never by the product path.  The wrapper only marshals arrays: bf16 /
fp32 inputs arrive as float32 arrays holding those values exactly and are widened to
float64, so every tolerance measures arithmetic and not input rounding.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gdn_oracle.cpp")
_LIB = os.path.join(_HERE, "libgdn_oracle.so")
_lib = None

DT = {"f32": 0, "bf16": 1, "none": 2}


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (plain IEEE double arithmetic, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-ffp-contract=off", "-std=c++17", "-shared", "-fPIC",
                               "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_round_bf16.restype = ctypes.c_double
        _lib.oracle_round_bf16.argtypes = [ctypes.c_double]
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def round_bf16(x: float) -> float:
    return _load().oracle_round_bf16(float(x))


def gates_from_raw(alpha_in, beta_in, a_log, dt_bias) -> Tuple[np.ndarray, np.ndarray]:
    """Raw gate inputs [B, Ns, Hv] -> the decay and write strength the recurrence consumes (fp64).

    Sec. "Sequential arithmetic and accepted-path replay" says the verifier takes raw gate inputs
    but prints no formula; the reading taken is the Gated DeltaNet parametrisation, per value head h:
    alpha = exp(-exp(a_log[h]) * softplus(alpha_in + dt_bias[h])), beta = 1 / (1 + exp(-beta_in)).
    Pins (tests/test_oracle_scan.py): closed-form values, limits, the softplus and sigmoid
    reflection identities, monotonicity."""
    x = _f64(alpha_in) + _f64(dt_bias)[None, None, :]
    softplus = np.where(x > 0, x, 0.0) + np.log1p(np.exp(-np.abs(x)))
    alpha = np.exp(-np.exp(_f64(a_log))[None, None, :] * softplus)
    beta = 1.0 / (1.0 + np.exp(-_f64(beta_in)))
    return alpha, beta


def conv(parent, slot, state_row, x, w, bias, hist, Ns: int, out_dtype: str = "none",
         threads: int = 0) -> np.ndarray:
    """Recorded operands y [B, Ns, C] (physical rows) of the ancestry-gathered conv + SiLU."""
    lib = _load()
    parent, slot, state_row = _i32(parent), _i32(slot), _i32(state_row)
    B, N = parent.shape
    x, w, hist = _f64(x), _f64(w), _f64(hist)
    bias = None if bias is None else _f64(bias)
    C = x.shape[-1]
    assert x.shape == (B, Ns, C) and w.shape == (C, 4) and hist.shape[1:] == (3, C)
    y = np.empty((B, Ns, C), dtype=np.float64)
    lib.oracle_conv(B, N, Ns, C, _p(parent), _p(slot), _p(state_row), _p(x), _p(w), _p(bias),
                    _p(hist), DT[out_dtype], _p(y), threads)
    return y


def scan(parent, slot, state_row, q, k, v, alpha, beta, state, *, scale: float = 1.0,
         l2norm: bool = False, eps: float = 1e-6, mode: str = "memo", snap_nodes=None,
         threads: int = 0) -> Tuple[np.ndarray, Optional[np.ndarray], int]:
    """(o [B,Ns,Hv,d], snapshots [B,E,Hv,d,d] or None, threads used)."""
    lib = _load()
    parent, slot, state_row = _i32(parent), _i32(slot), _i32(state_row)
    B, N = parent.shape
    q, k, v, alpha, beta, state = map(_f64, (q, k, v, alpha, beta, state))
    _, Ns, Hk, d = q.shape
    Hv = v.shape[2]
    assert k.shape == q.shape and v.shape == (B, Ns, Hv, d) and alpha.shape == (B, Ns, Hv)
    assert beta.shape == alpha.shape and state.shape[1:] == (Hv, d, d) and Hv % Hk == 0
    o = np.empty((B, Ns, Hv, d), dtype=np.float64)
    snap = None
    E = 0
    if snap_nodes is not None:
        snap_nodes = _i32(snap_nodes)
        E = snap_nodes.shape[1]
        snap = np.empty((B, E, Hv, d, d), dtype=np.float64)
    used = lib.oracle_scan(B, N, Ns, Hk, Hv, d, _p(parent), _p(slot), _p(state_row), _p(q), _p(k),
                           _p(v), _p(alpha), _p(beta), _p(state), ctypes.c_double(scale),
                           int(l2norm), ctypes.c_double(eps), {"walk": 0, "memo": 1}[mode], _p(o),
                           _p(snap_nodes), E, _p(snap), threads)
    return o, snap, used


def commit(parent, slot, state_row, q, k, v, alpha, beta, state, accepted, length, *,
           scale: float = 1.0, l2norm: bool = False, eps: float = 1e-6, x=None, hist=None,
           threads: int = 0):
    """(new state pool, new hist pool or None, status [B], threads used); inputs untouched."""
    lib = _load()
    parent, slot, state_row = _i32(parent), _i32(slot), _i32(state_row)
    accepted, length = _i32(accepted), _i32(length)
    B, N = parent.shape
    lmax = accepted.shape[1]
    q, k, v, alpha, beta = map(_f64, (q, k, v, alpha, beta))
    state = np.array(state, dtype=np.float64, order="C", copy=True)
    _, Ns, Hk, d = q.shape
    Hv = v.shape[2]
    C = 0
    if x is not None:
        x = _f64(x)
        hist = np.array(hist, dtype=np.float64, order="C", copy=True)
        C = x.shape[-1]
    status = np.zeros(B, dtype=np.int32)
    used = lib.oracle_commit(B, N, Ns, Hk, Hv, d, _p(parent), _p(slot), _p(state_row), _p(q), _p(k),
                             _p(v), _p(alpha), _p(beta), _p(state), ctypes.c_double(scale),
                             int(l2norm), ctypes.c_double(eps), _p(accepted), _p(length), lmax,
                             _p(x), C, _p(hist if x is not None else None), _p(status), threads)
    return state, (hist if x is not None else None), status, used
