"""ctypes loader for the plain-C PCG oracle (test infrastructure, not product code).

The arithmetic lives in ``pcg_oracle.c`` beside this file; this module only
compiles it with gcc, marshals numpy arrays and returns numpy arrays.  Logits
are passed as float32 or float16 arrays, or as uint16 arrays holding bf16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

F32 = 0
BF16 = 1
F16 = 2
FLAG_ZERO_RESIDUAL = 2
FLAG_THINNING_EXHAUSTED = 8

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pcg_oracle.c")
_LIB = os.path.join(_HERE, "libpcg_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile pcg_oracle.c into a shared object beside it (gcc, -O2, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_vp, c_i, c_i64, c_f, c_d = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_double
        lib.pcg_oracle_softmax.argtypes = [c_vp, c_i, c_i64, c_i, c_f, c_vp]
        lib.pcg_oracle_softmax.restype = c_i
        lib.pcg_oracle_group_probs.argtypes = [c_vp, c_i, c_i64, c_i, c_f, c_i, c_vp, c_vp, c_vp, c_vp, c_vp]
        lib.pcg_oracle_group_probs.restype = c_i
        lib.pcg_oracle_verify.argtypes = [c_vp, c_vp, c_i, c_i, c_i, c_i, c_vp, c_i, c_vp, c_vp, c_vp, c_vp, c_vp,
                                          c_f, c_d, c_vp, c_vp, c_vp, c_vp, c_vp, c_i]
        lib.pcg_oracle_verify.restype = c_i
        lib.pcg_oracle_verify_thinning.argtypes = [c_vp, c_vp, c_i, c_i, c_i, c_i, c_vp, c_i, c_vp, c_vp, c_vp, c_vp,
                                                   c_vp, c_vp, c_i, c_vp, c_f, c_d, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_i]
        lib.pcg_oracle_verify_thinning.restype = c_i
        lib.pcg_oracle_max_threads.argtypes = []
        lib.pcg_oracle_max_threads.restype = c_i
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().pcg_oracle_max_threads())


def _logits(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, F32
    if a.dtype == np.uint16:
        return a, BF16
    if a.dtype == np.float16:
        return a, F16
    raise TypeError("logits must be float32, float16 or uint16 (bf16 bit patterns)")


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def softmax(logits, temperature: float = 1.0) -> np.ndarray:
    """float64 softmax(logits / T) of every row of a [rows, V] array."""
    a, dt = _logits(logits)
    rows, V = a.shape
    out = np.empty((rows, V), dtype=np.float64)
    rc = _load().pcg_oracle_softmax(_ptr(a), dt, rows, V, temperature, _ptr(out))
    if rc:
        raise ValueError(f"pcg_oracle_softmax failed ({rc})")
    return out


def group_probs(logits, group_ptr, group_tok, tok_degree, temperature: float = 1.0, weights=None) -> np.ndarray:
    """float64 coarse-grained masses [rows, M] of every row of a [rows, V] array."""
    a, dt = _logits(logits)
    rows, V = a.shape
    gp, gt, dg = _i32(group_ptr), _i32(group_tok), _i32(tok_degree)
    M = gp.shape[0] - 1
    w = None if weights is None else np.ascontiguousarray(weights, dtype=np.float64)
    out = np.empty((rows, M), dtype=np.float64)
    rc = _load().pcg_oracle_group_probs(_ptr(a), dt, rows, V, temperature, M, _ptr(gp), _ptr(gt), _ptr(dg), _ptr(w),
                                        _ptr(out))
    if rc:
        raise ValueError(f"pcg_oracle_group_probs failed ({rc})")
    return out


@dataclass
class OracleResult:
    accept_len: np.ndarray  # [B] int32
    tokens: np.ndarray  # [B, K+1] int32, unused slots -1
    groups: np.ndarray  # [B, K+1] int32, unused slots -1
    flags: np.ndarray  # [B] int32
    margins: np.ndarray  # [B, K+1, 2] float64: [i<K] = (label, accept); [K] = (terminal group, terminal token)
    trials: np.ndarray = None  # [B] int32, thinning only: candidates drawn for the terminal group


def verify(target_logits, draft_logits, draft_tokens, group_ptr, group_tok, tok_degree, uniforms,
           temperature: float = 1.0, weights=None, accept_bias: float = 0.0, threads: int = 1,
           thin_uniforms=None, cand_order=None) -> OracleResult:
    """Run Algorithm 1's verification for a batch; see pcg_oracle.c for the layouts.

    With ``thin_uniforms`` ([B, n_trials, 3]) the terminal group comes from the thinning sampler of Sec. 2.2
    instead of the enumerated inverse CDF, and ``trials`` is filled in.  ``cand_order`` ([V], a permutation of the
    token ids; None = ascending token id) is the order in which the sampler's candidate draw walks the tokens.
    """
    tl, dt = _logits(target_logits)
    dl, dt2 = _logits(draft_logits)
    if dt != dt2:
        raise TypeError("target and draft logits must share a dtype")
    B, K1, V = tl.shape
    K = K1 - 1
    if dl.shape != (B, K, V):
        raise ValueError("draft_logits must be [B, K, V]")
    x = _i32(draft_tokens)
    u = np.ascontiguousarray(uniforms, dtype=np.float32)
    if x.shape != (B, K) or u.shape != (B, K + 1, 2):
        raise ValueError("draft_tokens must be [B, K] and uniforms [B, K+1, 2]")
    gp, gt, dg = _i32(group_ptr), _i32(group_tok), _i32(tok_degree)
    M = gp.shape[0] - 1
    w = None if weights is None else np.ascontiguousarray(weights, dtype=np.float64)
    res = OracleResult(
        accept_len=np.empty(B, np.int32),
        tokens=np.empty((B, K + 1), np.int32),
        groups=np.empty((B, K + 1), np.int32),
        flags=np.zeros(B, np.int32),
        margins=np.empty((B, K + 1, 2), np.float64),
    )
    if thin_uniforms is not None:
        tu = np.ascontiguousarray(thin_uniforms, dtype=np.float32)
        if tu.ndim != 3 or tu.shape[0] != B or tu.shape[1] < 1 or tu.shape[2] != 3:
            raise ValueError("thin_uniforms must be [B, n_trials >= 1, 3]")
        res.trials = np.zeros(B, np.int32)
        order = None if cand_order is None else _i32(cand_order)
        if order is not None and order.shape != (V,):
            raise ValueError("cand_order must be [V]")
        rc = _load().pcg_oracle_verify_thinning(_ptr(tl), _ptr(dl), dt, B, K, V, _ptr(x), M, _ptr(gp), _ptr(gt), _ptr(dg),
                                                _ptr(w), _ptr(u), _ptr(tu), tu.shape[1], _ptr(order), temperature, accept_bias,
                                                _ptr(res.accept_len), _ptr(res.tokens), _ptr(res.groups),
                                                _ptr(res.flags), _ptr(res.trials), _ptr(res.margins), threads)
        if rc:
            raise ValueError(f"pcg_oracle_verify_thinning failed ({rc})")
        return res
    rc = _load().pcg_oracle_verify(_ptr(tl), _ptr(dl), dt, B, K, V, _ptr(x), M, _ptr(gp), _ptr(gt), _ptr(dg), _ptr(w),
                                   _ptr(u), temperature, accept_bias, _ptr(res.accept_len), _ptr(res.tokens),
                                   _ptr(res.groups), _ptr(res.flags), _ptr(res.margins), threads)
    if rc:
        raise ValueError(f"pcg_oracle_verify failed ({rc})")
    return res
