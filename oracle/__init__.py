"""fp64 CPU oracle for the gated delta rule (paper, "Gated Delta Net" subsection).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports or calls it and
the two share no code.

The arithmetic lives in ``gdn_oracle.cpp`` (token-by-token recurrence, fp64).
This module compiles that file with g++ on first use and wraps the two entry
points for numpy arrays.  bf16 tensors are passed as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gdn_oracle.cpp")
_LIB = os.path.join(_HERE, "libgdn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle shared library next to its source; return its path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread",
             "-ffp-contract=off", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.c_void_p
        I = ctypes.c_int
        lib.gdn_oracle_default_threads.restype = I
        lib.gdn_oracle_decode.restype = I
        lib.gdn_oracle_decode.argtypes = [P, P, P, P, P, P, P, P, I, I, I, I, I, I,
                                          ctypes.c_double, I]
        lib.gdn_oracle_prefill.restype = I
        lib.gdn_oracle_prefill.argtypes = [P, P, P, P, P, P, P, P, P, P, I, I, I, I, I, I, I,
                                           ctypes.c_double, I]
        _lib = lib
    return _lib


def default_threads() -> int:
    return int(_load().gdn_oracle_default_threads())


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def decode(q, k, v, g, beta, pool, slot_idx=None, scale=1.0, n_threads=0):
    """One decode step.  ``pool`` (float64 [num_slots,Hv,dv,dk]) is updated IN PLACE.

    q,k: uint16 [B,Hqk,dk]; v: uint16 [B,Hv,dv]; g,beta: float32 [B,Hv];
    slot_idx: int32 [B] or None.  Returns (o float64 [B,Hv,dv], n_bad_slots).
    """
    q = _c(q, np.uint16); k = _c(k, np.uint16); v = _c(v, np.uint16)
    g = _c(g, np.float32); beta = _c(beta, np.float32)
    assert pool.dtype == np.float64 and pool.flags.c_contiguous
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    num_slots = pool.shape[0]
    assert pool.shape == (num_slots, Hv, dv, dk)
    assert k.shape == q.shape and g.shape == (B, Hv) and beta.shape == (B, Hv)
    if slot_idx is not None:
        slot_idx = _c(slot_idx, np.int32)
        assert slot_idx.shape == (B,)
    o = np.empty((B, Hv, dv), dtype=np.float64)
    rc = _load().gdn_oracle_decode(_p(q), _p(k), _p(v), _p(g), _p(beta), _p(pool),
                                   _p(slot_idx), _p(o), B, Hqk, Hv, dk, dv, num_slots,
                                   float(scale), int(n_threads))
    if rc < 0:
        raise ValueError(f"gdn_oracle_decode rejected its arguments ({rc})")
    return o, rc


def prefill(q, k, v, g, beta, cu_seqlens, init_state=None, slot_idx=None, scale=1.0,
            num_slots=None, final_state=None, n_threads=0):
    """Token-by-token prefill over packed sequences.

    q,k: uint16 [T,Hqk,dk]; v: uint16 [T,Hv,dv]; g,beta: float32 [T,Hv];
    cu_seqlens: int32 [N+1]; init_state: float64 [num_slots,Hv,dv,dk] or None (zeros).
    Returns (o float64 [T,Hv,dv], final_state float64 [num_slots,Hv,dv,dk], n_bad_slots).
    Slots no sequence maps to keep the values ``final_state`` had on entry
    (a fresh array is zero-filled unless ``final_state`` is given).
    """
    q = _c(q, np.uint16); k = _c(k, np.uint16); v = _c(v, np.uint16)
    g = _c(g, np.float32); beta = _c(beta, np.float32)
    cu = _c(cu_seqlens, np.int32)
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu.shape[0] - 1
    if num_slots is None:
        num_slots = init_state.shape[0] if init_state is not None else N
    if init_state is not None:
        assert init_state.dtype == np.float64 and init_state.flags.c_contiguous
        assert init_state.shape == (num_slots, Hv, dv, dk)
    if final_state is None:
        final_state = np.zeros((num_slots, Hv, dv, dk), dtype=np.float64)
    assert final_state.dtype == np.float64 and final_state.shape == (num_slots, Hv, dv, dk)
    if slot_idx is not None:
        slot_idx = _c(slot_idx, np.int32)
        assert slot_idx.shape == (N,)
    o = np.zeros((T, Hv, dv), dtype=np.float64)
    rc = _load().gdn_oracle_prefill(_p(q), _p(k), _p(v), _p(g), _p(beta), _p(cu),
                                    _p(init_state), _p(final_state), _p(slot_idx), _p(o),
                                    T, N, Hqk, Hv, dk, dv, num_slots, float(scale),
                                    int(n_threads))
    if rc < 0:
        raise ValueError(f"gdn_oracle_prefill rejected its arguments ({rc})")
    return o, final_state, rc


def gate(a_bits, b_bits, A_log, dt_bias):
    """Gate / beta preprocessing in fp64 (the paper names the helper without a formula; this is
    the published Gated DeltaNet parametrisation, the reading the library documents):
    g = -exp(A_log) * softplus(a + dt_bias), beta = sigmoid(b).

    a_bits, b_bits: uint16 bf16 patterns [T, Hv]; A_log, dt_bias: float [Hv].
    Returns (g, beta) float64 [T, Hv].
    """
    a = (np.ascontiguousarray(a_bits, np.uint16).astype(np.uint32) << 16).view(np.float32)
    b = (np.ascontiguousarray(b_bits, np.uint16).astype(np.uint32) << 16).view(np.float32)
    x = a.astype(np.float64) + np.asarray(dt_bias, np.float64)[None, :]
    softplus = np.maximum(x, 0.0) + np.log1p(np.exp(-np.abs(x)))
    g = -np.exp(np.asarray(A_log, np.float64))[None, :] * softplus
    beta = 1.0 / (1.0 + np.exp(-b.astype(np.float64)))
    return g, beta
