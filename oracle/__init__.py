"""TEST INFRASTRUCTURE, NOT THE PRODUCT: CPU oracle for the MDN forward.

`stepwise` evaluates the token-by-token recurrence of Section 3.1 (Eq. 5-6) in
fp64 through the plain C file next to this one; `chunkwise` (numpy, fp64) walks
the paper's chunkwise algorithm step by step.  Only tests, the smoke check and
the CPU-baseline leg of the benchmark may import this package; the CUDA path
never does, and this package imports nothing of the CUDA path.

Pins (tests/test_oracle_pins.py): mu=0 reduces to the gated delta rule; beta=0
leaves a purely decayed state; k=0 gives the closed-form decay of (S0, M0); a
brute-force unrolled closed form for T<=16; the second-order two-step form; the
summation-reordering identity; chunkwise == stepwise; the closed-form spectrum
of the transition matrix; state hand-off; a hand-computed scalar example.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "mdn_stepwise.c")
_SRC_BWD = os.path.join(_DIR, "mdn_stepwise_bwd.c")
_LIB = os.path.join(_DIR, "libmdn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, no fast-math, OpenMP)."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_BWD))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, _SRC_BWD, "-lm"],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p = ctypes.c_void_p
        lib.mdn_oracle_stepwise.restype = ctypes.c_int
        lib.mdn_oracle_stepwise.argtypes = [
            ctypes.c_int64, p, p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            p, p, p, p, p, p, p, ctypes.c_double, p, p, p, ctypes.c_int64, p, p, p]
        lib.mdn_oracle_num_threads.restype = ctypes.c_int
        lib.mdn_oracle_stepwise_bwd.restype = ctypes.c_int
        lib.mdn_oracle_stepwise_bwd.argtypes = [
            ctypes.c_int64, p, p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            p, p, p, p, p, p, p, ctypes.c_double, p, p, p, ctypes.c_int64] + [p] * 12
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().mdn_oracle_num_threads())


def _f32(x, shape=None):
    if x is None:
        return None
    a = np.ascontiguousarray(x, dtype=np.float32)
    if shape is not None:
        a = a.reshape(shape)
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def stepwise(q, k, v, beta, log_alpha, log_mu, eta=None, *, scale: float = 1.0,
             S0=None, M0=None, seq_start: Optional[Sequence[int]] = None,
             seq_len: Optional[Sequence[int]] = None, chains: Optional[Sequence[int]] = None):
    """fp64 stepwise recurrence (Eq. 5-6).

    q,k: [B,T,H,dk]; v: [B,T,H,dv]; gates: [B,T,H] (values exactly representable in
    float32).  The [B,T] axes are flattened into one token axis; sequences default to
    the B rows, or are given as token ranges (seq_start, seq_len) for packed input.
    S0, M0: [N,H,dk,dv] or None (zeros).  chains: optional ids n*H+h to evaluate.

    Returns (o [B,T,H,dv], S_final [N,H,dk,dv], M_final [N,H,dk,dv]) as float64;
    entries of chains not evaluated are NaN.
    """
    q = _f32(q); k = _f32(k); v = _f32(v)
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    beta = _f32(beta, (B, T, H)); log_alpha = _f32(log_alpha, (B, T, H))
    log_mu = _f32(log_mu, (B, T, H)); eta = _f32(eta, (B, T, H)) if eta is not None else None
    if seq_start is None:
        seq_start = np.arange(B, dtype=np.int64) * T
        seq_len = np.full(B, T, dtype=np.int64)
    seq_start = np.ascontiguousarray(seq_start, dtype=np.int64)
    seq_len = np.ascontiguousarray(seq_len, dtype=np.int64)
    N = len(seq_len)
    assert (seq_start >= 0).all() and (seq_start + seq_len <= B * T).all()
    S0 = _f32(S0, (N, H, dk, dv)) if S0 is not None else None
    M0 = _f32(M0, (N, H, dk, dv)) if M0 is not None else None
    o = np.full((B, T, H, dv), np.nan, dtype=np.float64)
    Sf = np.full((N, H, dk, dv), np.nan, dtype=np.float64)
    Mf = np.full((N, H, dk, dv), np.nan, dtype=np.float64)
    ch = None
    if chains is not None:
        ch = np.ascontiguousarray(chains, dtype=np.int32)
        assert ((ch >= 0) & (ch < N * H)).all()
    rc = _load().mdn_oracle_stepwise(
        N, _ptr(seq_start), _ptr(seq_len), H, dk, dv, _ptr(q), _ptr(k), _ptr(v),
        _ptr(beta), _ptr(log_alpha), _ptr(log_mu), _ptr(eta), float(scale),
        _ptr(S0), _ptr(M0), _ptr(ch), 0 if ch is None else len(ch), _ptr(o), _ptr(Sf), _ptr(Mf))
    if rc != 0:
        raise RuntimeError("mdn_oracle_stepwise failed (rc=%d)" % rc)
    return o, Sf, Mf


def stepwise_bwd(q, k, v, beta, log_alpha, log_mu, eta, d_o, *, scale: float = 1.0, S0=None, M0=None,
                 dS_final=None, dM_final=None, seq_start: Optional[Sequence[int]] = None,
                 seq_len: Optional[Sequence[int]] = None, chains: Optional[Sequence[int]] = None):
    """fp64 gradients of the stepwise recurrence (reverse mode, token by token; mdn_stepwise_bwd.c).

    Same layout as `stepwise`; d_o: [B,T,H,dv]; dS_final, dM_final: [N,H,dk,dv] or None (zeros).
    Returns a dict of float64 arrays: dq, dk, dv, dbeta, dlog_alpha, dlog_mu, deta (None when eta is None), dS0, dM0;
    entries of chains not evaluated are NaN.
    """
    q = _f32(q); k = _f32(k); v = _f32(v); d_o = _f32(d_o)
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    beta = _f32(beta, (B, T, H)); log_alpha = _f32(log_alpha, (B, T, H))
    log_mu = _f32(log_mu, (B, T, H)); eta = _f32(eta, (B, T, H)) if eta is not None else None
    if seq_start is None:
        seq_start = np.arange(B, dtype=np.int64) * T
        seq_len = np.full(B, T, dtype=np.int64)
    seq_start = np.ascontiguousarray(seq_start, dtype=np.int64)
    seq_len = np.ascontiguousarray(seq_len, dtype=np.int64)
    N = len(seq_len)
    st = (N, H, dk, dv)
    S0 = _f32(S0, st) if S0 is not None else None
    M0 = _f32(M0, st) if M0 is not None else None
    dSf = _f32(dS_final, st) if dS_final is not None else None
    dMf = _f32(dM_final, st) if dM_final is not None else None
    nan = lambda shape: np.full(shape, np.nan, dtype=np.float64)
    out = dict(dq=nan((B, T, H, dk)), dk=nan((B, T, H, dk)), dv=nan((B, T, H, dv)), dbeta=nan((B, T, H)),
               dlog_alpha=nan((B, T, H)), dlog_mu=nan((B, T, H)), deta=nan((B, T, H)) if eta is not None else None,
               dS0=nan(st), dM0=nan(st))
    ch = None
    if chains is not None:
        ch = np.ascontiguousarray(chains, dtype=np.int32)
        assert ((ch >= 0) & (ch < N * H)).all()
    rc = _load().mdn_oracle_stepwise_bwd(
        N, _ptr(seq_start), _ptr(seq_len), H, dk, dv, _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(log_alpha),
        _ptr(log_mu), _ptr(eta), float(scale), _ptr(S0), _ptr(M0), _ptr(ch), 0 if ch is None else len(ch),
        _ptr(d_o), _ptr(dSf), _ptr(dMf), _ptr(out["dq"]), _ptr(out["dk"]), _ptr(out["dv"]), _ptr(out["dbeta"]),
        _ptr(out["dlog_alpha"]), _ptr(out["dlog_mu"]), _ptr(out["deta"]), _ptr(out["dS0"]), _ptr(out["dM0"]))
    if rc != 0:
        raise RuntimeError("mdn_oracle_stepwise_bwd failed (rc=%d)" % rc)
    return out
