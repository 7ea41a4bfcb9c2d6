"""CPU oracle for the attention hot path -- TEST INFRASTRUCTURE, not the product.

Thin ctypes wrapper around ``lt_oracle.c`` (plain fp64 C, OpenMP over heads).
Only tests, the smoke check and the benchmark's CPU legs may import this
package; the CUDA library never does, and the two share no code.

Every function takes and returns numpy float64 arrays laid out ``[B, H, S, D]``
(LSE: ``[B, Hq, S]``).  fp16 inputs are widened exactly to float64 by the caller
(``x.astype(np.float64)``), which gives "fp64 math on fp16-rounded inputs".

The formulas follow the paper's Attention Backward (Section 4.1, Algorithm 1):
GP = GO V^T, GS = SoftmaxBackward(P, GP), GV = P^T GO, GQ = GS K, GK = GS^T Q,
with P the softmax of the scaled, optionally causally masked scores.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "lt_oracle.c"
_LIB = _HERE / "liblt_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile ``lt_oracle.c`` into ``liblt_oracle.so`` next to it (gcc, OpenMP)."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
    cmd = ["gcc", "-O3", "-march=native", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
           "-std=c11", "-o", str(tmp), str(_SRC), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        dp = ctypes.POINTER(ctypes.c_double)
        i, d = ctypes.c_int, ctypes.c_double
        lib.lt_oracle_attn_fwd_f64.argtypes = [dp] * 5 + [i] * 6 + [d]
        lib.lt_oracle_attn_fwd_f64.restype = i
        lib.lt_oracle_attn_bwd_f64.argtypes = [dp] * 9 + [i] * 6 + [d]
        lib.lt_oracle_attn_bwd_f64.restype = i
        lib.lt_oracle_delta_f64.argtypes = [dp] * 3 + [ctypes.c_longlong, i]
        lib.lt_oracle_delta_f64.restype = i
        lib.lt_oracle_num_threads.restype = i
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops will use (what the CPU baseline reports as cores)."""
    return int(_load().lt_oracle_num_threads())


def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x), dtype=np.float64)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _dims(Q, K):
    if Q.ndim != 4 or K.ndim != 4:
        raise ValueError("expected [B, H, S, D] arrays")
    B, Hq, S, D = Q.shape
    if K.shape[0] != B or K.shape[2] != S or K.shape[3] != D:
        raise ValueError("K/V shape does not match Q")
    return B, Hq, K.shape[1], S, D


def attn_fwd(Q, K, V, causal: bool, scale: float):
    """Return (O [B,Hq,S,D], LSE [B,Hq,S]) in float64; LSE is a natural log."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    B, Hq, Hkv, S, D = _dims(Q, K)
    O = np.empty_like(Q)
    LSE = np.empty((B, Hq, S), dtype=np.float64)
    rc = _load().lt_oracle_attn_fwd_f64(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(LSE),
                                        B, Hq, Hkv, S, D, int(bool(causal)), float(scale))
    if rc != 0:
        raise RuntimeError(f"lt_oracle_attn_fwd_f64 failed with code {rc}")
    return O, LSE


def attn_bwd(Q, K, V, dO, causal: bool, scale: float, O=None, LSE=None):
    """Return (dQ, dK, dV) in float64.

    With ``O`` and ``LSE`` omitted everything is recomputed from Q, K, V (the
    reference mode).  With both given they are used as the forward state
    (diagnostic mode: P = exp(scale*QK^T - LSE), delta = rowsum(dO*O)).
    """
    Q, K, V, dO = _f64(Q), _f64(K), _f64(V), _f64(dO)
    B, Hq, Hkv, S, D = _dims(Q, K)
    if dO.shape != Q.shape or V.shape != K.shape:
        raise ValueError("dO/V shape mismatch")
    if (O is None) != (LSE is None):
        raise ValueError("give both O and LSE or neither")
    if O is not None:
        O, LSE = _f64(O), _f64(LSE)
    dQ = np.empty_like(Q)
    dK = np.empty_like(K)
    dV = np.empty_like(K)
    rc = _load().lt_oracle_attn_bwd_f64(_ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(O), _ptr(LSE),
                                        _ptr(dQ), _ptr(dK), _ptr(dV),
                                        B, Hq, Hkv, S, D, int(bool(causal)), float(scale))
    if rc != 0:
        raise RuntimeError(f"lt_oracle_attn_bwd_f64 failed with code {rc}")
    return dQ, dK, dV


def delta(dO, O):
    """delta = rowsum(dO * O) over the last axis, float64."""
    dO, O = _f64(dO), _f64(O)
    out = np.empty(dO.shape[:-1], dtype=np.float64)
    rc = _load().lt_oracle_delta_f64(_ptr(dO), _ptr(O), _ptr(out), out.size, dO.shape[-1])
    if rc != 0:
        raise RuntimeError(f"lt_oracle_delta_f64 failed with code {rc}")
    return out


def gemm_nt(A, W):
    """C = A W^T in float64: A is [M, K] (activations), W is [N, K] (the weight matrix of a linear
    layer as it is stored), C is [M, N].  This is the product the paper's FP16 GEMM backend computes
    for the QKV, output and FFN projections (Section 4.1: C[M,N] accumulates A[M,K] B[K,N]; here
    B = W^T) and profiles in its table of GEMM shapes (Section 6.6).  numpy's matmul is the library
    step; nothing is blocked or reordered here."""
    A, W = _f64(A), _f64(W)
    if A.ndim != 2 or W.ndim != 2 or A.shape[1] != W.shape[1]:
        raise ValueError("expected A [M, K] and W [N, K]")
    return A @ W.T


def attn_probabilities(Q, K, causal: bool, scale: float):
    """P [B,Hq,S,S] in float64: the row softmax of the scaled, optionally causally masked scores,
    P[b,h,q,:] = softmax_k(scale * Q[b,h,q] . K[b,g,k]) with keys k > q hidden under the mask.
    This is the probability matrix the paper's forward pass saves tile by tile for Attention
    Backward (Section 4.1: the backward loads the saved tile P_ij).  Plain numpy, no blocking."""
    Q, K = _f64(Q), _f64(K)
    B, Hq, Hkv, S, D = _dims(Q, K)
    G = Hq // Hkv
    P = np.empty((B, Hq, S, S), dtype=np.float64)
    hidden = np.triu(np.ones((S, S), dtype=bool), k=1) if causal else None
    for b in range(B):
        for h in range(Hq):
            s = scale * (Q[b, h] @ K[b, h // G].T)
            if causal:
                s = np.where(hidden, -np.inf, s)
            s = s - s.max(axis=1, keepdims=True)
            e = np.exp(s)
            P[b, h] = e / e.sum(axis=1, keepdims=True)
    return P


def attn_bwd_from_p(P, Q, K, V, dO, scale: float):
    """(dQ, dK, dV) in float64 from a given probability matrix P [B,Hq,S,S], step by step as the
    paper's Attention Backward states them (Section 4.1, Algorithm 1): GV = P^T GO, GP = GO V^T,
    GS = P * (GP - rowsum(P * GP)) (the softmax backward), GQ = scale * GS K, GK = scale * GS^T Q;
    the kv head of a group receives the sum over the group's query heads.  P is used as given (a
    mask is already inside it as zeros)."""
    P, Q, K, V, dO = _f64(P), _f64(Q), _f64(K), _f64(V), _f64(dO)
    B, Hq, Hkv, S, D = _dims(Q, K)
    G = Hq // Hkv
    dQ = np.zeros_like(Q)
    dK = np.zeros_like(K)
    dV = np.zeros_like(K)
    for b in range(B):
        for h in range(Hq):
            g = h // G
            p = P[b, h]
            dV[b, g] += p.T @ dO[b, h]
            dP = dO[b, h] @ V[b, g].T
            dS = p * (dP - (p * dP).sum(axis=1, keepdims=True))
            dQ[b, h] = scale * (dS @ K[b, g])
            dK[b, g] += scale * (dS.T @ Q[b, h])
    return dQ, dK, dV
