"""ctypes wrapper of the fp64 CPU oracle (test infrastructure, not a product path).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It compiles ``moga_oracle.c`` with gcc on first use and never touches
the CUDA library.  All arrays are numpy; float inputs are float32 holding the
exact bf16/fp32 values the GPU sees, results are float64 / int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moga_oracle.c")
_LIB = os.path.join(_HERE, "libmoga_oracle.so")

GATE_SOFTMAX_ALL = 0   # Eq. 3-5: softmax over all M logits
GATE_SOFTMAX_TOPK = 1  # softmax over the k selected logits

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the .so is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.moga_oracle_threads.restype = ctypes.c_int
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def threads() -> int:
    return int(_load().moga_oracle_threads())


def route(X, Wr, bias, k, gate_mode, want_logits=False):
    """Eq. 2-4.  X [B,N,C], Wr [C,M] -> gid int32 [B,N,k], gate f64 [B,N,k], logits f64 or None."""
    X, Wr, bias = _f32(X), _f32(Wr), _f32(bias)
    B, N, C = X.shape
    M = Wr.shape[1]
    assert Wr.shape[0] == C
    gid = np.empty((B, N, k), np.int32)
    gate = np.empty((B, N, k), np.float64)
    logits = np.empty((B, N, M), np.float64) if want_logits else None
    rc = _load().moga_oracle_route(
        ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(C), ctypes.c_int(M), ctypes.c_int(k),
        ctypes.c_int(gate_mode), _p(X, ctypes.c_float), _p(Wr, ctypes.c_float),
        _p(bias, ctypes.c_float), _p(gid, ctypes.c_int32), _p(gate, ctypes.c_double),
        _p(logits, ctypes.c_double))
    if rc:
        raise ValueError(f"moga_oracle_route rc={rc}")
    return gid, gate, logits


def sort(gid, M):
    """Alg. 1 line 2, index part.  gid [B,N,k] -> offsets [B,M+1], perm [B,T], inv [B,N,k]."""
    gid = np.ascontiguousarray(gid, dtype=np.int32)
    B, N, k = gid.shape
    offsets = np.empty((B, M + 1), np.int32)
    perm = np.empty((B, N * k), np.int32)
    inv = np.empty((B, N, k), np.int32)
    rc = _load().moga_oracle_sort(
        ctypes.c_int(B), ctypes.c_int(N), ctypes.c_int(M), ctypes.c_int(k),
        _p(gid, ctypes.c_int32), _p(offsets, ctypes.c_int32), _p(perm, ctypes.c_int32),
        _p(inv, ctypes.c_int32))
    if rc:
        raise ValueError(f"moga_oracle_sort rc={rc}")
    return offsets, perm, inv


def attn_rows(Q, K, V, gid, gate, offsets, perm, scale, rows):
    """Eq. 1 + Eq. 5 for the listed (b, h, n) rows.  Q,K,V [B,H,N,D] -> f64 [nrows, D]."""
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    B, H, N, D = Q.shape
    gid = np.ascontiguousarray(gid, dtype=np.int32)
    gate = np.ascontiguousarray(gate, dtype=np.float64)
    offsets = np.ascontiguousarray(offsets, dtype=np.int32)
    perm = np.ascontiguousarray(perm, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    k = gid.shape[2]
    M = offsets.shape[1] - 1
    out = np.empty((rows.shape[0], D), np.float64)
    rc = _load().moga_oracle_attn_rows(
        ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(N), ctypes.c_int(D), ctypes.c_int(M),
        ctypes.c_int(k), ctypes.c_double(scale), _p(Q, ctypes.c_float), _p(K, ctypes.c_float),
        _p(V, ctypes.c_float), _p(gid, ctypes.c_int32), _p(gate, ctypes.c_double),
        _p(offsets, ctypes.c_int32), _p(perm, ctypes.c_int32), ctypes.c_longlong(rows.shape[0]),
        _p(rows, ctypes.c_int32), _p(out, ctypes.c_double))
    if rc:
        raise ValueError(f"moga_oracle_attn_rows rc={rc}")
    return out


def attn_all(Q, K, V, gid, gate, offsets, perm, scale):
    """attn_rows over every (b, h, n): f64 [B,H,N,D].  Used with a given routing."""
    B, H, N, D = Q.shape
    b, h, n = np.meshgrid(np.arange(B), np.arange(H), np.arange(N), indexing="ij")
    rows = np.stack([b.ravel(), h.ravel(), n.ravel()], axis=1).astype(np.int32)
    return attn_rows(Q, K, V, gid, gate, offsets, perm, scale, rows).reshape(B, H, N, D)


def forward(X, Wr, bias, Q, K, V, k, gate_mode, scale):
    """The whole MoGA forward.  Returns dict(O f64 [B,H,N,D], gid, gate, offsets, perm, inv)."""
    X, Wr, bias = _f32(X), _f32(Wr), _f32(bias)
    Q, K, V = _f32(Q), _f32(K), _f32(V)
    B, N, C = X.shape
    M = Wr.shape[1]
    _, H, _, D = Q.shape
    O = np.empty((B, H, N, D), np.float64)
    gid = np.empty((B, N, k), np.int32)
    gate = np.empty((B, N, k), np.float64)
    offsets = np.empty((B, M + 1), np.int32)
    perm = np.empty((B, N * k), np.int32)
    inv = np.empty((B, N, k), np.int32)
    rc = _load().moga_oracle_forward(
        ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(N), ctypes.c_int(C), ctypes.c_int(D),
        ctypes.c_int(M), ctypes.c_int(k), ctypes.c_int(gate_mode), ctypes.c_double(scale),
        _p(X, ctypes.c_float), _p(Wr, ctypes.c_float), _p(bias, ctypes.c_float),
        _p(Q, ctypes.c_float), _p(K, ctypes.c_float), _p(V, ctypes.c_float),
        _p(O, ctypes.c_double), _p(gid, ctypes.c_int32), _p(gate, ctypes.c_double),
        _p(offsets, ctypes.c_int32), _p(perm, ctypes.c_int32), _p(inv, ctypes.c_int32))
    if rc:
        raise ValueError(f"moga_oracle_forward rc={rc}")
    return dict(O=O, gid=gid, gate=gate, offsets=offsets, perm=perm, inv=inv)


def balance_stats(gid, gate, M, alpha):
    """Group-balancing loss of Eq. 6-8, written out per batch item in fp64.

    F[b,i] = (assignments of item b to group i) / N (Eq. 7), P[b,i] = (1/N) * sum of the
    routing probabilities (gates) of those assignments (Eq. 8: the sum runs over the tokens
    routed to i only), loss[b] = alpha * M * sum_i F_i P_i (Eq. 6).  The paper states it for
    top-1; with k > 1 every (token, slot) assignment counts once.
    Returns F [B,M], P [B,M], loss [B], all float64."""
    gid = np.asarray(gid)
    gate = np.asarray(gate, dtype=np.float64)
    B, N, k = gid.shape
    F = np.zeros((B, M))
    P = np.zeros((B, M))
    for b in range(B):
        for i in range(M):
            sel = gid[b] == i
            F[b, i] = sel.sum() / N
            P[b, i] = gate[b][sel].sum() / N
    loss = alpha * M * (F * P).sum(axis=1)
    return F, P, loss
