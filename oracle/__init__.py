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


# ----------------------------------------------------------------------------- static groups (STGA)
def stga_groups(F, Hh, Ww, wh, ww, shot_starts, tg, augment=True):
    """Static spatial-temporal groups of Sec. 3.2 ("Spatial-Temporal Group Attention").

    The latent video has F frames of Hh x Ww tokens, token index (f*Hh + y)*Ww + x.  Space is
    cut into wh x ww fixed windows, each shot (frames [shot_starts[s], shot_starts[s+1])) into
    runs of at most tg consecutive frames; frames of different shots never share a group.
    A group is (shot, run, window); its queries are its own tokens.  Its keys/values are the
    same tokens and, with ``augment``, the tokens of the same window in the last latent frame
    of the previous shot (for the first run of a shot) and in the first latent frame of the
    next shot (for the last run of a shot): the paper's "two latent frames from adjacent
    shots", keys/values only.  Returns two lists of int arrays (query tokens, key tokens) in
    the order (shot, run, window), tokens ascending, the augmenting frames before / after."""
    starts = list(shot_starts) + [F]
    assert starts[0] == 0 and all(a < b for a, b in zip(starts, starts[1:]))

    def window_tokens(f, wy, wx):
        return [(f * Hh + y) * Ww + x for y in range(Hh) if y * wh // Hh == wy
                for x in range(Ww) if x * ww // Ww == wx]

    q_groups, kv_groups = [], []
    for s in range(len(starts) - 1):
        f0, f1 = starts[s], starts[s + 1]
        runs = [(a, min(a + tg, f1)) for a in range(f0, f1, tg)]
        for r, (a, b) in enumerate(runs):
            for wy in range(wh):
                for wx in range(ww):
                    own = [t for f in range(a, b) for t in window_tokens(f, wy, wx)]
                    if not own:
                        continue
                    before = window_tokens(f0 - 1, wy, wx) if augment and r == 0 and s > 0 else []
                    after = (window_tokens(f1, wy, wx)
                             if augment and r == len(runs) - 1 and s < len(starts) - 2 else [])
                    q_groups.append(np.array(own, np.int64))
                    kv_groups.append(np.array(before + own + after, np.int64))
    return q_groups, kv_groups


def frame_groups(F, Hh, Ww):
    """Per-frame attention of Sec. 3.2: one group per latent frame, keys = queries."""
    g = [np.arange(f * Hh * Ww, (f + 1) * Hh * Ww, dtype=np.int64) for f in range(F)]
    return g, g


def static_group_attn(Q, K, V, q_groups, kv_groups, scale):
    """Eq. 1 inside caller-given groups whose query and key/value sets may differ:
    O[b,h,n,:] = softmax_m(scale * <Q[b,h,n], K[b,h,m]>) V[b,h,m] over the keys m of the group
    that holds query n.  Q,K,V [B,H,N,D] (exact float32 copies of the inputs); fp64 result
    [B,H,N,D]; tokens in no query group stay zero."""
    Q, K, V = (np.asarray(a, dtype=np.float64) for a in (Q, K, V))
    O = np.zeros_like(Q)
    for qi, ki in zip(q_groups, kv_groups):
        s = np.einsum("bhnd,bhmd->bhnm", Q[:, :, qi], K[:, :, ki]) * scale
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        p /= p.sum(axis=-1, keepdims=True)
        O[:, :, qi] = np.einsum("bhnm,bhmd->bhnd", p, V[:, :, ki])
    return O


def static_group_attn_rows(Q, K, V, q_groups, kv_groups, scale, rows):
    """Eq. 1 inside caller-given groups for the listed (b, h, token) rows only, one row at a
    time from the definition: scores of the token's query against the keys of the group that
    owns it, max-subtracted softmax, weighted sum of that group's values.  fp64 [nrows, D].
    Serves the paper-sized static-branch comparisons, where the full tensor of
    static_group_attn is out of reach on the host."""
    owner = {}
    for g, qi in enumerate(q_groups):
        for n in qi:
            owner[int(n)] = g
    out = np.empty((len(rows), Q.shape[-1]))
    for i, (b, h, n) in enumerate(rows):
        ki = kv_groups[owner[int(n)]]
        s = (np.asarray(K[b, h, ki], dtype=np.float64) @ np.asarray(Q[b, h, n], dtype=np.float64)) * scale
        p = np.exp(s - s.max())
        out[i] = (p / p.sum()) @ np.asarray(V[b, h, ki], dtype=np.float64)
    return out


def mean3(a, b, c):
    """Sec. 3.2: a token's output is the mean of its dynamic (MoGA) and two static group outputs."""
    return (np.asarray(a, np.float64) + np.asarray(b, np.float64) + np.asarray(c, np.float64)) / 3.0


# ----------------------------------------------------------------------------- backward
def backward(Q, K, V, gid, gate, dO, scale, M):
    """Gradients of the routed group attention with respect to Q, K, V and the gates.

    The paper states no backward pass; this is the chain rule applied to its forward definition,
    O[b,h,n] = sum_j gate[b,n,j] * SA(q_n, K_g, V_g) with g = gid[b,n,j] (Eq. 5 around Eq. 1), for a
    given upstream gradient dO = dL/dO, written out group by group in fp64 with dense matrices:
      p = softmax(scale * q k^T) (rows), o = p v
      do = gate * dO                      (gradient reaching the group's attention output)
      dgate = sum over heads and channels of dO * o
      dv = p^T do,  dp = do v^T,  ds = p * (dp - rowsum(dp * p)),  dq = scale * ds k,  dk = scale * ds^T q
    A token routed to k groups receives the sum of its k contributions.  The routing (gid) is a
    fixed integer decision and carries no gradient.
    Q, K, V, dO [B,H,N,D]; gid int [B,N,k]; gate [B,N,k].  Returns dQ, dK, dV [B,H,N,D], dgate [B,N,k] (fp64)."""
    Q, K, V, dO = (np.asarray(a, dtype=np.float64) for a in (Q, K, V, dO))
    gid = np.asarray(gid)
    gate = np.asarray(gate, dtype=np.float64)
    B, H, N, D = Q.shape
    k = gid.shape[2]
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    dgate = np.zeros((B, N, k))
    for b in range(B):
        for g in range(M):
            tok, slot = np.nonzero(gid[b] == g)            # assignments of group g, ascending token
            if tok.size == 0:
                continue
            gt = gate[b, tok, slot]
            for h in range(H):
                q, kk, v = Q[b, h, tok], K[b, h, tok], V[b, h, tok]
                s = scale * (q @ kk.T)
                s = s - s.max(axis=1, keepdims=True)
                p = np.exp(s)
                p /= p.sum(axis=1, keepdims=True)
                o = p @ v
                d_out = dO[b, h, tok]
                np.add.at(dgate[b], (tok, slot), (d_out * o).sum(axis=1))
                do = gt[:, None] * d_out
                dv = p.T @ do
                dp = do @ v.T
                ds = p * (dp - (dp * p).sum(axis=1, keepdims=True))
                np.add.at(dQ[b, h], tok, scale * (ds @ kk))
                np.add.at(dK[b, h], tok, scale * (ds.T @ q))
                np.add.at(dV[b, h], tok, dv)
    return dQ, dK, dV, dgate


def route_backward(X, Wr, bias, gid, dgate, gate_mode):
    """Gradient of the router (Eq. 2-3 and the gate of Eq. 5) for a given dgate = dL/dgate.

    The paper states no backward; this is the chain rule on its router: logits r = X W_r (+ bias),
    the selected groups gid are fixed integers, and the gates are
      mode ALL : gate_j = softmax(r)[g_j]                      -> dr_i = sum_j dgate_j p_{g_j} (delta(i, g_j) - p_i)
      mode TOPK: gate_j = softmax over the k selected logits   -> dr_{g_i} = z_i (dgate_i - sum_j dgate_j z_j), 0 elsewhere
    then dW_r = X^T dr, dbias = sum_n dr, dX = dr W_r^T.  All in fp64.
    X [B,N,C], Wr [C,M], gid [B,N,k], dgate [B,N,k].  Returns dr [B,N,M], dX [B,N,C], dWr [C,M], dbias [M]."""
    X = np.asarray(X, dtype=np.float64)
    Wr = np.asarray(Wr, dtype=np.float64)
    dgate = np.asarray(dgate, dtype=np.float64)
    gid = np.asarray(gid)
    B, N, C = X.shape
    M = Wr.shape[1]
    k = gid.shape[2]
    r = X @ Wr + (0.0 if bias is None else np.asarray(bias, dtype=np.float64))
    dr = np.zeros((B, N, M))
    for b in range(B):
        for n in range(N):
            g = gid[b, n]
            if gate_mode == GATE_SOFTMAX_ALL:
                e = np.exp(r[b, n] - r[b, n].max())
                p = e / e.sum()
                for j in range(k):
                    onehot = np.zeros(M)
                    onehot[g[j]] = 1.0
                    dr[b, n] += dgate[b, n, j] * p[g[j]] * (onehot - p)
            else:
                sel = r[b, n, g]
                e = np.exp(sel - sel.max())
                z = e / e.sum()
                dr[b, n, g] = z * (dgate[b, n] - (dgate[b, n] * z).sum())
    dX = dr @ Wr.T
    dWr = np.einsum("bnc,bnm->cm", X, dr)
    return dr, dX, dWr, dr.sum(axis=(0, 1))

