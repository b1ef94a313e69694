"""Thin ctypes binding of the C ABI in include/moga.h (argument marshalling only).

Every function takes torch CUDA tensors (used purely as device memory), passes
their pointers and the current stream to ``libmoga.so`` and raises ``MogaError``
on a non-OK status.  No arithmetic of the method happens in Python, and there is
no fallback: if the library is missing, importing this module fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .inputs import MogaConfig

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libmoga.so")

EXPORTS = ("moga_workspace_bytes", "moga_scratch_bytes", "moga_status_string", "moga_route",
           "moga_permute", "moga_group_attn", "moga_unpermute", "moga_forward",
           "moga_last_device_status", "moga_sort_static", "moga_balance_stats", "moga_stga_build", "moga_gather_rows",
           "moga_static_group_attn", "moga_mean3", "moga_forward_host_bytes", "moga_forward_host",
           "moga_visual_workspace_bytes", "moga_visual_forward", "moga_selftest_wait_timeout", "moga_set_attn_kernel", "moga_forward_routed", "moga_set_fused_topk", "moga_backward",
           "moga_backward_workspace_bytes", "moga_route_backward", "moga_route_backward_workspace_bytes")

MOGA_F32, MOGA_BF16 = 0, 1
MOGA_ROUTE_AUTO, MOGA_ROUTE_ALU = 0, 1
STATUS_NAMES = {0: "MOGA_OK", 1: "MOGA_ERR_INVALID_ARG", 2: "MOGA_ERR_UNSUPPORTED",
                3: "MOGA_ERR_WORKSPACE", 4: "MOGA_ERR_CUDA", 5: "MOGA_ERR_TIMEOUT",
                6: "MOGA_ERR_INTERNAL"}


class MogaShape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("N", ctypes.c_int32), ("H", ctypes.c_int32),
                ("C", ctypes.c_int32), ("D", ctypes.c_int32), ("M", ctypes.c_int32),
                ("k", ctypes.c_int32), ("dtype", ctypes.c_int32), ("gate_mode", ctypes.c_int32),
                ("scale", ctypes.c_float), ("q_stride_b", ctypes.c_int64),
                ("q_stride_h", ctypes.c_int64), ("q_stride_n", ctypes.c_int64),
                ("route_mode", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class MogaStaticLists(ctypes.Structure):
    _fields_ = [("G", ctypes.c_int32), ("Tkv", ctypes.c_int32), ("F", ctypes.c_int32),
                ("tokens_per_frame", ctypes.c_int32), ("q_idx", ctypes.c_void_p), ("q_inv", ctypes.c_void_p),
                ("q_offsets", ctypes.c_void_p), ("kv_idx", ctypes.c_void_p), ("kv_offsets", ctypes.c_void_p)]


class MogaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)} ({status_string(code)})")


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_18692_b200.build` "
                      "(there is no CPU fallback)")
lib = ctypes.CDLL(LIB_PATH)
for _n in EXPORTS:
    getattr(lib, _n).restype = ctypes.c_int
for _n in ("moga_workspace_bytes", "moga_scratch_bytes", "moga_static_scratch_bytes", "moga_forward_host_bytes",
           "moga_visual_workspace_bytes", "moga_backward_workspace_bytes", "moga_route_backward", "moga_route_backward_workspace_bytes"):
    getattr(lib, _n).restype = ctypes.c_size_t
lib.moga_status_string.restype = ctypes.c_char_p


def status_string(code: int) -> str:
    return lib.moga_status_string(ctypes.c_int(code)).decode()


def make_shape(cfg: MogaConfig, strides=None, scale=None, route_mode=MOGA_ROUTE_AUTO) -> MogaShape:
    sb, sh, sn = strides if strides is not None else (0, 0, 0)
    return MogaShape(cfg.B, cfg.N, cfg.H, cfg.C, cfg.D, cfg.M, cfg.k,
                     MOGA_F32 if cfg.dtype == "f32" else MOGA_BF16, cfg.gate_mode,
                     cfg.scale if scale is None else scale, sb, sh, sn, route_mode, 0)


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str):
    if code != 0:
        raise MogaError(code, where)


def moga_workspace_bytes(shape: MogaShape) -> int:
    return int(lib.moga_workspace_bytes(ctypes.byref(shape)))


def moga_scratch_bytes(shape: MogaShape) -> int:
    return int(lib.moga_scratch_bytes(ctypes.byref(shape)))


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """Device bytes for ``ws`` (torch's allocator returns 512-byte aligned blocks)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def moga_route(shape, X, Wr, bias, gid, gate, logits=None, ws=None):
    _check(lib.moga_route(ctypes.byref(shape), _ptr(X), _ptr(Wr), _ptr(bias), _ptr(gid), _ptr(gate),
                          _ptr(logits), _ptr(ws), ctypes.c_size_t(0 if ws is None else ws.numel()),
                          _stream()), "moga_route")


def moga_balance_stats(shape, gid, gate, alpha, F, P, loss, ws):
    _check(lib.moga_balance_stats(ctypes.byref(shape), _ptr(gid), _ptr(gate), ctypes.c_float(alpha), _ptr(F),
                                  _ptr(P), _ptr(loss), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()),
           "moga_balance_stats")


def moga_permute(shape, gid, Q, K, V, perm, inv, offsets, Qp, Kp, Vp, ws):
    _check(lib.moga_permute(ctypes.byref(shape), _ptr(gid), _ptr(Q), _ptr(K), _ptr(V), _ptr(perm),
                            _ptr(inv), _ptr(offsets), _ptr(Qp), _ptr(Kp), _ptr(Vp), _ptr(ws),
                            ctypes.c_size_t(ws.numel()), _stream()), "moga_permute")


def moga_sort_static(shape, gid, perm, inv, offsets, status_out=None):
    """Group sort with library-resident scratch: no workspace, no device allocation."""
    _check(lib.moga_sort_static(ctypes.byref(shape), _ptr(gid), _ptr(perm), _ptr(inv), _ptr(offsets),
                                _ptr(status_out), _stream()), "moga_sort_static")


def moga_group_attn(shape, Qp, Kp, Vp, offsets, Op, lse, ws):
    _check(lib.moga_group_attn(ctypes.byref(shape), _ptr(Qp), _ptr(Kp), _ptr(Vp), _ptr(offsets),
                               _ptr(Op), _ptr(lse), _ptr(ws), ctypes.c_size_t(ws.numel()),
                               _stream()), "moga_group_attn")


def moga_stga_build(F, Hh, Ww, wh, ww, shot_starts, tg, augment=True):
    """Host-side group lists of the spatial-temporal branch: dict of numpy int32 arrays
    q_idx, q_inv, q_offsets, kv_idx, kv_offsets (plus G, Tkv)."""
    import numpy as np
    shots = (ctypes.c_int32 * len(shot_starts))(*shot_starts)
    G, Tkv = ctypes.c_int32(0), ctypes.c_int32(0)
    null = ctypes.c_void_p(0)
    args = (ctypes.c_int32(F), ctypes.c_int32(Hh), ctypes.c_int32(Ww), ctypes.c_int32(wh), ctypes.c_int32(ww),
            shots, ctypes.c_int32(len(shot_starts)), ctypes.c_int32(tg), ctypes.c_int32(1 if augment else 0))
    _check(lib.moga_stga_build(*args, null, null, null, null, null, ctypes.byref(G), ctypes.byref(Tkv)),
           "moga_stga_build")
    N = F * Hh * Ww
    out = dict(q_idx=np.empty(N, np.int32), q_inv=np.empty(N, np.int32), q_offsets=np.empty(G.value + 1, np.int32),
               kv_idx=np.empty(Tkv.value, np.int32), kv_offsets=np.empty(G.value + 1, np.int32))
    p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib.moga_stga_build(*args, p(out["q_idx"]), p(out["q_inv"]), p(out["q_offsets"]), p(out["kv_idx"]),
                               p(out["kv_offsets"]), ctypes.byref(G), ctypes.byref(Tkv)), "moga_stga_build")
    out.update(G=G.value, Tkv=Tkv.value)
    return out


def moga_static_scratch_bytes(shape, G) -> int:
    return int(lib.moga_static_scratch_bytes(ctypes.byref(shape), ctypes.c_int32(G)))


def moga_gather_rows(shape, idx, src, dst):
    _check(lib.moga_gather_rows(ctypes.byref(shape), _ptr(idx), ctypes.c_int32(idx.numel()), _ptr(src), _ptr(dst),
                                _stream()), "moga_gather_rows")


def moga_static_group_attn(shape, G, Tq, Tkv, Qs, Ks, Vs, q_offsets, kv_offsets, Os, lse, ws):
    _check(lib.moga_static_group_attn(ctypes.byref(shape), ctypes.c_int32(G), ctypes.c_int32(Tq), ctypes.c_int32(Tkv),
                                      _ptr(Qs), _ptr(Ks), _ptr(Vs), _ptr(q_offsets), _ptr(kv_offsets), _ptr(Os),
                                      _ptr(lse), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()),
           "moga_static_group_attn")


def moga_mean3(shape, A, Bs, inv_b, C, O):
    _check(lib.moga_mean3(ctypes.byref(shape), _ptr(A), _ptr(Bs), _ptr(inv_b), _ptr(C), _ptr(O), _stream()),
           "moga_mean3")


def moga_unpermute(shape, Op, inv, gate, O):
    _check(lib.moga_unpermute(ctypes.byref(shape), _ptr(Op), _ptr(inv), _ptr(gate), _ptr(O),
                              _stream()), "moga_unpermute")


def moga_forward(shape, X, Wr, bias, Q, K, V, O, ws, gid_out=None, gate_out=None, perm_out=None,
                 offsets_out=None):
    _check(lib.moga_forward(ctypes.byref(shape), _ptr(X), _ptr(Wr), _ptr(bias), _ptr(Q), _ptr(K),
                            _ptr(V), _ptr(O), _ptr(gid_out), _ptr(gate_out), _ptr(perm_out),
                            _ptr(offsets_out), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()),
           "moga_forward")


def moga_forward_routed(shape, gid, gate, Q, K, V, O, ws, perm_out=None, offsets_out=None):
    _check(lib.moga_forward_routed(ctypes.byref(shape), _ptr(gid), _ptr(gate), _ptr(Q), _ptr(K), _ptr(V), _ptr(O),
                                   _ptr(perm_out), _ptr(offsets_out), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                   _stream()), "moga_forward_routed")


def moga_route_backward_workspace_bytes(shape) -> int:
    return int(lib.moga_route_backward_workspace_bytes(ctypes.byref(shape)))


def moga_route_backward(shape, X, Wr, logits, gid, dgate, dX, dWr, dbias, ws):
    _check(lib.moga_route_backward(ctypes.byref(shape), _ptr(X), _ptr(Wr), _ptr(logits), _ptr(gid), _ptr(dgate),
                                   _ptr(dX), _ptr(dWr), _ptr(dbias), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                   _stream()), "moga_route_backward")


def moga_backward_workspace_bytes(shape) -> int:
    return int(lib.moga_backward_workspace_bytes(ctypes.byref(shape)))


def moga_backward(shape, Qp, Kp, Vp, Op, lse, gate, perm, inv, offsets, dO, dQ, dK, dV, dgate, ws):
    _check(lib.moga_backward(ctypes.byref(shape), _ptr(Qp), _ptr(Kp), _ptr(Vp), _ptr(Op), _ptr(lse), _ptr(gate),
                             _ptr(perm), _ptr(inv), _ptr(offsets), _ptr(dO), _ptr(dQ), _ptr(dK), _ptr(dV),
                             _ptr(dgate), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "moga_backward")


def moga_forward_host_bytes(shape, heads_per_chunk) -> int:
    return int(lib.moga_forward_host_bytes(ctypes.byref(shape), ctypes.c_int32(heads_per_chunk)))


def moga_forward_host(shape, X, Wr, bias, Q, K, V, O, arena, heads_per_chunk, gid_out=None, gate_out=None):
    """Forward from host tensors (torch CPU tensors, ideally pinned); ``arena`` is a CUDA uint8 tensor."""
    _check(lib.moga_forward_host(ctypes.byref(shape), _ptr(X), _ptr(Wr), _ptr(bias), _ptr(Q), _ptr(K), _ptr(V),
                                 _ptr(O), _ptr(gid_out), _ptr(gate_out), _ptr(arena),
                                 ctypes.c_size_t(arena.numel()), ctypes.c_int32(heads_per_chunk), _stream()),
           "moga_forward_host")


def make_static_lists(lists, F, tokens_per_frame, device="cuda"):
    """Device copies of moga_stga_build's arrays wrapped for moga_visual_forward.  Returns the
    ctypes struct and the tensors that keep the device memory alive."""
    keep = {k: torch.from_numpy(lists[k]).to(device) for k in ("q_idx", "q_inv", "q_offsets", "kv_idx", "kv_offsets")}
    st = MogaStaticLists(lists["G"], lists["Tkv"], F, tokens_per_frame, *(keep[k].data_ptr() for k in
                         ("q_idx", "q_inv", "q_offsets", "kv_idx", "kv_offsets")))
    return st, keep


def moga_visual_workspace_bytes(shape, static_lists) -> int:
    return int(lib.moga_visual_workspace_bytes(ctypes.byref(shape), ctypes.byref(static_lists)))


def moga_visual_forward(shape, X, Wr, bias, Q, K, V, O, static_lists, ws):
    _check(lib.moga_visual_forward(ctypes.byref(shape), _ptr(X), _ptr(Wr), _ptr(bias), _ptr(Q), _ptr(K), _ptr(V),
                                   _ptr(O), ctypes.byref(static_lists), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                   _stream()), "moga_visual_forward")


def moga_selftest_wait_timeout(ws, limit_ns):
    _check(lib.moga_selftest_wait_timeout(_ptr(ws), ctypes.c_size_t(ws.numel()), ctypes.c_uint64(limit_ns),
                                          _stream()), "moga_selftest_wait_timeout")


MOGA_ATTN_AUTO, MOGA_ATTN_SINGLE, MOGA_ATTN_PAIR = 0, 1, 2


def moga_set_fused_topk(on: bool):
    _check(lib.moga_set_fused_topk(ctypes.c_int32(1 if on else 0)), "moga_set_fused_topk")


def moga_set_attn_kernel(mode: int):
    _check(lib.moga_set_attn_kernel(ctypes.c_int32(mode)), "moga_set_attn_kernel")


def moga_last_device_status(ws):
    """(status code, detail word) of the most recent call that used ``ws``; synchronises."""
    detail = ctypes.c_uint32(0)
    code = lib.moga_last_device_status(_ptr(ws), _stream(), ctypes.byref(detail))
    return int(code), int(detail.value)
