"""Helpers for the GPU-vs-oracle parity tests (the comparison protocol, no kernels).

Routing decides integers from floating point, so the comparison is staged:
  1. gid must equal the oracle's wherever the oracle's fp64 logits separate the
     candidates by more than 1e-5; elsewhere the GPU's pick must be one of the
     near-tied candidates.  Gates agree to 1e-5 where the picks agree.
  2. perm / inv / offsets are compared bit for bit with the oracle's sort run on
     the GPU's gid (identical to the oracle's own when step 1 found no flips).
  3. attention outputs are compared with the oracle evaluated on the GPU's routing.
"""
import numpy as np
import torch

import oracle

MARGIN = 1e-5
TOL = {"bf16": dict(max_abs=2e-2, mean_abs=2e-3), "f32": dict(max_abs=1e-4, mean_abs=1e-4)}


def to_np32(t):
    """Exact widening of a bf16/fp32 torch tensor to a float32 numpy array."""
    return None if t is None else t.detach().float().cpu().numpy()


def check_routing(gid_gpu, gate_gpu, logits64, gid_ref, gate_ref, k):
    """Step 1.  Returns the number of low-margin tokens whose pick differs."""
    gid_gpu = gid_gpu.cpu().numpy()
    gate_gpu = gate_gpu.cpu().numpy().astype(np.float64)
    srt = -np.sort(-logits64, axis=-1)                       # descending logits
    M = logits64.shape[-1]
    # a slot j is decided when logit_j and logit_{j+1} differ by more than the margin
    gaps = srt[..., :-1] - srt[..., 1:] if M > 1 else np.full(srt.shape[:-1] + (0,), np.inf)
    need = gaps[..., :k] if M > k else np.concatenate(
        [gaps[..., :k - 1], np.full(gaps.shape[:-1] + (1,), np.inf)], -1)
    decided = np.all(need > MARGIN, axis=-1)
    same = np.all(gid_gpu == gid_ref, axis=-1)
    assert np.all(same[decided]), "routing differs on a token with a clear margin"
    flips = ~same
    if flips.any():
        # the GPU's picks must be near-tied candidates: their logits within the margin of the oracle's
        lg = np.take_along_axis(logits64, gid_gpu.astype(np.int64), -1)
        lr = np.take_along_axis(logits64, gid_ref.astype(np.int64), -1)
        assert np.all(np.abs(lg - lr)[flips] <= MARGIN * 1.0001)
    assert np.abs(gate_gpu - gate_ref)[same].max(initial=0.0) <= 1e-5
    return int(flips.sum())


def check_sort(gid_gpu, perm, inv, offsets, M):
    """Step 2: bit-exact against the oracle's sort of the same assignments."""
    o_off, o_perm, o_inv = oracle.sort(gid_gpu.cpu().numpy(), M)
    assert np.array_equal(offsets.cpu().numpy(), o_off)
    assert np.array_equal(perm.cpu().numpy(), o_perm)
    assert np.array_equal(inv.cpu().numpy().reshape(o_inv.shape), o_inv)
    return o_off, o_perm, o_inv


# Relative bounds, beside the absolute ones above.  With N(0, 1) inputs and groups of ~17,000 keys
# the outputs are of the order 1e-3, below the absolute bounds, so those alone would accept an
# output that is scaled or zero.  REL_FRO bounds ||got - want||_F / ||want||_F over the whole
# comparison; ROW bounds each row's largest error by a fraction of that row's largest magnitude
# (bf16: 2^-6, i.e. a few units in the last place of the 8-bit mantissa after two roundings).
REL_FRO = {"bf16": 1e-2, "f32": 1e-5}
ROW_REL = {"bf16": 2.0 ** -6, "f32": 2.0 ** -16}
ROW_ABS = 1e-5


def check_output(got, want, dtype, what="O"):
    """Absolute bounds (max, mean), the relative Frobenius error and a per-row relative bound;
    rows are the last axis.  Returns (max abs err, mean abs err, relative Frobenius err)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, f"{what}: shape {got.shape} vs {want.shape}"
    if got.size == 0:
        return 0.0, 0.0, 0.0
    err = np.abs(got - want)
    tol = TOL[dtype]
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    assert err.max(initial=0.0) <= tol["max_abs"], f"{what}: max abs err {err.max():.3e}"
    assert err.mean() <= tol["mean_abs"], f"{what}: mean abs err {err.mean():.3e}"
    norm = float(np.sqrt((want ** 2).sum()))
    rel = float(np.sqrt((err ** 2).sum())) / norm if norm > 0 else float(err.max() > 0)
    assert rel <= REL_FRO[dtype], f"{what}: relative Frobenius err {rel:.3e}"
    row_err = err.reshape(-1, err.shape[-1]).max(axis=1)
    row_mag = np.abs(want).reshape(-1, want.shape[-1]).max(axis=1)
    excess = row_err - (ROW_REL[dtype] * row_mag + ROW_ABS)
    worst = int(np.argmax(excess))
    assert excess[worst] <= 0, (f"{what}: row {worst}: err {row_err[worst]:.3e} against row magnitude "
                                f"{row_mag[worst]:.3e}")
    print(f"{what}: max abs {err.max():.3e}  mean abs {err.mean():.3e}  rel fro {rel:.3e}  "
          f"worst row err/mag {float((row_err / np.maximum(row_mag, 1e-30)).max()):.3e}")
    return float(err.max(initial=0.0)), float(err.mean()), rel


def grouped_case(sizes, H, D, dtype, seed, B=1, qscale=1.0, device="cuda"):
    """Tokens already in group-major order with the given group sizes: perm is the
    identity, so Qp/Kp/Vp are Q/K/V and moga_group_attn can be tested alone."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    T = int(sum(sizes))
    dt = torch.float32 if dtype == "f32" else torch.bfloat16
    Q = (torch.randn(B, H, T, D, generator=g) * qscale).to(dt)
    K = torch.randn(B, H, T, D, generator=g).to(dt)
    V = torch.randn(B, H, T, D, generator=g).to(dt)
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    offsets = np.broadcast_to(offsets, (B, len(sizes) + 1)).copy()
    gid = np.repeat(np.arange(len(sizes)), sizes).astype(np.int32)
    gid = np.broadcast_to(gid[None, :, None], (B, T, 1)).copy()
    perm = np.broadcast_to(np.arange(T, dtype=np.int32), (B, T)).copy()
    return dict(Q=Q.to(device), K=K.to(device), V=V.to(device), offsets=offsets, gid=gid, perm=perm,
                T=T)
