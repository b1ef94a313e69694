"""Head-sharded MoGA forward for several GPUs (Sec. 3.2, last paragraph: routing composes with
sequence parallelism because routing scores are computed per token "with whole heads", and
the routing results are then aggregated across all tokens).

Layout per rank r of P: a token shard of X ([B, N/P, C], all channels) and a head shard of
Q, K, V ([B, H/P, N, D], all tokens) -- the state after the "sequence gather and head
scatter" exchange of the surrounding model.  The path has ONE exchange step: every rank
routes its own tokens, the (gid, gate) pairs are all-gathered (8*k bytes per token: 4.5 MB at
561,600 tokens), and every rank then sorts the same assignments (deterministic, identical
everywhere) and runs gather / group attention / gated inverse permutation on its own heads.
No collective touches Q, K, V or O.

torch.distributed is the plumbing (NCCL on GPUs, gloo in the CPU tests); every arithmetic step
is a C-ABI stage call.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_bounds(n: int, parts: int, index: int):
    """Contiguous split of n items in `parts` shards whose sizes differ by at most one."""
    base, extra = divmod(n, parts)
    lo = index * base + min(index, extra)
    return lo, lo + base + (1 if index < extra else 0)


def gather_routing(gid_local: torch.Tensor, gate_local: torch.Tensor, n_total: int, group=None):
    """All-gather the routing results of the token shards into [B, N, k] tensors.

    gid_local / gate_local: [B, n_r, k] for this rank's tokens [lo_r, hi_r) as given by
    shard_bounds(n_total, world, rank).  Shards may differ by one token, so they travel padded
    to the largest shard and are trimmed on arrival."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return gid_local, gate_local
    B, _, k = gid_local.shape
    n_max = -(-n_total // world)
    pad_g = gid_local.new_zeros(B, n_max, k)
    pad_t = gate_local.new_zeros(B, n_max, k)
    pad_g[:, :gid_local.shape[1]] = gid_local
    pad_t[:, :gate_local.shape[1]] = gate_local
    all_g = [torch.empty_like(pad_g) for _ in range(world)]
    all_t = [torch.empty_like(pad_t) for _ in range(world)]
    dist.all_gather(all_g, pad_g, group=group)
    dist.all_gather(all_t, pad_t, group=group)
    gid = gid_local.new_empty(B, n_total, k)
    gate = gate_local.new_empty(B, n_total, k)
    for r in range(world):
        lo, hi = shard_bounds(n_total, world, r)
        gid[:, lo:hi] = all_g[r][:, :hi - lo]
        gate[:, lo:hi] = all_t[r][:, :hi - lo]
    return gid, gate


def forward_head_sharded(mb, cfg, X_local, Wr, bias, Q_heads, K_heads, V_heads, O_heads, group=None):
    """One MoGA forward on this rank's shards.  cfg describes the WHOLE problem (N tokens,
    H heads); X_local holds tokens shard_bounds(N, world, rank), Q/K/V/O_heads hold heads
    shard_bounds(H, world, rank) as contiguous [B, h_r, N, D].  Returns (gid, gate, offsets) of
    the whole sequence (identical on every rank)."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    lo, hi = shard_bounds(cfg.N, world, rank)
    h_lo, h_hi = shard_bounds(cfg.H, world, rank)
    assert X_local.shape[1] == hi - lo and Q_heads.shape[1] == h_hi - h_lo
    dev = X_local.device
    # 1. route this rank's tokens (all heads share one routing: the whole hidden vector is local)
    cfg_tok = cfg.with_(N=hi - lo)
    sh_tok = mb.make_shape(cfg_tok)
    gid_l = torch.empty(cfg.B, hi - lo, cfg.k, dtype=torch.int32, device=dev)
    gate_l = torch.empty(cfg.B, hi - lo, cfg.k, dtype=torch.float32, device=dev)
    ws_tok = mb.alloc_workspace(mb.moga_scratch_bytes(sh_tok), dev)
    mb.moga_route(sh_tok, X_local, Wr, bias, gid_l, gate_l, None, ws_tok)
    # 2. the one exchange step
    gid, gate = gather_routing(gid_l, gate_l, cfg.N, group)
    # 3. sort + gather + attention + gated inverse permutation on this rank's heads
    cfg_h = cfg.with_(H=h_hi - h_lo)
    sh = mb.make_shape(cfg_h)
    T = cfg.N * cfg.k
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh), dev)
    perm = torch.empty(cfg.B, T, dtype=torch.int32, device=dev)
    inv = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device=dev)
    offsets = torch.empty(cfg.B, cfg.M + 1, dtype=torch.int32, device=dev)
    Qp, Kp, Vp, Op = (torch.empty(cfg.B, cfg_h.H, T, cfg.D, dtype=Q_heads.dtype, device=dev) for _ in range(4))
    mb.moga_permute(sh, gid, Q_heads, K_heads, V_heads, perm, inv, offsets, Qp, Kp, Vp, ws)
    mb.moga_group_attn(sh, Qp, Kp, Vp, offsets, Op, None, ws)
    mb.moga_unpermute(sh, Op, inv, gate, O_heads)
    return gid, gate, offsets
