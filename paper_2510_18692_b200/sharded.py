"""Head-sharded MoGA forward for several GPUs.

Sec. 3.2, last paragraph of the method: the router sees each token's whole hidden vector, so
routing can run on token shards before the model's sequence-to-head exchange, and the
routing results of all tokens are then collected on every rank.

Layout per rank r of P: a token shard of X ([B, N/P, C], all channels) and a head shard of
Q, K, V ([B, H/P, N, D], all tokens), i.e. the state after that exchange of the surrounding
model.  The path has ONE exchange step: every rank routes its own tokens, the (gid, gate)
pairs travel as packed 8-byte words in one all-gather (8*k bytes per token: 4.5 MB at 561,600
tokens), and every rank then runs ``moga_forward_routed`` -- sort, gather, group attention and
gated inverse permutation with the same kernels as the unsharded forward -- on its own
heads.  The sort is deterministic, so all ranks hold identical offsets.  No collective
touches Q, K, V or O.

torch.distributed is the plumbing (NCCL on GPUs, gloo in the CPU tests); every arithmetic step
is a C-ABI call.  All buffers are allocated once, in ``ShardPlan``.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_bounds(n: int, parts: int, index: int):
    """Contiguous split of n items in `parts` shards whose sizes differ by at most one."""
    base, extra = divmod(n, parts)
    lo = index * base + min(index, extra)
    return lo, lo + base + (1 if index < extra else 0)


def _world(group=None):
    if dist.is_available() and dist.is_initialized():
        return dist.get_world_size(group), dist.get_rank(group)
    return 1, 0


class RoutingExchange:
    """Buffers and index of the one all-gather: [B, n_r, k] (gid int32, gate fp32) per rank in,
    [B, N, k] of both out.  A pair travels as two 32-bit words side by side, shards padded to
    the largest shard; `valid` picks the real tokens out of the padded result."""

    def __init__(self, B: int, n_total: int, k: int, device, group=None):
        self.group = group
        self.world, self.rank = _world(group)
        self.B, self.N, self.k = B, n_total, k
        self.lo, self.hi = shard_bounds(n_total, self.world, self.rank)
        self.n_max = -(-n_total // self.world) if n_total else 0
        self.send = torch.zeros(B, self.n_max, k, 2, dtype=torch.int32, device=device)
        self.recv = torch.empty(self.world, B, self.n_max, k, 2, dtype=torch.int32, device=device)
        idx = []
        for r in range(self.world):
            lo, hi = shard_bounds(n_total, self.world, r)
            idx.append(torch.arange(hi - lo, dtype=torch.int64) + r * self.n_max)
        self.valid = torch.cat(idx).to(device) if idx else torch.empty(0, dtype=torch.int64, device=device)
        self.gid = torch.empty(B, n_total, k, dtype=torch.int32, device=device)
        self.gate = torch.empty(B, n_total, k, dtype=torch.float32, device=device)

    def __call__(self, gid_local: torch.Tensor, gate_local: torch.Tensor):
        """Returns (gid, gate) of all N tokens (views of buffers owned by this object)."""
        if self.world == 1:
            return gid_local, gate_local
        n = self.hi - self.lo
        self.send[:, :n, :, 0] = gid_local
        self.send[:, :n, :, 1] = gate_local.view(torch.int32)        # bit copy, no conversion
        dist.all_gather_into_tensor(self.recv.view(-1), self.send.view(-1), group=self.group)   # rank-major
        # [world, B, n_max, k, 2] -> [B, world * n_max, k, 2] -> the N real tokens
        flat = self.recv.permute(1, 0, 2, 3, 4).reshape(self.B, self.world * self.n_max, self.k, 2)
        both = flat.index_select(1, self.valid)
        self.gid.copy_(both[..., 0])
        self.gate.copy_(both[..., 1].contiguous().view(torch.float32))
        return self.gid, self.gate


def gather_routing(gid_local: torch.Tensor, gate_local: torch.Tensor, n_total: int, group=None):
    """One-off form of RoutingExchange (allocates its buffers): all-gather the routing results of
    the token shards into [B, N, k] tensors."""
    B, _, k = gid_local.shape
    return RoutingExchange(B, n_total, k, gid_local.device, group)(gid_local, gate_local)


class ShardPlan:
    """Everything a rank needs for repeated head-sharded forwards of one configuration: shapes of
    its token shard and head shard, the two workspaces, the local routing outputs and the
    exchange buffers.  `cfg` describes the WHOLE problem (N tokens, H heads)."""

    def __init__(self, mb, cfg, device, group=None):
        self.mb, self.cfg = mb, cfg
        self.world, self.rank = _world(group)
        self.tok = shard_bounds(cfg.N, self.world, self.rank)
        self.heads = shard_bounds(cfg.H, self.world, self.rank)
        n_r, h_r = self.tok[1] - self.tok[0], self.heads[1] - self.heads[0]
        self.sh_tok = mb.make_shape(cfg.with_(N=n_r))
        self.sh_heads = mb.make_shape(cfg.with_(H=max(h_r, 1)))
        self.h_r = h_r
        self.ws_tok = mb.alloc_workspace(mb.moga_scratch_bytes(self.sh_tok), device)
        self.ws = mb.alloc_workspace(mb.moga_workspace_bytes(self.sh_heads) if h_r else 256, device)
        self.gid_l = torch.empty(cfg.B, n_r, cfg.k, dtype=torch.int32, device=device)
        self.gate_l = torch.empty(cfg.B, n_r, cfg.k, dtype=torch.float32, device=device)
        self.exchange = RoutingExchange(cfg.B, cfg.N, cfg.k, device, group)
        self.offsets = torch.empty(cfg.B, cfg.M + 1, dtype=torch.int32, device=device)

    def forward(self, X_local, Wr, bias, Q_heads, K_heads, V_heads, O_heads):
        """One MoGA forward on this rank's shards: X_local holds tokens self.tok, Q/K/V/O_heads hold
        heads self.heads as contiguous [B, h_r, N, D].  Returns (gid, gate, offsets) of the whole
        sequence (identical on every rank)."""
        mb, cfg = self.mb, self.cfg
        assert X_local.shape[1] == self.tok[1] - self.tok[0] and Q_heads.shape[1] == self.h_r
        # 1. route this rank's tokens (all heads share one routing: the whole hidden vector is local)
        if self.gid_l.shape[1]:
            mb.moga_route(self.sh_tok, X_local, Wr, bias, self.gid_l, self.gate_l, None, self.ws_tok)
        # 2. the one exchange step
        gid, gate = self.exchange(self.gid_l, self.gate_l)
        # 3. sort + gather + attention + gated inverse permutation on this rank's heads
        if self.h_r:
            mb.moga_forward_routed(self.sh_heads, gid, gate, Q_heads, K_heads, V_heads, O_heads, self.ws,
                                   None, self.offsets)
        return gid, gate, self.offsets


def forward_head_sharded(mb, cfg, X_local, Wr, bias, Q_heads, K_heads, V_heads, O_heads, group=None, plan=None):
    """Convenience form: builds a ShardPlan when none is given (allocating; pass `plan` in a loop)."""
    plan = plan or ShardPlan(mb, cfg, X_local.device, group)
    return plan.forward(X_local, Wr, bias, Q_heads, K_heads, V_heads, O_heads)
