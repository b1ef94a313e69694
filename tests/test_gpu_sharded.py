"""Sharding semantics of the multi-GPU path checked on one GPU, rank by rank and without any
collective: routing token shards separately gives the bits of routing the whole sequence,
and running the stages on head shards gives the bits of running them on all heads."""
import numpy as np
import pytest
import torch

import oracle
from parity import check_output, to_np32
from paper_2510_18692_b200.inputs import GATE_SOFTMAX_TOPK, MogaConfig, make_inputs
from paper_2510_18692_b200.sharded import forward_head_sharded, shard_bounds

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mb():
    from paper_2510_18692_b200 import build
    build.build()
    from paper_2510_18692_b200 import binding
    return binding


def test_shards_reproduce_the_unsharded_stages(mb):
    cfg = MogaConfig("sh", 2, 5, 1777, 256, 128, 8, 2, "bf16", GATE_SOFTMAX_TOPK, 41)
    inp = make_inputs(cfg, device="cuda")
    # world size 1: the sharded driver is the staged forward
    O = torch.empty_like(inp["Q"])
    mb.moga_set_fused_topk(False)          # the staged top-2 path, which the stage calls below reproduce bit for bit
    try:
        gid, gate, offsets = forward_head_sharded(mb, cfg, inp["X"], inp["Wr"], inp["bias"], inp["Q"], inp["K"],
                                                  inp["V"], O)
        torch.cuda.synchronize()
    finally:
        mb.moga_set_fused_topk(False)
    host = {k: to_np32(v) for k, v in inp.items()}
    off, perm, _ = oracle.sort(gid.cpu().numpy(), cfg.M)
    want = oracle.attn_all(host["Q"], host["K"], host["V"], gid.cpu().numpy(), gate.double().cpu().numpy(), off,
                           perm, cfg.scale)
    check_output(O.float().cpu().numpy(), want, "bf16")
    world = 3
    # routing token shards one by one (what each rank would do) and concatenating
    parts_g, parts_t = [], []
    for r in range(world):
        lo, hi = shard_bounds(cfg.N, world, r)
        sh = mb.make_shape(cfg.with_(N=hi - lo))
        g = torch.empty(cfg.B, hi - lo, cfg.k, dtype=torch.int32, device="cuda")
        t = torch.empty(cfg.B, hi - lo, cfg.k, dtype=torch.float32, device="cuda")
        ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
        mb.moga_route(sh, inp["X"][:, lo:hi].contiguous(), inp["Wr"], inp["bias"], g, t, None, ws)
        parts_g.append(g)
        parts_t.append(t)
    assert torch.equal(torch.cat(parts_g, 1), gid) and torch.equal(torch.cat(parts_t, 1), gate)
    # head shards one by one with the gathered routing
    T = cfg.N * cfg.k
    for r in range(world):
        lo, hi = shard_bounds(cfg.H, world, r)
        cfg_h = cfg.with_(H=hi - lo)
        sh = mb.make_shape(cfg_h)
        ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
        perm_d = torch.empty(cfg.B, T, dtype=torch.int32, device="cuda")
        inv = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device="cuda")
        offs = torch.empty(cfg.B, cfg.M + 1, dtype=torch.int32, device="cuda")
        Qh, Kh, Vh = (inp[n][:, lo:hi].contiguous() for n in ("Q", "K", "V"))
        Qp, Kp, Vp, Op = (torch.empty(cfg.B, hi - lo, T, cfg.D, dtype=torch.bfloat16, device="cuda") for _ in range(4))
        Oh = torch.empty_like(Qh)
        mb.moga_permute(sh, gid, Qh, Kh, Vh, perm_d, inv, offs, Qp, Kp, Vp, ws)
        mb.moga_group_attn(sh, Qp, Kp, Vp, offs, Op, None, ws)
        mb.moga_unpermute(sh, Op, inv, gate, Oh)
        torch.cuda.synchronize()
        assert torch.equal(offs, offsets) and torch.equal(Oh, O[:, lo:hi])


@pytest.mark.parametrize("k,gate_mode", [(1, 0), (2, GATE_SOFTMAX_TOPK)])
def test_forward_from_a_given_routing_is_the_forward(mb, k, gate_mode):
    """moga_forward_routed fed with the routing moga_forward computed gives moga_forward's bits
    (same kernels, the fused epilogue included), for all heads and for a head shard."""
    cfg = MogaConfig("fr", 1, 4, 3001, 256, 128, 8, k, "bf16", gate_mode, 43)
    inp = make_inputs(cfg, device="cuda")
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_workspace_bytes(sh))
    O = torch.empty_like(inp["Q"])
    gid = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device="cuda")
    gate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device="cuda")
    offsets = torch.empty(cfg.B, cfg.M + 1, dtype=torch.int32, device="cuda")
    mb.moga_forward(sh, inp["X"], inp["Wr"], inp["bias"], inp["Q"], inp["K"], inp["V"], O, ws, gid, gate, None, offsets)
    assert mb.moga_last_device_status(ws) == (0, 0)
    O2 = torch.full_like(O, float("nan"))
    off2 = torch.empty_like(offsets)
    mb.moga_forward_routed(sh, gid, gate, inp["Q"], inp["K"], inp["V"], O2, ws, None, off2)
    assert mb.moga_last_device_status(ws) == (0, 0)
    assert torch.equal(O2, O) and torch.equal(off2, offsets)
    cfg_h = cfg.with_(H=1)
    sh_h = mb.make_shape(cfg_h)
    ws_h = mb.alloc_workspace(mb.moga_workspace_bytes(sh_h))
    Qh, Kh, Vh = (inp[n][:, 2:3].contiguous() for n in ("Q", "K", "V"))
    Oh = torch.empty_like(Qh)
    mb.moga_forward_routed(sh_h, gid, gate, Qh, Kh, Vh, Oh, ws_h)
    assert mb.moga_last_device_status(ws_h) == (0, 0)
    assert torch.equal(Oh, O[:, 2:3])
