"""GPU parity of the backward of the routed group attention (bf16 with d_head = 128 on the tensor
cores, fp32 with d_head 64 / 128 on the fp32 ALUs) against the fp64
oracle: the forward is run with the stage calls (which keep the sorted-order tensors and lse the
backward needs), an upstream gradient dO is drawn, and dQ, dK, dV, dgate are compared.

Tolerance: the kernels round the softmax weights, dS, the scaled upstream
gradient and the sorted-order results to bf16 (2^-9 each) and accumulate in fp32, and the forward
output they take as saved input is itself bf16: relative Frobenius error <= 1e-2 per gradient
(measured ~3e-3), largest error <= 2^-5 of the tensor's largest magnitude.  The fp32 path rounds
nothing below fp32 (sums of a few hundred fp32 products, exp to ~2 ulp): relative Frobenius error
<= 1e-5, largest error <= 2^-16 of the largest magnitude."""
import numpy as np
import pytest
import torch

import oracle
from parity import to_np32
from paper_2510_18692_b200.inputs import GATE_SOFTMAX_ALL, GATE_SOFTMAX_TOPK, MogaConfig, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mb():
    from paper_2510_18692_b200 import build
    build.build()
    from paper_2510_18692_b200 import binding
    return binding


def _staged_forward(mb, cfg, inp):
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    T = cfg.N * cfg.k
    dev = "cuda"
    gid = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device=dev)
    gate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device=dev)
    perm = torch.empty(cfg.B, T, dtype=torch.int32, device=dev)
    inv = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device=dev)
    offsets = torch.empty(cfg.B, cfg.M + 1, dtype=torch.int32, device=dev)
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    Qp, Kp, Vp, Op = (torch.empty(cfg.B, cfg.H, T, cfg.D, dtype=dt, device=dev) for _ in range(4))
    lse = torch.empty(cfg.B, cfg.H, T, dtype=torch.float32, device=dev)
    mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], gid, gate, None, ws)
    mb.moga_permute(sh, gid, inp["Q"], inp["K"], inp["V"], perm, inv, offsets, Qp, Kp, Vp, ws)
    mb.moga_group_attn(sh, Qp, Kp, Vp, offsets, Op, lse, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    return sh, dict(gid=gid, gate=gate, perm=perm, inv=inv, offsets=offsets, Qp=Qp, Kp=Kp, Vp=Vp, Op=Op, lse=lse)


CASES = [
    MogaConfig("b_top1", 1, 2, 1000, 128, 128, 4, 1, "bf16", GATE_SOFTMAX_ALL, 51),
    MogaConfig("b_top2", 2, 2, 700, 128, 128, 6, 2, "bf16", GATE_SOFTMAX_TOPK, 52),
    MogaConfig("b_ragged", 1, 3, 1111, 128, 128, 16, 1, "bf16", GATE_SOFTMAX_ALL, 53, zipf_bias=2.0),   # sizes 0, 1, ... hundreds
    MogaConfig("b_one_group", 1, 1, 385, 64, 128, 1, 1, "bf16", GATE_SOFTMAX_ALL, 54),
    MogaConfig("f_top1_d64", 2, 2, 333, 64, 64, 4, 1, "f32", GATE_SOFTMAX_ALL, 55),
    MogaConfig("f_top2_d128", 1, 2, 301, 64, 128, 5, 2, "f32", GATE_SOFTMAX_TOPK, 56),
    MogaConfig("f_ragged_d64", 1, 3, 500, 64, 64, 16, 1, "f32", GATE_SOFTMAX_ALL, 57, zipf_bias=2.0),
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_backward_matches_oracle(mb, cfg):
    inp = make_inputs(cfg, device="cuda")
    sh, fw = _staged_forward(mb, cfg, inp)
    g = torch.Generator(device="cuda").manual_seed(cfg.seed)
    dO = torch.randn(cfg.B, cfg.H, cfg.N, cfg.D, generator=g, device="cuda").to(inp["Q"].dtype)
    rel_bound, max_bound = (1e-2, 2.0 ** -5) if cfg.dtype == "bf16" else (1e-5, 2.0 ** -16)
    dQ, dK, dV = (torch.full_like(inp["Q"], float("nan")) for _ in range(3))
    dgate = torch.full((cfg.B, cfg.N, cfg.k), float("nan"), dtype=torch.float32, device="cuda")
    ws = mb.alloc_workspace(mb.moga_backward_workspace_bytes(sh))
    mb.moga_backward(sh, fw["Qp"], fw["Kp"], fw["Vp"], fw["Op"], fw["lse"], fw["gate"], fw["perm"], fw["inv"],
                     fw["offsets"], dO, dQ, dK, dV, dgate, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    want = oracle.backward(to_np32(inp["Q"]), to_np32(inp["K"]), to_np32(inp["V"]), fw["gid"].cpu().numpy(),
                           fw["gate"].double().cpu().numpy(), to_np32(dO), cfg.scale, cfg.M)
    for name, got, ref in (("dQ", dQ, want[0]), ("dK", dK, want[1]), ("dV", dV, want[2]), ("dgate", dgate, want[3])):
        got = got.double().cpu().numpy()
        assert np.all(np.isfinite(got)), name
        err = np.abs(got - ref)
        rel = float(np.sqrt((err ** 2).sum() / max((ref ** 2).sum(), 1e-300)))
        print(f"{name}: rel fro {rel:.3e}  max err {err.max():.3e}  max |ref| {np.abs(ref).max():.3e}")
        assert rel <= rel_bound, (name, rel)
        assert err.max() <= max_bound * np.abs(ref).max() + 1e-6, (name, err.max())
    # determinism: the same call twice gives the same bits
    dQ2, dK2, dV2 = (torch.empty_like(dQ) for _ in range(3))
    dg2 = torch.empty_like(dgate)
    mb.moga_backward(sh, fw["Qp"], fw["Kp"], fw["Vp"], fw["Op"], fw["lse"], fw["gate"], fw["perm"], fw["inv"],
                     fw["offsets"], dO, dQ2, dK2, dV2, dg2, ws)
    torch.cuda.synchronize()
    assert torch.equal(dQ, dQ2) and torch.equal(dK, dK2) and torch.equal(dV, dV2) and torch.equal(dgate, dg2)


def test_backward_rejects_unsupported_shapes(mb):
    cfg = MogaConfig("b_d64", 1, 1, 64, 64, 64, 2, 1, "bf16", GATE_SOFTMAX_ALL, 1)
    sh = mb.make_shape(cfg)
    t = torch.zeros(16, dtype=torch.int32, device="cuda")
    ws = mb.alloc_workspace(max(mb.moga_backward_workspace_bytes(sh), 256))
    with pytest.raises(mb.MogaError) as e:
        mb.moga_backward(sh, t, t, t, t, t, t, t, t, t, t, t, t, t, t, ws)
    assert e.value.code == 2


def test_backward_clip_size_one_head(mb):
    """The single-clip workload (32,760 tokens, groups of ~4,100: 32 tiles per item, 64-bit offsets
    in play for the other heads' rows): gradients of head 0 against the oracle run on that head
    alone (heads are independent in dQ, dK, dV; dgate sums over heads and is checked in the small
    cases)."""
    from paper_2510_18692_b200.inputs import CONFIGS
    cfg = CONFIGS["clip_bf16"]
    inp = make_inputs(cfg, device="cuda")
    sh, fw = _staged_forward(mb, cfg, inp)
    g = torch.Generator(device="cuda").manual_seed(7)
    dO = torch.randn(cfg.B, cfg.H, cfg.N, cfg.D, generator=g, device="cuda").to(torch.bfloat16)
    dQ, dK, dV = (torch.empty_like(inp["Q"]) for _ in range(3))
    dgate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device="cuda")
    ws = mb.alloc_workspace(mb.moga_backward_workspace_bytes(sh))
    mb.moga_backward(sh, fw["Qp"], fw["Kp"], fw["Vp"], fw["Op"], fw["lse"], fw["gate"], fw["perm"], fw["inv"],
                     fw["offsets"], dO, dQ, dK, dV, dgate, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    h = 0
    want = oracle.backward(to_np32(inp["Q"][:, h:h + 1]), to_np32(inp["K"][:, h:h + 1]), to_np32(inp["V"][:, h:h + 1]),
                           fw["gid"].cpu().numpy(), fw["gate"].double().cpu().numpy(), to_np32(dO[:, h:h + 1]),
                           cfg.scale, cfg.M)
    for name, got, ref in (("dQ", dQ, want[0]), ("dK", dK, want[1]), ("dV", dV, want[2])):
        got = got[:, h:h + 1].double().cpu().numpy()
        err = np.abs(got - ref)
        rel = float(np.sqrt((err ** 2).sum() / (ref ** 2).sum()))
        print(f"{name}: rel fro {rel:.3e}  max err {err.max():.3e}  max |ref| {np.abs(ref).max():.3e}")
        assert np.all(np.isfinite(got)) and rel <= 1e-2, (name, rel)


ROUTE_BWD = [
    MogaConfig("rb_all_top1", 2, 1, 1500, 256, 64, 8, 1, "bf16", GATE_SOFTMAX_ALL, 61),
    MogaConfig("rb_all_top2", 1, 1, 777, 136, 64, 5, 2, "bf16", GATE_SOFTMAX_ALL, 62),
    MogaConfig("rb_topk", 1, 1, 3000, 320, 64, 64, 2, "bf16", GATE_SOFTMAX_TOPK, 63, zipf_bias=2.0),
    MogaConfig("rb_f32", 1, 1, 1000, 96, 64, 16, 3, "f32", GATE_SOFTMAX_TOPK, 64),
    MogaConfig("rb_m1", 1, 1, 300, 64, 64, 1, 1, "bf16", GATE_SOFTMAX_ALL, 65),
]


@pytest.mark.parametrize("cfg", ROUTE_BWD, ids=lambda c: c.name)
def test_route_backward_matches_oracle(mb, cfg):
    """dX, dW_r, dbias of the router against the fp64 oracle, from the GPU's own routing and logits.
    Tolerances: dW_r and dbias are fp32 sums over the tokens (relative 1e-4 of the largest entry);
    dX is rounded to the type of X (bf16: 2^-8 of the row's magnitude); dr itself depends on the
    fp32 logits (2e-5) through a softmax."""
    inp = make_inputs(cfg, device="cuda", heads=[])
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    gid = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device="cuda")
    gate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device="cuda")
    logits = torch.empty(cfg.B, cfg.N, cfg.M, dtype=torch.float32, device="cuda")
    mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], gid, gate, logits, ws)
    g = torch.Generator(device="cuda").manual_seed(cfg.seed)
    dgate = torch.randn(cfg.B, cfg.N, cfg.k, generator=g, device="cuda")
    dX = torch.full_like(inp["X"], float("nan"))
    dWr = torch.full_like(inp["Wr"], float("nan"))
    dbias = torch.full((cfg.M,), float("nan"), device="cuda")
    wsb = mb.alloc_workspace(mb.moga_route_backward_workspace_bytes(sh))
    outs = []
    for _ in range(2):
        mb.moga_route_backward(sh, inp["X"], inp["Wr"], logits, gid, dgate, dX, dWr, dbias, wsb)
        torch.cuda.synchronize()
        outs.append((dX.clone(), dWr.clone(), dbias.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)                                   # fixed summation order: bit-reproducible
    _, o_dX, o_dWr, o_db = oracle.route_backward(to_np32(inp["X"]), inp["Wr"].cpu().numpy(),
                                                 None if inp["bias"] is None else inp["bias"].cpu().numpy(),
                                                 gid.cpu().numpy(), dgate.double().cpu().numpy(), cfg.gate_mode)
    got_w, got_b, got_x = dWr.double().cpu().numpy(), dbias.double().cpu().numpy(), dX.double().cpu().numpy()
    assert np.abs(got_w - o_dWr).max() <= 1e-4 * max(np.abs(o_dWr).max(), 1e-6) + 1e-7
    assert np.abs(got_b - o_db).max() <= 1e-4 * max(np.abs(o_db).max(), 1e-6) + 1e-6
    tol = (2.0 ** -8 if cfg.dtype == "bf16" else 1e-5) * np.abs(o_dX).max(axis=-1, keepdims=True) + 1e-6
    assert np.all(np.abs(got_x - o_dX) <= tol)
