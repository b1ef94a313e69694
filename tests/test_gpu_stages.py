"""GPU parity of each C-ABI stage against the fp64 oracle, on shapes that span
several tiles with ragged tails and on the degenerate cases (empty and 1-token
groups, M = 1, k = M)."""
import math

import numpy as np
import pytest
import torch

import oracle
from parity import check_output, check_routing, check_sort, grouped_case, to_np32
from paper_2510_18692_b200.inputs import (GATE_SOFTMAX_ALL, GATE_SOFTMAX_TOPK, MogaConfig,
                                          make_inputs)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mb():
    from paper_2510_18692_b200 import build
    build.build()
    from paper_2510_18692_b200 import binding
    return binding


def _cfg(**kw):
    base = dict(name="t", B=1, H=2, N=1000, C=128, D=64, M=8, k=1, dtype="f32",
                gate_mode=GATE_SOFTMAX_ALL, seed=0)
    base.update(kw)
    return MogaConfig(**base)


ROUTE_CASES = [
    _cfg(),                                                            # fp32, ragged token tail
    _cfg(M=1),
    _cfg(M=2, k=2, gate_mode=GATE_SOFTMAX_TOPK, N=777, C=72),          # k = M, C not a chunk multiple
    _cfg(dtype="bf16", M=8, C=1536, N=3001, seed=1),
    _cfg(dtype="bf16", M=16, k=2, gate_mode=GATE_SOFTMAX_TOPK, C=640, N=2500, B=2, seed=2),
    _cfg(dtype="bf16", M=32, C=1024, N=4099, seed=3),
    _cfg(dtype="bf16", M=64, k=2, gate_mode=GATE_SOFTMAX_TOPK, C=768, N=2051, zipf_bias=2.0, seed=4),
    _cfg(dtype="bf16", M=5, k=3, gate_mode=GATE_SOFTMAX_ALL, C=264, N=515, seed=5),
    _cfg(dtype="f32", M=33, k=8, gate_mode=GATE_SOFTMAX_TOPK, C=100, N=300, seed=6),
    _cfg(dtype="bf16", M=32, C=5120, N=20000, seed=7),                 # long accumulation, many tiles per CTA
    _cfg(dtype="bf16", M=3, k=2, gate_mode=GATE_SOFTMAX_TOPK, C=40, N=130, seed=8),   # less than one chunk
    _cfg(dtype="bf16", M=64, k=8, gate_mode=GATE_SOFTMAX_ALL, C=2048, N=1, seed=9),   # a single token
    _cfg(dtype="bf16", M=64, k=2, gate_mode=GATE_SOFTMAX_TOPK, C=5120, N=9000, seed=10),
    _cfg(dtype="bf16", M=16, k=2, gate_mode=GATE_SOFTMAX_TOPK, C=5120, N=9000, seed=11),
]


@pytest.mark.parametrize("path", ["alu", "tensor"])
@pytest.mark.parametrize("cfg", ROUTE_CASES, ids=lambda c: f"{c.dtype}-M{c.M}-k{c.k}-C{c.C}-N{c.N}")
def test_route(mb, cfg, path):
    """Both router kernels against the fp64 oracle: the fp32-ALU kernel (no workspace) and,
    for bf16 features, the tensor-core kernel (split weights, chosen when a workspace is given)."""
    if path == "tensor" and cfg.dtype != "bf16":
        pytest.skip("the tensor-core router takes bf16 features")
    inp = make_inputs(cfg, device="cuda", heads=[])
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh)) if path == "tensor" else None
    gid = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device="cuda")
    gate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device="cuda")
    logits = torch.empty(cfg.B, cfg.N, cfg.M, dtype=torch.float32, device="cuda")
    mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], gid, gate, logits, ws)
    if ws is not None:
        assert mb.moga_last_device_status(ws) == (0, 0)
    torch.cuda.synchronize()
    o_gid, o_gate, o_logits = oracle.route(to_np32(inp["X"]), to_np32(inp["Wr"]), to_np32(inp["bias"]),
                                           cfg.k, cfg.gate_mode, want_logits=True)
    assert np.abs(logits.cpu().numpy() - o_logits).max() <= 2e-5 * max(1.0, np.abs(o_logits).max())
    flips = check_routing(gid, gate, o_logits, o_gid, o_gate, cfg.k)
    assert flips <= max(2, int(cfg.B * cfg.N * cfg.k * 1e-3))
    # without the optional logits output the decisions are the same bits
    gid2, gate2 = torch.empty_like(gid), torch.empty_like(gate)
    mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], gid2, gate2, None, ws)
    torch.cuda.synchronize()
    assert torch.equal(gid, gid2) and torch.equal(gate, gate2)
    if path == "tensor":
        # route_mode = ALU overrides the choice even with a workspace: same bits as the ALU kernel alone
        sh_alu = mb.make_shape(cfg, route_mode=mb.MOGA_ROUTE_ALU)
        g3, g4 = torch.empty_like(gid), torch.empty_like(gid)
        t3, t4 = torch.empty_like(gate), torch.empty_like(gate)
        mb.moga_route(sh_alu, inp["X"], inp["Wr"], inp["bias"], g3, t3, None, ws)
        mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], g4, t4, None, None)
        torch.cuda.synchronize()
        assert torch.equal(g3, g4) and torch.equal(t3, t4)


def _random_gid(B, N, M, k, seed, skew=False, empty=()):
    rng = np.random.default_rng(seed)
    p = np.arange(1, M + 1, dtype=np.float64) ** (-2.0 if skew else 0.0)
    for e in empty:
        p[e] = 0.0
    p /= p.sum()
    gid = np.empty((B, N, k), np.int32)
    for b in range(B):
        for n in range(N):
            gid[b, n] = rng.choice(M, size=k, replace=False, p=p)
    return gid


SORT_CASES = [(1, 5000, 8, 1, False, ()), (2, 9001, 16, 2, False, (3,)), (1, 20000, 64, 2, True, (0, 63)),
              (1, 1, 4, 1, False, ()), (1, 4096, 1, 1, False, ()), (3, 4097, 2, 2, False, ()),
              (1, 12345, 32, 1, True, (5, 6, 7))]


@pytest.mark.parametrize("B,N,M,k,skew,empty", SORT_CASES)
def test_sort_and_gather(mb, B, N, M, k, skew, empty):
    cfg = _cfg(B=B, N=N, M=M, k=k, H=2, D=64, dtype="bf16", seed=7)
    rng = np.random.default_rng(N)
    if k <= M - len(empty):
        gid_np = _random_gid(B, N, M, k, seed=N, skew=skew, empty=empty)
    else:
        gid_np = np.broadcast_to(np.arange(k, dtype=np.int32), (B, N, k)).copy()
    gid = torch.from_numpy(gid_np).cuda()
    sh = mb.make_shape(cfg)
    T = N * k
    perm = torch.empty(B, T, dtype=torch.int32, device="cuda")
    inv = torch.empty(B, N, k, dtype=torch.int32, device="cuda")
    offsets = torch.empty(B, M + 1, dtype=torch.int32, device="cuda")
    g = torch.Generator().manual_seed(1)
    Q, K, V = (torch.randn(B, cfg.H, N, cfg.D, generator=g).bfloat16().cuda() for _ in range(3))
    Qp, Kp, Vp = (torch.empty(B, cfg.H, T, cfg.D, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    mb.moga_permute(sh, gid, Q, K, V, perm, inv, offsets, Qp, Kp, Vp, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    _, o_perm, _ = check_sort(gid, perm, inv, offsets, M)
    idx = torch.from_numpy(o_perm.astype(np.int64)).cuda()
    for src, dst in ((Q, Qp), (K, Kp), (V, Vp)):
        want = torch.gather(src, 2, idx[:, None, :, None].expand(B, cfg.H, T, cfg.D))
        assert torch.equal(dst, want)
    # indices only
    perm2, inv2, off2 = torch.empty_like(perm), torch.empty_like(inv), torch.empty_like(offsets)
    mb.moga_permute(sh, gid, None, None, None, perm2, inv2, off2, None, None, None, ws)
    torch.cuda.synchronize()
    assert torch.equal(perm, perm2) and torch.equal(inv, inv2) and torch.equal(offsets, off2)


def test_sort_reports_bad_group_id(mb):
    cfg = _cfg(N=100, M=4)
    gid = torch.zeros(1, 100, 1, dtype=torch.int32, device="cuda")
    gid[0, 17, 0] = 9
    sh = mb.make_shape(cfg)
    perm = torch.empty(1, 100, dtype=torch.int32, device="cuda")
    inv = torch.empty(1, 100, 1, dtype=torch.int32, device="cuda")
    offsets = torch.empty(1, 5, dtype=torch.int32, device="cuda")
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    mb.moga_permute(sh, gid, None, None, None, perm, inv, offsets, None, None, None, ws)
    code, detail = mb.moga_last_device_status(ws)
    assert code == 6 and (detail & 0x0fffffff) == 17
    assert mb.moga_last_device_status(ws) == (0, 0)            # reading clears it
    assert sorted(perm.cpu().numpy()[0].tolist()) == list(range(100))


def test_gather_strided_bnhd(mb):
    """Q/K/V stored as [B, N, H, D], expressed through the strides."""
    cfg = _cfg(B=2, N=333, H=3, D=128, M=4, dtype="f32")
    g = torch.Generator().manual_seed(2)
    Qs, Ks, Vs = (torch.randn(2, 333, 3, 128, generator=g).cuda() for _ in range(3))
    sh = mb.make_shape(cfg, strides=(333 * 3 * 128, 128, 3 * 128))
    gid = torch.from_numpy(_random_gid(2, 333, 4, 1, seed=3)).cuda()
    perm = torch.empty(2, 333, dtype=torch.int32, device="cuda")
    inv = torch.empty(2, 333, 1, dtype=torch.int32, device="cuda")
    offsets = torch.empty(2, 5, dtype=torch.int32, device="cuda")
    Qp, Kp, Vp = (torch.empty(2, 3, 333, 128, device="cuda") for _ in range(3))
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    mb.moga_permute(sh, gid, Qs, Ks, Vs, perm, inv, offsets, Qp, Kp, Vp, ws)
    torch.cuda.synchronize()
    idx = perm.long()
    for src, dst in ((Qs, Qp), (Ks, Kp), (Vs, Vp)):
        want = torch.gather(src.permute(0, 2, 1, 3), 2, idx[:, None, :, None].expand(2, 3, 333, 128))
        assert torch.equal(dst, want)
    # and the inverse writes through the same strides
    gate = torch.rand(2, 333, 1, device="cuda")
    O = torch.zeros(2, 333, 3, 128, device="cuda")
    mb.moga_unpermute(sh, Qp, inv, gate, O)
    torch.cuda.synchronize()
    want = (Qs.double() * gate.double()[..., None]).float()
    assert (O - want).abs().max().item() <= 1e-6


@pytest.mark.parametrize("dtype,k,D", [("f32", 1, 64), ("bf16", 2, 128), ("bf16", 1, 64), ("f32", 3, 128)])
def test_unpermute(mb, dtype, k, D):
    B, H, N, M = 2, 3, 1111, 8
    cfg = _cfg(B=B, H=H, N=N, D=D, M=M, k=k, dtype=dtype)
    sh = mb.make_shape(cfg)
    T = N * k
    dt = torch.float32 if dtype == "f32" else torch.bfloat16
    g = torch.Generator().manual_seed(4)
    Op = torch.randn(B, H, T, D, generator=g).to(dt).cuda()
    gate = torch.rand(B, N, k, generator=g).cuda()
    inv = torch.stack([torch.randperm(T, generator=g) for _ in range(B)]).int().reshape(B, N, k).cuda()
    O = torch.empty(B, H, N, D, dtype=dt, device="cuda")
    mb.moga_unpermute(sh, Op, inv, gate, O)
    torch.cuda.synchronize()
    op64, g64, iv = Op.double().cpu().numpy(), gate.double().cpu().numpy(), inv.cpu().numpy()
    want = np.zeros((B, H, N, D))
    for b in range(B):
        for j in range(k):
            want[b] += g64[b, :, j][None, :, None] * op64[b][:, iv[b, :, j]]
    tol = 1e-6 if dtype == "f32" else 2.0 ** -8 * np.abs(want).max()
    assert np.abs(O.double().cpu().numpy() - want).max() <= tol


ATTN_SIZES = [
    [512, 300, 129, 128, 127, 1, 0, 2, 65, 0, 1000],
    [1], [0, 0, 3], [257], [4096],
]


@pytest.mark.parametrize("dtype,D", [("f32", 64), ("f32", 128), ("bf16", 128), ("bf16", 64)])
@pytest.mark.parametrize("sizes", ATTN_SIZES, ids=lambda s: "g" + "_".join(map(str, s[:4])))
def test_group_attn(mb, dtype, D, sizes):
    H, B = 2, 2
    case = grouped_case(sizes, H, D, dtype, seed=len(sizes) + D, B=B)
    T, M = case["T"], len(sizes)
    cfg = _cfg(B=B, H=H, N=T, D=D, M=M, k=1, dtype=dtype)
    scale = 1.0 / math.sqrt(D)
    sh = mb.make_shape(cfg, scale=scale)
    Op = torch.full_like(case["Q"], float("nan"))
    lse = torch.empty(B, H, T, dtype=torch.float32, device="cuda")
    offsets = torch.from_numpy(case["offsets"]).cuda()
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    mb.moga_group_attn(sh, case["Q"], case["K"], case["V"], offsets, Op, lse, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    gate = np.ones((B, T, 1))
    want = oracle.attn_all(to_np32(case["Q"]), to_np32(case["K"]), to_np32(case["V"]), case["gid"], gate,
                           case["offsets"], case["perm"], scale)
    check_output(Op.float().cpu().numpy(), want, dtype, "Op")
    # log-sum-exp of the scaled scores, from library primitives in fp64
    q, k_ = case["Q"].double().cpu(), case["K"].double().cpu()
    for g in range(M):
        lo, hi = case["offsets"][0, g], case["offsets"][0, g + 1]
        if hi > lo:
            s = torch.einsum("bhnd,bhmd->bhnm", q[:, :, lo:hi], k_[:, :, lo:hi]) * scale
            ref = torch.logsumexp(s, -1)
            assert (lse[:, :, lo:hi].double().cpu() - ref).abs().max().item() <= (1e-4 if dtype == "f32" else 2e-2)


PAIR_SIZES = [
    [512, 300, 129, 128, 127, 1, 0, 2, 65, 0, 1000],
    [1], [0, 0, 3], [257], [513], [4096], [1500, 2600, 640],
]


@pytest.mark.parametrize("sizes", PAIR_SIZES, ids=lambda s: "g" + "_".join(map(str, s[:4])))
def test_group_attn_pair_kernel(mb, sizes):
    """The three tensor-core kernels for d_head = 128 (the CTA-pair kernel, the one-CTA kernel with one
    softmax thread per row, and the default with two softmax threads per row), each forced for
    every group size, against the oracle and against each other."""
    H, B, D = 2, 2, 128
    case = grouped_case(sizes, H, D, "bf16", seed=len(sizes) + 7, B=B)
    T, M = case["T"], len(sizes)
    cfg = _cfg(B=B, H=H, N=T, D=D, M=M, k=1, dtype="bf16")
    scale = 1.0 / math.sqrt(D)
    sh = mb.make_shape(cfg, scale=scale)
    offsets = torch.from_numpy(case["offsets"]).cuda()
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    want = oracle.attn_all(to_np32(case["Q"]), to_np32(case["K"]), to_np32(case["V"]), case["gid"],
                           np.ones((B, T, 1)), case["offsets"], case["perm"], scale)
    outs = {}
    try:
        for mode in (mb.MOGA_ATTN_PAIR, mb.MOGA_ATTN_SINGLE, mb.MOGA_ATTN_AUTO):
            mb.moga_set_attn_kernel(mode)
            Op = torch.full_like(case["Q"], float("nan"))
            lse = torch.empty(B, H, T, dtype=torch.float32, device="cuda")
            mb.moga_group_attn(sh, case["Q"], case["K"], case["V"], offsets, Op, lse, ws)
            assert mb.moga_last_device_status(ws) == (0, 0)
            check_output(Op.float().cpu().numpy(), want, "bf16", f"Op (kernel {mode})")
            outs[mode] = (Op, lse)
    finally:
        mb.moga_set_attn_kernel(mb.MOGA_ATTN_AUTO)
    # same arithmetic per row in both kernels: expected equal to the last bit; at the least very close
    b = outs[mb.MOGA_ATTN_SINGLE]
    for mode in (mb.MOGA_ATTN_PAIR, mb.MOGA_ATTN_AUTO):
        a = outs[mode]
        assert (a[0].float() - b[0].float()).abs().max().item() <= 2.0 ** -7 * b[0].float().abs().max().item() + 1e-6
        assert (a[1] - b[1]).abs().max().item() <= 1e-3
    a = outs[mb.MOGA_ATTN_PAIR]
    q, k_ = case["Q"].double().cpu(), case["K"].double().cpu()
    for g in range(M):
        lo, hi = case["offsets"][0, g], case["offsets"][0, g + 1]
        if hi > lo:
            ref = torch.logsumexp(torch.einsum("bhnd,bhmd->bhnm", q[:, :, lo:hi], k_[:, :, lo:hi]) * scale, -1)
            assert (a[1][:, :, lo:hi].double().cpu() - ref).abs().max().item() <= 2e-2


def test_group_attn_peaky_bf16(mb):
    """Large score spread (Q scaled x4): exercises the running-max rescale."""
    case = grouped_case([700, 333], 2, 128, "bf16", seed=9, B=1, qscale=4.0)
    cfg = _cfg(B=1, H=2, N=case["T"], D=128, M=2, k=1, dtype="bf16")
    scale = 1.0 / math.sqrt(128)
    sh = mb.make_shape(cfg, scale=scale)
    Op = torch.empty_like(case["Q"])
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    mb.moga_group_attn(sh, case["Q"], case["K"], case["V"], torch.from_numpy(case["offsets"]).cuda(), Op,
                       None, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    want = oracle.attn_all(to_np32(case["Q"]), to_np32(case["K"]), to_np32(case["V"]), case["gid"],
                           np.ones((1, case["T"], 1)), case["offsets"], case["perm"], scale)
    check_output(Op.float().cpu().numpy(), want, "bf16", "Op")
    rel = np.linalg.norm(Op.float().cpu().numpy() - want) / np.linalg.norm(want)
    assert rel < 2e-2


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("bf16", 64), ("f32", 64)])
def test_group_attn_scale_zero_is_the_group_mean(mb, dtype, D):
    """Closed form of Eq. 1: with scale = 0 every weight is 1 / n_g, so a row of the output is
    the mean of its group's V rows.  Ragged sizes, so the tail tile's masked columns are met."""
    sizes = [129, 300, 1, 0, 127, 513]
    case = grouped_case(sizes, 2, D, dtype, seed=31, B=1)
    cfg = _cfg(B=1, H=2, N=case["T"], D=D, M=len(sizes), k=1, dtype=dtype)
    sh = mb.make_shape(cfg, scale=0.0)
    Op = torch.full_like(case["Q"], float("nan"))
    lse = torch.empty(1, 2, case["T"], dtype=torch.float32, device="cuda")
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    mb.moga_group_attn(sh, case["Q"], case["K"], case["V"], torch.from_numpy(case["offsets"]).cuda(), Op, lse, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    V64 = case["V"].double().cpu().numpy()
    want = np.zeros_like(V64)
    off = case["offsets"][0]
    for g in range(len(sizes)):
        lo, hi = int(off[g]), int(off[g + 1])
        if hi > lo:
            want[:, :, lo:hi] = V64[:, :, lo:hi].mean(axis=2, keepdims=True)
            assert (lse[:, :, lo:hi].double().cpu() - math.log(hi - lo)).abs().max().item() <= 1e-5
    check_output(Op.float().cpu().numpy(), want, dtype, "Op at scale 0")
    # and the oracle says the same (its own closed-form pin lives in the CPU tests)
    ref = oracle.attn_all(to_np32(case["Q"]), to_np32(case["K"]), to_np32(case["V"]), case["gid"],
                          np.ones((1, case["T"], 1)), case["offsets"], case["perm"], 0.0)
    assert np.abs(ref - want).max() < 1e-12


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_group_attn_neighbour_group_does_not_leak(mb, dtype):
    """Group independence (Eq. 5: keys and values of the token's own group only): the second
    group's K rows are made huge and its V rows large, and the first group, whose tail tile
    shares a 128-row window with them, must come out bit-identical to the run where the second
    group holds ordinary numbers.  (Scores against the foreign keys overflow to inf / NaN in the
    masked columns; their weights must still be exact zeros.)  The fp32 kernel never loads a
    foreign row, so there the foreign V rows may even hold inf; the bf16 tensor-core kernel
    multiplies them by a zero weight, which requires them to be finite (documented in moga.h)."""
    sizes = [200, 150]
    case = grouped_case(sizes, 2, 128 if dtype == "bf16" else 64, dtype, seed=32, B=1)
    D = case["Q"].shape[-1]
    cfg = _cfg(B=1, H=2, N=case["T"], D=D, M=2, k=1, dtype=dtype)
    sh = mb.make_shape(cfg, scale=1.0 / math.sqrt(D))
    offsets = torch.from_numpy(case["offsets"]).cuda()
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    outs = []
    for poison in (False, True):
        K, V = case["K"].clone(), case["V"].clone()
        if poison:
            K[:, :, 200:] *= 1.0e30
            V[:, :, 200:] = float("inf") if dtype == "f32" else 3.0e38
        Op = torch.full_like(case["Q"], float("nan"))
        mb.moga_group_attn(sh, case["Q"], K, V, offsets, Op, None, ws)
        assert mb.moga_last_device_status(ws) == (0, 0)
        outs.append(Op[:, :, :200].clone())
    assert torch.isfinite(outs[1].float()).all()
    assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("kernel", ["single", "pair", "auto"])
@pytest.mark.parametrize("grow", [3.0, 24.0])
def test_group_attn_growing_scores_bf16(mb, grow, kernel):
    """All three kernels: the one-CTA kernel with one thread per row changes the reference inside the
    row; the default (two threads per row) and the CTA-pair kernel hand such items to that kernel's
    exact path afterwards.
    Keys late in each group are scaled up, so later K/V tiles hold scores far above the
    first tile's maximum: x3 stays on the kernel's fixed-reference path with large positive
    exponents, x24 overflows it and forces the mid-row change of reference.  Outputs are
    O(1) here (a few keys dominate each row), so the bound is relative."""
    sizes = [900, 515, 130]
    case = grouped_case(sizes, 2, 128, "bf16", seed=11, B=1)
    off = case["offsets"][0]
    for g in range(len(sizes)):
        lo, hi = int(off[g]), int(off[g + 1])
        case["K"][:, :, lo + (hi - lo) // 3:hi] *= grow
    cfg = _cfg(B=1, H=2, N=case["T"], D=128, M=len(sizes), k=1, dtype="bf16")
    scale = 1.0 / math.sqrt(128)
    sh = mb.make_shape(cfg, scale=scale)
    Op = torch.full_like(case["Q"], float("nan"))
    lse = torch.empty(1, 2, case["T"], dtype=torch.float32, device="cuda")
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    mb.moga_set_attn_kernel({"pair": mb.MOGA_ATTN_PAIR, "single": mb.MOGA_ATTN_SINGLE, "auto": mb.MOGA_ATTN_AUTO}[kernel])
    try:
        mb.moga_group_attn(sh, case["Q"], case["K"], case["V"], torch.from_numpy(case["offsets"]).cuda(), Op,
                           lse, ws)
        assert mb.moga_last_device_status(ws) == (0, 0)
    finally:
        mb.moga_set_attn_kernel(mb.MOGA_ATTN_AUTO)
    want = oracle.attn_all(to_np32(case["Q"]), to_np32(case["K"]), to_np32(case["V"]), case["gid"],
                           np.ones((1, case["T"], 1)), case["offsets"], case["perm"], scale)
    got = Op.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 1e-2
    assert np.abs(got - want).max() <= 2.0 ** -6 * np.abs(want).max()
    q, k_ = case["Q"].double().cpu(), case["K"].double().cpu()
    for g in range(len(sizes)):
        lo, hi = int(off[g]), int(off[g + 1])
        s = torch.einsum("bhnd,bhmd->bhnm", q[:, :, lo:hi], k_[:, :, lo:hi]) * scale
        ref = torch.logsumexp(s, -1)
        assert (lse[:, :, lo:hi].double().cpu() - ref).abs().max().item() <= 2e-2


@pytest.mark.parametrize("B,N,M,k,skew", [(1, 5000, 8, 1, False), (2, 9001, 16, 2, False), (1, 40000, 64, 2, True),
                                          (1, 1, 4, 1, False), (3, 4097, 1, 1, False)])
def test_balance_stats(mb, B, N, M, k, skew):
    """Eq. 6-8 from a routing result against the oracle, and reproducible bit for bit."""
    cfg = _cfg(B=B, N=N, M=M, k=k, dtype="bf16")
    gid_np = _random_gid(B, N, M, k, seed=N + 1, skew=skew) if k <= M else None
    rng = np.random.default_rng(N)
    gate_np = rng.random((B, N, k)).astype(np.float32)
    gid, gate = torch.from_numpy(gid_np).cuda(), torch.from_numpy(gate_np).cuda()
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    outs = []
    for _ in range(2):
        F = torch.empty(B, M, device="cuda")
        P = torch.empty(B, M, device="cuda")
        loss = torch.empty(B, device="cuda")
        mb.moga_balance_stats(sh, gid, gate, 0.1, F, P, loss, ws)
        torch.cuda.synchronize()
        outs.append((F, P, loss))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    oF, oP, oloss = oracle.balance_stats(gid_np, gate_np, M, 0.1)
    F, P, loss = (t.double().cpu().numpy() for t in outs[0])
    assert np.abs(F - oF).max() <= 1e-7                        # integer counts / N, rounded once to fp32
    assert np.abs(P - oP).max() <= 2e-6 * max(1.0, oP.max())
    assert np.abs(loss - oloss).max() <= 2e-6 * max(1.0, oloss.max())
