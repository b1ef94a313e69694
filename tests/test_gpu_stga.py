"""GPU parity of the static-group branch of the visual attention block (Sec. 3.2): group
attention with separate query and key sets, the row gather by a list, and the mean of the
three branches, each against the fp64 oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from parity import check_output, to_np32
from paper_2510_18692_b200.inputs import GATE_SOFTMAX_ALL, MogaConfig, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mb():
    from paper_2510_18692_b200 import build
    build.build()
    from paper_2510_18692_b200 import binding
    return binding


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_static(mb, cfg, Q, K, V, q_idx, kv_idx, q_offsets, kv_offsets, want_lse=False):
    """gather -> static group attention; returns Os [B,H,Tq,D] in query order (and lse)."""
    sh = mb.make_shape(cfg)
    G, Tq, Tkv = len(q_offsets) - 1, len(q_idx), len(kv_idx)
    dt = Q.dtype
    Qs = torch.empty(cfg.B, cfg.H, Tq, cfg.D, dtype=dt, device="cuda")
    Ks = torch.empty(cfg.B, cfg.H, Tkv, cfg.D, dtype=dt, device="cuda")
    Vs = torch.empty_like(Ks)
    mb.moga_gather_rows(sh, _dev(q_idx.astype(np.int32)), Q, Qs)
    kv_d = _dev(kv_idx.astype(np.int32))
    mb.moga_gather_rows(sh, kv_d, K, Ks)
    mb.moga_gather_rows(sh, kv_d, V, Vs)
    torch.cuda.synchronize()
    assert torch.equal(Ks, K[:, :, torch.from_numpy(kv_idx.astype(np.int64)).cuda()])
    Os = torch.full_like(Qs, float("nan"))
    lse = torch.empty(cfg.B, cfg.H, Tq, dtype=torch.float32, device="cuda") if want_lse else None
    ws = mb.alloc_workspace(mb.moga_static_scratch_bytes(sh, G))
    mb.moga_static_group_attn(sh, G, Tq, Tkv, Qs, Ks, Vs, _dev(q_offsets.astype(np.int32)),
                              _dev(kv_offsets.astype(np.int32)), Os, lse, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    return Os, lse


GRIDS = [
    # F, Hh, Ww, wh, ww, shots, tg
    (9, 4, 6, 2, 3, [0, 3, 4], 2),
    (6, 30, 52, 2, 2, [0, 2], 3),            # 480p grid: groups of 390..1170 queries, up to 1,560 keys
    (5, 9, 11, 1, 1, [0, 1, 4], 8),          # one window; a one-frame shot with both neighbours
]


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("bf16", 64), ("f32", 64)])
@pytest.mark.parametrize("grid", GRIDS, ids=lambda g: f"F{g[0]}_{g[1]}x{g[2]}_w{g[3]}x{g[4]}")
def test_spatial_temporal_branch(mb, grid, dtype, D):
    F, Hh, Ww, wh, ww, shots, tg = grid
    N = F * Hh * Ww
    cfg = MogaConfig("st", 2, 2, N, 64, D, 1, 1, dtype, GATE_SOFTMAX_ALL, 21)
    inp = make_inputs(cfg, device="cuda")
    lists = mb.moga_stga_build(F, Hh, Ww, wh, ww, shots, tg, True)
    Os, lse = run_static(mb, cfg, inp["Q"], inp["K"], inp["V"], lists["q_idx"], lists["kv_idx"],
                         lists["q_offsets"], lists["kv_offsets"], want_lse=True)
    qg, kg = oracle.stga_groups(F, Hh, Ww, wh, ww, shots, tg)
    want = oracle.static_group_attn(to_np32(inp["Q"]), to_np32(inp["K"]), to_np32(inp["V"]), qg, kg, cfg.scale)
    check_output(Os.float().cpu().numpy(), want[:, :, lists["q_idx"]], dtype, "Os")
    # log-sum-exp of one boundary group, from library primitives
    g = 1 if len(qg) > 1 else 0
    q = inp["Q"].double().cpu()[:, :, qg[g]]
    k = inp["K"].double().cpu()[:, :, kg[g]]
    ref = torch.logsumexp(torch.einsum("bhnd,bhmd->bhnm", q, k) * cfg.scale, -1)
    lo, hi = lists["q_offsets"][g], lists["q_offsets"][g + 1]
    assert (lse[:, :, lo:hi].double().cpu() - ref).abs().max().item() <= (1e-4 if dtype == "f32" else 2e-2)


def test_degenerate_static_groups(mb):
    """Hand-made lists: a group with queries but no keys and rows outside every group are left
    untouched; an empty group does nothing; a one-key group returns that key's V row."""
    cfg = MogaConfig("deg", 1, 2, 700, 64, 128, 1, 1, "bf16", GATE_SOFTMAX_ALL, 22)
    inp = make_inputs(cfg, device="cuda")
    sh = mb.make_shape(cfg)
    # queries: [0,300) | [300,300) | [300,310) no keys | [310,311) one key | rows 311.. unowned
    q_off = np.array([0, 300, 300, 310, 311], np.int32)
    kv_off = np.array([0, 450, 450, 450, 451], np.int32)
    Tq, Tkv = 700, 451
    Os = torch.full((1, 2, Tq, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    ws = mb.alloc_workspace(mb.moga_static_scratch_bytes(sh, 4))
    Ks, Vs = inp["K"][:, :, :Tkv].contiguous(), inp["V"][:, :, :Tkv].contiguous()
    mb.moga_static_group_attn(sh, 4, Tq, Tkv, inp["Q"], Ks, Vs, _dev(q_off), _dev(kv_off), Os, None, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    assert torch.all(Os[:, :, 300:310] == 7.0) and torch.all(Os[:, :, 311:] == 7.0)
    assert torch.equal(Os[:, :, 310], Vs[:, :, 450])
    want = oracle.static_group_attn(to_np32(inp["Q"]), to_np32(inp["K"]), to_np32(inp["V"]),
                                    [np.arange(300)], [np.arange(450)], cfg.scale)
    check_output(Os[:, :, :300].float().cpu().numpy(), want[:, :, :300], "bf16")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_visual_attention_block(mb, dtype):
    """Routed branch + spatial-temporal branch + per-frame branch, then their mean (Sec. 3.2)."""
    F, Hh, Ww, wh, ww, shots, tg = 8, 6, 10, 2, 2, [0, 3], 2
    N = F * Hh * Ww
    cfg = MogaConfig("va", 1, 2, N, 128, 64 if dtype == "f32" else 128, 4, 1, dtype, GATE_SOFTMAX_ALL, 23)
    inp = make_inputs(cfg, device="cuda")
    sh = mb.make_shape(cfg)
    # routed branch
    ws = mb.alloc_workspace(mb.moga_workspace_bytes(sh))
    A = torch.empty_like(inp["Q"])
    gid = torch.empty(1, N, 1, dtype=torch.int32, device="cuda")
    gate = torch.empty(1, N, 1, dtype=torch.float32, device="cuda")
    mb.moga_forward(sh, inp["X"], inp["Wr"], None, inp["Q"], inp["K"], inp["V"], A, ws, gid, gate)
    assert mb.moga_last_device_status(ws) == (0, 0)
    # static branches
    lists = mb.moga_stga_build(F, Hh, Ww, wh, ww, shots, tg, True)
    Bs, _ = run_static(mb, cfg, inp["Q"], inp["K"], inp["V"], lists["q_idx"], lists["kv_idx"],
                       lists["q_offsets"], lists["kv_offsets"])
    fr_off = (np.arange(F + 1) * Hh * Ww).astype(np.int32)
    C = torch.empty_like(inp["Q"])
    ws2 = mb.alloc_workspace(mb.moga_static_scratch_bytes(sh, F))
    mb.moga_static_group_attn(sh, F, N, N, inp["Q"], inp["K"], inp["V"], _dev(fr_off), _dev(fr_off), C, None, ws2)
    assert mb.moga_last_device_status(ws2) == (0, 0)
    O = torch.empty_like(inp["Q"])
    mb.moga_mean3(sh, A, Bs, _dev(lists["q_inv"]), C, O)
    torch.cuda.synchronize()
    # oracle: each branch in fp64 from the inputs (routed branch with the GPU's routing), then the mean
    host = {k: to_np32(v) for k, v in inp.items()}
    gid_np = gid.cpu().numpy()
    off, perm, _ = oracle.sort(gid_np, cfg.M)
    oA = oracle.attn_all(host["Q"], host["K"], host["V"], gid_np, gate.double().cpu().numpy(), off, perm, cfg.scale)
    qg, kg = oracle.stga_groups(F, Hh, Ww, wh, ww, shots, tg)
    oB = oracle.static_group_attn(host["Q"], host["K"], host["V"], qg, kg, cfg.scale)
    fq, fk = oracle.frame_groups(F, Hh, Ww)
    oC = oracle.static_group_attn(host["Q"], host["K"], host["V"], fq, fk, cfg.scale)
    check_output(C.float().cpu().numpy(), oC, dtype, "frame branch")
    check_output(O.float().cpu().numpy(), oracle.mean3(oA, oB, oC), dtype, "mean of three")
    # the same block through the single entry point: the same kernels, so the same bits
    st_lists, keep = mb.make_static_lists(lists, F, Hh * Ww)
    ws_v = mb.alloc_workspace(mb.moga_visual_workspace_bytes(sh, st_lists))
    O1 = torch.full_like(O, float("nan"))
    mb.moga_visual_forward(sh, inp["X"], inp["Wr"], None, inp["Q"], inp["K"], inp["V"], O1, st_lists, ws_v)
    assert mb.moga_last_device_status(ws_v) == (0, 0)
    assert torch.equal(O1, O)
    # the combine step alone, against the mean of the GPU's own branch outputs (fp32 sum, one rounding)
    Bt = Bs[:, :, torch.from_numpy(lists["q_inv"].astype(np.int64)).cuda()]
    ref = (A.double() + Bt.double() + C.double()) / 3
    tol = 2.0 ** -8 * ref.abs().max().item() if dtype == "bf16" else 1e-6
    assert (O.double() - ref).abs().max().item() <= tol


@pytest.mark.parametrize("name", ["clip_bf16", "minute_bf16"])
def test_static_branches_full_size_sampled(mb, name):
    """The static branches in the configuration bench.py --stage visual times (4 x 4 windows, runs of
    8 latent frames, shots of 45 latent frames) at paper sizes, checked on sampled rows: first and
    last query of a sample of groups (shot-boundary groups included) and random tokens."""
    from paper_2510_18692_b200.inputs import CONFIGS
    cfg = CONFIGS[name]
    free, _ = torch.cuda.mem_get_info()
    es = 2
    if free < 9 * cfg.B * cfg.H * cfg.N * cfg.D * es + cfg.B * cfg.N * cfg.C * es + (2 << 30):
        pytest.skip("not enough device memory for this size")
    Hh, Ww, wh, ww, tg, shot_len = 30, 52, 4, 4, 8, 45
    F = cfg.N // (Hh * Ww)
    shots = list(range(0, F, shot_len))
    inp = make_inputs(cfg, device="cuda")
    del inp["X"]
    lists = mb.moga_stga_build(F, Hh, Ww, wh, ww, shots, tg, True)
    Bs, _ = run_static(mb, cfg, inp["Q"], inp["K"], inp["V"], lists["q_idx"], lists["kv_idx"],
                       lists["q_offsets"], lists["kv_offsets"])
    sh = mb.make_shape(cfg)
    fr_off = (np.arange(F + 1) * Hh * Ww).astype(np.int32)
    C = torch.empty_like(inp["Q"])
    ws = mb.alloc_workspace(mb.moga_static_scratch_bytes(sh, F))
    mb.moga_static_group_attn(sh, F, cfg.N, cfg.N, inp["Q"], inp["K"], inp["V"], _dev(fr_off), _dev(fr_off), C, None, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    qg, kg = oracle.stga_groups(F, Hh, Ww, wh, ww, shots, tg)
    assert len(qg) == lists["G"]
    rng = np.random.default_rng(5)
    heads = [0, cfg.H - 1]
    pick = sorted(set(rng.choice(len(qg), size=min(24, len(qg)), replace=False).tolist()) | {0, len(qg) - 1} |
                  {g for g in range(len(qg)) if len(kg[g]) > len(qg[g])} & set(range(0, len(qg), 7)))
    toks = [int(qg[g][0]) for g in pick] + [int(qg[g][-1]) for g in pick] + rng.integers(0, cfg.N, 64).tolist()
    rows = [(0, h, n) for n in toks for h in heads]
    Qh, Kh, Vh = (to_np32(inp[n][:, heads]) for n in ("Q", "K", "V"))
    rows_h = [(b, heads.index(h), n) for b, h, n in rows]
    want_st = oracle.static_group_attn_rows(Qh, Kh, Vh, qg, kg, cfg.scale, rows_h)
    fq, fk = oracle.frame_groups(F, Hh, Ww)
    want_fr = oracle.static_group_attn_rows(Qh, Kh, Vh, fq, fk, cfg.scale, rows_h)
    q_inv = torch.from_numpy(lists["q_inv"].astype(np.int64)).cuda()
    bi = torch.tensor([r[0] for r in rows]).cuda()
    hi = torch.tensor([r[1] for r in rows]).cuda()
    ni = torch.tensor([r[2] for r in rows]).cuda()
    check_output(Bs[bi, hi, q_inv[ni]].float().cpu().numpy(), want_st, "bf16", "spatial-temporal rows")
    check_output(C[bi, hi, ni].float().cpu().numpy(), want_fr, "bf16", "per-frame rows")
