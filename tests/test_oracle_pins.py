"""Pins for the fp64 CPU oracle: each test checks it against something other than
itself -- a library routine (numpy matmul / argsort, torch SDPA), a pure-Python
brute force that never sorts, a closed form, or an invariant the paper fixes."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import GATE_SOFTMAX_ALL, GATE_SOFTMAX_TOPK


def _rand(shape, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)


def _case(B=1, H=2, N=40, C=16, D=8, M=4, seed=0, bias=False):
    X = _rand((B, N, C), seed)
    Wr = _rand((C, M), seed + 1, 1.0 / math.sqrt(C))
    b = _rand((M,), seed + 2) if bias else None
    Q = _rand((B, H, N, D), seed + 3)
    K = _rand((B, H, N, D), seed + 4)
    V = _rand((B, H, N, D), seed + 5)
    return X, Wr, b, Q, K, V


def _softmax64(a):
    a = a - a.max()
    e = np.exp(a)
    return e / e.sum()


# ---------------------------------------------------------------- route (Eq. 2-4)
@pytest.mark.parametrize("k,mode", [(1, GATE_SOFTMAX_ALL), (2, GATE_SOFTMAX_TOPK),
                                    (2, GATE_SOFTMAX_ALL), (1, GATE_SOFTMAX_TOPK)])
def test_route_against_library_matmul_and_argsort(k, mode):
    X, Wr, b, *_ = _case(B=2, N=300, C=48, M=8, seed=3, bias=True)
    gid, gate, logits = oracle.route(X, Wr, b, k, mode, want_logits=True)
    ref = X.astype(np.float64) @ Wr.astype(np.float64) + b.astype(np.float64)
    assert np.abs(logits - ref).max() < 1e-12
    order = np.argsort(-ref, axis=-1, kind="stable")[..., :k]
    assert np.array_equal(gid, order.astype(np.int32))
    for bi in range(X.shape[0]):
        for n in range(X.shape[1]):
            p_all = _softmax64(ref[bi, n])
            sel = order[bi, n]
            want = p_all[sel] if mode == GATE_SOFTMAX_ALL else _softmax64(ref[bi, n, sel])
            assert np.abs(gate[bi, n] - want).max() < 1e-14


def test_route_tie_goes_to_lower_index():
    X = _rand((1, 50, 8), 0)
    w = _rand((8, 1), 1)
    Wr = np.concatenate([w * 0.5, w, w, w * 0.25], axis=1)  # columns 1 and 2 tie exactly
    gid, gate, _ = oracle.route(X, Wr, None, 2, GATE_SOFTMAX_TOPK)
    lg = X[0].astype(np.float64) @ Wr.astype(np.float64)
    for n in range(50):
        if lg[n, 1] >= lg[n].max():  # the tied pair is on top
            assert list(gid[0, n]) == [1, 2]
            assert abs(gate[0, n, 0] - 0.5) < 1e-15 and abs(gate[0, n, 1] - 0.5) < 1e-15
        else:
            assert gid[0, n, 0] in (0, 3)


def test_gate_identities():
    X, Wr, b, *_ = _case(N=500, C=32, M=8, seed=7)
    gid, gate, logits = oracle.route(X, Wr, None, 1, GATE_SOFTMAX_ALL, want_logits=True)
    assert np.all(gate > 1.0 / 8 - 1e-15) and np.all(gate <= 1.0)      # top-1 of a softmax >= 1/M
    gid2, gate2, _ = oracle.route(X, Wr, None, 2, GATE_SOFTMAX_TOPK)
    assert np.abs(gate2.sum(-1) - 1.0).max() < 1e-15
    assert np.all(gate2[..., 0] >= gate2[..., 1])
    assert np.all(gid2[..., 0] != gid2[..., 1])
    assert np.array_equal(gid2[..., 0], gid[..., 0])
    # M = 1: the only gate is 1 in both modes
    _, g1, _ = oracle.route(X, Wr[:, :1], None, 1, GATE_SOFTMAX_ALL)
    assert np.all(g1 == 1.0)


# ---------------------------------------------------------------- sort (Alg. 1 line 2)
@pytest.mark.parametrize("k", [1, 2])
def test_sort_against_stable_argsort(k):
    rng = np.random.default_rng(5)
    B, N, M = 3, 777, 6
    if k == 1:
        gid = rng.integers(0, M, size=(B, N, 1)).astype(np.int32)
    else:
        a = rng.integers(0, M, size=(B, N))
        bb = (a + rng.integers(1, M, size=(B, N))) % M  # distinct second group
        gid = np.stack([a, bb], -1).astype(np.int32)
    if k == 1:
        gid[gid == 4] = 3  # leave group 4 empty
    offsets, perm, inv = oracle.sort(gid, M)
    for b in range(B):
        flat = gid[b].reshape(-1)
        order = np.argsort(flat, kind="stable")            # library stable sort of assignments
        assert np.array_equal(perm[b], (order // k).astype(np.int32))
        counts = np.bincount(flat, minlength=M)
        assert np.array_equal(offsets[b], np.concatenate([[0], np.cumsum(counts)]).astype(np.int32))
        # inv is the inverse: position of assignment (n, j)
        assert np.array_equal(order[inv[b].reshape(-1)], np.arange(N * k))
        assert np.array_equal(perm[b][inv[b]], np.repeat(np.arange(N)[:, None], k, 1))


# ---------------------------------------------------------------- attention (Eq. 1, 5)
@pytest.mark.parametrize("mode", [GATE_SOFTMAX_ALL, GATE_SOFTMAX_TOPK])
def test_m1_is_full_attention(mode):
    X, Wr, _, Q, K, V = _case(B=2, H=3, N=65, C=16, D=16, M=1, seed=11)
    scale = 1.0 / math.sqrt(16)
    out = oracle.forward(X, Wr, None, Q, K, V, 1, mode, scale)
    q, k_, v = (torch.from_numpy(t).double() for t in (Q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(q, k_, v, scale=scale).numpy()
    assert np.abs(out["O"] - ref).max() < 1e-13
    # and the textbook formula with numpy primitives
    s = np.einsum("bhnd,bhmd->bhnm", Q.astype(np.float64), K.astype(np.float64)) * scale
    p = np.exp(s - s.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    assert np.abs(out["O"] - p @ V.astype(np.float64)).max() < 1e-13
    assert np.all(out["gate"] == 1.0)
    assert np.array_equal(out["perm"][0], np.arange(65))


def _brute_force(X, Wr, bias, Q, K, V, k, mode, scale):
    """Definition of Eq. 2-5 with python loops: no sort, no offsets, no perm."""
    B, N, C = X.shape
    M = Wr.shape[1]
    H, D = Q.shape[1], Q.shape[3]
    O = np.zeros((B, H, N, D))
    for b in range(B):
        sel, gates = [], []
        for n in range(N):
            r = [sum(float(X[b, n, c]) * float(Wr[c, i]) for c in range(C)) +
                 (float(bias[i]) if bias is not None else 0.0) for i in range(M)]
            idx = sorted(range(M), key=lambda i: (-r[i], i))[:k]
            pool = range(M) if mode == GATE_SOFTMAX_ALL else idx
            mx = max(r)
            Z = sum(math.exp(r[i] - mx) for i in pool)
            sel.append(idx)
            gates.append([math.exp(r[i] - mx) / Z for i in idx])
        for h in range(H):
            for n in range(N):
                for j, g in enumerate(sel[n]):
                    mem = [m for m in range(N) if g in sel[m]]
                    a = np.array([float(np.dot(Q[b, h, n].astype(np.float64),
                                               K[b, h, m].astype(np.float64))) * scale for m in mem])
                    p = _softmax64(a)
                    for w, m in zip(p, mem):
                        O[b, h, n] += gates[n][j] * w * V[b, h, m].astype(np.float64)
    return O


@pytest.mark.parametrize("M,k,mode,bias", [(4, 1, GATE_SOFTMAX_ALL, False), (4, 2, GATE_SOFTMAX_TOPK, True),
                                           (3, 2, GATE_SOFTMAX_ALL, False), (2, 1, GATE_SOFTMAX_TOPK, True),
                                           (4, 4, GATE_SOFTMAX_TOPK, False)])
def test_forward_against_brute_force(M, k, mode, bias):
    X, Wr, b, Q, K, V = _case(B=2, H=2, N=37, C=8, D=8, M=M, seed=20 + M + k, bias=bias)
    out = oracle.forward(X, Wr, b, Q, K, V, k, mode, 0.3)
    ref = _brute_force(X, Wr, b, Q, K, V, k, mode, 0.3)
    assert np.abs(out["O"] - ref).max() < 1e-12


def test_attn_rows_matches_forward_rows():
    X, Wr, b, Q, K, V = _case(B=2, H=2, N=50, M=4, seed=31)
    out = oracle.forward(X, Wr, None, Q, K, V, 2, GATE_SOFTMAX_TOPK, 0.25)
    rows = np.array([[0, 0, 0], [1, 1, 49], [0, 1, 17], [1, 0, 3]], np.int32)
    got = oracle.attn_rows(Q, K, V, out["gid"], out["gate"], out["offsets"], out["perm"], 0.25, rows)
    for r, (bi, h, n) in enumerate(rows):
        assert np.array_equal(got[r], out["O"][bi, h, n])


def test_groups_are_independent():
    """Eq. 5: a token only sees the keys and values of its own group."""
    X, Wr, _, Q, K, V = _case(N=120, M=4, seed=40)
    base = oracle.forward(X, Wr, None, Q, K, V, 1, GATE_SOFTMAX_ALL, 0.35)
    g = base["gid"][0, :, 0]
    K2, V2 = K.copy(), V.copy()
    K2[:, :, g == 2] += 3.0
    V2[:, :, g == 2] *= -2.0
    pert = oracle.forward(X, Wr, None, Q, K2, V2, 1, GATE_SOFTMAX_ALL, 0.35)
    assert np.array_equal(base["O"][:, :, g != 2], pert["O"][:, :, g != 2])
    assert np.abs(base["O"][:, :, g == 2] - pert["O"][:, :, g == 2]).max() > 1e-3


def test_token_order_does_not_matter():
    """Eq. 1 is a set function of the group's (k, v) rows: shuffling tokens shuffles outputs."""
    X, Wr, _, Q, K, V = _case(N=90, M=3, seed=50)
    sh = np.random.default_rng(1).permutation(90)
    a = oracle.forward(X, Wr, None, Q, K, V, 2, GATE_SOFTMAX_TOPK, 0.35)
    b = oracle.forward(X[:, sh], Wr, None, Q[:, :, sh], K[:, :, sh], V[:, :, sh], 2,
                       GATE_SOFTMAX_TOPK, 0.35)
    assert np.array_equal(a["gid"][:, sh], b["gid"])
    assert np.abs(a["O"][:, :, sh] - b["O"]).max() < 1e-13


def test_closed_forms():
    X, Wr, _, Q, K, V = _case(N=100, M=4, D=8, seed=60)
    r = oracle.route(X, Wr, None, 1, GATE_SOFTMAX_ALL)
    g, gate = r[0][0, :, 0], r[1][0, :, 0]
    # (a) all V rows of a group equal v_g  ->  output = gate * v_g exactly (weights sum to 1)
    vg = _rand((4, 8), 61)
    Vc = np.broadcast_to(vg[g][None, None], V.shape).copy()
    out = oracle.forward(X, Wr, None, Q, K, Vc, 1, GATE_SOFTMAX_ALL, 0.5)["O"]
    want = gate[:, None] * vg[g].astype(np.float64)
    assert np.abs(out - want[None, None]).max() < 1e-14
    # (b) Q = 0  ->  uniform weights: output = gate * mean of the group's V rows
    out0 = oracle.forward(X, Wr, None, np.zeros_like(Q), K, V, 1, GATE_SOFTMAX_ALL, 0.5)["O"]
    for h in range(Q.shape[1]):
        for grp in range(4):
            mean = V[0, h, g == grp].astype(np.float64).mean(0)
            got = out0[0, h, g == grp] / gate[g == grp][:, None]
            assert np.abs(got - mean).max() < 1e-13
    # (c) scale = 0 gives the same uniform weights whatever Q is
    outs = oracle.forward(X, Wr, None, Q, K, V, 1, GATE_SOFTMAX_ALL, 0.0)["O"]
    assert np.abs(outs - out0).max() < 1e-13


def test_empty_and_single_token_groups():
    X, Wr, _, Q, K, V = _case(N=64, M=4, seed=70)
    bias = np.array([0.0, -1e4, 0.0, 0.0], np.float32)      # group 1 never chosen
    out = oracle.forward(X, Wr, bias, Q, K, V, 1, GATE_SOFTMAX_ALL, 0.5)
    assert out["offsets"][0, 1] == out["offsets"][0, 2]
    assert np.all(np.isfinite(out["O"]))
    # force token 5 alone into group 1: its output is gate * its own V row
    Xs = X.copy()
    Wb = Wr.copy()
    Xs[0, 5] = 0.0
    Xs[0, 5, 0] = 100.0
    Wb[0] = [0.0, 1000.0, 0.0, 0.0]
    Xs[0, :5, 0] = 0.0
    Xs[0, 6:, 0] = 0.0
    out = oracle.forward(Xs, Wb, bias, Q, K, V, 1, GATE_SOFTMAX_ALL, 0.5)
    assert out["gid"][0, 5, 0] == 1 and (out["gid"][0, :, 0] == 1).sum() == 1
    want = out["gate"][0, 5, 0] * V[0, :, 5].astype(np.float64)
    assert np.abs(out["O"][0, :, 5] - want).max() < 1e-15


def test_balanced_flops_are_one_over_m():
    """Sec. 3.2: cost drops to 1/M of full attention under uniform assignment."""
    from paper_2510_18692_b200.inputs import useful_flops
    N, M, H, D = 4096, 8, 2, 64
    assert useful_flops([N // M] * M, H, D) == pytest.approx(useful_flops([N], H, D) / M)


# ----------------------------------------------------------------------------- Eq. 6-8
def test_balance_loss_closed_forms_and_brute_force():
    """Eq. 6-8.  Uniform top-1 assignment with a constant probability p gives alpha * p
    (F_i = 1/M, P_i = p/M); all tokens in one group gives alpha * M * p; among assignments
    with equal probabilities the uniform one attains the minimum (the paper's remark after
    Eq. 8); a pure-Python loop over tokens reproduces F, P and the loss on random input."""
    M, N, alpha, p = 5, 1000, 0.1, 0.37
    gid = (np.arange(N) % M).astype(np.int32).reshape(1, N, 1)
    gate = np.full((1, N, 1), p)
    F, P, loss = oracle.balance_stats(gid, gate, M, alpha)
    assert np.allclose(F, 1.0 / M) and np.allclose(P, p / M) and np.isclose(loss[0], alpha * p)
    F, P, loss = oracle.balance_stats(np.full((1, N, 1), 3, np.int32), gate, M, alpha)
    assert np.isclose(loss[0], alpha * M * p) and F[0, 3] == 1.0 and F[0].sum() == 1.0
    rng = np.random.default_rng(0)
    for _ in range(20):                      # any other split of the tokens costs more
        gid_r = rng.integers(0, M, (1, N, 1)).astype(np.int32)
        assert oracle.balance_stats(gid_r, gate, M, alpha)[2][0] >= alpha * p - 1e-15
    # brute force, k = 2, two batch items
    B, N, k = 2, 57, 2
    gid = np.stack([np.stack([rng.choice(M, k, replace=False) for _ in range(N)]) for _ in range(B)]).astype(np.int32)
    gate = rng.random((B, N, k))
    F, P, loss = oracle.balance_stats(gid, gate, M, 0.25)
    for b in range(B):
        f, q = [0.0] * M, [0.0] * M
        for n in range(N):
            for j in range(k):
                f[gid[b, n, j]] += 1.0 / N
                q[gid[b, n, j]] += gate[b, n, j] / N
        assert np.allclose(F[b], f, rtol=0, atol=1e-12) and np.allclose(P[b], q, rtol=0, atol=1e-12)
        assert abs(loss[b] - 0.25 * M * sum(x * y for x, y in zip(f, q))) <= 1e-12
        assert abs(F[b].sum() - k) <= 1e-12


# ----------------------------------------------------------------------------- Sec. 3.2 static groups
def _token_coords(n, Hh, Ww):
    return n // (Hh * Ww), (n // Ww) % Hh, n % Ww


def test_stga_groups_against_the_membership_rule():
    """The group lists against the rule of Sec. 3.2 stated per token pair: query n sees key m
    iff both lie in the same window and either in the same run of the same shot, or m is in
    the frame just across the shot boundary that n's run touches."""
    F, Hh, Ww, wh, ww, tg = 9, 4, 6, 2, 3, 2
    shots = [0, 3, 4]                                   # shots of 3, 1 and 5 frames
    qg, kg = oracle.stga_groups(F, Hh, Ww, wh, ww, shots, tg)
    N = F * Hh * Ww
    seen = np.zeros(N, int)
    keyset = {}
    for qi, ki in zip(qg, kg):
        seen[qi] += 1
        assert len(set(ki.tolist())) == len(ki)
        for n in qi:
            keyset[int(n)] = set(ki.tolist())
    assert np.all(seen == 1)                            # every token queries in exactly one group
    bounds = shots + [F]
    shot_of = lambda f: max(s for s in range(len(shots)) if bounds[s] <= f)
    for n in range(N):
        f, y, x = _token_coords(n, Hh, Ww)
        s = shot_of(f)
        run = (f - bounds[s]) // tg
        last_run = (bounds[s + 1] - 1 - bounds[s]) // tg
        want = set()
        for m in range(N):
            g, v, u = _token_coords(m, Hh, Ww)
            if (v * wh // Hh, u * ww // Ww) != (y * wh // Hh, x * ww // Ww):
                continue
            same = shot_of(g) == s and (g - bounds[s]) // tg == run
            prev_edge = run == 0 and s > 0 and g == bounds[s] - 1
            next_edge = run == last_run and s < len(shots) - 1 and g == bounds[s + 1]
            if same or prev_edge or next_edge:
                want.add(m)
        assert keyset[n] == want, n
    # without augmentation keys = queries; a one-frame shot between two others gets both neighbours
    q2, k2 = oracle.stga_groups(F, Hh, Ww, wh, ww, shots, tg, augment=False)
    assert all(np.array_equal(a, b) for a, b in zip(q2, k2))
    per_win = (Hh // wh) * (Ww // ww)
    mid = [(a, b) for a, b in zip(qg, kg) if _token_coords(int(a[0]), Hh, Ww)[0] == 3]
    assert all(len(b) - len(a) == 2 * per_win for a, b in mid)


def test_static_group_attention_special_cases():
    """One shot, one window, one run: the static group is the whole sequence and the result is
    plain full attention (library routine).  Per-frame groups: each frame equals full
    attention on that frame alone.  Keys-only augmentation: changing K/V of an augmenting
    frame changes the neighbour shot's boundary group and nothing else."""
    rng = np.random.default_rng(3)
    F, Hh, Ww, D = 4, 3, 4, 8
    N = F * Hh * Ww
    Q, K, V = (rng.standard_normal((1, 2, N, D)).astype(np.float32) for _ in range(3))
    scale = 1 / np.sqrt(D)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q).double(), torch.from_numpy(K).double(), torch.from_numpy(V).double(), scale=scale).numpy()
    qg, kg = oracle.stga_groups(F, Hh, Ww, 1, 1, [0], F)
    assert len(qg) == 1
    assert np.abs(oracle.static_group_attn(Q, K, V, qg, kg, scale) - ref).max() < 1e-12
    fq, fk = oracle.frame_groups(F, Hh, Ww)
    Of = oracle.static_group_attn(Q, K, V, fq, fk, scale)
    for f in range(F):
        sl = slice(f * Hh * Ww, (f + 1) * Hh * Ww)
        r = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q[:, :, sl]).double(), torch.from_numpy(K[:, :, sl]).double(),
            torch.from_numpy(V[:, :, sl]).double(), scale=scale).numpy()
        assert np.abs(Of[:, :, sl] - r).max() < 1e-12
    # two shots of two frames, one run each: frame 1 augments shot 1, frame 2 augments shot 0
    qg, kg = oracle.stga_groups(F, Hh, Ww, 1, 2, [0, 2], 2)
    O1 = oracle.static_group_attn(Q, K, V, qg, kg, scale)
    K2, V2 = K.copy(), V.copy()
    f0 = slice(0, Hh * Ww)                              # frame 0 augments nobody
    K2[:, :, f0] += 1.0
    V2[:, :, f0] -= 2.0
    O2 = oracle.static_group_attn(Q, K2, V2, qg, kg, scale)
    shot1 = slice(2 * Hh * Ww, N)
    assert np.array_equal(O1[:, :, shot1], O2[:, :, shot1])          # shot 1 never sees frame 0
    assert np.abs(O1[:, :, f0] - O2[:, :, f0]).max() > 1e-3
    K3 = K.copy()
    K3[:, :, Hh * Ww:2 * Hh * Ww] *= 1.5                # frame 1: last frame of shot 0, seen by shot 1
    O3 = oracle.static_group_attn(Q, K3, V, qg, kg, scale)
    assert np.abs(O1[:, :, shot1] - O3[:, :, shot1]).max() > 1e-4
    assert np.abs(oracle.mean3(O1, O2, O3) - (O1 + O2 + O3) / 3).max() == 0


# ----------------------------------------------------------------------------- printed sparsity (Table 4)
def test_group_sizes_reproduce_the_printed_sparsity_steps():
    """Under uniform assignment the routed branch computes 1/M of the query-key pairs
    (Sec. 3.2, complexity paragraph).  The paper's sparsity column also contains the static
    branches, a constant density, so the DIFFERENCE between two rows is free of it:
    sparsity(M2) - sparsity(M1) = 1/M1 - 1/M2.  The pair count comes from the oracle's sort of
    a balanced assignment (sum of squared group sizes), the numbers from the printed table."""
    path = os.path.join(os.path.dirname(__file__), "golden", "table4_sparsity.txt")
    rows = [tuple(map(float, l.split())) for l in open(path) if l.strip() and not l.startswith("#")]
    N = 2 * 4 * 5 * 8 * 3
    density = {}
    for M, _ in rows:
        M = int(M)
        gid = (np.arange(N) % M).astype(np.int32).reshape(1, N, 1)
        offsets, _, _ = oracle.sort(gid, M)
        density[M] = float((np.diff(offsets[0]).astype(np.float64) ** 2).sum()) / N ** 2
        assert abs(density[M] - 1.0 / M) < 1e-15
    for (M1, s1), (M2, s2) in zip(rows, rows[1:]):
        assert abs((s2 - s1) / 100.0 - (density[int(M1)] - density[int(M2)])) < 1e-12


def test_static_group_attention_agrees_with_the_routed_oracle():
    """Two independently written oracle paths meet: the numpy group attention of Sec. 3.2 fed with
    the routed groups of a random assignment (queries = keys = the group's tokens) must reproduce
    the C oracle's per-group attention with unit gates."""
    rng = np.random.default_rng(8)
    B, H, N, D, M = 1, 2, 150, 16, 5
    Q, K, V = (rng.standard_normal((B, H, N, D)).astype(np.float32) for _ in range(3))
    gid = rng.integers(0, M, (B, N, 1)).astype(np.int32)
    offsets, perm, _ = oracle.sort(gid, M)
    groups = [perm[0, offsets[0, g]:offsets[0, g + 1]].astype(np.int64) for g in range(M)]
    groups = [g for g in groups if len(g)]
    a = oracle.static_group_attn(Q, K, V, groups, groups, 0.3)
    b = oracle.attn_all(Q, K, V, gid, np.ones((B, N, 1)), offsets, perm, 0.3)
    assert np.abs(a - b).max() < 1e-12


# ----------------------------------------------------------------------------- backward
def _torch_forward_masked(Q, K, V, gid, gate, scale):
    """The forward of Eq. 1 + Eq. 5 written a different way (dense N x N scores with a same-group
    mask per slot, torch fp64 ops), so that autograd gives gradients independent of the oracle."""
    B, H, N, D = Q.shape
    k = gid.shape[2]
    O = torch.zeros_like(Q)
    s = torch.einsum("bhnd,bhmd->bhnm", Q, K) * scale
    for j in range(k):
        # query n (slot j) may attend key m iff m is assigned, in any slot, to the group gid[n, j]
        same = (gid[:, :, j][:, :, None, None] == gid[:, None, :, :]).any(-1)        # [B, N, N]
        sj = s.masked_fill(~same[:, None], float("-inf"))
        O = O + gate[:, None, :, j, None] * torch.einsum("bhnm,bhmd->bhnd", torch.softmax(sj, -1), V)
    return O


@pytest.mark.parametrize("k", [1, 2])
def test_backward_oracle_against_autograd_and_finite_differences(k):
    rng = np.random.default_rng(17 + k)
    B, H, N, D, M = 2, 2, 37, 8, 4
    Q, K, V, dO = (rng.standard_normal((B, H, N, D)) for _ in range(4))
    gid = np.stack([rng.permutation(M)[:k] for _ in range(B * N)]).reshape(B, N, k).astype(np.int32)
    gate = rng.random((B, N, k)) + 0.1
    scale = 0.4
    dQ, dK, dV, dgate = oracle.backward(Q, K, V, gid, gate, dO, scale, M)
    tq, tk, tv, tg = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (Q, K, V, gate))
    out = _torch_forward_masked(tq, tk, tv, torch.tensor(gid.astype(np.int64)), tg, scale)
    # the masked torch forward is itself the oracle's forward
    off, perm, _ = oracle.sort(gid, M)
    want = oracle.attn_all(Q.astype(np.float32), K.astype(np.float32), V.astype(np.float32), gid, gate, off, perm, scale)
    ref32 = _torch_forward_masked(*(torch.tensor(a.astype(np.float32).astype(np.float64)) for a in (Q, K, V)),
                                  torch.tensor(gid.astype(np.int64)), torch.tensor(gate), scale)
    assert np.abs(ref32.numpy() - want).max() < 1e-12
    gq, gk, gv, gg = torch.autograd.grad(out, (tq, tk, tv, tg), torch.tensor(dO))
    for mine, ref in ((dQ, gq), (dK, gk), (dV, gv), (dgate, gg)):
        assert np.abs(mine - ref.numpy()).max() < 1e-11
    # central differences of L = sum(dO * O) on a few coordinates
    def loss(q, kk, v, g):
        return float((dO * _torch_forward_masked(*(torch.tensor(a) for a in (q, kk, v)),
                                                 torch.tensor(gid.astype(np.int64)), torch.tensor(g), scale).numpy()).sum())
    eps = 1e-6
    for arr, grad, name in ((Q, dQ, "q"), (K, dK, "k"), (V, dV, "v")):
        idx = (1, 0, 5, 3)
        hi, lo = arr.copy(), arr.copy()
        hi[idx] += eps
        lo[idx] -= eps
        args = {"q": (hi, K, V), "k": (Q, hi, V), "v": (Q, K, hi)}[name], {"q": (lo, K, V), "k": (Q, lo, V), "v": (Q, K, lo)}[name]
        fd = (loss(*args[0], gate) - loss(*args[1], gate)) / (2 * eps)
        assert abs(fd - grad[idx]) < 1e-6 * max(1.0, abs(fd))


def test_backward_oracle_special_cases():
    """One-token groups: o = v, so dV = gate * dO, dQ = dK = 0, dgate = <dO, v>.  Equal V rows in a
    group: the output does not depend on the scores, so dQ = dK = 0 there."""
    rng = np.random.default_rng(3)
    B, H, N, D, M = 1, 1, 6, 4, 6
    Q, K, V, dO = (rng.standard_normal((B, H, N, D)) for _ in range(4))
    gid = np.arange(N, dtype=np.int32).reshape(1, N, 1)          # every token alone in its group
    gate = rng.random((1, N, 1)) + 0.5
    dQ, dK, dV, dgate = oracle.backward(Q, K, V, gid, gate, dO, 0.7, M)
    assert np.abs(dQ).max() == 0 and np.abs(dK).max() == 0
    assert np.abs(dV - gate[:, None, :, 0, None] * dO).max() < 1e-15
    assert np.abs(dgate[..., 0] - (dO * V).sum(-1)[:, 0]).max() < 1e-15
    gid2 = np.zeros((1, N, 1), np.int32)
    V2 = np.broadcast_to(V[:, :, :1], V.shape).copy()
    dQ2, dK2, dV2, _ = oracle.backward(Q, K, V2, gid2, gate, dO, 0.7, 1)
    assert np.abs(dQ2).max() < 1e-15 and np.abs(dK2).max() < 1e-15


@pytest.mark.parametrize("gate_mode,k", [(GATE_SOFTMAX_ALL, 1), (GATE_SOFTMAX_ALL, 2), (GATE_SOFTMAX_TOPK, 2), (GATE_SOFTMAX_TOPK, 3)])
def test_route_backward_oracle_against_autograd(gate_mode, k):
    """The router's gradient against torch.autograd on the gate written with torch ops (softmax and
    gather), with the oracle's own routing decision as the fixed index."""
    rng = np.random.default_rng(5 + k)
    B, N, C, M = 2, 23, 12, 6
    X = rng.standard_normal((B, N, C)).astype(np.float32)
    Wr = (rng.standard_normal((C, M)) / np.sqrt(C)).astype(np.float32)
    bias = rng.standard_normal(M).astype(np.float32)
    gid, gate, _ = oracle.route(X, Wr, bias, k, gate_mode)
    dgate = rng.standard_normal((B, N, k))
    dr, dX, dWr, dbias = oracle.route_backward(X, Wr, bias, gid, dgate, gate_mode)
    tx, tw, tb = (torch.tensor(a.astype(np.float64), requires_grad=True) for a in (X, Wr, bias))
    r = tx @ tw + tb
    idx = torch.tensor(gid.astype(np.int64))
    if gate_mode == GATE_SOFTMAX_ALL:
        g = torch.softmax(r, -1).gather(-1, idx)
    else:
        g = torch.softmax(r.gather(-1, idx), -1)
    assert np.abs(g.detach().numpy() - gate).max() < 1e-12          # the forward gate is the oracle's
    gx, gw, gb = torch.autograd.grad(g, (tx, tw, tb), torch.tensor(dgate))
    assert np.abs(dX - gx.numpy()).max() < 1e-12
    assert np.abs(dWr - gw.numpy()).max() < 1e-12
    assert np.abs(dbias - gb.numpy()).max() < 1e-12
    assert np.abs(dr.sum(-1)).max() < 1e-12                          # softmax gradients sum to zero over the logits
