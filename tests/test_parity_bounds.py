"""The comparison helper itself must be able to fail (CPU only): at the magnitude of the
paper-sized outputs the absolute bounds alone accept a scaled or an all-zero result, so
check_output also carries relative bounds.  Expected rows come from the oracle; the "wrong"
results are made from them on the CPU."""
import numpy as np
import pytest

import oracle
from parity import check_output


def _minute_like_rows(nrows=96, n_g=17550, D=128, gate=0.08, seed=3):
    """Oracle rows of one group the size of a minute_bf16 group: N(0, 1) inputs rounded to bf16
    precision, gate of the order of the top-1 probability among 32 groups."""
    rng = np.random.default_rng(seed)

    def bf16(a):   # round to 8 mantissa bits, as the stored inputs are
        a = a.astype(np.float32)
        u = a.view(np.uint32)
        return (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16).astype(np.uint32).view(np.float32)

    Q, K, V = (bf16(rng.standard_normal((1, 1, n_g, D))) for _ in range(3))
    gid = np.zeros((1, n_g, 1), np.int32)
    offsets, perm, _ = oracle.sort(gid, 1)
    rows = np.stack([np.zeros(nrows, np.int32), np.zeros(nrows, np.int32),
                     rng.integers(0, n_g, nrows).astype(np.int32)], 1)
    return oracle.attn_rows(Q, K, V, gid, np.full((1, n_g, 1), gate), offsets, perm, 1.0 / np.sqrt(D), rows)


@pytest.fixture(scope="module")
def want():
    w = _minute_like_rows()
    # the situation the relative bounds exist for: the signal is below the absolute bounds
    assert np.abs(w).max() < 2e-2 and np.abs(w).mean() < 2e-3
    return w


def test_accepts_a_correctly_rounded_result(want):
    got = want.astype(np.float32)
    u = got.view(np.uint32)
    got = (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16).astype(np.uint32).view(np.float32)   # bf16 rounding
    check_output(got, want, "bf16")


@pytest.mark.parametrize("wrong", ["scaled_0.9", "zeros", "one_row_zero", "one_row_swapped"])
def test_rejects_wrong_results_at_paper_size_magnitude(want, wrong):
    got = want.copy()
    if wrong == "scaled_0.9":
        got *= 0.9
    elif wrong == "zeros":
        got[:] = 0.0
    elif wrong == "one_row_zero":
        got[7] = 0.0
    else:
        got[[3, 4]] = got[[4, 3]]
    with pytest.raises(AssertionError):
        check_output(got, want, "bf16")


def test_fp32_relative_bound(want):
    check_output(want.astype(np.float32), want, "f32")
    with pytest.raises(AssertionError):
        check_output(want * (1.0 + 1e-3), want, "f32")


def test_static_rows_agree_with_the_full_static_oracle():
    """static_group_attn_rows (one row at a time) against static_group_attn (whole groups with
    einsum), on the spatial-temporal lists of a small grid with augmented keys: two separately
    written evaluations of Eq. 1 over caller-given groups."""
    rng = np.random.default_rng(12)
    F, Hh, Ww = 6, 4, 6
    N = F * Hh * Ww
    Q, K, V = (rng.standard_normal((2, 2, N, 16)).astype(np.float32) for _ in range(3))
    qg, kg = oracle.stga_groups(F, Hh, Ww, 2, 3, [0, 2, 3], 2)
    full = oracle.static_group_attn(Q, K, V, qg, kg, 0.25)
    rows = [(b, h, n) for b in range(2) for h in range(2) for n in range(0, N, 5)]
    got = oracle.static_group_attn_rows(Q, K, V, qg, kg, 0.25, rows)
    want = np.stack([full[b, h, n] for b, h, n in rows])
    assert np.abs(got - want).max() < 1e-13
    # and a hand-checkable special case: a one-key group returns that key's value row
    one = oracle.static_group_attn_rows(Q, K, V, [np.array([5])], [np.array([9])], 0.25, [(1, 0, 5)])
    assert np.array_equal(one[0], V[1, 0, 9].astype(np.float64))
