"""Host-side construction of the static spatial-temporal groups (Sec. 3.2) in the C-ABI
library against the oracle's independent construction: bit for bit, no GPU involved."""
import numpy as np
import pytest

import oracle
from paper_2510_18692_b200 import build as moga_build

CASES = [
    (9, 4, 6, 2, 3, [0, 3, 4], 2, True),       # shots of 3, 1, 5 frames; runs of 2
    (5, 5, 7, 2, 2, [0], 5, True),              # one shot: nothing to augment; ragged windows
    (6, 3, 4, 1, 1, [0, 1, 2, 3, 4, 5], 3, True),   # one-frame shots: every group sees both neighbours
    (8, 6, 10, 3, 4, [0, 5], 3, False),         # augmentation off
    (7, 30, 52, 2, 2, [0, 2], 4, True),         # the 480p grid with 2 x 2 windows
    (4, 2, 2, 2, 2, [0, 2], 1, True),           # one token per window
]


@pytest.fixture(scope="module")
def binding():
    moga_build.build()
    from paper_2510_18692_b200 import binding as b
    return b


@pytest.mark.parametrize("F,Hh,Ww,wh,ww,shots,tg,aug", CASES)
def test_group_lists_match_the_oracle(binding, F, Hh, Ww, wh, ww, shots, tg, aug):
    got = binding.moga_stga_build(F, Hh, Ww, wh, ww, shots, tg, aug)
    qg, kg = oracle.stga_groups(F, Hh, Ww, wh, ww, shots, tg, aug)
    assert got["G"] == len(qg) and got["Tkv"] == sum(len(k) for k in kg)
    assert np.array_equal(got["q_offsets"], np.concatenate([[0], np.cumsum([len(q) for q in qg])]))
    assert np.array_equal(got["kv_offsets"], np.concatenate([[0], np.cumsum([len(k) for k in kg])]))
    assert np.array_equal(got["q_idx"], np.concatenate(qg))
    assert np.array_equal(got["kv_idx"], np.concatenate(kg))
    N = F * Hh * Ww
    assert np.array_equal(got["q_idx"][got["q_inv"]], np.arange(N))      # q_inv inverts q_idx


def test_bad_arguments(binding):
    import ctypes
    lib = binding.lib
    shots = (ctypes.c_int32 * 2)(0, 9)
    null = ctypes.c_void_p(0)
    G = ctypes.c_int32(0)
    call = lambda F, wh, starts, n: lib.moga_stga_build(
        ctypes.c_int32(F), ctypes.c_int32(4), ctypes.c_int32(4), ctypes.c_int32(wh), ctypes.c_int32(2), starts,
        ctypes.c_int32(n), ctypes.c_int32(2), ctypes.c_int32(1), null, null, null, null, null, ctypes.byref(G), null)
    assert call(8, 2, shots, 2) == 1            # a shot starting past the last frame
    assert call(0, 2, shots, 1) == 1
    assert call(8, 5, shots, 1) == 1            # more windows than rows
    bad = (ctypes.c_int32 * 2)(1, 3)
    assert call(8, 2, bad, 2) == 1              # first shot must start at frame 0
    assert call(8, 2, shots, 1) == 0 and G.value == 4 * 4
