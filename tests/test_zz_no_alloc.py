"""moga_sort_static: the group sort for hosts that cannot allocate device memory when
they need it (their framework's pool owns the GPU, or their budget was fixed at
start-up).  Its scratch is a device array inside the library, so the test checks that
two calls in a row -- which share that array and find the previous call's words in
it -- each give exactly what the workspace entry point (moga_permute, indices only)
gives, and exactly what the CPU oracle's sort of the same assignments gives.  Integer
outputs: the comparisons are bit for bit.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_18692_b200.inputs import GATE_SOFTMAX_ALL, MogaConfig

pytestmark = pytest.mark.gpu


def _gid(B, N, M, k, seed):
    rng = np.random.default_rng(seed)
    w = np.arange(1, M + 1, dtype=np.float64) ** -1.5
    first = rng.choice(M, size=(B, N), p=w / w.sum())
    cols = [first]
    for j in range(1, k):
        cols.append((first + j) % M)          # distinct groups per token
    return torch.from_numpy(np.stack(cols, -1).astype(np.int32)).cuda()


def test_static_sort_matches_workspace_sort_twice_in_a_row():
    from paper_2510_18692_b200 import build
    build.build()
    from paper_2510_18692_b200 import binding as mb

    calls = [(2, 70001, 64, 2, 1), (1, 9000, 8, 1, 2)]   # the second call is smaller: stale counters remain
    for B, N, M, k, seed in calls:
        cfg = MogaConfig("na", B, 2, N, 64, 64, M, k, "bf16", GATE_SOFTMAX_ALL, 0)
        sh = mb.make_shape(cfg)
        gid = _gid(B, N, M, k, seed)
        T = N * k
        ref = [torch.empty(B, T, dtype=torch.int32, device="cuda"),
               torch.empty(B, N, k, dtype=torch.int32, device="cuda"),
               torch.empty(B, M + 1, dtype=torch.int32, device="cuda")]
        ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
        mb.moga_permute(sh, gid, None, None, None, ref[0], ref[1], ref[2], None, None, None, ws)
        got = [torch.full_like(t, -1) for t in ref]
        status = torch.full((2,), 77, dtype=torch.int32, device="cuda")
        mb.moga_sort_static(sh, gid, got[0], got[1], got[2], status)
        torch.cuda.synchronize()
        for a, b in zip(ref, got):
            assert torch.equal(a, b)
        assert status.tolist() == [0, 0]
        o_off, o_perm, o_inv = oracle.sort(gid.cpu().numpy(), M)
        assert np.array_equal(got[0].cpu().numpy(), o_perm)
        assert np.array_equal(got[1].cpu().numpy(), o_inv)
        assert np.array_equal(got[2].cpu().numpy(), o_off)
    # a bad group id is clamped and reported through status_out, like the workspace variant
    gid[0, 5, 0] = 99
    mb.moga_sort_static(sh, gid, got[0], got[1], got[2], status)
    torch.cuda.synchronize()
    assert status[0].item() == 6 and (status[1].item() & 0x0fffffff) == 5
    # and the next call starts from a clean header again
    gid[0, 5, 0] = 0
    mb.moga_sort_static(sh, gid, got[0], got[1], got[2], status)
    torch.cuda.synchronize()
    assert status.tolist() == [0, 0]


def test_static_sort_of_no_tokens_is_a_no_op_with_zero_offsets():
    from paper_2510_18692_b200 import binding as mb
    cfg = MogaConfig("empty", 2, 1, 0, 64, 64, 8, 1, "bf16", GATE_SOFTMAX_ALL, 0)
    sh = mb.make_shape(cfg)
    offsets = torch.full((2, 9), 5, dtype=torch.int32, device="cuda")
    status = torch.full((2,), 77, dtype=torch.int32, device="cuda")
    mb.moga_sort_static(sh, None, None, None, offsets, status)
    torch.cuda.synchronize()
    assert not offsets.any() and status.tolist() == [0, 0]


def test_static_sort_rejects_what_does_not_fit():
    from paper_2510_18692_b200 import binding as mb
    # 16 batch items x 513 blocks x 64 groups of counters exceed the 1 MiB array
    cfg = MogaConfig("big", 16, 1, 2_100_000, 64, 64, 64, 1, "bf16", GATE_SOFTMAX_ALL, 0)
    sh = mb.make_shape(cfg)
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(mb.MogaError) as e:
        mb.moga_sort_static(sh, dummy, dummy, dummy, dummy, None)
    assert e.value.code == 3
