"""The bounded device wait, made to run out in the safe form: a one-block self-test kernel
waits, through the same routine the attention and router kernels use, on a barrier that
nothing signals.  The kernel must return by itself, the host must read MOGA_ERR_TIMEOUT with
the documented detail word, and the workspace must serve an ordinary call afterwards."""
import math

import numpy as np
import pytest
import torch

import oracle
from parity import check_output, grouped_case, to_np32
from paper_2510_18692_b200.inputs import GATE_SOFTMAX_ALL, MogaConfig

pytestmark = pytest.mark.gpu


def test_wait_that_runs_out_is_reported_and_the_workspace_stays_usable():
    from paper_2510_18692_b200 import build
    build.build()
    from paper_2510_18692_b200 import binding as mb

    case = grouped_case([300, 77], 2, 128, "bf16", seed=41, B=1)
    cfg = MogaConfig("to", 1, 2, case["T"], 64, 128, 2, 1, "bf16", GATE_SOFTMAX_ALL, 0)
    sh = mb.make_shape(cfg, scale=1.0 / math.sqrt(128))
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh))
    limit_ns = 1_000_000                                      # 1 ms
    mb.moga_selftest_wait_timeout(ws, limit_ns)
    torch.cuda.synchronize()
    words = ws[:20].view(torch.int32).cpu().numpy().astype(np.int64) & 0xFFFFFFFF
    waited = int(words[2]) | (int(words[3]) << 32)
    assert limit_ns < waited < 50 * limit_ns, waited          # it waited out the limit, and not much more
    assert int(words[4]) == 1                                 # the second warp left through the abort flag
    code, detail = mb.moga_last_device_status(ws)
    assert code == 5 and mb.STATUS_NAMES[code] == "MOGA_ERR_TIMEOUT"
    assert detail == 0x7E000000
    assert mb.moga_last_device_status(ws) == (0, 0)           # reading clears the word
    # argument checks: no launch
    with pytest.raises(mb.MogaError) as e:
        mb.moga_selftest_wait_timeout(ws, 10**9)
    assert e.value.code == 1
    # the same workspace, an ordinary call: correct and status OK
    Op = torch.full_like(case["Q"], float("nan"))
    mb.moga_group_attn(sh, case["Q"], case["K"], case["V"], torch.from_numpy(case["offsets"]).cuda(), Op, None, ws)
    assert mb.moga_last_device_status(ws) == (0, 0)
    want = oracle.attn_all(to_np32(case["Q"]), to_np32(case["K"]), to_np32(case["V"]), case["gid"],
                           np.ones((1, case["T"], 1)), case["offsets"], case["perm"], 1.0 / math.sqrt(128))
    check_output(Op.float().cpu().numpy(), want, "bf16", "Op after a reported time-out")
