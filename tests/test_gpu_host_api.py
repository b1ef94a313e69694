"""moga_forward_host (host buffers, chunked copy/compute overlap) against moga_forward on the
same inputs: the same kernels run per head, so the outputs must be the same bits."""
import pytest
import torch

from paper_2510_18692_b200.inputs import GATE_SOFTMAX_ALL, GATE_SOFTMAX_TOPK, MogaConfig, make_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mb():
    from paper_2510_18692_b200 import build
    build.build()
    from paper_2510_18692_b200 import binding
    return binding


CASES = [
    (MogaConfig("h_top1", 1, 5, 2000, 256, 128, 8, 1, "bf16", GATE_SOFTMAX_ALL, 31), 2),    # 3 chunks, ragged last
    (MogaConfig("h_top2", 2, 4, 900, 128, 128, 6, 2, "bf16", GATE_SOFTMAX_TOPK, 32), 1),    # B = 2, 4 chunks
    (MogaConfig("h_f32", 1, 3, 700, 96, 64, 4, 1, "f32", GATE_SOFTMAX_ALL, 33), 3),         # one chunk
    (MogaConfig("h_skew", 1, 6, 3000, 128, 64, 16, 2, "bf16", GATE_SOFTMAX_TOPK, 34, zipf_bias=2.0), 4),
]


@pytest.mark.parametrize("cfg,hc", CASES, ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_host_forward_matches_device_forward(mb, cfg, hc):
    inp = make_inputs(cfg, device="cuda")
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_workspace_bytes(sh))
    O_dev = torch.empty_like(inp["Q"])
    gid = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device="cuda")
    gate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device="cuda")
    mb.moga_forward(sh, inp["X"], inp["Wr"], inp["bias"], inp["Q"], inp["K"], inp["V"], O_dev, ws, gid, gate)
    assert mb.moga_last_device_status(ws) == (0, 0)
    host = {k: (None if v is None else v.cpu().pin_memory()) for k, v in inp.items()}
    O_host = torch.full(inp["Q"].shape, float("nan"), dtype=inp["Q"].dtype).pin_memory()
    gid_h = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32).pin_memory()
    gate_h = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32).pin_memory()
    arena = mb.alloc_workspace(mb.moga_forward_host_bytes(sh, hc))
    for _ in range(2):                      # twice: the event pool is reused across calls
        O_host.fill_(float("nan"))
        mb.moga_forward_host(sh, host["X"], host["Wr"], host["bias"], host["Q"], host["K"], host["V"], O_host,
                             arena, hc, gid_h, gate_h)
        assert mb.moga_last_device_status(arena) == (0, 0)      # synchronises the stream
        assert torch.equal(O_host, O_dev.cpu())
        assert torch.equal(gid_h, gid.cpu()) and torch.equal(gate_h, gate.cpu())


def test_host_forward_argument_checks(mb):
    import ctypes
    cfg = CASES[0][0]
    sh = mb.make_shape(cfg)
    assert mb.moga_forward_host_bytes(sh, 0) == 0 and mb.moga_forward_host_bytes(sh, 6) == 0
    assert mb.moga_forward_host_bytes(mb.make_shape(cfg.with_(H=200)), 1) == 0        # more than 64 chunks
    need = mb.moga_forward_host_bytes(sh, 2)
    f = ctypes.c_void_p(0x10000)
    args = [ctypes.byref(sh), f, f, None, f, f, f, f, None, None]
    assert mb.lib.moga_forward_host(*args, None, ctypes.c_size_t(need), ctypes.c_int32(2), None) == 3
    assert mb.lib.moga_forward_host(*args, f, ctypes.c_size_t(need - 1), ctypes.c_int32(2), None) == 3
    strided = mb.make_shape(cfg, strides=(cfg.N * cfg.H * cfg.D, cfg.D, cfg.H * cfg.D))
    args[0] = ctypes.byref(strided)
    assert mb.lib.moga_forward_host(*args, f, ctypes.c_size_t(need), ctypes.c_int32(2), None) == 2
