"""Seeded synthetic inputs shaped like the paper's 480p video-DiT workloads.

This module holds only shapes and random draws; none of the method's arithmetic
lives here, so the CUDA path and the CPU oracle can both be fed from it.

Token counts follow the paper's setting (Sec. 3.1 footnote: VAE stride (4, 8, 8),
patchify (1, 2, 2)): a 480x832 frame gives 30x52 = 1,560 tokens per latent frame.
Activations are iid N(0, 1) rounded to the storage dtype; the router weight is
N(0, 1/C) in fp32, so logits are close to iid N(0, 1) and routing is balanced.
The skewed case adds a per-group bias 2*ln(w_i), w_i proportional to i^-1.2.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch

GATE_SOFTMAX_ALL = 0
GATE_SOFTMAX_TOPK = 1


@dataclass(frozen=True)
class MogaConfig:
    name: str
    B: int
    H: int
    N: int
    C: int
    D: int
    M: int
    k: int
    dtype: str            # "f32" or "bf16"
    gate_mode: int
    seed: int
    zipf_bias: float = 0.0  # 0: no bias; else bias_i = zipf_bias * ln(w_i), w ~ i^-1.2

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.D)

    @property
    def T(self) -> int:
        return self.N * self.k

    def with_(self, **kw) -> "MogaConfig":
        return replace(self, **kw)


# Top-1 follows the paper (gate = softmax over all M logits, Eq. 3-5); the
# top-2 cases use a softmax over the two selected logits.
CONFIGS = {
    "tiny_f32": MogaConfig("tiny_f32", 1, 2, 4096, 128, 64, 8, 1, "f32", GATE_SOFTMAX_ALL, 0),
    # the same case with one group: MoGA must then equal full attention (gate = 1)
    "tiny_f32_m1": MogaConfig("tiny_f32_m1", 1, 2, 4096, 128, 64, 1, 1, "f32", GATE_SOFTMAX_ALL, 0),
    "clip_bf16": MogaConfig("clip_bf16", 1, 12, 32760, 1536, 128, 8, 1, "bf16", GATE_SOFTMAX_ALL, 1),
    "multishot_bf16": MogaConfig("multishot_bf16", 1, 40, 126360, 5120, 128, 16, 2, "bf16",
                                 GATE_SOFTMAX_TOPK, 2),
    "minute_bf16": MogaConfig("minute_bf16", 1, 40, 561600, 5120, 128, 32, 1, "bf16",
                              GATE_SOFTMAX_ALL, 3),
    "skew_bf16": MogaConfig("skew_bf16", 2, 24, 131072, 3072, 128, 64, 2, "bf16",
                            GATE_SOFTMAX_TOPK, 4, zipf_bias=2.0),
}


def torch_dtype(cfg: MogaConfig) -> torch.dtype:
    return torch.float32 if cfg.dtype == "f32" else torch.bfloat16


def make_inputs(cfg: MogaConfig, device="cpu", heads=None):
    """Draw X, W_r, bias, Q, K, V for ``cfg``.

    Each tensor has its own generator seeded from (cfg.seed, tensor index), so a
    subset of heads (``heads``: list of head indices) reproduces exactly the
    slices of the full draw: Q/K/V are drawn head by head.
    Returns a dict of tensors on ``device``; ``bias`` is None when there is none.
    """
    dt = torch_dtype(cfg)
    dev = torch.device(device)

    def gen(idx):
        g = torch.Generator(device=dev)
        g.manual_seed(cfg.seed * 1_000_003 + idx)
        return g

    X = torch.randn(cfg.B, cfg.N, cfg.C, generator=gen(0), device=dev, dtype=torch.float32).to(dt)
    Wr = torch.randn(cfg.C, cfg.M, generator=gen(1), device=dev, dtype=torch.float32) / math.sqrt(cfg.C)
    bias = None
    if cfg.zipf_bias != 0.0:
        w = torch.arange(1, cfg.M + 1, dtype=torch.float64) ** (-1.2)
        w = w / w.sum()
        bias = (cfg.zipf_bias * torch.log(w)).to(torch.float32).to(dev)
    head_list = list(range(cfg.H)) if heads is None else list(heads)
    out = {}
    for t_i, name in enumerate(("Q", "K", "V")):
        t = torch.empty(cfg.B, len(head_list), cfg.N, cfg.D, device=dev, dtype=dt)
        for j, h in enumerate(head_list):
            t[:, j] = torch.randn(cfg.B, cfg.N, cfg.D, generator=gen(10 + 1000 * t_i + h),
                                  device=dev, dtype=torch.float32).to(dt)
        out[name] = t
    out.update(X=X, Wr=Wr, bias=bias)
    return out


def useful_flops(group_sizes, H: int, D: int) -> float:
    """Attention FLOPs counted as the paper counts them (Appendix A: 4*n^2*d per
    head for QK^T and PV together), summed over groups: H * sum_g 4 n_g^2 D."""
    return float(H) * float(sum(4.0 * float(n) * float(n) * D for n in group_sizes))
