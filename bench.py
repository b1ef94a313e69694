#!/usr/bin/env python
"""Benchmark of the MoGA routed group-attention forward on B200.

One "step" is one pass of the whole hot path (route -> sort -> gather -> group
attention -> gated unpermute) over one layer-sized batch of synthetic input, by
default the minute-long 561,600-token context.  Prints ONE JSON line:
effective TFLOP/s (useful FLOPs = H * sum_g 4 n_g^2 D of the run's actual group
sizes), the per-stage breakdown, the roofline of the dominant kernel, the same
metric end to end from host buffers, and the CPU oracle timed beside it.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs
its own layer (weak scaling, no collective on the data path); time is the max
over ranks and `value` the whole-job aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2510_18692_b200.inputs import CONFIGS, make_inputs, useful_flops  # noqa: E402

METRIC = "MoGA fwd effective TFLOP/s (bf16)"
L2_FLUSH_BYTES = 256 << 20           # twice the 126 MB L2
SM_COUNT, FP32_LANES_PER_SM = 148, 128   # B200: fp32 FMA peak = SMs x lanes x 2 flop x clock
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes of the attention kernel / its algorithmic bytes, from the ncu capture of the
# clip-sized case (traffic grows with T*H: every Q/K/V/O byte crosses DRAM once).  The figure
# belongs to one version of the kernel source: when the source's hash differs, traffic is null.
ATTN_TRAFFIC = {"duo": {"file": "attn_bf16_duo.cu", "ratio": 0.9574, "source_sha16": "efd7d44a4d983365"},
                "single": {"file": "attn_bf16.cu", "ratio": 0.9565, "source_sha16": "6a7a8dee240eb5b1"}}


def attn_traffic_ratio(kernel):
    import hashlib
    rec = ATTN_TRAFFIC.get(kernel)
    if rec is None:
        return None
    path = os.path.join(ROOT, "paper_2510_18692_b200", "csrc", rec["file"])
    try:
        with open(path, "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()[:16]
    except OSError:
        return None
    return rec["ratio"] if sha == rec["source_sha16"] else None


def attn_kernel_name(cfg, choice):
    """Which group-attention kernel a forward of cfg runs under --attn-kernel `choice`."""
    if cfg.dtype != "bf16":
        return "alu"
    if cfg.D != 128 or choice == "single":
        return "single"
    return "pair" if choice == "pair" else "duo"


def schedule_tail(offsets_np, H, n_ctas=148, qblock=256, tile_n=128):
    """Imbalance of the attention kernel's static schedule for these group sizes: work items of
    `qblock` query rows, groups in order of decreasing cost inside each batch item, item w goes to
    CTA w mod n_ctas.  An item costs (query tiles) x (key tiles).  Returns max over CTAs of the
    assigned cost / mean."""
    load = np.zeros(n_ctas)
    w = 0
    for b in range(offsets_np.shape[0]):
        sizes = np.diff(offsets_np[b]).astype(np.int64)
        for g in np.argsort(-(sizes * sizes), kind="stable"):
            n = int(sizes[g])
            if n == 0:
                continue
            nqb, ktiles = -(-n // qblock), -(-n // tile_n)
            last_rows = n - (nqb - 1) * qblock
            costs = np.full(nqb, 2.0 * ktiles)
            costs[-1] = (2.0 if last_rows > tile_n else 1.0) * ktiles
            items = np.tile(costs, H)                 # head-major, query block fastest
            idx = (w + np.arange(items.size)) % n_ctas
            np.add.at(load, idx, items)
            w += items.size
    return float(load.max() / load.mean()) if load.mean() > 0 else 1.0


def kernels_per_forward(cfg, attn_kernel="duo"):
    """Kernels one moga_forward launches: router (bf16: weight split + tensor-core router; fp32: one
    ALU kernel), 3 sort kernels, gather, attention (bf16: schedule + attention, plus the launch of the
    exact kernel over the list of handed-over items when the default or the CTA-pair kernel runs),
    and the gated unpermute unless the bf16 top-1 attention epilogue already wrote token order."""
    if cfg.dtype == "bf16":
        return 2 + 3 + 1 + (3 if attn_kernel in ("duo", "pair") else 2) + (1 if cfg.k > 1 else 0)
    return 1 + 3 + 1 + 1 + 1


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# ----------------------------------------------------------------------------- distributed glue
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), \
        int(os.environ.get("WORLD_SIZE", 1))


def aggregate(ms_local: float, units_local: float, device=None):
    """Max of the per-rank times and sum of the per-rank work (all ranks get both)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms_local, units_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def barrier_sync():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
    torch.cuda.synchronize()


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        """`device`: a torch CUDA device.  The GPU is named to nvidia-smi by its UUID: the CUDA
        ordinal is not the physical index once CUDA_VISIBLE_DEVICES is set."""
        try:
            self.uuid = "GPU-" + str(torch.cuda.get_device_properties(device).uuid).removeprefix("GPU-")
        except Exception:   # noqa: BLE001  (older torch without the field)
            self.uuid = None
        self.index = str(device.index or 0) if self.uuid is None else self.uuid
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", self.index], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        if not out.strip():
            # the timed region was shorter than the tool's start-up: one query right after it
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i",
                                      self.index], capture_output=True, text=True, timeout=10).stdout
            except (OSError, subprocess.TimeoutExpired):
                out = ""
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "gpu_uuid": self.uuid}


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(cfg, host, routing, target_s=12.0):
    """Time the oracle, as it stands, on a bounded sample: routing of 1,024 tokens and
    attention rows of head 0 (calibrated on 64 rows to fill about `target_s` seconds)."""
    import oracle
    gid, gate, offsets, perm = routing
    rng = np.random.default_rng(0)
    tok = np.sort(rng.choice(cfg.N, size=min(1024, cfg.N), replace=False))
    t0 = time.perf_counter()
    oracle.route(host["X"][:, tok], host["Wr"], host["bias"], cfg.k, cfg.gate_mode)
    t_route = time.perf_counter() - t0
    sizes = np.diff(offsets[0])

    def run(nrows, seed):
        r = np.random.default_rng(seed)
        rows = np.stack([np.zeros(nrows, np.int32), np.zeros(nrows, np.int32),
                         r.integers(0, cfg.N, nrows).astype(np.int32)], 1)
        fl = sum(4.0 * sizes[g] * cfg.D for n in rows[:, 2] for g in gid[0, n])
        t0 = time.perf_counter()
        oracle.attn_rows(host["Q"], host["K"], host["V"], gid, gate, offsets, perm, cfg.scale, rows)
        return time.perf_counter() - t0, fl

    t_cal, _ = run(64, 1)                    # includes thread start-up: only good for a first guess
    n2 = int(max(64, min(50000, 64 * 2.0 / max(t_cal, 1e-4))))
    t2, _ = run(n2, 3)                       # a ~2 s run calibrates the real one
    nrows = int(max(64, min(400000, n2 * target_s / max(t2, 1e-4))))
    t, fl = run(nrows, 2)
    return dict(tflops=fl / t / 1e12, seconds=t, rows=nrows, flops=fl, route_tokens=len(tok),
                route_seconds=t_route, cores=oracle.threads())


def run_reference(args, cfg):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample of the workload."""
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle
    small = cfg.with_(H=1)
    inp = make_inputs(small, device="cpu", heads=[0])
    host = {k: (None if v is None else v.float().numpy()) for k, v in inp.items()}
    gid, gate, _ = oracle.route(host["X"], host["Wr"], host["bias"], cfg.k, cfg.gate_mode)
    offsets, perm, _ = oracle.sort(gid, cfg.M)
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals, secs, rows = [], [], 0
    for i in range(args.warmup + args.steps):
        r = oracle_sample(cfg, host, (gid, gate, offsets, perm), target_s=per_step)
        if i >= args.warmup:
            vals.append(r["tflops"])
            secs.append(r["seconds"])
            rows = r["rows"]
    v = float(np.mean(vals))
    sample = f"{rows} attention rows of head 0 per step (fp64 oracle, routing from the oracle)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_dict(cfg),
        "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))
    return 0


def config_dict(cfg):
    es = 2 if cfg.dtype == "bf16" else 4
    resident = cfg.B * cfg.N * (cfg.C + 3 * cfg.H * cfg.D) * es
    return {"workload": cfg.name, "B": cfg.B, "H": cfg.H, "N": cfg.N, "C": cfg.C, "D": cfg.D, "M": cfg.M,
            "k": cfg.k, "gate_mode": "softmax_all" if cfg.gate_mode == 0 else "softmax_topk",
            "l2": "inputs larger than L2 (no flush needed)" if resident >= L2_FLUSH_BYTES
                  else "L2 flushed before every timed step (a 256 MB buffer rewritten)"}


# ----------------------------------------------------------------------------- GPU arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="minute_bf16", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--sharding", default="auto", choices=["auto", "layers", "heads"],
                    help="with N > 1 ranks: 'heads' splits ONE layer: tokens of X for routing, heads of Q/K/V for "
                         "attention, with one all-gather of the routing results as the only exchange (strong "
                         "scaling; the default for N > 1); 'layers' gives every rank its own layer (weak scaling, no "
                         "collective; the default for N = 1)")
    ap.add_argument("--stage", default="all", choices=["all", "route", "visual", "backward"],
                    help="'route' times moga_route alone on the config's X (a small resident set, for profiling); "
                         "'visual' times the whole visual-attention block: routed branch, the two static-group "
                         "branches and their mean; 'backward' times moga_backward (gradients of the group attention and "
                         "the gates) after a staged forward of the config")
    ap.add_argument("--attn-kernel", default="auto", choices=["auto", "single", "pair"],
                    help="bf16 group-attention kernel (moga_set_attn_kernel): auto (two softmax threads per row where "
                         "the launch allows it), the one-thread-per-row kernel, or the CTA-pair kernel, for A/B runs "
                         "and profiles")
    ap.add_argument("--topk-epilogue", default="staged", choices=["staged", "add"],
                    help="bf16 top-2 output path (moga_set_fused_topk): permuted output + unpermute (default) or "
                         "gate * row added into token order by the attention epilogue")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = CONFIGS[args.config]
    if args.impl == "reference":
        return run_reference(args, cfg)

    rank, local_rank, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)

    from paper_2510_18692_b200 import build
    build.build()
    from paper_2510_18692_b200 import binding as mb   # raises if the CUDA library is missing

    mb.moga_set_attn_kernel({"auto": 0, "single": 1, "pair": 2}[args.attn_kernel])
    mb.moga_set_fused_topk(args.topk_epilogue == "add")
    cfg = cfg.with_(seed=cfg.seed + 100 * rank)       # every rank works on its own layer
    if args.sharding == "auto":
        args.sharding = "heads" if world > 1 else "layers"
    if args.sharding == "heads":
        return run_head_sharded(mb, CONFIGS[args.config], dev, args, rank, world)
    if args.stage == "route":
        return run_route_only(mb, cfg, dev, args)
    if args.stage == "visual":
        return run_visual_block(mb, cfg, dev, args)
    if args.stage == "backward":
        return run_backward(mb, cfg, dev, args)
    inp = make_inputs(cfg, device=dev)
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_workspace_bytes(sh), dev)
    O = torch.empty_like(inp["Q"])
    T = cfg.T
    gid = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device=dev)
    gate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device=dev)
    perm = torch.empty(cfg.B, T, dtype=torch.int32, device=dev)
    inv = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device=dev)
    offsets = torch.empty(cfg.B, cfg.M + 1, dtype=torch.int32, device=dev)

    def step():
        mb.moga_forward(sh, inp["X"], inp["Wr"], inp["bias"], inp["Q"], inp["K"], inp["V"], O, ws,
                        gid, gate, perm, offsets)

    for _ in range(args.warmup):
        step()
    code, detail = mb.moga_last_device_status(ws)
    if code != 0:
        raise RuntimeError(f"device status {code} detail {detail:#x} after warm-up")
    sizes = np.diff(offsets.cpu().numpy(), axis=1)
    flops = sum(useful_flops(sizes[b], cfg.H, cfg.D) for b in range(cfg.B))

    clocks = ClockSampler(dev)
    clocks.start()
    # exactly args.steps steps between two synchronisations, each between its own pair of events
    # (the headline is the median of the per-step times; their mean is kept beside it).  Inputs
    # smaller than L2 would stay cached from step to step: then a buffer larger than L2 is
    # rewritten before every step, outside that step's event pair.
    resident = sum(inp[n].numel() * inp[n].element_size() for n in ("X", "Q", "K", "V"))
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev) if resident < L2_FLUSH_BYTES else None
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier_sync()
    for e0, e1 in ev:
        if flush is not None:
            flush.fill_(1)
        e0.record()
        step()
        e1.record()
    barrier_sync()
    per_step = [e0.elapsed_time(e1) for e0, e1 in ev]
    ms_mean_local = float(np.mean(per_step))
    ms_local = float(statistics.median(per_step))

    # per-stage breakdown through the stage entry points (same kernels, same data)
    es = 2 if cfg.dtype == "bf16" else 4
    Qp, Kp, Vp, Op = (torch.empty(cfg.B, cfg.H, T, cfg.D, dtype=inp["Q"].dtype, device=dev) for _ in range(4))
    stage_names = ["route", "permute", "group_attn", "unpermute"]
    stage_ms = {n: [] for n in stage_names}
    for it in range(args.steps + 1):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        if flush is not None:
            flush.fill_(1)
        e[0].record()
        mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], gid, gate, None, ws)
        e[1].record()
        mb.moga_permute(sh, gid, inp["Q"], inp["K"], inp["V"], perm, inv, offsets, Qp, Kp, Vp, ws)
        e[2].record()
        mb.moga_group_attn(sh, Qp, Kp, Vp, offsets, Op, None, ws)
        e[3].record()
        mb.moga_unpermute(sh, Op, inv, gate, O)
        e[4].record()
        torch.cuda.synchronize()
        if it > 0:
            for i, n in enumerate(stage_names):
                stage_ms[n].append(e[i].elapsed_time(e[i + 1]))
    clk = clocks.stop()
    del Qp, Kp, Vp, Op
    stage = {n: float(statistics.median(v)) for n, v in stage_ms.items()}

    ms, total_flops = aggregate(ms_local, flops, dev)
    ms_mean, _ = aggregate(ms_mean_local, flops, dev)
    value = total_flops / (ms * 1e-3) / 1e12
    peaks = load_peaks()
    attn_tflops = flops / (stage["group_attn"] * 1e-3) / 1e12
    tok = cfg.B * cfg.N
    bytes_alg = {
        "route": tok * cfg.C * es + tok * cfg.k * 8,
        "permute": 3 * (1 + cfg.k) * tok * cfg.H * cfg.D * es + tok * cfg.k * 12,
        "unpermute": (cfg.k + 1) * tok * cfg.H * cfg.D * es + tok * cfg.k * 8,
    }
    stages_out = {n: {"ms": stage[n]} for n in stage_names}
    for n, by in bytes_alg.items():
        gbs = by / (stage[n] * 1e-3) / 1e9
        stages_out[n].update({"GB/s": gbs, "frac_hbm": gbs / peaks["hbm_gbs"]})
    mhz = clk.get("sm_mhz")
    stages_out["group_attn"].update({"TFLOP/s": attn_tflops,
                                     "frac_tensor_burst": attn_tflops / peaks["bf16_tflops"],
                                     "frac_tensor_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
                                     # time x clock: compares boxes whose power cap settles at different clocks
                                     "ms_x_sm_mhz": None if not mhz else stage["group_attn"] * mhz})
    akern = attn_kernel_name(cfg, args.attn_kernel)
    ratio = attn_traffic_ratio(akern)
    out = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "ms_per_step_mean": ms_mean,
        "timing": f"median of {args.steps} per-step CUDA-event times (max over ranks); mean over the region beside it",
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic", "config": config_dict(cfg),
        "route_kernel": "tensor" if cfg.dtype == "bf16" else "alu",
        "attn_kernel": akern,
        "topk_epilogue": args.topk_epilogue if (cfg.dtype == "bf16" and cfg.k == 2) else None,
        "ms_per_layer_head_batch": ms / (cfg.B * cfg.H), "useful_tflop_per_step": flops / 1e12,
        "group_sizes": {"min": int(sizes.min()), "max": int(sizes.max()), "empty": int((sizes == 0).sum())},
        "stages": stages_out, "gpu_launches": kernels_per_forward(cfg, akern) * args.steps, "clocks": clk,
        "schedule_tail": schedule_tail(offsets.cpu().numpy(), cfg.H) if cfg.dtype == "bf16" else None,
    }
    if cfg.dtype == "bf16":
        out["roofline"] = {
            "kernel": "moga_group_attn (tcgen05 varlen attention)", "bound": "tensor",
            "achieved": attn_tflops, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
            "frac": attn_tflops / peaks["bf16_tflops_sustained"],
            "peak_source": f"{peaks['source']} sustained bf16 GEMM",
            "frac_of_burst_peak": attn_tflops / peaks["bf16_tflops"],
            "algorithmic_bytes": 4.0 * tok * cfg.k * cfg.H * cfg.D * es,
            "traffic": None if ratio is None else ratio * 4.0 * tok * cfg.k * cfg.H * cfg.D * es,
            "traffic_unit": "bytes per launch (ncu dram bytes of the clip_bf16 capture, scaled by T*H; "
                            "null when the kernel source changed after the capture)"}
    else:
        # fp32 attention runs on the fp32 ALUs: 2 flop per lane per clock at the maximum SM clock
        alu_peak = SM_COUNT * FP32_LANES_PER_SM * 2 * (clk.get("sm_max_mhz") or peaks.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12
        out["roofline"] = {
            "kernel": "moga_group_attn (fp32 ALU varlen attention)", "bound": "alu", "achieved": attn_tflops,
            "peak": alu_peak, "unit": "TFLOP/s", "frac": attn_tflops / alu_peak,
            "peak_source": "148 SMs x 128 fp32 lanes x 2 flop x max SM clock", "traffic": None}

    if rank == 0 and not args.no_e2e:
        out["e2e"] = run_e2e(mb, cfg, sh, inp, ws, O, flops, args)
    if rank == 0 and not args.no_cpu and world == 1:
        host = {n: inp[n][:, :1].float().cpu().numpy() for n in ("Q", "K", "V")}
        host.update(Wr=inp["Wr"].cpu().numpy(), X=_LazyRows(inp["X"]),
                    bias=None if inp["bias"] is None else inp["bias"].cpu().numpy())
        # the sampled rows use the GPU's routing (same protocol as the parity tests)
        r = oracle_sample(cfg, host, (gid.cpu().numpy(), gate.double().cpu().numpy(),
                                      offsets.cpu().numpy(), perm.cpu().numpy()))
        out["cpu_baseline"] = {"value": r["tflops"], "unit": "TFLOP/s", "cores": r["cores"], "kind": "oracle",
                               "sample": f"{r['rows']} attention rows of head 0 in {r['seconds']:.1f} s "
                                         f"(plus routing of {r['route_tokens']} tokens in {r['route_seconds']:.2f} s)"}
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))
    return 0


def run_route_only(mb, cfg, dev, args):
    """moga_route alone through the C ABI: X, W_r and the routing outputs are all that is resident."""
    inp = make_inputs(cfg, device=dev, heads=[])
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh), dev)
    gid = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device=dev)
    gate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device=dev)
    for _ in range(args.warmup):
        mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], gid, gate, None, ws)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], gid, gate, None, ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    es = 2 if cfg.dtype == "bf16" else 4
    by = cfg.B * cfg.N * (cfg.C * es + cfg.k * 8)
    peaks = load_peaks()
    print(json.dumps({"stage": "route", "config": config_dict(cfg), "ms": ms, "GB/s": by / ms / 1e6,
                      "frac_hbm": by / ms / 1e6 / peaks["hbm_gbs"], "peak_source": peaks["source"],
                      "device_status": mb.moga_last_device_status(ws)[0]}))
    return 0


def run_backward(mb, cfg, dev, args):
    """moga_backward on the config's layer: a staged forward keeps the sorted-order tensors and lse, a
    random upstream gradient is drawn, and the backward call is timed (bf16, d_head = 128)."""
    inp = make_inputs(cfg, device=dev)
    sh = mb.make_shape(cfg)
    T = cfg.T
    ws = mb.alloc_workspace(mb.moga_scratch_bytes(sh), dev)
    gid = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device=dev)
    gate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device=dev)
    perm = torch.empty(cfg.B, T, dtype=torch.int32, device=dev)
    inv = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.int32, device=dev)
    offsets = torch.empty(cfg.B, cfg.M + 1, dtype=torch.int32, device=dev)
    Qp, Kp, Vp, Op = (torch.empty(cfg.B, cfg.H, T, cfg.D, dtype=inp["Q"].dtype, device=dev) for _ in range(4))
    lse = torch.empty(cfg.B, cfg.H, T, dtype=torch.float32, device=dev)
    logits = torch.empty(cfg.B, cfg.N, cfg.M, dtype=torch.float32, device=dev)
    mb.moga_route(sh, inp["X"], inp["Wr"], inp["bias"], gid, gate, logits, ws)
    mb.moga_permute(sh, gid, inp["Q"], inp["K"], inp["V"], perm, inv, offsets, Qp, Kp, Vp, ws)
    mb.moga_group_attn(sh, Qp, Kp, Vp, offsets, Op, lse, ws)
    dO = torch.randn(inp["Q"].shape, device=dev, dtype=torch.float32).to(inp["Q"].dtype)
    dQ, dK, dV = (torch.empty_like(inp["Q"]) for _ in range(3))
    dgate = torch.empty(cfg.B, cfg.N, cfg.k, dtype=torch.float32, device=dev)
    wsb = mb.alloc_workspace(mb.moga_backward_workspace_bytes(sh), dev)

    def step():
        mb.moga_backward(sh, Qp, Kp, Vp, Op, lse, gate, perm, inv, offsets, dO, dQ, dK, dV, dgate, wsb)

    for _ in range(args.warmup):
        step()
    code, detail = mb.moga_last_device_status(wsb)
    if code != 0:
        raise RuntimeError(f"device status {code} detail {detail:#x}")
    clocks = ClockSampler(dev)
    clocks.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    torch.cuda.synchronize()
    for e0, e1 in ev:
        e0.record()
        step()
        e1.record()
    torch.cuda.synchronize()
    clk = clocks.stop()
    ms = float(statistics.median(e0.elapsed_time(e1) for e0, e1 in ev))
    # the router's own backward from the dgate just computed
    dX = torch.empty_like(inp["X"])
    dWr = torch.empty_like(inp["Wr"])
    dbias = torch.empty(cfg.M, dtype=torch.float32, device=dev)
    wsr = mb.alloc_workspace(mb.moga_route_backward_workspace_bytes(sh), dev)
    rb = []
    for it in range(args.warmup + args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        mb.moga_route_backward(sh, inp["X"], inp["Wr"], logits, gid, dgate, dX, dWr, dbias, wsr)
        e1.record()
        torch.cuda.synchronize()
        if it >= args.warmup:
            rb.append(e0.elapsed_time(e1))
    ms_route = float(statistics.median(rb))
    sizes = np.diff(offsets.cpu().numpy(), axis=1)
    fwd = sum(useful_flops(sizes[b], cfg.H, cfg.D) for b in range(cfg.B))
    peaks = load_peaks()
    print(json.dumps({
        "stage": "backward", "config": config_dict(cfg), "ms": ms, "steps": args.steps,
        "route_backward_ms": ms_route,
        "route_backward_GFLOP": 4.0 * cfg.B * cfg.N * cfg.C * cfg.M / 1e9,
        "route_backward_TFLOP/s(fp32)": 4.0 * cfg.B * cfg.N * cfg.C * cfg.M / ms_route / 1e9,
        "useful_tflop": 2.5 * fwd / 1e12, "executed_tflop": 3.5 * fwd / 1e12,
        "useful_TFLOP/s": 2.5 * fwd / ms / 1e9, "executed_TFLOP/s": 3.5 * fwd / ms / 1e9,
        "frac_tensor_sustained_executed": 3.5 * fwd / ms / 1e9 / peaks["bf16_tflops_sustained"],
        "note": "useful = five GEMMs of 2 n^2 D per group (2.5 x the forward); executed = seven (the transposed "
                "products are recomputed for dK / dV)", "clocks": clk}))
    return 0


def run_head_sharded(mb, cfg, dev, args, rank, world):
    """One layer split over the ranks (strong scaling): see paper_2510_18692_b200/sharded.py."""
    from paper_2510_18692_b200.sharded import ShardPlan, shard_bounds
    lo, hi = shard_bounds(cfg.N, world, rank)
    h_lo, h_hi = shard_bounds(cfg.H, world, rank)
    inp = make_inputs(cfg, device=dev, heads=list(range(h_lo, h_hi)))      # every rank draws the same layer
    X_local = inp["X"][:, lo:hi].contiguous()
    del inp["X"]
    O = torch.empty_like(inp["Q"])
    plan = ShardPlan(mb, cfg, dev)          # workspaces, routing and exchange buffers: allocated once

    def step():
        return plan.forward(X_local, inp["Wr"], inp["bias"], inp["Q"], inp["K"], inp["V"], O)

    for _ in range(args.warmup):
        _, _, offsets = step()
    sizes = np.diff(offsets.cpu().numpy(), axis=1)
    flops_local = sum(useful_flops(sizes[b], h_hi - h_lo, cfg.D) for b in range(cfg.B))
    clocks = ClockSampler(dev)
    clocks.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    barrier_sync()
    ev[0].record()
    for _ in range(args.steps):
        step()
    ev[1].record()
    barrier_sync()
    clk = clocks.stop()
    ms, total_flops = aggregate(ev[0].elapsed_time(ev[1]) / args.steps, flops_local, dev)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": total_flops / (ms * 1e-3) / 1e12, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": dict(config_dict(cfg), sharding="tokens for routing, heads for attention; one all-gather of (gid, gate)"),
            "gpu_launches": kernels_per_forward(cfg, attn_kernel_name(cfg, args.attn_kernel)) * args.steps,
            "ms_per_layer_head_batch": ms * world / (cfg.B * cfg.H),
            "clocks": clk}))
    return 0


def run_visual_block(mb, cfg, dev, args):
    """The visual attention block of Sec. 3.2 on the config's layer: MoGA forward, the
    spatial-temporal static branch (4 x 4 windows, runs of 8 latent frames, synthetic shots of
    45 latent frames, keys augmented across shot boundaries), the per-frame branch, and the mean."""
    per_frame = 1560
    Hh, Ww, wh, ww, tg, shot_len = 30, 52, 4, 4, 8, 45
    if cfg.N % per_frame != 0:
        raise SystemExit("the visual block needs a token count that is a whole number of 30x52 frames")
    F = cfg.N // per_frame
    inp = make_inputs(cfg, device=dev)
    sh = mb.make_shape(cfg)
    ws = mb.alloc_workspace(mb.moga_workspace_bytes(sh), dev)
    lists = mb.moga_stga_build(F, Hh, Ww, wh, ww, list(range(0, F, shot_len)), tg, True)
    G, Tkv, N = lists["G"], lists["Tkv"], cfg.N
    d = lambda a: torch.from_numpy(a).to(dev)
    q_idx, q_inv, kv_idx = d(lists["q_idx"]), d(lists["q_inv"]), d(lists["kv_idx"])
    q_off, kv_off = d(lists["q_offsets"]), d(lists["kv_offsets"])
    fr_off = torch.arange(F + 1, dtype=torch.int32, device=dev) * per_frame
    dt = inp["Q"].dtype
    A, C, O = (torch.empty_like(inp["Q"]) for _ in range(3))
    Qs = torch.empty(cfg.B, cfg.H, N, cfg.D, dtype=dt, device=dev)
    Ks, Vs = (torch.empty(cfg.B, cfg.H, Tkv, cfg.D, dtype=dt, device=dev) for _ in range(2))
    Bs = torch.empty_like(Qs)
    ws_st = mb.alloc_workspace(mb.moga_static_scratch_bytes(sh, G), dev)
    ws_fr = mb.alloc_workspace(mb.moga_static_scratch_bytes(sh, F), dev)
    names = ["moga_forward", "st_gather", "st_attn", "frame_attn", "mean3"]
    times = {n: [] for n in names}
    for it in range(args.warmup + args.steps):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        e[0].record()
        mb.moga_forward(sh, inp["X"], inp["Wr"], inp["bias"], inp["Q"], inp["K"], inp["V"], A, ws)
        e[1].record()
        mb.moga_gather_rows(sh, q_idx, inp["Q"], Qs)
        mb.moga_gather_rows(sh, kv_idx, inp["K"], Ks)
        mb.moga_gather_rows(sh, kv_idx, inp["V"], Vs)
        e[2].record()
        mb.moga_static_group_attn(sh, G, N, Tkv, Qs, Ks, Vs, q_off, kv_off, Bs, None, ws_st)
        e[3].record()
        mb.moga_static_group_attn(sh, F, N, N, inp["Q"], inp["K"], inp["V"], fr_off, fr_off, C, None, ws_fr)
        e[4].record()
        mb.moga_mean3(sh, A, Bs, q_inv, C, O)
        e[5].record()
        torch.cuda.synchronize()
        if it >= args.warmup:
            for i, n in enumerate(names):
                times[n].append(e[i].elapsed_time(e[i + 1]))
    # the same block through the single C-ABI call
    del A, C, Qs, Ks, Vs, Bs
    st_lists, keep = mb.make_static_lists(lists, F, per_frame, dev)
    ws_v = mb.alloc_workspace(mb.moga_visual_workspace_bytes(sh, st_lists), dev)
    one = []
    for it in range(args.warmup + args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        mb.moga_visual_forward(sh, inp["X"], inp["Wr"], inp["bias"], inp["Q"], inp["K"], inp["V"], O, st_lists, ws_v)
        e1.record()
        torch.cuda.synchronize()
        if it >= args.warmup:
            one.append(e0.elapsed_time(e1))
    for w in (ws, ws_st, ws_fr, ws_v):
        code, detail = mb.moga_last_device_status(w)
        if code != 0:
            raise RuntimeError(f"device status {code} detail {detail:#x}")
    ms = {n: float(np.mean(v)) for n, v in times.items()}
    nq, nk = np.diff(lists["q_offsets"]).astype(np.float64), np.diff(lists["kv_offsets"]).astype(np.float64)
    fl_st = cfg.B * cfg.H * 4.0 * cfg.D * float((nq * nk).sum())
    fl_fr = cfg.B * cfg.H * 4.0 * cfg.D * F * float(per_frame) ** 2
    es = 2 if cfg.dtype == "bf16" else 4
    row = cfg.B * cfg.H * cfg.D * es
    peaks = load_peaks()
    print(json.dumps({
        "stage": "visual", "config": config_dict(cfg),
        "static_groups": {"frames": F, "windows": [wh, ww], "run_frames": tg, "shot_frames": shot_len, "groups": G,
                          "queries_per_group": [int(nq.min()), int(nq.max())], "keys_per_group": [int(nk.min()), int(nk.max())]},
        "ms": ms, "ms_total": sum(ms.values()), "ms_single_call": float(np.mean(one)),
        "st_attn_TFLOP/s": fl_st / ms["st_attn"] / 1e9, "frame_attn_TFLOP/s": fl_fr / ms["frame_attn"] / 1e9,
        "st_gather_GB/s": 2.0 * row * (N + 2 * Tkv) / ms["st_gather"] / 1e6,
        "mean3_GB/s": 4.0 * row * N / ms["mean3"] / 1e6, "hbm_peak_GB/s": peaks["hbm_gbs"],
        "useful_tflop": {"st": fl_st / 1e12, "frame": fl_fr / 1e12}}))
    return 0


class _LazyRows:
    """Host view of a large device X that materialises only the indexed token rows."""

    def __init__(self, X):
        self.X = X
        self.shape = tuple(X.shape)

    def __getitem__(self, idx):
        b, tok = idx
        assert b == slice(None)
        return self.X[:, torch.from_numpy(np.asarray(tok)).to(self.X.device)].float().cpu().numpy()


def run_e2e(mb, cfg, sh, inp, ws, O, flops, args):
    """Same step through moga_forward_host: inputs in pinned host memory, O returned to pinned
    host memory, every host<->device copy inside the timed region (chunked by heads so that
    copies and kernels overlap)."""
    names = ["X", "Q", "K", "V"]
    hc = max(1, (cfg.H + 7) // 8)
    try:
        host = {n: torch.empty(inp[n].shape, dtype=inp[n].dtype, pin_memory=True) for n in names}
        host_O = torch.empty(O.shape, dtype=O.dtype, pin_memory=True)
    except RuntimeError as e:   # not enough lockable host memory on this machine
        return {"value": None, "unit": "TFLOP/s", "error": f"pinned allocation failed: {e}"[:200]}
    for n in names:
        host[n].copy_(inp[n])
    host_Wr = inp["Wr"].cpu().pin_memory()
    host_bias = None if inp["bias"] is None else inp["bias"].cpu().pin_memory()
    arena = mb.alloc_workspace(mb.moga_forward_host_bytes(sh, hc), O.device)
    h2d = sum(host[n].numel() * host[n].element_size() for n in names) + host_Wr.numel() * 4
    d2h = host_O.numel() * host_O.element_size()
    steps = max(1, min(args.steps, 3))

    def step():
        mb.moga_forward_host(sh, host["X"], host_Wr, host_bias, host["Q"], host["K"], host["V"], host_O, arena, hc)

    step()
    mb.moga_forward(sh, inp["X"], inp["Wr"], inp["bias"], inp["Q"], inp["K"], inp["V"], O, ws)
    torch.cuda.synchronize()
    same = bool(torch.equal(host_O[:, :1].to(O.device), O[:, :1]))     # head 0 against moga_forward on device inputs
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    code, _ = mb.moga_last_device_status(arena)
    return {"value": flops / (ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms, "steps": steps,
            "api": "moga_forward_host", "heads_per_chunk": hc, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "host_link_GB/s": (h2d + d2h) / ms / 1e6,
            "matches_device_run": same, "device_status": code}


if __name__ == "__main__":
    sys.exit(main())
