#!/usr/bin/env python
"""Benchmark of the LAWCAT layer forward (prefill) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

One step = one pass of the whole layer forward (conv -> mix -> phi -> normalized GLA) over one batch of seeded
synthetic input through the C ABI (`lawcat_layer_fwd`). Prints ONE JSON line (rank 0). N > 1 runs N independent
replicas (the layer has no inter-GPU exchange); the time is the max over ranks.

`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_18467_b200 import inputs as I  # noqa: E402

METRIC = "prefill tokens/sec per LAWCAT layer"
UNIT = "tokens/s"
LAYER_NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["source"] = "measured"
        return d
    return dict(FALLBACK_PEAKS, source="fallback")


def alg_bytes_per_token(s: I.LayerShape) -> int:
    """Algorithmic HBM bytes per token of the fused layer: q, k, v, gate read once, o written once."""
    es = 2 if s.dtype == "bf16" else 4
    return es * (s.H * s.d_k + s.H_kv * s.d_k + s.H_kv * s.d_v + s.H * s.gd + s.H * s.d_v)


def alg_flops_per_token(s: I.LayerShape) -> float:
    """Algorithmic flops per token (recurrent minimum; chunk overhead not credited)."""
    G = s.H // s.H_kv
    return s.H * (4.0 * s.d_k * s.d_k + 4.0 * s.d_k * (s.d_v + 1) + 2.0 * s.conv_k * s.d_k * (1 + 1.0 / G))


# Per-kernel algorithmic bytes per token (what that kernel alone has to move), for the roofline of the dominant kernel.
def kernel_bytes_per_token(name: str, s: I.LayerShape) -> float:
    es = 2 if s.dtype == "bf16" else 4
    if name == "gla_fwd_rec":    # fp32 scratch qdot, kdot in; v, gate in; o out
        return 4 * 2 * s.H * s.d_k + es * (s.H_kv * s.d_v + s.H * s.gd + s.H * s.d_v)
    if name == "convmix_fwd":    # q, k in; fp32 qdot, kdot out
        return es * (s.H * s.d_k + s.H_kv * s.d_k) + 4 * 2 * s.H * s.d_k
    return alg_bytes_per_token(s)  # fused tensor-core kernels: the whole layer's traffic


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.th.start()
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.th.join(timeout=2)
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(s: I.LayerShape, x: dict, tokens: int):
    """Time the fp64 oracle, as it stands, on the first `tokens` tokens of the workload. Returns (seconds, outputs)."""
    from oracle import lawcat_oracle as O
    Ts = min(tokens, s.T)
    p = O.OracleParams(s.B, Ts, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, gate_tau=s.gate_tau)
    args = [x[n][:, :Ts] if n in ("q", "k", "v", "gate") else x[n] for n in LAYER_NAMES]
    O.threads()  # build / load outside the timed region
    t0 = time.perf_counter()
    r = O.layer_fwd(p, *args)
    return time.perf_counter() - t0, r, Ts, O.threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    s = I.CONFIGS[args.workload]
    sample = min(s.T, args.ref_tokens)
    x = I.make(dataclasses.replace(s, T=sample), LAYER_NAMES)
    s_small = dataclasses.replace(s, T=sample)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(s_small, x, sample)
    t, cores = 0.0, 1
    for _ in range(args.steps):
        dt, _, _, cores = oracle_sample(s_small, x, sample)
        t += dt
    value = s.B * sample * args.steps / t
    desc = f"a {sample}-token sequence of the workload's shape per step (T={s.T} in full), all {s.H} heads"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
        "config": {"workload": s.name, "B": s.B, "T": s.T, "H": s.H, "H_kv": s.H_kv, "d_k": s.d_k, "d_v": s.d_v,
                   "gate_dim": s.gd, "sample_tokens_per_step": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def dist_setup(backend: str, device=None):
    """(world, rank, local rank) from the launcher's environment; joins the process group when world > 1. The replicas
    exchange nothing on the data path: the group only serves the barrier and the max over ranks of the timed region."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        kw = {"device_id": device} if device is not None else {}
        dist.init_process_group(backend, **kw)
    return world, rank, local


def max_over_ranks(x: float, world: int, device) -> float:
    """The slowest rank's value (every rank gets it)."""
    if world <= 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64 if str(device) == "cpu" else torch.float32, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: int, steps: int, world: int, ms: float) -> float:
    """Units per second of the whole job: every rank processes units_per_rank per step (weak scaling)."""
    return world * units_per_rank * steps / (ms / 1e3)


def run_ours(args):
    import torch
    from paper_2509_18467_b200 import api

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    world, rank, local = dist_setup("nccl", dev)
    if world > 1:
        import torch.distributed as dist
    api.lib()

    s = I.CONFIGS[args.workload]
    if args.gate_dim:
        s = dataclasses.replace(s, gate_dim=args.gate_dim)
    x = I.make(s, LAYER_NAMES)
    d = {n: api.to_device(x[n], s.dtype, dev) for n in LAYER_NAMES}
    p = api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                   gate_tau=s.gate_tau, chunk=args.chunk)
    o = torch.empty(s.B, s.T, s.H, s.d_v, dtype=api.torch_dtype(p), device=dev)
    nws = api.workspace_bytes(p, api.OP_LAYER_FWD)
    ws = torch.empty(max(nws, 16), dtype=torch.uint8, device=dev)
    ins = [d[n] for n in LAYER_NAMES]

    def step():
        api.lawcat_layer_fwd(p, *ins, o=o, want_state=False, want_cache=False, ws=ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    n0 = api.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = api.launch_count() - n0
    # keep the GPU busy a little longer so that short runs still collect clock samples under load
    t_end = time.time() + max(0.0, 0.6 - ms / 1e3)
    while time.time() < t_end:
        step()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(ms, world, dev)
    tokens = s.B * s.T
    value = whole_job_value(tokens, args.steps, world, ms)

    # per-kernel device time over the same K steps (CUDA events on the launch stream, bracketing each kernel)
    api.trace_begin()
    for _ in range(args.steps):
        step()
    tr = api.trace_end()
    pk = peaks()
    dom = max(tr, key=lambda k: tr[k][1])
    n_l, tot_ms = tr[dom]
    launches_per_step = n_l / args.steps
    dom_ms = tot_ms / n_l
    kb = kernel_bytes_per_token(dom, s) * tokens / launches_per_step
    achieved = kb / (dom_ms / 1e3) / 1e9
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tpath):
        with open(tpath) as f:
            traffic = json.load(f).get(f"{dom}:{s.name}")
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / pk["hbm_gbs"], "traffic": traffic, "peak_source": f"of {pk['source']}",
                "kernel_ms": dom_ms, "kernel_share": tot_ms / sum(v[1] for v in tr.values()),
                "kernels_ms_per_step": {k: v[1] / args.steps for k, v in tr.items()}}
    # whole-layer roofline: slower of bytes at HBM bandwidth and flops at bf16 tensor peak
    t_hbm = alg_bytes_per_token(s) * tokens / (pk["hbm_gbs"] * 1e9)
    t_tc = alg_flops_per_token(s) * tokens / (pk["bf16_tflops"] * 1e12)
    layer = {"roofline_ms": 1e3 * max(t_hbm, t_tc), "bound": "hbm" if t_hbm >= t_tc else "tensor",
             "frac": max(t_hbm, t_tc) / (ms / 1e3 / args.steps), "alg_bytes_per_token": alg_bytes_per_token(s),
             "alg_flops_per_token": alg_flops_per_token(s)}

    # end to end through the C ABI with HOST buffers: pinned host -> device copies, the layer, o back to the host
    tdt = api.torch_dtype(p)
    hp = {n: torch.from_numpy(x[n]).to(tdt).pin_memory() for n in LAYER_NAMES}
    h_o = torch.empty(s.B, s.T, s.H, s.d_v, dtype=tdt).pin_memory()
    arena = torch.empty(api.host_arena_bytes(p), dtype=torch.uint8, device=dev)
    e2e_steps = max(1, min(args.steps, 5))
    api.lawcat_layer_fwd_host(p, *[hp[n] for n in LAYER_NAMES], h_o, arena)
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        api.lawcat_layer_fwd_host(p, *[hp[n] for n in LAYER_NAMES], h_o, arena)
    e1.record()
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev)
    h2d = sum(hp[n].numel() * hp[n].element_size() for n in LAYER_NAMES)
    e2e = {"value": whole_job_value(tokens, e2e_steps, world, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": h_o.numel() * h_o.element_size(), "steps": e2e_steps}
    same = bool(torch.equal(h_o.to(dev), o))

    cpu = None
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu:
        dt, ref, Ts, cores = oracle_sample(s, x, args.cpu_tokens)
        from paper_2509_18467_b200.metrics import err_bf16, err_f32
        got = o[:, :Ts].float().cpu().numpy()
        if s.dtype == "bf16":
            strict, comp = err_bf16(got, ref["o"])
            parity = {"tokens_checked": Ts, "err_rms_norm": comp, "err_rms_norm_incl_store_rounding": strict,
                      "tol": 1e-2}
        else:
            parity = {"tokens_checked": Ts, "err_rel": err_f32(got, ref["o"]), "tol": 1e-4}
        cpu = {"value": s.B * Ts / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {Ts} of {s.T} tokens, all {s.H} heads, one pass ({dt:.1f} s)"}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if s.dtype == "bf16" else "f32", "data": "synthetic (seeded)",
            "config": {"workload": s.name, "B": s.B, "T": s.T, "H": s.H, "H_kv": s.H_kv, "d_k": s.d_k, "d_v": s.d_v,
                       "conv_k": s.conv_k, "gate_dim": s.gd, "gate_tau": s.gate_tau, "chunk": args.chunk, "replicas": world,
                       "l2": "inputs larger than L2 (no flush)" if alg_bytes_per_token(s) * tokens > 126e6
                       else "inputs fit in L2"},
            "clocks": clocks, "e2e": e2e, "e2e_matches_device_path": same, "gpu_launches": launches,
            "roofline": roofline, "layer_roofline": layer, "cpu_baseline": cpu, "parity": parity}))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3"])
    ap.add_argument("--gate-dim", type=int, default=0, help="override the gate width (1 = one decay per head)")
    ap.add_argument("--chunk", type=int, default=0, choices=[0, 1, 64],
                    help="0: the library chooses (tensor-core kernel where it applies); 1: the exact recurrent path")
    ap.add_argument("--cpu-tokens", type=int, default=16384, help="tokens of the workload the CPU oracle is timed on")
    ap.add_argument("--ref-tokens", type=int, default=2048, help="tokens per step of the reference arm")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
