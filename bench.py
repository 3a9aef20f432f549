#!/usr/bin/env python
"""Benchmark of the LAWCAT layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

Workloads (seeded synthetic inputs of `paper_2509_18467_b200.inputs`, through the C ABI):
  c1, c2, c3, c5-T<N>   prefill: one step = one `lawcat_layer_fwd` (conv -> mix -> phi -> normalized GLA) over one batch,
                        returning the state and the conv caches a caller needs to continue; c3 is the headline
                        (Mistral-7B layer shape, T = 32768); c5-T<N> is the same shape at T = N
  c4                    distillation step: `lawcat_layer_fwd` (the output the loss needs) + `lawcat_layer_bwd` (every gradient of
                        the layer for a seeded upstream gradient) at B = 8, T = 1024
  c5-decode             one recurrent `lawcat_decode_step` for B = 64 sequences
  c3-gate-fn            the gate function in front of the c3 layer: one `lawcat_gate_fn_fwd` (hidden states of width 4096 ->
                        rank 32 -> 4096 gate logits per token) over the 32768 tokens
  c5-decode-gate-fn     the same gate function for the one new token of each of the B = 64 sequences of c5-decode
Prints ONE JSON line (rank 0). N > 1 runs N independent replicas (the layer has no inter-GPU exchange), one process per
GPU; the time is the max over ranks. Started without a launcher, `--gpus N` starts the N ranks itself.

`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_18467_b200 import inputs as I  # noqa: E402

UNIT = "tokens/s"
LAYER_NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
SWEEP_T = (1024, 4096, 16384, 65536, 131072)
WORKLOADS = ["c1", "c2", "c3", "c4", "c5-decode"] + [f"c5-T{t}" for t in SWEEP_T] + ["c3-gate-fn", "c5-decode-gate-fn"]
# the gate function in front of the headline layer: hidden width of the 7B model, the rank the paper settles on
GATE_FN = {"d_model": 4096, "rank": 32}


def workload_shape(name: str) -> I.LayerShape:
    if name.startswith("c5-T"):
        T = int(name[4:])
        return dataclasses.replace(I.CONFIGS["c3"], T=T, config_id=5, name=f"c5-mistral-7b-T{T}")
    if name == "c3-gate-fn":
        return dataclasses.replace(I.CONFIGS["c3"], name="c3-gate-fn-mistral-7b-T32768")
    if name == "c5-decode-gate-fn":
        return dataclasses.replace(I.CONFIGS["c5-decode"], name="c5-decode-gate-fn-mistral-7b-B64")
    return I.CONFIGS[name]


def workload_kind(name: str) -> str:
    return {"c4": "train", "c5-decode": "decode", "c3-gate-fn": "gatefn", "c5-decode-gate-fn": "gatefn"}.get(name, "prefill")


def metric_name(kind: str) -> str:
    return {"prefill": "prefill tokens/sec per LAWCAT layer",
            "train": "training tokens/sec per LAWCAT layer (forward + backward)",
            "decode": "decode tokens/sec per LAWCAT layer (one token per sequence and step)",
            "gatefn": "gate-function tokens/sec per LAWCAT layer (hidden states -> gate logits)"}[kind]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["source"] = "measured"
        return d
    return dict(FALLBACK_PEAKS, source="fallback")


# ---- algorithmic bytes and flops per step (what the method must move and compute; nothing a kernel design adds) ----------
def es(s: I.LayerShape) -> int:
    return 2 if s.dtype == "bf16" else 4


def io_bytes_per_token(s: I.LayerShape) -> dict:
    e = es(s)
    return {"q": e * s.H * s.d_k, "k": e * s.H_kv * s.d_k, "v": e * s.H_kv * s.d_v, "gate": e * s.H * s.gd,
            "o": e * s.H * s.d_v}


def alg_bytes_per_step(kind: str, s: I.LayerShape) -> float:
    b = io_bytes_per_token(s)
    fwd = b["q"] + b["k"] + b["v"] + b["gate"] + b["o"]
    if kind == "gatefn":    # hidden states read once, logits written once, the two weight matrices and the bias once
        dm, r, n_out = GATE_FN["d_model"], GATE_FN["rank"], s.H * s.gd
        return (es(s) * dm + b["gate"]) * s.B * s.T + es(s) * (r * dm + n_out * r + n_out)
    if kind == "prefill":   # q, k, v, gate read once, o written once
        return fwd * s.B * s.T
    if kind == "train":     # forward; backward: the inputs and dO read once, dq, dk, dv, dgate written once
        bwd = b["q"] + b["k"] + b["v"] + b["gate"] + b["o"] + b["q"] + b["k"] + b["v"] + b["gate"]
        return (fwd + bwd) * s.B * s.T
    # decode: the fp32 state [S | z] of every (sequence, head) read and written, W once, the token's tensors
    return 4 * s.B * s.H * 2 * (s.d_k * s.d_v + s.d_k) + es(s) * s.H * s.d_k * s.d_k + fwd * s.B


def alg_flops_per_step(kind: str, s: I.LayerShape) -> float:
    """Recurrent minimum (chunk overhead not credited): mix on both streams, state update + read-out, conv."""
    if kind == "gatefn":
        return 2.0 * GATE_FN["rank"] * (GATE_FN["d_model"] + s.H * s.gd) * s.B * s.T
    G = s.H // s.H_kv
    per_tok = s.H * (4.0 * s.d_k * s.d_k + 4.0 * s.d_k * (s.d_v + 1) + 2.0 * s.conv_k * s.d_k * (1 + 1.0 / G))
    tokens = s.B * (1 if kind == "decode" else s.T)
    return per_tok * tokens * (3.0 if kind == "train" else 1.0)


def kernel_bytes_per_step(name: str, kind: str, s: I.LayerShape) -> float:
    """Algorithmic bytes of ONE launch of kernel `name`: what that kernel's own interface has to move."""
    b, tok = io_bytes_per_token(s), s.B * s.T
    f32_feat = 4 * 2 * s.H * s.d_k            # qdot and kdot in fp32
    f32_dv = 4 * s.H * s.d_v                  # dv per query head in fp32 (before the group reduce)
    table = {
        "gla_fwd_rec": (f32_feat if kind == "prefill" else 2 * b["q"]) + b["v"] + b["gate"] + b["o"],
        "convmix_fwd": b["q"] + b["k"] + (f32_feat if kind == "prefill" else 2 * b["q"]),
        "convmix_tc_fwd": b["q"] + b["k"] + f32_feat,
        # chunkwise backward inside layer_bwd: fp32 features in, fp32 feature gradients out, v, gate, dO in, dgate out,
        # dv per query head out
        "gla_tc_bwd": 2 * f32_feat + b["v"] + b["gate"] + b["o"] + b["gate"] + f32_dv,
        "gla_tc_fwd": f32_feat + b["v"] + b["gate"] + b["o"],
        "gla_tc_bwd_sweep": f32_feat + b["v"] + b["gate"] + b["o"],   # features, v, gate, dO in
        "dv_reduce": f32_dv + b["v"],
        # raw q, k and the fp32 feature gradients in, fp32 du out (dW is negligible)
        "convmix_tc_bwd": b["q"] + b["k"] + f32_feat + 4 * (s.H + s.H_kv) * s.d_k,
        "conv_bwd": 4 * (s.H + s.H_kv) * s.d_k + 2 * (b["q"] + b["k"]),
    }
    if name in ("decode_state", "decode_features"):
        return alg_bytes_per_step("decode", s)
    if name in table:
        return table[name] * tok
    if name.startswith("gla_bwd") or name in ("convmix_bwd", "dv_group_reduce"):
        return alg_bytes_per_step("train", s) / 2  # the backward half of the step
    return alg_bytes_per_step(kind, s)              # fused kernels: the whole step's traffic


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


# ---- the CPU oracle, as it stands, on a bounded sample of the workload ------------------------------------------------------
def oracle_params_of(s: I.LayerShape, **kw):
    from oracle import lawcat_oracle as O
    return O.OracleParams(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim,
                          gate_tau=s.gate_tau, **kw)


def oracle_sample(kind: str, s: I.LayerShape, x: dict, tokens: int):
    """Time the fp64 oracle on a sample of the workload. Returns (seconds, results, units processed, cores, description).
    prefill: the first `tokens` tokens of every sequence and head; train: forward and backward of the first sequences
    that hold `tokens` tokens; decode: the step of every sequence."""
    from oracle import lawcat_oracle as O
    O.threads()  # build / load outside the timed region
    if kind == "gatefn":
        Ts = min(tokens, s.T)
        t0 = time.perf_counter()
        a = O.gate_logits(x["x"][:, :Ts], x["A1"], x["A2"], x["bias"])
        dt = time.perf_counter() - t0
        return dt, dict(gate=a.reshape(s.B, Ts, s.H, s.gd)), s.B * Ts, 1, f"first {Ts} of {s.T} tokens, one pass ({dt:.1f} s)"
    if kind == "prefill":
        Ts = min(tokens, s.T)
        p = oracle_params_of(dataclasses.replace(s, T=Ts))
        args = [x[n][:, :Ts] if n in LAYER_NAMES[:4] else x[n] for n in LAYER_NAMES]
        t0 = time.perf_counter()
        r = O.layer_fwd(p, *args)
        dt = time.perf_counter() - t0
        return dt, r, s.B * Ts, O.threads(), f"first {Ts} of {s.T} tokens, all {s.H} heads, one pass ({dt:.1f} s)"
    if kind == "train":
        Bs = max(1, min(s.B, tokens // s.T))
        sb = dataclasses.replace(s, B=Bs)
        p = oracle_params_of(sb)
        args = [x[n][:Bs] if n in LAYER_NAMES[:4] else x[n] for n in LAYER_NAMES]
        t0 = time.perf_counter()
        f = O.layer_fwd(p, *args)
        g1 = O.gla_bwd(p, f["qdot"], f["kdot"], args[2], args[3], x["dO"][:Bs])
        g2 = O.conv_bwd(p, args[0], args[1], x["w_q"], x["w_k"], x["W"], g1["d_qdot"], g1["d_kdot"])
        dt = time.perf_counter() - t0
        r = dict(o=f["o"], dv=g1["dv"], dgate=g1["dgate"], **g2)
        return dt, r, Bs * s.T, O.threads(), (f"forward + backward of the first {Bs} of {s.B} sequences "
                                              f"(T = {s.T}), all heads ({dt:.1f} s)")
    p = oracle_params_of(dataclasses.replace(s, T=1))
    t0 = time.perf_counter()
    r = O.decode_step(p, x["q"][:, 0], x["k"][:, 0], x["v"][:, 0], x["gate"][:, 0], x["w_q"], x["w_k"], x["W"],
                      x["S"], x["z"], x["cache_q"], x["cache_k"])
    dt = time.perf_counter() - t0
    return dt, r, s.B, O.threads(), f"one step of all {s.B} sequences ({dt:.2f} s)"


def make_inputs(kind: str, s: I.LayerShape) -> dict:
    """Seeded host tensors of the workload. The decode workload carries the state and the conv caches of a seeded
    stand-in prefill: S0, z0 and caches drawn by the same generator (positive states, as positive features produce)."""
    if kind == "prefill":
        return I.make(s, LAYER_NAMES)
    if kind == "gatefn":
        return I.make_gate_fn(s, GATE_FN["d_model"], GATE_FN["rank"])
    if kind == "train":
        return I.make(s, LAYER_NAMES + ["dO"])
    x = I.make(dataclasses.replace(s, T=1), LAYER_NAMES + ["S0", "z0", "cache_q", "cache_k"])
    x["S"], x["z"] = x.pop("S0") * np.float32(0.1), x.pop("z0") + np.float32(1.0)
    return x


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    kind = workload_kind(args.workload)
    s = workload_shape(args.workload)
    sample = args.ref_tokens
    if kind in ("prefill", "gatefn"):
        s_small = dataclasses.replace(s, T=min(s.T, sample))
    elif kind == "train":
        s_small = dataclasses.replace(s, B=max(1, min(s.B, sample // s.T)))
    else:
        s_small = s
    x = make_inputs(kind, s_small)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(kind, s_small, x, sample)
    t, units, cores, desc = 0.0, 0, 1, ""
    for _ in range(args.steps):
        dt, _, n, cores, desc = oracle_sample(kind, s_small, x, sample)
        t += dt
        units += n
    value = units / t
    print(json.dumps({
        "impl": "reference", "metric": metric_name(kind), "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded)",
        "config": {"workload": s.name, "B": s.B, "T": s.T, "H": s.H, "H_kv": s.H_kv, "d_k": s.d_k, "d_v": s.d_v,
                   "gate_dim": s.gd, "sample_per_step": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ---- rank plumbing -------------------------------------------------------------------------------------------------------
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


def replica_launch_plan(gpus: int, env: dict):
    """What `--gpus N` means for this process: 'run' (the launcher's world matches, or one GPU), 'spawn' (no launcher:
    start the N ranks), or an error string (a launcher whose world size contradicts --gpus)."""
    if "WORLD_SIZE" in env:
        world = int(env["WORLD_SIZE"])
        if world != gpus:
            return f"--gpus {gpus} contradicts the launcher's WORLD_SIZE={world}"
        return "run"
    return "run" if gpus <= 1 else "spawn"


def spawn_replicas(gpus: int):
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.call(cmd))


# ---- the GPU arm -----------------------------------------------------------------------------------------------------------
class Runner:
    """One workload staged on one GPU: `step()` enqueues one pass of the hot path on resident inputs, `e2e_step()` the same
    from pinned host buffers with the copies inside, `outputs()` what the parity leg compares."""

    def __init__(self, kind, s, x, dev, chunk):
        import torch
        from paper_2509_18467_b200 import api
        self.kind, self.s, self.x, self.dev, self.api, self.torch = kind, s, x, dev, api, torch
        self.p = api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                            gate_tau=s.gate_tau, chunk=chunk)
        self.tdt = api.torch_dtype(self.p)
        f32 = ("S", "z")
        self.d = {n: api.to_device(np.ascontiguousarray(v[:, 0]) if kind == "decode" and n in LAYER_NAMES[:4] else v,
                                   "f32" if n in f32 else s.dtype, dev) for n, v in x.items()}
        d, p = self.d, self.p
        if kind == "prefill":
            self.o = torch.empty(s.B, s.T, s.H, s.d_v, dtype=self.tdt, device=dev)
            self.ws = torch.empty(max(api.workspace_bytes(p, api.OP_LAYER_FWD), 16), dtype=torch.uint8, device=dev)
        elif kind == "gatefn":
            self.o = torch.empty(s.B, s.T, s.H, s.gd, dtype=self.tdt, device=dev)
        elif kind == "train":
            self.o = torch.empty(s.B, s.T, s.H, s.d_v, dtype=self.tdt, device=dev)
            self.ws = torch.empty(max(api.workspace_bytes(p, api.OP_LAYER_FWD), 16), dtype=torch.uint8, device=dev)
            self.ws_b = torch.empty(max(api.workspace_bytes(p, api.OP_LAYER_BWD), 16), dtype=torch.uint8, device=dev)
        else:
            self.ws = torch.empty(max(api.workspace_bytes(p, api.OP_DECODE_STEP), 16), dtype=torch.uint8, device=dev)
            self.o = torch.empty(s.B, s.H, s.d_v, dtype=self.tdt, device=dev)
            self.state0 = {n: d[n].clone() for n in ("S", "z", "cache_q", "cache_k")}
        self.res = None

    def step(self):
        api, d, p = self.api, self.d, self.p
        if self.kind == "prefill":   # the state and the caches are part of what a prefill hands back
            self.res = api.lawcat_layer_fwd(p, *[d[n] for n in LAYER_NAMES], o=self.o, ws=self.ws)
        elif self.kind == "gatefn":
            api.lawcat_gate_fn_fwd(p, GATE_FN["d_model"], GATE_FN["rank"], d["x"], d["A1"], d["A2"], d["bias"], gate=self.o)
        elif self.kind == "train":
            api.lawcat_layer_fwd(p, *[d[n] for n in LAYER_NAMES], o=self.o, want_state=False, want_cache=False, ws=self.ws)
            g = api.lawcat_layer_bwd(p, *[d[n] for n in LAYER_NAMES], d["dO"], ws=self.ws_b)
            self.res = dict(o=self.o, **g)
        else:
            api.lawcat_decode_step(p, d["q"], d["k"], d["v"], d["gate"], d["w_q"], d["w_k"], d["W"], d["S"], d["z"],
                                   d["cache_q"], d["cache_k"], o_t=self.o, ws=self.ws)

    def reset(self):
        if self.kind == "decode":   # the step advances the state in place: start the parity leg from the seeded state
            for n, v in self.state0.items():
                self.d[n].copy_(v)

    # -- end to end: inputs start in pinned host memory, results end there
    def e2e_setup(self):
        torch, api, s = self.torch, self.api, self.s
        # what arrives with every step: the whole batch for prefill and training; for decode the token's tensors (the
        # state and the conv caches live on the device and are advanced in place)
        names = {"prefill": LAYER_NAMES, "train": LAYER_NAMES[:4] + ["dO"], "decode": LAYER_NAMES[:4],
                 "gatefn": ["x"]}[self.kind]
        self.h = {n: (self.d[n].cpu().pin_memory()) for n in names}
        if self.kind == "prefill":
            self.h_o = torch.empty(s.B, s.T, s.H, s.d_v, dtype=self.tdt).pin_memory()
            self.arena = torch.empty(api.host_arena_bytes(self.p), dtype=torch.uint8, device=self.dev)
            self.h2d = sum(t.numel() * t.element_size() for t in self.h.values())
            self.d2h = self.h_o.numel() * self.h_o.element_size()
        elif self.kind == "train":
            self.h2d = sum(t.numel() * t.element_size() for t in self.h.values())
            self.h_out = None
        else:
            self.h2d = sum(t.numel() * t.element_size() for t in self.h.values())
            self.h_out = None

    def e2e_step(self):
        torch, api = self.torch, self.api
        if self.kind == "prefill":
            api.lawcat_layer_fwd_host(self.p, *[self.h[n] for n in LAYER_NAMES], self.h_o, self.arena)
            return
        for n, t in self.h.items():
            self.d[n].copy_(t, non_blocking=True)
        self.step()
        outs = self.res if self.kind == "train" else dict(o=self.o)
        if self.h_out is None:
            self.h_out = {n: torch.empty(t.shape, dtype=t.dtype).pin_memory() for n, t in outs.items() if t is not None}
            self.d2h = sum(t.numel() * t.element_size() for t in self.h_out.values())
        for n, t in self.h_out.items():
            t.copy_(outs[n], non_blocking=True)


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

    kind = workload_kind(args.workload)
    s = workload_shape(args.workload)
    if args.gate_dim:
        s = dataclasses.replace(s, gate_dim=args.gate_dim)
    x = make_inputs(kind, s)
    R = Runner(kind, s, x, dev, args.chunk)
    units = s.B * (1 if kind == "decode" else s.T)
    alg_bytes = alg_bytes_per_step(kind, s)
    flush = alg_bytes < 126e6 * 1.5   # inputs that (nearly) fit the 126 MB L2: write a larger buffer between steps
    scratch = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if flush else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_steps(fn, n):
        """Device time of n steps (CUDA events on the launch stream). With an L2 flush between steps each step is
        bracketed by its own pair of events and the flush stays outside."""
        if not flush:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b in ev:
            scratch.fill_(1)
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev)

    for _ in range(args.warmup):
        R.step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    n0 = api.launch_count()
    barrier()
    ms = timed_steps(R.step, args.steps)
    barrier()
    launches = api.launch_count() - n0
    # keep the GPU busy a little longer so that short runs still collect clock samples under load
    t_end = time.time() + max(0.0, 0.6 - ms / 1e3)
    while time.time() < t_end:
        R.step()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    ms = max_over_ranks(ms, world, dev)
    value = whole_job_value(units, args.steps, world, ms)

    # per-kernel device time over the same K steps (CUDA events on the launch stream, bracketing each kernel)
    api.trace_begin()
    for _ in range(args.steps):
        if flush:
            scratch.fill_(1)
        R.step()
    tr = api.trace_end()
    pk = peaks()
    dom = max(tr, key=lambda k: tr[k][1])
    n_l, tot_ms = tr[dom]
    dom_ms = tot_ms / n_l
    kb = kernel_bytes_per_step(dom, kind, s) / (n_l / args.steps)
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
    # whole-step roofline: slower of bytes at HBM bandwidth and flops at bf16 tensor peak
    t_hbm = alg_bytes / (pk["hbm_gbs"] * 1e9)
    t_tc = alg_flops_per_step(kind, s) / (pk["bf16_tflops"] * 1e12)
    layer = {"roofline_ms": 1e3 * max(t_hbm, t_tc), "bound": "hbm" if t_hbm >= t_tc else "tensor",
             "frac": max(t_hbm, t_tc) / (ms / 1e3 / args.steps), "alg_bytes_per_step": alg_bytes,
             "alg_flops_per_step": alg_flops_per_step(kind, s)}

    # end to end through the public API with HOST buffers: pinned host -> device copies, the step, results back
    R.e2e_setup()
    e2e_steps = max(1, min(args.steps, 5))
    R.e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        R.e2e_step()
    e1.record()
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev)
    e2e = {"value": whole_job_value(units, e2e_steps, world, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": R.h2d,
           "d2h_bytes_per_step": R.d2h, "steps": e2e_steps}

    cpu = None
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu:
        from paper_2509_18467_b200.metrics import err_bf16, err_f32
        R.reset()
        R.step()
        torch.cuda.synchronize()
        dt, ref, n_units, cores, desc = oracle_sample(kind, s, x, args.cpu_tokens)

        def err(got, want, f32_store=False):
            got = got.float().cpu().numpy()[tuple(slice(0, n) for n in want.shape)]
            if s.dtype != "bf16":
                return err_f32(got, want)
            strict, comp = err_bf16(got, want)
            return strict if f32_store else comp
        if kind == "prefill":
            errs = {"o": err(R.o, ref["o"])}
        elif kind == "gatefn":
            errs = {"gate": err(R.o, ref["gate"])}
        elif kind == "train":
            # the oracle differentiates the whole layer from the raw inputs
            errs = {n: err(R.res[n], ref[n], n in ("dw_q", "dw_k", "dW")) for n in ("o", "dq", "dk", "dv", "dgate",
                                                                                  "dw_q", "dw_k", "dW")
                    if n not in ("dw_q", "dw_k", "dW") or n_units == units}
        else:
            errs = {"o": err(R.o, ref["o"]), "S": err(R.d["S"], ref["S"], True), "z": err(R.d["z"], ref["z"], True)}
        parity = {"units_checked": n_units, "err_rms_norm": errs, "tol": 1e-2 if s.dtype == "bf16" else 1e-4}
        cpu = {"value": n_units / dt, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

    if rank == 0:
        print(json.dumps({
            "metric": metric_name(kind), "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if s.dtype == "bf16" else "f32", "data": "synthetic (seeded)",
            "config": {"workload": s.name, "B": s.B, "T": s.T, "H": s.H, "H_kv": s.H_kv, "d_k": s.d_k, "d_v": s.d_v,
                       "conv_k": s.conv_k, "gate_dim": s.gd, "gate_tau": s.gate_tau, "chunk": args.chunk, "replicas": world,
                       "returns": "o, S_T, z_T, conv caches" if kind == "prefill" else None,
                       "l2": "L2 flushed between steps (256 MB write, outside the timed events)" if flush
                       else "inputs larger than L2 (no flush)"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "roofline": roofline, "layer_roofline": layer, "cpu_baseline": cpu, "parity": parity}))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=WORKLOADS)
    ap.add_argument("--gate-dim", type=int, default=0, help="override the gate width (1 = one decay per head)")
    ap.add_argument("--chunk", type=int, default=0, choices=[0, 1, 64],
                    help="0: the library chooses (tensor-core kernel where it applies); 1: the exact recurrent path")
    ap.add_argument("--cpu-tokens", type=int, default=16384, help="tokens of the workload the CPU oracle is timed on")
    ap.add_argument("--ref-tokens", type=int, default=2048, help="tokens per step of the reference arm")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    plan = replica_launch_plan(args.gpus, os.environ)
    if plan == "spawn":
        spawn_replicas(args.gpus)
    elif plan != "run":
        sys.exit("bench.py: " + plan)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
