"""Times every benchmark configuration of the layer on one GPU and prints one JSON line per configuration.

    python -m paper_2509_18467_b200.sweep [--iters 20] [--only c2,c3,...]

Configurations: the prefill shapes c2 (Llama-3.2-1B, T = 8192) and c3 (Mistral-7B, T = 32768); the Mistral-shape prefill
sweep T in {1024, 4096, 16384, 65536, 131072}; c3 with one decay per head (gate_dim = 1); the distillation step c4
(conv_fwd -> gla_fwd -> gla_bwd -> conv_bwd at B = 8, T = 1024); the decode step at B = 64.

Inputs are seeded synthetic tensors of the recipe of `inputs.py` drawn on the device (q, k, v, gate logits ~ N(0,1), W ~
N(0, 1/d_k), conv taps ~ N(0, 1/K)): this script only times; parity of the same configurations is the test suite's
business. Each figure is the median of `iters` launches timed with CUDA events after 3 warm-up launches; inputs
smaller than the 126 MB L2 are followed by an L2 flush (a 256 MB write) between launches. The roofline of a configuration
is its algorithmic HBM bytes (inputs read once, outputs written once) at the measured copy bandwidth.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys

import torch

from . import api, inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def hbm_peak_gbs() -> tuple[float, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def draw(s: I.LayerShape, seed: int) -> dict:
    g = torch.Generator(device="cuda").manual_seed(seed)
    dt = torch.bfloat16 if s.dtype == "bf16" else torch.float32
    n = lambda *shape, std=1.0: (torch.randn(*shape, generator=g, device="cuda") * std).to(dt)
    return {"q": n(s.B, s.T, s.H, s.d_k), "k": n(s.B, s.T, s.H_kv, s.d_k), "v": n(s.B, s.T, s.H_kv, s.d_v),
            "gate": n(s.B, s.T, s.H, s.gd), "w_q": n(s.H * s.d_k, s.conv_k, std=s.conv_k ** -0.5),
            "w_k": n(s.H_kv * s.d_k, s.conv_k, std=s.conv_k ** -0.5), "W": n(s.H, s.d_k, s.d_k, std=s.d_k ** -0.5)}


def timed(fn, iters: int, flush: bool, batch: int = 1) -> float:
    """Median device time of one call. `batch` > 1 (only without a flush) puts that many calls between the two events:
    for a step of tens of microseconds the time from the first event to the first launch (argument marshalling on the
    host) would otherwise be counted as device time."""
    scratch = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if flush else None
    for _ in range(3):
        fn()
    ms = []
    for _ in range(iters):
        if flush:
            scratch.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(batch):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1) / batch)
    return statistics.median(ms)


def P(s: I.LayerShape):
    return api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                      gate_tau=s.gate_tau)


def es(s):
    return 2 if s.dtype == "bf16" else 4


def prefill(name: str, s: I.LayerShape, iters: int) -> dict:
    d = draw(s, 1000 + s.T)
    p = P(s)
    o = torch.empty(s.B, s.T, s.H, s.d_v, dtype=d["q"].dtype, device="cuda")
    args = [d[n] for n in ("q", "k", "v", "gate", "w_q", "w_k", "W")]
    api.trace_begin()
    api.lawcat_layer_fwd(p, *args, o=o)
    kernels = sorted(api.trace_end())
    nbytes = es(s) * s.B * s.T * (s.H * s.d_k + s.H_kv * s.d_k + s.H_kv * s.d_v + s.H * s.gd + s.H * s.d_v)
    ms = timed(lambda: api.lawcat_layer_fwd(p, *args, o=o), iters, nbytes < (126 << 20))
    return {"config": name, "what": "prefill (lawcat_layer_fwd)", "ms": ms, "tokens_per_s": s.B * s.T / ms * 1e3,
            "alg_bytes": nbytes, "kernels": kernels}


def training(name: str, s: I.LayerShape, iters: int) -> dict:
    d = draw(s, 4000)
    dO = torch.randn(s.B, s.T, s.H, s.d_v, device="cuda").to(d["q"].dtype)
    p = P(s)

    def step():
        qd, kd = api.lawcat_conv_fwd(p, d["q"], d["k"], d["w_q"], d["w_k"], d["W"])
        f = api.lawcat_gla_fwd(p, qd, kd, d["v"], d["gate"])
        g = api.lawcat_gla_bwd(p, qd, kd, d["v"], d["gate"], f["o"], f["den"], dO)
        api.lawcat_conv_bwd(p, d["q"], d["k"], d["w_q"], d["w_k"], d["W"], g["d_qdot"], g["d_kdot"])

    api.trace_begin()
    step()
    kernels = sorted(api.trace_end())
    e, tok = es(s), s.B * s.T
    fwd = e * tok * (s.H * s.d_k + s.H_kv * s.d_k + s.H_kv * s.d_v + s.H * s.gd + s.H * s.d_v)
    # the chain materializes qdot, kdot (written once, read by gla_fwd, gla_bwd and conv_bwd) and den; the backward reads
    # the inputs again and dO, and writes dq, dk, dv, dgate
    inter = e * tok * 2 * s.H * s.d_k * 4 + 4 * tok * s.H * 2
    bwd = fwd + e * tok * (s.H * s.d_v + 2 * s.H * s.d_k * 2 + s.H * s.d_k + s.H_kv * s.d_k + s.H_kv * s.d_v + s.H * s.gd)
    nbytes = fwd + inter + bwd
    ms = timed(step, iters, True)
    return {"config": name, "what": "forward + backward (conv_fwd, gla_fwd, gla_bwd, conv_bwd)", "ms": ms,
            "tokens_per_s": tok / ms * 1e3, "alg_bytes": nbytes, "kernels": kernels}


def decode(name: str, s: I.LayerShape, iters: int) -> dict:
    d = draw(dataclasses.replace(s, T=1), 5000)
    tok = {n: d[n][:, 0].contiguous() for n in ("q", "k", "v", "gate")}
    S = torch.randn(s.B, s.H, s.d_k, s.d_v, device="cuda") * 0.1
    z = torch.rand(s.B, s.H, s.d_k, device="cuda") + 1.0
    cq = torch.randn(s.B, s.conv_k - 1, s.H * s.d_k, device="cuda").to(d["q"].dtype)
    ck = torch.randn(s.B, s.conv_k - 1, s.H_kv * s.d_k, device="cuda").to(d["q"].dtype)
    p = P(s)
    o = torch.empty(s.B, s.H, s.d_v, dtype=d["q"].dtype, device="cuda")
    fn = lambda: api.lawcat_decode_step(p, tok["q"], tok["k"], tok["v"], tok["gate"], d["w_q"], d["w_k"], d["W"], S, z,
                                        cq, ck, o_t=o)
    api.trace_begin()
    fn()
    kernels = sorted(api.trace_end())
    # the state is read and written once per step; everything else is small beside it
    nbytes = 4 * s.B * s.H * (2 * s.d_k * s.d_v + 2 * s.d_k) + es(s) * s.H * s.d_k * s.d_k
    ms = timed(fn, iters, False, batch=50)  # 0.27 GB of state: larger than L2, no flush needed
    return {"config": name, "what": "decode step (lawcat_decode_step)", "ms": ms, "tokens_per_s": s.B / ms * 1e3,
            "alg_bytes": nbytes, "kernels": kernels}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--only", default="")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        sys.exit("sweep: needs a GPU")
    api.lib()
    c3 = I.CONFIGS["c3"]
    jobs = [("c2", prefill, I.CONFIGS["c2"]), ("c3", prefill, c3),
            ("c3-gate_dim1", prefill, dataclasses.replace(c3, gate_dim=1))]
    jobs += [(f"c5-prefill-T{T}", prefill, dataclasses.replace(c3, T=T)) for T in (1024, 4096, 16384, 65536, 131072)]
    jobs += [("c4", training, I.CONFIGS["c4"]), ("c5-decode", decode, I.CONFIGS["c5-decode"])]
    only = set(filter(None, args.only.split(",")))
    peak, src = hbm_peak_gbs()
    for name, fn, s in jobs:
        if only and name not in only:
            continue
        r = fn(name, s, args.iters)
        r["achieved_gbs"] = r["alg_bytes"] / (r["ms"] * 1e-3) / 1e9
        r["roofline_ms"] = r["alg_bytes"] / (peak * 1e9) * 1e3
        r["frac_of_hbm_roofline"] = r["roofline_ms"] / r["ms"]
        r["peak_gbs"], r["peak_source"] = peak, f"of {src}"
        print(json.dumps(r), flush=True)
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
