"""Randomized parity of the layer forward and backward through the C ABI against the fp64 oracle: seeded draws over head
width, batch, length (1 ... 6000, ragged), head grouping, conv width, gate sharpness (tau = 1 ... 64), gate mode (sigmoid
logits / log-decays), gate width, carried state, normalizer on/off, eps.

Tolerance: 1e-2 of the RMS on every tensor (outputs, final state, every gradient; bf16-stored tensors with the half-ulp
store allowance of metrics.py). Every draw also checks the routing rule of the header (helpers.tc_routed): sharp sigmoid
gates (tau < 8) and calls of fewer than 16 tokens must be served by the exact recurrence, everything else in the drawn
set by the tensor-core kernels, with dev_status = 0. Log-decay gates too sharp for 16-bit operands with an 11-bit
mantissa must be REPORTED (LAWCAT_ERR_NUMERIC), not silently degraded: test_sharp_log_decays_are_reported."""
import random

import numpy as np
import pytest

from helpers import tc_routed
from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I
from paper_2509_18467_b200.metrics import err_bf16

pytestmark = pytest.mark.gpu

NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]
LENGTHS = [1, 2, 3, 5, 15, 16, 17, 63, 64, 65, 100, 127, 129, 257, 513, 777, 1000, 1162, 2100, 3333, 4500, 6000]


def rel(x, y):
    return float(np.abs(x - y).max()) / max(float(np.sqrt((y ** 2).mean())), 1e-30)


def forward_draws():
    rng = random.Random(11)
    out = []
    for it in range(96):
        d = rng.choice([64, 128]); Hkv = rng.choice([1, 2, 3]); G = rng.choice([1, 2, 4])
        B = rng.choice([1, 2, 3]); T = rng.choice(LENGTHS)
        K = rng.choice([1, 2, 3, 4]); tau = rng.choice([1.0, 2.0, 4.0, 8.0, 16.0, 64.0]); gd = rng.choice([0, 1])
        state = rng.random() < 0.5
        norm = rng.choice([1, 1, 0]); eps = rng.choice([0.0, 0.0, 0.3]); mode = rng.choice([0, 0, 1])
        scale = rng.choice([0.02, 0.1])  # log-decay gates: g = -|N(0,1)| * scale per token
        out.append((it, d, B, T, Hkv * G, Hkv, K, tau, gd, state, norm, eps, mode, scale))
    return out


@pytest.mark.parametrize("case", forward_draws(), ids=lambda c: f"draw{c[0]}-d{c[1]}-T{c[3]}-tau{c[7]:g}-m{c[12]}")
def test_random_forward(case):
    import torch
    from paper_2509_18467_b200 import api
    it, d, B, T, H, Hkv, K, tau, gd, state, norm, eps, mode, scale = case
    s = I.LayerShape(B, T, H, Hkv, d, d, dtype="bf16", config_id=1200 + it, conv_k=K, gate_tau=tau, gate_dim=gd)
    extra = (["S0", "z0"] + (["cache_q", "cache_k"] if K > 1 else [])) if state else []
    x = I.make(s, NAMES + extra)
    if mode == 1:
        x["gate"] = I.round_to_bf16(-np.abs(x["gate"]) * np.float32(scale))
    dv = {n: api.to_device(x[n], "f32" if n in ("S0", "z0") else "bf16") for n in x}
    kw = dict(conv_k=K, gate_tau=tau, gate_dim=s.gate_dim, normalize=norm, eps=eps, gate_mode=mode)
    p = api.params(B, T, H, Hkv, d, d, **kw)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.trace_begin()
    r = api.lawcat_layer_fwd(p, *[dv[n] for n in NAMES], dv.get("cache_q"), dv.get("cache_k"), dv.get("S0"), dv.get("z0"),
                             dev_status=status)
    kernels = api.trace_end()
    assert any(k.startswith("layer_tc") for k in kernels) == tc_routed(s, gate_mode=mode), kernels
    assert int(status.item()) == 0
    ref = O.layer_fwd(O.OracleParams(B, T, H, Hkv, d, d, **kw), *[x[n] for n in NAMES], x.get("cache_q"),
                      x.get("cache_k"), x.get("S0"), x.get("z0"))
    o = r["o"].float().cpu().numpy()
    assert np.isfinite(o).all()
    _, e_o = err_bf16(o, ref["o"])
    assert e_o <= 1e-2, f"o: {e_o:.3e}"
    e_S = rel(r["S_T"].cpu().numpy(), ref["S_T"])
    assert e_S <= 1e-2, f"S_T: {e_S:.3e}"
    e_z = rel(r["z_T"].cpu().numpy(), ref["z_T"])
    assert e_z <= 1e-2, f"z_T: {e_z:.3e}"


def backward_draws():
    rng = random.Random(12)
    out = []
    for it in range(40):
        Hkv = rng.choice([1, 2]); G = rng.choice([1, 2, 4])
        B = rng.choice([1, 2]); T = rng.choice([1, 2, 5, 16, 63, 64, 65, 129, 300, 777, 1162, 1300])
        K = rng.choice([1, 2, 4]); tau = rng.choice([8.0, 16.0, 64.0]); gd = rng.choice([0, 1])
        norm = rng.choice([1, 1, 0]); eps = rng.choice([0.0, 0.3])
        out.append((it, B, T, Hkv * G, Hkv, K, tau, gd, norm, eps))
    return out


@pytest.mark.parametrize("case", backward_draws(), ids=lambda c: f"draw{c[0]}-T{c[2]}-tau{c[6]:g}")
def test_random_backward(case):
    """lawcat_layer_bwd (head width 64: the tensor-core backward from 16 tokens on) from the raw inputs: every gradient."""
    import torch
    from paper_2509_18467_b200 import api
    it, B, T, H, Hkv, K, tau, gd, norm, eps = case
    d = 64
    s = I.LayerShape(B, T, H, Hkv, d, d, dtype="bf16", config_id=1700 + it, conv_k=K, gate_tau=tau, gate_dim=gd)
    x = I.make(s, NAMES + ["dO"])
    dv = {n: api.to_device(x[n], "bf16") for n in x}
    kw = dict(conv_k=K, gate_tau=tau, gate_dim=s.gate_dim, normalize=norm, eps=eps)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.trace_begin()
    g = api.lawcat_layer_bwd(api.params(B, T, H, Hkv, d, d, **kw), *[dv[n] for n in NAMES], dv["dO"], dev_status=status)
    kernels = api.trace_end()
    assert ("gla_tc_bwd" in kernels) == (T >= 16), kernels
    assert int(status.item()) == 0
    op = O.OracleParams(B, T, H, Hkv, d, d, **kw)
    fwd = O.layer_fwd(op, *[x[n] for n in NAMES])
    g1 = O.gla_bwd(op, fwd["qdot"], fwd["kdot"], x["v"], x["gate"], x["dO"])
    g2 = O.conv_bwd(op, x["q"], x["k"], x["w_q"], x["w_k"], x["W"], g1["d_qdot"], g1["d_kdot"])
    want = dict(dq=g2["dq"], dk=g2["dk"], dv=g1["dv"], dgate=g1["dgate"], dw_q=g2["dw_q"], dw_k=g2["dw_k"], dW=g2["dW"])
    for n, w in want.items():
        got = g[n].float().cpu().numpy()
        assert np.isfinite(got).all(), n
        if T == 1 and n != "dv":
            # one token without a past returns its own value (o_1 = v_1): these gradients are zero in exact arithmetic,
            # so there is no RMS to normalize by; the bound is absolute
            assert float(np.abs(got - w).max()) <= 1e-3, n
            continue
        e = rel(got, w) if n in ("dw_q", "dw_k", "dW") else err_bf16(got, w)[1]
        assert e <= 1e-2, f"{n}: {e:.3e}"


def test_sharp_log_decays_are_reported():
    """Log-decay gates are the caller's numbers. When they are so sharp that half a chunk's accumulated log2-decay leaves
    +-8, the affected chunks run on 8-bit-mantissa operands: the result is delivered, finite, and dev_status says
    LAWCAT_ERR_NUMERIC (6); the same inputs with chunk = 1 (exact recurrence) report nothing and meet the tolerance."""
    import torch
    from paper_2509_18467_b200 import api
    s = I.LayerShape(1, 1000, 4, 2, 128, 128, dtype="bf16", config_id=1999)
    x = I.make(s, NAMES)
    x["gate"] = I.round_to_bf16(-np.abs(x["gate"]) * np.float32(0.5))
    dv = {n: api.to_device(x[n], "bf16") for n in x}
    ref = O.layer_fwd(O.OracleParams(1, 1000, 4, 2, 128, 128, gate_mode=1), *[x[n] for n in NAMES])
    for chunk, want in ((0, 6), (1, 0)):
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        r = api.lawcat_layer_fwd(api.params(1, 1000, 4, 2, 128, 128, gate_mode=1, chunk=chunk), *[dv[n] for n in NAMES],
                                 dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == want
        o = r["o"].float().cpu().numpy()
        assert np.isfinite(o).all()
        if chunk == 1:
            assert err_bf16(o, ref["o"])[1] <= 1e-2
