"""Parity of the chunkwise tensor-core attention kernels on given features (lawcat_gla_fwd / lawcat_gla_bwd, bf16,
d_k = d_v = 64) with the fp64 oracle, through the C ABI: outputs, denominators, final state, and every gradient, at lengths
around the chunk size (64 tokens), with ragged tails, carried states, grouped heads, one decay per head, sharper gates,
the log-decay gate mode, eps, and the numerator-only form. Tolerance: 1e-2 of the RMS of each tensor (helpers.check)."""
import numpy as np
import pytest

from helpers import check, oracle_params
from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I
from test_gpu_parity import gla_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    import torch
    from paper_2509_18467_b200 import api as A
    assert torch.cuda.is_available()
    A.lib()
    return A


def shape(B, T, H, Hkv, cid, **kw):
    return I.LayerShape(B, T, H, Hkv, 64, 64, dtype="bf16", config_id=cid, **kw)


def P(api, s, **kw):
    return api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                      gate_tau=s.gate_tau, **kw)


def run(api, s, with_state, backward=True, gate_mode=0, **pkw):
    x = gla_inputs(s, with_state, seed_offset=5)
    if gate_mode == 1:
        x["gate"] = -np.abs(x["gate"]) * np.float32(0.125)
    d = {k: (None if v is None else api.to_device(v, "f32" if k in ("S0", "z0") else s.dtype)) for k, v in x.items()}
    p = P(api, s, gate_mode=gate_mode, **pkw)
    op = oracle_params(s, gate_mode=gate_mode, **pkw)
    api.trace_begin()
    f = api.lawcat_gla_fwd(p, d["qdot"], d["kdot"], d["v"], d["gate"], d["S0"], d["z0"])
    kernels = api.trace_end()
    # (sharp sigmoid gates, tau < 8, and calls of fewer than 16 tokens are served by the exact recurrence: see the header)
    tc = (gate_mode == 1 or s.gate_tau >= 8.0) and s.T >= 16
    assert ("gla_tc_fwd" in kernels) == tc, kernels
    ref = O.gla_fwd(op, x["qdot"], x["kdot"], x["v"], x["gate"], x["S0"], x["z0"])
    check(f["o"], ref["o"], "bf16", "o")
    check(f["den"], ref["den"], "bf16", "den", f32_store=True)
    check(f["S_T"], ref["S_T"], "bf16", "S_T", f32_store=True)
    check(f["z_T"], ref["z_T"], "bf16", "z_T", f32_store=True)
    if not backward:
        return
    api.trace_begin()
    g = api.lawcat_gla_bwd(p, d["qdot"], d["kdot"], d["v"], d["gate"], f["o"], f["den"], d["dO"], d["S0"], d["z0"])
    kernels = api.trace_end()
    assert ("gla_tc_bwd" in kernels) == tc, kernels
    rg = O.gla_bwd(op, x["qdot"], x["kdot"], x["v"], x["gate"], x["dO"], x["S0"], x["z0"])
    for name in ("d_qdot", "d_kdot", "dv", "dgate"):
        if s.T == 1 and not with_state and name != "dv":
            # a single token without a past returns its own value (o_1 = v_1): these gradients are zero in theory, and
            # there is no RMS to normalize by; the bound is absolute, against gradients of order one elsewhere
            assert float(g[name].float().abs().max()) <= 1e-3 and float(np.abs(rg[name]).max()) <= 1e-9, name
            continue
        check(g[name], rg[name], "bf16", name)


@pytest.mark.parametrize("T", [1, 2, 5, 15, 16, 17, 63, 64, 65, 127, 128, 129, 200])
@pytest.mark.parametrize("with_state", [False, True])
def test_lengths_around_the_chunk_size(api, T, with_state):
    run(api, shape(2, T, 4, 2, 61), with_state)


@pytest.mark.parametrize("H,Hkv", [(2, 2), (4, 1), (8, 2)])
def test_head_grouping(api, H, Hkv):
    run(api, shape(1, 300, H, Hkv, 62), True)


@pytest.mark.parametrize("tau", [1.0, 4.0, 8.0, 16.0, 64.0])
def test_gate_sharpness(api, tau):
    run(api, shape(1, 260, 2, 1, 63, gate_tau=tau), False)


@pytest.mark.parametrize("T,with_state", [(64, False), (300, True), (1223, True)])
def test_one_decay_per_head(api, T, with_state):
    run(api, shape(1, T, 4, 2, 64, gate_dim=1), with_state)


@pytest.mark.parametrize("T", [1162, 1300])
def test_distillation_lengths(api, T):
    run(api, shape(1, T, 4, 2, 65), False)


def test_log_decay_gate_mode(api):
    run(api, shape(1, 200, 2, 1, 66), True, gate_mode=1)


def test_eps_and_numerator_only(api):
    run(api, shape(1, 150, 2, 1, 67), False, eps=0.5)
    run(api, shape(1, 150, 2, 1, 68), True, normalize=0)


@pytest.mark.parametrize("phi,T,with_state", [(1, 65, False), (1, 300, True), (1, 1223, True), (2, 200, False)])
def test_layer_forward_with_the_elementwise_feature_maps(api, phi, T, with_state):
    """The feature maps of Section 2 other than the softmax, phi = 1 + ELU (and the identity, with a positive mix so that
    the features stay positive), through lawcat_layer_fwd on head width 64: tensor-core conv + mix + phi, then the
    chunkwise tensor-core attention on fp32 features."""
    names = ["q", "k", "v", "gate", "w_q", "w_k", "W"]
    s = shape(2, T, 4, 2, 69)
    extra = ["S0", "z0", "cache_q", "cache_k"] if with_state else []
    x = I.make(s, names + extra)
    if phi == 2:  # identity: keep the features (hence the denominators) positive
        for n in ("q", "k", "w_q", "w_k", "W") + (("cache_q", "cache_k") if with_state else ()):
            x[n] = I.round_to_bf16(np.abs(x[n]))
    d = {n: api.to_device(v, "f32" if n in ("S0", "z0") else "bf16") for n, v in x.items()}
    api.trace_begin()
    r = api.lawcat_layer_fwd(P(api, s, phi=phi), *[d[n] for n in names], d.get("cache_q"), d.get("cache_k"), d.get("S0"),
                             d.get("z0"))
    kernels = api.trace_end()
    assert "convmix_tc_fwd" in kernels and "gla_tc_fwd" in kernels, kernels
    ref = O.layer_fwd(oracle_params(s, phi=phi), *[x[n] for n in names], x.get("cache_q"), x.get("cache_k"), x.get("S0"),
                      x.get("z0"))
    check(r["o"], ref["o"], "bf16", "o")
    check(r["S_T"], ref["S_T"], "bf16", "S_T", f32_store=True)
    check(r["z_T"], ref["z_T"], "bf16", "z_T", f32_store=True)
