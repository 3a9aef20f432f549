"""GPU-vs-oracle parity of every C-ABI entry point, element by element on the same seeded inputs.

Sizes are small enough for the fp64 oracle to finish in seconds and still span several staging batches / tiles and a
ragged tail. fp32 mode: max relative error 1e-4; bf16 mode: 1e-2 of the output RMS (see helpers.py).
"""
import dataclasses

import numpy as np
import pytest

from helpers import check, oracle_params
from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    import torch
    from paper_2509_18467_b200 import api as A
    assert torch.cuda.is_available()
    A.lib()
    return A


def shape(B, T, H, Hkv, dk, dv, dtype, gate_dim=0, conv_k=4, tau=16.0, cid=7):
    return I.LayerShape(B, T, H, Hkv, dk, dv, conv_k=conv_k, gate_dim=gate_dim, dtype=dtype, gate_tau=tau,
                        config_id=cid)


def P(api, s, **kw):
    return api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                      gate_tau=s.gate_tau, **kw)


def dev(api, x, s):
    return {k: api.to_device(v, "f32" if k in ("S0", "z0") else s.dtype) for k, v in x.items()}


SHAPES = [
    shape(2, 77, 4, 2, 32, 16, "f32"),
    shape(1, 65, 2, 2, 16, 64, "f32", gate_dim=1),
    shape(1, 130, 4, 1, 64, 128, "f32", conv_k=3),
    shape(2, 77, 4, 2, 32, 16, "bf16"),
    shape(1, 200, 8, 2, 64, 64, "bf16", gate_dim=1),
    shape(1, 96, 2, 1, 128, 128, "bf16"),
    shape(1, 33, 2, 2, 128, 32, "f32", conv_k=1),
    shape(1, 40, 2, 1, 16, 16, "bf16", conv_k=8, tau=1.0),
]
IDS = [f"B{s.B}T{s.T}H{s.H}/{s.H_kv}d{s.d_k}x{s.d_v}g{s.gd}K{s.conv_k}{s.dtype}" for s in SHAPES]


# ------------------------------------------------------------------------------------------------ conv (+ mix + phi)
@pytest.mark.parametrize("s", SHAPES, ids=IDS)
@pytest.mark.parametrize("with_cache", [False, True])
def test_conv_fwd_plain(api, s, with_cache):
    x = I.make(s, ["q", "k", "w_q", "w_k"] + (["cache_q", "cache_k"] if with_cache and s.conv_k > 1 else []))
    d = dev(api, x, s)
    qd, kd = api.lawcat_conv_fwd(P(api, s), d["q"], d["k"], d["w_q"], d["w_k"], None, d.get("cache_q"),
                                 d.get("cache_k"))
    check(qd, O.conv(x["q"], x["w_q"], x.get("cache_q"), s.conv_k), s.dtype, "conv(q)")
    check(kd, O.conv(x["k"], x["w_k"], x.get("cache_k"), s.conv_k), s.dtype, "conv(k)")


@pytest.mark.parametrize("s", SHAPES, ids=IDS)
@pytest.mark.parametrize("phi", [0, 1, 2])
def test_conv_fwd_mix_phi(api, s, phi):
    names = ["q", "k", "w_q", "w_k", "W"] + (["cache_q", "cache_k"] if s.conv_k > 1 else [])
    x = I.make(s, names)
    d = dev(api, x, s)
    qd, kd = api.lawcat_conv_fwd(P(api, s, phi=phi), d["q"], d["k"], d["w_q"], d["w_k"], d["W"], d.get("cache_q"),
                                 d.get("cache_k"))
    uq = O.conv(x["q"], x["w_q"], x.get("cache_q"), s.conv_k)
    uk = O.conv(x["k"], x["w_k"], x.get("cache_k"), s.conv_k)
    check(qd, O.mix_phi(uq, x["W"], s.H, phi), s.dtype, "qdot")
    check(kd, O.mix_phi(uk, x["W"], s.H, phi), s.dtype, "kdot")


@pytest.mark.parametrize("s", SHAPES, ids=IDS)
@pytest.mark.parametrize("phi,with_mix", [(0, True), (1, True), (2, True), (0, False)])
def test_conv_bwd(api, s, phi, with_mix):
    names = ["q", "k", "w_q", "w_k", "W", "d_qdot", "d_kdot"] + (["cache_q", "cache_k"] if s.conv_k > 1 else [])
    x = I.make(s, names)
    if not with_mix:
        x["d_kdot"] = x["d_kdot"][:, :, : s.H_kv].copy()
        x["W"] = None
    d = {k: (None if v is None else api.to_device(v, s.dtype)) for k, v in x.items()}
    g = api.lawcat_conv_bwd(P(api, s, phi=phi), d["q"], d["k"], d["w_q"], d["w_k"], d["W"], d["d_qdot"], d["d_kdot"],
                            d.get("cache_q"), d.get("cache_k"))
    ref = O.conv_bwd(oracle_params(s, phi=phi), x["q"], x["k"], x["w_q"], x["w_k"], x["W"], x["d_qdot"], x["d_kdot"],
                     x.get("cache_q"), x.get("cache_k"))
    check(g["dq"], ref["dq"], s.dtype, "dq")
    check(g["dk"], ref["dk"], s.dtype, "dk")
    check(g["dw_q"], ref["dw_q"], s.dtype, "dw_q", f32_store=True)
    check(g["dw_k"], ref["dw_k"], s.dtype, "dw_k", f32_store=True)
    if with_mix:
        check(g["dW"], ref["dW"], s.dtype, "dW", f32_store=True)
    else:
        assert g["dW"] is None


# ------------------------------------------------------------------------------------------------ GLA
def gla_inputs(s, with_state, seed_offset=0):
    """qdot, kdot positive like the outputs of a softmax feature map; bf16 mode rounds them to storage precision."""
    x = I.make(s, ["q", "k", "v", "gate", "dO"] + (["S0", "z0"] if with_state else []), seed_offset)
    kk = I.make(dataclasses.replace(s, H_kv=s.H), ["k"], seed_offset + 1)["k"]
    e = lambda a: np.exp(a - a.max(-1, keepdims=True)) / np.exp(a - a.max(-1, keepdims=True)).sum(-1, keepdims=True)
    qd, kd = e(x["q"].astype(np.float64)).astype(np.float32), e(kk.astype(np.float64)).astype(np.float32)
    if s.dtype == "bf16":
        qd, kd = I.round_to_bf16(qd), I.round_to_bf16(kd)
    return dict(qdot=qd, kdot=kd, v=x["v"], gate=x["gate"], dO=x["dO"], S0=x.get("S0"), z0=x.get("z0"))


@pytest.mark.parametrize("s", SHAPES, ids=IDS)
@pytest.mark.parametrize("with_state,gate_mode,normalize", [(False, 0, 1), (True, 0, 1), (True, 1, 1), (False, 0, 0)])
def test_gla_fwd(api, s, with_state, gate_mode, normalize):
    x = gla_inputs(s, with_state)
    if gate_mode == 1:
        x["gate"] = -np.abs(x["gate"]) * np.float32(0.125)   # log-decays, exactly representable scaling
    d = {k: (None if v is None else api.to_device(v, "f32" if k in ("S0", "z0") else s.dtype)) for k, v in x.items()}
    r = api.lawcat_gla_fwd(P(api, s, gate_mode=gate_mode, normalize=normalize), d["qdot"], d["kdot"], d["v"],
                           d["gate"], d["S0"], d["z0"])
    ref = O.gla_fwd(oracle_params(s, gate_mode=gate_mode, normalize=normalize), x["qdot"], x["kdot"], x["v"],
                    x["gate"], x["S0"], x["z0"])
    check(r["o"], ref["o"], s.dtype, "o")
    check(r["den"], ref["den"], s.dtype, "den", f32_store=True)
    check(r["S_T"], ref["S_T"], s.dtype, "S_T", f32_store=True)
    check(r["z_T"], ref["z_T"], s.dtype, "z_T", f32_store=True)


@pytest.mark.parametrize("s", SHAPES, ids=IDS)
@pytest.mark.parametrize("with_state,gate_mode,normalize", [(False, 0, 1), (True, 0, 1), (False, 1, 1), (False, 0, 0)])
def test_gla_bwd(api, s, with_state, gate_mode, normalize):
    x = gla_inputs(s, with_state, seed_offset=3)
    if gate_mode == 1:
        x["gate"] = -np.abs(x["gate"]) * np.float32(0.125)
    d = {k: (None if v is None else api.to_device(v, "f32" if k in ("S0", "z0") else s.dtype)) for k, v in x.items()}
    p = P(api, s, gate_mode=gate_mode, normalize=normalize)
    f = api.lawcat_gla_fwd(p, d["qdot"], d["kdot"], d["v"], d["gate"], d["S0"], d["z0"])
    g = api.lawcat_gla_bwd(p, d["qdot"], d["kdot"], d["v"], d["gate"], f["o"], f["den"], d["dO"], d["S0"], d["z0"])
    ref = O.gla_bwd(oracle_params(s, gate_mode=gate_mode, normalize=normalize), x["qdot"], x["kdot"], x["v"],
                    x["gate"], x["dO"], x["S0"], x["z0"])
    for name in ("d_qdot", "d_kdot", "dv", "dgate"):
        check(g[name], ref[name], s.dtype, name)


# ------------------------------------------------------------------------------------------------ whole layer
LAYER_NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]


@pytest.mark.parametrize("s", SHAPES, ids=IDS)
@pytest.mark.parametrize("with_state", [False, True])
def test_layer_fwd(api, s, with_state):
    extra = (["S0", "z0"] + (["cache_q", "cache_k"] if s.conv_k > 1 else [])) if with_state else []
    x = I.make(s, LAYER_NAMES + extra)
    d = dev(api, x, s)
    r = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in LAYER_NAMES], d.get("cache_q"), d.get("cache_k"),
                             d.get("S0"), d.get("z0"))
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in LAYER_NAMES], x.get("cache_q"), x.get("cache_k"),
                      x.get("S0"), x.get("z0"))
    check(r["o"], ref["o"], s.dtype, "o")
    check(r["S_T"], ref["S_T"], s.dtype, "S_T", f32_store=True)
    check(r["z_T"], ref["z_T"], s.dtype, "z_T", f32_store=True)
    if s.conv_k > 1:
        assert np.array_equal(r["cache_q"].float().cpu().numpy(), ref["cache_q"].astype(np.float32))
        assert np.array_equal(r["cache_k"].float().cpu().numpy(), ref["cache_k"].astype(np.float32))


@pytest.mark.parametrize("T", [1, 2, 3, 4, 5, 63, 65])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_layer_fwd_odd_lengths(api, T, dtype):
    s = shape(2, T, 4, 2, 32, 32, dtype, cid=8)
    x = I.make(s, LAYER_NAMES)
    d = dev(api, x, s)
    r = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in LAYER_NAMES])
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in LAYER_NAMES])
    check(r["o"], ref["o"], dtype, "o")
    assert np.array_equal(r["cache_q"].float().cpu().numpy(), ref["cache_q"].astype(np.float32))


def test_layer_fwd_empty_sequence(api):
    import torch
    s = shape(2, 0, 4, 2, 32, 32, "f32")
    x = I.make(dataclasses.replace(s, T=1), ["w_q", "w_k", "W", "S0", "z0", "cache_q", "cache_k"])
    d = dev(api, x, s)
    e = lambda *sh: torch.empty(*sh, device="cuda")
    r = api.lawcat_layer_fwd(P(api, s), e(2, 0, 4, 32), e(2, 0, 2, 32), e(2, 0, 2, 32), e(2, 0, 4, 32), d["w_q"],
                             d["w_k"], d["W"], d["cache_q"], d["cache_k"], d["S0"], d["z0"])
    assert r["o"].numel() == 0
    assert torch.equal(r["S_T"], d["S0"]) and torch.equal(r["z_T"], d["z0"])
    assert torch.equal(r["cache_q"], d["cache_q"]) and torch.equal(r["cache_k"], d["cache_k"])


def test_config_c1_fp32(api):
    """The fp32 parity configuration: B=1, T=512, H=4 (no GQA), d=64, conv width 4, gate = logsigmoid/16."""
    s = I.CONFIGS["c1"]
    x = I.make(s, LAYER_NAMES)
    d = dev(api, x, s)
    r = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in LAYER_NAMES])
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in LAYER_NAMES])
    e = check(r["o"], ref["o"], "f32", "o")
    print(f"c1 fp32 max relative error {e:.3e}")


@pytest.mark.parametrize("T", [1162, 1223, 1300])
def test_training_lengths_bf16(api, T):
    """Sequence lengths of the distillation runs (Section 5.1): not multiples of any tile or chunk."""
    s = shape(1, T, 4, 2, 64, 64, "bf16", cid=9)
    x = I.make(s, LAYER_NAMES)
    d = dev(api, x, s)
    r = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in LAYER_NAMES])
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in LAYER_NAMES])
    check(r["o"], ref["o"], "bf16", "o")


def test_split_prefill_equals_one_call(api):
    import torch
    s = shape(2, 150, 4, 2, 64, 64, "f32", cid=10)
    x = I.make(s, LAYER_NAMES)
    d = dev(api, x, s)
    full = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in LAYER_NAMES])
    cut = 70
    part = lambda lo, hi: [d[n][:, lo:hi].contiguous() for n in LAYER_NAMES[:4]] + [d[n] for n in LAYER_NAMES[4:]]
    s1, s2 = dataclasses.replace(s, T=cut), dataclasses.replace(s, T=s.T - cut)
    r1 = api.lawcat_layer_fwd(P(api, s1), *part(0, cut))
    r2 = api.lawcat_layer_fwd(P(api, s2), *part(cut, s.T), r1["cache_q"], r1["cache_k"], r1["S_T"], r1["z_T"])
    o = torch.cat([r1["o"], r2["o"]], 1)
    check(o, full["o"].double().cpu().numpy(), "f32", "split o")
    check(r2["S_T"], full["S_T"].double().cpu().numpy(), "f32", "split S_T")
    assert torch.equal(r2["cache_q"], full["cache_q"])


# ------------------------------------------------------------------------------------------------ decode
@pytest.mark.parametrize("s", [shape(3, 12, 4, 2, 32, 64, "f32"), shape(2, 10, 8, 2, 128, 128, "bf16"),
                               shape(2, 9, 4, 4, 64, 16, "bf16", gate_dim=1), shape(1, 6, 2, 1, 16, 32, "f32", conv_k=1),
                               shape(2, 5, 2, 1, 128, 128, "f32", conv_k=8), shape(9, 4, 4, 2, 64, 64, "bf16")],
                         ids=["f32-d32x64", "bf16-d128", "bf16-g1", "f32-K1", "f32-d128-K8", "bf16-d64-B9"])
def test_decode_steps_against_oracle(api, s):
    """T decode steps from a state and caches; every step's output, and the final state and caches, match the oracle."""
    import torch
    x = I.make(s, LAYER_NAMES + ["S0", "z0"] + (["cache_q", "cache_k"] if s.conv_k > 1 else []))
    d = dev(api, x, s)
    p = P(api, s)
    S, z = d["S0"].clone(), d["z0"].clone()
    cq = d["cache_q"].clone() if s.conv_k > 1 else None
    ck = d["cache_k"].clone() if s.conv_k > 1 else None
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in LAYER_NAMES], x.get("cache_q"), x.get("cache_k"), x["S0"],
                      x["z0"])
    outs = []
    for t in range(s.T):
        tok = [d[n][:, t].contiguous() for n in LAYER_NAMES[:4]]
        outs.append(api.lawcat_decode_step(p, *tok, d["w_q"], d["w_k"], d["W"], S, z, cq, ck))
    check(torch.stack(outs, 1), ref["o"], s.dtype, "decode o")
    check(S, ref["S_T"], s.dtype, "S", f32_store=True)
    check(z, ref["z_T"], s.dtype, "z", f32_store=True)
    if s.conv_k > 1:
        assert np.array_equal(cq.float().cpu().numpy(), ref["cache_q"].astype(np.float32))
        assert np.array_equal(ck.float().cpu().numpy(), ref["cache_k"].astype(np.float32))


@pytest.mark.parametrize("B,dk,dv,conv_k,gate_dim,kw", [
    (70, 128, 128, 4, 0, {}),                       # two groups of sequences, the second ragged
    (64, 64, 64, 2, 0, {"phi": 1}),                 # 1 + ELU, conv width 2
    (3, 128, 64, 1, 1, {"phi": 2}),                 # identity feature map, no conv, one decay per head
    (5, 64, 128, 3, 0, {"gate_mode": 1}),           # log-decay gates
    (2, 128, 128, 4, 0, {"eps": 0.3, "normalize": 1}),
    (2, 64, 64, 4, 0, {"normalize": 0}),
], ids=["B70-d128", "elu1-K2", "identity-K1-g1", "logdecay", "eps", "no-normalizer"])
def test_decode_steps_tensor_core_features(api, B, dk, dv, conv_k, gate_dim, kw):
    """bf16 decode with d_k = 64 / 128 computes the mix of a step's query and key vectors on the tensor cores: the
    variants of the feature map, gate and normalizer, and a batch that spans two groups of 64 sequences."""
    import torch
    s = shape(B, 4, 4, 2, dk, dv, "bf16", gate_dim=gate_dim, conv_k=conv_k, cid=12)
    names = LAYER_NAMES + ["S0", "z0"] + (["cache_q", "cache_k"] if conv_k > 1 else [])
    x = I.make(s, names)
    if kw.get("gate_mode") == 1:
        x["gate"] = I.round_to_bf16(-np.abs(x["gate"]) * 0.1)
    if kw.get("phi") == 2:  # the identity map needs positive features for a positive denominator
        for n in ("q", "k", "w_q", "w_k", "W"):
            x[n] = np.abs(x[n])
    d = dev(api, x, s)
    p = P(api, s, **kw)
    S, z = d["S0"].clone(), d["z0"].clone()
    cq = d["cache_q"].clone() if conv_k > 1 else None
    ck = d["cache_k"].clone() if conv_k > 1 else None
    ref = O.layer_fwd(oracle_params(s, **kw), *[x[n] for n in LAYER_NAMES], x.get("cache_q"), x.get("cache_k"),
                      x["S0"], x["z0"])
    outs = []
    for t in range(s.T):
        tok = [d[n][:, t].contiguous() for n in LAYER_NAMES[:4]]
        outs.append(api.lawcat_decode_step(p, *tok, d["w_q"], d["w_k"], d["W"], S, z, cq, ck))
    check(torch.stack(outs, 1), ref["o"], "bf16", "decode o")
    check(S, ref["S_T"], "bf16", "S", f32_store=True)
    check(z, ref["z_T"], "bf16", "z", f32_store=True)
