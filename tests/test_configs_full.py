"""The benchmark configurations other than the headline one, at their full sizes, through the C ABI against the oracle:
c2 (Llama-3.2-1B shape prefill, T = 8192), c4 (distillation step: forward and backward at B = 8, T = 1024) and the c5
decode step (B = 64 sequences, 32 x 128 x 128 fp32 state each, conv caches of width 4). The oracle checks every output
where it finishes in seconds, and a sampled prefix where it does not."""
import dataclasses

import numpy as np
import pytest

from helpers import check, oracle_params
from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I

pytestmark = pytest.mark.gpu

NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]


@pytest.fixture(scope="module")
def api():
    import torch
    from paper_2509_18467_b200 import api as A
    assert torch.cuda.is_available()
    A.lib()
    return A


def P(api, s, **kw):
    return api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                      gate_tau=s.gate_tau, **kw)


def test_c2_llama_shape_prefill(api):
    import torch
    s = I.CONFIGS["c2"]
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    r = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in NAMES])
    torch.cuda.synchronize()
    Ts = 2048  # the oracle checks every output of the first 2048 tokens of all 32 heads ...
    ref = O.layer_fwd(oracle_params(dataclasses.replace(s, T=Ts)), *[x[n][:, :Ts] for n in NAMES[:4]],
                      *[x[n] for n in NAMES[4:]])
    check(r["o"][:, :Ts], ref["o"], "bf16", "o[:2048]")
    # ... and the tail through the state: a second call over the last quarter, started from the state and caches of a
    # call over the first three quarters, must reproduce the tail of the single call
    cut = 3 * s.T // 4
    part = lambda lo, hi: [d[n][:, lo:hi].contiguous() for n in NAMES[:4]] + [d[n] for n in NAMES[4:]]
    r1 = api.lawcat_layer_fwd(P(api, dataclasses.replace(s, T=cut)), *part(0, cut))
    r2 = api.lawcat_layer_fwd(P(api, dataclasses.replace(s, T=s.T - cut)), *part(cut, s.T), r1["cache_q"], r1["cache_k"],
                              r1["S_T"], r1["z_T"])
    check(r2["o"], r["o"][:, cut:].double().cpu().numpy(), "bf16", "tail o")
    check(r2["S_T"], r["S_T"].double().cpu().numpy(), "bf16", "S_T", f32_store=True)


def test_c4_distillation_step_forward_and_backward(api):
    """conv_fwd -> gla_fwd -> gla_bwd -> conv_bwd at B = 8, T = 1024, 32/8 heads, d = 64, bf16, against the oracle's
    whole-layer gradients for an upstream gradient ~ N(0,1)."""
    import torch
    s = I.CONFIGS["c4"]
    x = I.make(s, NAMES + ["dO"])
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    p = P(api, s)
    qd, kd = api.lawcat_conv_fwd(p, d["q"], d["k"], d["w_q"], d["w_k"], d["W"])
    f = api.lawcat_gla_fwd(p, qd, kd, d["v"], d["gate"])
    g = api.lawcat_gla_bwd(p, qd, kd, d["v"], d["gate"], f["o"], f["den"], d["dO"])
    c = api.lawcat_conv_bwd(p, d["q"], d["k"], d["w_q"], d["w_k"], d["W"], g["d_qdot"], g["d_kdot"])
    torch.cuda.synchronize()
    op = oracle_params(s)
    ref_f = O.layer_fwd(op, *[x[n] for n in NAMES])
    check(qd, ref_f["qdot"], "bf16", "qdot")
    check(kd, ref_f["kdot"], "bf16", "kdot")
    # each call against the oracle on the inputs that call was given: the stored (bf16-rounded) features for the attention
    qd_h, kd_h = qd.float().cpu().numpy(), kd.float().cpu().numpy()
    check(f["o"], O.gla_fwd(op, qd_h, kd_h, x["v"], x["gate"])["o"], "bf16", "o")
    ref_g = O.gla_bwd(op, qd_h, kd_h, x["v"], x["gate"], x["dO"], None, None)
    for name in ("d_qdot", "d_kdot", "dv", "dgate"):
        check(g[name], ref_g[name], "bf16", name)
    ref_c = O.conv_bwd(op, x["q"], x["k"], x["w_q"], x["w_k"], x["W"], g["d_qdot"].float().cpu().numpy(),
                       g["d_kdot"].float().cpu().numpy(), None, None)
    check(c["dq"], ref_c["dq"], "bf16", "dq")
    check(c["dk"], ref_c["dk"], "bf16", "dk")
    check(c["dw_q"], ref_c["dw_q"], "bf16", "dw_q", f32_store=True)
    check(c["dw_k"], ref_c["dw_k"], "bf16", "dw_k", f32_store=True)
    check(c["dW"], ref_c["dW"], "bf16", "dW", f32_store=True)


def test_c5_decode_step_full_size(api):
    """One decode step for B = 64 sequences on the Mistral shape; the carried state and caches come from a seeded
    256-token prefill of the same layer (computed by the oracle), so the denominators are well conditioned."""
    import torch
    s = I.CONFIGS["c5-decode"]
    pre = dataclasses.replace(s, T=256, config_id=51)
    xp = I.make(pre, NAMES)
    refp = O.layer_fwd(oracle_params(pre), *[xp[n] for n in NAMES])
    xt = I.make(dataclasses.replace(s, T=1, config_id=52), NAMES[:4])
    tok = {n: xt[n][:, 0] for n in NAMES[:4]}
    d = {n: api.to_device(np.ascontiguousarray(v), s.dtype) for n, v in tok.items()}
    w = {n: api.to_device(xp[n], s.dtype) for n in NAMES[4:]}
    S = torch.from_numpy(refp["S_T"].astype(np.float32)).cuda()
    z = torch.from_numpy(refp["z_T"].astype(np.float32)).cuda()
    cq = api.to_device(refp["cache_q"].astype(np.float32), s.dtype)
    ck = api.to_device(refp["cache_k"].astype(np.float32), s.dtype)
    o = api.lawcat_decode_step(P(api, s), d["q"], d["k"], d["v"], d["gate"], w["w_q"], w["w_k"], w["W"], S, z, cq, ck)
    torch.cuda.synchronize()
    ref = O.decode_step(oracle_params(dataclasses.replace(s, T=1)), tok["q"], tok["k"], tok["v"], tok["gate"], xp["w_q"],
                        xp["w_k"], xp["W"], refp["S_T"].astype(np.float32).astype(np.float64),
                        refp["z_T"].astype(np.float32).astype(np.float64), refp["cache_q"], refp["cache_k"])
    check(o, ref["o"], "bf16", "o_t")
    check(S, ref["S"], "bf16", "S", f32_store=True)
    check(z, ref["z"], "bf16", "z", f32_store=True)
    assert np.array_equal(cq.float().cpu().numpy(), ref["cache_q"].astype(np.float32))
