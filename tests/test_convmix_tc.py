"""Parity of the tensor-core conv -> mix -> softmax kernels (lawcat_conv_fwd with W, bf16, head width 64 or 128) and of the
tensor-core backward through mix and softmax (lawcat_conv_bwd, head width 64) with the fp64 oracle, through the C ABI:
tile boundaries (128 tokens), ragged tails, conv caches, conv widths 1-4, grouped heads."""
import numpy as np
import pytest

from helpers import check
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


def P(api, s, **kw):
    return api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                      gate_tau=s.gate_tau, **kw)


def features(s, x):
    uq = O.conv(x["q"], x["w_q"], x.get("cache_q"), s.conv_k)
    uk = O.conv(x["k"], x["w_k"], x.get("cache_k"), s.conv_k)
    return O.mix_phi(uq, x["W"], s.H, 0), O.mix_phi(uk, x["W"], s.H, 0)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("T,with_cache", [(1, False), (5, True), (127, False), (128, True), (129, False), (300, True)])
def test_forward_lengths_around_the_tile(api, d, T, with_cache):
    s = I.LayerShape(2, T, 4, 2, d, d, dtype="bf16", config_id=71)
    x = I.make(s, ["q", "k", "w_q", "w_k", "W"] + (["cache_q", "cache_k"] if with_cache else []))
    dv = {n: api.to_device(v, "bf16") for n, v in x.items()}
    api.trace_begin()
    qd, kd = api.lawcat_conv_fwd(P(api, s), dv["q"], dv["k"], dv["w_q"], dv["w_k"], dv["W"], dv.get("cache_q"),
                                 dv.get("cache_k"))
    assert "convmix_tc_fwd" in api.trace_end()
    rq, rk = features(s, x)
    check(qd, rq, "bf16", "qdot")
    check(kd, rk, "bf16", "kdot")


@pytest.mark.parametrize("H,Hkv,conv_k", [(2, 2, 4), (4, 1, 3), (8, 2, 2), (3, 3, 1)])
def test_forward_grouping_and_conv_widths(api, H, Hkv, conv_k):
    s = I.LayerShape(1, 200, H, Hkv, 64, 64, dtype="bf16", conv_k=conv_k, config_id=72)
    x = I.make(s, ["q", "k", "w_q", "w_k", "W"] + (["cache_q", "cache_k"] if conv_k > 1 else []))
    dv = {n: api.to_device(v, "bf16") for n, v in x.items()}
    qd, kd = api.lawcat_conv_fwd(P(api, s), dv["q"], dv["k"], dv["w_q"], dv["w_k"], dv["W"], dv.get("cache_q"),
                                 dv.get("cache_k"))
    rq, rk = features(s, x)
    check(qd, rq, "bf16", "qdot")
    check(kd, rk, "bf16", "kdot")


@pytest.mark.parametrize("T,H,Hkv,conv_k,with_cache", [(1, 2, 1, 4, False), (127, 4, 2, 4, True), (128, 4, 1, 3, False),
                                                       (129, 2, 2, 2, True), (300, 8, 2, 4, True), (77, 3, 3, 1, False)])
def test_backward(api, T, H, Hkv, conv_k, with_cache):
    s = I.LayerShape(2, T, H, Hkv, 64, 64, dtype="bf16", conv_k=conv_k, config_id=73)
    names = ["q", "k", "w_q", "w_k", "W", "d_qdot", "d_kdot"] + (["cache_q", "cache_k"] if with_cache and conv_k > 1 else [])
    x = I.make(s, names)
    dv = {n: api.to_device(v, "bf16") for n, v in x.items()}
    api.trace_begin()
    g = api.lawcat_conv_bwd(P(api, s), dv["q"], dv["k"], dv["w_q"], dv["w_k"], dv["W"], dv["d_qdot"], dv["d_kdot"],
                            dv.get("cache_q"), dv.get("cache_k"))
    assert "convmix_tc_bwd" in api.trace_end()
    op = O.OracleParams(s.B, s.T, s.H, s.H_kv, 64, 64, conv_k=conv_k)
    ref = O.conv_bwd(op, x["q"], x["k"], x["w_q"], x["w_k"], x["W"], x["d_qdot"], x["d_kdot"], x.get("cache_q"),
                     x.get("cache_k"))
    check(g["dq"], ref["dq"], "bf16", "dq")
    check(g["dk"], ref["dk"], "bf16", "dk")
    for n in ("dw_q", "dw_k", "dW"):
        check(g[n], ref[n], "bf16", n, f32_store=True)
