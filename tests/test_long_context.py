"""The long-context sweep (Mistral-7B layer shape, T = 32768 = the headline configuration, 65536 and 131072) in the launch
configuration the benchmark times, against the oracle on a stated subset of heads over ALL tokens: query heads
{0, 7, 13, 31} (key/value heads {0, 1, 3, 7}), every output of every token, and the final state. The oracle runs those
four heads as a four-head layer of its own (the heads of the layer do not interact)."""
import numpy as np
import pytest

from helpers import check
from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I

pytestmark = pytest.mark.gpu

NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]
HEADS = [0, 7, 13, 31]


@pytest.mark.parametrize("T", [32768, 65536, 131072])
def test_all_tokens_of_four_heads(T):
    import dataclasses
    import torch
    from paper_2509_18467_b200 import api
    s = dataclasses.replace(I.CONFIGS["c3"], T=T, config_id=5 if T != 32768 else 3)
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    p = api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.trace_begin()
    r = api.lawcat_layer_fwd(p, *[d[n] for n in NAMES], dev_status=status)
    kernels = api.trace_end()
    assert "layer_tc" in kernels and "layer_tc_state" in kernels and int(status.item()) == 0
    G, dk = s.H // s.H_kv, s.d_k
    kv = [h // G for h in HEADS]
    rows = lambda w, heads: w.reshape(-1, dk, s.conv_k)[heads].reshape(-1, s.conv_k)
    sub = dict(q=x["q"][:, :, HEADS], k=x["k"][:, :, kv], v=x["v"][:, :, kv], gate=x["gate"][:, :, HEADS],
               w_q=rows(x["w_q"], HEADS), w_k=rows(x["w_k"], kv), W=x["W"][HEADS])
    op = O.OracleParams(1, T, len(HEADS), len(HEADS), dk, s.d_v)
    ref = O.layer_fwd(op, *[np.ascontiguousarray(sub[n]) for n in NAMES])
    check(r["o"][:, :, HEADS], ref["o"], "bf16", f"o of heads {HEADS}, all {T} tokens")
    check(r["S_T"][:, HEADS], ref["S_T"], "bf16", "S_T", f32_store=True)
    check(r["z_T"][:, HEADS], ref["z_T"], "bf16", "z_T", f32_store=True)
