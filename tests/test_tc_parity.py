"""Parity of the chunkwise tensor-core layer forward (bf16, d_k = d_v = 128) with the fp64 oracle, through the C ABI.

The kernel works in chunks of 64 tokens and (for long sequences) splits a sequence into segments handled by different
thread blocks; the cases below span one partial chunk, exact chunk multiples, ragged tails, several segments, carried
state and conv caches, GQA and no GQA, narrower convs, sharper gates, and the distillation lengths of Section 5.1.
Tolerance: 1e-2 of the output RMS (bf16 mode), see helpers.check.
"""
import dataclasses

import numpy as np
import pytest

from helpers import check, oracle_params, tc_routed
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


def shape(B, T, H, Hkv, cid, **kw):
    return I.LayerShape(B, T, H, Hkv, 128, 128, dtype="bf16", config_id=cid, **kw)


def P(api, s, **kw):
    return api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                      gate_tau=s.gate_tau, **kw)


def run_case(api, s, with_state, expect_tc=None, **pkw):
    """One call of lawcat_layer_fwd against the oracle; expect_tc: whether the tensor-core layer kernel must have run
    (default: what the routing rule of the header says for this shape)."""
    import torch
    if expect_tc is None:
        expect_tc = tc_routed(s, **pkw)
    extra = (["S0", "z0"] + (["cache_q", "cache_k"] if s.conv_k > 1 else [])) if with_state else []
    x = I.make(s, NAMES + extra)
    d = {n: api.to_device(v, "f32" if n in ("S0", "z0") else s.dtype) for n, v in x.items()}
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    n0 = api.launch_count()
    api.trace_begin()
    r = api.lawcat_layer_fwd(P(api, s, **pkw), *[d[n] for n in NAMES], d.get("cache_q"), d.get("cache_k"),
                             d.get("S0"), d.get("z0"), dev_status=status)
    kernels = api.trace_end()
    assert any(k.startswith("layer_tc") for k in kernels) == expect_tc, f"unexpected kernels: {kernels}"
    assert api.launch_count() > n0
    assert int(status.item()) == 0
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in NAMES], x.get("cache_q"), x.get("cache_k"), x.get("S0"),
                      x.get("z0"))
    e = check(r["o"], ref["o"], "bf16", "o")
    check(r["S_T"], ref["S_T"], "bf16", "S_T", f32_store=True)
    check(r["z_T"], ref["z_T"], "bf16", "z_T", f32_store=True)
    if s.conv_k > 1:
        assert np.array_equal(r["cache_q"].float().cpu().numpy(), ref["cache_q"].astype(np.float32))
        assert np.array_equal(r["cache_k"].float().cpu().numpy(), ref["cache_k"].astype(np.float32))
    return e, r, ref


@pytest.mark.parametrize("T", [1, 2, 3, 5, 15, 16, 17, 31, 63, 64, 65, 127, 128, 129, 200])
@pytest.mark.parametrize("with_state", [False, True])
def test_lengths_around_the_chunk_size(api, T, with_state):
    """(calls of fewer than 16 tokens are served by the exact recurrence)"""
    run_case(api, shape(2, T, 4, 2, 41), with_state)


@pytest.mark.parametrize("H,Hkv", [(2, 2), (4, 1), (8, 2)])
def test_head_grouping(api, H, Hkv):
    run_case(api, shape(1, 300, H, Hkv, 42), True)


@pytest.mark.parametrize("conv_k", [1, 2, 3, 4])
def test_conv_widths(api, conv_k):
    run_case(api, shape(1, 150, 2, 1, 43, conv_k=conv_k), True)


@pytest.mark.parametrize("tau", [1.0, 4.0, 8.0, 16.0, 64.0])
def test_gate_sharpness(api, tau):
    """tau = 1 is the plain sigmoid gate of Section 4.2: per-token decays down to a few percent. Sigmoid gates with tau < 8
    take the exact recurrence, from tau = 8 on the tensor-core kernel."""
    _, _, _ = run_case(api, shape(1, 260, 2, 1, 44, gate_tau=tau), False, expect_tc=tau >= 8.0)


@pytest.mark.parametrize("T", [1162, 1223, 1300])
def test_distillation_lengths(api, T):
    run_case(api, shape(1, T, 4, 2, 45), False)


@pytest.mark.parametrize("T,with_state", [(1, False), (64, False), (65, True), (300, False), (1223, True), (8269, True)])
def test_one_decay_per_head(api, T, with_state):
    """gate_dim = 1: the decay of a token is shared by all key channels of a head (the scalar-gate reading of Section
    4.2); short, ragged, carried-state and many-segment lengths."""
    run_case(api, shape(1, T, 4, 2, 50, gate_dim=1), with_state)


def test_one_decay_per_head_sharp_gate(api):
    """One plain-sigmoid decay per head (gate_dim = 1, tau = 1): the library serves it with the exact recurrence, because
    the state then sits on the last one or two tokens; tau = 8 is on the tensor-core kernel."""
    run_case(api, shape(2, 200, 2, 1, 51, gate_dim=1, gate_tau=1.0), False, expect_tc=False)
    run_case(api, shape(2, 200, 2, 1, 51, gate_dim=1, gate_tau=2.0), True, expect_tc=False)
    run_case(api, shape(2, 200, 2, 1, 51, gate_dim=1, gate_tau=8.0), True, expect_tc=True)


def shape64(B, T, H, Hkv, cid, **kw):
    return I.LayerShape(B, T, H, Hkv, 64, 64, dtype="bf16", config_id=cid, **kw)


@pytest.mark.parametrize("T,with_state", [(1, False), (63, True), (64, False), (65, True), (200, False), (1300, True),
                                          (4133, True)])
def test_heads_of_width_64(api, T, with_state):
    """d_k = d_v = 64 (the Llama-3.2-1B shape): the kernel runs such a head as a 128-wide one with zero upper channels;
    the feature map, the outputs and the states must not see the padding."""
    run_case(api, shape64(2, T, 4, 2, 52), with_state)


@pytest.mark.parametrize("kw", [dict(gate_dim=1), dict(conv_k=2), dict(gate_tau=1.0)])
def test_heads_of_width_64_variants(api, kw):
    run_case(api, shape64(1, 333, 8, 2, 53, **kw), True)


def test_long_sequence_many_segments(api):
    """Long enough for the sequence to be split into segments whose states are handed across thread blocks."""
    e, _, _ = run_case(api, shape(1, 8192 + 77, 2, 1, 46), True)
    print(f"T=8269 error {e:.3e}")


@pytest.mark.parametrize("chunk", [0, 1])
@pytest.mark.parametrize("which", ["S", "z"])
def test_state_outputs_are_optional_one_by_one(api, chunk, which):
    """S_T without z_T and z_T without S_T, on the tensor-core kernel (chunk = 0) and on the exact path (chunk = 1)."""
    s = shape(1, 150, 2, 1, 56)
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    r = api.lawcat_layer_fwd(P(api, s, chunk=chunk), *[d[n] for n in NAMES], want_state=which)
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in NAMES])
    check(r["o"], ref["o"], "bf16", "o")
    if which == "S":
        assert r["z_T"] is None
        check(r["S_T"], ref["S_T"], "bf16", "S_T", f32_store=True)
    else:
        assert r["S_T"] is None
        check(r["z_T"], ref["z_T"], "bf16", "z_T", f32_store=True)


def test_log_decay_gate_mode(api):
    import torch
    s = shape(1, 200, 2, 1, 47)
    x = I.make(s, NAMES)
    x["gate"] = I.round_to_bf16(-np.abs(x["gate"]) * np.float32(0.125))
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    r = api.lawcat_layer_fwd(P(api, s, gate_mode=1), *[d[n] for n in NAMES])
    ref = O.layer_fwd(oracle_params(s, gate_mode=1), *[x[n] for n in NAMES])
    check(r["o"], ref["o"], "bf16", "o")
    check(r["S_T"], ref["S_T"], "bf16", "S_T", f32_store=True)


def test_eps_in_the_denominator(api):
    s = shape(1, 100, 2, 1, 48)
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    r = api.lawcat_layer_fwd(P(api, s, eps=0.5), *[d[n] for n in NAMES])
    ref = O.layer_fwd(oracle_params(s, eps=0.5), *[x[n] for n in NAMES])
    # with eps the per-token scale of the query features no longer cancels: this checks that the kernel normalizes them
    check(r["o"], ref["o"], "bf16", "o")


@pytest.mark.parametrize("d", [128, 64])
def test_without_normalization(api, d):
    """normalize = 0 (the ablation without the normalizer, Section 5.4): the output is the numerator of Eq. 8, with the
    query features properly normalized by their softmax sum."""
    s = I.LayerShape(1, 300, 4, 2, d, d, dtype="bf16", config_id=54)
    x = I.make(s, NAMES)
    dv = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    api.trace_begin()
    r = api.lawcat_layer_fwd(P(api, s, normalize=0), *[dv[n] for n in NAMES])
    assert any(k.startswith("layer_tc") for k in api.trace_end())
    ref = O.layer_fwd(oracle_params(s, normalize=0), *[x[n] for n in NAMES])
    check(r["o"], ref["o"], "bf16", "o")
    check(r["S_T"], ref["S_T"], "bf16", "S_T", f32_store=True)


def test_exponent_clamp_is_reported(api):
    """Gate logits so negative that the decay exponents within half a chunk leave +-120: the kernel clamps them, says so
    through dev_status (LAWCAT_ERR_NUMERIC = 6) and still returns finite numbers; moderate logits report nothing."""
    import torch
    s = shape(1, 128, 2, 1, 55, gate_tau=16.0)
    x = I.make(s, NAMES)
    for scale, want in ((1.0, 0), (60.0, 6)):
        g = I.round_to_bf16(-np.abs(x["gate"]) * np.float32(scale))
        d = {n: api.to_device(g if n == "gate" else v, s.dtype) for n, v in x.items()}
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        r = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in NAMES], dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == want
        assert torch.isfinite(r["o"].float()).all() and torch.isfinite(r["S_T"]).all()


def test_agrees_with_exact_path_and_split_calls(api):
    """Tensor-core path vs the CUDA-core recurrent path (chunk = 1) on the same device inputs, and one call vs two calls
    that carry the state and the conv caches."""
    import torch
    s = shape(2, 333, 4, 2, 49)
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    tc = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in NAMES])
    ex = api.lawcat_layer_fwd(P(api, s, chunk=1), *[d[n] for n in NAMES])
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in NAMES])
    check(tc["o"], ref["o"], "bf16", "tc o")
    check(ex["o"], ref["o"], "bf16", "exact o")
    check(tc["S_T"], ex["S_T"].double().cpu().numpy(), "bf16", "tc vs exact S_T", f32_store=True)
    cut = 150
    part = lambda lo, hi: [d[n][:, lo:hi].contiguous() for n in NAMES[:4]] + [d[n] for n in NAMES[4:]]
    r1 = api.lawcat_layer_fwd(P(api, dataclasses.replace(s, T=cut)), *part(0, cut))
    r2 = api.lawcat_layer_fwd(P(api, dataclasses.replace(s, T=s.T - cut)), *part(cut, s.T), r1["cache_q"],
                              r1["cache_k"], r1["S_T"], r1["z_T"])
    o = torch.cat([r1["o"], r2["o"]], 1)
    check(o, ref["o"], "bf16", "split o")
    check(r2["S_T"], ex["S_T"].double().cpu().numpy(), "bf16", "split S_T", f32_store=True)


def test_bench_configuration_sampled_heads(api):
    """The headline shape (T = 32768, 32/8 heads, d = 128) in the launch configuration the benchmark times: the oracle
    checks every output of the first 2048 tokens of all 32 heads; properties that hold at any length (outputs inside the
    running range of the values; a second call that carries state and caches from the middle reproduces the tail and the
    final state of the single call) cover the rest. All tokens of four heads against the oracle: test_long_context.py."""
    import torch
    s = I.CONFIGS["c3"]
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    r = api.lawcat_layer_fwd(P(api, s), *[d[n] for n in NAMES])
    torch.cuda.synchronize()
    Ts = 2048
    ref = O.layer_fwd(oracle_params(dataclasses.replace(s, T=Ts)), *[x[n][:, :Ts] for n in NAMES[:4]],
                      *[x[n] for n in NAMES[4:]])
    check(r["o"][:, :Ts], ref["o"], "bf16", "o[:2048]")
    o = r["o"].float()
    assert torch.isfinite(o).all()
    # property that holds at any length (Section 5.3: the output is a normalized weighted sum of the values):
    # every output lies inside the range of the values seen so far (up to bf16 rounding)
    v = d["v"].float().repeat_interleave(s.H // s.H_kv, dim=2)
    hi, lo = torch.cummax(v, 1).values, torch.cummin(v, 1).values
    tol = 2.0 ** -7 * torch.maximum(hi.abs(), lo.abs()) + 1e-3
    assert bool(((o <= hi + tol) & (o >= lo - tol)).all())
    # a second call that carries the state from the middle reproduces the tail
    half = s.T // 2
    part = lambda lo_, hi_: [d[n][:, lo_:hi_].contiguous() for n in NAMES[:4]] + [d[n] for n in NAMES[4:]]
    r1 = api.lawcat_layer_fwd(P(api, dataclasses.replace(s, T=half)), *part(0, half))
    r2 = api.lawcat_layer_fwd(P(api, dataclasses.replace(s, T=half)), *part(half, s.T), r1["cache_q"], r1["cache_k"],
                              r1["S_T"], r1["z_T"])
    check(r2["o"], r["o"][:, half:].double().cpu().numpy(), "bf16", "second half o")
    check(r2["S_T"], r["S_T"].double().cpu().numpy(), "bf16", "final S_T", f32_store=True)
