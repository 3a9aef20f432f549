"""The gate function (two consecutive low-rank linear layers producing the gate logits; Section 4.2 and the appendix's
ablation on its rank) through the C ABI against the fp64 oracle: the tensor-core kernel for bf16 and rank 16 / 32 / 64 /
128 and more than 1024 tokens (ragged token tiles, hidden widths that are not a multiple of the stage width, output widths
that are not a multiple of the product width, with and without a bias), the latency-oriented kernel for up to 1024 tokens,
the exact kernels for everything else, the logits feeding the layer, the benchmark's size on sampled tokens, and the edge
cases.

Tolerance, bf16 storage: the logits are rounded to bf16 once, so beyond that rounding (half an ulp, allowed by
metrics.err_bf16) the error must stay below 1e-3 of the RMS (bottleneck activations carry 16 significant bits, products
accumulate in fp32); fp32 storage: 1e-5 of the RMS."""
import numpy as np
import pytest

from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I
from paper_2509_18467_b200.metrics import err_bf16, err_f32

pytestmark = pytest.mark.gpu


def run(B, T, H, d, gd, dm, rank, dtype="bf16", bias=True, chunk=0, cfg=900, expect_tc=None, expect_kernel=None):
    import torch
    from paper_2509_18467_b200 import api
    s = I.LayerShape(B, T, H, H, d, d, dtype=dtype, gate_dim=gd, config_id=cfg)
    x = I.make_gate_fn(s, dm, rank)
    dv = {n: api.to_device(v, dtype) for n, v in x.items()}
    p = api.params(B, T, H, H, d, d, gate_dim=gd, dtype=dtype, chunk=chunk)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.trace_begin()
    g = api.lawcat_gate_fn_fwd(p, dm, rank, dv["x"], dv["A1"], dv["A2"], dv["bias"] if bias else None, dev_status=status)
    kernels = api.trace_end()
    assert int(status.item()) == 0
    if expect_tc is not None:
        assert ("gate_fn_tc" in kernels) == expect_tc, kernels
    if expect_kernel is not None:
        assert expect_kernel in kernels, kernels
    want = O.gate_logits(x["x"], x["A1"], x["A2"], x["bias"] if bias else None).reshape(B, T, H, s.gd)
    got = g.float().cpu().numpy()
    assert got.shape == want.shape and np.isfinite(got).all()
    return got, want


@pytest.mark.parametrize("rank", [16, 32, 64, 128])
@pytest.mark.parametrize("B,T,H,d,gd,dm", [
    (6, 193, 3, 64, 0, 256),     # 1158 tokens: nine full tiles and a ragged one; 192 outputs = 1.5 products
    (9, 128, 2, 128, 0, 320),    # whole tiles only; five stages (more than the ring holds)
    (15, 70, 8, 64, 1, 72),      # one decay per head: 8 outputs; hidden width 72 = one stage and an eighth
    (21, 50, 4, 128, 0, 1024),   # 16 stages, 512 outputs
    (8, 1024, 10, 128, 0, 64),   # 64 token tiles, 10 output tiles: a token tile's outputs are shared out 3 + 3 + 3 + 1
])
def test_tensor_core_kernel(rank, B, T, H, d, gd, dm):
    """More than 1024 tokens: the tensor-core kernel."""
    got, want = run(B, T, H, d, gd, dm, rank, expect_tc=True, cfg=900 + rank)
    _, e = err_bf16(got, want)
    assert e <= 1e-3, f"{e:.3e}"


@pytest.mark.parametrize("rank", [8, 24, 32, 128])
@pytest.mark.parametrize("B,T,H,d,gd,dm", [
    (1, 1, 2, 64, 0, 128),       # one token (a decode step of one sequence)
    (64, 1, 32, 128, 0, 4096),   # the decode step of the benchmark's batch at the 7B model's widths
    (2, 193, 3, 64, 0, 256),     # 386 tokens: blocks of four tokens, the last one ragged
    (1, 70, 8, 64, 1, 72),       # 8 outputs; hidden width 72 (fewer octets than lanes)
    (1, 1024, 1, 64, 0, 64),     # the largest call of this kernel
])
def test_few_tokens_kernel(rank, B, T, H, d, gd, dm):
    """Up to 1024 tokens (bf16, widths multiples of 8; any rank that is a multiple of 8): the latency-oriented kernel."""
    import ctypes
    from paper_2509_18467_b200 import api
    got, want = run(B, T, H, d, gd, dm, rank, expect_tc=False, expect_kernel="gate_fn_small", cfg=930 + rank)
    assert err_bf16(got, want)[1] <= 1e-4
    p = api.params(B, T, H, H, d, d, gate_dim=gd)
    f = api.lib().lawcat_gate_fn_workspace_bytes
    f.restype = ctypes.c_size_t
    f.argtypes = [ctypes.POINTER(api.Params), ctypes.c_int32, ctypes.c_int32]
    assert f(ctypes.byref(p), dm, rank) == 0   # (no scratch: the bottleneck activations stay in shared memory)


def test_without_bias():
    got, want = run(1, 1, 2, 64, 0, 128, 32, bias=False, expect_tc=False)
    assert err_bf16(got, want)[1] <= 1e-3
    got, want = run(9, 129, 2, 64, 0, 128, 16, bias=False, expect_tc=True)
    assert err_bf16(got, want)[1] <= 1e-3


@pytest.mark.parametrize("dtype,rank,dm,H,d,gd,chunk", [
    ("f32", 5, 50, 3, 16, 0, 0),        # nothing about the shape suits the tensor-core kernel
    ("f32", 32, 256, 2, 64, 0, 0),      # fp32 storage
    ("bf16", 20, 96, 2, 64, 0, 0),      # a rank neither bf16 kernel takes
    ("bf16", 32, 256, 2, 64, 0, 1),     # chunk = 1 asks for the exact kernels
    ("bf16", 16, 132, 2, 64, 0, 0),     # hidden width not a multiple of 8
    ("bf16", 16, 128, 3, 64, 1, 0),     # 3 outputs
])
def test_exact_kernels(dtype, rank, dm, H, d, gd, chunk):
    got, want = run(2, 37, H, d, gd, dm, rank, dtype=dtype, chunk=chunk, expect_tc=False, expect_kernel="gate_fn_h", cfg=950)
    if dtype == "f32":
        assert err_f32(got, want) <= 1e-5
    else:
        assert err_bf16(got, want)[1] <= 1e-4


def test_logits_feed_the_layer():
    """gate function -> layer forward, both through the C ABI, against the same chain in the oracle (which keeps the
    logits in fp64: the tolerance of the layer output, 1e-2 of the RMS, covers their rounding to bf16)."""
    from paper_2509_18467_b200 import api
    names = ["q", "k", "v", "gate", "w_q", "w_k", "W"]
    B, T, H, Hkv, d, dm, rank = 1, 200, 4, 2, 128, 256, 32
    s = I.LayerShape(B, T, H, Hkv, d, d, config_id=960)
    x = I.make(s, names)
    gx = I.make_gate_fn(s, dm, rank)
    dv = {n: api.to_device(v, "bf16") for n, v in {**x, **gx}.items()}
    p = api.params(B, T, H, Hkv, d, d)
    gate = api.lawcat_gate_fn_fwd(p, dm, rank, dv["x"], dv["A1"], dv["A2"], dv["bias"])
    r = api.lawcat_layer_fwd(p, dv["q"], dv["k"], dv["v"], gate, dv["w_q"], dv["w_k"], dv["W"])
    a = O.gate_logits(gx["x"], gx["A1"], gx["A2"], gx["bias"]).reshape(B, T, H, d)
    ref = O.layer_fwd(O.OracleParams(B, T, H, Hkv, d, d), x["q"], x["k"], x["v"], a, x["w_q"], x["w_k"], x["W"])
    assert err_bf16(r["o"].float().cpu().numpy(), ref["o"])[1] <= 1e-2


def test_benchmark_size_on_sampled_tokens():
    """The Mistral-7B layer of the headline configuration (32768 tokens, hidden width 4096, rank 32, 4096 logits per token),
    in the launch configuration the benchmark times: 192 sampled tokens, among them the first and the last of the
    sequence and both sides of a tile boundary, against the oracle one by one."""
    import torch
    from paper_2509_18467_b200 import api
    s = I.CONFIGS["c3"]
    dm, rank = 4096, 32
    x = I.make_gate_fn(s, dm, rank)
    dv = {n: api.to_device(v, "bf16") for n, v in x.items()}
    p = api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    g = api.lawcat_gate_fn_fwd(p, dm, rank, dv["x"], dv["A1"], dv["A2"], dv["bias"], dev_status=status)
    assert int(status.item()) == 0
    rng = np.random.default_rng(4)
    rows = np.unique(np.concatenate([[0, 127, 128, s.T - 129, s.T - 128, s.T - 1], rng.integers(0, s.T, 186)]))
    want = O.gate_logits(x["x"][:, rows], x["A1"], x["A2"], x["bias"]).reshape(1, len(rows), s.H, s.d_k)
    got = g[:, torch.from_numpy(rows).cuda()].float().cpu().numpy()
    assert err_bf16(got, want)[1] <= 1e-3


def test_empty_and_invalid_calls():
    import torch
    from paper_2509_18467_b200 import api
    p0 = api.params(0, 16, 2, 2, 64, 64)
    A1 = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    A2 = torch.zeros(128, 16, dtype=torch.bfloat16, device="cuda")
    x0 = torch.zeros(0, 16, 64, dtype=torch.bfloat16, device="cuda")
    g = api.lawcat_gate_fn_fwd(p0, 64, 16, x0, A1, A2)       # no tokens: nothing to do, no error
    assert g.numel() == 0
    p = api.params(1, 16, 2, 2, 64, 64)
    x = torch.zeros(1, 16, 64, dtype=torch.bfloat16, device="cuda")
    for dm, rank in ((0, 16), (64, 0), (-8, 16)):
        with pytest.raises(api.LawcatError) as e:
            api.lawcat_gate_fn_fwd(p, dm, rank, x, A1, A2)
        assert e.value.status == 1
    with pytest.raises(api.LawcatError) as e:
        api.lawcat_gate_fn_fwd(p, 32768, 16, x, A1, A2)
    assert e.value.status == 2
    buf = torch.zeros(16 * 64 + 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.LawcatError) as e:                 # a weight pointer off the 16-byte grid
        api.lawcat_gate_fn_fwd(p, 64, 16, x, buf[4:4 + 16 * 64], A2)
    assert e.value.status == 1
