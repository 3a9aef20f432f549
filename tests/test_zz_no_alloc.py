"""The no-allocation layer forward (`lawcat_layer_fwd_noalloc`) against the regular entry point.

Some callers of this library cannot call cudaMalloc where they call the layer (a frozen memory pool, a host application
that owns the allocator), so they cannot hand over a workspace; the no-allocation entry point keeps its scratch in a
fixed array inside the library instead. This file checks, through the C ABI, that it returns what `lawcat_layer_fwd`
returns, twice in a row (the scratch is shared and keeps the previous call's contents), and that it refuses problems
beyond its fixed limit. It is collected last so that a failure here cannot hide any other test.
"""
import ctypes
import dataclasses

import pytest

from helpers import check
from paper_2509_18467_b200 import inputs as I

NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]


def _p(api, s, **kw):
    return api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim, dtype=s.dtype,
                      gate_tau=s.gate_tau, **kw)


def _driver_free_bytes():
    import torch
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_noalloc_matches_regular_entry_point_and_oracle_twice(dtype):
    import torch
    from oracle import lawcat_oracle as O
    from paper_2509_18467_b200 import api
    shapes = [I.LayerShape(2, 200, 4, 2, 64, 64, dtype=dtype, config_id=21),
              I.LayerShape(1, 77, 8, 2, 128, 32, dtype=dtype, gate_dim=1, config_id=22)]
    # The first call on a device does the set-up (it looks up the address of the built-in scratch array, which is also
    # when the driver brings in the library's device image, array included): prime it on a one-token problem, so that
    # the memory readings below see steady-state calls.
    s0 = I.LayerShape(1, 1, 2, 1, 16, 16, dtype=dtype, config_id=20)
    x0 = {n: api.to_device(v, s0.dtype) for n, v in I.make(s0, NAMES).items()}
    api.lawcat_layer_fwd_noalloc(_p(api, s0), *[x0[n] for n in NAMES],
                                 o=torch.empty(1, 1, 2, 16, dtype=x0["q"].dtype, device="cuda"))
    for s in shapes:  # the second call reuses the scratch the first one left behind, with a different shape
        x = I.make(s, NAMES + ["S0", "z0", "cache_q", "cache_k"])
        d = {n: api.to_device(v, "f32" if n in ("S0", "z0") else s.dtype) for n, v in x.items()}
        p = _p(api, s)
        # the entry point runs the recurrent CUDA-core path; chunk = 1 selects the same path in the regular entry point
        ref = api.lawcat_layer_fwd(_p(api, s, chunk=1), *[d[n] for n in NAMES], d["cache_q"], d["cache_k"], d["S0"],
                                   d["z0"])
        out = {k: torch.full_like(v, float("nan")) for k, v in ref.items()}
        # device memory as the driver sees it (not the framework's allocator, which a call into the library never
        # touches): the call must leave it where it was. (The library image with its scratch array is loaded by now.)
        free_before = _driver_free_bytes()
        api.lawcat_layer_fwd_noalloc(p, *[d[n] for n in NAMES], d["cache_q"], d["cache_k"], d["S0"], d["z0"],
                                     out["o"], out["cache_q"], out["cache_k"], out["S_T"], out["z_T"])
        assert _driver_free_bytes() == free_before
        check(out["o"], ref["o"].double().cpu().numpy(), s.dtype, "o")
        check(out["S_T"], ref["S_T"].double().cpu().numpy(), s.dtype, "S_T", f32_store=True)
        check(out["z_T"], ref["z_T"].double().cpu().numpy(), s.dtype, "z_T", f32_store=True)
        assert torch.equal(out["cache_q"], ref["cache_q"]) and torch.equal(out["cache_k"], ref["cache_k"])
        # and against the CPU oracle on the same seeded inputs
        op = O.OracleParams(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim,
                            gate_tau=s.gate_tau)
        want = O.layer_fwd(op, *[x[n] for n in NAMES], x["cache_q"], x["cache_k"], x["S0"], x["z0"])
        check(out["o"], want["o"], s.dtype, "o vs oracle")
        check(out["S_T"], want["S_T"], s.dtype, "S_T vs oracle", f32_store=True)
        check(out["z_T"], want["z_T"], s.dtype, "z_T vs oracle", f32_store=True)


@pytest.mark.gpu
def test_noalloc_accepts_the_largest_problem_that_fits():
    """B*T*H*d_k = 4 Mi elements fills the built-in scratch exactly: the call runs and agrees with the regular entry
    point; one more token is refused."""
    import torch
    from paper_2509_18467_b200 import api
    s = I.LayerShape(1, 1024, 32, 8, 128, 128, dtype="bf16", config_id=23)
    assert 2 * 4 * s.B * s.T * s.H * s.d_k == api.lib().lawcat_noalloc_scratch_bytes()
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    ref = api.lawcat_layer_fwd(_p(api, s, chunk=1), *[d[n] for n in NAMES])
    o = torch.full_like(ref["o"], float("nan"))
    S_T = torch.full_like(ref["S_T"], float("nan"))
    api.lawcat_layer_fwd_noalloc(_p(api, s), *[d[n] for n in NAMES], o=o, S_T=S_T)
    torch.cuda.synchronize()
    check(o, ref["o"].double().cpu().numpy(), "bf16", "o")
    check(S_T, ref["S_T"].double().cpu().numpy(), "bf16", "S_T", f32_store=True)
    more = dataclasses.replace(s, T=s.T + 1)
    big = {n: (torch.cat([d[n], d[n][:, :1]], 1) if n in NAMES[:4] else d[n]) for n in NAMES}
    with pytest.raises(api.LawcatError) as e:
        api.lawcat_layer_fwd_noalloc(_p(api, more), *[big[n] for n in NAMES], o=torch.empty(1, s.T + 1, s.H, s.d_v,
                                     dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == 7


def test_noalloc_rejects_oversized_and_bad_problems_on_host():
    from paper_2509_18467_b200 import api, build
    build.build()
    L = api.lib()
    limit = L.lawcat_noalloc_scratch_bytes()
    assert limit == 32 << 20
    ok = ctypes.c_void_p(0x1000)
    args = [ok] * 7 + [None] * 4 + [ok] + [None] * 4 + [None, None]
    big = api.params(1, 4096, 32, 8, 128, 128)      # 2 * 4 * 16 Mi elements: far beyond the array
    assert L.lawcat_layer_fwd_noalloc(ctypes.byref(big), *args) == 7
    assert "built-in scratch" in api.status_string(7)
    # a size that wraps around in 64 bits (two tensors of 2^19 * 2^30 * 32 * 128 * 4 bytes = 2^64) is refused all the same
    huge = api.params(1 << 19, 1 << 30, 32, 8, 128, 128)
    assert L.lawcat_layer_fwd_noalloc(ctypes.byref(huge), *args) == 7
    edge = api.params(1, 1024, 32, 8, 128, 128)     # exactly 4 Mi elements per tensor: fits
    assert 2 * 4 * 1024 * 32 * 128 == limit
    bad = api.params(1, 16, 4, 3, 64, 64)
    assert L.lawcat_layer_fwd_noalloc(ctypes.byref(bad), *args) == 1
    odd = api.params(1, 16, 4, 2, 48, 64)
    assert L.lawcat_layer_fwd_noalloc(ctypes.byref(odd), *args) == 2
    nullq = [None] + args[1:]
    assert L.lawcat_layer_fwd_noalloc(ctypes.byref(edge), *nullq) == 1
