"""Packed variable-length sequences (lawcat_layer_fwd_varlen): every sequence of the pack against the oracle run on that
sequence alone (so the state and the conv are reset at every boundary), with and without carried-in states and caches, on
the tensor-core path (bf16, d = 128) and on the exact path (fp32)."""
import numpy as np
import pytest

from helpers import check, oracle_params
from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I



NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("bf16", 64), ("f32", 32)])
@pytest.mark.parametrize("with_state", [False, True])
def test_packed_sequences_match_the_oracle_one_by_one(dtype, d, with_state):
    import dataclasses
    import torch
    from paper_2509_18467_b200 import api
    lens = [1, 63, 0, 200, 700, 64]
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    s = I.LayerShape(1, cu[-1], 4, 2, d, d, dtype=dtype, config_id=95)
    x = I.make(s, NAMES)
    st = I.make(dataclasses.replace(s, B=len(lens)), ["S0", "z0", "cache_q", "cache_k"]) if with_state else {}
    dv = {n: api.to_device(v, dtype) for n, v in x.items()}
    ds = {n: api.to_device(v, "f32" if n in ("S0", "z0") else dtype) for n, v in st.items()}
    p = api.params(1, s.T, s.H, s.H_kv, d, d, dtype=dtype)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    r = api.lawcat_layer_fwd_varlen(p, cu, *[dv[n] for n in NAMES], ds.get("cache_q"), ds.get("cache_k"), ds.get("S0"),
                                    ds.get("z0"), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for i, n in enumerate(lens):
        lo, hi = cu[i], cu[i + 1]
        sub = dataclasses.replace(s, T=n)
        init = {k2: (v[i:i + 1] if k2 in st else None) for k2, v in st.items()}
        if n == 0:  # an empty sequence hands its state through
            want_S = st["S0"][i] if with_state else np.zeros_like(r["S_T"][i].cpu().numpy())
            assert np.array_equal(r["S_T"][i].cpu().numpy(), want_S)
            continue
        ref = O.layer_fwd(oracle_params(sub), *[x[m][:, lo:hi] for m in NAMES[:4]], *[x[m] for m in NAMES[4:]],
                          init.get("cache_q"), init.get("cache_k"), init.get("S0"), init.get("z0"))
        check(r["o"][:, lo:hi], ref["o"], dtype, f"o of sequence {i}")
        check(r["S_T"][i:i + 1], ref["S_T"], dtype, f"S_T of sequence {i}", f32_store=True)
        check(r["z_T"][i:i + 1], ref["z_T"], dtype, f"z_T of sequence {i}", f32_store=True)
        assert np.array_equal(r["cache_q"][i:i + 1].float().cpu().numpy(), ref["cache_q"].astype(np.float32))
        assert np.array_equal(r["cache_k"][i:i + 1].float().cpu().numpy(), ref["cache_k"].astype(np.float32))


def test_bad_offsets_are_refused_on_the_host():
    import ctypes
    from paper_2509_18467_b200 import api
    L = api.lib()
    p = api.params(1, 10, 2, 1, 64, 64)
    ok = ctypes.c_void_p(0x1000)
    f = L.lawcat_layer_fwd_varlen
    f.restype = ctypes.c_int
    f.argtypes = [ctypes.POINTER(api.Params), ctypes.c_void_p, ctypes.c_int] + [ctypes.c_void_p] * 17 + \
                 [ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
    args = [ok] * 7 + [None] * 4 + [ok] + [None] * 4 + [ok, 1 << 30, None, None]
    for bad in ([0, 4, 9], [1, 4, 10], [0, 6, 4, 10]):
        cu = (ctypes.c_int32 * len(bad))(*bad)
        assert f(ctypes.byref(p), cu, len(bad) - 1, *args) == 1
    p2 = api.params(2, 10, 2, 1, 64, 64)
    cu = (ctypes.c_int32 * 2)(0, 10)
    assert f(ctypes.byref(p2), cu, 1, *args) == 1
