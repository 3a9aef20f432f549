"""lawcat_layer_fwd_host: tensors in pinned HOST memory in, o in host memory out. The call slices the sequence along T and
overlaps the copies of the next slice, the layer on the current one (started from the state and conv caches the previous
slice left) and the copy back of the last one on three streams; the result must match the oracle's one-pass forward."""
import numpy as np
import pytest

from helpers import check, oracle_params
from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I

NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,B,T,d,conv_k", [("bf16", 2, 5000, 128, 4),   # three slices per batch element, ragged last
                                                ("bf16", 1, 2049, 64, 4),    # a last slice of one token
                                                ("bf16", 1, 4096, 64, 1),    # no conv: no caches between slices
                                                ("f32", 2, 2500, 32, 3),     # exact path
                                                ("bf16", 3, 300, 128, 4)])   # one slice per batch element
def test_host_path_matches_the_oracle(dtype, B, T, d, conv_k):
    import torch
    from paper_2509_18467_b200 import api
    s = I.LayerShape(B, T, 4, 2, d, d, conv_k=conv_k, dtype=dtype, config_id=97)
    x = I.make(s, NAMES)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    h = {n: api.to_device(v, dtype).cpu().pin_memory() for n, v in x.items()}
    h_o = torch.zeros(B, T, s.H, d, dtype=tdt).pin_memory()
    p = api.params(B, T, s.H, s.H_kv, d, d, conv_k=conv_k, dtype=dtype)
    arena = torch.empty(api.host_arena_bytes(p), dtype=torch.uint8, device="cuda")
    for _ in range(2):  # the second call reuses the arena behind the first
        api.lawcat_layer_fwd_host(p, *[h[n] for n in NAMES], h_o, arena)
    torch.cuda.synchronize()
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in NAMES])
    check(h_o, ref["o"], dtype, "o")


@pytest.mark.gpu
def test_host_path_refuses_a_small_arena():
    import torch
    from paper_2509_18467_b200 import api
    p = api.params(1, 256, 4, 2, 64, 64)
    need = api.host_arena_bytes(p)
    assert need > 0
    h = torch.zeros(16, dtype=torch.bfloat16).pin_memory()
    arena = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(api.LawcatError):
        api.lawcat_layer_fwd_host(p, h, h, h, h, h, h, h, h, arena)
