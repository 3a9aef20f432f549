"""Randomized parity of the tensor-core layer forward: 36 seeded draws of (head width, batch, length, head grouping,
conv width, gate sharpness, gate width, carried state, normalizer on/off, eps) against the fp64 oracle, through the C ABI.

Tolerance: 1e-2 of the RMS on every tensor (outputs and the final state). Under the plain sigmoid gate (tau < 2) one decay
per head (gate_dim = 1) and the numerator-only form (normalize = 0) are served by the exact recurrence (see the header of
lawcat_layer_fwd); every other draw must run on the tensor-core kernel."""
import random

import numpy as np
import pytest

from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I
from paper_2509_18467_b200.metrics import err_bf16

pytestmark = pytest.mark.gpu

NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]


def draws():
    rng = random.Random(7)
    out = []
    for it in range(36):
        d = rng.choice([64, 128]); Hkv = rng.choice([1, 2, 3]); G = rng.choice([1, 2, 4])
        B = rng.choice([1, 2, 3]); T = rng.choice([1, 7, 64, 100, 257, 513, 1000, 2100, 4500])
        K = rng.choice([1, 2, 3, 4]); tau = rng.choice([1.0, 4.0, 16.0]); gd = rng.choice([0, 1])
        state = rng.random() < 0.5
        norm = rng.choice([1, 1, 0]); eps = rng.choice([0.0, 0.0, 0.3])
        out.append((it, d, B, T, Hkv * G, Hkv, K, tau, gd, state, norm, eps))
    return out


@pytest.mark.parametrize("case", draws(), ids=lambda c: f"draw{c[0]}-d{c[1]}-T{c[3]}")
def test_random_configuration(case):
    import torch
    from paper_2509_18467_b200 import api
    it, d, B, T, H, Hkv, K, tau, gd, state, norm, eps = case
    s = I.LayerShape(B, T, H, Hkv, d, d, dtype="bf16", config_id=900 + it, conv_k=K, gate_tau=tau, gate_dim=gd)
    extra = (["S0", "z0"] + (["cache_q", "cache_k"] if K > 1 else [])) if state else []
    x = I.make(s, NAMES + extra)
    dv = {n: api.to_device(x[n], "f32" if n in ("S0", "z0") else "bf16") for n in x}
    p = api.params(B, T, H, Hkv, d, d, conv_k=K, gate_tau=tau, gate_dim=s.gate_dim, normalize=norm, eps=eps)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.trace_begin()
    r = api.lawcat_layer_fwd(p, *[dv[n] for n in NAMES], dv.get("cache_q"), dv.get("cache_k"), dv.get("S0"), dv.get("z0"),
                             dev_status=status)
    kernels = api.trace_end()
    exact = tau < 2.0 and (s.gate_dim == 1 or norm == 0)
    assert any(k.startswith("layer_tc") for k in kernels) != exact, kernels
    assert int(status.item()) == 0
    ref = O.layer_fwd(O.OracleParams(B, T, H, Hkv, d, d, conv_k=K, gate_tau=tau, gate_dim=s.gate_dim, normalize=norm,
                                     eps=eps),
                      *[x[n] for n in NAMES], x.get("cache_q"), x.get("cache_k"), x.get("S0"), x.get("z0"))
    o = r["o"].float().cpu().numpy()
    assert np.isfinite(o).all()
    _, e_o = err_bf16(o, ref["o"])
    assert e_o <= 1e-2, f"o: {e_o:.3e}"
    rms = max(float(np.sqrt((ref["S_T"] ** 2).mean())), 1e-30)
    e_S = float(np.abs(r["S_T"].cpu().numpy() - ref["S_T"]).max()) / rms
    assert e_S <= 1e-2, f"S_T: {e_S:.3e}"
    rz = max(float(np.sqrt((ref["z_T"] ** 2).mean())), 1e-30)
    e_z = float(np.abs(r["z_T"].cpu().numpy() - ref["z_T"]).max()) / rz
    assert e_z <= 1e-2, f"z_T: {e_z:.3e}"
