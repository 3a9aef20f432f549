"""Shared helpers of the GPU parity tests: input staging, oracle calls and the two error metrics."""
import numpy as np

from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I

from paper_2509_18467_b200.metrics import TOL_BF16, TOL_F32, err_bf16, err_f32  # noqa: F401


def check(x, y, dtype, what, f32_store=False):
    """Assert parity of GPU result x (tensor or array) with oracle y for storage type dtype ('f32' | 'bf16').
    f32_store: the tensor is stored in fp32 even in bf16 mode (states, denominators, weight gradients)."""
    import torch
    if isinstance(x, torch.Tensor):
        x = x.detach().float().cpu().numpy()
    assert x.shape == tuple(np.shape(y)), (what, x.shape, np.shape(y))
    assert np.isfinite(x).all(), f"{what}: non-finite values"
    if dtype == "f32":
        e = err_f32(x, y)
        assert e <= TOL_F32, f"{what}: fp32 error {e:.3e} > {TOL_F32}"
    else:
        strict, comp = err_bf16(x, y)
        e = strict if f32_store else comp
        assert e <= TOL_BF16, f"{what}: bf16 error {e:.3e} (strict {strict:.3e}) > {TOL_BF16}"
    return e


def oracle_params(s: I.LayerShape, **kw):
    return O.OracleParams(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v, conv_k=s.conv_k, gate_dim=s.gate_dim,
                          gate_tau=s.gate_tau, **kw)


def tc_routed(s: I.LayerShape, phi=0, gate_mode=0, chunk=0, mix_unshared=0, **_):
    """Whether lawcat_layer_fwd serves this shape with the chunkwise tensor-core layer kernel (the rule its header states):
    bf16, d_k = d_v in {64, 128}, softmax feature map, conv width <= 4, one linear layer for both streams, at least 16
    tokens, and log-decay gates or sigmoid gates with tau >= 8; chunk = 1 forces the exact recurrence."""
    return (s.dtype == "bf16" and s.d_k == s.d_v and s.d_k in (64, 128) and phi == 0 and s.conv_k <= 4 and chunk != 1
            and not mix_unshared and s.B > 0 and s.T >= 16 and (gate_mode == 1 or s.gate_tau >= 8.0))
