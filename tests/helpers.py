"""Shared helpers of the GPU parity tests: input staging, oracle calls and the two error metrics."""
import numpy as np

from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I

# Tolerances (stated by the benchmark definition): fp32 mode max relative error 1e-4, bf16 mode 1e-2 of the output RMS.
TOL_F32 = 1e-4
TOL_BF16 = 1e-2
BF16_HALF_ULP = 2.0 ** -8   # worst relative error of rounding a value to bfloat16 storage


def err_f32(x, y):
    """max_i |x_i - y_i| / max(|y_i|, rms(y))"""
    x, y = np.asarray(x, np.float64), np.asarray(y, np.float64)
    if y.size == 0:
        return 0.0
    rms = np.sqrt(np.mean(y * y)) + 1e-300
    return float(np.max(np.abs(x - y) / np.maximum(np.abs(y), rms)))


def err_bf16(x, y):
    """Returns (strict, computed): strict = max_i |x_i - y_i| / rms(y); computed discounts, per element, the half ulp
    that storing the result in bfloat16 costs whatever was computed: max_i (|x_i - y_i| - 2^-8 |y_i|)+ / rms(y)."""
    x, y = np.asarray(x, np.float64), np.asarray(y, np.float64)
    if y.size == 0:
        return 0.0, 0.0
    rms = np.sqrt(np.mean(y * y)) + 1e-300
    d = np.abs(x - y)
    return float(np.max(d) / rms), float(np.max(np.maximum(d - BF16_HALF_ULP * np.abs(y), 0.0)) / rms)


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
