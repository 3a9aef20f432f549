"""Error metrics of the parity checks (no arithmetic of the method).

fp32 mode:  max_i |x_i - y_i| / max(|y_i|, rms(y))            <= 1e-4
bf16 mode:  max_i |x_i - y_i| / rms(y)                        <= 1e-2, where a tensor STORED in bfloat16 is allowed,
            per element, the half unit in the last place of bfloat16 at y_i, 2^(floor(log2 |y_i|) - 8), that the final
            store costs whatever was computed.
"""
import numpy as np

TOL_F32 = 1e-4
TOL_BF16 = 1e-2


def bf16_half_ulp(y):
    """Half a unit in the last place of bfloat16 (8 significant bits) at each |y|: 2^(floor(log2 |y|) - 8); 0 at 0."""
    _, e = np.frexp(np.abs(np.asarray(y, np.float64)))  # |y| = m 2^e with m in [0.5, 1): floor(log2 |y|) = e - 1
    return np.where(np.asarray(y) != 0, np.ldexp(1.0, e - 9), 0.0)


def err_f32(x, y) -> float:
    x, y = np.asarray(x, np.float64), np.asarray(y, np.float64)
    if y.size == 0:
        return 0.0
    rms = np.sqrt(np.mean(y * y)) + 1e-300
    return float(np.max(np.abs(x - y) / np.maximum(np.abs(y), rms)))


def err_bf16(x, y):
    """Returns (strict, computed): strict counts everything; computed discounts the half ulp of the bf16 store."""
    x, y = np.asarray(x, np.float64), np.asarray(y, np.float64)
    if y.size == 0:
        return 0.0, 0.0
    rms = np.sqrt(np.mean(y * y)) + 1e-300
    d = np.abs(x - y)
    return float(np.max(d) / rms), float(np.max(np.maximum(d - bf16_half_ulp(y), 0.0)) / rms)
