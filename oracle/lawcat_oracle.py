"""ctypes front end of the fp64 CPU oracle (``lawcat_oracle.c``).

TEST INFRASTRUCTURE, not part of the product: only the tests, the smoke check and the benchmark's CPU-baseline leg
may import this module. It compiles the C file with gcc on first use and exchanges numpy float64 arrays with it.
Nothing here touches the CUDA library or its Python binding.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lawcat_oracle.c")
_LIB = os.path.join(_HERE, "liblawcat_oracle.so")

PHI_SOFTMAX, PHI_ELU1, PHI_IDENTITY = 0, 1, 2
GATE_LOGITS, GATE_LOGDECAY = 0, 1


class _CParams(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("B", "T", "H", "H_kv", "d_k", "d_v", "conv_k", "gate_dim", "phi", "gate_mode", "normalize")] + \
               [("gate_tau", ctypes.c_double), ("eps", ctypes.c_double)]


@dataclass
class OracleParams:
    B: int
    T: int
    H: int
    H_kv: int
    d_k: int
    d_v: int
    conv_k: int = 4
    gate_dim: int = 0          # 0 -> d_k
    phi: int = PHI_SOFTMAX
    gate_mode: int = GATE_LOGITS
    normalize: int = 1
    gate_tau: float = 16.0
    eps: float = 0.0

    def c(self) -> _CParams:
        gd = self.gate_dim or self.d_k
        return _CParams(self.B, self.T, self.H, self.H_kv, self.d_k, self.d_v, self.conv_k, gd, self.phi,
                        self.gate_mode, self.normalize, float(self.gate_tau), float(self.eps))

    @property
    def gd(self) -> int:
        return self.gate_dim or self.d_k


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, no fast-math) and return the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_L().oracle_threads())


def _p(a):
    if a is None:
        return None
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def conv(x, w, cache, K):
    """x [B,T,NH,d], w [NH*d,K], cache [B,K-1,NH*d] or None -> conv(x) [B,T,NH,d] (Section 4.1)."""
    x, w, cache = _f64(x), _f64(w), _f64(cache)
    B, T, NH, d = x.shape
    out = np.empty_like(x)
    _L().oracle_conv(_p(x), _p(w), _p(cache), B, T, NH, d, K, _p(out))
    return out


def mix_phi(u, W, H, phi=PHI_SOFTMAX):
    """u [B,T,NH_in,d], W [H,d,d] -> phi(u W_h) [B,T,H,d]; head h reads input head h // (H/NH_in)."""
    u, W = _f64(u), _f64(W)
    B, T, NH, d = u.shape
    out = np.empty((B, T, H, d))
    _L().oracle_mix_phi(_p(u), _p(W), B, T, NH, H, d, phi, _p(out))
    return out


def gla_fwd(p: OracleParams, qdot, kdot, v, gate, S0=None, z0=None):
    """Eq. 4 + Eq. 8 token by token. Returns dict(o, den, S_T, z_T)."""
    qdot, kdot, v, gate, S0, z0 = map(_f64, (qdot, kdot, v, gate, S0, z0))
    cp = p.c()
    o = np.empty((p.B, p.T, p.H, p.d_v))
    den = np.empty((p.B, p.T, p.H))
    S_T = np.empty((p.B, p.H, p.d_k, p.d_v))
    z_T = np.empty((p.B, p.H, p.d_k))
    _L().oracle_gla_fwd(ctypes.byref(cp), _p(qdot), _p(kdot), _p(v), _p(gate), _p(S0), _p(z0), _p(o), _p(den),
                        _p(S_T), _p(z_T))
    return dict(o=o, den=den, S_T=S_T, z_T=z_T)


def gla_bwd(p: OracleParams, qdot, kdot, v, gate, dO, S0=None, z0=None):
    """Reverse recurrence for the gradients of gla_fwd. Returns dict(d_qdot, d_kdot, dv, dgate)."""
    qdot, kdot, v, gate, dO, S0, z0 = map(_f64, (qdot, kdot, v, gate, dO, S0, z0))
    cp = p.c()
    d_qdot = np.empty_like(qdot)
    d_kdot = np.empty_like(kdot)
    d_v = np.empty_like(v)
    d_gate = np.empty_like(gate)
    _L().oracle_gla_bwd(ctypes.byref(cp), _p(qdot), _p(kdot), _p(v), _p(gate), _p(S0), _p(z0), _p(dO),
                        _p(d_qdot), _p(d_kdot), _p(d_v), _p(d_gate))
    return dict(d_qdot=d_qdot, d_kdot=d_kdot, dv=d_v, dgate=d_gate)


def conv_bwd(p: OracleParams, q, k, w_q, w_k, W, d_qdot, d_kdot, cache_q=None, cache_k=None):
    """Backward of conv (-> mix -> phi when W is given) on both streams. Returns dict(dq, dk, dw_q, dw_k, dW).
    W [H,d,d]: one linear layer for both streams (dW sums both); W [2,H,d,d]: one per stream (dW likewise)."""
    q, k, w_q, w_k, W, d_qdot, d_kdot, cache_q, cache_k = map(
        _f64, (q, k, w_q, w_k, W, d_qdot, d_kdot, cache_q, cache_k))
    B, T, H, Hkv, d, K = p.B, p.T, p.H, p.H_kv, p.d_k, p.conv_k
    dq, dk = np.empty_like(q), np.empty_like(k)
    dw_q, dw_k = np.empty_like(w_q), np.empty_like(w_k)
    dW = None if W is None else np.zeros_like(W)
    unshared = W is not None and W.ndim == 4
    Wq, Wk = (np.ascontiguousarray(W[0]), np.ascontiguousarray(W[1])) if unshared else (W, W)
    dWq, dWk = (np.zeros_like(Wq), np.zeros_like(Wk)) if unshared else (dW, dW)
    L = _L()
    L.oracle_conv_mix_bwd(_p(q), _p(w_q), _p(cache_q), _p(Wq), _p(d_qdot), B, T, H, H, d, K, p.phi, _p(dq),
                          _p(dw_q), _p(dWq))
    L.oracle_conv_mix_bwd(_p(k), _p(w_k), _p(cache_k), _p(Wk), _p(d_kdot), B, T, Hkv, H if W is not None else Hkv,
                          d, K, p.phi, _p(dk), _p(dw_k), _p(dWk))
    if unshared:
        dW = np.stack([dWq, dWk])
    return dict(dq=dq, dk=dk, dw_q=dw_q, dw_k=dw_k, dW=dW)


def layer_fwd(p: OracleParams, q, k, v, gate, w_q, w_k, W, cache_q=None, cache_k=None, S0=None, z0=None):
    """The whole layer (Fig. 1). Returns dict(o, den, qdot, kdot, cache_q, cache_k, S_T, z_T).
    W [2,H,d,d] = a separate linear layer per stream (appendix table on sharing): the same steps, composed here."""
    if W is not None and np.ndim(W) == 4:
        return _layer_fwd_unshared(p, q, k, v, gate, w_q, w_k, W, cache_q, cache_k, S0, z0)
    q, k, v, gate, w_q, w_k, W, cache_q, cache_k, S0, z0 = map(
        _f64, (q, k, v, gate, w_q, w_k, W, cache_q, cache_k, S0, z0))
    cp = p.c()
    B, T, H, Hkv, dk, dv, K = p.B, p.T, p.H, p.H_kv, p.d_k, p.d_v, p.conv_k
    o = np.empty((B, T, H, dv))
    den = np.empty((B, T, H))
    qd = np.empty((B, T, H, dk))
    kd = np.empty((B, T, H, dk))
    cq = np.empty((B, K - 1, H * dk))
    ck = np.empty((B, K - 1, Hkv * dk))
    S_T = np.empty((B, H, dk, dv))
    z_T = np.empty((B, H, dk))
    _L().oracle_layer_fwd(ctypes.byref(cp), _p(q), _p(k), _p(v), _p(gate), _p(w_q), _p(w_k), _p(W), _p(cache_q),
                          _p(cache_k), _p(S0), _p(z0), _p(o), _p(den), _p(qd), _p(kd), _p(cq), _p(ck), _p(S_T),
                          _p(z_T))
    return dict(o=o, den=den, qdot=qd, kdot=kd, cache_q=cq, cache_k=ck, S_T=S_T, z_T=z_T)


def _layer_fwd_unshared(p, q, k, v, gate, w_q, w_k, W, cache_q, cache_k, S0, z0):
    """conv (Section 4.1) -> linear layer of the stream + phi -> Eq. 4 / Eq. 8, from the same primitives as the shared form;
    the conv caches are the last K - 1 raw rows of [cache, x]."""
    W = _f64(W)
    K = p.conv_k
    qd = mix_phi(conv(q, w_q, cache_q, K), W[0], p.H, p.phi)
    kd = mix_phi(conv(k, w_k, cache_k, K), W[1], p.H, p.phi)
    r = gla_fwd(p, qd, kd, v, gate, S0, z0)
    def tail(x, cache):
        x = _f64(x).reshape(p.B, p.T, -1)
        c = np.zeros((p.B, K - 1, x.shape[2])) if cache is None else _f64(cache).reshape(p.B, K - 1, -1)
        return np.concatenate([c, x], 1)[:, p.T:]
    return dict(o=r["o"], den=r["den"], qdot=qd, kdot=kd, cache_q=tail(q, cache_q), cache_k=tail(k, cache_k),
                S_T=r["S_T"], z_T=r["z_T"])


def decode_step(p: OracleParams, q_t, k_t, v_t, gate_t, w_q, w_k, W, S, z, cache_q, cache_k):
    """One recurrent step = the layer at T = 1 with caches and state. Returns dict(o, S, z, cache_q, cache_k)."""
    B, H, Hkv, dk, dv = p.B, p.H, p.H_kv, p.d_k, p.d_v
    p1 = OracleParams(**{**p.__dict__, "T": 1})
    r = layer_fwd(p1, np.reshape(q_t, (B, 1, H, dk)), np.reshape(k_t, (B, 1, Hkv, dk)),
                  np.reshape(v_t, (B, 1, Hkv, dv)), np.reshape(gate_t, (B, 1, H, p.gd)), w_q, w_k, W,
                  cache_q, cache_k, S, z)
    return dict(o=r["o"].reshape(B, H, dv), S=r["S_T"], z=r["z_T"], cache_q=r["cache_q"], cache_k=r["cache_k"])


def gate_logits(x, A1, A2, bias=None):
    """The gate function in front of the layer (Section 4.2: additional linear layers whose output goes through a sigmoid;
    appendix, ablation on the rank of the gate function: two consecutive low-rank linear layers).
    x [B,T,d_model], A1 [rank,d_model] (first layer), A2 [n_out,rank] (second layer), bias [n_out] or None ->
    logits a [B,T,n_out] with a_t = A2 (A1 x_t) + bias. n_out = H * gate_dim: reshaped to [B,T,H,gate_dim] they are the
    `gate` input of gla_fwd / layer_fwd, where the sigmoid and the power 1/tau are applied (GATE_LOGITS)."""
    x, A1, A2, bias = map(_f64, (x, A1, A2, bias))
    B, T, dm = x.shape
    rank, n_out = A1.shape[0], A2.shape[0]
    assert A1.shape == (rank, dm) and A2.shape == (n_out, rank)
    h = np.empty((B, T, rank))
    for b in range(B):
        for t in range(T):
            h[b, t] = A1 @ x[b, t]          # bottleneck activations of token t
    a = np.empty((B, T, n_out))
    for b in range(B):
        for t in range(T):
            a[b, t] = A2 @ h[b, t]
            if bias is not None:
                a[b, t] += bias
    return a


def gate_log_decay(a, tau):
    """Section 4.2: the gate is the sigmoid of the logits; with the exponent 1/tau of the gate scaling the log of the decay
    of one entry is log(sigmoid(a)) / tau (what GATE_LOGDECAY inputs hold). Written as -(max(-a, 0) + log1p(exp(-|a|))) / tau,
    the form without overflow."""
    a = _f64(a)
    return -(np.maximum(-a, 0.0) + np.log1p(np.exp(-np.abs(a)))) / float(tau)
