"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix (no GPU involved).

Each test compares the oracle with something that is not the oracle: a brute-force statement of a closed form the
paper gives (Eq. 2, Eq. 6-8), a special case with a known answer, an invariant, a library routine, or finite
differences of the oracle's own forward for the hand-derived backward.
"""
import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

from oracle import lawcat_oracle as O

RNG = np.random.default_rng(20250918)


def rnd(*shape):
    return RNG.standard_normal(shape)


def logsigmoid(a):
    return -np.logaddexp(0.0, -a)


# --------------------------------------------------------------------------- conv (Section 4.1)
def brute_conv(x, w, cache, K):
    B, T, NH, d = x.shape
    C = NH * d
    xf = x.reshape(B, T, C)
    pre = np.zeros((B, K - 1, C)) if cache is None else cache
    full = np.concatenate([pre, xf], axis=1)  # token t sits at row t + K - 1
    out = np.zeros((B, T, C))
    for t in range(T):
        for delta in range(K):
            out[:, t] += w[:, delta][None, :] * full[:, t + K - 1 - delta]
    return out.reshape(B, T, NH, d)


@pytest.mark.parametrize("T,K", [(1, 4), (3, 4), (9, 4), (17, 2), (6, 1), (12, 8)])
def test_conv_direct_sum(T, K):
    x, w = rnd(2, T, 3, 8), rnd(24, K)
    np.testing.assert_allclose(O.conv(x, w, None, K), brute_conv(x, w, None, K), rtol=0, atol=1e-13)
    cache = rnd(2, K - 1, 24)
    np.testing.assert_allclose(O.conv(x, w, cache, K), brute_conv(x, w, cache, K), rtol=0, atol=1e-13)


def test_conv_unit_taps_are_shifts():
    x = rnd(1, 10, 2, 4)
    for delta in range(4):
        w = np.zeros((8, 4))
        w[:, delta] = 1.0
        y = O.conv(x, w, None, 4)
        want = np.zeros_like(x)
        want[:, delta:] = x[:, : 10 - delta]
        assert np.array_equal(y, want)


def test_conv_cache_equals_prepended_tokens():
    K = 4
    x, w = rnd(2, 11, 2, 4), rnd(8, K)
    head, tail = x[:, : K - 1], x[:, K - 1:]
    full = O.conv(x, w, None, K)
    part = O.conv(tail, w, head.reshape(2, K - 1, 8), K)
    np.testing.assert_allclose(part, full[:, K - 1:], rtol=0, atol=1e-14)


def test_conv_linear_and_causal():
    K = 4
    x1, x2, w = rnd(1, 12, 2, 4), rnd(1, 12, 2, 4), rnd(8, K)
    np.testing.assert_allclose(O.conv(2 * x1 - 3 * x2, w, None, K),
                               2 * O.conv(x1, w, None, K) - 3 * O.conv(x2, w, None, K), atol=1e-13)
    x3 = x1.copy()
    x3[:, 7:] += rnd(1, 5, 2, 4)
    assert np.array_equal(O.conv(x3, w, None, K)[:, :7], O.conv(x1, w, None, K)[:, :7])


# --------------------------------------------------------------------------- mix + phi (Section 4.1)
def test_mix_identity_passthrough():
    u = rnd(2, 5, 3, 8)
    W = np.broadcast_to(np.eye(8), (3, 8, 8)).copy()
    assert np.array_equal(O.mix_phi(u, W, 3, O.PHI_IDENTITY), u)


def test_mix_against_library_routines():
    u, W = rnd(2, 7, 2, 8), rnd(4, 8, 8)
    y = np.einsum("btnc,nce->btne", np.repeat(u, 2, axis=2), W)  # head h reads input head h // 2
    np.testing.assert_allclose(O.mix_phi(u, W, 4, O.PHI_IDENTITY), y, atol=1e-13)
    np.testing.assert_allclose(O.mix_phi(u, W, 4, O.PHI_SOFTMAX), sp_softmax(y, axis=-1), atol=1e-14)
    np.testing.assert_allclose(O.mix_phi(u, W, 4, O.PHI_ELU1), np.where(y > 0, y + 1, np.exp(y)), atol=1e-14)


def test_softmax_phi_positive_and_normalised():
    p = O.mix_phi(5 * rnd(1, 9, 2, 16), rnd(2, 16, 16), 2, O.PHI_SOFTMAX)
    assert (p > 0).all()
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-14)


def test_same_map_for_query_and_key():
    # identical conv outputs pushed through the shared layer give identical features (Section 4.1)
    u, W = rnd(1, 6, 2, 8), rnd(2, 8, 8)
    assert np.array_equal(O.mix_phi(u, W, 2), O.mix_phi(u.copy(), W, 2))


# --------------------------------------------------------------------------- GLA forward (Eq. 4 - Eq. 8)
def quadratic_form(qd, kd, v, alpha, normalize=True):
    """Eq. 8 for one head with J_{i,t} built as an explicit running product of the gates (Eq. 6)."""
    T, dk = qd.shape
    o = np.zeros((T, v.shape[1]))
    den = np.zeros(T)
    for t in range(T):
        num = np.zeros(v.shape[1])
        dn = 0.0
        for i in range(t + 1):
            J = np.ones(dk)
            for zz in range(i + 1, t + 1):
                J = J * alpha[zz]
            wti = np.sum(qd[t] * J * kd[i])
            num += wti * v[i]
            dn += wti
        o[t] = num / dn if normalize else num
        den[t] = dn
    return o, den


@pytest.mark.parametrize("gate_dim,T", [(0, 1), (0, 13), (1, 24), (0, 40)])
def test_recurrence_equals_quadratic_form(gate_dim, T):
    H, dk, dv = 2, 6, 5
    p = O.OracleParams(1, T, H, H, dk, dv, gate_dim=gate_dim, gate_tau=2.0)
    qd, kd = np.abs(rnd(1, T, H, dk)), np.abs(rnd(1, T, H, dk))
    v, a = rnd(1, T, H, dv), 2 * rnd(1, T, H, p.gd)
    r = O.gla_fwd(p, qd, kd, v, a)
    alpha = np.broadcast_to(np.exp(logsigmoid(a) / 2.0), (1, T, H, dk))
    for h in range(H):
        o, den = quadratic_form(qd[0, :, h], kd[0, :, h], v[0, :, h], alpha[0, :, h])
        np.testing.assert_allclose(r["o"][0, :, h], o, rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(r["den"][0, :, h], den, rtol=1e-11)
    # numerator-only variant
    p0 = O.OracleParams(1, T, H, H, dk, dv, gate_dim=gate_dim, gate_tau=2.0, normalize=0)
    r0 = O.gla_fwd(p0, qd, kd, v, a)
    o0, _ = quadratic_form(qd[0, :, 1], kd[0, :, 1], v[0, :, 1], alpha[0, :, 1], normalize=False)
    np.testing.assert_allclose(r0["o"][0, :, 1], o0, rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("gate_dim", [0, 1])
def test_eps_sits_in_the_denominator_of_eq8(gate_dim):
    # Eq. 8 with eps: o_t = (sum_i w_ti v_i) / (sum_i w_ti + eps), w_ti = qdot_t . (J_{i,t} kdot_i); the weights are
    # built here from the explicit running product of the gates, eps is added to the explicit denominator only
    T, H, dk, dv, eps = 14, 2, 5, 4, 0.37
    p = O.OracleParams(1, T, H, H, dk, dv, gate_dim=gate_dim, gate_tau=2.0, eps=eps)
    qd, kd = np.abs(rnd(1, T, H, dk)), np.abs(rnd(1, T, H, dk))
    v, a = rnd(1, T, H, dv), 2 * rnd(1, T, H, p.gd)
    r = O.gla_fwd(p, qd, kd, v, a)
    alpha = np.broadcast_to(np.exp(logsigmoid(a) / 2.0), (1, T, H, dk))
    for h in range(H):
        num, den = quadratic_form(qd[0, :, h], kd[0, :, h], v[0, :, h], alpha[0, :, h], normalize=False)
        np.testing.assert_allclose(r["o"][0, :, h], num / (den + eps)[:, None], rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(r["den"][0, :, h], den + eps, rtol=1e-11)
    # a wrong place for eps (added to the numerator, or scaled by anything) would show against the eps = 0 result too
    r0 = O.gla_fwd(O.OracleParams(1, T, H, H, dk, dv, gate_dim=gate_dim, gate_tau=2.0), qd, kd, v, a)
    np.testing.assert_allclose(r["o"] * r["den"][..., None], r0["o"] * r0["den"][..., None], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(r["den"] - r0["den"], eps, rtol=1e-10)


@pytest.mark.parametrize("gate_dim,with_state", [(0, False), (1, True), (0, True)])
def test_final_state_equals_eq7_explicit_sum(gate_dim, with_state):
    # Eq. 7: S_T = J_{0,T} S_0 + sum_i J_{i,T} (kdot_i^T v_i), z_T likewise with 1 for v_i, where J_{i,T} is the
    # explicit product of the gates of tokens i+1..T (Eq. 6); a given initial state is decayed by every gate
    T, H, dk, dv = 11, 2, 4, 3
    p = O.OracleParams(1, T, H, H, dk, dv, gate_dim=gate_dim, gate_tau=2.0)
    qd, kd = np.abs(rnd(1, T, H, dk)), np.abs(rnd(1, T, H, dk))
    v, a = rnd(1, T, H, dv), 2 * rnd(1, T, H, p.gd)
    S0 = rnd(1, H, dk, dv) if with_state else None
    z0 = np.abs(rnd(1, H, dk)) if with_state else None
    r = O.gla_fwd(p, qd, kd, v, a, S0, z0)
    alpha = np.broadcast_to(np.exp(logsigmoid(a) / 2.0), (1, T, H, dk))
    for h in range(H):
        S, z = np.zeros((dk, dv)), np.zeros(dk)
        for i in range(-1, T):  # i = -1 stands for the given initial state
            J = np.ones(dk)
            for zz in range(i + 1, T):
                J = J * alpha[0, zz, h]
            if i < 0:
                if with_state:
                    S += J[:, None] * S0[0, h]
                    z += J * z0[0, h]
            else:
                S += J[:, None] * np.outer(kd[0, i, h], v[0, i, h])
                z += J * kd[0, i, h]
        np.testing.assert_allclose(r["S_T"][0, h], S, rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(r["z_T"][0, h], z, rtol=1e-11, atol=1e-13)


def test_zero_decay_is_kernel_linear_attention():
    # all gates 1 -> Eq. 2 by direct double sum
    T, dk, dv = 19, 5, 4
    p = O.OracleParams(1, T, 1, 1, dk, dv, gate_mode=O.GATE_LOGDECAY)
    qd, kd, v = np.abs(rnd(1, T, 1, dk)), np.abs(rnd(1, T, 1, dk)), rnd(1, T, 1, dv)
    r = O.gla_fwd(p, qd, kd, v, np.zeros((1, T, 1, dk)))
    for t in range(T):
        wts = np.array([qd[0, t, 0] @ kd[0, i, 0] for i in range(t + 1)])
        want = (wts[:, None] * v[0, : t + 1, 0]).sum(0) / wts.sum()
        np.testing.assert_allclose(r["o"][0, t, 0], want, rtol=1e-12, atol=1e-14)


def test_total_decay_returns_current_value():
    # alpha = 0: S_t = kdot_t^T v_t, so o_t = v_t exactly up to one rounding of the division
    T, dk, dv = 9, 4, 6
    p = O.OracleParams(1, T, 1, 1, dk, dv, gate_mode=O.GATE_LOGDECAY)
    qd, kd, v = np.abs(rnd(1, T, 1, dk)), np.abs(rnd(1, T, 1, dk)), rnd(1, T, 1, dv)
    r = O.gla_fwd(p, qd, kd, v, np.full((1, T, 1, dk), -1e9))
    np.testing.assert_allclose(r["o"], v, rtol=1e-14)


def test_normaliser_properties():
    T, H, dk, dv = 30, 2, 8, 7
    p = O.OracleParams(2, T, H, 1, dk, dv)
    qd, kd = np.abs(rnd(2, T, H, dk)) + 0.1, np.abs(rnd(2, T, H, dk)) + 0.1
    v, a = rnd(2, T, 1, dv), rnd(2, T, H, dk)
    o = O.gla_fwd(p, qd, kd, v, a)["o"]
    np.testing.assert_allclose(o[:, 0], np.repeat(v[:, 0], H, axis=1), rtol=1e-14)  # first output is v_1
    vmin = np.minimum.accumulate(v, axis=1)
    vmax = np.maximum.accumulate(v, axis=1)
    assert (o >= vmin - 1e-12).all() and (o <= vmax + 1e-12).all()                 # convex combination of values
    const = np.broadcast_to(rnd(1, 1, 1, dv), v.shape).copy()
    oc = O.gla_fwd(p, qd, kd, const, a)["o"]
    np.testing.assert_allclose(oc, np.broadcast_to(const[:, :, :1], oc.shape), rtol=1e-12)
    o_scaled = O.gla_fwd(p, 3.7 * qd, kd, v, a)["o"]                               # scale of qdot cancels
    np.testing.assert_allclose(o_scaled, o, rtol=1e-12, atol=1e-14)


def test_causality_bitwise():
    T, t0 = 21, 12
    sh = dict(B=1, T=T, H=2, H_kv=1, d_k=8, d_v=8)
    p = O.OracleParams(**sh)
    q, k, v, a = rnd(1, T, 2, 8), rnd(1, T, 1, 8), rnd(1, T, 1, 8), rnd(1, T, 2, 8)
    wq, wk, W = rnd(16, 4), rnd(8, 4), rnd(2, 8, 8)
    base = O.layer_fwd(p, q, k, v, a, wq, wk, W)["o"]
    q2, k2, v2, a2 = q.copy(), k.copy(), v.copy(), a.copy()
    for x in (q2, k2, v2, a2):
        x[:, t0 + 1:] += rnd(*x[:, t0 + 1:].shape)
    pert = O.layer_fwd(p, q2, k2, v2, a2, wq, wk, W)["o"]
    assert np.array_equal(base[:, : t0 + 1], pert[:, : t0 + 1])
    assert not np.array_equal(base[:, t0 + 1:], pert[:, t0 + 1:])


def _layer_inputs(B, T, H, Hkv, dk, dv, gd=0):
    gd = gd or dk
    return dict(q=rnd(B, T, H, dk), k=rnd(B, T, Hkv, dk), v=rnd(B, T, Hkv, dv), gate=rnd(B, T, H, gd),
                w_q=rnd(H * dk, 4) / 2, w_k=rnd(Hkv * dk, 4) / 2, W=rnd(H, dk, dk) / np.sqrt(dk))


@pytest.mark.parametrize("split", [1, 2, 3, 10])
def test_split_calls_carry_state_and_caches(split):
    B, T, H, Hkv, dk, dv = 2, 17, 4, 2, 8, 6
    x = _layer_inputs(B, T, H, Hkv, dk, dv)
    full = O.layer_fwd(O.OracleParams(B, T, H, Hkv, dk, dv), **x)
    sl = lambda a, lo, hi: a[:, lo:hi]
    r1 = O.layer_fwd(O.OracleParams(B, split, H, Hkv, dk, dv), sl(x["q"], 0, split), sl(x["k"], 0, split),
                     sl(x["v"], 0, split), sl(x["gate"], 0, split), x["w_q"], x["w_k"], x["W"])
    r2 = O.layer_fwd(O.OracleParams(B, T - split, H, Hkv, dk, dv), sl(x["q"], split, T), sl(x["k"], split, T),
                     sl(x["v"], split, T), sl(x["gate"], split, T), x["w_q"], x["w_k"], x["W"],
                     r1["cache_q"], r1["cache_k"], r1["S_T"], r1["z_T"])
    np.testing.assert_allclose(np.concatenate([r1["o"], r2["o"]], 1), full["o"], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(r2["S_T"], full["S_T"], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(r2["z_T"], full["z_T"], rtol=1e-12)
    assert np.array_equal(r2["cache_q"], full["cache_q"]) and np.array_equal(r2["cache_k"], full["cache_k"])
    assert np.array_equal(full["cache_q"], x["q"][:, -3:].reshape(B, 3, -1))


def test_decode_steps_equal_prefill():
    B, T, H, Hkv, dk, dv = 2, 9, 4, 2, 8, 8
    x = _layer_inputs(B, T, H, Hkv, dk, dv, gd=1)
    p = O.OracleParams(B, T, H, Hkv, dk, dv, gate_dim=1)
    full = O.layer_fwd(p, **x)
    S, z = np.zeros((B, H, dk, dv)), np.zeros((B, H, dk))
    cq, ck = np.zeros((B, 3, H * dk)), np.zeros((B, 3, Hkv * dk))
    for t in range(T):
        r = O.decode_step(p, x["q"][:, t], x["k"][:, t], x["v"][:, t], x["gate"][:, t], x["w_q"], x["w_k"],
                          x["W"], S, z, cq, ck)
        np.testing.assert_allclose(r["o"], full["o"][:, t], rtol=1e-12, atol=1e-14)
        S, z, cq, ck = r["S"], r["z"], r["cache_q"], r["cache_k"]
    np.testing.assert_allclose(S, full["S_T"], rtol=1e-12, atol=1e-14)


def test_gqa_equals_mha_with_repeated_kv():
    B, T, H, Hkv, dk, dv = 1, 11, 4, 2, 8, 8
    x = _layer_inputs(B, T, H, Hkv, dk, dv)
    a = O.layer_fwd(O.OracleParams(B, T, H, Hkv, dk, dv), **x)["o"]
    y = dict(x)
    y["k"] = np.repeat(x["k"], 2, axis=2)
    y["v"] = np.repeat(x["v"], 2, axis=2)
    y["w_k"] = np.repeat(x["w_k"].reshape(Hkv, dk, 4), 2, axis=0).reshape(H * dk, 4)
    b = O.layer_fwd(O.OracleParams(B, T, H, H, dk, dv), **y)["o"]
    np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-15)


# --------------------------------------------------------------------------- gradients
def _fd(fun, x, dO, h=1e-6):
    """Central finite differences of sum(dO * fun(x)) with respect to every entry of x."""
    g = np.zeros_like(x)
    flat, gf = x.reshape(-1), g.reshape(-1)
    for i in range(flat.size):
        old = flat[i]
        flat[i] = old + h
        fp = np.sum(dO * fun())
        flat[i] = old - h
        fm = np.sum(dO * fun())
        flat[i] = old
        gf[i] = (fp - fm) / (2 * h)
    return g


@pytest.mark.parametrize("gate_dim,gate_mode,normalize,with_state",
                         [(0, O.GATE_LOGITS, 1, False), (1, O.GATE_LOGITS, 1, True),
                          (0, O.GATE_LOGDECAY, 1, True), (0, O.GATE_LOGITS, 0, False)])
def test_gla_bwd_finite_differences(gate_dim, gate_mode, normalize, with_state):
    B, T, H, Hkv, dk, dv = 1, 6, 2, 1, 4, 3
    p = O.OracleParams(B, T, H, Hkv, dk, dv, gate_dim=gate_dim, gate_mode=gate_mode, normalize=normalize,
                       gate_tau=2.0)
    qd, kd = np.abs(rnd(B, T, H, dk)) + 0.2, np.abs(rnd(B, T, H, dk)) + 0.2
    v, dO = rnd(B, T, Hkv, dv), rnd(B, T, H, dv)
    a = rnd(B, T, H, p.gd)
    if gate_mode == O.GATE_LOGDECAY:
        a = -np.abs(a) * 0.3
    S0 = np.abs(rnd(B, H, dk, dv)) if with_state else None
    z0 = np.abs(rnd(B, H, dk)) + 0.5 if with_state else None
    g = O.gla_bwd(p, qd, kd, v, a, dO, S0, z0)
    f = lambda: O.gla_fwd(p, qd, kd, v, a, S0, z0)["o"]
    for name, x in (("d_qdot", qd), ("d_kdot", kd), ("dv", v), ("dgate", a)):
        np.testing.assert_allclose(g[name], _fd(f, x, dO), rtol=2e-6, atol=1e-8, err_msg=name)


@pytest.mark.parametrize("gate_dim", [0, 1])
def test_gla_bwd_finite_differences_with_eps(gate_dim):
    # eps = 0.3 is of the size of the denominators here: a misplaced eps in the backward (in do' or in the
    # -(dO . o) / d term) changes every gradient by tens of percent
    B, T, H, Hkv, dk, dv = 1, 6, 2, 1, 4, 3
    p = O.OracleParams(B, T, H, Hkv, dk, dv, gate_dim=gate_dim, gate_tau=2.0, eps=0.3)
    qd, kd = np.abs(rnd(B, T, H, dk)) * 0.3 + 0.05, np.abs(rnd(B, T, H, dk)) * 0.3 + 0.05
    v, dO, a = rnd(B, T, Hkv, dv), rnd(B, T, H, dv), rnd(B, T, H, p.gd)
    S0, z0 = np.abs(rnd(B, H, dk, dv)) * 0.2, np.abs(rnd(B, H, dk)) * 0.2
    g = O.gla_bwd(p, qd, kd, v, a, dO, S0, z0)
    f = lambda: O.gla_fwd(p, qd, kd, v, a, S0, z0)["o"]
    for name, x in (("d_qdot", qd), ("d_kdot", kd), ("dv", v), ("dgate", a)):
        np.testing.assert_allclose(g[name], _fd(f, x, dO), rtol=2e-6, atol=1e-8, err_msg=name)
    g0 = O.gla_bwd(O.OracleParams(B, T, H, Hkv, dk, dv, gate_dim=gate_dim, gate_tau=2.0), qd, kd, v, a, dO, S0, z0)
    assert np.abs(g["d_qdot"] - g0["d_qdot"]).max() > 0.05 * np.abs(g0["d_qdot"]).max()  # eps matters at this size


def test_gate_gradient_reverse_cumsum_identity():
    # o' depends on the log-decays only through their running sum, hence
    # dg_s = sum_{t>=s} (qdot_t * dqdot_t - kdot_t * dkdot_t)
    B, T, H, dk, dv = 1, 12, 2, 5, 4
    p = O.OracleParams(B, T, H, H, dk, dv, gate_mode=O.GATE_LOGDECAY)
    qd, kd = np.abs(rnd(B, T, H, dk)) + 0.1, np.abs(rnd(B, T, H, dk)) + 0.1
    v, dO, g_in = rnd(B, T, H, dv), rnd(B, T, H, dv), -np.abs(rnd(B, T, H, dk)) * 0.2
    g = O.gla_bwd(p, qd, kd, v, g_in, dO)
    per_t = qd * g["d_qdot"] - kd * g["d_kdot"]
    want = np.flip(np.cumsum(np.flip(per_t, 1), 1), 1)
    np.testing.assert_allclose(g["dgate"], want, rtol=1e-10, atol=1e-12)


def test_value_shift_identity():
    # v -> v + c shifts every o_t by c (weights sum to one), so sum_t dv = sum_{t,h} dO per value channel
    B, T, H, Hkv, dk, dv = 2, 10, 4, 2, 4, 5
    p = O.OracleParams(B, T, H, Hkv, dk, dv)
    qd, kd = np.abs(rnd(B, T, H, dk)) + 0.1, np.abs(rnd(B, T, H, dk)) + 0.1
    v, dO, a = rnd(B, T, Hkv, dv), rnd(B, T, H, dv), rnd(B, T, H, dk)
    g = O.gla_bwd(p, qd, kd, v, a, dO)
    want = dO.reshape(B, T, Hkv, 2, dv).sum(axis=(1, 3))  # per (b, kv head, channel)
    np.testing.assert_allclose(g["dv"].sum(axis=1), want, rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("phi,with_cache,with_mix",
                         [(O.PHI_SOFTMAX, False, True), (O.PHI_ELU1, True, True), (O.PHI_IDENTITY, True, True),
                          (O.PHI_SOFTMAX, True, False)])
def test_conv_bwd_finite_differences(phi, with_cache, with_mix):
    B, T, H, Hkv, d, K = 1, 5, 2, 1, 3, 3
    p = O.OracleParams(B, T, H, Hkv, d, d, conv_k=K, phi=phi)
    q, k = rnd(B, T, H, d), rnd(B, T, Hkv, d)
    wq, wk = rnd(H * d, K), rnd(Hkv * d, K)
    W = rnd(H, d, d) if with_mix else None
    cq = rnd(B, K - 1, H * d) if with_cache else None
    ck = rnd(B, K - 1, Hkv * d) if with_cache else None
    dqd = rnd(B, T, H, d)
    dkd = rnd(B, T, H if with_mix else Hkv, d)
    g = O.conv_bwd(p, q, k, wq, wk, W, dqd, dkd, cq, ck)

    def fq():
        u = O.conv(q, wq, cq, K)
        return O.mix_phi(u, W, H, phi) if with_mix else u

    def fk():
        u = O.conv(k, wk, ck, K)
        return O.mix_phi(u, W, H, phi) if with_mix else u

    np.testing.assert_allclose(g["dq"], _fd(fq, q, dqd), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(g["dk"], _fd(fk, k, dkd), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(g["dw_q"], _fd(fq, wq, dqd), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(g["dw_k"], _fd(fk, wk, dkd), rtol=2e-6, atol=1e-8)
    if with_mix:
        total = lambda: np.concatenate([fq().ravel(), fk().ravel()])
        dboth = np.concatenate([dqd.ravel(), dkd.ravel()])
        np.testing.assert_allclose(g["dW"], _fd(total, W, dboth), rtol=2e-6, atol=1e-8)


def test_whole_layer_gradient_chain():
    # composition gla_bwd -> conv_bwd against finite differences of the whole layer forward
    B, T, H, Hkv, d = 1, 5, 2, 1, 3
    p = O.OracleParams(B, T, H, Hkv, d, d, gate_tau=1.0)
    x = _layer_inputs(B, T, H, Hkv, d, d)
    dO = rnd(B, T, H, d)
    fwd = O.layer_fwd(p, **x)
    g1 = O.gla_bwd(p, fwd["qdot"], fwd["kdot"], x["v"], x["gate"], dO)
    g2 = O.conv_bwd(p, x["q"], x["k"], x["w_q"], x["w_k"], x["W"], g1["d_qdot"], g1["d_kdot"])
    f = lambda: O.layer_fwd(p, **x)["o"]
    for name, got in (("q", g2["dq"]), ("k", g2["dk"]), ("v", g1["dv"]), ("gate", g1["dgate"]),
                      ("w_q", g2["dw_q"]), ("w_k", g2["dw_k"]), ("W", g2["dW"])):
        np.testing.assert_allclose(got, _fd(f, x[name], dO), rtol=5e-6, atol=1e-8, err_msg=name)


# --------------------------------------------------------------------------- a separate linear layer per stream
def test_unshared_linear_with_equal_matrices_is_the_shared_layer():
    """Appendix table on sharing: the unshared form with W_q = W_k is the shared layer, and its two weight gradients add
    up to the shared one."""
    B, T, H, Hkv, d = 2, 7, 4, 2, 3
    p = O.OracleParams(B, T, H, Hkv, d, d)
    x = _layer_inputs(B, T, H, Hkv, d, d)
    a = O.layer_fwd(p, **x)
    y = dict(x)
    y["W"] = np.stack([x["W"], x["W"]])
    b = O.layer_fwd(p, **y)
    for n in ("o", "qdot", "kdot", "S_T", "z_T", "cache_q", "cache_k"):
        np.testing.assert_allclose(b[n], a[n], rtol=1e-13, atol=1e-15, err_msg=n)
    dqd, dkd = rnd(B, T, H, d), rnd(B, T, H, d)
    g = O.conv_bwd(p, x["q"], x["k"], x["w_q"], x["w_k"], x["W"], dqd, dkd)
    gu = O.conv_bwd(p, x["q"], x["k"], x["w_q"], x["w_k"], y["W"], dqd, dkd)
    np.testing.assert_allclose(gu["dW"][0] + gu["dW"][1], g["dW"], rtol=1e-12, atol=1e-14)
    for n in ("dq", "dk", "dw_q", "dw_k"):
        np.testing.assert_allclose(gu[n], g[n], rtol=1e-13, atol=1e-15, err_msg=n)


def test_unshared_linear_streams_are_independent_and_gradients_match_finite_differences():
    B, T, H, Hkv, d, K = 1, 5, 2, 1, 3, 3
    p = O.OracleParams(B, T, H, Hkv, d, d, conv_k=K, gate_tau=1.0)
    q, k, v, gate = rnd(B, T, H, d), rnd(B, T, Hkv, d), rnd(B, T, Hkv, d), rnd(B, T, H, d)
    wq, wk, W = rnd(H * d, K), rnd(Hkv * d, K), rnd(2, H, d, d)
    base = O.layer_fwd(p, q, k, v, gate, wq, wk, W)
    # the key stream's matrices do not touch qdot, and the other way round
    W2 = W.copy()
    W2[1] += 0.5
    np.testing.assert_array_equal(O.layer_fwd(p, q, k, v, gate, wq, wk, W2)["qdot"], base["qdot"])
    W3 = W.copy()
    W3[0] += 0.5
    np.testing.assert_array_equal(O.layer_fwd(p, q, k, v, gate, wq, wk, W3)["kdot"], base["kdot"])
    # whole-layer gradient chain against finite differences
    dO = rnd(B, T, H, d)
    g1 = O.gla_bwd(p, base["qdot"], base["kdot"], v, gate, dO)
    g2 = O.conv_bwd(p, q, k, wq, wk, W, g1["d_qdot"], g1["d_kdot"])
    f = lambda: O.layer_fwd(p, q, k, v, gate, wq, wk, W)["o"]
    for name, arr, got in (("q", q, g2["dq"]), ("k", k, g2["dk"]), ("w_q", wq, g2["dw_q"]), ("w_k", wk, g2["dw_k"]),
                           ("W", W, g2["dW"])):
        np.testing.assert_allclose(got, _fd(f, arr, dO), rtol=5e-6, atol=1e-8, err_msg=name)


# ---- gate function (Section 4.2; appendix on the rank of the gate function) -------------------------------------------
def _gate_fn_inputs(B=2, T=5, dm=12, rank=3, n_out=8, seed=77):
    g = np.random.default_rng(seed)
    return (g.standard_normal((B, T, dm)), g.standard_normal((rank, dm)), g.standard_normal((n_out, rank)),
            g.standard_normal(n_out))


def test_gate_function_brute_force_sums():
    """Every logit written out as the double sum over the bottleneck units and the hidden channels."""
    x, A1, A2, b = _gate_fn_inputs()
    got = O.gate_logits(x, A1, A2, b)
    for bb in range(x.shape[0]):
        for t in range(x.shape[1]):
            for j in range(A2.shape[0]):
                want = b[j]
                for r in range(A1.shape[0]):
                    hr = 0.0
                    for c in range(A1.shape[1]):
                        hr += A1[r, c] * x[bb, t, c]
                    want += A2[j, r] * hr
                assert abs(got[bb, t, j] - want) <= 1e-12 * (1 + abs(want))


def test_gate_function_is_one_matrix_of_bounded_rank():
    """Two consecutive linear layers are the single linear layer A2 A1 (library product), whose rank is at most the
    bottleneck width; without a bias the map is linear in x."""
    x, A1, A2, b = _gate_fn_inputs(rank=3)
    M = A2 @ A1
    assert np.linalg.matrix_rank(M) <= 3
    np.testing.assert_allclose(O.gate_logits(x, A1, A2, None), np.einsum("jc,btc->btj", M, x), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(O.gate_logits(x, A1, A2, b) - O.gate_logits(x, A1, A2, None),
                               np.broadcast_to(b, (2, 5, 8)), rtol=0, atol=1e-12)
    y = np.random.default_rng(5).standard_normal(x.shape)
    np.testing.assert_allclose(O.gate_logits(2.0 * x - 3.0 * y, A1, A2, None),
                               2.0 * O.gate_logits(x, A1, A2, None) - 3.0 * O.gate_logits(y, A1, A2, None),
                               rtol=1e-11, atol=1e-11)


def test_gate_function_special_cases():
    """Rank 1: logit j of token t is (u . x_t) w_j. Full rank with an identity first layer: a plain linear layer.
    A transposed operand or swapped layers would change the shape or the value in each of these."""
    g = np.random.default_rng(3)
    x = g.standard_normal((1, 4, 6)); u = g.standard_normal((1, 6)); w = g.standard_normal((5, 1))
    got = O.gate_logits(x, u, w)
    for t in range(4):
        np.testing.assert_allclose(got[0, t], float(u[0] @ x[0, t]) * w[:, 0], rtol=1e-12)
    A2 = g.standard_normal((5, 6)); b = g.standard_normal(5)
    np.testing.assert_allclose(O.gate_logits(x, np.eye(6), A2, b), x @ A2.T + b, rtol=1e-12, atol=1e-12)
    # a first layer that picks hidden channel 2 and a second layer that routes it to logit 4 only
    A1 = np.zeros((1, 6)); A1[0, 2] = 1.0
    A2 = np.zeros((5, 1)); A2[4, 0] = 2.0
    want = np.zeros((1, 4, 5)); want[0, :, 4] = 2.0 * x[0, :, 2]
    np.testing.assert_array_equal(O.gate_logits(x, A1, A2), want)


def test_gate_function_feeds_the_decay_of_eq4():
    """The logits are the layer's `gate` input: through gla_fwd the decay of channel c at token t is
    sigmoid(a_tc)^(1/tau) (Section 4.2). One token after a known state isolates it."""
    x, A1, A2, b = _gate_fn_inputs(B=1, T=1, dm=7, rank=2, n_out=2 * 4)
    a = O.gate_logits(x, A1, A2, b).reshape(1, 1, 2, 4)
    p = O.OracleParams(1, 1, 2, 2, 4, 4, gate_tau=3.0)
    S0 = np.ones((1, 2, 4, 4)); z0 = np.ones((1, 2, 4))
    zero = np.zeros((1, 1, 2, 4))
    r = O.gla_fwd(p, zero + 1.0, zero, zero, a, S0, z0)     # k = 0: the state only decays
    alpha = (1.0 / (1.0 + np.exp(-a[0, 0]))) ** (1.0 / 3.0)  # [H, d_k]
    np.testing.assert_allclose(r["S_T"][0], alpha[:, :, None] * S0[0], rtol=1e-12)
    np.testing.assert_allclose(r["z_T"][0], alpha * z0[0], rtol=1e-12)


def test_gate_log_decay_is_the_log_of_the_gate():
    """exp(log-decay) = sigmoid(a)^(1/tau) by the textbook sigmoid (moderate logits), the far tails behave like a / tau and
    like -exp(-a) / tau, and the layer run on log-decays (GATE_LOGDECAY) equals the layer run on the logits themselves."""
    a = np.linspace(-20.0, 20.0, 81)
    for tau in (1.0, 3.0, 16.0):
        g = O.gate_log_decay(a, tau)
        np.testing.assert_allclose(np.exp(g), (1.0 / (1.0 + np.exp(-a))) ** (1.0 / tau), rtol=1e-12)
        assert (g < 0).all() and (np.diff(g) > 0).all()
    np.testing.assert_allclose(O.gate_log_decay(np.array([-800.0]), 4.0), [-200.0], rtol=1e-12)
    np.testing.assert_allclose(O.gate_log_decay(np.array([40.0]), 2.0), [-np.exp(-40.0) / 2.0], rtol=1e-9)
    g = np.random.default_rng(8)
    B, T, H, d = 1, 9, 2, 4
    q, k, v = (np.abs(g.standard_normal((B, T, H, d))) for _ in range(3))
    logits = 2.0 * g.standard_normal((B, T, H, d))
    r0 = O.gla_fwd(O.OracleParams(B, T, H, H, d, d, gate_tau=5.0), q, k, v, logits)
    r1 = O.gla_fwd(O.OracleParams(B, T, H, H, d, d, gate_mode=O.GATE_LOGDECAY), q, k, v, O.gate_log_decay(logits, 5.0))
    for n in ("o", "S_T", "z_T"):
        np.testing.assert_allclose(r1[n], r0[n], rtol=1e-11, atol=1e-13)
