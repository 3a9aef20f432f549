/*
 * lawcat_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what the LAWCAT layer computes, written from the paper's equations in the
 * paper's order: token by token, no chunking, no fusion. Only tests, the smoke check and the CPU-baseline leg of the
 * benchmark may call it. It shares no code, header, table or helper with the CUDA library.
 *
 * Pin status (what the CPU tests check each function against):
 *   oracle_conv          direct-sum brute force, unit taps = shifts, cache == prepended tokens      (pinned)
 *   oracle_mix_phi       identity pass-through, softmax rows sum to 1, library matmul               (pinned)
 *   oracle_gla_fwd       quadratic form of Eq. 8 with J as an explicit running product, zero-decay
 *                        reduction to Eq. 2, alpha = 0 reduction to o_t = v_t, convex-combination
 *                        bounds, causality, split-call state hand-off; eps against the explicit
 *                        denominator of Eq. 8; S_T, z_T against the explicit sum of Eq. 7           (pinned)
 *   oracle_gla_bwd       central finite differences of oracle_gla_fwd (eps = 0 and eps = 0.3),
 *                        reverse-cumsum gate identity, value-shift identity                         (pinned)
 *   oracle_conv_bwd      central finite differences of oracle_conv + oracle_mix_phi                 (pinned)
 *   choice of phi, gate_tau, eps: the paper does not fix them -> parameters; parity unpinned by the paper.
 *
 * Layouts (row-major, last index fastest), G = H / H_kv:
 *   q, qdot, kdot [B,T,H,d_k]   k [B,T,H_kv,d_k]   v [B,T,H_kv,d_v]   gate [B,T,H,gate_dim]   o [B,T,H,d_v]
 *   w [(head*d + c)*K + delta]   W [H,d_k,d_k] (y[e] = sum_c u[c] W[h][c][e])
 *   S [B,H,d_k,d_v]   z [B,H,d_k]   conv cache [B,K-1,heads*d_k] (raw tokens before t=0, oldest first)
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int B, T, H, H_kv, d_k, d_v, conv_k, gate_dim;
  int phi;       /* 0 softmax over the d_k outputs, 1 = 1+ELU, 2 identity */
  int gate_mode; /* 0: g = logsigmoid(gate)/tau ; 1: g = gate */
  int normalize; /* 1: Eq. 8 ; 0: numerator only */
  double gate_tau, eps;
} oracle_params;

int oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---- Section 4.1: causal depthwise Conv1D, xtilde_t = sum_{delta=0..r} w_delta x_{t-delta} ---------------- */
void oracle_conv(const double* x, const double* w, const double* cache, int B, int T, int NH, int d, int K,
                 double* out) {
  const long C = (long)NH * d;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < T; ++t)
      for (long c = 0; c < C; ++c) {
        double acc = 0.0;
        for (int delta = 0; delta < K; ++delta) {
          int s = t - delta;
          double xv;
          if (s >= 0) xv = x[((long)b * T + s) * C + c];
          else if (cache) xv = cache[((long)b * (K - 1) + (s + K - 1)) * C + c];
          else xv = 0.0;
          acc += w[c * K + delta] * xv;
        }
        out[((long)b * T + t) * C + c] = acc;
      }
}

static void phi_forward(const double* y, int d, int phi, double* p) {
  if (phi == 0) {
    double m = y[0], s = 0.0;
    for (int e = 1; e < d; ++e) if (y[e] > m) m = y[e];
    for (int e = 0; e < d; ++e) { p[e] = exp(y[e] - m); s += p[e]; }
    for (int e = 0; e < d; ++e) p[e] /= s;
  } else if (phi == 1) {
    for (int e = 0; e < d; ++e) p[e] = y[e] > 0.0 ? y[e] + 1.0 : exp(y[e]);
  } else {
    for (int e = 0; e < d; ++e) p[e] = y[e];
  }
}

/* ---- Section 4.1: shared linear layer + nonlinearity. u [B,T,NH_in,d] -> out [B,T,H,d], head h reads input head
 *      h / (H/NH_in) and weights W[h] (the same W[h] for the query and the key stream). ------------------------- */
void oracle_mix_phi(const double* u, const double* W, int B, int T, int NH_in, int H, int d, int phi,
                    double* out) {
  const int G = H / NH_in;
#pragma omp parallel for collapse(2)
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < T; ++t) {
      double* y = (double*)malloc(sizeof(double) * d);
      for (int h = 0; h < H; ++h) {
        const double* ur = u + (((long)b * T + t) * NH_in + h / G) * d;
        const double* Wh = W + (long)h * d * d;
        for (int e = 0; e < d; ++e) {
          double acc = 0.0;
          for (int c = 0; c < d; ++c) acc += ur[c] * Wh[(long)c * d + e];
          y[e] = acc;
        }
        phi_forward(y, d, phi, out + (((long)b * T + t) * H + h) * d);
      }
      free(y);
    }
}

/* log-decay of one gate entry: logsigmoid(a)/tau (Section 4.2, "sigmoid activation") or a itself */
static double log_decay(double a, int gate_mode, double tau) {
  if (gate_mode == 1) return a;
  double ls = (a < 0.0 ? a : 0.0) - log1p(exp(-fabs(a))); /* log sigmoid(a) */
  return ls / tau;
}

/* ---- Eq. 4 + Eq. 8, one token at a time -------------------------------------------------------------------- */
void oracle_gla_fwd(const oracle_params* p, const double* qdot, const double* kdot, const double* v,
                    const double* gate, const double* S0, const double* z0, double* o, double* den, double* S_T,
                    double* z_T) {
  const int B = p->B, T = p->T, H = p->H, Hkv = p->H_kv, dk = p->d_k, dv = p->d_v, gd = p->gate_dim;
  const int G = H / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < H; ++h) {
      double* S = (double*)calloc((size_t)dk * dv, sizeof(double));
      double* z = (double*)calloc((size_t)dk, sizeof(double));
      double* num = (double*)malloc(sizeof(double) * dv);
      if (S0) memcpy(S, S0 + ((long)b * H + h) * dk * dv, sizeof(double) * dk * dv);
      if (z0) memcpy(z, z0 + ((long)b * H + h) * dk, sizeof(double) * dk);
      for (int t = 0; t < T; ++t) {
        const long th = ((long)b * T + t) * H + h;
        const double* qd = qdot + th * dk;
        const double* kd = kdot + th * dk;
        const double* vt = v + (((long)b * T + t) * Hkv + h / G) * dv;
        const double* gt = gate + th * gd;
        /* S_t = G_t (.) S_{t-1} + kdot_t^T v_t ;  z_t = alpha_t (.) z_{t-1} + kdot_t */
        for (int c = 0; c < dk; ++c) {
          double alpha = exp(log_decay(gt[gd == 1 ? 0 : c], p->gate_mode, p->gate_tau));
          for (int e = 0; e < dv; ++e) S[(long)c * dv + e] = alpha * S[(long)c * dv + e] + kd[c] * vt[e];
          z[c] = alpha * z[c] + kd[c];
        }
        /* o_t = qdot_t S_t / (qdot_t . z_t + eps) */
        double dn = p->eps;
        for (int c = 0; c < dk; ++c) dn += qd[c] * z[c];
        for (int e = 0; e < dv; ++e) num[e] = 0.0;
        for (int c = 0; c < dk; ++c)
          for (int e = 0; e < dv; ++e) num[e] += qd[c] * S[(long)c * dv + e];
        for (int e = 0; e < dv; ++e) o[th * dv + e] = p->normalize ? num[e] / dn : num[e];
        if (den) den[th] = dn;
      }
      if (S_T) memcpy(S_T + ((long)b * H + h) * dk * dv, S, sizeof(double) * dk * dv);
      if (z_T) memcpy(z_T + ((long)b * H + h) * dk, z, sizeof(double) * dk);
      free(S); free(z); free(num);
    }
}

/* ---- Backward of Eq. 4 + Eq. 8 by the chain rule, as a reverse recurrence.
 * With v' = [v, 1], S' = [S, z] (d_k x (d_v+1)) and o' = qdot S' = [n, d]:
 *   do'_t = [dO_t / d_t, -(dO_t . o_t) / d_t]           (normalize = 0: [dO_t, 0])
 *   for t = T..1:  dS' += qdot_t^T do'_t ; dqdot_t = do'_t S'_t^T ; dkdot_t = dS' v'_t ; dv'_t = kdot_t dS' ;
 *                  dalpha_t = rowsum(dS' (.) S'_{t-1}) ; dS' <- diag(alpha_t) dS'
 *   dg_t = dalpha_t (.) alpha_t ; logits mode: dgate = dg (1 - sigmoid(a)) / tau
 * All S'_t of one (b,h) are kept in memory; this is test infrastructure for small T. */
void oracle_gla_bwd(const oracle_params* p, const double* qdot, const double* kdot, const double* v,
                    const double* gate, const double* S0, const double* z0, const double* dO, double* d_qdot,
                    double* d_kdot, double* d_v, double* d_gate) {
  const int B = p->B, T = p->T, H = p->H, Hkv = p->H_kv, dk = p->d_k, dv = p->d_v, gd = p->gate_dim;
  const int G = H / Hkv, dv1 = dv + 1;
  memset(d_v, 0, sizeof(double) * (size_t)B * T * Hkv * dv);
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int b = 0; b < B; ++b)
    for (int j = 0; j < Hkv; ++j)
      for (int h = j * G; h < (j + 1) * G; ++h) { /* heads of one group run in sequence: they share d_v */
        const size_t SZ = (size_t)dk * dv1;
        double* Sall = (double*)calloc(SZ * (size_t)(T + 1), sizeof(double)); /* S'_0 .. S'_T */
        double* dS = (double*)calloc(SZ, sizeof(double));
        double* alpha = (double*)malloc(sizeof(double) * (size_t)T * dk);
        double* dop = (double*)malloc(sizeof(double) * dv1);
        if (S0) for (int c = 0; c < dk; ++c)
          for (int e = 0; e < dv; ++e) Sall[(size_t)c * dv1 + e] = S0[(((long)b * H + h) * dk + c) * dv + e];
        if (z0) for (int c = 0; c < dk; ++c) Sall[(size_t)c * dv1 + dv] = z0[((long)b * H + h) * dk + c];
        for (int t = 0; t < T; ++t) {
          const long th = ((long)b * T + t) * H + h;
          const double* kd = kdot + th * dk;
          const double* vt = v + (((long)b * T + t) * Hkv + j) * dv;
          const double* Sp = Sall + SZ * (size_t)t;
          double* Sn = Sall + SZ * (size_t)(t + 1);
          for (int c = 0; c < dk; ++c) {
            double a = exp(log_decay(gate[th * gd + (gd == 1 ? 0 : c)], p->gate_mode, p->gate_tau));
            alpha[(size_t)t * dk + c] = a;
            for (int e = 0; e < dv; ++e) Sn[(size_t)c * dv1 + e] = a * Sp[(size_t)c * dv1 + e] + kd[c] * vt[e];
            Sn[(size_t)c * dv1 + dv] = a * Sp[(size_t)c * dv1 + dv] + kd[c];
          }
        }
        for (int t = T - 1; t >= 0; --t) {
          const long th = ((long)b * T + t) * H + h;
          const double* qd = qdot + th * dk;
          const double* kd = kdot + th * dk;
          const double* vt = v + (((long)b * T + t) * Hkv + j) * dv;
          const double* dOt = dO + th * dv;
          const double* Sp = Sall + SZ * (size_t)t;
          const double* Sn = Sall + SZ * (size_t)(t + 1);
          /* o'_t = qdot_t S'_t */
          double dn = p->eps, dot_dO_o = 0.0;
          for (int c = 0; c < dk; ++c) dn += qd[c] * Sn[(size_t)c * dv1 + dv];
          if (p->normalize) {
            for (int e = 0; e < dv; ++e) {
              double n = 0.0;
              for (int c = 0; c < dk; ++c) n += qd[c] * Sn[(size_t)c * dv1 + e];
              dot_dO_o += dOt[e] * (n / dn);
              dop[e] = dOt[e] / dn;
            }
            dop[dv] = -dot_dO_o / dn;
          } else {
            for (int e = 0; e < dv; ++e) dop[e] = dOt[e];
            dop[dv] = 0.0;
          }
          double* dvt = d_v + (((long)b * T + t) * Hkv + j) * dv;
          double dg_scalar = 0.0;
          for (int c = 0; c < dk; ++c) {
            double* dSr = dS + (size_t)c * dv1;
            double dq = 0.0, dkk = 0.0, dal = 0.0;
            for (int e = 0; e < dv1; ++e) {
              dSr[e] += qd[c] * dop[e];
              dq += dop[e] * Sn[(size_t)c * dv1 + e];
              double vp = e < dv ? vt[e] : 1.0;
              dkk += dSr[e] * vp;
              dal += dSr[e] * Sp[(size_t)c * dv1 + e];
            }
            for (int e = 0; e < dv; ++e) dvt[e] += kd[c] * dSr[e];
            d_qdot[th * dk + c] = dq;
            d_kdot[th * dk + c] = dkk;
            const double a = alpha[(size_t)t * dk + c];
            double dg = dal * a;
            for (int e = 0; e < dv1; ++e) dSr[e] *= a;
            if (gd == 1) dg_scalar += dg;
            else {
              double araw = gate[th * gd + c];
              d_gate[th * gd + c] = p->gate_mode == 1 ? dg : dg * (1.0 - 1.0 / (1.0 + exp(-araw))) / p->gate_tau;
            }
          }
          if (gd == 1) {
            double araw = gate[th];
            d_gate[th] = p->gate_mode == 1 ? dg_scalar
                                           : dg_scalar * (1.0 - 1.0 / (1.0 + exp(-araw))) / p->gate_tau;
          }
        }
        free(Sall); free(dS); free(alpha); free(dop);
      }
}

/* ---- Backward of conv -> mix -> phi for one stream (chain rule; Section 4.1 defines the forward).
 * x [B,T,NH,d] raw stream, w its taps, cache nullable; W [H,d,d] or NULL (then d_out is [B,T,NH,d], else [B,T,H,d]).
 * Outputs: dx [B,T,NH,d], dw [NH*d,K]; dW [H,d,d] is ACCUMULATED into (caller zeroes it; two streams share it). */
void oracle_conv_mix_bwd(const double* x, const double* w, const double* cache, const double* W,
                         const double* d_out, int B, int T, int NH, int H, int d, int K, int phi, double* dx,
                         double* dw, double* dW) {
  const long C = (long)NH * d;
  const int G = H / NH;
  double* u = (double*)malloc(sizeof(double) * (size_t)B * T * C);
  double* du = (double*)calloc((size_t)B * T * C, sizeof(double));
  oracle_conv(x, w, cache, B, T, NH, d, K, u);
  if (!W) {
    memcpy(du, d_out, sizeof(double) * (size_t)B * T * C);
  } else {
#pragma omp parallel for schedule(dynamic)
    for (int n = 0; n < NH; ++n) {
      double* y = (double*)malloc(sizeof(double) * d);
      double* pp = (double*)malloc(sizeof(double) * d);
      double* dy = (double*)malloc(sizeof(double) * d);
      for (int h = n * G; h < (n + 1) * G; ++h) {
        const double* Wh = W + (long)h * d * d;
        double* dWh = dW + (long)h * d * d;
        for (int b = 0; b < B; ++b)
          for (int t = 0; t < T; ++t) {
            const double* ur = u + (((long)b * T + t) * NH + n) * d;
            double* dur = du + (((long)b * T + t) * NH + n) * d;
            const double* dp = d_out + (((long)b * T + t) * H + h) * d;
            for (int e = 0; e < d; ++e) {
              double acc = 0.0;
              for (int c = 0; c < d; ++c) acc += ur[c] * Wh[(long)c * d + e];
              y[e] = acc;
            }
            phi_forward(y, d, phi, pp);
            if (phi == 0) { /* softmax Jacobian: dy = p (.) (dp - p.dp) */
              double s = 0.0;
              for (int e = 0; e < d; ++e) s += pp[e] * dp[e];
              for (int e = 0; e < d; ++e) dy[e] = pp[e] * (dp[e] - s);
            } else if (phi == 1) {
              for (int e = 0; e < d; ++e) dy[e] = dp[e] * (y[e] > 0.0 ? 1.0 : exp(y[e]));
            } else {
              for (int e = 0; e < d; ++e) dy[e] = dp[e];
            }
            for (int c = 0; c < d; ++c) {
              double acc = 0.0;
              for (int e = 0; e < d; ++e) {
                dWh[(long)c * d + e] += ur[c] * dy[e];
                acc += dy[e] * Wh[(long)c * d + e];
              }
              dur[c] += acc;
            }
          }
      }
      free(y); free(pp); free(dy);
    }
  }
  /* conv transpose: dx[t] = sum_delta w_delta du[t+delta] ; dw_delta = sum_{b,t} du[t] x[t-delta] */
  memset(dw, 0, sizeof(double) * (size_t)C * K);
#pragma omp parallel for
  for (long c = 0; c < C; ++c)
    for (int b = 0; b < B; ++b)
      for (int t = 0; t < T; ++t) {
        double acc = 0.0;
        for (int delta = 0; delta < K; ++delta) {
          if (t + delta < T) acc += w[c * K + delta] * du[((long)b * T + t + delta) * C + c];
          int s = t - delta;
          double xv = s >= 0 ? x[((long)b * T + s) * C + c]
                             : (cache ? cache[((long)b * (K - 1) + (s + K - 1)) * C + c] : 0.0);
          dw[c * K + delta] += du[((long)b * T + t) * C + c] * xv;
        }
        dx[((long)b * T + t) * C + c] = acc;
      }
  free(u); free(du);
}

/* ---- The whole layer, Fig. 1: conv on q and k, shared mix + phi, normalized GLA; also hands back the conv caches
 *      (the last K-1 raw tokens seen, Section 4.1 on caching). T = 1 with caches and a state is one decode step. */
void oracle_layer_fwd(const oracle_params* p, const double* q, const double* k, const double* v,
                      const double* gate, const double* w_q, const double* w_k, const double* W,
                      const double* cache_q_in, const double* cache_k_in, const double* S0, const double* z0,
                      double* o, double* den, double* qdot_out, double* kdot_out, double* cache_q_out,
                      double* cache_k_out, double* S_T, double* z_T) {
  const int B = p->B, T = p->T, H = p->H, Hkv = p->H_kv, dk = p->d_k, K = p->conv_k;
  const size_t nq = (size_t)B * T * H * dk, nk = (size_t)B * T * Hkv * dk;
  double* uq = (double*)malloc(sizeof(double) * nq);
  double* uk = (double*)malloc(sizeof(double) * nk);
  double* qd = qdot_out ? qdot_out : (double*)malloc(sizeof(double) * nq);
  double* kd = kdot_out ? kdot_out : (double*)malloc(sizeof(double) * nq);
  oracle_conv(q, w_q, cache_q_in, B, T, H, dk, K, uq);
  oracle_conv(k, w_k, cache_k_in, B, T, Hkv, dk, K, uk);
  oracle_mix_phi(uq, W, B, T, H, H, dk, p->phi, qd);
  oracle_mix_phi(uk, W, B, T, Hkv, H, dk, p->phi, kd);
  oracle_gla_fwd(p, qd, kd, v, gate, S0, z0, o, den, S_T, z_T);
  for (int s = 0; s < 2; ++s) {
    double* co = s ? cache_k_out : cache_q_out;
    const double* ci = s ? cache_k_in : cache_q_in;
    const double* x = s ? k : q;
    const long C = (long)(s ? Hkv : H) * dk;
    if (!co) continue;
    for (int b = 0; b < B; ++b)
      for (int r = 0; r < K - 1; ++r) { /* row r holds token T-(K-1)+r of the concatenated [cache, x] stream */
        int tok = T - (K - 1) + r;
        for (long c = 0; c < C; ++c) {
          double val;
          if (tok >= 0) val = x[((long)b * T + tok) * C + c];
          else val = ci ? ci[((long)b * (K - 1) + (tok + K - 1)) * C + c] : 0.0;
          co[((long)b * (K - 1) + r) * C + c] = val;
        }
      }
  }
  free(uq); free(uk);
  if (!qdot_out) free(qd);
  if (!kdot_out) free(kd);
}
