// Causal depthwise Conv1D across tokens, the shared per-head linear layer and the feature map phi (Section 4.1),
// forward and backward, CUDA-core (fp32 FMA) kernels. Storage type T is float or bfloat16; arithmetic is fp32.
#include <type_traits>

#include "common.cuh"

namespace lawcat {

// One raw token of a stream, or a conv-cache row for negative token indices, or zero (Section 4.1: the conv only
// looks at earlier tokens; the cache holds the K-1 raw tokens that precede t = 0, oldest first).
template <typename T>
__device__ __forceinline__ float raw_token(const T* x, const T* cache, int b, int s, int Tn, int C, int K, int ch) {
  if (s >= 0) return ldf(x + ((size_t)b * Tn + s) * C + ch);
  if (cache) return ldf(cache + ((size_t)b * (K - 1) + (s + K - 1)) * C + ch);
  return 0.f;
}

// ------------------------------------------------------------------------------------------------ plain conv
// out[b,t,ch] = sum_delta w[ch,delta] x[b,t-delta,ch]. One thread owns one channel for a run of TR tokens and
// slides a register window over them, so every input is read once; neighbouring threads take neighbouring channels.
template <typename T, int TR>
__global__ void conv_plain_kernel(const T* __restrict__ x, const T* __restrict__ w, const T* __restrict__ cache,
                                  T* __restrict__ out, int B, int Tn, int C, int K) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int runs = (Tn + TR - 1) / TR;
  const size_t total = (size_t)B * runs * C;
  if (idx >= total) return;
  const int ch = (int)(idx % C);
  const int run = (int)((idx / C) % runs);
  const int b = (int)(idx / ((size_t)C * runs));
  float wt[8], win[8];
#pragma unroll
  for (int d = 0; d < 8; ++d) wt[d] = d < K ? ldf(w + (size_t)ch * K + d) : 0.f;
  const int t0 = run * TR;
#pragma unroll
  for (int d = 1; d < 8; ++d) win[d] = d < K ? raw_token(x, cache, b, t0 - d, Tn, C, K, ch) : 0.f;
#pragma unroll
  for (int i = 0; i < TR; ++i) {
    const int t = t0 + i;
    if (t >= Tn) break;
    win[0] = ldf(x + ((size_t)b * Tn + t) * C + ch);
    float acc = 0.f;
#pragma unroll
    for (int d = 0; d < 8; ++d) acc = fmaf(wt[d], win[d], acc);
    stf(out + ((size_t)b * Tn + t) * C + ch, acc);
#pragma unroll
    for (int d = 7; d > 0; --d) win[d] = win[d - 1];
  }
}

int launch_conv_plain(const Ctx& c, const void* x, const void* w, const void* cache, void* out, int NH) {
  const lawcat_params& p = *c.p;
  const int C = NH * p.d_k;
  constexpr int TR = 16;
  const size_t total = (size_t)p.B * ((p.T + TR - 1) / TR) * C;
  if (total == 0) return LAWCAT_OK;
  const int threads = 256;
  const unsigned blocks = (unsigned)((total + threads - 1) / threads);
  LaunchScope _ls("conv_plain", c.stream);
  if (p.dtype == LAWCAT_F32)
    conv_plain_kernel<float, TR><<<blocks, threads, 0, c.stream>>>((const float*)x, (const float*)w,
                                                                     (const float*)cache, (float*)out, p.B, p.T, C,
                                                                     p.conv_k);
  else
    conv_plain_kernel<bf16, TR><<<blocks, threads, 0, c.stream>>>((const bf16*)x, (const bf16*)w,
                                                                    (const bf16*)cache, (bf16*)out, p.B, p.T, C,
                                                                    p.conv_k);
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

// ------------------------------------------------------------------------------------------------ phi helpers
// A warp holds one token's d mix outputs, lane l owning entries l, l+32, l+64, l+96 (those < d).
__device__ __forceinline__ void phi_forward_warp(float (&y)[4], int d, int lane, int phi) {
  if (phi == LAWCAT_PHI_SOFTMAX) {
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (lane + 32 * j < d) m = fmaxf(m, y[j]);
    m = warp_max(m);
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      y[j] = (lane + 32 * j < d) ? expf(y[j] - m) : 0.f;
      s += y[j];
    }
    s = warp_sum(s);
    const float inv = 1.f / s;
#pragma unroll
    for (int j = 0; j < 4; ++j) y[j] *= inv;
  } else if (phi == LAWCAT_PHI_ELU1) {
#pragma unroll
    for (int j = 0; j < 4; ++j) y[j] = y[j] > 0.f ? y[j] + 1.f : expf(y[j]);
  }
}

// ------------------------------------------------------------------------------------------------ conv+mix+phi fwd
// One block = TT tokens of one head of one stream (blockIdx.z: 0 query, 1 key). The conv output tile and W[h] sit in
// shared memory; each warp owns TT/8 whole tokens so the feature map is a warp-local reduction.
constexpr int CM_TT = 32;
constexpr int CM_THREADS = 256;

struct ConvMixArgs {
  const void *q, *k, *w_q, *w_k, *W, *cache_q, *cache_k;
  void *qdot, *kdot;
  int B, T, H, Hkv, d, K, phi;
  int unshared;  // 1: W is [2,H,d,d], the key stream uses the second set
};

template <typename TI, typename TO>
__global__ void __launch_bounds__(CM_THREADS) convmix_fwd_kernel(ConvMixArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int d = a.d, K = a.K, Tn = a.T;
  float* Ws = smem;          // [d][d]
  float* us = smem + d * d;  // [TT][d]
  const int stream = blockIdx.z, h = blockIdx.y;
  const int tiles = (Tn + CM_TT - 1) / CM_TT;
  const int b = blockIdx.x / tiles, t0 = (blockIdx.x % tiles) * CM_TT;
  const int G = a.H / a.Hkv;
  const int NH = stream ? a.Hkv : a.H, n = stream ? h / G : h;
  const TI* x = (const TI*)(stream ? a.k : a.q);
  const TI* w = (const TI*)(stream ? a.w_k : a.w_q);
  const TI* cache = (const TI*)(stream ? a.cache_k : a.cache_q);
  TO* out = (TO*)(stream ? a.kdot : a.qdot);
  const TI* Wh = (const TI*)a.W + ((size_t)(stream && a.unshared ? a.H : 0) + h) * d * d;
  const int tid = threadIdx.x, C = NH * d;
  for (int i = tid; i < d * d; i += CM_THREADS) Ws[i] = ldf(Wh + i);
  for (int i = tid; i < CM_TT * d; i += CM_THREADS) {
    const int tl = i / d, ch = i % d, t = t0 + tl;
    float acc = 0.f;
    if (t < Tn)
      for (int dl = 0; dl < K; ++dl)
        acc = fmaf(ldf(w + ((size_t)n * d + ch) * K + dl), raw_token(x, cache, b, t - dl, Tn, C, K, n * d + ch), acc);
    us[i] = acc;
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  constexpr int TPW = CM_TT / (CM_THREADS / 32);  // tokens per warp
  float acc[TPW][4];
#pragma unroll
  for (int i = 0; i < TPW; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int cc = 0; cc < d; ++cc) {
    float wv[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) wv[j] = (lane + 32 * j < d) ? Ws[cc * d + lane + 32 * j] : 0.f;
#pragma unroll
    for (int i = 0; i < TPW; ++i) {
      const float u = us[(warp * TPW + i) * d + cc];
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(u, wv[j], acc[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < TPW; ++i) {
    const int t = t0 + warp * TPW + i;
    if (t >= Tn) continue;  // warp-uniform
    phi_forward_warp(acc[i], d, lane, a.phi);
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (lane + 32 * j < d) stf(out + (((size_t)b * Tn + t) * a.H + h) * d + lane + 32 * j, acc[i][j]);
  }
}

int launch_convmix_fwd(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                       const void* cache_q, const void* cache_k, void* qdot, void* kdot, bool out_f32, bool exact) {
  const lawcat_params& p = *c.p;
  if (p.B * p.T == 0) return LAWCAT_OK;
  if (convmix_tc_fwd_supported(p) && !exact)  // tensor-core kernel
    return launch_convmix_tc_fwd(c, q, k, w_q, w_k, W, cache_q, cache_k, qdot, kdot, out_f32);
  ConvMixArgs a{q, k, w_q, w_k, W, cache_q, cache_k, qdot, kdot, p.B, p.T, p.H, p.H_kv, p.d_k, p.conv_k, p.phi,
                p.mix_unshared};
  const size_t smem = sizeof(float) * ((size_t)p.d_k * p.d_k + (size_t)CM_TT * p.d_k);
  dim3 grid(p.B * ((p.T + CM_TT - 1) / CM_TT), p.H, 2);
#define LAUNCH_CM(TI, TO)                                                                                      \
  do {                                                                                                         \
    if (cudaFuncSetAttribute(convmix_fwd_kernel<TI, TO>, cudaFuncAttributeMaxDynamicSharedMemorySize,          \
                             (int)smem) != cudaSuccess)                                                        \
      return LAWCAT_ERR_CUDA;                                                                                  \
    convmix_fwd_kernel<TI, TO><<<grid, CM_THREADS, smem, c.stream>>>(a);                                       \
  } while (0)
  LaunchScope _ls("convmix_fwd", c.stream);
  if (p.dtype == LAWCAT_F32) LAUNCH_CM(float, float);
  else if (out_f32) LAUNCH_CM(bf16, float);
  else LAUNCH_CM(bf16, bf16);
#undef LAUNCH_CM
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

// ------------------------------------------------------------------------------------------------ conv+mix+phi bwd
// Chain rule on conv -> mix -> phi. One block = one (batch, span of tokens, key/value head j). It walks the G query
// heads of the group and, for each, the query stream and the key stream (both use W[h]): recompute the conv tile and
// the mix output, apply the phi Jacobian to the incoming gradient, then
//   d(conv out) = dy W[h]^T   (query stream: stored per query head; key stream: summed over the group),
//   dW[h]      += (conv out)^T dy   (registers across the span, one atomic add per entry at the end).
constexpr int CB_SPAN = 64;

struct ConvMixBwdArgs {
  const void *q, *k, *w_q, *w_k, *W, *cache_q, *cache_k, *d_qdot, *d_kdot;
  float *du_q, *du_k, *dW;
  int B, T, H, Hkv, K, phi;
  int unshared;  // 1: W and dW are [2,H,D,D], the key stream uses the second set
};

template <typename TI, int D>
__global__ void __launch_bounds__(CM_THREADS) convmix_bwd_kernel(ConvMixBwdArgs a) {
  extern __shared__ __align__(16) float smem[];
  constexpr int LDW = D + 1;
  float* Ws = smem;                    // [D][D+1]
  float* us = Ws + D * LDW;            // [TT][D]
  float* dys = us + CM_TT * D;         // [TT][D]
  // dW is accumulated in 4 x 4 register blocks (two 16-byte shared-memory reads per 16 multiply-adds)
  constexpr int DB = D / 4, NB = (DB * DB + CM_THREADS - 1) / CM_THREADS;
  constexpr int TPW = CM_TT / (CM_THREADS / 32);
  const int Tn = a.T, K = a.K, G = a.H / a.Hkv;
  const int spans = (Tn + CB_SPAN - 1) / CB_SPAN;
  const int b = blockIdx.x / spans, span0 = (blockIdx.x % spans) * CB_SPAN;
  const int span1 = min(Tn, span0 + CB_SPAN);
  const int j = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int gi = 0; gi < G; ++gi) {
    const int h = j * G + gi;
    for (int stream = 0; stream < 2; ++stream) {
      const size_t wset = (size_t)(stream && a.unshared ? a.H : 0) + h;  // which matrix of W / dW
      if (stream == 0 || a.unshared) {
        const TI* Wh = (const TI*)a.W + wset * D * D;
        __syncthreads();
        for (int i = tid; i < D * D; i += CM_THREADS) Ws[(i / D) * LDW + (i % D)] = ldf(Wh + i);
      }
      const int NH = stream ? a.Hkv : a.H, n = stream ? j : h, C = NH * D;
      const TI* x = (const TI*)(stream ? a.k : a.q);
      const TI* w = (const TI*)(stream ? a.w_k : a.w_q);
      const TI* cache = (const TI*)(stream ? a.cache_k : a.cache_q);
      const TI* dout = (const TI*)(stream ? a.d_kdot : a.d_qdot);
      float dWacc[NB][16];
#pragma unroll
      for (int m = 0; m < NB; ++m)
#pragma unroll
        for (int i = 0; i < 16; ++i) dWacc[m][i] = 0.f;
      for (int t0 = span0; t0 < span1; t0 += CM_TT) {
        __syncthreads();
        for (int i = tid; i < CM_TT * D; i += CM_THREADS) {
          const int tl = i / D, ch = i % D, t = t0 + tl;
          float acc = 0.f;
          if (t < span1)
            for (int dl = 0; dl < K; ++dl)
              acc = fmaf(ldf(w + ((size_t)n * D + ch) * K + dl),
                         raw_token(x, cache, b, t - dl, Tn, C, K, n * D + ch), acc);
          us[i] = acc;
        }
        __syncthreads();
        float acc[TPW][4];
#pragma unroll
        for (int i = 0; i < TPW; ++i)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) acc[i][jj] = 0.f;
        for (int cc = 0; cc < D; ++cc) {
          float wv[4];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) wv[jj] = (lane + 32 * jj < D) ? Ws[cc * LDW + lane + 32 * jj] : 0.f;
#pragma unroll
          for (int i = 0; i < TPW; ++i) {
            const float u = us[(warp * TPW + i) * D + cc];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) acc[i][jj] = fmaf(u, wv[jj], acc[i][jj]);
          }
        }
#pragma unroll
        for (int i = 0; i < TPW; ++i) {
          const int tl = warp * TPW + i, t = t0 + tl;
          float dp[4], dy[4];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int e = lane + 32 * jj;
            dp[jj] = (t < span1 && e < D) ? ldf(dout + (((size_t)b * Tn + t) * a.H + h) * D + e) : 0.f;
          }
          if (a.phi == LAWCAT_PHI_SOFTMAX) {
            phi_forward_warp(acc[i], D, lane, a.phi);
            float s = 0.f;
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) s = fmaf(acc[i][jj], dp[jj], s);
            s = warp_sum(s);
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) dy[jj] = acc[i][jj] * (dp[jj] - s);
          } else if (a.phi == LAWCAT_PHI_ELU1) {
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) dy[jj] = dp[jj] * (acc[i][jj] > 0.f ? 1.f : expf(acc[i][jj]));
          } else {
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) dy[jj] = dp[jj];
          }
#pragma unroll
          for (int jj = 0; jj < 4; ++jj)
            if (lane + 32 * jj < D) dys[tl * D + lane + 32 * jj] = dy[jj];
        }
        __syncthreads();
        // d(conv out)[tl][ch] = sum_e dy[tl][e] W[ch][e]
        float du[TPW][4];
#pragma unroll
        for (int i = 0; i < TPW; ++i)
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) du[i][jj] = 0.f;
        for (int e = 0; e < D; ++e) {
          float wv[4];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) wv[jj] = (lane + 32 * jj < D) ? Ws[(lane + 32 * jj) * LDW + e] : 0.f;
#pragma unroll
          for (int i = 0; i < TPW; ++i) {
            const float dyv = dys[(warp * TPW + i) * D + e];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) du[i][jj] = fmaf(dyv, wv[jj], du[i][jj]);
          }
        }
#pragma unroll
        for (int i = 0; i < TPW; ++i) {
          const int t = t0 + warp * TPW + i;
          if (t >= span1) continue;
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int ch = lane + 32 * jj;
            if (ch >= D) continue;
            if (stream == 0) {
              a.du_q[(((size_t)b * Tn + t) * a.H + h) * D + ch] = du[i][jj];
            } else {
              float* dst = a.du_k + (((size_t)b * Tn + t) * a.Hkv + j) * D + ch;
              *dst = (gi == 0 ? 0.f : *dst) + du[i][jj];
            }
          }
        }
        // dW[ch][e] += sum_tl u[tl][ch] dy[tl][e]
#pragma unroll
        for (int m = 0; m < NB; ++m) {
          const int blk = tid + CM_THREADS * m;
          if (blk < DB * DB) {
            const int cb = blk / DB, eb = blk % DB;
#pragma unroll 4
            for (int tl = 0; tl < CM_TT; ++tl) {
              const float4 u4 = *reinterpret_cast<const float4*>(us + tl * D + 4 * cb);
              const float4 d4 = *reinterpret_cast<const float4*>(dys + tl * D + 4 * eb);
              const float uu[4] = {u4.x, u4.y, u4.z, u4.w}, dd[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
              for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) dWacc[m][4 * i + jj] = fmaf(uu[i], dd[jj], dWacc[m][4 * i + jj]);
            }
          }
        }
      }
      if (a.dW) {
#pragma unroll
        for (int m = 0; m < NB; ++m) {
          const int blk = tid + CM_THREADS * m;
          if (blk < DB * DB) {
            const int cb = blk / DB, eb = blk % DB;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int jj = 0; jj < 4; ++jj)
                atomicAdd(a.dW + wset * D * D + (size_t)(4 * cb + i) * D + 4 * eb + jj, dWacc[m][4 * i + jj]);
          }
        }
      }
    }
  }
}

// The conv's own backward for one stream, both results in one sweep:
//   dx[b,t,ch] = sum_delta w[ch,delta] du[b,t+delta,ch]   (transpose of the causal conv)
//   dw[ch,delta] = sum_{b,t} du[b,t,ch] x[b,t-delta,ch]
// One thread = one channel over a span of tokens, neighbouring threads neighbouring channels: it slides one register
// window over du (the tokens ahead) and one over x (the tokens behind), so every input is read once; the span's part of
// dw goes out with atomic adds. Either result may be absent.
constexpr int CBW_SPAN = 64;
template <typename TD, typename TX, int KM>
__global__ void __launch_bounds__(128) conv_bwd_kernel(const TD* __restrict__ du, const TX* __restrict__ x,
                                                      const TX* __restrict__ w, const TX* __restrict__ cache,
                                                      TX* __restrict__ dx, float* __restrict__ dw, int B, int Tn, int C,
                                                      int K) {
  const int ch = blockIdx.y * blockDim.x + threadIdx.x;
  if (ch >= C) return;
  const int spans = (Tn + CBW_SPAN - 1) / CBW_SPAN;
  const int b = blockIdx.x / spans, t0 = (blockIdx.x % spans) * CBW_SPAN;
  const int t1 = min(Tn, t0 + CBW_SPAN);
  float tap[KM], acc[KM], xw[KM], dwin[KM];
#pragma unroll
  for (int d = 0; d < KM; ++d) {
    tap[d] = d < K ? ldf(w + (size_t)ch * K + d) : 0.f;
    acc[d] = 0.f;
    xw[d] = (d >= 1 && d < K) ? raw_token(x, cache, b, t0 - d, Tn, C, K, ch) : 0.f;   // xw[d] = x[t - d]
    dwin[d] = (d + 1 < K && t0 + d < Tn) ? ldf(du + ((size_t)b * Tn + t0 + d) * C + ch) : 0.f;  // shifted below
  }
  // entering token t the window holds du[t .. t+K-2] in dwin[0 .. K-2]; the newest entry du[t+K-1] comes from the batch
  // of loads that opens every group of 8 tokens (all of a group's loads are in flight together)
  for (int tg = t0; tg < t1; tg += 8) {
    float ahead[8], xin[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int ta = tg + j + K - 1;
      ahead[j] = (tg + j < t1 && ta < Tn) ? ldf(du + ((size_t)b * Tn + ta) * C + ch) : 0.f;
      xin[j] = tg + j < t1 ? ldf(x + ((size_t)b * Tn + tg + j) * C + ch) : 0.f;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int t = tg + j;
      if (t < t1) {
#pragma unroll
        for (int d = 0; d < KM; ++d)
          if (d == K - 1) dwin[d] = ahead[j];
        xw[0] = xin[j];
        float o = 0.f;
        const float g = dwin[0];
#pragma unroll
        for (int d = 0; d < KM; ++d) {
          o = fmaf(tap[d], dwin[d], o);
          acc[d] = fmaf(g, xw[d], acc[d]);
        }
        if (dx) stf(dx + ((size_t)b * Tn + t) * C + ch, o);
#pragma unroll
        for (int d = 0; d < KM - 1; ++d) dwin[d] = dwin[d + 1];
        dwin[KM - 1] = 0.f;
#pragma unroll
        for (int d = KM - 1; d > 0; --d) xw[d] = xw[d - 1];
      }
    }
  }
  if (dw) {
    for (int d = 0; d < K; ++d) atomicAdd(dw + (size_t)ch * K + d, acc[d]);
  }
}

template <typename TI, typename TD>
static int conv_bwd_stream(const Ctx& c, const TD* du, const TI* x, const TI* w, const TI* cache, TI* dx, float* dw,
                           int NH) {
  const lawcat_params& p = *c.p;
  const int C = NH * p.d_k;
  if (!dx && !dw) return LAWCAT_OK;
  if (dw && cudaMemsetAsync(dw, 0, sizeof(float) * (size_t)C * p.conv_k, c.stream) != cudaSuccess) return LAWCAT_ERR_CUDA;
  dim3 grid(p.B * ((p.T + CBW_SPAN - 1) / CBW_SPAN), (C + 127) / 128);
  LaunchScope _ls("conv_bwd", c.stream);
  if (p.conv_k <= 4)
    conv_bwd_kernel<TD, TI, 4><<<grid, 128, 0, c.stream>>>(du, x, w, cache, dx, dw, p.B, p.T, C, p.conv_k);
  else
    conv_bwd_kernel<TD, TI, 8><<<grid, 128, 0, c.stream>>>(du, x, w, cache, dx, dw, p.B, p.T, C, p.conv_k);
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

template <typename TI>
static int conv_bwd_typed(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k,
                          const void* W, const void* cache_q, const void* cache_k, const void* d_qdot,
                          const void* d_kdot, void* dq, void* dk, float* dw_q, float* dw_k, float* dW, void* ws,
                          bool grads_f32) {
  const lawcat_params& p = *c.p;
  if (p.B * p.T == 0) {
    if (dw_q && cudaMemsetAsync(dw_q, 0, sizeof(float) * (size_t)p.H * p.d_k * p.conv_k, c.stream)) return LAWCAT_ERR_CUDA;
    if (dw_k && cudaMemsetAsync(dw_k, 0, sizeof(float) * (size_t)p.H_kv * p.d_k * p.conv_k, c.stream)) return LAWCAT_ERR_CUDA;
    if (dW && cudaMemsetAsync(dW, 0, sizeof(float) * (size_t)(1 + p.mix_unshared) * p.H * p.d_k * p.d_k, c.stream)) return LAWCAT_ERR_CUDA;
    return LAWCAT_OK;
  }
  if (!W) {
    int r = conv_bwd_stream<TI, TI>(c, (const TI*)d_qdot, (const TI*)q, (const TI*)w_q, (const TI*)cache_q, (TI*)dq,
                                    dw_q, p.H);
    if (r) return r;
    return conv_bwd_stream<TI, TI>(c, (const TI*)d_kdot, (const TI*)k, (const TI*)w_k, (const TI*)cache_k, (TI*)dk,
                                   dw_k, p.H_kv);
  }
  float* du_q = (float*)ws;
  float* du_k = (float*)((char*)ws + align_up(sizeof(float) * (size_t)p.B * p.T * p.H * p.d_k, 256));
  if (dW && cudaMemsetAsync(dW, 0, sizeof(float) * (size_t)(1 + p.mix_unshared) * p.H * p.d_k * p.d_k, c.stream) != cudaSuccess)
    return LAWCAT_ERR_CUDA;
  ConvMixBwdArgs a{q, k, w_q, w_k, W, cache_q, cache_k, d_qdot, d_kdot, du_q, du_k, dW,
                   p.B, p.T, p.H, p.H_kv, p.conv_k, p.phi, p.mix_unshared};
  if (std::is_same<TI, bf16>::value && convmix_tc_bwd_supported(p) && p.chunk != 1) {
    // tensor-core kernel for the mix and the softmax Jacobian; the conv's own backward follows on du as below
    int r0 = launch_convmix_tc_bwd(c, q, k, w_q, w_k, W, cache_q, cache_k, d_qdot, d_kdot, grads_f32, du_q, du_k, dW);
    if (r0) return r0;
    r0 = conv_bwd_stream<TI, float>(c, du_q, (const TI*)q, (const TI*)w_q, (const TI*)cache_q, (TI*)dq, dw_q, p.H);
    if (r0) return r0;
    return conv_bwd_stream<TI, float>(c, du_k, (const TI*)k, (const TI*)w_k, (const TI*)cache_k, (TI*)dk, dw_k, p.H_kv);
  }
  if (grads_f32) return LAWCAT_ERR_UNSUPPORTED;  // (fp32 gradients only reach the tensor-core kernel)
  dim3 grid(p.B * ((p.T + CB_SPAN - 1) / CB_SPAN), p.H_kv);
#define LAUNCH_CB(D)                                                                                             \
  do {                                                                                                           \
    const size_t smem = sizeof(float) * ((size_t)D * (D + 1) + 2 * (size_t)CM_TT * D);                           \
    if (cudaFuncSetAttribute(convmix_bwd_kernel<TI, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,             \
                             (int)smem) != cudaSuccess)                                                          \
      return LAWCAT_ERR_CUDA;                                                                                    \
    convmix_bwd_kernel<TI, D><<<grid, CM_THREADS, smem, c.stream>>>(a);                                          \
  } while (0)
  LaunchScope _ls("convmix_bwd", c.stream);
  switch (p.d_k) {
    case 16: LAUNCH_CB(16); break;
    case 32: LAUNCH_CB(32); break;
    case 64: LAUNCH_CB(64); break;
    case 128: LAUNCH_CB(128); break;
    default: return LAWCAT_ERR_UNSUPPORTED;
  }
#undef LAUNCH_CB
  LAWCAT_CHECK_LAUNCH();
  int r = conv_bwd_stream<TI, float>(c, du_q, (const TI*)q, (const TI*)w_q, (const TI*)cache_q, (TI*)dq, dw_q, p.H);
  if (r) return r;
  return conv_bwd_stream<TI, float>(c, du_k, (const TI*)k, (const TI*)w_k, (const TI*)cache_k, (TI*)dk, dw_k,
                                    p.H_kv);
}

int launch_conv_bwd(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                    const void* cache_q, const void* cache_k, const void* d_qdot, const void* d_kdot, void* dq,
                    void* dk, float* dw_q, float* dw_k, float* dW, void* ws, bool grads_f32) {
  if (c.p->dtype == LAWCAT_F32)
    return conv_bwd_typed<float>(c, q, k, w_q, w_k, W, cache_q, cache_k, d_qdot, d_kdot, dq, dk, dw_q, dw_k, dW, ws, false);
  return conv_bwd_typed<bf16>(c, q, k, w_q, w_k, W, cache_q, cache_k, d_qdot, d_kdot, dq, dk, dw_q, dw_k, dW, ws, grads_f32);
}

// ------------------------------------------------------------------------------------------------ conv cache out
// cache_out[b,r,:] = token T-(K-1)+r of the stream [cache_in, x] (Section 4.1: the cache is bounded by the kernel size)
template <typename T>
__global__ void cache_out_kernel(const T* __restrict__ x, const T* __restrict__ cin, T* __restrict__ cout, int B,
                                 int Tn, int C, int K) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)B * (K - 1) * C) return;
  const int ch = (int)(idx % C);
  const int r = (int)((idx / C) % (K - 1));
  const int b = (int)(idx / ((size_t)C * (K - 1)));
  const int tok = Tn - (K - 1) + r;
  T val;
  if (tok >= 0) val = x[((size_t)b * Tn + tok) * C + ch];
  else if (cin) val = cin[((size_t)b * (K - 1) + (tok + K - 1)) * C + ch];
  else stf(&val, 0.f);
  cout[idx] = val;
}

template <typename T>
static int cache_out_typed(const Ctx& c, const void* x, const void* cin, void* cout, int NH) {
  const lawcat_params& p = *c.p;
  const size_t total = (size_t)p.B * (p.conv_k - 1) * NH * p.d_k;
  if (!cout || total == 0) return LAWCAT_OK;
  LaunchScope _ls("cache_out", c.stream);
  cache_out_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, c.stream>>>((const T*)x, (const T*)cin, (T*)cout,
                                                                              p.B, p.T, NH * p.d_k, p.conv_k);
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

int launch_cache_out(const Ctx& c, const void* q, const void* k, const void* cache_q_in, const void* cache_k_in,
                     void* cache_q_out, void* cache_k_out) {
  int r;
  if (c.p->dtype == LAWCAT_F32) {
    if ((r = cache_out_typed<float>(c, q, cache_q_in, cache_q_out, c.p->H))) return r;
    return cache_out_typed<float>(c, k, cache_k_in, cache_k_out, c.p->H_kv);
  }
  if ((r = cache_out_typed<bf16>(c, q, cache_q_in, cache_q_out, c.p->H))) return r;
  return cache_out_typed<bf16>(c, k, cache_k_in, cache_k_out, c.p->H_kv);
}

}  // namespace lawcat
