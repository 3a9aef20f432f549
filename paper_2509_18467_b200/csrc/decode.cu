// Recurrent single-token decode (streaming inference, Section 6): the layer at one token with the conv cache of
// Section 4.1 and the constant-size state of Eq. 4. One block per (sequence, query head); the fp32 state is streamed
// through HBM once (read + write), which is the whole cost of the step.
#include "common.cuh"

namespace lawcat {

struct DecodeArgs {
  const void *q_t, *k_t, *v_t, *gate_t, *w_q, *w_k, *W;
  float *S, *z;
  const void *cache_q, *cache_k;
  void* o_t;
  int B, H, Hkv, dk, dv, K, gd, phi, gate_mode, normalize;
  float inv_tau, eps;
};

constexpr int DEC_THREADS = 256;

__device__ __forceinline__ float block_reduce(float v, float* red, bool is_max) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  v = is_max ? warp_max(v) : warp_sum(v);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float r = red[0];
  for (int i = 1; i < DEC_THREADS / 32; ++i) r = is_max ? fmaxf(r, red[i]) : r + red[i];
  return r;
}

template <typename T>
__global__ void __launch_bounds__(DEC_THREADS) decode_kernel(DecodeArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int dk = a.dk, dv = a.dv, K = a.K, H = a.H;
  float* s_u = smem;              // [2][dk] conv outputs (query, key)
  float* s_f = s_u + 2 * dk;      // [2][dk] qdot, kdot
  float* s_alpha = s_f + 2 * dk;  // [dk]
  float* s_v = s_alpha + dk;      // [dv]
  float* s_part = s_v + dv;       // [RGmax][dv]
  float* s_red = s_part + (DEC_THREADS / 16) * dv;  // [8]
  const int b = blockIdx.x / H, h = blockIdx.x % H, G = H / a.Hkv, j = h / G;
  const int tid = threadIdx.x;
  // conv tap sum: delta = 0 is the new token, delta >= 1 reads cache row K-1-delta (the newest row is the last)
  for (int i = tid; i < 2 * dk; i += DEC_THREADS) {
    const int stream = i / dk, c = i % dk;
    const int NH = stream ? a.Hkv : H, n = stream ? j : h, C = NH * dk;
    const T* xt = (const T*)(stream ? a.k_t : a.q_t);
    const T* w = (const T*)(stream ? a.w_k : a.w_q);
    const T* cache = (const T*)(stream ? a.cache_k : a.cache_q);
    float acc = ldf(w + ((size_t)n * dk + c) * K) * ldf(xt + (size_t)b * C + n * dk + c);
    for (int dl = 1; dl < K; ++dl)
      acc = fmaf(ldf(w + ((size_t)n * dk + c) * K + dl), ldf(cache + ((size_t)b * (K - 1) + (K - 1 - dl)) * C + n * dk + c), acc);
    s_u[i] = acc;
  }
  for (int i = tid; i < dk; i += DEC_THREADS)
    s_alpha[i] = expf(log_decay(ldf((const T*)a.gate_t + ((size_t)b * H + h) * a.gd + (a.gd == 1 ? 0 : i)), a.gate_mode,
                                a.inv_tau));
  for (int i = tid; i < dv; i += DEC_THREADS) s_v[i] = ldf((const T*)a.v_t + ((size_t)b * a.Hkv + j) * dv + i);
  __syncthreads();
  // shared linear layer: thread (stream, e) sums over input channels; W[h][c][e] is read coalesced along e
  {
    const T* Wh = (const T*)a.W + (size_t)h * dk * dk;
    const int stream = tid / dk, e = tid % dk;
    float y = 0.f;
    const bool act = tid < 2 * dk;
    if (act)
      for (int c = 0; c < dk; ++c) y = fmaf(s_u[stream * dk + c], ldf(Wh + (size_t)c * dk + e), y);
    if (a.phi == LAWCAT_PHI_SOFTMAX) {
      const float mq = block_reduce(act && stream == 0 ? y : -INFINITY, s_red, true);
      const float mk = block_reduce(act && stream == 1 ? y : -INFINITY, s_red, true);
      const float ex = act ? expf(y - (stream ? mk : mq)) : 0.f;
      const float sq = block_reduce(act && stream == 0 ? ex : 0.f, s_red, false);
      const float sk = block_reduce(act && stream == 1 ? ex : 0.f, s_red, false);
      y = ex / (stream ? sk : sq);
    } else if (a.phi == LAWCAT_PHI_ELU1) {
      y = y > 0.f ? y + 1.f : expf(y);
    }
    if (act) s_f[tid] = y;
  }
  __syncthreads();
  const float* qd = s_f;
  const float* kd = s_f + dk;
  // state update and read-out: thread (rg, e) walks rows rg, rg+RG, ... of column e
  const int RG = DEC_THREADS / dv, rg = tid / dv, e = tid % dv;
  float* Sbh = a.S + ((size_t)b * H + h) * dk * dv;
  float acc = 0.f;
  if (rg < RG) {
    const float ve = s_v[e];
#pragma unroll 8
    for (int c = rg; c < dk; c += RG) {
      const float s = fmaf(s_alpha[c], Sbh[(size_t)c * dv + e], kd[c] * ve);
      Sbh[(size_t)c * dv + e] = s;
      acc = fmaf(qd[c], s, acc);
    }
    s_part[rg * dv + e] = acc;
  }
  float zq = 0.f;
  if (tid < dk) {
    float* zp = a.z + ((size_t)b * H + h) * dk + tid;
    const float zn = fmaf(s_alpha[tid], *zp, kd[tid]);
    *zp = zn;
    zq = qd[tid] * zn;
  }
  const float den = block_reduce(zq, s_red, false) + a.eps;  // contains the barrier that publishes s_part
  if (tid < dv) {
    float num = 0.f;
    for (int g = 0; g < RG; ++g) num += s_part[g * dv + tid];
    stf((T*)a.o_t + ((size_t)b * H + h) * dv + tid, a.normalize ? num / den : num);
  }
}

// Drop the oldest cache row and append the new raw token; one thread per (sequence, channel), in place.
template <typename T>
__global__ void cache_shift_kernel(T* __restrict__ cache, const T* __restrict__ xt, int B, int C, int K) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)B * C) return;
  const int ch = (int)(idx % C);
  const int b = (int)(idx / C);
  T* base = cache + (size_t)b * (K - 1) * C + ch;
  for (int r = 0; r + 1 < K - 1; ++r) base[(size_t)r * C] = base[(size_t)(r + 1) * C];
  base[(size_t)(K - 2) * C] = xt[idx];
}

template <typename T>
static int decode_typed(const Ctx& c, DecodeArgs& a, void* cache_q, void* cache_k) {
  const lawcat_params& p = *c.p;
  if (p.B * p.H == 0) return LAWCAT_OK;
  const size_t smem = sizeof(float) * ((size_t)5 * p.d_k + p.d_v + (size_t)(DEC_THREADS / 16) * p.d_v + 8);
  LAWCAT_LAUNCH("decode", c.stream, decode_kernel<T><<<p.B * p.H, DEC_THREADS, smem, c.stream>>>(a));
  LAWCAT_CHECK_LAUNCH();
  if (p.conv_k > 1) {
    const size_t nq = (size_t)p.B * p.H * p.d_k, nk = (size_t)p.B * p.H_kv * p.d_k;
    LAWCAT_LAUNCH("cache_shift", c.stream,
                  cache_shift_kernel<T><<<(unsigned)((nq + 255) / 256), 256, 0, c.stream>>>(
                      (T*)cache_q, (const T*)a.q_t, p.B, p.H * p.d_k, p.conv_k));
    LAWCAT_CHECK_LAUNCH();
    LAWCAT_LAUNCH("cache_shift", c.stream,
                  cache_shift_kernel<T><<<(unsigned)((nk + 255) / 256), 256, 0, c.stream>>>(
                      (T*)cache_k, (const T*)a.k_t, p.B, p.H_kv * p.d_k, p.conv_k));
    LAWCAT_CHECK_LAUNCH();
  }
  return LAWCAT_OK;
}

int launch_decode(const Ctx& c, const void* q_t, const void* k_t, const void* v_t, const void* gate_t,
                  const void* w_q, const void* w_k, const void* W, float* S, float* z, void* cache_q, void* cache_k,
                  void* o_t) {
  const lawcat_params& p = *c.p;
  DecodeArgs a{q_t, k_t, v_t, gate_t, w_q, w_k, W, S, z, cache_q, cache_k, o_t,
               p.B, p.H, p.H_kv, p.d_k, p.d_v, p.conv_k, p.gate_dim, p.phi, p.gate_mode, p.normalize,
               1.f / p.gate_tau, p.eps};
  if (p.dtype == LAWCAT_F32) return decode_typed<float>(c, a, cache_q, cache_k);
  return decode_typed<bf16>(c, a, cache_q, cache_k);
}

}  // namespace lawcat
