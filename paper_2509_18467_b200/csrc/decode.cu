// Recurrent single-token decode (streaming inference, Section 6): the layer at one token with the conv cache of
// Section 4.1 and the constant-size state of Eq. 4. Two launches:
//   decode_features  (one block per head and group of 8 sequences, which share the head's W) conv -> shared linear layer
//                    -> feature map for the token's query and key, decay alpha = exp(g), the normalizer state z (Eq. 8's
//                    denominator) advanced in place; writes qdot, kdot, alpha and the denominator to the workspace
//   decode_state     (one block per sequence and head) S <- diag(alpha) S + kdot^T v (Eq. 4), o = qdot S / denominator (Eq. 8): the fp32 state is streamed
//                    through HBM once (read + write), which is the whole cost of the step; the same blocks then shift
//                    the conv caches (every reader of the caches belongs to the first launch, which has completed)
#include "common.cuh"

namespace lawcat {

struct DecodeArgs {
  const void *q_t, *k_t, *v_t, *gate_t, *w_q, *w_k, *W;
  float *S, *z;
  void *cache_q, *cache_k;
  void* o_t;
  float* vecs;  // workspace [B*H][3][dk]: qdot, kdot, alpha
  float* den;   // workspace [B*H]
  int B, H, Hkv, dk, dv, K, gd, phi, gate_mode, normalize;
  int w_smem;  // 1: W of the head is staged in shared memory
  float inv_tau, eps;
};

constexpr int DEC_THREADS = 256;
constexpr int DEC_ROWS = 16;  // state rows a thread holds in registers on the fast path

// Read-only load through the non-coherent path: the compiler may then hoist the loads of several loop iterations in
// front of the shared-memory stores between them, so that they are all in flight together.
template <typename T> __device__ __forceinline__ float ldro(const T* p);
template <> __device__ __forceinline__ float ldro<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldro<bf16>(const bf16* p) {
  return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}

constexpr int DEC_SEQ = 8;          // sequences per block of decode_features (they share the head's W)
constexpr int DEC_NV = 2 * DEC_SEQ;  // vectors per block: query and key stream of every sequence
constexpr int DEC_MAXW = 16, DEC_MAXR = 8, DEC_ZR = 4;  // 16-byte units (W, raw rows) and z entries a thread stages

// One block per (query head, group of DEC_SEQ sequences): W_h is staged in shared memory once for the whole group.
template <typename T>
__global__ void __launch_bounds__(DEC_THREADS) decode_features_kernel(DecodeArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int dk = a.dk, K = a.K, H = a.H;
  float* s_u = smem;                     // [dk][DEC_NV] conv outputs, vector index innermost (vector = 2 seq + stream)
  float* s_y = s_u + dk * DEC_NV;        // [DEC_NV][dk] mix outputs, then features
  float* s_alpha = s_y + DEC_NV * dk;    // [DEC_SEQ][dk]
  T* s_raw = reinterpret_cast<T*>(s_alpha + DEC_SEQ * dk);  // [DEC_NV][K][dk] raw rows of the conv, row delta of vector v
  T* s_tap = s_raw + DEC_NV * K * dk;                        // [2][dk][K] conv taps of the query head and of its kv head
  T* s_W = s_tap + 2 * dk * K;                               // [dk][dk] this head's W (only when it fits, a.w_smem)
  const int h = blockIdx.x % H, b0 = (blockIdx.x / H) * DEC_SEQ, G = H / a.Hkv, j = h / G;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // ---- every global read of the block goes out here, with 16-byte loads, before anything waits for any of them: the
  // head's W, the raw rows the conv needs (the token and the K-1 cache rows of both streams of every sequence), the taps
  // and the normalizer states. One round trip to memory instead of one per stage.
  const int U = dk * (int)sizeof(T) / 16;  // 16-byte units per row of dk entries
  const int nW = a.w_smem ? dk * U : 0, nR = DEC_NV * K * U, nT = 2 * K * U;
  uint4 wreg[DEC_MAXW], rreg[DEC_MAXR], treg = make_uint4(0u, 0u, 0u, 0u);
  float zreg[DEC_ZR];
  {
    const uint4* src = reinterpret_cast<const uint4*>((const T*)a.W + (size_t)h * dk * dk);
#pragma unroll
    for (int k = 0; k < DEC_MAXW; ++k) {
      const int i = tid + k * DEC_THREADS;
      if (i < nW) wreg[k] = __ldg(src + i);
    }
  }
  // unit i of the raw rows: vector v = i / (K U), row delta = (i / U) % K; zeros past the last sequence
  auto raw_unit = [&](int i) -> uint4 {
    const int v = i / (K * U), dl = (i / U) % K, off = i % U, seq = v >> 1, stream = v & 1, b = b0 + seq;
    if (b >= a.B) return make_uint4(0u, 0u, 0u, 0u);
    const int NH = stream ? a.Hkv : H, n = stream ? j : h, C = NH * dk;
    // delta = 0 is the new token, delta >= 1 is cache row K-1-delta (the newest row is the last)
    const T* row = dl == 0 ? (const T*)(stream ? a.k_t : a.q_t) + (size_t)b * C + n * dk
                           : (const T*)(stream ? a.cache_k : a.cache_q) + ((size_t)b * (K - 1) + (K - 1 - dl)) * C + n * dk;
    return __ldg(reinterpret_cast<const uint4*>(row) + off);
  };
  auto tap_unit = [&](int i) -> uint4 {
    const int stream = i / (K * U), off = i % (K * U);
    const T* w = stream ? (const T*)a.w_k + (size_t)j * dk * K : (const T*)a.w_q + (size_t)h * dk * K;
    return __ldg(reinterpret_cast<const uint4*>(w) + off);
  };
#pragma unroll
  for (int k = 0; k < DEC_MAXR; ++k) {
    const int i = tid + k * DEC_THREADS;
    if (i < nR) rreg[k] = raw_unit(i);
  }
  if (tid < nT) treg = tap_unit(tid);
#pragma unroll
  for (int k = 0; k < DEC_ZR; ++k) {  // (the per-sequence pass at the end: warp = sequence, lane + 32 k = channel)
    const int c = lane + 32 * k, b = b0 + warp;
    zreg[k] = (c < dk && warp < DEC_SEQ && b < a.B) ? a.z[((size_t)b * H + h) * dk + c] : 0.f;
  }
  // the blocks of decode_state may be scheduled from here on: they start with loads of S, which this kernel never
  // touches, and wait for the end of this grid before they read anything it writes
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- ... and into shared memory
  {
    uint4* dW = reinterpret_cast<uint4*>(s_W);
    uint4* dR = reinterpret_cast<uint4*>(s_raw);
#pragma unroll
    for (int k = 0; k < DEC_MAXW; ++k) {
      const int i = tid + k * DEC_THREADS;
      if (i < nW) dW[i] = wreg[k];
    }
#pragma unroll
    for (int k = 0; k < DEC_MAXR; ++k) {
      const int i = tid + k * DEC_THREADS;
      if (i < nR) dR[i] = rreg[k];
    }
    if (tid < nT) reinterpret_cast<uint4*>(s_tap)[tid] = treg;
    // (shapes with more units than a thread holds in registers: the rest goes the plain way)
    const uint4* srcW = reinterpret_cast<const uint4*>((const T*)a.W + (size_t)h * dk * dk);
    for (int i = tid + DEC_MAXW * DEC_THREADS; i < nW; i += DEC_THREADS) dW[i] = __ldg(srcW + i);
    for (int i = tid + DEC_MAXR * DEC_THREADS; i < nR; i += DEC_THREADS) dR[i] = raw_unit(i);
    for (int i = tid + DEC_THREADS; i < nT; i += DEC_THREADS) reinterpret_cast<uint4*>(s_tap)[i] = tap_unit(i);
  }
#pragma unroll 4
  for (int i = tid; i < DEC_SEQ * dk; i += DEC_THREADS) {
    const int seq = i / dk, c = i % dk, b = b0 + seq;
    s_alpha[i] = b < a.B ? expf(log_decay(ldro((const T*)a.gate_t + ((size_t)b * H + h) * a.gd + (a.gd == 1 ? 0 : c)),
                                          a.gate_mode, a.inv_tau))
                         : 0.f;
  }
  __syncthreads();
  // conv tap sum from the staged rows
  for (int i = tid; i < DEC_NV * dk; i += DEC_THREADS) {
    const int v = i / dk, c = i % dk, stream = v & 1;
    const T* tap = s_tap + (stream * dk + c) * K;
    const T* raw = s_raw + (size_t)v * K * dk + c;
    float acc = ldf(tap) * ldf(raw);
    for (int dl = 1; dl < K; ++dl) acc = fmaf(ldf(tap + dl), ldf(raw + dl * dk), acc);
    s_u[c * DEC_NV + v] = acc;
  }
  __syncthreads();
  // shared linear layer: work item (e, group of 4 vectors) sums over the input channels in order; one read of W[c][e]
  // serves the four vectors
  {
    const T* Wh = (const T*)a.W + (size_t)h * dk * dk;
    for (int it = tid; it < dk * (DEC_NV / 4); it += DEC_THREADS) {
      const int e = it % dk, vg = it / dk;
      float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
      for (int c = 0; c < dk; ++c) {
        const float w = a.w_smem ? ldf(s_W + c * dk + e) : ldf(Wh + (size_t)c * dk + e);
        const float4 u = *reinterpret_cast<const float4*>(s_u + c * DEC_NV + 4 * vg);
        y.x = fmaf(u.x, w, y.x); y.y = fmaf(u.y, w, y.y); y.z = fmaf(u.z, w, y.z); y.w = fmaf(u.w, w, y.w);
      }
      s_y[(4 * vg + 0) * dk + e] = y.x; s_y[(4 * vg + 1) * dk + e] = y.y;
      s_y[(4 * vg + 2) * dk + e] = y.z; s_y[(4 * vg + 3) * dk + e] = y.w;
    }
  }
  __syncthreads();
  // feature map, one warp per vector
  for (int v = warp; v < DEC_NV; v += DEC_THREADS / 32) {
    float* yv = s_y + v * dk;
    if (a.phi == LAWCAT_PHI_SOFTMAX) {
      float m = -INFINITY;
      for (int e = lane; e < dk; e += 32) m = fmaxf(m, yv[e]);
      m = warp_max(m);
      float sum = 0.f;
      for (int e = lane; e < dk; e += 32) {
        const float ex = expf(yv[e] - m);
        yv[e] = ex;
        sum += ex;
      }
      sum = warp_sum(sum);
      for (int e = lane; e < dk; e += 32) yv[e] = yv[e] / sum;
    } else if (a.phi == LAWCAT_PHI_ELU1) {
      for (int e = lane; e < dk; e += 32) yv[e] = yv[e] > 0.f ? yv[e] + 1.f : expf(yv[e]);
    }
  }
  __syncthreads();
  // per sequence (one warp each): features and decays to the workspace, z advanced in place, denominator of Eq. 8
  static_assert(DEC_SEQ == DEC_THREADS / 32, "one warp per sequence");
  {
    const int seq = warp, b = b0 + seq;
    if (b >= a.B) return;
    const size_t bh = (size_t)b * H + h;
    const float* qd = s_y + (2 * seq) * dk;
    const float* kd = qd + dk;
    const float* al = s_alpha + seq * dk;
    float* out = a.vecs + bh * 3 * dk;
    float zq = 0.f;
#pragma unroll
    for (int k = 0; k < DEC_ZR; ++k) {
      const int c = lane + 32 * k;
      if (c < dk) {
        out[c] = qd[c];
        out[dk + c] = kd[c];
        out[2 * dk + c] = al[c];
        const float zn = fmaf(al[c], zreg[k], kd[c]);
        a.z[bh * dk + c] = zn;
        zq = fmaf(qd[c], zn, zq);
      }
    }
    zq = warp_sum(zq);
    if (lane == 0) a.den[bh] = zq + a.eps;
  }
}

template <typename T>
__global__ void __launch_bounds__(DEC_THREADS, 3) decode_state_kernel(DecodeArgs a) {
  extern __shared__ __align__(16) float smem[];
  const int dk = a.dk, dv = a.dv, K = a.K, H = a.H;
  float* s_q = smem;           // [dk]
  float* s_k = s_q + dk;       // [dk]
  float* s_alpha = s_k + dk;   // [dk]
  float* s_v = s_alpha + dk;   // [dv]
  float* s_part = s_v + dv;    // [row groups][dv]
  const int bh = blockIdx.x, b = bh / H, h = bh % H, G = H / a.Hkv, j = h / G;
  const int tid = threadIdx.x;
  float* Sbh = a.S + (size_t)bh * dk * dv;
  // Fast path: thread (row group, 4 columns) holds up to DEC_ROWS rows x 4 columns of the state in registers; the loads
  // go out first, the small vectors arrive while the state streams in.
  const int cols4 = dv >> 2;
  const int RGv = cols4 > 0 ? DEC_THREADS / cols4 : 0;  // row groups
  const bool fast = (dv & 3) == 0 && cols4 <= DEC_THREADS && DEC_THREADS % cols4 == 0 && RGv <= DEC_THREADS / 16 &&
                    dk % RGv == 0 && dk / RGv <= DEC_ROWS;
  const int nr = fast ? dk / RGv : 0, e4 = fast ? tid % cols4 : 0, rgv = fast ? tid / cols4 : 0;
  float4 sreg[DEC_ROWS];
  if (fast) {
#pragma unroll
    for (int i = 0; i < DEC_ROWS; ++i)
      if (i < nr) sreg[i] = __ldcs(reinterpret_cast<const float4*>(Sbh + (size_t)(rgv + RGv * i) * dv) + e4);
  }
  // (launched with programmatic stream serialization: everything above ran beside decode_features; from here on that
  // grid has completed, its writes are visible, and it reads the conv caches no more)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const float* in = a.vecs + (size_t)bh * 3 * dk;
  for (int i = tid; i < 3 * dk; i += DEC_THREADS) s_q[i] = in[i];
  for (int i = tid; i < dv; i += DEC_THREADS) s_v[i] = ldf((const T*)a.v_t + ((size_t)b * a.Hkv + j) * dv + i);
  __syncthreads();
  // state update and read-out
  const int RG = fast ? RGv : DEC_THREADS / dv;
  if (fast) {
    const float4 v4 = *reinterpret_cast<const float4*>(s_v + 4 * e4);
    float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < DEC_ROWS; ++i) {
      if (i < nr) {
        const int c = rgv + RGv * i;
        const float al = s_alpha[c], kc = s_k[c], qc = s_q[c];
        float4 s4 = sreg[i];
        s4.x = fmaf(al, s4.x, kc * v4.x); s4.y = fmaf(al, s4.y, kc * v4.y);
        s4.z = fmaf(al, s4.z, kc * v4.z); s4.w = fmaf(al, s4.w, kc * v4.w);
        __stcs(reinterpret_cast<float4*>(Sbh + (size_t)c * dv) + e4, s4);
        acc4.x = fmaf(qc, s4.x, acc4.x); acc4.y = fmaf(qc, s4.y, acc4.y);
        acc4.z = fmaf(qc, s4.z, acc4.z); acc4.w = fmaf(qc, s4.w, acc4.w);
      }
    }
    *reinterpret_cast<float4*>(s_part + rgv * dv + 4 * e4) = acc4;
  } else {
    // any shape: thread (rg, e) walks rows rg, rg + RG, ... of column e
    const int rg = tid / dv, e = tid % dv;
    if (rg < RG) {
      const float ve = s_v[e];
      float acc = 0.f;
#pragma unroll 8
      for (int c = rg; c < dk; c += RG) {
        const float s = fmaf(s_alpha[c], Sbh[(size_t)c * dv + e], s_k[c] * ve);
        Sbh[(size_t)c * dv + e] = s;
        acc = fmaf(s_q[c], s, acc);
      }
      s_part[rg * dv + e] = acc;
    }
  }
  __syncthreads();
  const float den = a.den[bh];
  for (int e = tid; e < dv; e += DEC_THREADS) {
    float num = 0.f;
    for (int g = 0; g < RG; ++g) num += s_part[g * dv + e];
    stf((T*)a.o_t + (size_t)bh * dv + e, a.normalize ? num / den : num);
  }
  // conv caches: drop the oldest row, append the new raw token. This block owns the query channels of its head, and the
  // first head of a group the key channels of its kv head.
  if (K > 1) {
    for (int i = tid; i < 2 * dk; i += DEC_THREADS) {
      const int stream = i / dk, c = i % dk;
      if (stream == 1 && h % G != 0) continue;
      const int NH = stream ? a.Hkv : H, n = stream ? j : h, C = NH * dk;
      T* base = (T*)(stream ? a.cache_k : a.cache_q) + (size_t)b * (K - 1) * C + n * dk + c;
      for (int r = 0; r + 1 < K - 1; ++r) base[(size_t)r * C] = base[(size_t)(r + 1) * C];
      base[(size_t)(K - 2) * C] = ((const T*)(stream ? a.k_t : a.q_t))[(size_t)b * C + n * dk + c];
    }
  }
}

size_t decode_workspace_bytes(const lawcat_params& p) {
  return sizeof(float) * (size_t)p.B * p.H * (3 * (size_t)p.d_k + 1);
}

template <typename T>
static int decode_typed(const Ctx& c, DecodeArgs& a) {
  const lawcat_params& p = *c.p;
  if (p.B * p.H == 0) return LAWCAT_OK;
  size_t smem1 = sizeof(float) * (size_t)p.d_k * (2 * DEC_NV + DEC_SEQ) + sizeof(T) * (size_t)p.d_k * p.conv_k * (DEC_NV + 2);
  if (p.d_k > 32 * DEC_ZR) return LAWCAT_ERR_UNSUPPORTED;  // (one warp holds a sequence's normalizer state)
  const size_t wbytes = sizeof(T) * (size_t)p.d_k * p.d_k;
  a.w_smem = smem1 + wbytes <= 100 * 1024 ? 1 : 0;
  if (a.w_smem) smem1 += wbytes;
  if (smem1 > 48 * 1024 &&
      cudaFuncSetAttribute(decode_features_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1) != cudaSuccess)
    return LAWCAT_ERR_CUDA;
  LAWCAT_LAUNCH("decode_features", c.stream, decode_features_kernel<T><<<p.H * ((p.B + DEC_SEQ - 1) / DEC_SEQ), DEC_THREADS, smem1, c.stream>>>(a));
  LAWCAT_CHECK_LAUNCH();
  const size_t smem2 = sizeof(float) * ((size_t)3 * p.d_k + p.d_v + (size_t)(DEC_THREADS / 16) * p.d_v);
  if (smem2 > 48 * 1024 &&
      cudaFuncSetAttribute(decode_state_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2) != cudaSuccess)
    return LAWCAT_ERR_CUDA;
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.B * p.H));
    cfg.blockDim = dim3(DEC_THREADS);
    cfg.dynamicSmemBytes = smem2;
    cfg.stream = c.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    LAWCAT_LAUNCH("decode_state", c.stream, cudaLaunchKernelEx(&cfg, decode_state_kernel<T>, a));
  }
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

int launch_decode(const Ctx& c, const void* q_t, const void* k_t, const void* v_t, const void* gate_t,
                  const void* w_q, const void* w_k, const void* W, float* S, float* z, void* cache_q, void* cache_k,
                  void* o_t, void* ws) {
  const lawcat_params& p = *c.p;
  DecodeArgs a{};
  a.q_t = q_t; a.k_t = k_t; a.v_t = v_t; a.gate_t = gate_t; a.w_q = w_q; a.w_k = w_k; a.W = W;
  a.S = S; a.z = z; a.cache_q = cache_q; a.cache_k = cache_k; a.o_t = o_t;
  a.vecs = (float*)ws;
  a.den = a.vecs + (size_t)p.B * p.H * 3 * p.d_k;
  a.B = p.B; a.H = p.H; a.Hkv = p.H_kv; a.dk = p.d_k; a.dv = p.d_v; a.K = p.conv_k; a.gd = p.gate_dim;
  a.phi = p.phi; a.gate_mode = p.gate_mode; a.normalize = p.normalize;
  a.inv_tau = 1.f / p.gate_tau; a.eps = p.eps;
  if (p.dtype == LAWCAT_F32) return decode_typed<float>(c, a);
  return decode_typed<bf16>(c, a);
}

}  // namespace lawcat
