// Recurrent single-token decode (streaming inference, Section 6): the layer at one token with the conv cache of
// Section 4.1 and the constant-size state of Eq. 4. Two launches:
//   decode_features  conv -> shared linear layer -> feature map for the token's query and key, decay alpha = exp(g), the
//                    normalizer state z (Eq. 8's denominator) advanced in place; writes qdot, kdot, alpha and the
//                    denominator to the workspace. Two kernels: decode_features_tc_kernel (bf16, d_k = 64 or 128: one
//                    block per head and group of 16 or 32 sequences, the mix of all their vectors as one tensor-core
//                    product) and decode_features_kernel (any shape and type: one block per head and group of 8
//                    sequences, which share the head's W, fp32 FMA)
//   decode_state     (one block per sequence and head) S <- diag(alpha) S + kdot^T v (Eq. 4), o = qdot S / denominator (Eq. 8): the fp32 state is streamed
//                    through HBM once (read + write), which is the whole cost of the step; the same blocks then shift
//                    the conv caches (every reader of the caches belongs to the first launch, which has completed)
#include <mutex>
#include <type_traits>

#include "common.cuh"
#include "octet_tile.cuh"

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
  int unshared;  // 1: W is [2,H,dk,dk], the key stream's vectors mix with the second set
  float inv_tau, eps;
  int* dev_status;
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
    const T* Wk = Wh + (a.unshared ? (size_t)H * dk * dk : 0);  // (vectors 4 vg + 1, 4 vg + 3 are key-stream vectors)
    for (int it = tid; it < dk * (DEC_NV / 4); it += DEC_THREADS) {
      const int e = it % dk, vg = it / dk;
      float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
      for (int c = 0; c < dk; ++c) {
        const float w = a.w_smem ? ldf(s_W + c * dk + e) : ldf(Wh + (size_t)c * dk + e);
        const float wk = a.unshared ? ldf(Wk + (size_t)c * dk + e) : w;
        const float4 u = *reinterpret_cast<const float4*>(s_u + c * DEC_NV + 4 * vg);
        y.x = fmaf(u.x, w, y.x); y.y = fmaf(u.y, wk, y.y); y.z = fmaf(u.z, w, y.z); y.w = fmaf(u.w, wk, y.w);
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

// ---- decode_features on the tensor cores (bf16 storage, d_k = 64 or 128, conv width up to 4) -----------------------------
// One block per (query head, group of NSEQ sequences): the query vectors and the key vectors of the group share W_h
// (Section 4.1), so their mix is ONE product Y = U W_h on the tensor cores (fp32 accumulator in tensor memory). U, the conv
// outputs, goes in as a two-term fp16 pair hi + lo (two accumulating passes), which keeps about 21 bits of it; W_h is
// exact in fp16. The 2 NSEQ vectors of a group (query stream first) are written to the M = 128 operand several times
// over, once per group of 2 NSEQ rows: a warp reads only its own 32 lanes of tensor memory, and with the copies every warp
// of the block finds every vector in its lanes. Thread = (vector, 16 of its channels): conv from global memory in fp32,
// then, straight from tensor memory, phi, the decay, the normalizer state z advanced in place, and the denominator of
// Eq. 8; same workspace layout as decode_features_kernel. Small groups (16 sequences at d_k = 128) give enough blocks to
// fill the GPU at batch 64: the step is a chain of dependent memory round trips, not arithmetic.
constexpr int DFT_THREADS = 256;

template <int D>
struct DftLay {
  using L = ctc::Lay<D>;
  static constexpr int NSEQ = 2048 / D;        // sequences per block: 16 (d_k = 128), 32 (d_k = 64)
  static constexpr int LR = 2 * NSEQ;          // vectors per block
  static constexpr int NP = 2 * (128 / LR);    // threads per vector
  static constexpr int HC = D / NP;            // channels per thread
  static_assert(HC == 16, "one 16-column tensor-memory load per thread");
  static constexpr uint32_t OFF_WT = 0, OFF_U = OFF_WT + L::TILE_W, OFF_UL = OFF_U + L::TILE_U;
  static constexpr uint32_t OFF_Z = OFF_UL + L::TILE_U;                    // fp32 [NSEQ][D + 1]: z after the update
  static constexpr uint32_t OFF_TAPS = OFF_Z + NSEQ * (D + 1) * 4;         // fp32 [2][D][4]
  static constexpr uint32_t OFF_RED = OFF_TAPS + 2 * D * 4 * 4;            // fp32 [NP][LR]: exchange between a vector's threads
  static constexpr uint32_t OFF_BAR = (OFF_RED + 256 * 4 + 15) / 16 * 16;
  static constexpr uint32_t BYTES = OFF_BAR + 64;
};

template <int D>
__global__ void __launch_bounds__(DFT_THREADS) decode_features_tc_kernel(DecodeArgs a) {
  using namespace ctc;
  using L = Lay<D>;
  using M = DftLay<D>;
  constexpr int NSEQ = M::NSEQ, LR = M::LR, NP = M::NP, HC = M::HC;
  extern __shared__ __align__(128) uint8_t sg[];
  const uint32_t sb = smem_u32(sg);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int r = tid & 127, lr = r % LR, part = (r / LR) * 2 + (tid >> 7);
  const int stream = lr / NSEQ, seq = lr % NSEQ, c0 = part * HC;
  const int h = blockIdx.x, G = a.H / a.Hkv, j = h / G, K = a.K;
  const int b = blockIdx.y * NSEQ + seq;
  const bool valid = b < a.B;
  volatile int* const s_flags = reinterpret_cast<volatile int*>(sg + M::OFF_BAR + 16);  // [0] tmem base, [1] abort
  float* const s_taps = reinterpret_cast<float*>(sg + M::OFF_TAPS);
  float* const s_red = reinterpret_cast<float*>(sg + M::OFF_RED);
  float* const s_z = reinterpret_cast<float*>(sg + M::OFF_Z);
  const size_t bh = (size_t)(valid ? b : 0) * a.H + h;
  // ---- every global read that does not depend on another goes out first: W_h, the taps, this thread's conv rows (the
  // token, delta = 0, and the cache rows, delta >= 1: row K - 1 - delta), its gate values and its part of z
  uint4 wreg[D * L::OPR / DFT_THREADS];
  {
    const bf16* Wh = (const bf16*)a.W + (size_t)h * D * D;
#pragma unroll
    for (int k = 0; k < D * L::OPR / DFT_THREADS; ++k) {
      const int idx = tid + k * DFT_THREADS, c = idx / L::OPR, o = idx % L::OPR;
      wreg[k] = __ldg(reinterpret_cast<const uint4*>(Wh + (size_t)c * D + o * 8));
    }
  }
  uint4 xreg[4][HC / 8];
  {
    const int NH = stream ? a.Hkv : a.H, head = stream ? j : h;
    const bf16* tok = (const bf16*)(stream ? a.k_t : a.q_t) + ((size_t)(valid ? b : 0) * NH + head) * D + c0;
    const bf16* cache = (const bf16*)(stream ? a.cache_k : a.cache_q) + ((size_t)(valid ? b : 0) * (K - 1) * NH + head) * D + c0;
#pragma unroll
    for (int dl = 0; dl < 4; ++dl) {
#pragma unroll
      for (int o = 0; o < HC / 8; ++o) {
        xreg[dl][o] = make_uint4(0u, 0u, 0u, 0u);
        if (valid && dl < K)
          xreg[dl][o] = __ldg(reinterpret_cast<const uint4*>(dl == 0 ? tok + o * 8 : cache + (size_t)(K - 1 - dl) * NH * D + o * 8));
      }
    }
  }
  float zold[HC], graw[HC];
#pragma unroll
  for (int i = 0; i < HC; ++i) zold[i] = graw[i] = 0.f;
  if (stream == 1 && valid) {
    const bf16* gt = (const bf16*)a.gate_t + bh * a.gd;
    if (a.gd == 1) {
      graw[0] = __bfloat162float(gt[0]);
    } else {
#pragma unroll
      for (int o = 0; o < HC / 8; ++o) unpack8b(__ldg(reinterpret_cast<const uint4*>(gt + c0 + o * 8)), graw + o * 8);
    }
#pragma unroll
    for (int i = 0; i < HC; i += 4) {
      const float4 z4 = *reinterpret_cast<const float4*>(a.z + bh * D + c0 + i);
      zold[i] = z4.x; zold[i + 1] = z4.y; zold[i + 2] = z4.z; zold[i + 3] = z4.w;
    }
  }
  float treg[2 * D * 4 / DFT_THREADS];
#pragma unroll
  for (int k = 0; k < 2 * D * 4 / DFT_THREADS; ++k) {
    const int idx = tid + k * DFT_THREADS, st = idx / (D * 4), c = (idx >> 2) % D, dl = idx & 3;
    const bf16* w = st ? (const bf16*)a.w_k + ((size_t)j * D + c) * K : (const bf16*)a.w_q + ((size_t)h * D + c) * K;
    treg[k] = dl < K ? __bfloat162float(w[dl]) : 0.f;
  }
  // the blocks of decode_state may be scheduled from here on: they start with loads of S, which this kernel never
  // touches, and wait for the end of this grid before they read anything it writes
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#pragma unroll
  for (int k = 0; k < 2 * D * 4 / DFT_THREADS; ++k) s_taps[tid + k * DFT_THREADS] = treg[k];
  if (tid == 0) {
    mbar_init(sb + M::OFF_BAR, 1);
    mbar_fence_init();
    s_flags[1] = 0;
  }
  if (warp == 0) {
    tmem_alloc(sb + M::OFF_BAR + 16, D);
    tmem_relinquish();
  }
#pragma unroll
  for (int k = 0; k < D * L::OPR / DFT_THREADS; ++k) {  // W[h][c][e] (exact in fp16) as a tile with rows c, columns e
    const int idx = tid + k * DFT_THREADS, c = idx / L::OPR, o = idx % L::OPR;
    float f[8];
    unpack8b(wreg[k], f);
    *reinterpret_cast<uint4*>(sg + M::OFF_WT + toff(L::SLAB_W, c, o * 8)) = pack8f16(f);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = (uint32_t)s_flags[0];
  const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)c0;
  Waiter wt{sb + M::OFF_BAR, 0u, s_flags + 1, a.dev_status};

  // ---- conv of this thread's channels, written to every copy of its vector's row -------------------------------------------
  {
    const float* tp = s_taps + (stream * D + c0) * 4;
#pragma unroll
    for (int o = 0; o < HC / 8; ++o) {
      float u[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int dl = 0; dl < 4; ++dl) {
        float x[8];
        unpack8b(xreg[dl][o], x);
#pragma unroll
        for (int i = 0; i < 8; ++i) u[i] = fmaf(tp[(o * 8 + i) * 4 + dl], x[i], u[i]);
      }
      const uint4 ph = pack8f16(u);
      const __half2* h2 = reinterpret_cast<const __half2*>(&ph);
      float lo[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h2[i]);
        lo[2 * i] = u[2 * i] - f.x;
        lo[2 * i + 1] = u[2 * i + 1] - f.y;
      }
      const uint4 pl = pack8f16(lo);
#pragma unroll
      for (int cp = 0; cp < 128 / LR; ++cp) {
        *reinterpret_cast<uint4*>(sg + M::OFF_U + toff(L::SLAB_U, lr + cp * LR, c0 + o * 8)) = ph;
        *reinterpret_cast<uint4*>(sg + M::OFF_UL + toff(L::SLAB_U, lr + cp * LR, c0 + o * 8)) = pl;
      }
    }
  }
  fence_proxy_async();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (tid == 0) {  // Y = (U_hi + U_lo) W_h
    const uint32_t idesc = instr_desc(128, D, FMT_F16, MAJOR_K, MAJOR_MN);
    const uint64_t dh = kview(sb + M::OFF_U, L::SLAB_U), dl = kview(sb + M::OFF_UL, L::SLAB_U);
    const uint64_t db = mview(sb + M::OFF_WT, L::SLAB_W);
    for (int kk = 0; kk < D / 16; ++kk) mma_f16(tmem, dadv(dh, 2 * L::SLAB_U * kk), dadv(db, 256 * kk), idesc, kk > 0);
    for (int kk = 0; kk < D / 16; ++kk) mma_f16(tmem, dadv(dl, 2 * L::SLAB_U * kk), dadv(db, 256 * kk), idesc, 1);
    mma_commit(sb + M::OFF_BAR);
  }
  wt.wait();

  // ---- phi over this thread's channels of its vector ------------------------------------------------------------------------
  float y[HC];
  tmem_ld16(lane_base, y);
  tmem_wait_ld();
  if (a.phi == LAWCAT_PHI_SOFTMAX) {
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < HC; ++i) m = fmaxf(m, y[i]);
    s_red[part * LR + lr] = m;
    __syncthreads();
#pragma unroll
    for (int q = 0; q < NP; ++q) m = fmaxf(m, s_red[q * LR + lr]);
    const float mb = m * 1.4426950408889634f;
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < HC; ++i) {
      y[i] = ex2f(fmaf(y[i], 1.4426950408889634f, -mb));
      sum += y[i];
    }
    __syncthreads();  // (every thread of the vector has read the maxima)
    s_red[part * LR + lr] = sum;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int q = 0; q < NP; ++q) tot += s_red[q * LR + lr];
    const float inv = 1.f / tot;
#pragma unroll
    for (int i = 0; i < HC; ++i) y[i] *= inv;
  } else if (a.phi == LAWCAT_PHI_ELU1) {
#pragma unroll
    for (int i = 0; i < HC; ++i) y[i] = y[i] > 0.f ? y[i] + 1.f : expf(y[i]);
  }
  __syncthreads();  // (the exchange buffer is used again below)

  // ---- features and decays to the workspace, z advanced in place, denominator of Eq. 8 ----------------------------------------
  float* out = a.vecs + bh * 3 * D + stream * D + c0;
  if (valid) {
#pragma unroll
    for (int i = 0; i < HC; i += 4) *reinterpret_cast<float4*>(out + i) = make_float4(y[i], y[i + 1], y[i + 2], y[i + 3]);
  }
  if (stream == 1) {
    float* al = a.vecs + bh * 3 * D + 2 * D + c0;
    float* zg = a.z + bh * D + c0;
    float alpha[HC], zn[HC];
    const float a1 = (valid && a.gd == 1) ? expf(log_decay(graw[0], a.gate_mode, a.inv_tau)) : 0.f;
#pragma unroll
    for (int i = 0; i < HC; ++i) {
      alpha[i] = a.gd == 1 ? a1 : (valid ? expf(log_decay(graw[i], a.gate_mode, a.inv_tau)) : 0.f);
      zn[i] = fmaf(alpha[i], zold[i], y[i]);
      s_z[seq * (D + 1) + c0 + i] = zn[i];
    }
    if (valid) {
#pragma unroll
      for (int i = 0; i < HC; i += 4) {
        *reinterpret_cast<float4*>(al + i) = make_float4(alpha[i], alpha[i + 1], alpha[i + 2], alpha[i + 3]);
        *reinterpret_cast<float4*>(zg + i) = make_float4(zn[i], zn[i + 1], zn[i + 2], zn[i + 3]);
      }
    }
  }
  __syncthreads();
  if (stream == 0) {
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < HC; ++i) dot = fmaf(y[i], s_z[seq * (D + 1) + c0 + i], dot);
    s_red[part * LR + lr] = dot;
  }
  __syncthreads();
  if (stream == 0 && part == 0 && valid) {
    float den = a.eps;
#pragma unroll
    for (int q = 0; q < NP; ++q) den += s_red[q * LR + lr];
    a.den[bh] = den;
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, D);
  }
}

bool decode_tc_supported(const lawcat_params& p) {
  return p.dtype == LAWCAT_BF16 && (p.d_k == 64 || p.d_k == 128) && p.conv_k <= 4 && p.chunk != 1 && !p.mix_unshared;
}

template <int D>
static int launch_decode_features_tc(const Ctx& c, const DecodeArgs& a) {
  static std::mutex mu;
  static bool done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LAWCAT_ERR_CUDA;
  {
    std::lock_guard<std::mutex> lk(mu);
    if (!done[dev]) {
      if (cudaFuncSetAttribute(decode_features_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)DftLay<D>::BYTES) != cudaSuccess)
        return LAWCAT_ERR_CUDA;
      done[dev] = true;
    }
  }
  const dim3 grid((unsigned)a.H, (unsigned)((a.B + DftLay<D>::NSEQ - 1) / DftLay<D>::NSEQ));
  LAWCAT_LAUNCH("decode_features", c.stream,
                decode_features_tc_kernel<D><<<grid, DFT_THREADS, DftLay<D>::BYTES, c.stream>>>(a));
  return LAWCAT_OK;
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
  if (std::is_same<T, bf16>::value && decode_tc_supported(p)) {
    const int r = p.d_k == 64 ? launch_decode_features_tc<64>(c, a) : launch_decode_features_tc<128>(c, a);
    if (r) return r;
    LAWCAT_CHECK_LAUNCH();
  } else {
    size_t smem1 = sizeof(float) * (size_t)p.d_k * (2 * DEC_NV + DEC_SEQ) + sizeof(T) * (size_t)p.d_k * p.conv_k * (DEC_NV + 2);
    if (p.d_k > 32 * DEC_ZR) return LAWCAT_ERR_UNSUPPORTED;  // (one warp holds a sequence's normalizer state)
    const size_t wbytes = sizeof(T) * (size_t)p.d_k * p.d_k;
    a.w_smem = (!p.mix_unshared && smem1 + wbytes <= 100 * 1024) ? 1 : 0;  // (two sets of W are read from L2 in place)
    if (a.w_smem) smem1 += wbytes;
    if (smem1 > 48 * 1024 &&
        cudaFuncSetAttribute(decode_features_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1) != cudaSuccess)
      return LAWCAT_ERR_CUDA;
    LAWCAT_LAUNCH("decode_features", c.stream, decode_features_kernel<T><<<p.H * ((p.B + DEC_SEQ - 1) / DEC_SEQ), DEC_THREADS, smem1, c.stream>>>(a));
    LAWCAT_CHECK_LAUNCH();
  }
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
  a.inv_tau = 1.f / p.gate_tau; a.eps = p.eps; a.dev_status = c.dev_status; a.unshared = p.mix_unshared;
  if (p.dtype == LAWCAT_F32) return decode_typed<float>(c, a);
  return decode_typed<bf16>(c, a);
}

}  // namespace lawcat
