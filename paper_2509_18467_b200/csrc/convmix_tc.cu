// Tensor-core kernels for conv -> shared linear layer -> softmax feature map (Section 4.1) and for the chain rule back
// through them (distillation step, Section 5.1), bf16 storage.
//
// Forward: one thread block = one (batch, query head, tile of 128 tokens), both streams one after the other (they share
// W_h): raw rows (with the conv_k - 1 rows in front) into shared memory, depthwise causal conv in fp32 -> fp16 operand,
// Y = u W_h as one tcgen05 product per 16 channels (fp32 accumulator in tensor memory), phi (softmax over the row, or the
// elementwise 1 + ELU / identity of Section 2) by the thread that owns the row's TMEM lane, 16-bit or fp32 store.
// Backward (head width 64): one block = one (batch, key head, tile); for each query head of
// the group and each stream it recomputes u and p = softmax(u W_h), applies the softmax Jacobian dy = p (dp - p . dp),
// and forms du = dy W_h^T (the key stream summed over the group in registers) and dW_h += u^T dy (accumulators of two
// heads at a time in tensor memory, flushed with atomic adds). The conv's own backward then runs on du.
// Tiles are unswizzled 8x8 core matrices with every 8-column slab contiguous (see gla_tc.cu): W_h serves as the
// MN-major B of the forward mix and, without a second copy, as the K-major B of dy W_h^T.
#include <cuda.h>
#include <cuda_fp16.h>

#include <mutex>

#include "common.cuh"
#include "octet_tile.cuh"
#include "tc_common.cuh"

namespace lawcat {
namespace ctc {

struct CArgs {
  const bf16 *q, *k, *w_q, *w_k, *W, *cache_q, *cache_k;
  void *qdot, *kdot;                 // forward outputs (bf16 or fp32)
  const void *d_qdot, *d_kdot;       // backward inputs (bf16 or fp32)
  float *du_q, *du_k, *dW;           // backward outputs: d(conv out) per stream (fp32), dW (fp32, atomic adds)
  int* dev_status;
  int B, T, H, Hkv, K, phi;
  int unshared;  // 1: W is [2,H,D,D], the key stream mixes with the second set (forward kernel only)
};

// hint: fetch the 128-byte line at p towards L2 (these kernels walk their tiles in lock-step; the hint lets the next
// tile's rows travel while the current one is computed)
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// raw rows [t0 - HALO, t0 + TT) of one head into shared memory (rows before the sequence come from the conv cache or are
// zero, rows past its end are zero), and the head's taps as fp32 [D][4] (zero beyond the conv width)
template <int D>
__device__ __forceinline__ void load_raw_and_taps(uint8_t* s_raw, float* s_w, const bf16* x, const bf16* w, const bf16* cache,
                                                  int b, int t0, int T, int NH, int head, int K, int tid, int nthreads) {
  using L = Lay<D>;
  for (int idx = tid; idx < (TT + HALO) * L::OPR; idx += nthreads) {
    const int rr = idx / L::OPR, o = idx % L::OPR, t = t0 - HALO + rr;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (t >= 0 && t < T) {
      v = *reinterpret_cast<const uint4*>(x + (((size_t)b * T + t) * NH + head) * D + o * 8);
    } else if (t < 0 && cache != nullptr && t + (K - 1) >= 0) {
      v = *reinterpret_cast<const uint4*>(cache + (((size_t)b * (K - 1) + t + (K - 1)) * NH + head) * D + o * 8);
    }
    *reinterpret_cast<uint4*>(s_raw + rr * L::RAW_STRIDE + o * 16) = v;
  }
  for (int idx = tid; idx < D * 4; idx += nthreads) {
    const int c = idx >> 2, dl = idx & 3;
    s_w[idx] = dl < K ? __bfloat162float(w[((size_t)head * D + c) * K + dl]) : 0.f;
  }
}

// depthwise causal conv of the tile in fp32, result as the fp16 A operand of the mix; s_ul (nullable): the low part
// u - fp16(u), again in fp16, for products that take u as a two-term operand
template <int D>
__device__ __forceinline__ void conv_tile(const uint8_t* s_raw, const float* s_w, uint8_t* s_u, int tid, int nthreads,
                                          uint8_t* s_ul = nullptr) {
  using L = Lay<D>;
  const int o = tid % L::OPR;
  float w[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float4 t4 = *reinterpret_cast<const float4*>(s_w + (o * 8 + i) * 4);
    w[i][0] = t4.x; w[i][1] = t4.y; w[i][2] = t4.z; w[i][3] = t4.w;
  }
#pragma unroll 1
  for (int r = tid / L::OPR; r < TT; r += nthreads / L::OPR) {
    float u[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int dl = 0; dl < 4; ++dl) {
      float x[8];
      unpack8b(*reinterpret_cast<const uint4*>(s_raw + (r + HALO - dl) * L::RAW_STRIDE + o * 16), x);
#pragma unroll
      for (int i = 0; i < 8; ++i) u[i] = fmaf(w[i][dl], x[i], u[i]);
    }
    const uint4 ph = pack8f16(u);
    *reinterpret_cast<uint4*>(s_u + toff(L::SLAB_U, r, o * 8)) = ph;
    if (s_ul != nullptr) {
      const __half2* h2 = reinterpret_cast<const __half2*>(&ph);
      float lo[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h2[i]);
        lo[2 * i] = u[2 * i] - f.x;
        lo[2 * i + 1] = u[2 * i + 1] - f.y;
      }
      *reinterpret_cast<uint4*>(s_ul + toff(L::SLAB_U, r, o * 8)) = pack8f16(lo);
    }
  }
}

template <int D, typename TO>
__global__ void __launch_bounds__(128) convmix_tc_fwd_kernel(const CArgs a) {
  using L = Lay<D>;
  extern __shared__ __align__(128) uint8_t sg[];
  // fp32 outputs (the features a fused caller keeps in fp32) take the conv output as a two-term fp16 pair: about 21 bits
  // instead of 11, so that the features carry no visible rounding into the gradients computed from them
  constexpr bool TWO = sizeof(TO) == 4;
  constexpr uint32_t OFF_WT = 0, OFF_U = OFF_WT + L::TILE_W, OFF_UL = OFF_U + L::TILE_U;
  constexpr uint32_t OFF_RAW = OFF_UL + (TWO ? L::TILE_U : 0) + 2048 /* rows past the tile */;
  constexpr uint32_t OFF_TAPS = OFF_RAW + (L::RAW_BYTES + 15) / 16 * 16, OFF_BAR = OFF_TAPS + D * 4 * 4;
  const uint32_t sb = smem_u32(sg);
  const int tid = threadIdx.x, warp = tid >> 5;
  volatile int* const s_flags = reinterpret_cast<volatile int*>(sg + OFF_BAR + 16);  // [0] tmem base, [1] abort
  const int t0 = blockIdx.x * TT, bh = blockIdx.y, h = bh % a.H, b = bh / a.H;
  const int G = a.H / a.Hkv, j = h / G;
  if (tid == 0) {
    mbar_init(sb + OFF_BAR, 1);
    mbar_fence_init();
    s_flags[1] = 0;
  }
  if (warp == 0) {
    tmem_alloc(sb + OFF_BAR + 16, D);
    tmem_relinquish();
  }
  load_w_tile<D>(sg + OFF_WT, a.W + (size_t)h * D * D, tid, 128);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = (uint32_t)s_flags[0];
  const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
  Waiter wt{sb + OFF_BAR, 0u, s_flags + 1, a.dev_status};
#pragma unroll 1
  for (int stream = 0; stream < 2; ++stream) {
    const bf16* x = stream ? a.k : a.q;
    const int NH = stream ? a.Hkv : a.H, head = stream ? j : h;
    // (a separate linear layer per stream: the key stream's W_h replaces the tile; the product that read the query
    // stream's has completed, and the barriers below publish the new tile together with the conv output)
    if (stream == 1 && a.unshared) load_w_tile<D>(sg + OFF_WT, a.W + ((size_t)a.H + h) * D * D, tid, 128);
    load_raw_and_taps<D>(sg + OFF_RAW, reinterpret_cast<float*>(sg + OFF_TAPS), x, stream ? a.w_k : a.w_q,
                         stream ? a.cache_k : a.cache_q, b, t0, a.T, NH, head, a.K, tid, 128);
    if (stream == 0 && t0 + tid < a.T) {  // the key stream's raw row of this thread, towards L2 meanwhile
      const bf16* kr = a.k + (((size_t)b * a.T + t0 + tid) * a.Hkv + j) * D;
      prefetch_l2(kr);
      if (D * 2 > 128) prefetch_l2(kr + 64);
    }
    __syncthreads();
    conv_tile<D>(sg + OFF_RAW, reinterpret_cast<const float*>(sg + OFF_TAPS), sg + OFF_U, tid, 128,
                 TWO ? sg + OFF_UL : nullptr);
    fence_proxy_async();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (tid == 0) {
      const uint32_t idesc = instr_desc(128, D, FMT_F16, MAJOR_K, MAJOR_MN);
      const uint64_t da = kview(sb + OFF_U, L::SLAB_U), db = mview(sb + OFF_WT, L::SLAB_W);
      for (int kk = 0; kk < D / 16; ++kk) mma_f16(tmem, dadv(da, 2 * L::SLAB_U * kk), dadv(db, 256 * kk), idesc, kk > 0);
      if (TWO) {
        const uint64_t dl = kview(sb + OFF_UL, L::SLAB_U);
        for (int kk = 0; kk < D / 16; ++kk) mma_f16(tmem, dadv(dl, 2 * L::SLAB_U * kk), dadv(db, 256 * kk), idesc, 1);
      }
      mma_commit(sb + OFF_BAR);
    }
    wt.wait();
    // phi over the row this thread owns (row = token t0 + tid): softmax, or elementwise 1 + ELU / identity
    if (a.phi != LAWCAT_PHI_SOFTMAX) {
      const int t = t0 + tid;
      float y[32];
      TO* out = reinterpret_cast<TO*>(stream ? a.kdot : a.qdot) + (((size_t)b * a.T + t) * a.H + h) * D;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        tmem_ld32(lane_base + c0, y);
        tmem_wait_ld();
        if (a.phi == LAWCAT_PHI_ELU1) {
#pragma unroll
          for (int i = 0; i < 32; ++i) y[i] = y[i] > 0.f ? y[i] + 1.f : __expf(y[i]);
        }
        if (t < a.T) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) store_row8(out + c0 + i, y + i);
        }
      }
    } else {
      const int t = t0 + tid;
      float y[32], m = -INFINITY, sum = 0.f;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        tmem_ld32(lane_base + c0, y);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) m = fmaxf(m, y[i]);
      }
      const float mb = m * 1.4426950408889634f;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        tmem_ld32(lane_base + c0, y);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) sum += ex2f(fmaf(y[i], 1.4426950408889634f, -mb));
      }
      const float inv = 1.f / sum;
      TO* out = reinterpret_cast<TO*>(stream ? a.kdot : a.qdot) + (((size_t)b * a.T + t) * a.H + h) * D;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        tmem_ld32(lane_base + c0, y);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) y[i] = ex2f(fmaf(y[i], 1.4426950408889634f, -mb)) * inv;
        if (t < a.T) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) store_row8(out + c0 + i, y + i);
        }
      }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
  }
  if (warp == 0) tmem_dealloc(tmem, D);
}

// Backward through phi and the mix for head width 64: du_q [B,T,H,64], du_k [B,T,Hkv,64] (fp32), dW [H,64,64] (atomic adds
// into a zeroed array). TG: type of the incoming gradients d_qdot, d_kdot.
template <typename TG>
__global__ void __launch_bounds__(128, 2) convmix_tc_bwd_kernel(const CArgs a) {
  constexpr int D = 64;
  using L = Lay<D>;
  extern __shared__ __align__(128) uint8_t sg[];
  constexpr uint32_t OFF_WT = 0, OFF_U = OFF_WT + L::TILE_W, OFF_DY = OFF_U + L::TILE_U, OFF_DYL = OFF_DY + L::TILE_U;
  constexpr uint32_t OFF_UL = OFF_DYL + L::TILE_U;  // low part of the conv output (second term of u in dW)
  constexpr uint32_t OFF_RAW = OFF_UL + L::TILE_U + 2048, OFF_TAPS = OFF_RAW + (L::RAW_BYTES + 15) / 16 * 16;
  constexpr uint32_t OFF_BAR = OFF_TAPS + D * 4 * 4;
  constexpr uint32_t COL_Y = 0, COL_DW = 64, TMEM_COLS = 256;  // Y / du, and the dW accumulators of two heads at a time
  const uint32_t sb = smem_u32(sg);
  const int tid = threadIdx.x, warp = tid >> 5;
  volatile int* const s_flags = reinterpret_cast<volatile int*>(sg + OFF_BAR + 16);
  const int t0 = blockIdx.x * TT, bj = blockIdx.y, j = bj % a.Hkv, b = bj / a.Hkv;
  const int G = a.H / a.Hkv;
  if (tid == 0) {
    mbar_init(sb + OFF_BAR, 1);
    mbar_fence_init();
    s_flags[1] = 0;
  }
  if (warp == 0) {
    tmem_alloc(sb + OFF_BAR + 16, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = (uint32_t)s_flags[0];
  const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
  Waiter wt{sb + OFF_BAR, 0u, s_flags + 1, a.dev_status};
  const int t = t0 + tid;       // the row this thread owns in the epilogues
  const bool valid = t < a.T;
  float duk[D];                 // d(conv out) of the key stream, summed over the heads of the group
#pragma unroll
  for (int i = 0; i < D; ++i) duk[i] = 0.f;
#pragma unroll 1
  for (int g = 0; g < G; ++g) {
    const int h = j * G + g;
    load_w_tile<D>(sg + OFF_WT, a.W + (size_t)h * D * D, tid, 128);
#pragma unroll 1
    for (int stream = 0; stream < 2; ++stream) {
      const bf16* x = stream ? a.k : a.q;
      const int NH = stream ? a.Hkv : a.H, head = stream ? j : h;
      load_raw_and_taps<D>(sg + OFF_RAW, reinterpret_cast<float*>(sg + OFF_TAPS), x, stream ? a.w_k : a.w_q,
                           stream ? a.cache_k : a.cache_q, b, t0, a.T, NH, head, a.K, tid, 128);
      if (valid) {
        // towards L2 while conv and mix run: this thread's row of the incoming gradient (read in the epilogue below),
        // and its raw row of the next (head, stream) step
        const char* dpr = reinterpret_cast<const char*>(stream ? a.d_kdot : a.d_qdot) +
                          ((((size_t)b * a.T + t) * a.H + h) * D) * sizeof(TG);
        prefetch_l2(dpr);
        if (sizeof(TG) * D > 128) prefetch_l2(dpr + 128);
        const int ns = stream ^ 1, ng = g + stream;  // the step that follows
        if (ng < G) {
          const bf16* nx = ns ? a.k : a.q;
          const int nNH = ns ? a.Hkv : a.H, nhead = ns ? j : j * G + ng;
          prefetch_l2(nx + (((size_t)b * a.T + t) * nNH + nhead) * D);
        }
      }
      __syncthreads();
      conv_tile<D>(sg + OFF_RAW, reinterpret_cast<const float*>(sg + OFF_TAPS), sg + OFF_U, tid, 128, sg + OFF_UL);
      fence_proxy_async();
      tc_fence_before_sync();
      __syncthreads();
      tc_fence_after_sync();
      if (tid == 0) {  // Y = u W_h
        const uint32_t idesc = instr_desc(128, D, FMT_F16, MAJOR_K, MAJOR_MN);
        const uint64_t da = kview(sb + OFF_U, L::SLAB_U), db = mview(sb + OFF_WT, L::SLAB_W);
        for (int kk = 0; kk < D / 16; ++kk) mma_f16(tmem + COL_Y, dadv(da, 2 * L::SLAB_U * kk), dadv(db, 256 * kk), idesc, kk > 0);
        const uint64_t dal = kview(sb + OFF_UL, L::SLAB_U);  // (second term of u: the same features as the forward recompute)
        for (int kk = 0; kk < D / 16; ++kk) mma_f16(tmem + COL_Y, dadv(dal, 2 * L::SLAB_U * kk), dadv(db, 256 * kk), idesc, 1);
        mma_commit(sb + OFF_BAR);
      }
      wt.wait();
      // p = softmax(y), dy = p (dp - p . dp): this thread's row, two-term fp16 operand (rows past the end: zero)
      {
        float y[D];
        tmem_ld32(lane_base + COL_Y, y);
        tmem_ld32(lane_base + COL_Y + 32, y + 32);
        tmem_wait_ld();
        float m = -INFINITY, sum = 0.f, dot = 0.f;
#pragma unroll
        for (int i = 0; i < D; ++i) m = fmaxf(m, y[i]);
        const float mb = m * 1.4426950408889634f;
#pragma unroll
        for (int i = 0; i < D; ++i) {
          y[i] = ex2f(fmaf(y[i], 1.4426950408889634f, -mb));
          sum += y[i];
        }
        const float inv = 1.f / sum;
        const TG* dp = reinterpret_cast<const TG*>(stream ? a.d_kdot : a.d_qdot) + (((size_t)b * a.T + t) * a.H + h) * D;
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
          for (int c0 = 0; c0 < D; c0 += 8) {
            float g8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (valid) load_row8(dp + c0, g8);
            if (pass == 0) {
#pragma unroll
              for (int i = 0; i < 8; ++i) dot = fmaf(y[c0 + i] * inv, g8[i], dot);
            } else {
              float dy[8], hi[8], lo[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) dy[i] = valid ? y[c0 + i] * inv * (g8[i] - dot) : 0.f;
              const uint4 ph = pack8f16(dy);
              const __half2* h2 = reinterpret_cast<const __half2*>(&ph);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(h2[i]);
                hi[2 * i] = f.x; hi[2 * i + 1] = f.y;
              }
#pragma unroll
              for (int i = 0; i < 8; ++i) lo[i] = dy[i] - hi[i];
              *reinterpret_cast<uint4*>(sg + OFF_DY + toff(L::SLAB_U, tid, c0)) = ph;
              *reinterpret_cast<uint4*>(sg + OFF_DYL + toff(L::SLAB_U, tid, c0)) = pack8f16(lo);
            }
          }
        }
      }
      fence_proxy_async();
      tc_fence_before_sync();
      __syncthreads();
      tc_fence_after_sync();
      if (tid == 0) {
        // du = dy W_h^T (two-term dy) into Y's columns; dW_h += u^T dy
        const uint32_t id_du = instr_desc(128, D, FMT_F16, MAJOR_K, MAJOR_K);
        const uint64_t dh = kview(sb + OFF_DY, L::SLAB_U), dl = kview(sb + OFF_DYL, L::SLAB_U), dw = kview(sb + OFF_WT, L::SLAB_W);
        for (int kk = 0; kk < D / 16; ++kk) mma_f16(tmem + COL_Y, dadv(dh, 2 * L::SLAB_U * kk), dadv(dw, 2 * L::SLAB_W * kk), id_du, kk > 0);
        for (int kk = 0; kk < D / 16; ++kk) mma_f16(tmem + COL_Y, dadv(dl, 2 * L::SLAB_U * kk), dadv(dw, 2 * L::SLAB_W * kk), id_du, 1);
        const uint32_t id_dw = instr_desc(128, D, FMT_F16, MAJOR_MN, MAJOR_MN);
        // (both factors two-term: u_hi dy_hi + u_lo dy_hi + u_hi dy_lo; with few tokens in a call the weight gradient is
        // a sum of few products and the rounding of single 16-bit operands would show in its largest entries)
        const uint64_t ua = mview(sb + OFF_U, L::SLAB_U), ual = mview(sb + OFF_UL, L::SLAB_U);
        const uint64_t yb = mview(sb + OFF_DY, L::SLAB_U), ybl = mview(sb + OFF_DYL, L::SLAB_U);
        for (int kk = 0; kk < TT / 16; ++kk)
          mma_f16(tmem + COL_DW + 64 * (g & 1), dadv(ua, 256 * kk), dadv(yb, 256 * kk), id_dw, (stream > 0 || kk > 0) ? 1u : 0u);
        for (int kk = 0; kk < TT / 16; ++kk)
          mma_f16(tmem + COL_DW + 64 * (g & 1), dadv(ual, 256 * kk), dadv(yb, 256 * kk), id_dw, 1u);
        for (int kk = 0; kk < TT / 16; ++kk)
          mma_f16(tmem + COL_DW + 64 * (g & 1), dadv(ua, 256 * kk), dadv(ybl, 256 * kk), id_dw, 1u);
        mma_commit(sb + OFF_BAR);
      }
      wt.wait();
      {
        float du[D];
        tmem_ld32(lane_base + COL_Y, du);
        tmem_ld32(lane_base + COL_Y + 32, du + 32);
        tmem_wait_ld();
        if (stream == 0) {
          if (valid) {
            float* dst = a.du_q + (((size_t)b * a.T + t) * a.H + h) * D;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 8) store_row8(dst + c0, du + c0);
          }
        } else {
#pragma unroll
          for (int i = 0; i < D; ++i) duk[i] += du[i];
        }
      }
      tc_fence_before_sync();
      __syncthreads();
      tc_fence_after_sync();
    }
    // dW of the last two heads (or the last one): row c of each accumulator is owned by thread c
    if (((g & 1) || g == G - 1) && warp < 2 && a.dW) {
#pragma unroll 1
      for (int gg = g & ~1; gg <= g; ++gg) {
        float r[32];
#pragma unroll 1
        for (int c0 = 0; c0 < D; c0 += 32) {
          tmem_ld32(lane_base + COL_DW + 64 * (gg & 1) + c0, r);
          tmem_wait_ld();
          float* dst = a.dW + ((size_t)(j * G + gg) * D + tid) * D + c0;
#pragma unroll
          for (int i = 0; i < 32; ++i) atomicAdd(dst + i, r[i]);
        }
      }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
  }
  if (valid) {
    float* dst = a.du_k + (((size_t)b * a.T + t) * a.Hkv + j) * D;
#pragma unroll
    for (int c0 = 0; c0 < D; c0 += 8) store_row8(dst + c0, duk + c0);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

template <int D, typename TO>
constexpr uint32_t fwd_smem() {
  using L = Lay<D>;
  return L::TILE_W + (sizeof(TO) == 4 ? 2 : 1) * L::TILE_U + 2048 + (L::RAW_BYTES + 15) / 16 * 16 + D * 16 + 64;
}
constexpr uint32_t bwd_smem() {
  using L = Lay<64>;
  return L::TILE_W + 4 * L::TILE_U + 2048 + (L::RAW_BYTES + 15) / 16 * 16 + 64 * 16 + 64;
}

template <typename K>
static int raise_smem(K kernel, uint32_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess ? LAWCAT_OK : LAWCAT_ERR_CUDA;
}

}  // namespace ctc

bool convmix_tc_fwd_supported(const lawcat_params& p) {
  return p.dtype == LAWCAT_BF16 && (p.d_k == 64 || p.d_k == 128) && p.conv_k <= ctc::HALO + 1 && p.B > 0 && p.T > 0;
}
bool convmix_tc_bwd_supported(const lawcat_params& p) {
  return p.dtype == LAWCAT_BF16 && p.d_k == 64 && p.phi == LAWCAT_PHI_SOFTMAX && p.conv_k <= ctc::HALO + 1 && p.B > 0 &&
         p.T > 0 && !p.mix_unshared;
}

static ctc::CArgs convmix_tc_args(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                                  const void* cache_q, const void* cache_k) {
  const lawcat_params& p = *c.p;
  ctc::CArgs a{};
  a.q = (const bf16*)q; a.k = (const bf16*)k; a.w_q = (const bf16*)w_q; a.w_k = (const bf16*)w_k; a.W = (const bf16*)W;
  a.cache_q = (const bf16*)cache_q; a.cache_k = (const bf16*)cache_k;
  a.dev_status = c.dev_status;
  a.B = p.B; a.T = p.T; a.H = p.H; a.Hkv = p.H_kv; a.K = p.conv_k; a.phi = p.phi; a.unshared = p.mix_unshared;
  return a;
}

// qdot, kdot = softmax((conv x) W_h) for both streams; out_f32: fp32 outputs (scratch of a fused caller) instead of bf16
int launch_convmix_tc_fwd(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                          const void* cache_q, const void* cache_k, void* qdot, void* kdot, bool out_f32) {
  using namespace ctc;
  const lawcat_params& p = *c.p;
  CArgs a = convmix_tc_args(c, q, k, w_q, w_k, W, cache_q, cache_k);
  a.qdot = qdot; a.kdot = kdot;
  static std::mutex mu;
  static bool done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LAWCAT_ERR_CUDA;
  {
    std::lock_guard<std::mutex> lk(mu);
    if (!done[dev]) {
      if (raise_smem(convmix_tc_fwd_kernel<64, bf16>, fwd_smem<64, bf16>()) || raise_smem(convmix_tc_fwd_kernel<64, float>, fwd_smem<64, float>()) ||
          raise_smem(convmix_tc_fwd_kernel<128, bf16>, fwd_smem<128, bf16>()) || raise_smem(convmix_tc_fwd_kernel<128, float>, fwd_smem<128, float>()))
        return LAWCAT_ERR_CUDA;
      done[dev] = true;
    }
  }
  const dim3 grid((unsigned)((p.T + TT - 1) / TT), (unsigned)(p.B * p.H));
  LaunchScope _ls("convmix_tc_fwd", c.stream);
  if (p.d_k == 64) {
    if (out_f32) convmix_tc_fwd_kernel<64, float><<<grid, 128, fwd_smem<64, float>(), c.stream>>>(a);
    else convmix_tc_fwd_kernel<64, bf16><<<grid, 128, fwd_smem<64, bf16>(), c.stream>>>(a);
  } else {
    if (out_f32) convmix_tc_fwd_kernel<128, float><<<grid, 128, fwd_smem<128, float>(), c.stream>>>(a);
    else convmix_tc_fwd_kernel<128, bf16><<<grid, 128, fwd_smem<128, bf16>(), c.stream>>>(a);
  }
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

// du_q, du_k (fp32) and dW (atomic adds into the caller-zeroed array) from d_qdot, d_kdot (bf16, or fp32 when grads_f32)
int launch_convmix_tc_bwd(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                          const void* cache_q, const void* cache_k, const void* d_qdot, const void* d_kdot, bool grads_f32,
                          float* du_q, float* du_k, float* dW) {
  using namespace ctc;
  const lawcat_params& p = *c.p;
  CArgs a = convmix_tc_args(c, q, k, w_q, w_k, W, cache_q, cache_k);
  a.d_qdot = d_qdot; a.d_kdot = d_kdot; a.du_q = du_q; a.du_k = du_k; a.dW = dW;
  static std::mutex mu;
  static bool done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LAWCAT_ERR_CUDA;
  {
    std::lock_guard<std::mutex> lk(mu);
    if (!done[dev]) {
      if (raise_smem(convmix_tc_bwd_kernel<bf16>, bwd_smem()) || raise_smem(convmix_tc_bwd_kernel<float>, bwd_smem())) return LAWCAT_ERR_CUDA;
      done[dev] = true;
    }
  }
  const dim3 grid((unsigned)((p.T + TT - 1) / TT), (unsigned)(p.B * p.H_kv));
  LaunchScope _ls("convmix_tc_bwd", c.stream);
  if (grads_f32) convmix_tc_bwd_kernel<float><<<grid, 128, bwd_smem(), c.stream>>>(a);
  else convmix_tc_bwd_kernel<bf16><<<grid, 128, bwd_smem(), c.stream>>>(a);
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

}  // namespace lawcat
