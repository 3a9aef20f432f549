// The whole layer forward of Fig. 1 as ONE chunkwise tensor-core kernel for bf16 storage, d_k = d_v = 128:
// conv (Section 4.1) -> shared linear layer + softmax feature map (Section 4.1) -> normalized gated linear attention
// (Eq. 4 - Eq. 8) in its chunkwise-parallel form, with the d_k x (d_v+1) state [S | z] kept in tensor memory in fp32.
//
// One CTA walks one (batch, query head, segment of the sequence) in chunks of C = 64 tokens. Per chunk:
//   TMA      raw q, k (with the 3 halo rows the conv needs), gate logits and v tiles -> 128-byte-swizzled shared memory
//   conv     u = sum_delta w_delta * x_{t-delta} in fp32 -> fp16 rows of one stacked A operand (rows 0-63 the query
//            tokens, rows 64-127 the key tokens: both streams share W_h, so ONE M=128 MMA mixes both)
//   gate     g = log2 sigmoid(a) / tau per entry, then a scan outwards from the middle token gives the exponents
//            x_t = b_t - b_mid (b the running sum of g) in fp32. The middle reference keeps every factor 2^x within
//            2^(+-32 max|g|).
//   MMA 1    Y = [u_q; u_k] W_h      (fp16 operands: 3 more mantissa bits than bf16 for u; fp32 accumulate in TMEM)
//   phi      row softmax, one thread per token row, 32 columns at a time straight from tensor memory. Query rows keep
//            exp(y - max) unnormalized: a positive per-token factor cancels in Eq. 8. The decay factors ride in the
//            exponent of the softmax: qs = 2^(y' + x_t), ks = phi_k 2^(-x_i), kh = phi_k 2^(b_C - b_i) (fp16, <= phi_k)
//   MMA 2    P = qs ks^T ; O' = qs (2^b_mid [S|z]) ; [S|z] = 2^b_C [S|z] + kh^T [v|1]
//   mask     P_ti = 0 for i > t, rounded to fp16
//   MMA 3    O' += P [v|1]   (fp16 operands; v converts from bf16 to fp16 exactly)
//   out      o_t = O'_t[:d_v] / (O'_t[d_v] + eps) -> bf16 -> TMA store
// Operand precision: qs, ks and the state operand are fp16 (11-bit mantissa) while the chunk's x stay within
// +-8 and the state within +-3e4 -- the usual case -- and bf16 otherwise (range first). bf16 score weights would
// cost up to 2^-9 relative error per weight, which the first tokens of a sequence do not average out.
// Every MMA uses M = 128; where only 64 rows are meaningful (P, O') the upper 64 TMEM lanes hold unused results.
// Loops over column blocks are deliberately NOT unrolled: the chunk loop must stay well inside the instruction cache.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace lawcat {
namespace tc {

constexpr int D = 128;       // d_k = d_v
constexpr int C = 64;        // tokens per chunk
constexpr int MID = 31;      // reference token of the in-chunk decay factorization
constexpr int HALO = 3;      // halo rows loaded in front of a chunk (conv width up to 4)
constexpr int RAW_ROWS = C + HALO;
constexpr int THREADS = 256;

// shared memory map (byte offsets from a 1024-byte aligned base)
constexpr uint32_t OFF_W = 0;                       // W_h^T fp16, K-major, 2 slabs x [128 x 128 B]
constexpr uint32_t OFF_SBF = OFF_W + 32768;         // 2^b_mid * S, 16 bit, MN-major, 2 slabs x [128 x 128 B]
constexpr uint32_t OFF_A = OFF_SBF + 32768;         // stacked A operand: conv outputs, then qs / ks in place
constexpr uint32_t OFF_KH = OFF_A + 32768;          // kh^T, fp16, K-major A of the state update, [128 channels x 64 tokens]
constexpr uint32_t OFF_G = OFF_KH + 16384;          // gate logits (bf16), 2 slabs x [64 x 128 B]
constexpr uint32_t OFF_V = OFF_G + 16384;           // v bf16, then fp16 in place, MN-major B, 2 slabs x [64 x 128 B]
constexpr uint32_t RAW_SLAB = 9216;                 // 67 rows x 128 B rounded up to 1024
constexpr uint32_t OFF_QRAW = OFF_V + 16384;        // raw q tile (2 slabs); later the masked scores P (fp16, 16 KB)
constexpr uint32_t OFF_X = OFF_QRAW;                // after the conv: exponents x fp32 [64 x 128] over the raw tiles (32 KB)
constexpr uint32_t OFF_KRAW = OFF_QRAW + 2 * RAW_SLAB;  // raw k tile (2 slabs); later the output staging (16 KB)
constexpr uint32_t OFF_SZ = OFF_KRAW + 2 * RAW_SLAB;    // 2^b_mid * z as a [128 x 16] operand (column 0 is z)
constexpr uint32_t OFF_ONES = OFF_SZ + 4096;        // [64 x 16] fp16 operand whose column 0 is 1 (the "1" of [v|1])
constexpr uint32_t OFF_VEC = OFF_ONES + 2048;       // bm[128], ft[128], e63[128], qsum[64] fp32
constexpr uint32_t OFF_BAR = OFF_VEC + 3 * 512 + 256;  // mbarriers and scalars
constexpr uint32_t SMEM_BYTES = OFF_BAR + 64;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;  // slack for the manual 1024-byte alignment
static_assert(SMEM_ALLOC <= 232448, "shared memory budget");
constexpr float SMAX_F16 = 3.0e4f;  // largest |state entry| for which the operands are kept in fp16
constexpr float RMAX_F16 = 8.f;     // largest |log2 E| for which the operands are kept in fp16

// tensor memory map (32-bit columns)
constexpr uint32_t COL_Y = 0;      // [128 x 128] mix output
constexpr uint32_t COL_S = 128;    // [128 x 128] state S
constexpr uint32_t COL_O = 256;    // [128 x 128] numerator (lanes 0-63 meaningful)
constexpr uint32_t COL_P = 384;    // [128 x 64] scores (lanes 0-63 meaningful)
constexpr uint32_t COL_SZ = 448;   // [128 x 16] column 0: normalizer state z
constexpr uint32_t COL_OZ = 464;   // [128 x 16] column 0: denominator
constexpr uint32_t TMEM_COLS = 512;

constexpr uint32_t LOAD_BYTES = 4 * RAW_ROWS * 128 + 4 * C * 128;

struct TcArgs {
  const bf16 *w_q, *w_k, *W, *cache_q, *cache_k;
  const float *S0, *z0;  // state before the first token of the CTA's segment
  float *S_T, *z_T;      // state after the last token of the CTA's segment
  float* dtot;           // [B,H,nseg,128]: log2 of the total decay of the segment per key channel (nullable)
  int* dev_status;
  int T, H, Hkv, K;
  int nseg, seg_len;     // segments per sequence and tokens per segment (a multiple of C)
  int grid_nseg;         // segments of each sequence covered by this launch (the first grid_nseg of nseg)
  int seg_in;            // 1: S0/z0 are indexed [b,h,seg]; 0: [b,h] and they apply to segment 0 only
  int seg_out;           // 1: S_T/z_T are indexed [b,h,seg]; 0: [b,h] and only the last segment writes them
  int gate_mode;
  float inv_tau, eps;
};

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
  f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
}
__device__ __forceinline__ void unpack8h(const uint4& v, float* f) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __half22float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}
// 8 values -> 8 packed 16-bit values, fp16 or bf16
__device__ __forceinline__ uint4 pack8(const float* v, bool f16) {
  return f16 ? make_uint4(pack_f16(v[0], v[1]), pack_f16(v[2], v[3]), pack_f16(v[4], v[5]), pack_f16(v[6], v[7]))
             : make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
__device__ __forceinline__ uint16_t to16(float x, bool f16) {
  return f16 ? __half_as_ushort(__float2half_rn(x)) : __bfloat16_as_ushort(__float2bfloat16_rn(x));
}
__device__ __forceinline__ float from16(uint16_t x, bool f16) {
  return f16 ? __half2float(__ushort_as_half(x)) : __uint_as_float((uint32_t)x << 16);
}

// channels [8 jj, 8 jj + 8) of row t of the fp32 exponent tile (see the gate pass for its layout)
__device__ __forceinline__ void load_x8(uint32_t base, int t, int jj, float* x) {
  const uint4 lo = lds128(base + t * 512 + (((2 * jj) ^ (t & 7)) << 4));
  const uint4 hi = lds128(base + t * 512 + (((2 * jj + 1) ^ (t & 7)) << 4));
  x[0] = __uint_as_float(lo.x); x[1] = __uint_as_float(lo.y); x[2] = __uint_as_float(lo.z); x[3] = __uint_as_float(lo.w);
  x[4] = __uint_as_float(hi.x); x[5] = __uint_as_float(hi.y); x[6] = __uint_as_float(hi.z); x[7] = __uint_as_float(hi.w);
}

// log2 of the decay of one gate entry: LOGITS: log2(sigmoid(a)) / tau, LOGDECAY: a * log2(e).
__device__ __forceinline__ float log2_decay(float a, int gate_mode, float inv_tau) {
  const float L2E = 1.4426950408889634f;
  if (gate_mode == LAWCAT_GATE_LOGDECAY) return a * L2E;
  // -log2(1 + 2^x) with 2^x = exp(-a), branch-free: the clamp keeps 2^x finite, and beyond it log2(1 + 2^x) = x
  const float x = -a * L2E;
  return -fmaxf(x, lg2f(1.f + ex2f(fminf(x, 126.f)))) * inv_tau;
}

// MODE 0: the layer forward. MODE 1: state only (no query stream, no output): the end state of a segment that starts
// from the given state, used to hand the state across segments of one sequence.
template <int MODE>
__global__ void __launch_bounds__(THREADS, 1)
layer_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_g,
                const __grid_constant__ CUtensorMap tm_o, const TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sb = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* const sg = smem_raw + (sb - smem_u32(smem_raw));  // generic pointer to the aligned base
  float* const s_bm = reinterpret_cast<float*>(sg + OFF_VEC);  // per key channel: b_mid (log2)
  float* const s_ft = s_bm + 128;                             // per key channel: b_C - b_mid (log2)
  float* const s_e63 = s_bm + 256;                            // 2^ft
  float* const s_qsum = s_bm + 384;  // per query token: sum of exp(y - max), the dropped softmax normalizer
  volatile int* const s_flags = reinterpret_cast<volatile int*>(sg + OFF_BAR + 32);  // [0] tmem base, [1] abort
  // Range tracking (all as bits of non-negative floats): largest |log2 E| of the chunk; largest |state entry| seen by
  // the last state pass; largest |v| of the chunk; and the resulting bound on the state the NEXT state pass converts
  // (|S_new| <= |S_old| + 64 max|v| because kh <= 1).
  int* const s_rmax = const_cast<int*>(s_flags) + 2;
  int* const s_smax = s_rmax + 1;
  int* const s_vmax = s_rmax + 2;
  int* const s_sbound = s_rmax + 3;
  const uint32_t bar_load = sb + OFF_BAR, bar_mma = sb + OFF_BAR + 8;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int seg = blockIdx.x % a.grid_nseg;
  const int bh = blockIdx.x / a.grid_nseg;
  const int h = bh % a.H, b = bh / a.H;
  const int G = a.H / a.Hkv, j = h / G;
  const int t_begin = seg * a.seg_len;
  const int t_end = min(a.T, t_begin + a.seg_len);
  const int nchunks = (t_end - t_begin + C - 1) / C;
  const size_t seg_idx = (size_t)bh * a.nseg + seg;
  const size_t in_idx = a.seg_in ? seg_idx : (size_t)bh, out_idx = a.seg_out ? seg_idx : (size_t)bh;
  float dsum = 0.f;  // gate threads: log2 of this channel's total decay over the segment

  // ---- one-time setup --------------------------------------------------------------------------------------------
  if (tid == 0) {
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    mbar_fence_init();
    s_flags[1] = 0;
    *s_rmax = 0; *s_smax = 0; *s_vmax = 0; *s_sbound = 0;
    tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_g);
    tma_prefetch_desc(&tm_o);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(sb + OFF_BAR + 32, TMEM_COLS);
    tmem_relinquish();
  }
  // W_h^T into its K-major slabs as fp16: row e holds W[h][c][e] over c
  {
    const bf16* Wh = a.W + (size_t)h * D * D;
#pragma unroll 1
    for (int idx = tid; idx < 16 * D; idx += THREADS) {
      const int e = idx & (D - 1), oc = idx >> 7;
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        w[i] = pack_f16(__bfloat162float(Wh[(size_t)(oc * 8 + 2 * i) * D + e]),
                        __bfloat162float(Wh[(size_t)(oc * 8 + 2 * i + 1) * D + e]));
      sts128(sb + OFF_W + (oc >> 3) * 16384 + sw128(e, oc & 7), make_uint4(w[0], w[1], w[2], w[3]));
    }
  }
  // constant "ones" operand and a zeroed z operand (unswizzled 8x8 core matrices)
  for (int i = tid; i < (4096 + 2048) / 4; i += THREADS) reinterpret_cast<uint32_t*>(sg + OFF_SZ)[i] = 0u;
  __syncthreads();
  if (tid < C) *reinterpret_cast<__half*>(sg + OFF_ONES + (tid >> 3) * 128 + (tid & 7) * 16) = __float2half(1.f);
  // conv taps of this thread's channel octet (see the conv pass below)
  const int cv_stream = tid >> 7, cv_oct = tid & 15, cv_rg = (tid >> 4) & 7;
  float cw[8][4];
  {
    const bf16* w = cv_stream ? a.w_k : a.w_q;
    const int head = cv_stream ? j : h;
#pragma unroll
    for (int ch = 0; ch < 8; ++ch)
#pragma unroll
      for (int dl = 0; dl < 4; ++dl)
        cw[ch][dl] = dl < a.K ? __bfloat162float(w[((size_t)head * D + cv_oct * 8 + ch) * a.K + dl]) : 0.f;
  }
  fence_proxy_async();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = (uint32_t)s_flags[0];
  const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);

  // initial state into tensor memory: thread c owns row c of [S | z]
  if (tid < D) {
    const bool have = a.S0 != nullptr && (a.seg_in || seg == 0);
    float s[32], mx = 0.f;
#pragma unroll 1
    for (int blk = 0; blk < 4; ++blk) {
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        s[i] = have ? a.S0[(in_idx * D + tid) * D + blk * 32 + i] : 0.f;
        mx = fmaxf(mx, fabsf(s[i]));
      }
      tmem_st32(lane_base + COL_S + blk * 32, s);
    }
    const bool havez = a.z0 != nullptr && (a.seg_in || seg == 0);
    const float z0v = havez ? a.z0[in_idx * D + tid] : 0.f;
    tmem_st1(lane_base + COL_SZ, z0v);
    tmem_wait_st();
    mx = fmaxf(mx, fabsf(z0v));
    if (!(mx < 3.0e38f)) mx = 3.0e38f;  // NaN or inf in the given state: no fp16 operand
    atomicMax(s_sbound, __float_as_int(mx));
  }
  tc_fence_before_sync();
  __syncthreads();

  uint32_t ph_load = 0, ph_mma = 0;
  bool store_pending = false;

#define LAWCAT_WAIT_ALL(bar, phase)               \
  do {                                            \
    if (!mbar_wait(bar, phase)) s_flags[1] = 1;   \
    phase ^= 1u;                                  \
    __syncthreads();                              \
    if (s_flags[1]) goto done;                    \
  } while (0)

  // shared-memory descriptors of the MMA operands (all tiles sit at fixed addresses); a K step adds a constant
  const uint64_t dsc_a = smem_desc(sb + OFF_A, 16, 1024, LAYOUT_SW128);                // stacked A, K-major
  const uint64_t dsc_w = smem_desc(sb + OFF_W, 16, 1024, LAYOUT_SW128);                // W^T, K-major
  const uint64_t dsc_ks = smem_desc(sb + OFF_A + 8192, 16, 1024, LAYOUT_SW128);        // rows 64-127 of the stacked A
  const uint64_t dsc_s = smem_desc(sb + OFF_SBF, 16384, 1024, LAYOUT_SW128);           // state operand, MN-major
  const uint64_t dsc_sz = smem_desc(sb + OFF_SZ, 128, 2048, LAYOUT_NONE);
  const uint64_t dsc_kh = smem_desc(sb + OFF_KH, 16, 1024, LAYOUT_SW128);              // kh^T, K-major
  const uint64_t dsc_v = smem_desc(sb + OFF_V, 8192, 1024, LAYOUT_SW128);              // v, MN-major
  const uint64_t dsc_one = smem_desc(sb + OFF_ONES, 128, 1024, LAYOUT_NONE);
  const uint64_t dsc_p = smem_desc(sb + OFF_QRAW, 16, 1024, LAYOUT_SW128);             // masked scores, K-major
  // start-address field steps (units of 16 bytes): K-major operand 32 B per K step, the second 64-column slab 16 KB
  // further; MN-major swizzled operand 2048 B per K step; unswizzled [rows x 16] operand 256 B per K step
  auto kmajor_step = [](int k) -> uint64_t { return (uint64_t)((k >> 2) * (16384 >> 4) + (k & 3) * 2); };

  for (int n = 0; n < nchunks; ++n) {
    const int t0 = t_begin + n * C;
    const int nvalid = min(C, t_end - t0);

    // ---- TMA: raw q, k (with halo), gate, v -----------------------------------------------------------------------
    if (tid == 0) {
      if (store_pending) tma_store_wait_read();  // the output staging aliases the raw k tile
      mbar_arrive_expect_tx(bar_load, MODE == 0 ? LOAD_BYTES : LOAD_BYTES - 2 * RAW_ROWS * 128);
#pragma unroll 1
      for (int s = 0; s < 2; ++s) {
        if (MODE == 0) tma_load_4d(sb + OFF_QRAW + s * RAW_SLAB, &tm_q, bar_load, s * 64, h, t0 - HALO, b);
        tma_load_4d(sb + OFF_KRAW + s * RAW_SLAB, &tm_k, bar_load, s * 64, j, t0 - HALO, b);
        tma_load_4d(sb + OFF_G + s * 8192, &tm_g, bar_load, s * 64, h, t0, b);
        tma_load_4d(sb + OFF_V + s * 8192, &tm_v, bar_load, s * 64, j, t0, b);
      }
    }
    store_pending = false;
    LAWCAT_WAIT_ALL(bar_load, ph_load);
    if (tid == 0) *s_rmax = 0;

    // rows before the first token of the sequence come from the conv cache (TMA zero-filled them)
    if (t0 == 0 && a.K > 1 && (a.cache_q || a.cache_k)) {
      if (tid < 96) {
        const int st = tid / 48, r = (tid % 48) / 16, oc = tid % 16;
        const bf16* cache = st ? a.cache_k : a.cache_q;
        const int ci = r - (HALO + 1) + a.K;  // cache row of token r - HALO
        if (cache && ci >= 0 && (MODE == 0 || st == 1)) {
          const int NH = st ? a.Hkv : a.H, head = st ? j : h;
          const uint4 v = *reinterpret_cast<const uint4*>(cache + ((size_t)b * (a.K - 1) + ci) * NH * D + head * D + oc * 8);
          sts128(sb + (st ? OFF_KRAW : OFF_QRAW) + (oc >> 3) * RAW_SLAB + sw128(r, oc & 7), v);
        }
      }
      __syncthreads();
    }

    // ---- conv: thread = (stream, channel octet, 8 consecutive tokens), sliding window over the raw rows -------------
    if (MODE == 0 || cv_stream == 1) {
      const uint32_t raw = sb + (cv_stream ? OFF_KRAW : OFF_QRAW) + (cv_oct >> 3) * RAW_SLAB;
      const uint32_t dst = sb + OFF_A + (cv_oct >> 3) * 16384;
      const int jc = cv_oct & 7, r0 = cv_rg * 8;
      float x1[8], x2[8], x3[8], x0[8];
      unpack8(lds128(raw + sw128(r0 + 0, jc)), x3);
      unpack8(lds128(raw + sw128(r0 + 1, jc)), x2);
      unpack8(lds128(raw + sw128(r0 + 2, jc)), x1);
#pragma unroll 2
      for (int i = 0; i < 8; ++i) {
        unpack8(lds128(raw + sw128(r0 + 3 + i, jc)), x0);
        float u[8];
#pragma unroll
        for (int ch = 0; ch < 8; ++ch)
          u[ch] = fmaf(cw[ch][0], x0[ch], fmaf(cw[ch][1], x1[ch], fmaf(cw[ch][2], x2[ch], cw[ch][3] * x3[ch])));
        sts128(dst + sw128(cv_stream * 64 + r0 + i, jc), pack8(u, true));
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) { x3[ch] = x2[ch]; x2[ch] = x1[ch]; x1[ch] = x0[ch]; }
      }
    }

    __syncthreads();  // the raw q, k tiles are dead from here on: the exponents x take their place

    // ---- gate: thread = (key channel, half of the chunk). Exponents x_t = b_t - b_mid, scanned outwards from MID. ------
    {
      const int c = tid & 127, half = tid >> 7, jc = (c & 63) >> 3;
      const uint8_t* gcol = sg + OFF_G + (c >> 6) * 8192 + (c & 7) * 2;
      // x[t][c] fp32, 512-byte rows whose 16-byte chunks are XOR-swizzled with t & 7 (conflict-free for this
      // column-wise writer and for the row-wise readers of the phi pass)
      float* const xcol = reinterpret_cast<float*>(sg + OFF_X) + (c & 3);
      auto putx = [&](int t, float x) { xcol[t * 128 + (((c >> 2) ^ (t & 7)) << 2)] = x; };
      float g[32];  // log-decays of tokens [32 half, 32 half + 32): all loaded and evaluated before the serial scan
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const int t = half * 32 + i;
        const uint32_t raw = *reinterpret_cast<const uint16_t*>(gcol + sw128(t, jc));
        g[i] = t < nvalid ? log2_decay(__uint_as_float(raw << 16), a.gate_mode, a.inv_tau) : 0.f;
      }
      float acc = 0.f;
      if (half) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          acc += g[i];
          putx(32 + i, fmaxf(acc, -120.f));
        }
        s_ft[c] = acc;
      } else {
        putx(MID, 0.f);
#pragma unroll
        for (int i = MID - 1; i >= 0; --i) {
          acc += g[i + 1];
          putx(i, fminf(-acc, 120.f));
        }
        s_bm[c] = acc + g[0];
      }
      // exponents are clamped to +-120 so that no factor overflows or vanishes; a clamp is reported
      if (-acc > 120.f && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_NUMERIC);
      const float am = warp_max(-acc);
      if ((tid & 31) == 0) atomicMax(s_rmax, __float_as_int(am));  // g <= 0: the largest exponent magnitude
    }
    // ---- v: bf16 -> fp16 in place (exact for |v| in the fp16 normal range) --------------------------------------------
    {
      float vm = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t ad = sb + OFF_V + (uint32_t)(tid + THREADS * i) * 16;
        float x[8];
        unpack8(lds128(ad), x);
#pragma unroll
        for (int e = 0; e < 8; ++e) vm = fmaxf(vm, fabsf(x[e]));
        sts128(ad, pack8(x, true));
      }
      vm = warp_max(vm);
      if ((tid & 31) == 0) atomicMax(s_vmax, __float_as_int(vm < 3.0e38f ? vm : 3.0e38f));
    }
    fence_proxy_async();
    __syncthreads();
    // Operand type of this chunk (see the header): fp16 while the exponents and the state stay in range, else bf16.
    const bool f16 = __int_as_float(*s_rmax) <= RMAX_F16 && __int_as_float(*s_sbound) < SMAX_F16;

    // ---- MMA 1: Y = [u_q; u_k] W_h ------------------------------------------------------------------------------------
    if (tid == 0) {
      tc_fence_after_sync();
      constexpr uint32_t ID = instr_desc(128, 128, FMT_F16, MAJOR_K, MAJOR_K);
#pragma unroll 1
      for (int k = 0; k < 8; ++k) mma_f16(tmem + COL_Y, dsc_a + kmajor_step(k), dsc_w + kmajor_step(k), ID, k > 0);
      mma_commit(bar_mma);
    }

    // ---- state pass (overlaps MMA 1): operand 2^b_mid * [S|z] in 16 bit, accumulator [S|z] *= 2^b_C -----------------
    if (tid < D) {
      const int c = tid;
      const float bm = s_bm[c], ft = s_ft[c];
      const float dm = ex2f(bm), dC = ex2f(bm + ft);
      s_e63[c] = ex2f(fmaxf(ft, -120.f));
      dsum += bm + ft;
      float s[32], mx = 0.f;
#pragma unroll 1
      for (int blk = 0; blk < 4; ++blk) {
        tmem_ld32(lane_base + COL_S + blk * 32, s);
        tmem_wait_ld();
        if (MODE == 0) {
#pragma unroll
          for (int i = 0; i < 32; ++i) mx = fmaxf(mx, fabsf(s[i]));
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            float w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i] = dm * s[8 * q4 + i];
            sts128(sb + OFF_SBF + (blk >> 1) * 16384 + sw128(c, (blk & 1) * 4 + q4), pack8(w, f16));
          }
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) s[i] *= dC;
        tmem_st32(lane_base + COL_S + blk * 32, s);
      }
      const float z = tmem_ld1(lane_base + COL_SZ);
      tmem_wait_ld();
      if (MODE == 0) {
        *reinterpret_cast<uint16_t*>(sg + OFF_SZ + (c >> 3) * 128 + (c & 7) * 16) = to16(dm * z, f16);
        mx = warp_max(fmaxf(mx, fabsf(z)));
        if ((tid & 31) == 0) atomicMax(s_smax, __float_as_int(mx < 3.0e38f ? mx : 3.0e38f));
      }
      tmem_st1(lane_base + COL_SZ, dC * z);
      tmem_wait_st();
    }
    LAWCAT_WAIT_ALL(bar_mma, ph_mma);
    tc_fence_after_sync();

    // ---- phi: one thread per row of Y, 32 columns at a time -------------------------------------------------------
    if (tid < D && (MODE == 0 || tid >= C)) {
      const float L2E = 1.4426950408889634f;
      const int row = tid < C ? tid : tid - C;  // token of this row (query rows 0-63, key rows 64-127 of Y)
      float y[32];
      float m = -INFINITY;
#pragma unroll 1
      for (int blk = 0; blk < 4; ++blk) {
        tmem_ld32(lane_base + COL_Y + blk * 32, y);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) m = fmaxf(m, y[i]);
      }
      const float mb = m * L2E;
      if (tid < C) {
        float qsum = 0.f;
        const bool need_qsum = a.eps != 0.f;  // the dropped normalizer only matters next to eps
#pragma unroll 1
        for (int blk = 0; blk < 4; ++blk) {
          tmem_ld32(lane_base + COL_Y + blk * 32, y);
          tmem_wait_ld();
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            float x[8], v[8];
            load_x8(sb + OFF_X, row, blk * 4 + q4, x);
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = ex2f(fmaf(y[q4 * 8 + i], L2E, x[i] - mb));
            if (need_qsum) {
#pragma unroll
              for (int i = 0; i < 8; ++i) qsum += ex2f(fmaf(y[q4 * 8 + i], L2E, -mb));
            }
            sts128(sb + OFF_A + (blk >> 1) * 16384 + sw128(row, (blk & 1) * 4 + q4), pack8(v, f16));
          }
        }
        s_qsum[row] = qsum;
      } else {
        // key rows: a first sweep for the softmax sum, a second for ks = phi_k 2^-x and kh = ks 2^(b_C - b_mid)
        float sum = 0.f;
#pragma unroll 1
        for (int blk = 0; blk < 4; ++blk) {
          tmem_ld32(lane_base + COL_Y + blk * 32, y);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) sum += ex2f(fmaf(y[i], L2E, -mb));
        }
        const float inv = row < nvalid ? 1.f / sum : 0.f;  // tokens past the end contribute nothing
#pragma unroll 1
        for (int blk = 0; blk < 4; ++blk) {
          tmem_ld32(lane_base + COL_Y + blk * 32, y);
          tmem_wait_ld();
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int jj = blk * 4 + q4;  // channels [8 jj, 8 jj + 8)
            float x[8], ks[8];
            load_x8(sb + OFF_X, row, jj, x);
            const float4 ea = *reinterpret_cast<const float4*>(s_e63 + jj * 8);
            const float4 eb = *reinterpret_cast<const float4*>(s_e63 + jj * 8 + 4);
            const float e63[8] = {ea.x, ea.y, ea.z, ea.w, eb.x, eb.y, eb.z, eb.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) ks[i] = ex2f(fmaf(y[q4 * 8 + i], L2E, -mb - x[i])) * inv;
            if (MODE == 0) sts128(sb + OFF_A + (jj >> 3) * 16384 + sw128(C + row, jj & 7), pack8(ks, f16));
            // kh^T: row = key channel, 64 tokens (128 bytes) per row, so that the state update reads a K-major A operand
#pragma unroll
            for (int i = 0; i < 8; ++i)
              *reinterpret_cast<__half*>(sg + OFF_KH + (jj * 8 + i) * 128 + (((row >> 3) ^ i) << 4) + (row & 7) * 2) =
                  __float2half_rn(ks[i] * e63[i]);
          }
        }
      }
    }
    fence_proxy_async();
    tc_fence_before_sync();
    __syncthreads();

    // ---- MMA 2: scores, inter-chunk read-out, state update ---------------------------------------------------------
    if (tid == 0) {
      tc_fence_after_sync();
      if (MODE == 0) {
        const int fmt = f16 ? FMT_F16 : FMT_BF16;
        const uint32_t ID_P = instr_desc(128, 64, fmt, MAJOR_K, MAJOR_K);
        const uint32_t ID_O = instr_desc(128, 128, fmt, MAJOR_K, MAJOR_MN);
        const uint32_t ID_OZ = instr_desc(128, 16, fmt, MAJOR_K, MAJOR_MN);
        // bound on the state after this chunk's update, for the next chunk's choice of operand type
        *s_sbound = __float_as_int(__int_as_float(*s_smax) + 64.f * fmaxf(__int_as_float(*s_vmax), 1.f));
        *s_smax = 0;
        *s_vmax = 0;
#pragma unroll 1
        for (int k = 0; k < 8; ++k) {
          const uint64_t ad = dsc_a + kmajor_step(k);
          mma_f16(tmem + COL_P, ad, dsc_ks + kmajor_step(k), ID_P, k > 0);
          mma_f16(tmem + COL_O, ad, dsc_s + (uint64_t)(k * (2048 >> 4)), ID_O, k > 0);
          mma_f16(tmem + COL_OZ, ad, dsc_sz + (uint64_t)(k * (256 >> 4)), ID_OZ, k > 0);
        }
      }
      constexpr uint32_t ID_S = instr_desc(128, 128, FMT_F16, MAJOR_K, MAJOR_MN);
      constexpr uint32_t ID_SZ = instr_desc(128, 16, FMT_F16, MAJOR_K, MAJOR_MN);
#pragma unroll 1
      for (int k = 0; k < 4; ++k) {
        const uint64_t ad = dsc_kh + (uint64_t)(k * 2);
        mma_f16(tmem + COL_S, ad, dsc_v + (uint64_t)(k * (2048 >> 4)), ID_S, 1);
        mma_f16(tmem + COL_SZ, ad, dsc_one + (uint64_t)(k * (256 >> 4)), ID_SZ, 1);
      }
      mma_commit(bar_mma);
    }
    LAWCAT_WAIT_ALL(bar_mma, ph_mma);
    tc_fence_after_sync();

    if (MODE == 0) {
      // ---- causal mask, fp16 scores ---------------------------------------------------------------------------------
      if (tid < C) {
        const int t = tid;
        float p[32];
#pragma unroll 1
        for (int blk = 0; blk < 2; ++blk) {
          tmem_ld32(lane_base + COL_P + blk * 32, p);
          tmem_wait_ld();
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (blk * 32 + q4 * 8 + i <= t) ? p[q4 * 8 + i] : 0.f;
            sts128(sb + OFF_QRAW + sw128(t, blk * 4 + q4), pack8(v, true));
          }
        }
      }
      fence_proxy_async();
      tc_fence_before_sync();
      __syncthreads();

      // ---- MMA 3: O' += P [v|1] ---------------------------------------------------------------------------------------
      if (tid == 0) {
        tc_fence_after_sync();
        constexpr uint32_t ID_O = instr_desc(128, 128, FMT_F16, MAJOR_K, MAJOR_MN);
        constexpr uint32_t ID_OZ = instr_desc(128, 16, FMT_F16, MAJOR_K, MAJOR_MN);
#pragma unroll 1
        for (int k = 0; k < 4; ++k) {
          const uint64_t ad = dsc_p + (uint64_t)(k * 2);
          mma_f16(tmem + COL_O, ad, dsc_v + (uint64_t)(k * (2048 >> 4)), ID_O, 1);
          mma_f16(tmem + COL_OZ, ad, dsc_one + (uint64_t)(k * (256 >> 4)), ID_OZ, 1);
        }
        mma_commit(bar_mma);
      }
      LAWCAT_WAIT_ALL(bar_mma, ph_mma);
      tc_fence_after_sync();

      // ---- normalize (Eq. 8), stage, store ----------------------------------------------------------------------------
      if (tid < C) {
        const int t = tid;
        const float den = tmem_ld1(lane_base + COL_OZ);
        tmem_wait_ld();
        // the query features went in scaled by qsum (unnormalized softmax), so eps scales the same way
        const float inv = 1.f / (den + a.eps * s_qsum[t]);
        float o[32];
#pragma unroll 1
        for (int blk = 0; blk < 4; ++blk) {
          tmem_ld32(lane_base + COL_O + blk * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] *= inv;
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)
            sts128(sb + OFF_KRAW + (blk >> 1) * 8192 + sw128(t, (blk & 1) * 4 + q4), pack8(o + 8 * q4, false));
        }
      }
      fence_proxy_async();
      tc_fence_before_sync();
      __syncthreads();
      if (tid == 0) {
        tma_store_4d(&tm_o, sb + OFF_KRAW, 0, h, t0, b);
        tma_store_4d(&tm_o, sb + OFF_KRAW + 8192, 64, h, t0, b);
        tma_store_commit();
      }
      store_pending = true;
    }
  }

  // ---- final state ---------------------------------------------------------------------------------------------------
  tc_fence_after_sync();
  if (tid < D && a.dtot != nullptr) a.dtot[seg_idx * D + tid] = dsum;
  if (tid < D && a.S_T != nullptr && (a.seg_out || seg == a.nseg - 1)) {
    float s[32];
#pragma unroll 1
    for (int blk = 0; blk < 4; ++blk) {
      tmem_ld32(lane_base + COL_S + blk * 32, s);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; i += 4)
        *reinterpret_cast<float4*>(a.S_T + (out_idx * D + tid) * D + blk * 32 + i) = make_float4(s[i], s[i + 1], s[i + 2], s[i + 3]);
    }
    const float z = tmem_ld1(lane_base + COL_SZ);
    tmem_wait_ld();
    if (a.z_T) a.z_T[out_idx * D + tid] = z;
  }

done:
  if (tid == 0) {
    tma_store_wait_all();
    if (s_flags[1] && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_TIMEOUT);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
#undef LAWCAT_WAIT_ALL
}

}  // namespace tc
}  // namespace lawcat
