// The whole layer forward of Fig. 1 as ONE chunkwise tensor-core kernel for bf16 storage, d_k = d_v = 128:
// conv (Section 4.1) -> shared linear layer + softmax feature map (Section 4.1) -> normalized gated linear attention
// (Eq. 4 - Eq. 8) in its chunkwise-parallel form, with the d_k x (d_v+1) state [S | z] kept in tensor memory in fp32.
//
// One CTA walks one (batch, query head, segment of the sequence) in chunks of C = 64 tokens. Per chunk:
//   TMA      raw q, k (with the 3 halo rows the conv needs), gate logits and v tiles -> 128-byte-swizzled shared memory
//   conv     u = sum_delta w_delta * x_{t-delta} in fp32 -> fp16 rows of one stacked A operand (rows 0-63 the query
//            tokens, rows 64-127 the key tokens: both streams share W_h, so ONE M=128 MMA mixes both)
//   gate     g = logsigmoid(a)/tau, b = running sum of g inside the chunk, E_t = exp(b_t - b_mid) per channel (a scan
//            outwards from the middle token keeps every factor within exp(+-32 max|g|))
//   MMA 1    Y = [u_q; u_k] W_h      (fp16 operands: 3 more mantissa bits than bf16 for u; fp32 accumulate in TMEM)
//   phi      row softmax in registers (one thread per token row). Query rows keep exp(y - max) unnormalized: a positive
//            per-token factor cancels in Eq. 8. qs = phi_q * E_t, ks = phi_k / E_i: fp16 while the chunk's E stay
//            within 2^+-8 (3 more mantissa bits; the usual case), bf16 otherwise (range); kh = phi_k * exp(b_C - b_i)
//            (fp16, <= phi_k)
//   MMA 2    P = qs ks^T ; O' = qs (exp(b_mid) S_prev) ; [S|z] = exp(b_C) [S|z] + kh^T [v|1]
//   mask     P_ti = 0 for i > t, rounded to fp16 (bf16 weights would cost up to 2^-9 relative error per weight, which
//            the early tokens of a sequence do not average out)
//   MMA 3    O' += P [v|1]   (fp16 operands; v converts from bf16 to fp16 exactly)
//   out      o_t = O'_t[:d_v] / (O'_t[d_v] + eps) -> bf16 -> TMA store
// Every MMA uses M = 128; where only 64 rows are meaningful (P, O') the upper 64 TMEM lanes hold unused results.
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
constexpr uint32_t OFF_W = 0;                       // W_h^T, K-major, 2 slabs x [128 x 128 B]
constexpr uint32_t OFF_SBF = OFF_W + 32768;         // exp(b_mid) * S, bf16, MN-major, 2 slabs x [128 x 128 B]
constexpr uint32_t OFF_A = OFF_SBF + 32768;         // stacked A operand: conv outputs, then qs / ks in place
constexpr uint32_t OFF_KH = OFF_A + 32768;          // kh, fp16, MN-major A of the state update, 2 slabs x [64 x 128 B]
constexpr uint32_t OFF_G = OFF_KH + 16384;          // gate logits (bf16), 2 slabs x [64 x 128 B]
constexpr uint32_t OFF_V = OFF_G + 16384;           // v bf16, then fp16 in place, MN-major B, 2 slabs x [64 x 128 B]
constexpr uint32_t RAW_SLAB = 9216;                 // 67 rows x 128 B rounded up to 1024
constexpr uint32_t OFF_QRAW = OFF_V + 16384;        // raw q tile (2 slabs); later the masked scores P (fp16, 16 KB)
constexpr uint32_t OFF_E = OFF_QRAW;                // after the conv: E fp32 [64 x 128] over the raw q and k tiles (32 KB)
constexpr uint32_t OFF_KRAW = OFF_QRAW + 2 * RAW_SLAB;  // raw k tile (2 slabs); later the output staging (16 KB)
constexpr uint32_t OFF_SZ = OFF_KRAW + 2 * RAW_SLAB;    // exp(b_mid) * z as a [128 x 16] bf16 operand (column 0 is z)
constexpr uint32_t OFF_ONES = OFF_SZ + 4096;        // [64 x 16] fp16 operand whose column 0 is 1 (the "1" of [v|1])
constexpr uint32_t OFF_QB = OFF_ONES + 2048;        // qs in bf16 for the read-out MMA, K-major, 2 slabs x [64 x 128 B]
constexpr uint32_t OFF_VEC = OFF_QB + 16384;        // dm[128], dC[128], e63[128], qsum[64] fp32
constexpr uint32_t OFF_BAR = OFF_VEC + 3 * 512 + 256;  // mbarriers and scalars
constexpr uint32_t SMEM_BYTES = OFF_BAR + 64;
// The M = 128 read-out MMA reads 128 rows per slab of the 64-row qs tile: its (unused) rows 64-127 reach 8 KB past the
// tile, so the allocation extends that far; plus slack for the manual 1024-byte alignment.
constexpr uint32_t SMEM_ALLOC = OFF_QB + 16384 + 8192 + 1024;
static_assert(SMEM_ALLOC >= SMEM_BYTES + 1024 && SMEM_ALLOC <= 232448, "shared memory budget");
constexpr float SMAX_F16 = 3.0e4f;  // largest |state entry| for which the read-out operands are kept in fp16
constexpr float RMAX_F16 = 8.f;  // largest log2 range of E for which the score operands are kept in fp16

// tensor memory map (32-bit columns)
constexpr uint32_t COL_Y = 0;      // [128 x 128] mix output
constexpr uint32_t COL_P = 128;    // [128 x 64] scores (lanes 0-63 meaningful)
constexpr uint32_t COL_O = 192;    // [128 x 144] numerator | denominator (lanes 0-63 meaningful)
constexpr uint32_t COL_S = 336;    // [128 x 144] state S | z
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

// channels [8 jj, 8 jj + 8) of row t of the fp32 E tile (see the gate pass for its layout)
__device__ __forceinline__ void load_E8(uint32_t base, int t, int jj, float* E) {
  const uint4 lo = lds128(base + t * 512 + (((2 * jj) ^ (t & 7)) << 4));
  const uint4 hi = lds128(base + t * 512 + (((2 * jj + 1) ^ (t & 7)) << 4));
  E[0] = __uint_as_float(lo.x); E[1] = __uint_as_float(lo.y); E[2] = __uint_as_float(lo.z); E[3] = __uint_as_float(lo.w);
  E[4] = __uint_as_float(hi.x); E[5] = __uint_as_float(hi.y); E[6] = __uint_as_float(hi.z); E[7] = __uint_as_float(hi.w);
}

// log2 of the decay of one gate entry: LOGITS: log2(sigmoid(a)) / tau, LOGDECAY: a * log2(e).
__device__ __forceinline__ float log2_decay(float a, int gate_mode, float inv_tau) {
  const float L2E = 1.4426950408889634f;
  if (gate_mode == LAWCAT_GATE_LOGDECAY) return a * L2E;
  const float x = -a * L2E;  // 2^x = exp(-a)
  const float r = x > 30.f ? -x : -lg2f(1.f + ex2f(x));
  return r * inv_tau;
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
  float* const s_dm = reinterpret_cast<float*>(sg + OFF_VEC);
  float* const s_dC = s_dm + 128;
  float* const s_e63 = s_dm + 256;
  float* const s_qsum = s_dm + 384;  // per query token: sum of exp(y - max), the dropped softmax normalizer
  volatile int* const s_flags = reinterpret_cast<volatile int*>(sg + OFF_BAR + 32);  // [0] tmem base, [1] abort, [2] rmax
  int* const s_rmax = const_cast<int*>(s_flags) + 2;  // bits of the largest |log2 E| of the chunk (a non-negative float)
  // Range tracking for the fp16 read-out operand (all as bits of non-negative floats): largest |state entry| seen by the
  // last state pass, largest |v| of the chunk, and the resulting bound on the state the NEXT state pass will convert
  // (|S_new| <= |S_old| + 64 max|v| because kh <= 1).
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
    *s_smax = 0; *s_vmax = 0; *s_sbound = 0;
    tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_g);
    tma_prefetch_desc(&tm_o);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(sb + OFF_BAR + 32, TMEM_COLS);
    tmem_relinquish();
  }
  // W_h^T into its K-major slabs: row e holds W[h][c][e] over c
  {
    const bf16* Wh = a.W + (size_t)h * D * D;
    for (int idx = tid; idx < 16 * D; idx += THREADS) {
      const int e = idx & (D - 1), oc = idx >> 7;
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        w[i] = pack_f16(__bfloat162float(Wh[(size_t)(oc * 8 + 2 * i) * D + e]),
                        __bfloat162float(Wh[(size_t)(oc * 8 + 2 * i + 1) * D + e]));
      }
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
#pragma unroll
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
    tmem_st1(lane_base + COL_S + D, z0v);
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

  for (int n = 0; n < nchunks; ++n) {
    const int t0 = t_begin + n * C;
    const int nvalid = min(C, t_end - t0);

    // ---- TMA: raw q, k (with halo), gate, v -----------------------------------------------------------------------
    if (tid == 0) {
      if (store_pending) tma_store_wait_read();  // the output staging aliases the raw k tile
      mbar_arrive_expect_tx(bar_load, MODE == 0 ? LOAD_BYTES : LOAD_BYTES - 2 * RAW_ROWS * 128 - 0);
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
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        unpack8(lds128(raw + sw128(r0 + 3 + i, jc)), x0);
        float u[8];
#pragma unroll
        for (int ch = 0; ch < 8; ++ch)
          u[ch] = fmaf(cw[ch][0], x0[ch], fmaf(cw[ch][1], x1[ch], fmaf(cw[ch][2], x2[ch], cw[ch][3] * x3[ch])));
        sts128(dst + sw128(cv_stream * 64 + r0 + i, jc),
               make_uint4(pack_f16(u[0], u[1]), pack_f16(u[2], u[3]), pack_f16(u[4], u[5]), pack_f16(u[6], u[7])));
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) { x3[ch] = x2[ch]; x2[ch] = x1[ch]; x1[ch] = x0[ch]; }
      }
    }

    __syncthreads();  // the raw q, k tiles are dead from here on: E takes their place
    if (tid < D) {
      // ---- gate: thread = channel; scans outwards from the middle token ------------------------------------------------
      const int c = tid;
      const uint32_t gb = sb + OFF_G + (c >> 6) * 8192 + (c & 7) * 2;
      const int jc = (c & 63) >> 3;
      auto gaddr = [&](int t) { return gb + sw128(t, jc); };
      auto g2 = [&](int t) -> float {
        if (t >= nvalid) return 0.f;
        uint16_t raw;
        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(raw) : "r"(gaddr(t)));
        return log2_decay(__uint_as_float((uint32_t)raw << 16), a.gate_mode, a.inv_tau);
      };
      // E[t][c] fp32, 512-byte rows whose 16-byte chunks are XOR-swizzled with t & 7 (conflict-free for this
      // column-wise writer and for the row-wise readers of the phi pass)
      auto putE = [&](int t, float e) {
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(sb + OFF_E + t * 512 + (((c >> 2) ^ (t & 7)) << 4) + (c & 3) * 4), "f"(e)
                     : "memory");
      };
      bool clamped = false;
      float f = 0.f;
#pragma unroll 8
      for (int t = MID + 1; t < C; ++t) {
        f += g2(t);
        putE(t, ex2f(f));
      }
      float r = 0.f, cur = g2(MID);
#pragma unroll 8
      for (int t = MID - 1; t >= 0; --t) {
        r += cur;
        cur = g2(t);
        float ex = -r;
        if (ex > 120.f) { ex = 120.f; clamped = true; }
        putE(t, ex2f(ex));
      }
      const float g0 = cur;
      putE(MID, 1.f);
      const float bm = r + g0;
      s_dm[c] = ex2f(bm);
      s_dC[c] = ex2f(bm + f);
      dsum += bm + f;
      s_e63[c] = ex2f(f);
      atomicMax(s_rmax, __float_as_int(fmaxf(-r, -f)));  // r, f <= 0: the largest exponent magnitude of this channel
      if (clamped && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_NUMERIC);
    } else {
      // ---- v: bf16 -> fp16 in place (exact for |v| in the fp16 normal range) ------------------------------------------
      const int vt = tid - D;
      float vm = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t ad = sb + OFF_V + (uint32_t)(vt + 128 * i) * 16;
        float x[8];
        unpack8(lds128(ad), x);
#pragma unroll
        for (int e = 0; e < 8; ++e) vm = fmaxf(vm, fabsf(x[e]));
        sts128(ad, make_uint4(pack_f16(x[0], x[1]), pack_f16(x[2], x[3]), pack_f16(x[4], x[5]), pack_f16(x[6], x[7])));
      }
      vm = warp_max(vm);
      if ((tid & 31) == 0) atomicMax(s_vmax, __float_as_int(vm < 3.0e38f ? vm : 3.0e38f));
    }
    fence_proxy_async();
    __syncthreads();

    // ---- MMA 1: Y = [u_q; u_k] W_h ------------------------------------------------------------------------------------
    if (tid == 0) {
      tc_fence_after_sync();
      constexpr uint32_t ID = instr_desc(128, 128, FMT_F16, MAJOR_K, MAJOR_K);
#pragma unroll
      for (int k = 0; k < 8; ++k)
        mma_f16(tmem + COL_Y, smem_desc(sb + OFF_A + (k >> 2) * 16384 + (k & 3) * 32, 16, 1024, LAYOUT_SW128),
                smem_desc(sb + OFF_W + (k >> 2) * 16384 + (k & 3) * 32, 16, 1024, LAYOUT_SW128), ID, k > 0);
      mma_commit(bar_mma);
    }

    // ---- state pass (overlaps MMA 1): operand exp(b_mid)*[S|z] in bf16, accumulator [S|z] *= exp(b_C) --------------
    if (tid < D) {
      const int c = tid;
      const float dm = s_dm[c], dC = s_dC[c];
      const bool sf16 = __int_as_float(*s_rmax) <= RMAX_F16 && __int_as_float(*s_sbound) < SMAX_F16;
      float s[32], mx = 0.f;
#pragma unroll
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
            sts128(sb + OFF_SBF + (blk >> 1) * 16384 + sw128(c, (blk & 1) * 4 + q4),
                   sf16 ? make_uint4(pack_f16(w[0], w[1]), pack_f16(w[2], w[3]), pack_f16(w[4], w[5]), pack_f16(w[6], w[7]))
                        : make_uint4(pack_bf16(w[0], w[1]), pack_bf16(w[2], w[3]), pack_bf16(w[4], w[5]), pack_bf16(w[6], w[7])));
          }
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) s[i] *= dC;
        tmem_st32(lane_base + COL_S + blk * 32, s);
      }
      const float z = tmem_ld1(lane_base + COL_S + D);
      tmem_wait_ld();
      if (MODE == 0) {
        const uint16_t zb = sf16 ? __half_as_ushort(__float2half_rn(dm * z)) : __bfloat16_as_ushort(__float2bfloat16_rn(dm * z));
        *reinterpret_cast<uint16_t*>(sg + OFF_SZ + (c >> 3) * 128 + (c & 7) * 16) = zb;
        mx = warp_max(fmaxf(mx, fabsf(z)));
        if ((tid & 31) == 0) atomicMax(s_smax, __float_as_int(mx < 3.0e38f ? mx : 3.0e38f));
      }
      tmem_st1(lane_base + COL_S + D, dC * z);
      tmem_wait_st();
    }
    LAWCAT_WAIT_ALL(bar_mma, ph_mma);
    tc_fence_after_sync();

    // ---- phi: one thread per row of Y -----------------------------------------------------------------------------
    if (tid < D && (MODE == 0 || tid >= C)) {
      const float L2E = 1.4426950408889634f;
      float y[D];
#pragma unroll
      for (int blk = 0; blk < 4; ++blk) tmem_ld32(lane_base + COL_Y + blk * 32, y + blk * 32);
      tmem_wait_ld();
      float m = y[0];
#pragma unroll
      for (int i = 1; i < D; ++i) m = fmaxf(m, y[i]);
      const float mb = m * L2E;
      const bool f16 = __int_as_float(*s_rmax) <= RMAX_F16;
      const bool sf16 = f16 && __int_as_float(*s_sbound) < SMAX_F16;
      if (tid < C) {
        const int t = tid;
        float qsum = 0.f;
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) {
          float E[8];
          load_E8(sb + OFF_E, t, jj, E);
          float v[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float ex = ex2f(fmaf(y[jj * 8 + i], L2E, -mb));
            qsum += ex;
            v[i] = ex * E[i];
          }
          const uint4 vb = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
          const uint4 vh = make_uint4(pack_f16(v[0], v[1]), pack_f16(v[2], v[3]), pack_f16(v[4], v[5]), pack_f16(v[6], v[7]));
          sts128(sb + OFF_QB + (jj >> 3) * 8192 + sw128(t, jj & 7), sf16 ? vh : vb);
          sts128(sb + OFF_A + (jj >> 3) * 16384 + sw128(t, jj & 7), f16 ? vh : vb);
        }
        s_qsum[t] = qsum;
      } else {
        const int i_tok = tid - C;
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < D; ++i) {
          y[i] = ex2f(fmaf(y[i], L2E, -mb));
          sum += y[i];
        }
        const float inv = i_tok < nvalid ? 1.f / sum : 0.f;
#pragma unroll
        for (int jj = 0; jj < 16; ++jj) {
          float E[8];
          load_E8(sb + OFF_E, i_tok, jj, E);
          const float4 ea = *reinterpret_cast<const float4*>(s_e63 + jj * 8);
          const float4 eb = *reinterpret_cast<const float4*>(s_e63 + jj * 8 + 4);
          const float e63[8] = {ea.x, ea.y, ea.z, ea.w, eb.x, eb.y, eb.z, eb.w};
          float ks[8], kh[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            ks[i] = y[jj * 8 + i] * inv * rcpf(E[i]);
            kh[i] = ks[i] * e63[i];
          }
          if (MODE == 0)
            sts128(sb + OFF_A + (jj >> 3) * 16384 + sw128(C + i_tok, jj & 7),
                   f16 ? make_uint4(pack_f16(ks[0], ks[1]), pack_f16(ks[2], ks[3]), pack_f16(ks[4], ks[5]), pack_f16(ks[6], ks[7]))
                       : make_uint4(pack_bf16(ks[0], ks[1]), pack_bf16(ks[2], ks[3]), pack_bf16(ks[4], ks[5]), pack_bf16(ks[6], ks[7])));
          sts128(sb + OFF_KH + (jj >> 3) * 8192 + sw128(i_tok, jj & 7),
                 make_uint4(pack_f16(kh[0], kh[1]), pack_f16(kh[2], kh[3]), pack_f16(kh[4], kh[5]), pack_f16(kh[6], kh[7])));
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
        const uint32_t ID_P = __int_as_float(*s_rmax) <= RMAX_F16 ? instr_desc(128, 64, FMT_F16, MAJOR_K, MAJOR_K)
                                                                  : instr_desc(128, 64, FMT_BF16, MAJOR_K, MAJOR_K);
        const bool sf16 = __int_as_float(*s_rmax) <= RMAX_F16 && __int_as_float(*s_sbound) < SMAX_F16;
        const uint32_t ID_O = instr_desc(128, 128, sf16 ? FMT_F16 : FMT_BF16, MAJOR_K, MAJOR_MN);
        const uint32_t ID_OZ = instr_desc(128, 16, sf16 ? FMT_F16 : FMT_BF16, MAJOR_K, MAJOR_MN);
        // bound on the state after this chunk's update, for the next chunk's choice of operand type
        *s_sbound = __float_as_int(__int_as_float(*s_smax) + 64.f * fmaxf(__int_as_float(*s_vmax), 1.f));
        *s_smax = 0;
        *s_vmax = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint64_t ad = smem_desc(sb + OFF_A + (k >> 2) * 16384 + (k & 3) * 32, 16, 1024, LAYOUT_SW128);
          mma_f16(tmem + COL_P, ad, smem_desc(sb + OFF_A + (k >> 2) * 16384 + 8192 + (k & 3) * 32, 16, 1024, LAYOUT_SW128),
                  ID_P, k > 0);
          const uint64_t qb = smem_desc(sb + OFF_QB + (k >> 2) * 8192 + (k & 3) * 32, 16, 1024, LAYOUT_SW128);
          mma_f16(tmem + COL_O, qb, smem_desc(sb + OFF_SBF + k * 2048, 16384, 1024, LAYOUT_SW128), ID_O, k > 0);
          mma_f16(tmem + COL_O + D, qb, smem_desc(sb + OFF_SZ + k * 256, 128, 2048, LAYOUT_NONE), ID_OZ, k > 0);
        }
      }
      constexpr uint32_t ID_S = instr_desc(128, 128, FMT_F16, MAJOR_MN, MAJOR_MN);
      constexpr uint32_t ID_SZ = instr_desc(128, 16, FMT_F16, MAJOR_MN, MAJOR_MN);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint64_t ad = smem_desc(sb + OFF_KH + k * 2048, 8192, 1024, LAYOUT_SW128);
        mma_f16(tmem + COL_S, ad, smem_desc(sb + OFF_V + k * 2048, 8192, 1024, LAYOUT_SW128), ID_S, 1);
        mma_f16(tmem + COL_S + D, ad, smem_desc(sb + OFF_ONES + k * 256, 128, 1024, LAYOUT_NONE), ID_SZ, 1);
      }
      mma_commit(bar_mma);
    }
    LAWCAT_WAIT_ALL(bar_mma, ph_mma);
    tc_fence_after_sync();

    if (MODE == 0) {
      // ---- causal mask, fp16 scores ---------------------------------------------------------------------------------
      if (tid < C) {
        const int t = tid;
        float p[C];
        tmem_ld32(lane_base + COL_P, p);
        tmem_ld32(lane_base + COL_P + 32, p + 32);
        tmem_wait_ld();
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          float v[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) v[i] = (jj * 8 + i <= t) ? p[jj * 8 + i] : 0.f;
          sts128(sb + OFF_QRAW + sw128(t, jj),
                 make_uint4(pack_f16(v[0], v[1]), pack_f16(v[2], v[3]), pack_f16(v[4], v[5]), pack_f16(v[6], v[7])));
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
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint64_t ad = smem_desc(sb + OFF_QRAW + k * 32, 16, 1024, LAYOUT_SW128);
          mma_f16(tmem + COL_O, ad, smem_desc(sb + OFF_V + k * 2048, 8192, 1024, LAYOUT_SW128), ID_O, 1);
          mma_f16(tmem + COL_O + D, ad, smem_desc(sb + OFF_ONES + k * 256, 128, 1024, LAYOUT_NONE), ID_OZ, 1);
        }
        mma_commit(bar_mma);
      }
      LAWCAT_WAIT_ALL(bar_mma, ph_mma);
      tc_fence_after_sync();

      // ---- normalize (Eq. 8), stage, store ----------------------------------------------------------------------------
      if (tid < C) {
        const int t = tid;
        const float den = tmem_ld1(lane_base + COL_O + D);
        float o[32];
#pragma unroll
        for (int blk = 0; blk < 4; ++blk) {
          tmem_ld32(lane_base + COL_O + blk * 32, o);
          tmem_wait_ld();
          // the query features went in scaled by qsum (unnormalized softmax), so eps scales the same way
          const float inv = 1.f / (den + a.eps * s_qsum[t]);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)
            sts128(sb + OFF_KRAW + (blk >> 1) * 8192 + sw128(t, (blk & 1) * 4 + q4),
                   make_uint4(pack_bf16(o[8 * q4 + 0] * inv, o[8 * q4 + 1] * inv), pack_bf16(o[8 * q4 + 2] * inv, o[8 * q4 + 3] * inv),
                              pack_bf16(o[8 * q4 + 4] * inv, o[8 * q4 + 5] * inv), pack_bf16(o[8 * q4 + 6] * inv, o[8 * q4 + 7] * inv)));
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
#pragma unroll
    for (int blk = 0; blk < 4; ++blk) {
      tmem_ld32(lane_base + COL_S + blk * 32, s);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; i += 4)
        *reinterpret_cast<float4*>(a.S_T + (out_idx * D + tid) * D + blk * 32 + i) = make_float4(s[i], s[i + 1], s[i + 2], s[i + 3]);
    }
    const float z = tmem_ld1(lane_base + COL_S + D);
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

// ---------------------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

// [B, T, heads, 128] bf16 tensor as a 4-D map (channel, head, token, batch) with boxes of 64 channels x rows tokens
static bool make_map(CUtensorMap* m, const void* ptr, int heads, int T, int B, int rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)T, (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)heads * D * 2, (cuuint64_t)T * heads * D * 2};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)rows, 1};
  const cuuint32_t es[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// State at the start of every segment from the per-segment end states (computed from zero) and total decays:
// start[0] = given state; start[s] = decay[s-1] * start[s-1] + local[s-1]  (Eq. 4 unrolled over whole segments).
// One thread per state entry (the d_k x d_v entries of S, then the d_k entries of z) of one (batch, head).
__global__ void segment_scan_kernel(const float* __restrict__ S0, const float* __restrict__ z0,
                                    const float* __restrict__ loc_S, const float* __restrict__ loc_z,
                                    const float* __restrict__ dtot, float* __restrict__ start_S,
                                    float* __restrict__ start_z, int BH, int nseg) {
  const int per = D * D + D;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= BH * per) return;
  const int bh = idx / per, r = idx % per;
  const bool isz = r >= D * D;
  const int c = isz ? r - D * D : r / D;  // key channel: the decay is per row of the state
  const int e = isz ? 0 : r % D;
  float cur = isz ? (z0 ? z0[(size_t)bh * D + c] : 0.f) : (S0 ? S0[((size_t)bh * D + c) * D + e] : 0.f);
  for (int sgm = 0; sgm < nseg; ++sgm) {
    const size_t si = (size_t)bh * nseg + sgm;
    if (isz) start_z[si * D + c] = cur; else start_S[(si * D + c) * D + e] = cur;
    if (sgm + 1 < nseg) {
      const float loc = isz ? loc_z[si * D + c] : loc_S[(si * D + c) * D + e];
      cur = fmaf(exp2f(dtot[si * D + c]), cur, loc);
    }
  }
}

}  // namespace tc

// Segments per sequence: enough thread blocks to fill the SMs (one block per SM), but at least 16 chunks per segment.
int layer_tc_segments(const lawcat_params& p) {
  const int chunks = (p.T + tc::C - 1) / tc::C;
  int n = 148 / (p.B * p.H);
  if (n > chunks / 16) n = chunks / 16;
  return n < 1 ? 1 : n;
}

size_t layer_tc_workspace_bytes(const lawcat_params& p) {
  const int nseg = layer_tc_segments(p);
  if (nseg == 1) return 0;
  return sizeof(float) * (size_t)p.B * p.H * nseg * (2 * (tc::D * tc::D + tc::D) + tc::D);
}

bool layer_tc_supported(const lawcat_params& p) {
  return p.dtype == LAWCAT_BF16 && p.d_k == tc::D && p.d_v == tc::D && p.gate_dim == p.d_k &&
         p.phi == LAWCAT_PHI_SOFTMAX && p.normalize == 1 && p.conv_k <= tc::HALO + 1 && p.B > 0 && p.T > 0 &&
         (p.chunk == 0 || p.chunk == tc::C);
}

int launch_layer_tc(const Ctx& c, const void* q, const void* k, const void* v, const void* gate, const void* w_q,
                    const void* w_k, const void* W, const void* cache_q_in, const void* cache_k_in, const float* S0,
                    const float* z0, void* o, float* S_T, float* z_T, void* ws) {
  using namespace tc;
  const lawcat_params& p = *c.p;
  CUtensorMap tq, tk, tv, tg, to;
  if (!make_map(&tq, q, p.H, p.T, p.B, RAW_ROWS) || !make_map(&tk, k, p.H_kv, p.T, p.B, RAW_ROWS) ||
      !make_map(&tv, v, p.H_kv, p.T, p.B, C) || !make_map(&tg, gate, p.H, p.T, p.B, C) ||
      !make_map(&to, o, p.H, p.T, p.B, C))
    return LAWCAT_ERR_CUDA;
  TcArgs a{};
  a.w_q = (const bf16*)w_q; a.w_k = (const bf16*)w_k; a.W = (const bf16*)W;
  a.cache_q = (const bf16*)cache_q_in; a.cache_k = (const bf16*)cache_k_in;
  a.dev_status = c.dev_status;
  a.T = p.T; a.H = p.H; a.Hkv = p.H_kv; a.K = p.conv_k;
  a.gate_mode = p.gate_mode; a.inv_tau = 1.f / p.gate_tau; a.eps = p.eps;
  const int nseg = layer_tc_segments(p);
  a.nseg = nseg;
  a.seg_len = ((p.T + nseg - 1) / nseg + C - 1) / C * C;
  if (cudaFuncSetAttribute(layer_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess ||
      cudaFuncSetAttribute(layer_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess)
    return LAWCAT_ERR_CUDA;
  const int BH = p.B * p.H;
  if (nseg == 1) {
    a.S0 = S0; a.z0 = z0; a.S_T = S_T; a.z_T = z_T; a.dtot = nullptr;
    a.grid_nseg = 1; a.seg_in = 0; a.seg_out = 0;
    LaunchScope _ls("layer_tc", c.stream);
    layer_tc_kernel<0><<<BH, THREADS, SMEM_ALLOC, c.stream>>>(tq, tk, tv, tg, to, a);
    LAWCAT_CHECK_LAUNCH();
    return LAWCAT_OK;
  }
  // Several segments per sequence: (1) every segment but the last computes its end state from a zero state, and the
  // total decay of the segment; (2) a scan over the segments turns these into the state at each segment's start;
  // (3) the layer runs on all segments at once, each from its start state.
  const size_t nS = (size_t)BH * nseg * D * D, nz = (size_t)BH * nseg * D;
  float* loc_S = (float*)ws;
  float* loc_z = loc_S + nS;
  float* dtot = loc_z + nz;
  float* start_S = dtot + nz;
  float* start_z = start_S + nS;
  {
    TcArgs b1 = a;
    b1.S0 = nullptr; b1.z0 = nullptr; b1.S_T = loc_S; b1.z_T = loc_z; b1.dtot = dtot;
    b1.grid_nseg = nseg - 1; b1.seg_in = 1; b1.seg_out = 1;
    LaunchScope _ls("layer_tc_state", c.stream);
    layer_tc_kernel<1><<<BH * (nseg - 1), THREADS, SMEM_ALLOC, c.stream>>>(tq, tk, tv, tg, to, b1);
    LAWCAT_CHECK_LAUNCH();
  }
  {
    const int total = BH * (D * D + D);
    LaunchScope _ls("segment_scan", c.stream);
    segment_scan_kernel<<<(total + 255) / 256, 256, 0, c.stream>>>(S0, z0, loc_S, loc_z, dtot, start_S, start_z, BH, nseg);
    LAWCAT_CHECK_LAUNCH();
  }
  a.S0 = start_S; a.z0 = start_z; a.S_T = S_T; a.z_T = z_T; a.dtot = nullptr;
  a.grid_nseg = nseg; a.seg_in = 1; a.seg_out = 0;
  LaunchScope _ls("layer_tc", c.stream);
  layer_tc_kernel<0><<<BH * nseg, THREADS, SMEM_ALLOC, c.stream>>>(tq, tk, tv, tg, to, a);
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

}  // namespace lawcat
