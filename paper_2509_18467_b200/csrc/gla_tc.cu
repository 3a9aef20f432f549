// Chunkwise tensor-core kernels for the normalized gated linear attention on GIVEN feature-mapped streams (Eq. 4 - Eq. 8)
// and for its backward (the distillation step of Section 5.1), bf16 storage, d_k = d_v = 64.
//
// One thread block walks one (batch, query head) in chunks of C = 64 tokens, lock-step: every phase of a chunk is done by
// all threads together, the products are issued by one thread (tcgen05.mma, fp32 accumulators in tensor memory) and the
// block waits for them on an mbarrier. With b_t the running sum of the log-decays inside a chunk (log2 units) and the
// reference token m = 31,  x_t = b_t - b_m,  qs_t = qdot_t 2^{x_t},  ks_i = kdot_i 2^{-x_i},  v' = [v | 1]:
//
//   forward    P = mask_{i<=t}(qs ks^T)        O' = P v' + qs (2^{b_m} S')        S' <- 2^{b_C} S' + (ks 2^{b_C - b_m})^T v'
//              o_t = O'_t[:d_v] / (O'_t[d_v] + eps)                                (S' = [S | z], Eq. 4 and Eq. 8)
//   backward   (chain rule on the above; do'_t = [dO_t / den_t | -(dO_t . o_t) / den_t], R = adjoint of S' from later chunks)
//              dP = mask(do' v'^T) = mask((dO v^T - dO_t . o_t) / den_t): the product dO v^T takes dO and v unrounded (both
//                   are exact in 16 bits) and the row terms are applied in fp32, because for the first tokens of a
//                   sequence the two terms cancel (o_1 = v_1) and rounded operands would leave only their rounding
//              dqdot = 2^{x_t}  (dP ks + do' (2^{b_m} S'_prev)^T)
//              dkdot = 2^{-x_i} (dP^T qs + v' (2^{b_C - b_m} R)^T)
//              dv'   = P^T do' + ks (2^{b_C - b_m} R)
//              R <- 2^{b_C} R + (qs 2^{b_m})^T do'
//              dg_s  = sum_{t >= s} (qdot_t dqdot_t - kdot_t dkdot_t)   (the decays enter only through their running sum);
//                      the part of that sum behind the chunk equals sum_e S'[c,e] R[c,e] at the chunk's end
// The backward kernel first runs the forward sweep (it needs the state in front of every chunk, the denominators and
// dO . o in fp32), keeping the 16-bit state operand of every chunk in scratch memory, then the reverse sweep.
//
// Operand tiles live in shared memory as unswizzled 8x8 core matrices, every 8-column slab of a tile contiguous:
// element (r, c) of a tile with R rows sits at (c / 8) * (16 R + 16) + 16 r + 2 (c % 8). The same bytes serve as a
// K-major operand (rows = M or N, columns = K: LBO = slab stride, SBO = 128) and as an MN-major one (rows = K, columns =
// M or N: LBO = 128, SBO = slab stride), so a tile and its transpose need no second copy. The 16 spare bytes per slab keep
// the row-wise writers (8 lanes on one row, one per slab) off each other's banks.
// Every product uses M = 128; where 64 rows are meaningful the upper 64 TMEM lanes hold unused results computed from
// whatever follows the tile in shared memory. Operands are fp16 while the chunk's exponents stay within +-8 and the state
// below 3e4, bf16 otherwise. Every wait is bounded; a wait that runs out reports LAWCAT_ERR_TIMEOUT and the block finishes
// without waiting again.
#include <cuda.h>
#include <cuda_fp16.h>

#include <mutex>

#include "common.cuh"
#include "tc_common.cuh"

namespace lawcat {
namespace gtc {

using namespace tc;

#ifdef LAWCAT_TIMELINE
__device__ long long g_gla_timeline[32];
#define GTL(i) do { if (blockIdx.x == 0 && tid == 0 && n == 8) g_gla_timeline[i] = clock64(); } while (0)
#else
#define GTL(i) do { } while (0)
#endif

constexpr int C = 64, MID = 31, THREADS = 256;
constexpr int D = 64;           // d_k = d_v
constexpr int NV = D + 16;      // columns of v' and do': the value channels, the "1" / denominator column, zero padding
constexpr uint32_t SLAB_T = C * 16 + 16;  // slab stride of tiles with 64 (token) rows
constexpr uint32_t SLAB_C = D * 16 + 16;  // slab stride of tiles with D (key channel) rows
constexpr uint32_t TILE_TD = (D / 8) * SLAB_T, TILE_TV = (NV / 8) * SLAB_T, TILE_TT = (C / 8) * SLAB_T;
constexpr uint32_t TILE_CV = (NV / 8) * SLAB_C;
constexpr float RMAX_F16 = 8.f, SMAX_F16 = 3.0e4f;

// shared memory map (bytes). The forward kernel uses the first part only (two thread blocks per SM).
constexpr uint32_t OFF_X = 0;                        // fp32 [64][D] log-decays, then exponents x
constexpr uint32_t OFF_VEC = OFF_X + C * D * 4;      // fp32 bm[D], ft[D], dm[D] = 2^bm, e63[D] = 2^ft, dC[D] = 2^(bm+ft)
constexpr uint32_t OFF_ROW = OFF_VEC + 5 * D * 4;    // fp32 [2][64] per-row scalars
constexpr uint32_t OFF_BAR = OFF_ROW + 2 * C * 4;    // mbarrier and flags
constexpr uint32_t OFF_QS = (OFF_BAR + 64 + 127) / 128 * 128;  // operand tiles from here on
constexpr uint32_t OFF_KS = OFF_QS + TILE_TD;
constexpr uint32_t OFF_KQ = OFF_KS + TILE_TD;        // forward sweep: kh = ks 2^ft ; reverse sweep: qh = qs 2^bm
constexpr uint32_t OFF_VP = OFF_KQ + TILE_TD;        // v' [64 x NV]
constexpr uint32_t OFF_PM = OFF_VP + TILE_TV;        // masked scores [64 x 64]
constexpr uint32_t OFF_S16 = OFF_PM + TILE_TT;       // 2^bm S' [D x NV]
constexpr uint32_t SMEM_FWD = OFF_S16 + TILE_CV + 2048;  // (M = 128 operands read rows / slabs past a 64-row tile)
// backward only: low parts of the two-term operands (value minus its 16-bit rounding, again in 16 bits), do', adjoint
constexpr uint32_t OFF_S16L = OFF_S16 + TILE_CV;
constexpr uint32_t OFF_QSL = OFF_S16L + TILE_CV;
constexpr uint32_t OFF_KSL = OFF_QSL + TILE_TD;
constexpr uint32_t OFF_PML = OFF_KSL + TILE_TD;
constexpr uint32_t OFF_DPM = OFF_PML + TILE_TT;      // masked score gradients [64 x 64]
constexpr uint32_t OFF_DPL = OFF_DPM + TILE_TT;
constexpr uint32_t OFF_DO = OFF_DPL + TILE_TT;       // do' [64 x NV] (scaled)
constexpr uint32_t OFF_DOL = OFF_DO + TILE_TV;
constexpr uint32_t OFF_DOX = OFF_DOL + TILE_TV;      // dO itself [64 x D] (exact in 16 bits): A of the score gradients
constexpr uint32_t OFF_R16 = OFF_DOX + TILE_TD;      // 2^ft R [D x NV]
constexpr uint32_t OFF_R16L = OFF_R16 + TILE_CV;
constexpr uint32_t OFF_KQL = OFF_R16L + TILE_CV;     // low part of kh / qh
constexpr uint32_t OFF_DT = (OFF_KQL + TILE_TD + 127) / 128 * 128;   // fp32 [64][D]: qdot dqdot - kdot dkdot and its running sum
constexpr uint32_t SMEM_BWD = OFF_DT + C * D * 4;    // (the fp32 tile doubles as the pad behind the last operand)
// The forward sweep of the backward (its own launch, two thread blocks per SM) keeps the low parts of its two-term operands
// right behind the state operand, in an order of its own (see the kernel): the tile that is read as an MN-major M = 128
// operand -- sixteen slabs from its start -- must not be the last one.
constexpr uint32_t SMEM_SWEEP = OFF_PML + TILE_TD + 2048;
static_assert(SMEM_BWD <= 232448 && 2 * SMEM_SWEEP + 2048 <= 232448, "shared memory budget");
static_assert(OFF_R16L + 16 * SLAB_C <= SMEM_BWD + 16 * SLAB_C, "");

// tensor memory map (32-bit columns): the forward kernel allocates 256 columns, the backward 512
constexpr uint32_t COL_P = 0, COL_A = 64 /* O' | dQ */, COL_ST = 144 /* S' or R */, COL_DP = 256, COL_B = 320 /* dK */,
                   COL_V = 384 /* dV */;

struct GArgs {
  const void *qdot, *kdot;   // features: bf16, or fp32 when feat_f32 (scratch of the fused layer backward)
  const bf16 *v, *gate, *dO;
  const float *S0, *z0;
  bf16* o;
  float *den, *S_T, *z_T;
  void *d_qdot, *d_kdot;     // bf16, or fp32 when feat_f32
  bf16* dgate;
  int feat_f32;
  float* dvh;         // [B,T,H,D] per-head dv (fp32), reduced over the heads of a group afterwards
  uint8_t* ws_s16;    // [B*H][chunks][2 TILE_CV + 16] the (two-term) state operand of every chunk and its format
  float *ws_den, *ws_delta;  // [B,T,H]: 1 / den_t and dO_t . o_t
  float* ws_scale;           // [B*H]: largest |do'| of the head
  int* dev_status;
  int B, T, H, Hkv, gate_dim, gate_mode, normalize;
  float inv_tau, eps;
};

__device__ __forceinline__ uint32_t toff(uint32_t slab, int r, int c) { return (uint32_t)(c >> 3) * slab + (uint32_t)r * 16u + (uint32_t)(c & 7) * 2u; }
// K-major view (rows = M or N, columns = K) and MN-major view (rows = K, columns = M or N) of a tile
__device__ __forceinline__ uint64_t kview(uint32_t addr, uint32_t slab) { return smem_desc(addr, slab, 128, LAYOUT_NONE); }
__device__ __forceinline__ uint64_t mview(uint32_t addr, uint32_t slab) { return smem_desc(addr, 128, slab, LAYOUT_NONE); }
__device__ __forceinline__ uint64_t dadv(uint64_t d, uint32_t bytes) {
  return (d & 0xFFFFFFFF00000000ull) | (uint64_t)((uint32_t)d + (bytes >> 4));
}
__device__ __forceinline__ float log2_sigmoid(float a) {
  const float x = -a * 1.4426950408889634f;
  return -fmaxf(x, lg2f(1.f + ex2f(fminf(x, 126.f))));
}
__device__ __forceinline__ uint4 pack8h(const float* v, bool f16) {
  return f16 ? make_uint4(pack_f16(v[0], v[1]), pack_f16(v[2], v[3]), pack_f16(v[4], v[5]), pack_f16(v[6], v[7]))
             : make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
// 16-bit values back to fp32
__device__ __forceinline__ void unpack8h(const uint4& v, bool f16, float* f) {
  if (f16) {
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 x = __half22float2(h[i]);
      f[2 * i] = x.x; f[2 * i + 1] = x.y;
    }
  } else {
    f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
    f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
  }
}
// v = hi + lo with hi the 16-bit rounding of v and lo the 16-bit rounding of the rest
__device__ __forceinline__ void split8h(const float* v, bool f16, uint4& hi, uint4& lo) {
  hi = pack8h(v, f16);
  float h[8], r[8];
  unpack8h(hi, f16, h);
#pragma unroll
  for (int i = 0; i < 8; ++i) r[i] = v[i] - h[i];
  lo = pack8h(r, f16);
}
__device__ __forceinline__ void unpack8b(const uint4& v, float* f) {
  f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
  f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const float* v) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
                 "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
                 "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7]))
               : "memory");
}

// MODE 0: the forward (o, den, S_T, z_T). The backward is two launches: MODE 1, the forward sweep for the scratch quantities
// (state operand of every chunk, 1 / den, dO . o, the scale of do'), two thread blocks per SM; MODE 2, the reverse sweep. In
// the backward every product whose few, large terms decide the first tokens of a sequence (small denominators, gradients a
// hundred times the typical size) runs on two-term operands x = hi + lo (hi hi + lo hi + hi lo, about 21 significant bits).
template <int MODE>
__global__ void __launch_bounds__(THREADS, MODE == 2 ? 1 : 2) gla_tc_kernel(const GArgs a) {
  extern __shared__ __align__(128) uint8_t sg[];
  constexpr bool BWD = MODE != 0, SPLIT = BWD;
  constexpr uint32_t TMEM_COLS = MODE == 2 ? 512 : 256;
  // Low-part tiles. The sweep kernel (MODE 1) packs them into the three tile slots behind the state operand: low part of
  // kh first (it is read as an MN-major M = 128 operand, sixteen slabs from its start, so two tile slots must follow its
  // start), then that of qs -- whose slot the low part of the masked scores takes over once the first batch of products
  // has consumed it -- then that of ks (a B operand of 64 rows: nothing is read behind it).
  constexpr uint32_t oKQL = MODE == 1 ? OFF_QSL : OFF_KQL, oQSL = MODE == 1 ? OFF_KSL : OFF_QSL;
  constexpr uint32_t oKSL = MODE == 1 ? OFF_PML : OFF_KSL, oPML = MODE == 1 ? OFF_KSL : OFF_PML;
  const uint32_t sb = smem_u32(sg);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float* const s_x = reinterpret_cast<float*>(sg + OFF_X);
  float* const s_dt = reinterpret_cast<float*>(sg + OFF_DT);
  float* const s_bm = reinterpret_cast<float*>(sg + OFF_VEC);
  float* const s_ft = s_bm + D;
  float* const s_dm = s_bm + 2 * D;
  float* const s_e63 = s_bm + 3 * D;
  float* const s_dC = s_bm + 4 * D;
  float* const s_row = reinterpret_cast<float*>(sg + OFF_ROW);
  volatile int* const s_flags = reinterpret_cast<volatile int*>(sg + OFF_BAR + 16);  // [0] tmem base, [1] abort, [2] rmax, [3] smax, [4] vmax / domax
  const uint32_t bar = sb + OFF_BAR;
  const int bh = blockIdx.x, h = bh % a.H, b = bh / a.H;
  const int G = a.H / a.Hkv, j = h / G;
  const int nchunks = (a.T + C - 1) / C;

  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_fence_init();
    s_flags[1] = 0; s_flags[2] = 0; s_flags[3] = 0; s_flags[4] = 0;
  }
  if (warp == 0) {
    tmem_alloc(sb + OFF_BAR + 16, TMEM_COLS);
    tmem_relinquish();
  }
  // the two extra slabs of v' and do' (column D: the "1" of [v | 1] / the denominator's gradient; the rest zero)
  for (int i = tid; i < 2 * C; i += THREADS) {
    const int r = i & (C - 1), sl = i >> 6;
    const uint4 w = make_uint4(0u, 0u, 0u, 0u);
    *reinterpret_cast<uint4*>(sg + OFF_VP + toff(SLAB_T, r, D + 8 * sl)) = w;
    if (MODE == 2) {
      *reinterpret_cast<uint4*>(sg + OFF_DO + toff(SLAB_T, r, D + 8 * sl)) = w;
      *reinterpret_cast<uint4*>(sg + OFF_DOL + toff(SLAB_T, r, D + 8 * sl)) = w;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = (uint32_t)s_flags[0];
  // threads that own a row of the 64-row accumulators (token rows; for D = 64 also the state's key-channel rows)
  const bool row_thr = (warp & 3) < 2;
  const int row = (warp & 3) * 32 + lane, half = warp >> 2;
  const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
  uint32_t phase = 0;  // parity of the next completion of the one mbarrier
  // (a batch of products completes within microseconds; the limit is 2e8 cycles, about a tenth of a second)
  auto bounded_wait = [&](uint32_t parity) -> bool {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
      for (int i = 0; i < 16; ++i)
        if (mbar_try_wait(bar, parity)) return true;
      if (s_flags[1] || clock64() - t0 > 200000000LL) return false;
    }
  };
  auto wait_mma = [&]() {
    if (!s_flags[1] && !bounded_wait(phase)) {
      s_flags[1] = 1;
      if (a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_TIMEOUT);
    }
    phase ^= 1u;
    tc_fence_after_sync();
  };
  // before the issuing thread may read what the others wrote to shared memory / tensor memory
  auto publish = [&]() {
    fence_proxy_async();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
  };
  // 8 values of row r, columns [c, c + 8) of a tile (and of its low-part tile)
  auto put8 = [&](uint32_t off_hi, uint32_t off_lo, uint32_t slab, int r, int c, const float* v, bool f16, bool split) {
    if (split) {
      uint4 hi, lo;
      split8h(v, f16, hi, lo);
      *reinterpret_cast<uint4*>(sg + off_hi + toff(slab, r, c)) = hi;
      *reinterpret_cast<uint4*>(sg + off_lo + toff(slab, r, c)) = lo;
    } else {
      *reinterpret_cast<uint4*>(sg + off_hi + toff(slab, r, c)) = pack8h(v, f16);
    }
  };

  // ---- state [S | z] into tensor memory (zeros without a given state) ---------------------------------------------------
  auto load_state = [&](bool given) {
    if (row_thr) {
      float s[8];
#pragma unroll 1
      for (int c0 = half * 48; c0 < (half ? NV : 48); c0 += 8) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int e = c0 + i;
          float v = 0.f;
          if (given && e < D && a.S0) v = a.S0[((size_t)bh * D + row) * D + e];
          if (given && e == D && a.z0) v = a.z0[(size_t)bh * D + row];
          s[i] = v;
        }
        tmem_st8(lane_base + COL_ST + c0, s);
      }
      tmem_wait_st();
    }
  };
  load_state(MODE != 2);  // (the reverse sweep starts from a zero adjoint state)
  if (MODE != 2 && row_thr && (a.S0 || a.z0)) {  // bound on the given state: decides the operand format of the first chunks
    float mx = 0.f;
    for (int e = 0; e < D; ++e)
      if (a.S0) mx = fmaxf(mx, fabsf(a.S0[((size_t)bh * D + row) * D + e]));
    if (a.z0) mx = fmaxf(mx, fabsf(a.z0[(size_t)bh * D + row]));
    if (!(mx < 3.0e38f)) mx = 3.0e38f;
    atomicMax(const_cast<int*>(&s_flags[3]), __float_as_int(mx));
  }
  float sbound = 0.f;  // bound on the state entries (every thread keeps the same copy)
  __syncthreads();
  sbound = __int_as_float(s_flags[3]);

  // rows of the next chunk towards L2 (one 128-byte line per row and tensor)
  auto prefetch_chunk = [&](int m) {
    if (m < 0 || m >= nchunks) return;
    const int r = tid >> 2, which = tid & 3, t = m * C + r;
    if (t >= a.T) return;
    const size_t tq = ((size_t)b * a.T + t) * a.H + h, tv = ((size_t)b * a.T + t) * a.Hkv + j;
    const size_t fb = a.feat_f32 ? 4 : 2;
    const void* ptr = which == 0 ? (const void*)((const char*)a.qdot + tq * D * fb) : which == 1 ? (const void*)((const char*)a.kdot + tq * D * fb)
                    : which == 2 ? (const void*)(a.v + tv * D)
                    : (a.gate_dim == 1 ? (const void*)(a.gate + tq) : (const void*)(a.gate + tq * D));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
    if (BWD && which == 3) asm volatile("prefetch.global.L2 [%0];" ::"l"(a.dO + tq * D));
  };

  // ---- gate pass of a chunk: exponents x, per-channel sums, largest exponent ----------------------------------------------
  auto gate_pass = [&](int t0, int nvalid) {
    const float L2E = 1.4426950408889634f;
    if (tid == 0) s_flags[2] = 0;
    // log-decays (log2 units) of the chunk, all threads, 16-byte loads
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
      const int o8 = tid & 7, r = (tid >> 3) + 32 * pass;
      float g[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (r < nvalid) {
        const size_t gi = ((size_t)b * a.T + t0 + r) * a.H + h;
        if (a.gate_dim == 1) {
          const float av = __bfloat162float(a.gate[gi]);
          const float gv = a.gate_mode == LAWCAT_GATE_LOGDECAY ? av * L2E : log2_sigmoid(av) * a.inv_tau;
#pragma unroll
          for (int i = 0; i < 8; ++i) g[i] = gv;
        } else {
          unpack8b(*reinterpret_cast<const uint4*>(a.gate + gi * D + o8 * 8), g);
#pragma unroll
          for (int i = 0; i < 8; ++i) g[i] = a.gate_mode == LAWCAT_GATE_LOGDECAY ? g[i] * L2E : log2_sigmoid(g[i]) * a.inv_tau;
        }
      }
      *reinterpret_cast<float4*>(s_x + r * D + o8 * 8) = make_float4(g[0], g[1], g[2], g[3]);
      *reinterpret_cast<float4*>(s_x + r * D + o8 * 8 + 4) = make_float4(g[4], g[5], g[6], g[7]);
    }
    __syncthreads();
    // scan outwards from the middle token, in place: thread = (channel, half of the chunk)
    if (tid < 2 * D) {
      const int c = tid & (D - 1), gh = tid >> 6;
      float g[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) g[i] = s_x[(gh * 32 + i) * D + c];
      float acc = 0.f;
      if (gh) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          acc += g[i];
          s_x[(32 + i) * D + c] = fmaxf(acc, -120.f);
        }
        s_ft[c] = acc;
        s_e63[c] = ex2f(fmaxf(acc, -120.f));
      } else {
        s_x[MID * D + c] = 0.f;
#pragma unroll
        for (int i = MID - 1; i >= 0; --i) {
          acc += g[i + 1];
          s_x[i * D + c] = fminf(-acc, 120.f);
        }
        s_bm[c] = acc + g[0];
        s_dm[c] = ex2f(fmaxf(acc + g[0], -126.f));
      }
      if (-acc > 120.f && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_NUMERIC);
      const float am = warp_max(-acc);
      if (lane == 0) atomicMax(const_cast<int*>(&s_flags[2]), __float_as_int(am));
    }
    __syncthreads();
    if (tid < D) s_dC[tid] = ex2f(fmaxf(s_bm[tid] + s_ft[tid], -126.f));
  };

  // ---- products (issued by thread 0) -----------------------------------------------------------------------------------------
  // D[M=128 x N] (+)= A B over `ksteps` steps of 16; astep / bstep: byte advance of the operand per step
  auto mma_chain = [&](uint32_t col, uint64_t da, uint32_t astep, uint64_t db, uint32_t bstep, int ksteps, uint32_t idesc,
                       bool accumulate) {
    for (int k = 0; k < ksteps; ++k) mma_f16(tmem + col, dadv(da, astep * k), dadv(db, bstep * k), idesc, (accumulate || k > 0) ? 1u : 0u);
  };
  // the same on two-term operands: hi hi (+ lo hi + hi lo); a missing low part is passed as 0
  auto mma_split = [&](uint32_t col, uint64_t ah, uint64_t al, uint32_t astep, uint64_t bh_, uint64_t bl, uint32_t bstep,
                       int ksteps, uint32_t idesc, bool accumulate) {
    mma_chain(col, ah, astep, bh_, bstep, ksteps, idesc, accumulate);
    if (al) mma_chain(col, al, astep, bh_, bstep, ksteps, idesc, true);
    if (bl) mma_chain(col, ah, astep, bl, bstep, ksteps, idesc, true);
  };
  constexpr uint32_t KST_T = 2 * SLAB_T, KST_C = 2 * SLAB_C, MST = 256;  // K-major step (two slabs), MN-major step (16 rows)
  auto KV = [&](uint32_t off, uint32_t slab) -> uint64_t { return kview(sb + off, slab); };
  auto MV = [&](uint32_t off, uint32_t slab) -> uint64_t { return mview(sb + off, slab); };
  const uint64_t NONE = 0;

  // ---- operands of a chunk: qs, ks (two-term in the backward), kh (forward sweep) or qh (reverse sweep), v';
  // reverse sweep also do' (scaled, two-term), dO, and the row scalars dO.o and 1/den ---------------------------------------
  auto operand_pass = [&](int t0, int nvalid, bool f16, bool reverse, float sc, float& vmax) {
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
      const int o8 = tid & 7, r = (tid >> 3) + 32 * pass;
      float q[8], k[8], vv[8], x[8], w[8];
      uint4 zq = make_uint4(0u, 0u, 0u, 0u), zk = zq, zv = zq, zg = zq;
      float inv = 0.f, dl = 0.f;
      if (r < nvalid) {
        const size_t tq = ((size_t)b * a.T + t0 + r) * a.H + h, tv = ((size_t)b * a.T + t0 + r) * a.Hkv + j;
        if (a.feat_f32) {
          const float* fq = reinterpret_cast<const float*>(a.qdot) + tq * D + o8 * 8;
          const float* fk = reinterpret_cast<const float*>(a.kdot) + tq * D + o8 * 8;
          const float4 q0 = *reinterpret_cast<const float4*>(fq), q1 = *reinterpret_cast<const float4*>(fq + 4);
          const float4 k0 = *reinterpret_cast<const float4*>(fk), k1 = *reinterpret_cast<const float4*>(fk + 4);
          q[0] = q0.x; q[1] = q0.y; q[2] = q0.z; q[3] = q0.w; q[4] = q1.x; q[5] = q1.y; q[6] = q1.z; q[7] = q1.w;
          k[0] = k0.x; k[1] = k0.y; k[2] = k0.z; k[3] = k0.w; k[4] = k1.x; k[5] = k1.y; k[6] = k1.z; k[7] = k1.w;
        } else {
          zq = *reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(a.qdot) + tq * D + o8 * 8);
          zk = *reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(a.kdot) + tq * D + o8 * 8);
        }
        zv = *reinterpret_cast<const uint4*>(a.v + tv * D + o8 * 8);
        if (BWD && reverse) {
          zg = *reinterpret_cast<const uint4*>(a.dO + tq * D + o8 * 8);
          inv = a.ws_den[tq] * sc;
          dl = a.ws_delta[tq];
        }
      }
      if (!a.feat_f32 || r >= nvalid) { unpack8b(zq, q); unpack8b(zk, k); }
      unpack8b(zv, vv);
      const float4 xa = *reinterpret_cast<const float4*>(s_x + r * D + o8 * 8), xb = *reinterpret_cast<const float4*>(s_x + r * D + o8 * 8 + 4);
      x[0] = xa.x; x[1] = xa.y; x[2] = xa.z; x[3] = xa.w; x[4] = xb.x; x[5] = xb.y; x[6] = xb.z; x[7] = xb.w;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        q[i] *= ex2f(x[i]);
        k[i] *= ex2f(-x[i]);
        w[i] = reverse ? q[i] * s_dm[o8 * 8 + i] : k[i] * s_e63[o8 * 8 + i];
        vmax = fmaxf(vmax, fabsf(vv[i]));
      }
      put8(OFF_QS, oQSL, SLAB_T, r, o8 * 8, q, f16, SPLIT);
      put8(OFF_KS, oKSL, SLAB_T, r, o8 * 8, k, f16, SPLIT);
      put8(OFF_KQ, oKQL, SLAB_T, r, o8 * 8, w, f16, SPLIT);
      put8(OFF_VP, 0, SLAB_T, r, o8 * 8, vv, f16, false);
      const float one[8] = {1.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (o8 == 0) put8(OFF_VP, 0, SLAB_T, r, D, one, f16, false);
      if (BWD && reverse) {
        float g[8], gs[8];
        unpack8b(zg, g);
#pragma unroll
        for (int i = 0; i < 8; ++i) gs[i] = g[i] * inv;
        put8(OFF_DOX, 0, SLAB_T, r, o8 * 8, g, f16, false);
        put8(OFF_DO, OFF_DOL, SLAB_T, r, o8 * 8, gs, f16, true);
        if (o8 == 0) {
          const float dd[8] = {-dl * inv, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
          put8(OFF_DO, OFF_DOL, SLAB_T, r, D, dd, f16, true);
          s_row[r] = dl;
          s_row[C + r] = inv;
        }
      }
    }
  };

  // ====================================================================================================== forward sweep
  float domax = 0.f;
  if (MODE != 2) prefetch_chunk(0);
  for (int n = 0; MODE != 2 && n < nchunks; ++n) {
    const int t0 = n * C, nvalid = min(C, a.T - t0);
    GTL(0);
    prefetch_chunk(n + 1);
    gate_pass(t0, nvalid);
    __syncthreads();
    GTL(1);
    const bool f16 = __int_as_float(s_flags[2]) <= RMAX_F16 && sbound < SMAX_F16;
    // (the 8-bit-mantissa operands keep the range but not the accuracy bound: the caller is told)
    if (!f16 && tid == 0 && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_NUMERIC);
    const int fmt = f16 ? FMT_F16 : FMT_BF16;
    float vmax = 0.f;
    operand_pass(t0, nvalid, f16, false, 0.f, vmax);
    GTL(2);
    // ---- state pass: 16-bit operand 2^bm S', accumulator S' *= 2^bC; largest entry for the next chunk's format ------------
    float smax = 0.f;
    if (row_thr) {
      const float dm = s_dm[row], dC = s_dC[row];
      float s[8], w[8];
#pragma unroll 1
      for (int c0 = half * 48; c0 < (half ? NV : 48); c0 += 8) {
        tmem_ld8(lane_base + COL_ST + c0, s);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          smax = fmaxf(smax, fabsf(s[i]));
          w[i] = dm * s[i];
          s[i] *= dC;
        }
        put8(OFF_S16, OFF_S16L, SLAB_C, row, c0, w, f16, SPLIT);
        tmem_st8(lane_base + COL_ST + c0, s);
      }
      tmem_wait_st();
    }
    smax = fmaxf(warp_max(smax), 0.f);
    vmax = warp_max(vmax);
    if (lane == 0) {
      atomicMax(const_cast<int*>(&s_flags[3]), __float_as_int(smax < 3.0e38f ? smax : 3.0e38f));
      atomicMax(const_cast<int*>(&s_flags[4]), __float_as_int(vmax < 3.0e38f ? vmax : 3.0e38f));
    }
    publish();
    GTL(3);
    if (BWD) {  // the reverse sweep needs this chunk's state operand (two-term, and its format) again
      uint8_t* dst = a.ws_s16 + ((size_t)bh * nchunks + n) * (2 * TILE_CV + 16);
      for (int i = tid; i < (int)(2 * TILE_CV / 16); i += THREADS)
        reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(sg + OFF_S16)[i];
      if (tid == 0) *reinterpret_cast<int*>(dst + 2 * TILE_CV) = fmt;
    }
    if (tid == 0) {
      mma_split(COL_P, KV(OFF_QS, SLAB_T), SPLIT ? KV(oQSL, SLAB_T) : NONE, KST_T, KV(OFF_KS, SLAB_T),
                SPLIT ? KV(oKSL, SLAB_T) : NONE, KST_T, D / 16, instr_desc(128, C, fmt, MAJOR_K, MAJOR_K), false);
      mma_split(COL_A, KV(OFF_QS, SLAB_T), SPLIT ? KV(oQSL, SLAB_T) : NONE, KST_T, MV(OFF_S16, SLAB_C),
                SPLIT ? MV(OFF_S16L, SLAB_C) : NONE, MST, D / 16, instr_desc(128, NV, fmt, MAJOR_K, MAJOR_MN), false);
      mma_commit(bar);
    }
    sbound = __int_as_float(s_flags[3]) + 64.f * fmaxf(__int_as_float(s_flags[4]), 1.f);  // |S_new| <= |S_old| + 64 max|v|
    wait_mma();
    GTL(4);
    // ---- mask ----------------------------------------------------------------------------------------------------------------
    if (row_thr) {
      float s[8], w[8];
#pragma unroll 1
      for (int c0 = half * 32; c0 < half * 32 + 32; c0 += 8) {
        tmem_ld8(lane_base + COL_P + c0, s);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = (c0 + i <= row) ? s[i] : 0.f;
        put8(OFF_PM, oPML, SLAB_T, row, c0, w, f16, SPLIT);
      }
    }
    __syncthreads();
    if (tid == 0) { s_flags[3] = 0; s_flags[4] = 0; }
    publish();
    GTL(5);
    if (tid == 0) {
      mma_split(COL_A, KV(OFF_PM, SLAB_T), SPLIT ? KV(oPML, SLAB_T) : NONE, KST_T, MV(OFF_VP, SLAB_T), NONE, MST, C / 16,
                instr_desc(128, NV, fmt, MAJOR_K, MAJOR_MN), true);
      // (two-term kh in the backward: the state must hold each key's contribution exactly as the reverse sweep's own
      // products see that key, or the pairs that cancel in the gate gradient leave their rounding behind)
      mma_split(COL_ST, MV(OFF_KQ, SLAB_T), SPLIT ? MV(oKQL, SLAB_T) : NONE, MST, MV(OFF_VP, SLAB_T), NONE, MST, C / 16,
                instr_desc(128, NV, fmt, MAJOR_MN, MAJOR_MN), true);
      mma_commit(bar);
    }
    wait_mma();
    GTL(6);
    // ---- output: o = O'[:D] / (O'[D] + eps) ; backward: 1 / den and dO . o for the reverse sweep ------------------------
    if (row_thr) {
      const float den = tmem_ld1(lane_base + COL_A + D) + a.eps;
      tmem_wait_ld();
      const float inv = a.normalize ? 1.f / den : 1.f;
      const size_t th = ((size_t)b * a.T + t0 + row) * a.H + h;
      const bool valid = row < nvalid;
      float dot = 0.f, dmx = 0.f;
      float s[8];
#pragma unroll 1
      for (int c0 = half * 32; c0 < half * 32 + 32; c0 += 8) {
        tmem_ld8(lane_base + COL_A + c0, s);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i) s[i] *= inv;
        if (valid && !BWD) *reinterpret_cast<uint4*>(a.o + th * D + c0) = pack8h(s, false);
        if (BWD && valid) {
          float g[8];
          unpack8b(*reinterpret_cast<const uint4*>(a.dO + th * D + c0), g);
#pragma unroll
          for (int i = 0; i < 8; ++i) { dot = fmaf(g[i], s[i], dot); dmx = fmaxf(dmx, fabsf(g[i])); }
        }
      }
      if (!BWD && valid && half == 0 && a.den) a.den[th] = den;
      if (BWD) {
        s_row[half * C + row] = dot;
        domax = fmaxf(domax, valid ? fmaxf(dmx, 0.f) * fabsf(inv) : 0.f);
      }
    }
    if (BWD) {
      __syncthreads();
      if (row_thr && half == 0) {  // (tensor-memory loads are warp-collective: only the stores depend on the row)
        const float den = tmem_ld1(lane_base + COL_A + D) + a.eps;
        tmem_wait_ld();
        if (row < nvalid) {
          const size_t th = ((size_t)b * a.T + t0 + row) * a.H + h;
          const float inv = a.normalize ? 1.f / den : 1.f, dl = a.normalize ? s_row[row] + s_row[C + row] : 0.f;
          a.ws_den[th] = inv;
          a.ws_delta[th] = dl;
          domax = fmaxf(domax, fabsf(dl * inv));
        }
      }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    GTL(7);
  }
  // ---- final state -------------------------------------------------------------------------------------------------------
  if (!BWD && row_thr) {
    float s[8];
#pragma unroll 1
    for (int c0 = half * 48; c0 < (half ? NV : 48); c0 += 8) {
      tmem_ld8(lane_base + COL_ST + c0, s);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int e = c0 + i;
        if (e < D && a.S_T) a.S_T[((size_t)bh * D + row) * D + e] = s[i];
        if (e == D && a.z_T) a.z_T[(size_t)bh * D + row] = s[i];
      }
    }
  }

  if (MODE == 1) {  // the largest |do'| of the head, for the reverse sweep's scale
    domax = warp_max(domax);
    if (lane == 0) atomicMax(const_cast<int*>(&s_flags[4]), __float_as_int(domax < 3.0e38f ? domax : 3.0e38f));
    __syncthreads();
    if (tid == 0) a.ws_scale[bh] = __int_as_float(s_flags[4]);
  }
  // ====================================================================================================== reverse sweep
  if (MODE == 2) {
    // one power-of-two scale for do' over the whole head (every gradient is linear in do'): the largest |do'| lands just
    // below 2^8. The first tokens of a sequence have small denominators and a do' a hundred times the typical size; the
    // typical entries, and the adjoint state built from them, must stay clear of the fp16 subnormals. The masked score
    // gradients, sums of up to 65 such products, are saturated at the fp16 maximum.
    const float dm_all = fmaxf(a.ws_scale[bh], 1e-30f);
    const int ex = ((__float_as_int(dm_all) >> 23) & 0xff) - 127 + 1 - 8;           // 2^(ex + 8) > max |do'|
    const float sc = __int_as_float((127 - min(max(ex, -100), 100)) << 23);        // 2^-ex
    const float isc = __int_as_float((127 + min(max(ex, -100), 100)) << 23);       // 2^ex
    bool prev_f16 = true;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    prefetch_chunk(nchunks - 1);
    for (int n = nchunks - 1; n >= 0; --n) {
      const int t0 = n * C, nvalid = min(C, a.T - t0);
      prefetch_chunk(n - 1);
      GTL(8);
      // ---- what crosses the end of this chunk: all pairs (key at or before the chunk, query behind it) feel every decay of
      // the chunk; their sum per key channel is the row-wise product of the state after the chunk with its adjoint,
      // sum_e S'_n[c,e] R_n[c,e]. S'_n is taken from the next chunk's state operand 2^bm S'_n (two-term, still in shared
      // memory), R_n from tensor memory. Nothing is carried from chunk to chunk: rounding noise does not add up along T.
      float carry = 0.f;  // (threads tid < D) channel tid
      if (n < nchunks - 1) {
        if (row_thr) {
          float r[8], sv[8], sl[8], dot = 0.f;
#pragma unroll 1
          for (int c0 = half * 48; c0 < (half ? NV : 48); c0 += 8) {
            tmem_ld8(lane_base + COL_ST + c0, r);
            tmem_wait_ld();
            unpack8h(*reinterpret_cast<const uint4*>(sg + OFF_S16 + toff(SLAB_C, row, c0)), prev_f16, sv);
            unpack8h(*reinterpret_cast<const uint4*>(sg + OFF_S16L + toff(SLAB_C, row, c0)), prev_f16, sl);
#pragma unroll
            for (int i = 0; i < 8; ++i) dot = fmaf(sv[i] + sl[i], r[i], dot);
          }
          s_row[half * C + row] = dot;
        }
        __syncthreads();
        if (tid < D) carry = (s_row[tid] + s_row[C + tid]) * ex2f(fminf(-s_bm[tid], 126.f)) * isc;
      }
      GTL(9);
      gate_pass(t0, nvalid);
      GTL(10);
      const uint8_t* src = a.ws_s16 + ((size_t)bh * nchunks + n) * (2 * TILE_CV + 16);
      const int fmt = *reinterpret_cast<const int*>(src + 2 * TILE_CV);
      const bool f16 = fmt == FMT_F16;
      prev_f16 = f16;
      for (int i = tid; i < (int)(2 * TILE_CV / 16); i += THREADS)
        reinterpret_cast<uint4*>(sg + OFF_S16)[i] = reinterpret_cast<const uint4*>(src)[i];
      __syncthreads();
      float vmax_unused = 0.f;
      operand_pass(t0, nvalid, f16, true, sc, vmax_unused);
      GTL(11);
      // ---- adjoint-state pass: two-term operand 2^ft R, accumulator R *= 2^bC --------------------------------------------
      if (row_thr) {
        const float e63 = s_e63[row], dC = s_dC[row];
        float s[8], w[8];
#pragma unroll 1
        for (int c0 = half * 48; c0 < (half ? NV : 48); c0 += 8) {
          tmem_ld8(lane_base + COL_ST + c0, s);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            w[i] = e63 * s[i];
            s[i] *= dC;
          }
          put8(OFF_R16, OFF_R16L, SLAB_C, row, c0, w, f16, true);
          tmem_st8(lane_base + COL_ST + c0, s);
        }
        tmem_wait_st();
      }
      publish();
      GTL(12);
      if (tid == 0) {
        mma_split(COL_P, KV(OFF_QS, SLAB_T), KV(oQSL, SLAB_T), KST_T, KV(OFF_KS, SLAB_T), KV(oKSL, SLAB_T), KST_T,
                  D / 16, instr_desc(128, C, fmt, MAJOR_K, MAJOR_K), false);
        // dO v^T with both operands exact: the row terms are applied in fp32 by the mask pass
        mma_chain(COL_DP, KV(OFF_DOX, SLAB_T), KST_T, KV(OFF_VP, SLAB_T), KST_T, D / 16,
                  instr_desc(128, C, fmt, MAJOR_K, MAJOR_K), false);
        mma_commit(bar);
      }
      wait_mma();
      GTL(13);
      if (row_thr) {
        const float dl = s_row[row], inv = s_row[C + row];  // dO_t . o_t and (scaled) 1 / den_t of this row
        float s[8], w[8];
#pragma unroll 1
        for (int c0 = half * 32; c0 < half * 32 + 32; c0 += 8) {
          tmem_ld8(lane_base + COL_P + c0, s);
          tmem_ld8(lane_base + COL_DP + c0, w);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            s[i] = (c0 + i <= row) ? s[i] : 0.f;
            w[i] = (c0 + i <= row) ? fminf(fmaxf((w[i] - dl) * inv, -65000.f), 65000.f) : 0.f;
          }
          put8(OFF_PM, oPML, SLAB_T, row, c0, s, f16, true);
          put8(OFF_DPM, OFF_DPL, SLAB_T, row, c0, w, f16, true);
        }
      }
      publish();
      GTL(14);
      if (tid == 0) {
        const uint32_t ID_KM = instr_desc(128, D, fmt, MAJOR_K, MAJOR_MN), ID_MM = instr_desc(128, D, fmt, MAJOR_MN, MAJOR_MN),
                       ID_KK = instr_desc(128, D, fmt, MAJOR_K, MAJOR_K);
        const uint32_t IV_MM = instr_desc(128, NV, fmt, MAJOR_MN, MAJOR_MN), IV_KM = instr_desc(128, NV, fmt, MAJOR_K, MAJOR_MN);
        // dQ = dP ks + do' (2^bm S')^T
        mma_split(COL_A, KV(OFF_DPM, SLAB_T), KV(OFF_DPL, SLAB_T), KST_T, MV(OFF_KS, SLAB_T), MV(oKSL, SLAB_T), MST,
                  C / 16, ID_KM, false);
        mma_split(COL_A, KV(OFF_DO, SLAB_T), KV(OFF_DOL, SLAB_T), KST_T, KV(OFF_S16, SLAB_C), KV(OFF_S16L, SLAB_C), KST_C,
                  NV / 16, ID_KK, true);
        // dK = dP^T qs + v' (2^ft R)^T
        mma_split(COL_B, MV(OFF_DPM, SLAB_T), MV(OFF_DPL, SLAB_T), MST, MV(OFF_QS, SLAB_T), MV(oQSL, SLAB_T), MST,
                  C / 16, ID_MM, false);
        mma_split(COL_B, KV(OFF_VP, SLAB_T), NONE, KST_T, KV(OFF_R16, SLAB_C), KV(OFF_R16L, SLAB_C), KST_C, NV / 16, ID_KK,
                  true);
        // dV' = P^T do' + ks (2^ft R)
        mma_split(COL_V, MV(OFF_PM, SLAB_T), MV(oPML, SLAB_T), MST, MV(OFF_DO, SLAB_T), MV(OFF_DOL, SLAB_T), MST, C / 16,
                  IV_MM, false);
        mma_split(COL_V, KV(OFF_KS, SLAB_T), KV(oKSL, SLAB_T), KST_T, MV(OFF_R16, SLAB_C), MV(OFF_R16L, SLAB_C), MST,
                  D / 16, IV_KM, true);
        // R += (qs 2^bm)^T do'
        mma_split(COL_ST, MV(OFF_KQ, SLAB_T), MV(oKQL, SLAB_T), MST, MV(OFF_DO, SLAB_T), MV(OFF_DOL, SLAB_T), MST, C / 16,
                  IV_MM, true);
        mma_commit(bar);
      }
      wait_mma();
      GTL(15);
      // ---- gradients of this chunk's rows ----------------------------------------------------------------------------------
      if (row_thr) {
        const size_t th = ((size_t)b * a.T + t0 + row) * a.H + h;
        const bool valid = row < nvalid;
        float dq[8], dk[8], dvv[8], rq[8], rk[8];
#pragma unroll 1
        for (int c0 = half * 32; c0 < half * 32 + 32; c0 += 8) {
          tmem_ld8(lane_base + COL_A + c0, dq);
          tmem_ld8(lane_base + COL_B + c0, dk);
          tmem_ld8(lane_base + COL_V + c0, dvv);
          tmem_wait_ld();
          // qdot dqdot - kdot dkdot = qs dQ - ks dK with qs, ks as the products saw them (hi + lo): every pair of tokens
          // inside the chunk then contributes the same number to both terms, and the reverse running sum below (in which
          // all pairs behind a token cancel) keeps only what it should
          {
            float lo[8];
            unpack8h(*reinterpret_cast<const uint4*>(sg + OFF_QS + toff(SLAB_T, row, c0)), f16, rq);
            unpack8h(*reinterpret_cast<const uint4*>(sg + oQSL + toff(SLAB_T, row, c0)), f16, lo);
#pragma unroll
            for (int i = 0; i < 8; ++i) rq[i] += lo[i];
            unpack8h(*reinterpret_cast<const uint4*>(sg + OFF_KS + toff(SLAB_T, row, c0)), f16, rk);
            unpack8h(*reinterpret_cast<const uint4*>(sg + oKSL + toff(SLAB_T, row, c0)), f16, lo);
#pragma unroll
            for (int i = 0; i < 8; ++i) rk[i] += lo[i];
          }
          float dd[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float xv = s_x[row * D + c0 + i];
            dd[i] = (rq[i] * dq[i] - rk[i] * dk[i]) * isc;
            dq[i] *= ex2f(xv) * isc;
            dk[i] *= ex2f(-xv) * isc;
            dvv[i] *= isc;
          }
          *reinterpret_cast<float4*>(s_dt + row * D + c0) = make_float4(dd[0], dd[1], dd[2], dd[3]);
          *reinterpret_cast<float4*>(s_dt + row * D + c0 + 4) = make_float4(dd[4], dd[5], dd[6], dd[7]);
          if (valid) {
            if (a.feat_f32) {
              float* gq = reinterpret_cast<float*>(a.d_qdot) + th * D + c0;
              float* gk = reinterpret_cast<float*>(a.d_kdot) + th * D + c0;
              *reinterpret_cast<float4*>(gq) = make_float4(dq[0], dq[1], dq[2], dq[3]);
              *reinterpret_cast<float4*>(gq + 4) = make_float4(dq[4], dq[5], dq[6], dq[7]);
              *reinterpret_cast<float4*>(gk) = make_float4(dk[0], dk[1], dk[2], dk[3]);
              *reinterpret_cast<float4*>(gk + 4) = make_float4(dk[4], dk[5], dk[6], dk[7]);
            } else {
              *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(a.d_qdot) + th * D + c0) = pack8h(dq, false);
              *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(a.d_kdot) + th * D + c0) = pack8h(dk, false);
            }
            *reinterpret_cast<float4*>(a.dvh + th * D + c0) = make_float4(dvv[0], dvv[1], dvv[2], dvv[3]);
            *reinterpret_cast<float4*>(a.dvh + th * D + c0 + 4) = make_float4(dvv[4], dvv[5], dvv[6], dvv[7]);
          }
        }
      }
      tc_fence_before_sync();
      __syncthreads();
      tc_fence_after_sync();
      GTL(16);
      // ---- gate gradient: reverse running sum over the chunk's tokens on top of what crosses its end, then the derivative
      // of the log-decay ----------------------------------------------------------------------------------------------------
      {
        // thread = (channel, quarter of the chunk): running sums inside the quarter, then the totals of the quarters behind
        // it and what crosses the chunk's end on top (rows past the end hold zeros: their operands were zero)
        const int c = tid & (D - 1), seg = tid >> 6;
        float* const s_tot = s_ft;  // [4][D]: s_ft, s_dm, s_e63, s_dC are free until the next chunk's gate pass
        if (tid < D) s_row[tid] = carry;
        float v[16], acc = 0.f;
#pragma unroll
        for (int i = 15; i >= 0; --i) {
          acc += s_dt[(seg * 16 + i) * D + c];
          v[i] = acc;
        }
        s_tot[seg * D + c] = acc;
        __syncthreads();
        float off = s_row[c];
#pragma unroll
        for (int s2 = 3; s2 >= 1; --s2)
          if (s2 > seg) off += s_tot[s2 * D + c];
#pragma unroll
        for (int i = 0; i < 16; ++i) s_dt[(seg * 16 + i) * D + c] = v[i] + off;
      }
      __syncthreads();
      if (a.gate_dim == 1) {
        if (tid < nvalid) {
          float sum = 0.f;
          for (int c = 0; c < D; ++c) sum += s_dt[tid * D + ((c + tid) & (D - 1))];
          const size_t gi = ((size_t)b * a.T + t0 + tid) * a.H + h;
          const float av = __bfloat162float(a.gate[gi]);
          const float dv_ = a.gate_mode == LAWCAT_GATE_LOGDECAY ? 1.f : (1.f - 1.f / (1.f + __expf(-av))) * a.inv_tau;
          a.dgate[gi] = __float2bfloat16_rn(sum * dv_);
        }
      } else {
#pragma unroll 1
        for (int pass = 0; pass < 2; ++pass) {
          const int o8 = tid & 7, r = (tid >> 3) + 32 * pass;
          if (r < nvalid) {
            const size_t gi = (((size_t)b * a.T + t0 + r) * a.H + h) * D + o8 * 8;
            float av[8], out[8];
            unpack8b(*reinterpret_cast<const uint4*>(a.gate + gi), av);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float dv_ = a.gate_mode == LAWCAT_GATE_LOGDECAY ? 1.f : (1.f - 1.f / (1.f + __expf(-av[i]))) * a.inv_tau;
              out[i] = s_dt[r * D + o8 * 8 + i] * dv_;
            }
            *reinterpret_cast<uint4*>(a.dgate + gi) = pack8h(out, false);
          }
        }
      }
      __syncthreads();
      GTL(17);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

// dv[b,t,j,:] = sum over the G query heads of group j of the per-head gradients (keys and values are shared in a group)
__global__ void dv_reduce_kernel(const float* __restrict__ dvh, bf16* __restrict__ dv, size_t total, int G) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;  // one thread per 8 channels of one (b, t, kv head)
  if (idx >= total) return;
  const size_t btj = idx / (D / 8);
  const int o8 = (int)(idx % (D / 8));
  float s[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int g = 0; g < G; ++g) {
    const float4* p = reinterpret_cast<const float4*>(dvh + (btj * G + g) * D + o8 * 8);
    const float4 x = p[0], y = p[1];
    s[0] += x.x; s[1] += x.y; s[2] += x.z; s[3] += x.w; s[4] += y.x; s[5] += y.y; s[6] += y.z; s[7] += y.w;
  }
  *reinterpret_cast<uint4*>(dv + btj * D + o8 * 8) = pack8h(s, false);
}

static int set_smem_once() {
  static std::mutex mu;
  static bool done[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LAWCAT_ERR_CUDA;
  std::lock_guard<std::mutex> lk(mu);
  if (!done[dev]) {
    cudaError_t e = cudaFuncSetAttribute(gla_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_FWD);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gla_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_SWEEP);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gla_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BWD);
    if (e != cudaSuccess) {
      note_cuda_error(e, __FILE__, __LINE__);
      return LAWCAT_ERR_CUDA;
    }
    done[dev] = true;
  }
  return LAWCAT_OK;
}

}  // namespace gtc

// Under a sharp gate (LOGITS with tau < 8: the decay exponents of half a chunk leave the fp16 range and the operands fall
// back to 8 significant bits) results and gradients miss the accuracy bound, and so does the state of a call of fewer than
// 16 tokens (too few terms to average the rounding of single operands): both take the exact recurrence.
bool gla_tc_bwd_supported(const lawcat_params& p) { return gla_tc_supported(p); }

bool gla_tc_supported(const lawcat_params& p) {
  const bool sharp = p.gate_mode == LAWCAT_GATE_LOGITS && p.gate_tau < 8.f;
  return p.dtype == LAWCAT_BF16 && p.d_k == gtc::D && p.d_v == gtc::D && (p.gate_dim == p.d_k || p.gate_dim == 1) &&
         !sharp && p.B > 0 && p.T >= 16 && (p.chunk == 0 || p.chunk == gtc::C);
}

// scratch of the backward: per-head dv (fp32), 1/den and dO.o per token and head, the state operand of every chunk
size_t gla_tc_bwd_workspace_bytes(const lawcat_params& p) {
  const size_t bth = (size_t)p.B * p.T * p.H, chunks = (p.T + gtc::C - 1) / gtc::C;
  return align_up(sizeof(float) * bth * gtc::D, 256) + 2 * align_up(sizeof(float) * bth, 256) +
         align_up(sizeof(float) * (size_t)p.B * p.H, 256) +
         align_up((size_t)p.B * p.H * chunks * (2 * gtc::TILE_CV + 16), 256);
}

static gtc::GArgs gla_tc_args(const Ctx& c) {
  const lawcat_params& p = *c.p;
  gtc::GArgs a{};
  a.dev_status = c.dev_status;
  a.B = p.B; a.T = p.T; a.H = p.H; a.Hkv = p.H_kv; a.gate_dim = p.gate_dim; a.gate_mode = p.gate_mode;
  a.normalize = p.normalize; a.inv_tau = 1.f / p.gate_tau; a.eps = p.eps;
  return a;
}

int launch_gla_fwd_tc(const Ctx& c, const void* qdot, const void* kdot, const void* v, const void* gate, const float* S0,
                      const float* z0, void* o, float* den, float* S_T, float* z_T, bool feat_f32) {
  using namespace gtc;
  const lawcat_params& p = *c.p;
  int r = set_smem_once();
  if (r) return r;
  GArgs a = gla_tc_args(c);
  a.qdot = qdot; a.kdot = kdot; a.v = (const bf16*)v; a.gate = (const bf16*)gate;
  a.S0 = S0; a.z0 = z0; a.o = (bf16*)o; a.den = den; a.S_T = S_T; a.z_T = z_T; a.feat_f32 = feat_f32 ? 1 : 0;
  LaunchScope _ls("gla_tc_fwd", c.stream);
  gla_tc_kernel<0><<<p.B * p.H, THREADS, SMEM_FWD, c.stream>>>(a);
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

int launch_gla_bwd_tc(const Ctx& c, const void* qdot, const void* kdot, const void* v, const void* gate, const float* S0,
                      const float* z0, const void* dO, void* d_qdot, void* d_kdot, void* dv, void* dgate, void* ws,
                      bool feat_f32) {
  using namespace gtc;
  const lawcat_params& p = *c.p;
  int r = set_smem_once();
  if (r) return r;
  GArgs a = gla_tc_args(c);
  a.qdot = qdot; a.kdot = kdot; a.v = (const bf16*)v; a.gate = (const bf16*)gate;
  a.dO = (const bf16*)dO; a.S0 = S0; a.z0 = z0;
  a.d_qdot = d_qdot; a.d_kdot = d_kdot; a.dgate = (bf16*)dgate; a.feat_f32 = feat_f32 ? 1 : 0;
  const size_t bth = (size_t)p.B * p.T * p.H;
  char* w = (char*)ws;
  a.dvh = (float*)w; w += align_up(sizeof(float) * bth * D, 256);
  a.ws_den = (float*)w; w += align_up(sizeof(float) * bth, 256);
  a.ws_delta = (float*)w; w += align_up(sizeof(float) * bth, 256);
  a.ws_scale = (float*)w; w += align_up(sizeof(float) * (size_t)p.B * p.H, 256);
  a.ws_s16 = (uint8_t*)w;
  {
    LaunchScope _ls("gla_tc_bwd_sweep", c.stream);
    gla_tc_kernel<1><<<p.B * p.H, THREADS, SMEM_SWEEP, c.stream>>>(a);
    LAWCAT_CHECK_LAUNCH();
  }
  {
    LaunchScope _ls("gla_tc_bwd", c.stream);
    gla_tc_kernel<2><<<p.B * p.H, THREADS, SMEM_BWD, c.stream>>>(a);
    LAWCAT_CHECK_LAUNCH();
  }
  const size_t total = (size_t)p.B * p.T * p.H_kv * (D / 8);
  LaunchScope _ls("dv_reduce", c.stream);
  dv_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, c.stream>>>(a.dvh, (bf16*)dv, total, p.H / p.H_kv);
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

}  // namespace lawcat

#ifdef LAWCAT_TIMELINE
extern "C" int lawcat_gla_timeline_read(long long* host, size_t n) {
  return cudaMemcpyFromSymbol(host, lawcat::gtc::g_gla_timeline, sizeof(long long) * (n < 32 ? n : 32)) == cudaSuccess
             ? LAWCAT_OK : LAWCAT_ERR_CUDA;
}
#endif
