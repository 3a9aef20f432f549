// The whole layer forward of Fig. 1 as ONE chunkwise tensor-core kernel for bf16 storage, d_k = d_v = 128:
// conv (Section 4.1) -> shared linear layer + softmax feature map (Section 4.1) -> normalized gated linear attention
// (Eq. 4 - Eq. 8) in its chunkwise-parallel form, with the d_k x (d_v+1) state [S | z] kept in tensor memory in fp32.
//
// One CTA walks one (batch, query head, segment of the sequence) in chunks of C = 64 tokens. The work of a chunk is
// split over specialized warps that hand tiles to one another through mbarriers, so that consecutive chunks overlap:
//   TMA warp    raw q, k tiles (one stacked [128 x 128] tile: rows 0-63 query tokens, rows 64-127 key tokens), gate
//               logits and v tiles -> 128-byte-swizzled shared memory
//   prep warps  conv: u = sum_delta w_delta * x_{t-delta} in fp32 -> fp16, IN PLACE over the raw tile, which thereby
//               becomes the stacked A operand of the mix (both streams share W_h, so ONE M=128 MMA mixes both);
//               gate: g = log2 sigmoid(a) / tau per entry, then a scan outwards from the middle token gives the
//               exponents x_t = b_t - b_mid (b the running sum of g) in fp32 (the middle reference keeps every factor
//               2^x within 2^(+-32 max|g|)); v: bf16 -> fp16 in place (exact)
//   MMA warp    MMA 1: Y = [u_q; u_k] W_h  (fp16 operands, fp32 accumulate in TMEM)
//   row warps   (two threads per token row, 64 columns each, straight from tensor memory)
//               phi: row softmax. Query rows keep exp(y - max) unnormalized: a positive per-token factor cancels in
//               Eq. 8. The decay factors ride in the exponent of the softmax: qs = 2^(y' + x_t), ks = phi_k 2^(-x_i),
//               kh = phi_k 2^(b_C - b_i) (<= phi_k)
//   row warps   state pass: 2^b_mid [S|z] as a 16-bit operand, accumulator [S|z] *= 2^b_C
//   MMA warp    MMA 2: P = qs ks^T ; O' = qs (2^b_mid [S|z]) ; [S|z] += kh^T [v|1]
//   row warps   mask: P_ti = 0 for i > t, rounded to fp16 (behind the reading sweeps of the next chunk)
//   MMA warp    MMA 3: O' += P [v|1]
//   prep warps  o_t = O'_t[:d_v] / (O'_t[d_v] + eps) -> bf16 -> global memory (the warps of TMEM quadrants 0-1)
// Operand precision: qs, ks and the state operand are fp16 (11-bit mantissa) while the chunk's x stay within
// +-8 and the state within +-3e4 -- the usual case -- and bf16 otherwise (range first). bf16 score weights would
// cost up to 2^-9 relative error per weight, which the first tokens of a sequence do not average out.
// Every MMA uses M = 128; where only 64 rows are meaningful (P, O') the upper 64 TMEM lanes hold unused results.
// Loops over column blocks are deliberately NOT unrolled: each role's loop must stay inside the instruction cache.
// Every wait is bounded: a wait that runs out raises the abort flag, every role leaves its loop, the CTA frees its
// tensor memory and reports LAWCAT_ERR_TIMEOUT through dev_status.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace lawcat {
namespace tc {

// Optional time line (profiling builds only, -DLAWCAT_TIMELINE): one lane per role of thread block 0 stamps the clock at
// fixed points of four consecutive chunks into a device array that lawcat_timeline_read copies out.
#ifdef LAWCAT_TIMELINE
#ifndef LAWCAT_TIMELINE_MODE
#define LAWCAT_TIMELINE_MODE 0   // which kernel mode stamps: 0 the layer, 1 the state-only pass
#endif
#ifndef LAWCAT_TIMELINE_N0
#define LAWCAT_TIMELINE_N0 40    // first of the four chunks that stamp
#endif
#ifndef LAWCAT_TL_BLOCK
#define LAWCAT_TL_BLOCK 0        // the thread block whose pending waits are recorded when a wait runs out
#endif
constexpr int TL_ROLES = 6, TL_IDS = 16, TL_N0 = LAWCAT_TIMELINE_N0, TL_NCH = 4;
__device__ long long g_timeline[TL_ROLES * TL_IDS * TL_NCH];
#define TL(role, id, n, who)                                                                        \
  do {                                                                                              \
    if (MODE == LAWCAT_TIMELINE_MODE && blockIdx.x == 0 && (who) && (n) >= TL_N0 && (n) < TL_N0 + TL_NCH) \
      g_timeline[((role) * TL_IDS + (id)) * TL_NCH + ((n) - TL_N0)] = clock64();                    \
  } while (0)
#else
#define TL(role, id, n, who) do { } while (0)
#endif

constexpr int D = 128;       // d_k = d_v
constexpr int C = 64;        // tokens per chunk
constexpr int MID = 31;      // reference token of the in-chunk decay factorization
constexpr int HALO = 3;      // raw rows in front of a chunk that the conv needs (conv width up to 4)

// warps: 0-7 prep, 8-15 row warps (TMEM quadrant = warp & 3, column half = (warp - 8) >> 2), 16 TMA, 17 MMA
constexpr int PREP_THREADS = 256;
constexpr int ROW_WARP0 = 8, TMA_WARP = 16, MMA_WARP = 17;
constexpr int THREADS = 18 * 32;

// shared memory map (byte offsets from a 1024-byte aligned base)
constexpr uint32_t OFF_W = 0;                     // W_h^T fp16, K-major, 2 slabs x [128 x 128 B]
constexpr uint32_t OFF_SBF = OFF_W + 32768;       // 2^b_mid * [S | z], 16 bit, MN-major B operand of the read-out product,
                                                  // unswizzled 8x8 core matrices: block of 8 columns nb at nb * 2048,
                                                  // key channel c at (c / 8) * 128 + (c % 8) * 16 inside a block; the
                                                  // blocks of S are followed by two blocks whose first column is z
constexpr uint32_t OFF_PH2 = OFF_SBF + 20480;     // (two 64-wide heads per block: the state operand has 80 columns = 20 KB;
                                                  // the second head's masked scores [64 x 128 B] use the rest, and the 8 KB an
                                                  // M = 128 product reads behind them stay inside this tile)
constexpr uint32_t OFF_AU = OFF_SBF + 36864;      // raw q|k tile, then conv output in place: A of MMA 1, 2 slabs
constexpr uint32_t OFF_QK = OFF_AU + 32768;       // qs (rows 0-63) | ks (rows 64-127), 16 bit, K-major, 2 slabs
constexpr uint32_t OFF_X = OFF_QK + 32768;        // exponents x fp32 [64 x 128], XOR-swizzled 16-byte chunks
constexpr uint32_t OFF_KH = OFF_X + 32768;        // kh fp16, MN-major A of the state update, 2 slabs x [64 tokens x 128 B]
constexpr uint32_t OFF_G = OFF_KH + 16384;        // gate logits bf16, 2 slabs x [64 x 128 B]
constexpr uint32_t OFF_PH = OFF_G + 16384;        // masked scores fp16, K-major, [64 x 128 B]; an M=128 MMA also reads
                                                  // (and ignores) the 8 KB that follow (the first half of the v tile)
constexpr uint32_t OFF_V = OFF_PH + 8192;         // v bf16, then fp16 in place, MN-major B, 2 slabs x [64 x 128 B]
constexpr uint32_t OFF_ONES = OFF_V + 16384;      // [64 x 16] fp16 operand whose column 0 is 1 (the "1" of [v|1])
constexpr uint32_t OFF_HALO = OFF_ONES + 2048;    // [2 streams][3 rows][16 x 16 B]: raw rows in front of the next chunk
constexpr uint32_t OFF_VEC = OFF_HALO + 1536;     // per parity: bm[128], ft[128], e63[128] fp32 (2 x 1536 B)
constexpr uint32_t OFF_BAR = OFF_VEC + 3072;      // mbarriers (8 B each) and scalars
constexpr uint32_t SMEM_BYTES = OFF_BAR + 256;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES;  // all dynamic, declared 1024-byte aligned (the kernel checks it)
static_assert(OFF_PH + 16384 <= SMEM_BYTES, "the unused rows of the score operand must stay inside the allocation");
static_assert(SMEM_ALLOC <= 232448, "shared memory budget");
constexpr float SMAX_F16 = 3.0e4f;  // largest |state entry| for which the operands are kept in fp16
constexpr float RMAX_F16 = 8.f;     // largest |x| for which the operands are kept in fp16

// tensor memory map (32-bit columns)
constexpr uint32_t COL_Y = 0;      // [128 x 128] mix output
constexpr uint32_t COL_S = 128;    // [128 x 128] state S
constexpr uint32_t COL_O = 256;    // [128 x (128 + 16)] numerator, directly followed by the state's part of the denominator
                                   // (column COL_O + head width); lanes 0-63 meaningful
constexpr uint32_t COL_P = 400;    // [128 x 64] scores (lanes 0-63 meaningful)
constexpr uint32_t COL_SZ = 464;   // [128 x 16] column 0: normalizer state z
constexpr uint32_t COL_MAIL = 480; // spare columns used as per-row mailboxes between threads of one TMEM lane:
                                   // +2, +3: row max / softmax sum of the two column halves; +4 p + half (p = chunk
                                   // parity): the dropped query normalizer (softmax sum) of that half, row warps -> output
                                   // pass; +8 + 2 p + half: the chunk's own part of the denominator (row sum of the masked
                                   // scores of that half), mask pass -> output pass
constexpr uint32_t TMEM_COLS = 512;

// mbarrier indices. "full": producer -> consumer, "free": consumer -> producer. Each completes once per chunk, so the
// wait parity of chunk n is n & 1.
enum {
  B_RAW_FULL = 0,  // TMA: raw q|k tile landed                      -> prep (conv)
  B_G_FULL,        // TMA: gate tile landed                          -> prep (gate)
  B_V_FULL,        // TMA: v tile landed                             -> prep (v convert)
  B_G_FREE,        // prep: gate tile consumed                       -> TMA
  B_U_FULL,        // prep: conv output written                      -> MMA 1
  B_X_FULL,        // prep: exponents, per-channel sums, range flags -> row warps
  B_VH_FULL,       // prep: v converted                              -> MMA 2, row warps
  B_MMA1,          // MMA 1 complete: Y ready -> row warps; raw tile free -> TMA
  B_Y_FREE,        // row warps: Y consumed                          -> MMA 1 of the next chunk
  B_X_FREE,        // row warps: exponents consumed                  -> prep (gate of the next chunk)
  B_QK_FULL,       // row warps: qs, ks, kh written                  -> MMA 2
  B_SBF_FULL,      // row warps: state operand written, S decayed    -> MMA 2
  B_P,             // score product complete: P ready                -> row warps (mask)
  B_MMA2,          // MMA 2 complete: state updated, read-out started O', qs/ks/kh/state operand free
  B_PH_FULL,       // row warps: masked scores written               -> MMA 3
  B_MMA3,          // MMA 3 complete: O' ready -> row warps; v tile free -> TMA
  B_O_FREE,        // row warps: O' consumed                         -> MMA 2 of the next chunk
  NUM_BARS
};

struct TcArgs {
  const bf16 *q, *k;     // raw streams (for the halo rows in front of a segment)
  const bf16* gate;      // gate logits; read directly when there is one per token and head (gate_dim = 1)
  int gate_dim;          // d_k: one decay per key channel (tile loads); 1: one per head, shared by all channels
  int dh;                // d_k = d_v of the tensors: 128, or 64. A 64-wide head runs as a 128-wide one whose upper 64
                         // channels (of q, k, gate, v, W, the state) are zero: the tiles' second 64-channel slabs are
                         // zeroed once and never loaded, and the feature map leaves the padded outputs out
  const bf16 *w_q, *w_k, *W, *cache_q, *cache_k;
  const float *S0, *z0;  // state before the first token of the CTA's segment
  float *S_T, *z_T;      // state after the last token of the CTA's segment
  float* dtot;           // [B,H,nseg,128]: log2 of the total decay of the segment per key channel (nullable)
  bf16* o;               // [B,T,H,128]
  bf16 *cache_q_out, *cache_k_out;  // conv caches after the last token (nullable): [B,K-1,H*dh], [B,K-1,Hkv*dh]
  int* dev_status;
  int T, H, Hkv, K;
  int nseg, seg_len;     // segments per sequence and tokens per segment (a multiple of C)
  int grid_nseg;         // segments of each sequence covered by this launch (the first grid_nseg of nseg)
  int nsub;              // pieces each segment is cut into by this launch (whole chunks; 1 = the segment itself)
  int seg_in;            // 1: S0/z0 are indexed [b,h,seg*nsub+sub]; 0: [b,h] and they apply to segment 0 only
  int seg_out;           // 1: S_T/z_T (and dtot) are indexed [b,h,seg*nsub+sub]; 0: [b,h], written by the last segment
  int gate_mode;
  int normalize;         // 1: Eq. 8; 0: the numerator alone (the query features then carry their softmax normalizer)
  float inv_tau, eps;
  long long wait_limit;  // clock cycles a device-side wait may take before the block gives up (about 2 s by default)
};

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
  f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
}
// 8 bf16 values -> 4 packed pairs of fp32
__device__ __forceinline__ void unpack8p(const uint4& v, uint64_t* f) {
  f[0] = f2_pack(bf16_lo(v.x), bf16_hi(v.x)); f[1] = f2_pack(bf16_lo(v.y), bf16_hi(v.y));
  f[2] = f2_pack(bf16_lo(v.z), bf16_hi(v.z)); f[3] = f2_pack(bf16_lo(v.w), bf16_hi(v.w));
}
// 4 packed pairs of fp32 -> 8 packed 16-bit values, fp16 or bf16
__device__ __forceinline__ uint4 pack8p(const uint64_t* v, bool f16) {
  float f[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) f2_unpack(v[i], f[2 * i], f[2 * i + 1]);
  return f16 ? make_uint4(pack_f16(f[0], f[1]), pack_f16(f[2], f[3]), pack_f16(f[4], f[5]), pack_f16(f[6], f[7]))
             : make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
}
// 8 values -> 8 packed 16-bit values, fp16 or bf16
__device__ __forceinline__ uint4 pack8(const float* v, bool f16) {
  return f16 ? make_uint4(pack_f16(v[0], v[1]), pack_f16(v[2], v[3]), pack_f16(v[4], v[5]), pack_f16(v[6], v[7]))
             : make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
__device__ __forceinline__ uint16_t to16(float x, bool f16) {
  return f16 ? __half_as_ushort(__float2half_rn(x)) : __bfloat16_as_ushort(__float2bfloat16_rn(x));
}

// channels [8 jj, 8 jj + 8) of row t of the fp32 exponent tile (see the gate pass for its layout)
__device__ __forceinline__ void load_x8(uint32_t base, int t, int jj, float* x) {
  const uint4 lo = lds128(base + t * 512 + (((2 * jj) ^ (t & 7)) << 4));
  const uint4 hi = lds128(base + t * 512 + (((2 * jj + 1) ^ (t & 7)) << 4));
  x[0] = __uint_as_float(lo.x); x[1] = __uint_as_float(lo.y); x[2] = __uint_as_float(lo.z); x[3] = __uint_as_float(lo.w);
  x[4] = __uint_as_float(hi.x); x[5] = __uint_as_float(hi.y); x[6] = __uint_as_float(hi.z); x[7] = __uint_as_float(hi.w);
}

// log2(sigmoid(a)) = -log2(1 + 2^x) with 2^x = exp(-a); branch-free: the clamp keeps 2^x finite, and beyond it
// log2(1 + 2^x) = x to fp32 accuracy.
__device__ __forceinline__ float log2_sigmoid(float a) {
  const float x = -a * 1.4426950408889634f;
  return -fmaxf(x, lg2f(1.f + ex2f(fminf(x, 126.f))));
}

// Bounded wait that also gives up as soon as another role has raised the abort flag.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  const int batch = limit < 1000000LL ? 1 : 256;  // polls between two looks at the clock (a short limit is looked at often)
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < batch; ++i)
      if (mbar_try_wait(bar, parity)) return true;
#ifdef LAWCAT_TIMELINE
    // (profiling builds) when a wait runs out, every warp of one block notes the barrier it is waiting for: entry 0 of the
    // time line counts the notes, each note = barrier index | parity << 8 | thread << 16 | kind << 40
    if ((*abort_flag || clock64() - t0 > limit) && blockIdx.x == LAWCAT_TL_BLOCK && (threadIdx.x & 31) == 0) {
      const unsigned long long i = atomicAdd(reinterpret_cast<unsigned long long*>(&g_timeline[0]), 1ull);
      if (i < 40) g_timeline[1 + i] = (long long)(((bar & 1023u) - (OFF_BAR & 1023u)) / 8u) | ((long long)parity << 8) | ((long long)threadIdx.x << 16) | (1ll << 40);
    }
#endif
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      return false;
    }
  }
}

// Warp-collective bounded wait on a SET of mbarriers: lane l polls barrier l of the set, so the whole set costs one
// round of polling. (A wait that is already satisfied still takes a few hundred cycles of latency here, and waits issued
// one after the other add up on the critical path of a chunk.) `mask` selects the barriers, bit l of `parities` is the
// parity barrier l is waited with. All 32 lanes must call it together. A lane stops polling once its barrier's phase has
// completed: the barrier may run on into its next phase while the other lanes still wait.
__device__ __forceinline__ bool wait_set_or_abort(uint32_t bar0, uint32_t mask, uint32_t parities, int lane,
                                                  volatile int* abort_flag, long long limit) {
  const uint32_t b = bar0 + 8u * (uint32_t)lane, par = (parities >> lane) & 1u;
  bool ok = ((mask >> lane) & 1u) == 0u || mbar_try_wait(b, par);
  if (__all_sync(0xffffffffu, ok)) {
    __syncwarp();
    return true;
  }
  const long long t0 = clock64();
  const int batch = limit < 1000000LL ? 1 : 256;
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < batch; ++i) {
      if (!ok) ok = mbar_try_wait(b, par);
      if (__all_sync(0xffffffffu, ok)) {
        __syncwarp();
        return true;
      }
    }
    bool stop = *abort_flag != 0;
#ifdef LAWCAT_TIMELINE
    if ((stop || clock64() - t0 > limit) && !ok && blockIdx.x == LAWCAT_TL_BLOCK) {
      const unsigned long long i = atomicAdd(reinterpret_cast<unsigned long long*>(&g_timeline[0]), 1ull);
      if (i < 40) g_timeline[1 + i] = (long long)(((b & 1023u) - (OFF_BAR & 1023u)) / 8u) | ((long long)par << 8) | ((long long)threadIdx.x << 16) | (2ll << 40);
    }
#endif
    if (!stop && clock64() - t0 > limit) {
      *abort_flag = 1;
      stop = true;
    }
    if (__any_sync(0xffffffffu, stop)) return false;
  }
}

// MODE 0: the layer forward. MODE 1: state only (no query stream, no output): the end state of a segment that starts
// from the given state, used to hand the state across segments of one sequence.
// WIDTH: 0 = heads of 128 channels; 1 = one head of 64 channels per block (padded to 128); 2 = two 64-wide heads of one
// key/value group per block. A compile-time switch, so that the 128-wide kernel carries none of the others' tests.
template <int MODE, int WIDTH>
__global__ void __launch_bounds__(THREADS, 1)
layer_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_g, const TcArgs a) {
  extern __shared__ __align__(1024) uint8_t sg[];
  const uint32_t sb = smem_u32(sg);
  volatile int* const s_flags = reinterpret_cast<volatile int*>(sg + OFF_BAR + 8 * NUM_BARS);  // [0] tmem base, [1] abort
  // Range tracking, all as bits of non-negative floats. Per chunk parity: largest |x| of the chunk (rmax), largest |v|
  // of the chunk (vmax), bound on the state entries the chunk's state pass converts (sbound); smax: largest |state
  // entry| seen by the running state pass.  |S_new| <= |S_old| + 64 max|v| because kh <= 1.
  int* const s_rmax = const_cast<int*>(s_flags) + 2;   // [2]
  int* const s_vmax = s_rmax + 2;                      // [2]
  int* const s_sbound = s_rmax + 4;                    // [2]
  int* const s_smax = s_rmax + 6;                      // [1]
  volatile int* const s_abort = s_flags + 1;
  auto bar = [&](int i) -> uint32_t { return sb + OFF_BAR + 8 * i; };
  auto vec = [&](int parity, int which) -> float* {  // which: 0 bm, 1 ft, 2 e63
    return reinterpret_cast<float*>(sg + OFF_VEC + parity * 1536 + which * 512);
  };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // WIDTH 0: heads of 128 channels. WIDTH 1 (narrow): one head of 64 channels, run as a 128-wide one whose upper 64
  // channels are zero. WIDTH 2 (pair): two 64-wide heads of one key/value group side by side -- channels 0-63 belong to head
  // 2 h, channels 64-127 to head 2 h + 1; q, gate and o of the two are contiguous in memory and are addressed as one head
  // of 128 channels, the shared k is loaded into both halves, W is block-diagonal, and everything that contracts over the
  // channels (scores, read-out) is issued per half into accumulators of its own.
  constexpr bool narrow = WIDTH == 1, pair = WIDTH == 2, wide = WIDTH == 0;
  constexpr int dh = narrow ? 64 : 128, nslab = dh >> 6;  // width of the q / gate / o tiles as addressed, and their slabs
  constexpr int hd = wide ? 128 : 64, vslab = hd >> 6;    // width of a real head: of k and v as stored, of the state's value side
  // tensor memory columns (the pair keeps two read-out and two score accumulators where the state needs half the columns)
  constexpr uint32_t cS = COL_S, cSZ = pair ? 192u : COL_SZ, cO = pair ? 208u : COL_O, cO2 = 288u;
  constexpr uint32_t cP = pair ? 368u : COL_P, cP2 = 432u, cMAIL = pair ? 496u : COL_MAIL;
  const int sub = blockIdx.x % a.nsub;
  const int seg = (blockIdx.x / a.nsub) % a.grid_nseg;
  const int bh = blockIdx.x / (a.nsub * a.grid_nseg);
  const int Hn = pair ? a.H / 2 : a.H;   // heads as addressed (units of dh channels)
  const int h = bh % Hn, b = bh / Hn;
  const int h0 = pair ? 2 * h : h;       // first real head of this block
  const int G = a.H / a.Hkv, j = h0 / G;
  const int cps = a.seg_len / C;  // chunks per segment; piece `sub` covers chunks [sub cps / nsub, (sub + 1) cps / nsub)
  const int t_begin = min(a.T, seg * a.seg_len + (sub * cps / a.nsub) * C);
  const int t_end = min(a.T, seg * a.seg_len + ((sub + 1) * cps / a.nsub) * C);
  const int nchunks = max(0, (t_end - t_begin + C - 1) / C);
  // index of the state of the real head that owns state row c (rows 64-127 of a pair: the second head)
  auto state_idx = [&](int c, int per_segment) -> size_t {
    const size_t hr = (size_t)b * a.H + h0 + (pair ? (c >> 6) : 0);
    return per_segment ? (hr * a.nseg + seg) * a.nsub + sub : hr;
  };

  if ((sb & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base
    if (tid == 0 && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_CUDA);
    return;
  }

  // ---- one-time setup --------------------------------------------------------------------------------------------
  if (MODE == 1) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // (the scan may be scheduled behind)
  if (tid == 0) {
    const int nphi = MODE == 0 ? 256 : 128;  // threads of the phi pass: all row threads, or the key rows only
    mbar_init(bar(B_RAW_FULL), 1);
    mbar_init(bar(B_G_FULL), 1);
    mbar_init(bar(B_V_FULL), 1);
    mbar_init(bar(B_G_FREE), PREP_THREADS);
    mbar_init(bar(B_U_FULL), PREP_THREADS);
    mbar_init(bar(B_X_FULL), PREP_THREADS);
    mbar_init(bar(B_VH_FULL), PREP_THREADS);
    mbar_init(bar(B_MMA1), 1);
    mbar_init(bar(B_Y_FREE), nphi);
    mbar_init(bar(B_X_FREE), 256);  // every row thread: it reads bm, ft and (phi threads) the exponents
    mbar_init(bar(B_QK_FULL), nphi);
    mbar_init(bar(B_SBF_FULL), 256);
    mbar_init(bar(B_P), 1);
    mbar_init(bar(B_MMA2), 1);
    mbar_init(bar(B_PH_FULL), 128);
    mbar_init(bar(B_MMA3), 1);
    mbar_init(bar(B_O_FREE), 128);
    mbar_fence_init();
    s_flags[1] = 0;
    for (int i = 0; i < 7; ++i) s_rmax[i] = 0;
    tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_g);
  }
  if (warp == MMA_WARP) {
    tmem_alloc(sb + OFF_BAR + 8 * NUM_BARS, TMEM_COLS);
    tmem_relinquish();
  }
  // W_h^T into its K-major slabs as fp16: row e holds W[h][c][e] over c
  // (pair: block-diagonal, W of head 2 h in the upper left 64 x 64 block, W of head 2 h + 1 in the lower right)
  {
    const bf16* Wh = a.W + (size_t)h0 * hd * hd;
#pragma unroll 1
    for (int idx = tid; idx < 16 * D; idx += THREADS) {
      const int e = idx & (D - 1), oc = idx >> 7;
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      if (pair) {
        if ((e >> 6) == (oc >> 3)) {
          const bf16* Wp = Wh + (size_t)(oc >> 3) * hd * hd;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            w[i] = pack_f16(__bfloat162float(Wp[(size_t)((oc & 7) * 8 + 2 * i) * hd + (e & 63)]),
                            __bfloat162float(Wp[(size_t)((oc & 7) * 8 + 2 * i + 1) * hd + (e & 63)]));
        }
      } else if (e < dh && oc * 8 < dh) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          w[i] = pack_f16(__bfloat162float(Wh[(size_t)(oc * 8 + 2 * i) * dh + e]),
                          __bfloat162float(Wh[(size_t)(oc * 8 + 2 * i + 1) * dh + e]));
      }
      sts128(sb + OFF_W + (oc >> 3) * 16384 + sw128(e, oc & 7), make_uint4(w[0], w[1], w[2], w[3]));
    }
  }
  // a 64-wide head: the products run over the first 64 channels / columns only (K = 64, N = 64), so the second slabs of
  // the tiles are never read; the one exception is the kh operand of the state update, whose M = 128 rows are the key
  // channels: its second slab is zeroed here and never written
  if (narrow)
    for (int i = tid; i < 8192 / 16; i += THREADS) reinterpret_cast<uint4*>(sg + OFF_KH + 8192)[i] = make_uint4(0u, 0u, 0u, 0u);
  // constant "ones" operand and the zeroed column blocks of the state operand that carry z (unswizzled 8x8 core matrices)
  for (int i = tid; i < 2048 / 4; i += THREADS) reinterpret_cast<uint32_t*>(sg + OFF_ONES)[i] = 0u;
  for (int i = tid; i < 4096 / 4; i += THREADS) reinterpret_cast<uint32_t*>(sg + OFF_SBF + (hd >> 3) * 2048)[i] = 0u;
  // raw rows in front of the segment: earlier tokens, or the conv cache, or zeros (Section 4.1)
  if (tid < 96) {
    const int st = tid / 48, r = (tid % 48) / 16, oc = tid % 16;
    // row stride and offset of this block's channels in the stream as stored (pair: the key stream's 64 channels serve
    // both halves of the tile)
    const size_t rstride = st ? (size_t)a.Hkv * hd : (size_t)Hn * dh;
    const size_t coff = (st ? (size_t)j * hd : (size_t)h * dh) + (size_t)((st && pair) ? (oc & 7) : oc) * 8;
    const int t = t_begin - HALO + r;  // token of halo row r
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (oc * 8 >= dh) {
      // padded channels: zero
    } else if (t >= 0) {
      v = *reinterpret_cast<const uint4*>((st ? a.k : a.q) + ((size_t)b * a.T + t) * rstride + coff);
    } else {
      const bf16* cache = st ? a.cache_k : a.cache_q;
      const int ci = t + (a.K - 1);  // the cache holds tokens -(K-1) .. -1, oldest first
      if (cache && ci >= 0) v = *reinterpret_cast<const uint4*>(cache + ((size_t)b * (a.K - 1) + ci) * rstride + coff);
    }
    *reinterpret_cast<uint4*>(sg + OFF_HALO + ((st * 3 + r) * 16 + oc) * 16) = v;
  }
  __syncthreads();
  // conv caches after the last token (Section 4.1: the last K - 1 raw rows of [cache_in, x]): they depend on the raw
  // inputs alone, so the block of a head's last segment writes them here (the key stream by the first head of a group)
  if (MODE == 0 && seg == a.nseg - 1 && sub == 0 && a.K > 1 && tid < PREP_THREADS) {
    const int per = (a.K - 1) * (dh / 8);  // 16-byte units per stream (the key stream of a pair uses the first hd / 8 per row)
    for (int idx = tid; idx < 2 * per; idx += PREP_THREADS) {
      const int st = idx / per, r = (idx % per) / (dh / 8), oc = idx % (dh / 8);
      bf16* dst = st ? a.cache_k_out : a.cache_q_out;
      if (dst == nullptr || (st == 1 && (h0 % G != 0 || oc * 8 >= hd))) continue;
      const size_t rstride = st ? (size_t)a.Hkv * hd : (size_t)Hn * dh;
      const size_t coff = (st ? (size_t)j * hd : (size_t)h * dh) + (size_t)oc * 8;
      const int tok = a.T - (a.K - 1) + r;
      const bf16* x = st ? a.k : a.q;
      const bf16* cin = st ? a.cache_k : a.cache_q;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (tok >= 0) v = *reinterpret_cast<const uint4*>(x + ((size_t)b * a.T + tok) * rstride + coff);
      else if (cin != nullptr) v = *reinterpret_cast<const uint4*>(cin + ((size_t)b * (a.K - 1) + tok + a.K - 1) * rstride + coff);
      *reinterpret_cast<uint4*>(dst + ((size_t)b * (a.K - 1) + r) * rstride + coff) = v;
    }
  }
  if (tid < C) *reinterpret_cast<__half*>(sg + OFF_ONES + (tid >> 3) * 128 + (tid & 7) * 16) = __float2half(1.f);
  fence_proxy_async();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = (uint32_t)s_flags[0];
  const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);

  // Launched with programmatic stream serialization: the set-up above may run beside the tail of the kernel in front
  // (the scan over the segments, whose results are the start states read next); from here on that kernel has completed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // initial state into tensor memory: row thread (c, half) owns 64 columns of row c of [S | z]
  if (warp >= ROW_WARP0 && warp < ROW_WARP0 + 8) {
    // (pair: the state is [128 key channels x 64 value columns], the thread owns 32 columns; rows 64-127 are the second head)
    const int tw = tid - ROW_WARP0 * 32, c = tw & 127, chh = tw >> 7;
    const bool have = a.S0 != nullptr && (a.seg_in || seg == 0);
    const size_t in_idx = state_idx(c, a.seg_in);
    const int cr = c & (hd - 1);  // row inside the real head's state
    float s[32], mx = 0.f;
#pragma unroll 1
    for (int b2 = 0; b2 < (pair ? 1 : 2); ++b2) {
      const int blk = pair ? chh : chh * 2 + b2;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        s[i] = (have && c < dh && blk * 32 < hd) ? a.S0[(in_idx * hd + cr) * hd + blk * 32 + i] : 0.f;
        mx = fmaxf(mx, fabsf(s[i]));
      }
      tmem_st32(lane_base + cS + blk * 32, s);
    }
    if (chh == 1) {
      const bool havez = a.z0 != nullptr && (a.seg_in || seg == 0);
      const float z0v = (havez && c < dh) ? a.z0[in_idx * hd + cr] : 0.f;
      tmem_st1(lane_base + cSZ, z0v);
      mx = fmaxf(mx, fabsf(z0v));
    }
    tmem_wait_st();
    if (!(mx < 3.0e38f)) mx = 3.0e38f;  // NaN or inf in the given state: no fp16 operand
    atomicMax(s_sbound, __float_as_int(mx));
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();

#define WAIT(b, par)                                     \
  if (!wait_or_abort(bar(b), (uint32_t)(par), s_abort, a.wait_limit)) break
  // for roles with barriers of their own: remember the failure, skip the work, leave at the role's next OR-barrier
#define WAITF(b, par)                                    \
  if (!fail && !wait_or_abort(bar(b), (uint32_t)(par), s_abort, a.wait_limit)) fail = true
  // several barriers at once (whole warp): BIT(barrier) selects, PAR(barrier, parity) gives its parity
#define BIT(b) (1u << (b))
#define PAR(b, par) ((uint32_t)(par) << (b))
#define WAITSET(mask, pars)                              \
  if (!wait_set_or_abort(bar(0), (mask), (pars), lane, s_abort, a.wait_limit)) break
#define WAITSETF(mask, pars)                             \
  if (!fail && !wait_set_or_abort(bar(0), (mask), (pars), lane, s_abort, a.wait_limit)) fail = true

  if (warp == TMA_WARP) {
    // ================================================================================================ TMA producer
    if (lane == 0) {
      int ar_raw = -1, ar_g = -1, ar_v = -1;  // last chunk whose copies were started, per tile
      for (int n = 0; n < nchunks; ++n) {
        const int t0 = t_begin + n * C;
        const uint32_t pp = (uint32_t)((n - 1) & 1);
        if (n > 0) WAIT(B_MMA1, pp);  // MMA 1 of the previous chunk has read the in-place conv output
        mbar_arrive_expect_tx(bar(B_RAW_FULL), (MODE == 0 ? 16384u : 8192u) * (uint32_t)nslab);
#pragma unroll 1
        for (int s = 0; s < nslab; ++s) {
          if (MODE == 0) tma_load_4d(sb + OFF_AU + s * 16384, &tm_q, bar(B_RAW_FULL), s * 64, h, t0, b);
          // (pair: the same 64 key channels into both halves of the tile)
          tma_load_4d(sb + OFF_AU + s * 16384 + 8192, &tm_k, bar(B_RAW_FULL), pair ? 0 : s * 64, j, t0, b);
        }
        ar_raw = n;
        if (a.gate_dim != 1) {
          if (n > 0) WAIT(B_G_FREE, pp);
          mbar_arrive_expect_tx(bar(B_G_FULL), 8192u * (uint32_t)nslab);
          tma_load_4d(sb + OFF_G, &tm_g, bar(B_G_FULL), 0, h, t0, b);
          if (nslab == 2) tma_load_4d(sb + OFF_G + 8192, &tm_g, bar(B_G_FULL), 64, h, t0, b);
          ar_g = n;
        }
        if (n > 0) WAIT(MODE == 0 ? B_MMA3 : B_MMA2, pp);  // the last MMA that reads v
        mbar_arrive_expect_tx(bar(B_V_FULL), 8192u * (uint32_t)vslab);
        tma_load_4d(sb + OFF_V, &tm_v, bar(B_V_FULL), 0, j, t0, b);
        if (vslab == 2) tma_load_4d(sb + OFF_V + 8192, &tm_v, bar(B_V_FULL), 64, j, t0, b);
        ar_v = n;
      }
      if (*s_abort) {
        // leaving early: give the copies that are still in flight a bounded time to land before the CTA exits
        if (ar_raw >= 0) mbar_wait(bar(B_RAW_FULL), (uint32_t)(ar_raw & 1));
        if (ar_g >= 0) mbar_wait(bar(B_G_FULL), (uint32_t)(ar_g & 1));
        if (ar_v >= 0) mbar_wait(bar(B_V_FULL), (uint32_t)(ar_v & 1));
      }
    }
  } else if (warp == MMA_WARP) {
    // ================================================================================================ MMA issuer
    // The whole warp walks the loop and waits (one lane per barrier of a set); lane 0 issues.
    {
      // shared-memory descriptors of the operands (all tiles sit at fixed addresses); a K step adds a constant to the
      // start-address field (units of 16 bytes): K-major operand 32 B per step and 16 KB to the second 64-column slab;
      // MN-major swizzled operand 2048 B per step; unswizzled [rows x 16] operand 256 B per step
      const uint64_t dsc_u = smem_desc(sb + OFF_AU, 16, 1024, LAYOUT_SW128);
      const uint64_t dsc_w = smem_desc(sb + OFF_W, 16, 1024, LAYOUT_SW128);
      const uint64_t dsc_qk = smem_desc(sb + OFF_QK, 16, 1024, LAYOUT_SW128);
      const uint64_t dsc_ks = smem_desc(sb + OFF_QK + 8192, 16, 1024, LAYOUT_SW128);  // rows 64-127
      const uint64_t dsc_s = smem_desc(sb + OFF_SBF, 128, 2048, LAYOUT_NONE);  // [S | z]: one operand
      const uint64_t dsc_kh = smem_desc(sb + OFF_KH, 8192, 1024, LAYOUT_SW128);
      const uint64_t dsc_v = smem_desc(sb + OFF_V, 8192, 1024, LAYOUT_SW128);
      const uint64_t dsc_one = smem_desc(sb + OFF_ONES, 128, 1024, LAYOUT_NONE);
      const uint64_t dsc_p = smem_desc(sb + OFF_PH, 16, 1024, LAYOUT_SW128);
      // (pair: the masked scores of the second head; see OFF_PH2)
      const uint64_t dsc_p2 = smem_desc(sb + OFF_PH2, 16, 1024, LAYOUT_SW128);
      // only the 14-bit start-address field (bits 0-13) moves, and it cannot carry: a 32-bit add on the low word
      auto adv = [](uint64_t d, uint32_t off16) -> uint64_t {
        return (d & 0xFFFFFFFF00000000ull) | (uint64_t)((uint32_t)d + off16);
      };
      auto kstep = [](int k) -> uint32_t { return (uint32_t)((k >> 2) * (16384 >> 4) + (k & 3) * 2); };
      // (a 64-wide head: 4 instead of 8 K steps over the channels, 64 instead of 128 output columns)
      const int ksteps = narrow ? 4 : 8, NW = narrow ? 64 : 128;  // (the mix: channels contracted, output columns)
      constexpr int NV = hd;  // value columns of the state and of the read-out
      auto issue_mma1 = [&]() {
        const uint32_t ID = instr_desc(128, NW, FMT_F16, MAJOR_K, MAJOR_K);
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (k < ksteps) mma_f16(tmem + COL_Y, adv(dsc_u, kstep(k)), adv(dsc_w, kstep(k)), ID, k > 0);
        mma_commit(bar(B_MMA1));
      };
      bool ok = nchunks > 0;
      if (ok) ok = wait_set_or_abort(bar(0), BIT(B_U_FULL), 0u, lane, s_abort, a.wait_limit);
      if (ok && lane == 0) {
        tc_fence_after_sync();
        issue_mma1();
      }
      for (int n = 0; ok && n < nchunks; ++n) {
        const uint32_t p = (uint32_t)(n & 1), pp = p ^ 1u;
        WAITSET(BIT(B_QK_FULL) | BIT(B_SBF_FULL) | BIT(B_VH_FULL) | (MODE == 0 && n > 0 ? BIT(B_O_FREE) : 0u),
                PAR(B_QK_FULL, p) | PAR(B_SBF_FULL, p) | PAR(B_VH_FULL, p) | PAR(B_O_FREE, pp));
        TL(0, 0, n, lane == 0);
        const bool f16 = __int_as_float(s_rmax[p]) <= RMAX_F16 && __int_as_float(s_sbound[p]) < SMAX_F16;
        const int fmt = f16 ? FMT_F16 : FMT_BF16;
        if (MODE == 0 && lane == 0) {
          // the scores first: their mask pass is the longest chain behind this hand-over
          tc_fence_after_sync();
          // (pair: channels 0-63 give the first head's scores, channels 64-127 the second head's, in accumulators of their own)
          const uint32_t ID_P = instr_desc(128, 64, fmt, MAJOR_K, MAJOR_K);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            if (k < ksteps)
              mma_f16(tmem + ((pair && k >= 4) ? cP2 : cP), adv(dsc_qk, kstep(k)), adv(dsc_ks, kstep(k)), ID_P,
                      pair ? (k & 3) > 0 : k > 0);
          mma_commit(bar(B_P));
        }
        TL(0, 1, n, lane == 0);
        if (n + 1 < nchunks) {
          // then the mix of the next chunk: its phi sweeps read Y while this chunk's read-out and state update execute
          WAITSET(BIT(B_U_FULL) | BIT(B_Y_FREE), PAR(B_U_FULL, pp) | PAR(B_Y_FREE, p));
          if (lane == 0) {
            tc_fence_after_sync();
            issue_mma1();
          }
        }
        TL(0, 2, n, lane == 0);
        if (lane == 0) {
          tc_fence_after_sync();
          if (MODE == 0) {
            // read-out O' | denominator = qs [2^b_mid S | 2^b_mid z] in one product per K step
            // (pair: the first head's read-out contracts channels 0-63 with state rows 0-63, the second head's the rest)
            const uint32_t ID_O = instr_desc(128, NV + 16, fmt, MAJOR_K, MAJOR_MN);
#pragma unroll
            for (int k = 0; k < 8; ++k)
              if (k < ksteps)
                mma_f16(tmem + ((pair && k >= 4) ? cO2 : cO), adv(dsc_qk, kstep(k)), adv(dsc_s, k * (256 >> 4)), ID_O,
                        pair ? (k & 3) > 0 : k > 0);
          }
          const uint32_t ID_S = instr_desc(128, NV, FMT_F16, MAJOR_MN, MAJOR_MN);
          constexpr uint32_t ID_SZ = instr_desc(128, 16, FMT_F16, MAJOR_MN, MAJOR_MN);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint64_t ad = adv(dsc_kh, k * (2048 >> 4));
            mma_f16(tmem + cS, ad, adv(dsc_v, k * (2048 >> 4)), ID_S, 1);
            mma_f16(tmem + cSZ, ad, adv(dsc_one, k * (256 >> 4)), ID_SZ, 1);
          }
          mma_commit(bar(B_MMA2));
        }
        TL(0, 3, n, lane == 0);
        if (MODE == 0) {
          WAITSET(BIT(B_PH_FULL), PAR(B_PH_FULL, p));
          TL(0, 4, n, lane == 0);
          if (lane == 0) {
            // O' += P v  (the scores' part of the denominator is summed by the mask pass)
            tc_fence_after_sync();
            const uint32_t ID_O = instr_desc(128, NV, FMT_F16, MAJOR_K, MAJOR_MN);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              mma_f16(tmem + cO, adv(dsc_p, k * 2), adv(dsc_v, k * (2048 >> 4)), ID_O, 1);
            if (pair) {
#pragma unroll
              for (int k = 0; k < 4; ++k)
                mma_f16(tmem + cO2, adv(dsc_p2, k * 2), adv(dsc_v, k * (2048 >> 4)), ID_O, 1);
            }
            mma_commit(bar(B_MMA3));
          }
          TL(0, 5, n, lane == 0);
        }
      }
    }
  } else if (warp < ROW_WARP0) {
    // ================================================================================================ prep warps
    // conv mapping: thread = (stream, channel octet, 8 consecutive tokens); gate mapping: thread = (channel, half chunk)
    const int cv_stream = tid >> 7, cv_oct = tid & 15, cv_rg = (tid >> 4) & 7;
    const bool cv_on = (MODE == 0 || cv_stream == 1) && cv_oct * 8 < dh;
    uint64_t cw[4][4];  // [channel pair][tap], packed pairs of fp32
    {
      const bf16* w = cv_stream ? a.w_k : a.w_q;
      // first channel of this thread's octet among the stream's taps (pair: both halves of the key tile are the same 64 channels)
      const size_t ch0 = cv_stream ? (size_t)j * hd + (size_t)(pair ? (cv_oct & 7) : cv_oct) * 8 : (size_t)h * dh + cv_oct * 8;
#pragma unroll
      for (int cp = 0; cp < 4; ++cp)
#pragma unroll
        for (int dl = 0; dl < 4; ++dl) {
          const size_t i0 = (ch0 + 2 * cp) * a.K + dl;
          cw[cp][dl] = (dl < a.K && cv_oct * 8 < dh) ? f2_pack(__bfloat162float(w[i0]), __bfloat162float(w[i0 + a.K]))
                                                    : f2_pack(0.f, 0.f);
        }
    }
    const uint32_t au = sb + OFF_AU + (cv_oct >> 3) * 16384;  // this thread's 64-channel slab
    const int cjc = cv_oct & 7, crow0 = cv_stream * 64 + cv_rg * 8;
    const int gc = tid & 127, ghalf = tid >> 7, gjc = (gc & 63) >> 3;
    // Output pass (threads of TMEM quadrants 0 and 1: 64 query rows x 2 column halves): o = O' / (denominator + eps),
    // Eq. 8, straight from tensor memory to global memory.
    auto warp_free_o = [&]() {
      tc_fence_before_sync();
      mbar_arrive(bar(B_O_FREE));
    };
    auto out_pass = [&](int m) {
      if ((warp & 3) >= 2) return;
      const int orow_i = (warp & 3) * 32 + lane, och = tid >> 7;
      if (och >= nslab) {  // 64-wide head: no such columns
        warp_free_o();
        return;
      }
      const int ot0 = t_begin + m * C;
      const int onvalid = min(C, t_end - ot0);
      tc_fence_after_sync();
      // (pair: column half = head; each head has its own read-out accumulator, denominator parts and dropped normalizer)
      const uint32_t ocol = pair ? (och ? cO2 : cO) : cO + och * 64;
      float den = tmem_ld1(lane_base + (pair ? ocol + hd : cO + dh));
      const float den_p0 = tmem_ld1(lane_base + cMAIL + 8 + 2 * (m & 1) + (pair ? och : 0));
      const float den_p1 = pair ? 0.f : tmem_ld1(lane_base + cMAIL + 8 + 2 * (m & 1) + 1);
      // The query features went in as exp(y - max), without their softmax normalizer: it cancels in Eq. 8 except next to
      // eps, which therefore gets scaled by it; without normalization the numerator is divided by it.
      float qs = 0.f;
      if (a.eps != 0.f || !a.normalize) {
        qs = tmem_ld1(lane_base + cMAIL + 4 * (m & 1) + (pair ? och : 0));
        if (wide) qs += tmem_ld1(lane_base + cMAIL + 4 * (m & 1) + 1);
      }
      tmem_wait_ld();
      den += den_p0 + den_p1;
      const float inv = 1.f / (a.normalize ? fmaf(a.eps, qs, den) : qs);
      bf16* orow = a.o + (((size_t)b * a.T + ot0 + orow_i) * Hn + h) * dh + och * 64;
      float y[32];
#pragma unroll 1
      for (int b2 = 0; b2 < 2; ++b2) {
        tmem_ld32(lane_base + ocol + b2 * 32, y);
        tmem_wait_ld();
        if (b2 == 1) {  // O' is in registers: the next chunk's products may overwrite it
          tc_fence_before_sync();
          mbar_arrive(bar(B_O_FREE));
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) y[i] *= inv;
        if (orow_i < onvalid && och * 64 < dh) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) *reinterpret_cast<uint4*>(orow + b2 * 32 + q4 * 8) = pack8(y + 8 * q4, false);
        }
      }
    };
    // One decay per head (gate_dim = 1): thread t < C reads the logit of token t of the chunk straight from global memory,
    // one chunk ahead, and the log-decays of the chunk go to the other threads through (the unused) gate tile.
    float* const s_g1 = reinterpret_cast<float*>(sg + OFF_G);
    auto gate1_load = [&](int m) -> float {
      const int t = t_begin + m * C + tid;
      return (a.gate_dim == 1 && tid < C && m < nchunks && t < t_end)
                 ? __bfloat162float(a.gate[((size_t)b * a.T + t) * a.H + h]) : 0.f;
    };
    float g1_next = gate1_load(0);
    bool fail = false;
    for (int n = 0; n < nchunks; ++n) {
      const uint32_t p = (uint32_t)(n & 1), pp = p ^ 1u;
      const int nvalid = min(C, t_end - (t_begin + n * C));
      // ---- conv, in place: the three rows in front of this thread's rows belong to another thread (or to the previous
      // chunk), so they are read before the barrier and every row is overwritten only after it ------------------------
      WAITF(B_RAW_FULL, p);
      TL(warp == 0 ? 3 : 4, 0, n, (warp == 0 || warp == 2) && lane == 0);
      uint64_t x1[4], x2[4], x3[4], x0[4];  // sliding window of raw rows, packed pairs of fp32
      if (cv_on && !fail) {
        if (cv_rg == 0) {
          const uint4* hl = reinterpret_cast<const uint4*>(sg + OFF_HALO) + cv_stream * 48 + cv_oct;
          unpack8p(hl[0], x3); unpack8p(hl[16], x2); unpack8p(hl[32], x1);
        } else {
          unpack8p(lds128(au + sw128(crow0 - 3, cjc)), x3);
          unpack8p(lds128(au + sw128(crow0 - 2, cjc)), x2);
          unpack8p(lds128(au + sw128(crow0 - 1, cjc)), x1);
        }
      }
      if (tid == 0) { s_rmax[p] = 0; s_vmax[p] = 0; }
      fail = named_bar_or(1, PREP_THREADS, fail);
      if (fail) break;
      if (cv_on) {
#pragma unroll 4
        for (int i = 0; i < 8; ++i) {
          const uint32_t ad = au + sw128(crow0 + i, cjc);
          unpack8p(lds128(ad), x0);
          uint64_t u[4];
#pragma unroll
          for (int cp = 0; cp < 4; ++cp)
            u[cp] = f2_fma(cw[cp][0], x0[cp], f2_fma(cw[cp][1], x1[cp], f2_fma(cw[cp][2], x2[cp], f2_mul(cw[cp][3], x3[cp]))));
          sts128(ad, pack8p(u, true));
#pragma unroll
          for (int cp = 0; cp < 4; ++cp) { x3[cp] = x2[cp]; x2[cp] = x1[cp]; x1[cp] = x0[cp]; }
        }
        if (cv_rg == 7) {  // the last three raw rows of the chunk are the next chunk's halo (bf16 values: exact repack)
          uint4* hl = reinterpret_cast<uint4*>(sg + OFF_HALO) + cv_stream * 48 + cv_oct;
          hl[0] = pack8p(x3, false); hl[16] = pack8p(x2, false); hl[32] = pack8p(x1, false);
        }
      }
      fence_proxy_async();
      named_bar_sync(1, PREP_THREADS);
      mbar_arrive(bar(B_U_FULL));
      TL(warp == 0 ? 3 : 4, 1, n, (warp == 0 || warp == 2) && lane == 0);

      // ---- gate: exponents x_t = b_t - b_mid, scanned outwards from MID ------------------------------------------------
      if (a.gate_dim != 1) WAITF(B_G_FULL, p);
      TL(warp == 0 ? 3 : 4, 2, n, (warp == 0 || warp == 2) && lane == 0);
      {
        const uint8_t* gcol = sg + OFF_G + (gc >> 6) * 8192 + (gc & 7) * 2;
        // x[t][c] fp32, 512-byte rows whose 16-byte chunks are XOR-swizzled with t & 7 (conflict-free for this
        // column-wise writer and for the row-wise readers of the phi pass)
        float* const xcol = reinterpret_cast<float*>(sg + OFF_X) + (gc & 3);
        auto putx = [&](int t, float x) { xcol[t * 128 + (((gc >> 2) ^ (t & 7)) << 2)] = x; };
        // log-decays of tokens [32 half, 32 half + 32): all evaluated before the serial scan. The mode and the ragged
        // tail are decided outside the loops: a branch around each special-function instruction costs more than it.
        float g[32];
        const float L2E = 1.4426950408889634f;
        const bool g_on = gc < dh;  // (warp-uniform) the upper channels of a 64-wide head have no gate and no exponents
        if (a.gate_dim == 1) {
          if (tid < C)
            s_g1[tid] = a.gate_mode == LAWCAT_GATE_LOGDECAY ? g1_next * L2E : log2_sigmoid(g1_next) * a.inv_tau;
          g1_next = gate1_load(n + 1);
          fail = named_bar_or(1, PREP_THREADS, fail);
          if (fail) break;
#pragma unroll
          for (int i = 0; i < 32; ++i) g[i] = s_g1[ghalf * 32 + i];
        } else if (!g_on) {
#pragma unroll
          for (int i = 0; i < 32; ++i) g[i] = 0.f;
        } else if (a.gate_mode == LAWCAT_GATE_LOGDECAY) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const uint32_t raw = *reinterpret_cast<const uint16_t*>(gcol + sw128(ghalf * 32 + i, gjc));
            g[i] = __uint_as_float(raw << 16) * L2E;
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const uint32_t raw = *reinterpret_cast<const uint16_t*>(gcol + sw128(ghalf * 32 + i, gjc));
            g[i] = log2_sigmoid(__uint_as_float(raw << 16)) * a.inv_tau;
          }
        }
        if (nvalid < C) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (ghalf * 32 + i >= nvalid) g[i] = 0.f;  // tokens past the end: no decay
        }

        // the exponent tile is free once the previous chunk's phi pass has read it; the log-decays above did not need it
        mbar_arrive(bar(B_G_FREE));
        TL(warp == 0 ? 3 : 4, 3, n, (warp == 0 || warp == 2) && lane == 0);
        if (n > 0) WAITF(B_X_FREE, pp);
        TL(warp == 0 ? 3 : 4, 4, n, (warp == 0 || warp == 2) && lane == 0);
        float acc = 0.f;
        if (!g_on) {
          // nothing: nobody reads these channels' exponents or sums
        } else if (ghalf) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            acc += g[i];
            putx(32 + i, fmaxf(acc, -120.f));
          }
          vec(p, 1)[gc] = acc;                           // ft = b_C - b_mid
          vec(p, 2)[gc] = ex2f(fmaxf(acc, -120.f));      // 2^ft
        } else {
          putx(MID, 0.f);
#pragma unroll
          for (int i = MID - 1; i >= 0; --i) {
            acc += g[i + 1];
            putx(i, fminf(-acc, 120.f));
          }
          vec(p, 0)[gc] = acc + g[0];                    // bm = b_mid
        }
        // exponents are clamped to +-120 so that no factor overflows or vanishes; a clamp is reported
        if (-acc > 120.f && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_NUMERIC);
        const float am = warp_max(-acc);
        if (lane == 0) atomicMax(&s_rmax[p], __float_as_int(am));  // g <= 0: the largest exponent magnitude
      }
      mbar_arrive(bar(B_X_FULL));
      TL(warp == 0 ? 3 : 4, 5, n, (warp == 0 || warp == 2) && lane == 0);

      // ---- output of the previous chunk (its last product completes about now; the v tile is loaded after it) -----------
      if (MODE == 0 && n > 0) {
        WAITF(B_MMA3, pp);
        TL(warp == 0 ? 3 : 4, 6, n, (warp == 0 || warp == 2) && lane == 0);
        if (!fail) out_pass(n - 1);
        TL(warp == 0 ? 3 : 4, 7, n, (warp == 0 || warp == 2) && lane == 0);
      }

      // ---- v: bf16 -> fp16 in place (exact for |v| in the fp16 normal range) ------------------------------------------
      WAITF(B_V_FULL, p);
      TL(warp == 0 ? 3 : 4, 8, n, (warp == 0 || warp == 2) && lane == 0);
      // (layer mode: by the warps of TMEM quadrants 2-3 only; those of quadrants 0-1 carry the output pass)
      if (!fail && (MODE == 1 || (warp & 3) >= 2)) {
        const int vthreads = MODE == 1 ? PREP_THREADS : PREP_THREADS / 2;
        const int vt = MODE == 1 ? tid : (tid >> 7) * 64 + ((warp & 3) - 2) * 32 + lane;
        float vm = 0.f;
#pragma unroll 4
        for (int i = 0; i < vslab * 512 / vthreads; ++i) {
          const uint32_t ad = sb + OFF_V + (uint32_t)(vt + vthreads * i) * 16;
          float x[8];
          unpack8(lds128(ad), x);
#pragma unroll
          for (int e = 0; e < 8; ++e) vm = fmaxf(vm, fabsf(x[e]));
          sts128(ad, pack8(x, true));
        }
        vm = warp_max(vm);
        if (lane == 0) atomicMax(&s_vmax[p], __float_as_int(vm < 3.0e38f ? vm : 3.0e38f));
      }
      fence_proxy_async();
      mbar_arrive(bar(B_VH_FULL));
      TL(warp == 0 ? 3 : 4, 9, n, (warp == 0 || warp == 2) && lane == 0);
    }
    if (MODE == 0 && nchunks > 0 && !fail && !*s_abort &&
        wait_or_abort(bar(B_MMA3), (uint32_t)((nchunks - 1) & 1), s_abort, a.wait_limit))
      out_pass(nchunks - 1);
  } else {
    // ================================================================================================ row warps
    // 8 warps, two per TMEM quadrant. Thread = (row, half of the columns): rows 0-63 are the query tokens, rows 64-127 the
    // key tokens of Y; the same threads own row c of [S | z] (state pass), and the query-row threads also mask the
    // scores. The two threads of a row share a TMEM lane and meet through two spare TMEM columns (row max, softmax sum).
    // Order inside a chunk: the sweeps of phi that only READ (row max; key rows: exp and its sum) run while the previous
    // chunk's MMA 2 is still executing; the state pass and the sweep that writes qs / ks / kh wait for it.
    const int tw = tid - ROW_WARP0 * 32;
    const int ch = tw >> 7;                       // column half: columns [64 ch, 64 ch + 64)
    const int r128 = (tw & 127);                  // row of Y and of the state (= TMEM lane)
    const bool is_q = r128 < C;
    const int row = is_q ? r128 : r128 - C;       // token inside the chunk
    const bool phi_on = MODE == 0 || !is_q;       // the state-only pass has no query rows
    const bool padded = ch >= nslab;              // this thread's 64 columns are the zero padding of a 64-wide head
    const int phi_bar = is_q ? 3 : 4;             // the query rows and the key rows meet among themselves (128 threads each)
    const float L2E = 1.4426950408889634f;
    // the dropped softmax normalizer of the query rows only matters next to eps, and without normalization
    const bool need_qsum = a.eps != 0.f || !a.normalize;
    const uint32_t mail_mine = lane_base + cMAIL + 2 + ch, mail_other = lane_base + cMAIL + 2 + (ch ^ 1);
    const uint32_t ycol = lane_base + COL_Y + ch * 64;
    float dsum = 0.f;  // log2 of this state row's total decay over the segment
    bool fail = false;
    // ---- causal mask of chunk m, fp16 scores: this (query-row) thread's 32 columns of row `row`. It runs behind the
    // reading sweeps of chunk m + 1, which do not have to wait for MMA 2 of chunk m.
    auto mask_chunk = [&](int m) {
      // (MMA 3 of the chunk before: the score tile was its operand)
      WAITSETF(BIT(B_P) | (m > 0 ? BIT(B_MMA3) : 0u), PAR(B_P, m & 1) | PAR(B_MMA3, (m - 1) & 1));
      if (fail) return;
      tc_fence_after_sync();
      // The chunk's own part of the denominator is the row sum of the masked scores AS ROUNDED to fp16: numerator and
      // denominator then carry the same weights (the first tokens of a sequence do not average a mismatch out).
      // (pair: this thread masks all 64 columns of its own head's scores, two blocks of 32, into that head's tile)
      float rs = 0.f;
#pragma unroll 1
      for (int hb = 0; hb < (pair ? 2 : 1); ++hb) {
        const int c32 = pair ? hb : ch;  // which block of 32 key tokens
        float s[32];
        tmem_ld32(lane_base + (pair ? (ch ? cP2 : cP) : cP) + c32 * 32, s);
        tmem_wait_ld();
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int col = c32 * 32 + q4 * 8 + 2 * i;
            const __half2 h2 = __floats2half2_rn(col <= row ? s[q4 * 8 + 2 * i] : 0.f, col + 1 <= row ? s[q4 * 8 + 2 * i + 1] : 0.f);
            const float2 f2 = __half22float2(h2);
            rs += f2.x + f2.y;
            w[i] = *reinterpret_cast<const uint32_t*>(&h2);
          }
          sts128(sb + ((pair && ch) ? OFF_PH2 : OFF_PH) + sw128(row, c32 * 4 + q4), make_uint4(w[0], w[1], w[2], w[3]));
        }
      }
      tmem_st1(lane_base + cMAIL + 8 + 2 * (m & 1) + ch, rs);
      tmem_wait_st();
      fence_proxy_async();
      tc_fence_before_sync();
      mbar_arrive(bar(B_PH_FULL));
    };
    for (int n = 0; n < nchunks; ++n) {
      const uint32_t p = (uint32_t)(n & 1), pp = p ^ 1u;
      const int nvalid = min(C, t_end - (t_begin + n * C));
      float y[32], ya[16], yb[16];
      float mb = 0.f, sum = 0.f;
      TL(warp == 8 ? 1 : 2, 0, n, (warp == 8 || warp == 10) && lane == 0);
      // ---- mask of the previous chunk: its scores are the first product issued after the hand-over, ahead of this
      // chunk's mix ---------------------------------------------------------------------------------------------------
      if (MODE == 0 && is_q && n > 0) mask_chunk(n - 1);
      TL(warp == 8 ? 1 : 2, 1, n, (warp == 8 || warp == 10) && lane == 0);
      // ---- phi, reading sweeps ----------------------------------------------------------------------------------------
      if (phi_on) {
        WAITF(B_MMA1, p);
        fail = __any_sync(0xffffffffu, fail);  // (the collective waits below need the whole warp)
        TL(warp == 8 ? 1 : 2, 2, n, (warp == 8 || warp == 10) && lane == 0);
        tc_fence_after_sync();
        float m = -INFINITY;
        // (64-wide head: the threads of the upper 64 columns have no outputs: they skip every sweep, and the two threads
        // of a row have nothing to exchange)
        if (!fail && !padded) {
          tmem_ld16(ycol, ya);  // 16 columns at a time, the next load in flight while a block is processed
#pragma unroll 1
          for (int b2 = 0; b2 < 2; ++b2) {
            tmem_wait_ld();
            tmem_ld16(ycol + b2 * 32 + 16, yb);
#pragma unroll
            for (int i = 0; i < 16; ++i) m = fmaxf(m, ya[i]);
            tmem_wait_ld();
            tmem_ld16(ycol + ((b2 * 32 + 32) & 63), ya);  // wraps to the first block: the next sweep starts there
#pragma unroll
            for (int i = 0; i < 16; ++i) m = fmaxf(m, yb[i]);
          }
        }
        if (wide) {  // (narrow, pair: a row's softmax lives in one thread's 64 columns)
          if (!fail) {
            tmem_st1(mail_mine, m);
            tmem_wait_st();
          }
          named_bar_sync(phi_bar, 128);
          if (!fail) {
            m = fmaxf(m, tmem_ld1(mail_other));  // (the load of `ya` issued above completes with this wait as well)
            tmem_wait_ld();
          }
        }
        mb = m * L2E;
        TL(warp == 8 ? 1 : 2, 3, n, (warp == 8 || warp == 10) && lane == 0);
        if (!is_q) {
          // key rows: e = exp(y - max) and its sum; e is parked in Y's own columns for the writing sweep
          if (!fail && !padded) {
#pragma unroll 1
            for (int b2 = 0; b2 < 2; ++b2) {
              tmem_wait_ld();
              tmem_ld16(ycol + b2 * 32 + 16, yb);
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                ya[i] = ex2f(fmaf(ya[i], L2E, -mb));
                sum += ya[i];
              }
              tmem_st16(ycol + b2 * 32, ya);
              tmem_wait_ld();
              if (b2 < 1) tmem_ld16(ycol + b2 * 32 + 32, ya);
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                yb[i] = ex2f(fmaf(yb[i], L2E, -mb));
                sum += yb[i];
              }
              tmem_st16(ycol + b2 * 32 + 16, yb);
            }
          }
          if (wide) {
            named_bar_sync(phi_bar, 128);  // the partner has read the row max out of the mailbox
            if (!fail) {
              tmem_st1(mail_mine, sum);
              tmem_wait_st();
            }
            named_bar_sync(phi_bar, 128);
            if (!fail) {
              sum += tmem_ld1(mail_other);
              tmem_wait_ld();
            }
          }
        }
      }
      // ---- the previous chunk's MMA 2 has completed: the state is updated; qs / ks / kh / state operand are free ---------
      TL(warp == 8 ? 1 : 2, 4, n, (warp == 8 || warp == 10) && lane == 0);
      WAITSETF(BIT(B_X_FULL) | (n > 0 ? BIT(B_MMA2) : 0u), PAR(B_X_FULL, p) | PAR(B_MMA2, pp));
      TL(warp == 8 ? 1 : 2, 5, n, (warp == 8 || warp == 10) && lane == 0);
      tc_fence_after_sync();
      const bool f16 = __int_as_float(s_rmax[p]) <= RMAX_F16 && __int_as_float(s_sbound[p]) < SMAX_F16;
      // (the 8-bit-mantissa operands keep the range but not the accuracy bound: the caller is told)
      if (MODE == 0 && !f16 && tw == 0 && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_NUMERIC);
      // ---- state pass: 16-bit operand 2^b_mid [S|z], accumulator [S|z] *= 2^b_C (this thread: 64 columns of row r128)
      // (64-wide head: only the rows and columns that exist)
      const bool s_on = !narrow || (!padded && r128 < dh);
      // The largest state entry (which decides between fp16 and bf16 operands) is measured every 8th chunk; in between
      // its bound grows by 64 max|v| per chunk (kh <= 1), a few thousand at most against the threshold of 3e4.
      const bool track = (n & 7) == 0;
      if (!fail && !s_on && !phi_on) mbar_arrive(bar(B_X_FREE));  // (see the end of the pass)
      if (!fail && s_on) {
        const int c = r128;
        const float bm = vec(p, 0)[c], ft = vec(p, 1)[c];
        const float dm = ex2f(bm), dC = ex2f(bm + ft);
        if (ch == 0) dsum += bm + ft;
        float mx = 0.f;
        // (pair: 64 value columns, 32 per thread)
#pragma unroll 1
        for (int b2 = 0; b2 < (pair ? 1 : 2); ++b2) {
          const int blk = pair ? ch : ch * 2 + b2;
          tmem_ld32(lane_base + cS + blk * 32, y);
          tmem_wait_ld();
          if (MODE == 0) {
            if (track) {
#pragma unroll
              for (int i = 0; i < 32; ++i) mx = fmaxf(mx, fabsf(y[i]));
            }
            const uint64_t dm2 = f2_pack(dm, dm);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              uint64_t w[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) w[i] = f2_mul(dm2, f2_pack(y[8 * q4 + 2 * i], y[8 * q4 + 2 * i + 1]));
              // columns [8 nb, 8 nb + 8) of row c: block nb of the unswizzled operand (a warp's 32 rows: 512 contiguous bytes)
              sts128(sb + OFF_SBF + (uint32_t)(blk * 4 + q4) * 2048u + (uint32_t)c * 16u, pack8p(w, f16));
            }
          }
          {
            const uint64_t dC2 = f2_pack(dC, dC);
#pragma unroll
            for (int i = 0; i < 32; i += 2) f2_unpack(f2_mul(dC2, f2_pack(y[i], y[i + 1])), y[i], y[i + 1]);
          }
          tmem_st32(lane_base + cS + blk * 32, y);
        }
        if (ch == (narrow ? 0 : 1)) {  // (the thread of the row's last existing column half also carries z)
          const float z = tmem_ld1(lane_base + cSZ);
          tmem_wait_ld();
          if (MODE == 0) {
            *reinterpret_cast<uint16_t*>(sg + OFF_SBF + (hd >> 3) * 2048 + c * 16) = to16(dm * z, f16);
            if (track) mx = fmaxf(mx, fabsf(z));
          }
          tmem_st1(lane_base + cSZ, dC * z);
        }
        if (MODE == 0 && track) {
          mx = warp_max(mx);
          if (lane == 0) atomicMax(s_smax, __float_as_int(mx < 3.0e38f ? mx : 3.0e38f));
        }
        tmem_wait_st();
        if (!phi_on) mbar_arrive(bar(B_X_FREE));  // (state-only pass) this thread has read bm, ft and reads no exponents
      }
      TL(warp == 8 ? 1 : 2, 6, n, (warp == 8 || warp == 10) && lane == 0);
      // ---- phi, writing sweep -------------------------------------------------------------------------------------------
      if (phi_on && !fail && !padded) {
        if (is_q) {
          float qsum = 0.f;
          auto q_block = [&](const float* yy, int jj0) {  // 16 columns = channel groups jj0, jj0 + 1
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
              const int jj = jj0 + h2;
              float x[8], v[8];
              load_x8(sb + OFF_X, row, jj, x);
#pragma unroll
              for (int i = 0; i < 8; ++i) v[i] = ex2f(fmaf(yy[h2 * 8 + i], L2E, x[i] - mb));
              if (need_qsum) {
#pragma unroll
                for (int i = 0; i < 8; ++i) qsum += ex2f(fmaf(yy[h2 * 8 + i], L2E, -mb));
              }
              sts128(sb + OFF_QK + ch * 16384 + sw128(row, jj & 7), pack8(v, f16));
            }
          };
          // (`ya` holds the first 16 columns since the row-max sweep)
#pragma unroll 1
          for (int b2 = 0; b2 < 2; ++b2) {
            tmem_wait_ld();
            tmem_ld16(ycol + b2 * 32 + 16, yb);
            q_block(ya, ch * 8 + b2 * 4);
            tmem_wait_ld();
            if (b2 < 1) tmem_ld16(ycol + b2 * 32 + 32, ya);
            q_block(yb, ch * 8 + b2 * 4 + 2);
          }
          if (need_qsum) {
            // the dropped normalizer travels to the output pass through tensor memory: each half adds its part
            tmem_st1(lane_base + cMAIL + 4 * p + ch, qsum);
            tmem_wait_st();
          }
        } else {
          const float inv = row < nvalid ? 1.f / sum : 0.f;  // tokens past the end contribute nothing
          const float* e63v = vec(p, 2);
          auto k_block = [&](const float* ee, int jj0) {  // 16 columns = channel groups jj0, jj0 + 1
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
              const int jj = jj0 + h2;  // channels [8 jj, 8 jj + 8)
              float x[8], ks[8];
              load_x8(sb + OFF_X, row, jj, x);
              const float4 ea = *reinterpret_cast<const float4*>(e63v + jj * 8);
              const float4 eb = *reinterpret_cast<const float4*>(e63v + jj * 8 + 4);
              const float e63[8] = {ea.x, ea.y, ea.z, ea.w, eb.x, eb.y, eb.z, eb.w};
#pragma unroll
              for (int i = 0; i < 8; ++i) ks[i] = ee[h2 * 8 + i] * inv * ex2f(-x[i]);
              if (MODE == 0) sts128(sb + OFF_QK + ch * 16384 + sw128(C + row, jj & 7), pack8(ks, f16));
#pragma unroll
              for (int i = 0; i < 8; ++i) ks[i] *= e63[i];
              // kh: row = token, MN-major A operand of the state update (slab = column half)
              sts128(sb + OFF_KH + ch * 8192 + sw128(row, jj & 7), pack8(ks, true));
            }
          };
          tmem_ld16(ycol, ya);
#pragma unroll 1
          for (int b2 = 0; b2 < 2; ++b2) {
            tmem_wait_ld();
            tmem_ld16(ycol + b2 * 32 + 16, yb);
            k_block(ya, ch * 8 + b2 * 4);
            tmem_wait_ld();
            if (b2 < 1) tmem_ld16(ycol + b2 * 32 + 32, ya);
            k_block(yb, ch * 8 + b2 * 4 + 2);
          }
        }
      }
      // ---- hand-over to MMA 2: state operand, qs / ks / kh, and the bound on the state for the next chunk ------------
      TL(warp == 8 ? 1 : 2, 7, n, (warp == 8 || warp == 10) && lane == 0);
      WAITF(B_VH_FULL, p);  // the chunk's max|v| is known
      TL(warp == 8 ? 1 : 2, 8, n, (warp == 8 || warp == 10) && lane == 0);
      fence_proxy_async();
      tc_fence_before_sync();
      fail = named_bar_or(2, 256, fail);
      TL(warp == 8 ? 1 : 2, 9, n, (warp == 8 || warp == 10) && lane == 0);
      if (fail) break;
      if (MODE == 0 && tw == 0) {
        // |S_new| <= |S_old| + 64 max|v|: the next chunk's choice of operand type
        s_sbound[pp] = __float_as_int(__int_as_float(track ? *s_smax : s_sbound[p]) + 64.f * fmaxf(__int_as_float(s_vmax[p]), 1.f));
        *s_smax = 0;
        __threadfence_block();
      }
      mbar_arrive(bar(B_SBF_FULL));
      if (phi_on) {
        mbar_arrive(bar(B_Y_FREE));
        mbar_arrive(bar(B_X_FREE));
        mbar_arrive(bar(B_QK_FULL));
      }
    }
    if (MODE == 0 && is_q && nchunks > 0) mask_chunk(nchunks - 1);
    // ---- final state -------------------------------------------------------------------------------------------------
    if (!fail && !*s_abort && (nchunks == 0 || wait_or_abort(bar(B_MMA2), (uint32_t)((nchunks - 1) & 1), s_abort, a.wait_limit))) {
      tc_fence_after_sync();
      const int c = r128, cr = c & (hd - 1);  // state row, and the row inside its real head's state
      const size_t out_idx = state_idx(c, a.seg_out);
      if (a.dtot != nullptr && ch == 0 && c < dh) a.dtot[state_idx(c, 1) * hd + cr] = dsum;
      const bool last = a.seg_out || seg == a.nseg - 1;  // (each of the two outputs is optional on its own)
      if (a.S_T != nullptr && last) {
        float s[32];
#pragma unroll 1
        for (int b2 = 0; b2 < (pair ? 1 : 2); ++b2) {
          const int blk = pair ? ch : ch * 2 + b2;
          tmem_ld32(lane_base + cS + blk * 32, s);
          tmem_wait_ld();
          if (c < dh && blk * 32 < hd) {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<float4*>(a.S_T + (out_idx * hd + cr) * hd + blk * 32 + i) = make_float4(s[i], s[i + 1], s[i + 2], s[i + 3]);
          }
        }
      }
      if (a.z_T != nullptr && last && ch == 1) {
        const float z = tmem_ld1(lane_base + cSZ);
        tmem_wait_ld();
        if (c < dh) a.z_T[out_idx * hd + cr] = z;
      }
    }
  }
#undef WAIT
#undef WAITF
#undef WAITSET
#undef WAITSETF
#undef BIT
#undef PAR

  // ---- teardown --------------------------------------------------------------------------------------------------------
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0 && *s_abort && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_TIMEOUT);
  if (warp == MMA_WARP) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

}  // namespace tc
}  // namespace lawcat
