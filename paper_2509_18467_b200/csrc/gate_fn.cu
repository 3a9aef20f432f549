// The gate function in front of the layer (Section 4.2: additional linear layers whose output goes through a sigmoid;
// appendix, ablation on the rank of the gate function: two consecutive low-rank linear layers of rank 16 ... 128):
//   logits a_t = A2 (A1 x_t) + bias,   x [N, d_model] (N = B T tokens), A1 [rank, d_model], A2 [n_out, rank], bias [n_out],
// written as the [B, T, H, gate_dim] gate tensor the layer consumes (n_out = H * gate_dim); the sigmoid and the power
// 1 / tau are applied where the logits are read.
//
// Tensor-core kernel (bf16 storage, rank 16 / 32 / 64 / 128): one thread block per 128 tokens, three roles (10 warps).
//   copy warp      first layer: x tiles [128 tokens x 64 hidden channels] and A1 tiles [rank x 64] through a ring of
//                  stages (TMA, 128-byte swizzle)
//   product warp   H = X A1^T accumulated over d_model in tensor memory (M = 128, N = rank); then per 128 outputs
//                  OUT = [H_hi | H_lo] [A2 | A2]^T (M = 128, N = 128) into one of two accumulators
//   2 x 4 epilogue A2 tiles [128 outputs x rank] from L2 into the operand layout, two tiles ahead of the products (rows
//     warps        of 2 * rank bytes are too short for efficient TMA boxes; the loads of a tile are issued before the
//                  epilogue of the tile two earlier and stored behind it);
//                  H: tensor memory -> two-term bf16 (hi + lo, 16 significant bits) -> shared-memory operand;
//                  OUT: tensor memory -> + bias -> bf16 -> swizzled staging tile -> TMA store (clipped at the tensor's edge).
//                  Two groups of four warps take the output tiles in turn, each with an accumulator, an A2 buffer and a
//                  staging tile of its own: a tile's chain of waits (product, tensor-memory load, store) is long compared
//                  with its arithmetic, and two chains side by side hide most of it.
// x and the logits cross HBM once each (the roofline of the kernel); A1 and A2 are re-read from L2 by every block.
// The buffers of the second layer alias the ring of the first (which is drained by then) except the A2 tiles, so that
// the first two of those are in place while the first layer runs.
// Every wait is bounded: a wait that runs out raises the block's abort flag, every role leaves its loop, the block lets
// its copies land, frees its tensor memory and reports LAWCAT_ERR_TIMEOUT through dev_status.
//
// Few tokens (a decode step, a short call; bf16, widths multiples of 8): one block of the tensor-core kernel walks its
// 64 stages and 32 output tiles one after the other, about 50 us whatever the number of tokens. Up to 1024 tokens
// gate_fn_small_kernel takes over: one thread block per token (or per four), both layers on the CUDA cores in fp32 with
// the bottleneck activations in shared memory, every load a 16-byte one and many in flight; the weights come from L2.
// Above that, while there are fewer token tiles than the SMs hold blocks, the output tiles of a token tile are shared out
// over several blocks (gridDim.y), each of which repeats the first layer.
//
// Exact kernels (any storage type and shape): fp32 accumulation on the CUDA cores, h in fp32 scratch.
#include <cuda.h>

#include <algorithm>
#include <atomic>

#include "common.cuh"
#include "octet_tile.cuh"
#include "tc_common.cuh"

namespace lawcat {

namespace gfn {

using namespace tc;
using ctc::dadv;
using ctc::kview;
using ctc::toff;

constexpr int TT = 128;        // tokens per thread block
constexpr int NT = 128;        // outputs per product of the second layer
constexpr int KS = 64;         // hidden channels per stage of the first layer
constexpr int THREADS = 320;   // warp 0 copies, warp 1 products, warps 2-5 and 6-9 epilogue groups (TMEM quadrant = warp & 3)
constexpr int EPI_THREADS = 128;  // per group
constexpr uint32_t TMEM_COLS = 256;  // accumulator 0 = columns 0-127 (H uses its first `rank` columns first), 1 = 128-255
constexpr long long WAIT_LIMIT = 400000000LL;  // clock cycles (about a fifth of a second)

template <int R>
struct Lay {
  static constexpr int ST = R == 128 ? 3 : 4;                       // stages of the first layer's ring
  static constexpr uint32_t X_BYTES = TT * 128;                     // [128 x 64] bf16, swizzled
  static constexpr uint32_t A1_BYTES = R * 128;                     // [R x 64] bf16, swizzled
  static constexpr uint32_t STAGE = X_BYTES + A1_BYTES;
  static constexpr uint32_t OUT_BYTES = TT * NT * 2;                // staging: 2 slabs of [128 x 128 B], swizzled
  static constexpr uint32_t SLAB_H = TT * 16 + 16;                  // H operand: octet slabs of 128 rows (padded)
  static constexpr uint32_t H_BYTES = (2 * R / 8) * SLAB_H;         // columns [0, R) hi, [R, 2R) lo
  static constexpr uint32_t SLAB_B = NT * 16 + 16;                  // A2 operand: octet slabs of 128 rows (padded)
  static constexpr uint32_t B_BYTES = (R / 8) * SLAB_B;
  static constexpr uint32_t OFF_RING = 0;
  static constexpr uint32_t OFF_OUT = 0;                            // (second layer: over the drained ring)
  static constexpr uint32_t OFF_H = 2 * OUT_BYTES;
  static constexpr uint32_t P2_BYTES = OFF_H + H_BYTES;
  static constexpr uint32_t RING_BYTES = ST * STAGE;
  static constexpr uint32_t OFF_B = ((P2_BYTES > RING_BYTES ? P2_BYTES : RING_BYTES) + 1023) / 1024 * 1024;
  static constexpr uint32_t OFF_BIAS = OFF_B + 2 * B_BYTES;         // fp32 [2][128]
  static constexpr uint32_t OFF_BAR = OFF_BIAS + 2 * NT * 4;
  static constexpr uint32_t BYTES = OFF_BAR + 256;
  static_assert(BYTES <= 232448, "shared memory budget");
};

// mbarriers
enum { B_FULL0 = 0, B_EMPTY0 = 4, B_HFULL = 8, B_HREADY, B_BFULL0, B_ACCFULL0 = B_BFULL0 + 2, B_ACCFREE0 = B_ACCFULL0 + 2,
       NUM_BARS = B_ACCFREE0 + 2 };

struct GArgs {
  const bf16* A2;     // [n_out, rank]
  const bf16* bias;   // [n_out] or null
  int N, dm, n_out;
  int* dev_status;
};

__device__ __forceinline__ bool gwait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > WAIT_LIMIT) {
      *abort_flag = 1;
      return false;
    }
  }
}

template <int R>
__global__ void __launch_bounds__(THREADS, R <= 32 ? 2 : 1)   // (rank <= 32: two blocks per SM, so at most 102 registers)
gate_fn_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_a1,
                  const __grid_constant__ CUtensorMap tm_out, const GArgs a) {
  using L = Lay<R>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sb = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bars = sb + L::OFF_BAR;
  volatile int* const s_flags = reinterpret_cast<volatile int*>(smem + L::OFF_BAR + 8 * NUM_BARS);  // [0] tmem base, [1] abort
  volatile int* const s_abort = s_flags + 1;
  float* const s_bias = reinterpret_cast<float*>(smem + L::OFF_BIAS);
  auto BAR = [&](int i) { return bars + 8u * (uint32_t)i; };
  const int n0 = blockIdx.x * TT;
  // With fewer token tiles than SMs the output tiles of a token tile are shared out over gridDim.y blocks (each repeats the
  // first layer, whose x tile then comes from L2): this block's tiles are nt0 ... nt0 + ntile - 1, `nt` below counts from 0.
  const int nk = (a.dm + KS - 1) / KS, ntile_all = (a.n_out + NT - 1) / NT;
  const int per_y = (ntile_all + (int)gridDim.y - 1) / (int)gridDim.y, nt0 = (int)blockIdx.y * per_y;
  const int ntile = min(per_y, ntile_all - nt0);

  if (tid == 0) {
    if (sb & 1023u) { s_flags[1] = 1; } else { s_flags[1] = 0; }
    for (int i = 0; i < NUM_BARS; ++i) {
      const bool many = i == B_HREADY || i == B_ACCFREE0 || i == B_ACCFREE0 + 1 || i == B_BFULL0 || i == B_BFULL0 + 1;
      mbar_init(BAR(i), many ? EPI_THREADS : 1);
    }
    mbar_fence_init();
    tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_a1); tma_prefetch_desc(&tm_out);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<int*>(s_flags)), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = (uint32_t)s_flags[0];

  if (warp == 0) {
    // ------------------------------------------------------------------------------------------------ copies
    if (lane == 0) {
      bool ok = true;
      for (int i = 0; i < nk && ok; ++i) {
        const int s = i % L::ST;
        if (i >= L::ST) ok = gwait(BAR(B_EMPTY0 + s), ((i / L::ST) - 1) & 1, s_abort);
        if (!ok) break;
        mbar_arrive_expect_tx(BAR(B_FULL0 + s), L::STAGE);
        tma_load_2d(sb + L::OFF_RING + s * L::STAGE, &tm_x, BAR(B_FULL0 + s), i * KS, n0);
        tma_load_2d(sb + L::OFF_RING + s * L::STAGE + L::X_BYTES, &tm_a1, BAR(B_FULL0 + s), i * KS, 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------------------------ products
    if (lane == 0) {
      constexpr uint32_t idesc1 = instr_desc(128, R, FMT_BF16, MAJOR_K, MAJOR_K);
      constexpr uint32_t idesc2 = instr_desc(128, NT, FMT_BF16, MAJOR_K, MAJOR_K);
      bool ok = true;
      for (int i = 0; i < nk && ok; ++i) {
        const int s = i % L::ST;
        ok = gwait(BAR(B_FULL0 + s), (i / L::ST) & 1, s_abort);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t xs = sb + L::OFF_RING + s * L::STAGE;
#pragma unroll
        for (int kk = 0; kk < KS / 16; ++kk)
          mma_f16(tmem, smem_desc(xs + kk * 32, 16, 1024, LAYOUT_SW128),
                  smem_desc(xs + L::X_BYTES + kk * 32, 16, 1024, LAYOUT_SW128), idesc1, (i | kk) != 0);
        mma_commit(BAR(B_EMPTY0 + s));
      }
      if (ok) {
        mma_commit(BAR(B_HFULL));
        ok = gwait(BAR(B_HREADY), 0, s_abort);
      }
      const uint64_t dh = kview(sb + L::OFF_H, L::SLAB_H);
      for (int nt = 0; nt < ntile && ok; ++nt) {
        const int b = nt & 1;
        ok = gwait(BAR(B_BFULL0 + b), (nt >> 1) & 1, s_abort);
        if (ok && nt >= 2) ok = gwait(BAR(B_ACCFREE0 + b), ((nt >> 1) - 1) & 1, s_abort);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t db = kview(sb + L::OFF_B + b * L::B_BYTES, L::SLAB_B);
        const uint32_t acc = tmem + (uint32_t)b * NT;
#pragma unroll
        for (int part = 0; part < 2; ++part)
#pragma unroll
          for (int kk = 0; kk < R / 16; ++kk)
            mma_f16(acc, dadv(dh, (uint32_t)(part * (R / 8) + 2 * kk) * L::SLAB_H), dadv(db, (uint32_t)(2 * kk) * L::SLAB_B),
                    idesc2, (part | kk) != 0);
        mma_commit(BAR(B_ACCFULL0 + b));  // (also: the A2 tile in buffer b has been read)
      }
    }
  } else {
    // ------------------------------------------------------------------------------------------------ epilogue
    const int g = (warp - 2) >> 2;               // group: output tiles g, g + 2, ...
    const int et = (tid - 64) & 127;             // thread of the group
    const int row = (warp & 3) * 32 + lane;      // token row of the tile = TMEM lane
    const uint32_t tlane = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    // A2 tile nt as registers of this thread: 16-byte piece idx = et + 128 k is octet idx % (R / 8) of output row idx / (R / 8)
    constexpr int BPT = NT * (R / 8) / EPI_THREADS;  // pieces per thread
    uint4 breg[BPT];
    auto b_load = [&](int nt) {
#pragma unroll
      for (int k = 0; k < BPT; ++k) {
        const int idx = et + k * EPI_THREADS, j = (nt0 + nt) * NT + idx / (R / 8), o = idx % (R / 8);
        breg[k] = j < a.n_out ? __ldg(reinterpret_cast<const uint4*>(a.A2 + (size_t)j * R + o * 8)) : make_uint4(0u, 0u, 0u, 0u);
      }
    };
    auto b_store = [&](int b) {
#pragma unroll
      for (int k = 0; k < BPT; ++k) {
        const int idx = et + k * EPI_THREADS;
        *reinterpret_cast<uint4*>(smem + L::OFF_B + b * L::B_BYTES + (idx % (R / 8)) * L::SLAB_B + (idx / (R / 8)) * 16) = breg[k];
      }
      fence_proxy_async();
      mbar_arrive(BAR(B_BFULL0 + b));
    };
    if (g < ntile) {   // (each group's first tile: while the first layer runs)
      b_load(g);
      b_store(g);
    }
    // this thread's entry of a tile's bias, fetched one tile ahead (its latency must not sit between two tiles)
    auto bias_load = [&](int nt) -> float {
      const int j = (nt0 + nt) * NT + et;
      return (a.bias && nt < ntile && j < a.n_out) ? __bfloat162float(a.bias[j]) : 0.f;
    };
    float bias_next = bias_load(g);
    bool fail = g == 0 && !gwait(BAR(B_HFULL), 0, s_abort);
    if (g == 0 && !fail) {
      tc_fence_after_sync();
#pragma unroll 1
      for (int c0 = 0; c0 < R; c0 += 16) {
        float v[16], lo[16];
        tmem_ld16(tlane + (uint32_t)c0, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float hi = __bfloat162float(__float2bfloat16_rn(v[i]));
          lo[i] = v[i] - hi;
          v[i] = hi;
        }
        *reinterpret_cast<uint4*>(smem + L::OFF_H + toff(L::SLAB_H, row, c0)) = ctc::pack8bf16(v);
        *reinterpret_cast<uint4*>(smem + L::OFF_H + toff(L::SLAB_H, row, c0 + 8)) = ctc::pack8bf16(v + 8);
        *reinterpret_cast<uint4*>(smem + L::OFF_H + toff(L::SLAB_H, row, R + c0)) = ctc::pack8bf16(lo);
        *reinterpret_cast<uint4*>(smem + L::OFF_H + toff(L::SLAB_H, row, R + c0 + 8)) = ctc::pack8bf16(lo + 8);
      }
      fence_proxy_async();
      tc_fence_before_sync();
      mbar_arrive(BAR(B_HREADY));
    }
    for (int nt = g; nt < ntile; nt += 2) {
      const int b = g;
      if (!fail) fail = !gwait(BAR(B_ACCFULL0 + b), (nt >> 1) & 1, s_abort);
      s_bias[b * NT + et] = bias_next;
      bias_next = bias_load(nt + 2);
      if (et == 0) tma_store_wait_read();  // the group's previous store is through with the staging tile
      fail = named_bar_or(1 + 2 * g, EPI_THREADS, fail);
      if (fail) break;
      tc_fence_after_sync();
      const bool more = nt + 2 < ntile;
      if (more) b_load(nt + 2);   // (in flight during this tile's epilogue)
      const uint32_t acc = tlane + (uint32_t)b * NT;
      uint8_t* const stg = smem + L::OFF_OUT + b * L::OUT_BYTES;
#pragma unroll 1
      for (int sl = 0; sl < NT / 64; ++sl) {   // one 64-column slab of the staging tile per round: both loads, one wait
        float v[64];
        tmem_ld32(acc + (uint32_t)sl * 64, v);
        tmem_ld32(acc + (uint32_t)sl * 64 + 32, v + 32);
        tmem_wait_ld();
        const float4* bs = reinterpret_cast<const float4*>(s_bias + b * NT + sl * 64);
        uint8_t* const slab = stg + sl * (TT * 128);
#pragma unroll
        for (int o = 0; o < 8; ++o) {
          const float4 b0 = bs[2 * o], b1 = bs[2 * o + 1];
          v[8 * o] += b0.x; v[8 * o + 1] += b0.y; v[8 * o + 2] += b0.z; v[8 * o + 3] += b0.w;
          v[8 * o + 4] += b1.x; v[8 * o + 5] += b1.y; v[8 * o + 6] += b1.z; v[8 * o + 7] += b1.w;
          *reinterpret_cast<uint4*>(slab + sw128(row, o)) = ctc::pack8bf16(v + 8 * o);
        }
      }
      tc_fence_before_sync();
      mbar_arrive(BAR(B_ACCFREE0 + b));
      if (more) b_store(b);       // (the products of tile nt, which read buffer b, completed before this tile's accumulator did)
      fence_proxy_async();
      named_bar_sync(2 + 2 * g, EPI_THREADS);
      if (et == 0) {
        tma_store_2d(&tm_out, smem_u32(stg), (nt0 + nt) * NT, n0);
        if ((nt0 + nt) * NT + 64 < a.n_out) tma_store_2d(&tm_out, smem_u32(stg) + TT * 128, (nt0 + nt) * NT + 64, n0);
        tma_store_commit();
      }
    }
    if (et == 0) tma_store_wait_all();
  }
  __syncthreads();
  if (*s_abort) {
    // let copies that are still in flight land before the block gives up its shared memory
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
    if (tid == 0 && a.dev_status) atomicMax(a.dev_status, (int)LAWCAT_ERR_TIMEOUT);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

// ---------------------------------------------------------------------------------------------------- exact kernels
// h[n][r] = A1[r] . x[n]: one block per token, the row of x in shared memory, one warp per bottleneck unit in turn
template <typename T>
__global__ void __launch_bounds__(256) gate_fn_h_kernel(const T* __restrict__ x, const T* __restrict__ A1,
                                                        float* __restrict__ h, int dm, int rank) {
  extern __shared__ float s_x[];
  const size_t n = blockIdx.x;
  for (int c = threadIdx.x; c < dm; c += blockDim.x) s_x[c] = ldf(x + n * dm + c);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int r = warp; r < rank; r += nw) {
    float acc = 0.f;
    for (int c = lane; c < dm; c += 32) acc = fmaf(ldf(A1 + (size_t)r * dm + c), s_x[c], acc);
    acc = warp_sum(acc);
    if (lane == 0) h[n * rank + r] = acc;
  }
}
// a[n][j] = A2[j] . h[n] + bias[j]: one block per token, one thread per output in turn
template <typename T>
__global__ void __launch_bounds__(256) gate_fn_out_kernel(const float* __restrict__ h, const T* __restrict__ A2,
                                                          const T* __restrict__ bias, T* __restrict__ out, int rank,
                                                          int n_out) {
  extern __shared__ float s_h[];
  const size_t n = blockIdx.x;
  for (int r = threadIdx.x; r < rank; r += blockDim.x) s_h[r] = h[n * rank + r];
  __syncthreads();
  for (int j = threadIdx.x; j < n_out; j += blockDim.x) {
    float acc = 0.f;
    for (int r = 0; r < rank; ++r) acc = fmaf(ldf(A2 + (size_t)j * rank + r), s_h[r], acc);
    if (bias) acc += ldf(bias + j);
    stf(out + n * n_out + j, acc);
  }
}

// ---------------------------------------------------------------------------------------------------- few tokens
// One block per TOK tokens, 256 threads. First layer: warp w takes the bottleneck units w, w + 8, ...; its lanes stride
// over the hidden channels in octets and meet in a shuffle sum. Second layer: a thread takes 8 consecutive outputs at a
// time (their rows of A2 are contiguous) and keeps TOK x 8 sums.
template <int TOK>
__global__ void __launch_bounds__(256) gate_fn_small_kernel(const bf16* __restrict__ x, const bf16* __restrict__ A1,
                                                            const bf16* __restrict__ A2, const bf16* __restrict__ bias,
                                                            bf16* __restrict__ out, int N, int dm, int rank, int n_out) {
  extern __shared__ __align__(16) uint8_t sm_small[];
  uint4* const s_x = reinterpret_cast<uint4*>(sm_small);                           // [TOK][dm / 8] octets of bf16
  float* const s_h = reinterpret_cast<float*>(sm_small + (size_t)TOK * dm * 2);    // [TOK][rank]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n0 = blockIdx.x * TOK, oct = dm >> 3;
  for (int i = tid; i < TOK * oct; i += 256) {
    const int t = i / oct, o = i - t * oct;
    s_x[i] = n0 + t < N ? __ldg(reinterpret_cast<const uint4*>(x + (size_t)(n0 + t) * dm) + o) : make_uint4(0u, 0u, 0u, 0u);
  }
  __syncthreads();
  // (four units at a time, so that a lane has 16 loads of A1 in flight)
  for (int r0 = warp; r0 < rank; r0 += 32) {
    float acc[4][TOK];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int t = 0; t < TOK; ++t) acc[u][t] = 0.f;
#pragma unroll 4
    for (int c = lane; c < oct; c += 32) {
      uint4 wa[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        wa[u] = r0 + 8 * u < rank ? __ldg(reinterpret_cast<const uint4*>(A1 + (size_t)(r0 + 8 * u) * dm) + c)
                                  : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int t = 0; t < TOK; ++t) {
        float fx[8];
        ctc::unpack8b(s_x[t * oct + c], fx);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          float fa[8];
          ctc::unpack8b(wa[u], fa);
#pragma unroll
          for (int i = 0; i < 8; ++i) acc[u][t] = fmaf(fa[i], fx[i], acc[u][t]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int t = 0; t < TOK; ++t) {
        const float v = warp_sum(acc[u][t]);
        if (lane == 0 && r0 + 8 * u < rank) s_h[t * rank + r0 + 8 * u] = v;
      }
  }
  __syncthreads();
  for (int jo = tid; jo * 8 < n_out; jo += 256) {
    const int j0 = jo * 8;
    float acc[TOK][8];
    {
      float fb[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (bias) ctc::unpack8b(__ldg(reinterpret_cast<const uint4*>(bias + j0)), fb);
#pragma unroll
      for (int t = 0; t < TOK; ++t)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[t][e] = fb[e];
    }
#pragma unroll 4
    for (int rr = 0; rr < rank; rr += 8) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float fa[8];
        ctc::unpack8b(__ldg(reinterpret_cast<const uint4*>(A2 + (size_t)(j0 + e) * rank + rr)), fa);
#pragma unroll
        for (int t = 0; t < TOK; ++t)
#pragma unroll
          for (int i = 0; i < 8; ++i) acc[t][e] = fmaf(fa[i], s_h[t * rank + rr + i], acc[t][e]);
      }
    }
#pragma unroll
    for (int t = 0; t < TOK; ++t)
      if (n0 + t < N) *reinterpret_cast<uint4*>(out + (size_t)(n0 + t) * n_out + j0) = ctc::pack8bf16(acc[t]);
  }
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
// row-major [rows, cols] bf16 matrix with boxes of box_rows x 64 columns, 128-byte swizzle
static bool map_2d(CUtensorMap* m, const void* ptr, size_t rows, size_t cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t es[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// SMs of the current device (looked up once per device)
static int sm_count_gfn() {
  static std::atomic<int> cached[64] = {};
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if ((n = cached[dev].load()) > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  cached[dev].store(n);
  return n;
}

template <int R>
static int launch_tc(const Ctx& c, int d_model, const void* x, const void* A1, const void* A2, const void* bias,
                     void* gate, size_t N, int n_out) {
  using L = Lay<R>;
  CUtensorMap tx, ta1, to;
  if (!map_2d(&tx, x, N, d_model, TT) || !map_2d(&ta1, A1, R, d_model, R) || !map_2d(&to, gate, N, n_out, TT))
    return LAWCAT_ERR_CUDA;
  static std::atomic<bool> raised[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LAWCAT_ERR_CUDA;
  if (!raised[dev].load()) {
    if (cudaFuncSetAttribute(gate_fn_tc_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L::BYTES) != cudaSuccess)
      return LAWCAT_ERR_CUDA;
    raised[dev].store(true);
  }
  GArgs a{(const bf16*)A2, (const bf16*)bias, (int)N, d_model, n_out, c.dev_status};
  // fewer token tiles than the SMs can hold (two blocks each for rank <= 32): share each tile's outputs out over up to 8
  // blocks, every one of them with output tiles of its own
  const size_t tiles = (N + TT - 1) / TT;
  const int ntile_all = (n_out + NT - 1) / NT, room = (R <= 32 ? 2 : 1) * sm_count_gfn();
  int ysplit = (int)std::min<size_t>(8, std::max<size_t>(1, room / tiles));
  ysplit = std::min(ysplit, ntile_all);
  ysplit = (ntile_all + ((ntile_all + ysplit - 1) / ysplit) - 1) / ((ntile_all + ysplit - 1) / ysplit);  // (no empty block)
  LAWCAT_LAUNCH("gate_fn_tc", c.stream,
                gate_fn_tc_kernel<R><<<dim3((unsigned)tiles, (unsigned)ysplit), THREADS, L::BYTES, c.stream>>>(tx, ta1, to, a));
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

template <int TOK>
static int launch_small(const Ctx& c, int d_model, int rank, const void* x, const void* A1, const void* A2,
                        const void* bias, void* gate, size_t N, int n_out) {
  const size_t smem = (size_t)TOK * d_model * 2 + sizeof(float) * (size_t)TOK * rank;
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(gate_fn_small_kernel<TOK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return LAWCAT_ERR_CUDA;
  LAWCAT_LAUNCH("gate_fn_small", c.stream,
                gate_fn_small_kernel<TOK><<<(unsigned)((N + TOK - 1) / TOK), 256, smem, c.stream>>>(
                    (const bf16*)x, (const bf16*)A1, (const bf16*)A2, (const bf16*)bias, (bf16*)gate, (int)N, d_model, rank,
                    n_out));
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

template <typename T>
static int launch_exact(const Ctx& c, int d_model, int rank, const void* x, const void* A1, const void* A2,
                        const void* bias, void* gate, size_t N, int n_out, void* ws) {
  float* h = (float*)ws;
  const size_t smem1 = sizeof(float) * (size_t)d_model;
  if (smem1 > 48 * 1024 &&
      cudaFuncSetAttribute(gate_fn_h_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1) != cudaSuccess)
    return LAWCAT_ERR_CUDA;
  LAWCAT_LAUNCH("gate_fn_h", c.stream,
                gate_fn_h_kernel<T><<<(unsigned)N, 256, smem1, c.stream>>>((const T*)x, (const T*)A1, h, d_model, rank));
  LAWCAT_CHECK_LAUNCH();
  LAWCAT_LAUNCH("gate_fn_out", c.stream,
                gate_fn_out_kernel<T><<<(unsigned)N, 256, sizeof(float) * (size_t)rank, c.stream>>>(
                    h, (const T*)A2, (const T*)bias, (T*)gate, rank, n_out));
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

}  // namespace gfn

bool gate_fn_tc_supported(const lawcat_params& p, int d_model, int rank) {
  const long long n_out = (long long)p.H * p.gate_dim;
  return p.dtype == LAWCAT_BF16 && (rank == 16 || rank == 32 || rank == 64 || rank == 128) && d_model % 8 == 0 &&
         n_out % 8 == 0 && p.chunk != 1;
}

// Few tokens: the latency-oriented CUDA-core kernel (see the head of this file). SMALL_1: tokens up to which one block per
// token is used, SMALL_4: up to which one block per four tokens; beyond, the tensor-core kernel where it applies.
constexpr size_t SMALL_1 = 128, SMALL_4 = 1024;
// tokens per block of the few-token kernel for this call, 0 = not its case
static int gate_fn_small_tok(const lawcat_params& p, int d_model, int rank) {
  const long long n_out = (long long)p.H * p.gate_dim;
  const size_t N = (size_t)p.B * p.T;
  if (p.dtype != LAWCAT_BF16 || rank % 8 != 0 || d_model % 8 != 0 || n_out % 8 != 0 || p.chunk == 1) return 0;
  if (N <= SMALL_1) return 1;
  if (N <= SMALL_4 && d_model <= 8192) return 4;
  return 0;
}

size_t gate_fn_workspace_bytes(const lawcat_params& p, int d_model, int rank) {
  if (gate_fn_tc_supported(p, d_model, rank)) return 0;
  if (gate_fn_small_tok(p, d_model, rank)) return 0;
  return sizeof(float) * (size_t)p.B * p.T * rank;
}

int launch_gate_fn(const Ctx& c, int d_model, int rank, const void* x, const void* A1, const void* A2, const void* bias,
                   void* gate, void* ws) {
  const lawcat_params& p = *c.p;
  const size_t N = (size_t)p.B * p.T;
  const int n_out = p.H * p.gate_dim;
  if (N == 0) return LAWCAT_OK;
  switch (gate_fn_small_tok(p, d_model, rank)) {
    case 1: return gfn::launch_small<1>(c, d_model, rank, x, A1, A2, bias, gate, N, n_out);
    case 4: return gfn::launch_small<4>(c, d_model, rank, x, A1, A2, bias, gate, N, n_out);
    default: break;
  }
  if (gate_fn_tc_supported(p, d_model, rank)) {
    switch (rank) {
      case 16: return gfn::launch_tc<16>(c, d_model, x, A1, A2, bias, gate, N, n_out);
      case 32: return gfn::launch_tc<32>(c, d_model, x, A1, A2, bias, gate, N, n_out);
      case 64: return gfn::launch_tc<64>(c, d_model, x, A1, A2, bias, gate, N, n_out);
      default: return gfn::launch_tc<128>(c, d_model, x, A1, A2, bias, gate, N, n_out);
    }
  }
  if (p.dtype == LAWCAT_F32) return gfn::launch_exact<float>(c, d_model, rank, x, A1, A2, bias, gate, N, n_out, ws);
  return gfn::launch_exact<bf16>(c, d_model, rank, x, A1, A2, bias, gate, N, n_out, ws);
}

}  // namespace lawcat
