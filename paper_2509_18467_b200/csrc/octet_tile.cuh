// Operand tiles of the lock-step tensor-core kernels (conv + mix forward and backward, decode features): unswizzled 8x8
// core matrices with every 8-column slab contiguous. Element (r, c) of a tile with R rows sits at
// (c / 8) * (16 R + 16) + 16 r + 2 (c % 8); the same bytes serve as a K-major operand (LBO = slab stride, SBO = 128) and
// as an MN-major one (LBO = 128, SBO = slab stride). Plus the small helpers these kernels share.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace lawcat {
namespace ctc {

using namespace tc;

constexpr int TT = 128;   // tokens per tile
constexpr int HALO = 3;   // raw rows kept in front of a tile (conv width up to 4)

template <int D>
struct Lay {
  static constexpr int OPR = D / 8;                         // 16-byte octets per row
  static constexpr uint32_t SLAB_W = D * 16 + 16;           // slab stride of the W tile (D rows)
  static constexpr uint32_t SLAB_U = TT * 16 + 16;          // slab stride of tiles with 128 token rows
  static constexpr uint32_t TILE_W = OPR * SLAB_W, TILE_U = OPR * SLAB_U;
  static constexpr uint32_t RAW_STRIDE = D * 2 + 16;        // bytes per raw row (padded: the conv reads 4 rows per warp)
  static constexpr uint32_t RAW_BYTES = (TT + HALO) * RAW_STRIDE;
};

__device__ __forceinline__ uint32_t toff(uint32_t slab, int r, int c) { return (uint32_t)(c >> 3) * slab + (uint32_t)r * 16u + (uint32_t)(c & 7) * 2u; }
__device__ __forceinline__ uint64_t kview(uint32_t addr, uint32_t slab) { return smem_desc(addr, slab, 128, LAYOUT_NONE); }
__device__ __forceinline__ uint64_t mview(uint32_t addr, uint32_t slab) { return smem_desc(addr, 128, slab, LAYOUT_NONE); }
__device__ __forceinline__ uint64_t dadv(uint64_t d, uint32_t bytes) {
  return (d & 0xFFFFFFFF00000000ull) | (uint64_t)((uint32_t)d + (bytes >> 4));
}
__device__ __forceinline__ void unpack8b(const uint4& v, float* f) {
  f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
  f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
}
__device__ __forceinline__ uint4 pack8f16(const float* v) {
  return make_uint4(pack_f16(v[0], v[1]), pack_f16(v[2], v[3]), pack_f16(v[4], v[5]), pack_f16(v[6], v[7]));
}
__device__ __forceinline__ uint4 pack8bf16(const float* v) {
  return make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
__device__ __forceinline__ void store_row8(bf16* p, const float* v) { *reinterpret_cast<uint4*>(p) = pack8bf16(v); }
__device__ __forceinline__ void store_row8(float* p, const float* v) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void load_row8(const bf16* p, float* v) { unpack8b(*reinterpret_cast<const uint4*>(p), v); }
__device__ __forceinline__ void load_row8(const float* p, float* v) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// one mbarrier, bounded wait (a product batch completes within microseconds; 2e8 cycles is about a tenth of a second)
struct Waiter {
  uint32_t bar, phase;
  volatile int* abort_flag;
  int* dev_status;
  __device__ __forceinline__ void wait() {
    if (!*abort_flag) {
      bool ok = mbar_try_wait(bar, phase);
      if (!ok) {
        const long long t0 = clock64();
        while (!ok) {
#pragma unroll 1
          for (int i = 0; i < 16 && !ok; ++i) ok = mbar_try_wait(bar, phase);
          if (!ok && (*abort_flag || clock64() - t0 > 200000000LL)) break;
        }
      }
      if (!ok) {
        *abort_flag = 1;
        if (dev_status) atomicMax(dev_status, (int)LAWCAT_ERR_TIMEOUT);
      }
    }
    phase ^= 1u;
    tc_fence_after_sync();
  }
};

// W[h][c][e] (bf16, exact in fp16) as a tile with rows c, columns e
template <int D>
__device__ __forceinline__ void load_w_tile(uint8_t* s_wt, const bf16* Wh, int tid, int nthreads) {
  using L = Lay<D>;
  for (int idx = tid; idx < D * L::OPR; idx += nthreads) {
    const int c = idx / L::OPR, o = idx % L::OPR;
    float f[8];
    unpack8b(*reinterpret_cast<const uint4*>(Wh + (size_t)c * D + o * 8), f);
    *reinterpret_cast<uint4*>(s_wt + toff(L::SLAB_W, c, o * 8)) = pack8f16(f);
  }
}

}  // namespace ctc
}  // namespace lawcat
