// Host side of the chunkwise tensor-core layer forward: tensor maps, segment split, launches.
#include <atomic>
#include <mutex>

#include "layer_tc_kernel.cuh"

namespace lawcat {
namespace tc {

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

// [B, T, heads, dh] bf16 tensor as a 4-D map (channel, head, token, batch) with boxes of 64 channels x rows tokens.
// A map depends only on the pointer and the shape, so the last few are kept per host thread: a serving loop that calls
// with the same buffers encodes each map once.
static bool make_map(CUtensorMap* m, const void* ptr, int heads, int T, int B, int rows, int dh) {
  struct Slot {
    const void* ptr;
    int heads, T, B, rows, dh;
    bool used;
    CUtensorMap map;
  };
  constexpr int NSLOT = 16;
  thread_local Slot cache[NSLOT] = {};
  thread_local int next = 0;
  for (int i = 0; i < NSLOT; ++i) {
    const Slot& c = cache[i];
    if (c.used && c.ptr == ptr && c.heads == heads && c.T == T && c.B == B && c.rows == rows && c.dh == dh) {
      *m = c.map;
      return true;
    }
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)dh, (cuuint64_t)heads, (cuuint64_t)T, (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)dh * 2, (cuuint64_t)heads * dh * 2, (cuuint64_t)T * heads * dh * 2};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)rows, 1};
  const cuuint32_t es[4] = {1, 1, 1, 1};
  if (fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, es,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  Slot& c = cache[next];
  next = (next + 1) % NSLOT;
  c.ptr = ptr; c.heads = heads; c.T = T; c.B = B; c.rows = rows; c.dh = dh; c.map = *m; c.used = true;
  return true;
}

// State at the start of every segment from the end states of its pieces (each computed from a zero state) and their
// total decays: running state cur = given state; after piece i: cur = decay[i] * cur + local[i] (Eq. 4 unrolled over
// whole pieces); start[seg] = cur in front of the segment's first piece.
// One thread per state entry (the d_k x d_v entries of S, then the d_k entries of z) of one (batch, head).
__global__ void segment_scan_kernel(const float* __restrict__ S0, const float* __restrict__ z0,
                                    const float* __restrict__ loc_S, const float* __restrict__ loc_z,
                                    const float* __restrict__ dtot, float* __restrict__ start_S,
                                    float* __restrict__ start_z, int BH, int nseg, int nsub, int dh) {
  const int D = dh;  // (rows and columns of the state as stored)
  const int per = D * D + D;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // the layer kernel may start its set-up
  asm volatile("griddepcontrol.wait;" ::: "memory");               // (this kernel itself: behind the state-only pass)
  if (idx >= BH * per) return;
  const int bh = idx / per, r = idx % per;
  const bool isz = r >= D * D;
  const int c = isz ? r - D * D : r / D;  // key channel: the decay is per row of the state
  const int e = isz ? 0 : r % D;
  float cur = isz ? (z0 ? z0[(size_t)bh * D + c] : 0.f) : (S0 ? S0[((size_t)bh * D + c) * D + e] : 0.f);
  for (int sgm = 0; sgm < nseg; ++sgm) {
    const size_t so = (size_t)bh * nseg + sgm;
    if (isz) start_z[so * D + c] = cur; else start_S[(so * D + c) * D + e] = cur;
    if (sgm + 1 < nseg) {
      for (int sb = 0; sb < nsub; ++sb) {
        const size_t si = so * nsub + sb;
        const float loc = isz ? loc_z[si * D + c] : loc_S[(si * D + c) * D + e];
        cur = fmaf(exp2f(dtot[si * D + c]), cur, loc);
      }
    }
  }
}

}  // namespace tc

// Number of SMs of the current device (cached per device; 148 on a B200).
static int sm_count() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

// How a sequence is cut: nseg segments of seg_len tokens (a multiple of the chunk; every segment holds tokens), and the
// pieces per segment of the state-only pre-pass.
struct TcPlan {
  int nseg, seg_len, nsub;
};

// Segments per sequence: enough thread blocks to fill the SMs (one block per SM), but at least MIN_SEG_CHUNKS chunks per
// segment (a thread block spends about three chunk times on its set-up and on filling its pipeline). Pieces per segment
// in the state-only pre-pass: its thread blocks are independent, so cutting the segments finer lets them fill the SMs in
// whole waves; the split with the fewest chunks per SM wins (a small charge per extra piece).
// Two 64-wide heads share a thread block when they can: an even number of query heads per key/value head (the two heads
// of a block read the same k and v) and one decay per key channel.
static bool layer_tc_paired(const lawcat_params& p) {
  return p.d_k == 64 && p.gate_dim == p.d_k && (p.H / p.H_kv) % 2 == 0;
}

static TcPlan layer_tc_plan(const lawcat_params& p) {
  constexpr int MIN_SEG_CHUNKS = 4;
  const int sms = sm_count();
  const int chunks = (p.T + tc::C - 1) / tc::C;
  const int seqs = p.B * (layer_tc_paired(p) ? p.H / 2 : p.H);  // sequences of thread blocks
  int n = sms / seqs;
  if (n > chunks / MIN_SEG_CHUNKS) n = chunks / MIN_SEG_CHUNKS;
  if (n < 1) n = 1;
  TcPlan pl;
  pl.seg_len = ((chunks + n - 1) / n) * tc::C;
  pl.nseg = (p.T + pl.seg_len - 1) / pl.seg_len;  // (rounding the length up may leave fewer segments than asked for)
  if (pl.nseg < 1) pl.nseg = 1;
  const int cps = pl.seg_len / tc::C;
  int best = 1, best_cost = 1 << 30;
  for (int ns = 1; ns <= 8 && ns * 4 <= cps; ++ns) {
    const int ctas = seqs * (pl.nseg - 1) * ns;
    const int cost = ((ctas + sms - 1) / sms) * ((cps + ns - 1) / ns + 2);
    if (cost < best_cost) { best_cost = cost; best = ns; }
  }
  pl.nsub = best;
  return pl;
}

int layer_tc_segments(const lawcat_params& p) { return layer_tc_plan(p).nseg; }

// Limit of the kernels' device-side waits in clock cycles (about two seconds); a test hook may shorten it.
static std::atomic<long long> g_wait_limit{4000000000LL};

size_t layer_tc_workspace_bytes(const lawcat_params& p) {
  const TcPlan pl = layer_tc_plan(p);
  if (pl.nseg == 1) return 0;
  const size_t pieces = (size_t)pl.nseg * pl.nsub;
  return sizeof(float) * (size_t)p.B * p.H * ((pieces + pl.nseg) * ((size_t)p.d_k * p.d_k + p.d_k) + pieces * p.d_k);
}

bool layer_tc_supported(const lawcat_params& p) {
  // Sharp sigmoid gates (tau < 8: a token's decay reaches a half at tau = 1) drive the exponents of the in-chunk
  // factorization out of the fp16 range within half a chunk; the operands then fall back to bf16 (8 significant bits)
  // and a seeded random sweep finds outputs and states beyond 1e-2 of their RMS for tau = 1, 2 and 4 (numerator-only
  // form, one decay per head, eps != 0, carried states). Those gates take the exact recurrence. Very short calls do too:
  // with fewer than 16 tokens the state is a sum of so few terms that the rounding of single 16-bit operands shows in
  // its largest entries, and the exact kernels are as fast there.
  const bool sharp = p.gate_mode == LAWCAT_GATE_LOGITS && p.gate_tau < 8.f;
  return p.dtype == LAWCAT_BF16 && (p.d_k == tc::D || p.d_k == 64) && p.d_v == p.d_k &&
         (p.gate_dim == p.d_k || p.gate_dim == 1) && !sharp && p.T >= 16 &&
         p.phi == LAWCAT_PHI_SOFTMAX && p.conv_k <= tc::HALO + 1 && p.B > 0 && p.T > 0 &&
         (p.chunk == 0 || p.chunk == tc::C) &&
         !p.mix_unshared;  // (one W_h is what lets both streams share the M = 128 mix)
}

int launch_layer_tc(const Ctx& c, const void* q, const void* k, const void* v, const void* gate, const void* w_q,
                    const void* w_k, const void* W, const void* cache_q_in, const void* cache_k_in, const float* S0,
                    const float* z0, void* o, void* cache_q_out, void* cache_k_out, float* S_T, float* z_T, void* ws) {
  using namespace tc;
  const lawcat_params& p = *c.p;
  CUtensorMap tq, tk, tv, tg;
  const int dh = p.d_k;
  const bool paired = layer_tc_paired(p);
  // (pair: q, gate and o of two neighbouring heads are 128 contiguous channels and are mapped as one head of 128)
  const int Hmap = paired ? p.H / 2 : p.H, dmap = paired ? 128 : dh;
  if (!make_map(&tq, q, Hmap, p.T, p.B, C, dmap) || !make_map(&tk, k, p.H_kv, p.T, p.B, C, dh) ||
      !make_map(&tv, v, p.H_kv, p.T, p.B, C, dh))
    return LAWCAT_ERR_CUDA;
  if (p.gate_dim == 1) tg = tq;  // (never used: one logit per token and head is read without a tensor map)
  else if (!make_map(&tg, gate, Hmap, p.T, p.B, C, dmap)) return LAWCAT_ERR_CUDA;
  TcArgs a{};
  a.q = (const bf16*)q; a.k = (const bf16*)k; a.o = (bf16*)o;
  a.gate = (const bf16*)gate; a.gate_dim = p.gate_dim; a.dh = dh;
  a.w_q = (const bf16*)w_q; a.w_k = (const bf16*)w_k; a.W = (const bf16*)W;
  a.cache_q = (const bf16*)cache_q_in; a.cache_k = (const bf16*)cache_k_in;
  a.cache_q_out = (bf16*)cache_q_out; a.cache_k_out = (bf16*)cache_k_out;
  a.dev_status = c.dev_status;
  a.T = p.T; a.H = p.H; a.Hkv = p.H_kv; a.K = p.conv_k;
  a.gate_mode = p.gate_mode; a.normalize = p.normalize; a.inv_tau = 1.f / p.gate_tau; a.eps = p.eps;
  a.wait_limit = g_wait_limit.load();
  const TcPlan pl = layer_tc_plan(p);
  const int nseg = pl.nseg;
  a.nseg = nseg;
  a.seg_len = pl.seg_len;
  auto* const k_layer = paired ? layer_tc_kernel<0, 2> : dh == 64 ? layer_tc_kernel<0, 1> : layer_tc_kernel<0, 0>;
  auto* const k_state = paired ? layer_tc_kernel<1, 2> : dh == 64 ? layer_tc_kernel<1, 1> : layer_tc_kernel<1, 0>;
  {
    // the kernels' shared-memory limit is raised once per device
    static std::mutex mu;
    static bool done[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LAWCAT_ERR_CUDA;
    std::lock_guard<std::mutex> lk(mu);
    if (!done[dev]) {
      if (cudaFuncSetAttribute(layer_tc_kernel<0, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess ||
          cudaFuncSetAttribute(layer_tc_kernel<0, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess ||
          cudaFuncSetAttribute(layer_tc_kernel<0, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess ||
          cudaFuncSetAttribute(layer_tc_kernel<1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess ||
          cudaFuncSetAttribute(layer_tc_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess ||
          cudaFuncSetAttribute(layer_tc_kernel<1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess)
        return LAWCAT_ERR_CUDA;
      done[dev] = true;
    }
  }
  const int BH = p.B * p.H;                       // real heads: the states in the workspace are per real head
  const int NB = paired ? BH / 2 : BH;            // sequences of thread blocks
  if (nseg == 1) {
    a.S0 = S0; a.z0 = z0; a.S_T = S_T; a.z_T = z_T; a.dtot = nullptr;
    a.grid_nseg = 1; a.nsub = 1; a.seg_in = 0; a.seg_out = 0;
    LaunchScope _ls("layer_tc", c.stream);
    k_layer<<<NB, THREADS, SMEM_ALLOC, c.stream>>>(tq, tk, tv, tg, a);
    LAWCAT_CHECK_LAUNCH();
    return LAWCAT_OK;
  }
  // Several segments per sequence: (1) every segment but the last computes its end state from a zero state, and the
  // total decay of the segment; (2) a scan over the segments turns these into the state at each segment's start;
  // (3) the layer runs on all segments at once, each from its start state.
  const int nsub = pl.nsub;
  const size_t nS = (size_t)BH * nseg * dh * dh, nz = (size_t)BH * nseg * dh;
  float* loc_S = (float*)ws;              // [BH, nseg, nsub, D, D]
  float* loc_z = loc_S + nS * nsub;       // [BH, nseg, nsub, D]
  float* dtot = loc_z + nz * nsub;        // [BH, nseg, nsub, D]
  float* start_S = dtot + nz * nsub;      // [BH, nseg, D, D]
  float* start_z = start_S + nS;          // [BH, nseg, D]
  {
    TcArgs b1 = a;
    b1.S0 = nullptr; b1.z0 = nullptr; b1.S_T = loc_S; b1.z_T = loc_z; b1.dtot = dtot;
    b1.grid_nseg = nseg - 1; b1.nsub = nsub; b1.seg_in = 1; b1.seg_out = 1;
    LaunchScope _ls("layer_tc_state", c.stream);
    k_state<<<NB * (nseg - 1) * nsub, THREADS, SMEM_ALLOC, c.stream>>>(tq, tk, tv, tg, b1);
    LAWCAT_CHECK_LAUNCH();
  }
  {
    const int total = BH * (dh * dh + dh);
    LaunchScope _ls("segment_scan", c.stream);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((total + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = c.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, segment_scan_kernel, S0, z0, (const float*)loc_S, (const float*)loc_z, (const float*)dtot,
                       start_S, start_z, BH, nseg, nsub, dh);
    LAWCAT_CHECK_LAUNCH();
  }
  a.S0 = start_S; a.z0 = start_z; a.S_T = S_T; a.z_T = z_T; a.dtot = nullptr;
  a.grid_nseg = nseg; a.nsub = 1; a.seg_in = 1; a.seg_out = 0;
  LaunchScope _ls("layer_tc", c.stream);
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(NB * nseg));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_ALLOC;
    cfg.stream = c.stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, k_layer, tq, tk, tv, tg, a);
  }
  LAWCAT_CHECK_LAUNCH();
  return LAWCAT_OK;
}

}  // namespace lawcat

// Test hook: the limit (clock cycles) of every bounded device-side wait of the tensor-core layer kernels launched from
// now on; 0 restores the default. A limit of a few cycles makes the first unsatisfied wait give up, which exercises the
// path that reports LAWCAT_ERR_TIMEOUT (nothing faults or hangs: the block leaves its loops, lets its copies land, frees
// its tensor memory and returns).
extern "C" void lawcat_test_set_wait_limit(long long cycles) {
  lawcat::g_wait_limit.store(cycles > 0 ? cycles : 4000000000LL);
}

#ifdef LAWCAT_TIMELINE
// (profiling builds only) copies the clock stamps of the last layer-kernel launch to the host
extern "C" int lawcat_timeline_read(long long* host, size_t n) {
  const size_t have = sizeof(lawcat::tc::g_timeline) / sizeof(long long);
  return cudaMemcpyFromSymbol(host, lawcat::tc::g_timeline, sizeof(long long) * (n < have ? n : have)) == cudaSuccess
             ? LAWCAT_OK : LAWCAT_ERR_CUDA;
}
#endif
