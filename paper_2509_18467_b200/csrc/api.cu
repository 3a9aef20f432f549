// The C ABI: argument validation on the host, then dispatch to the kernels. Nothing here allocates device memory or
// synchronizes (the host-buffer variant creates its two copy streams and its events on first use and keeps them).
#include <mutex>
#include <vector>

#include "common.cuh"

using namespace lawcat;

namespace {

bool pow2_dim(int d) { return d == 16 || d == 32 || d == 64 || d == 128; }

int check_params(const lawcat_params* p, bool need_T) {
  if (!p) return LAWCAT_ERR_INVALID_ARG;
  if (p->B < 0 || p->H <= 0 || p->H_kv <= 0 || (need_T && p->T < 0)) return LAWCAT_ERR_INVALID_ARG;
  if (p->H % p->H_kv != 0) return LAWCAT_ERR_INVALID_ARG;
  if (p->dtype != LAWCAT_F32 && p->dtype != LAWCAT_BF16) return LAWCAT_ERR_INVALID_ARG;
  if (p->phi < LAWCAT_PHI_SOFTMAX || p->phi > LAWCAT_PHI_IDENTITY) return LAWCAT_ERR_INVALID_ARG;
  if (p->gate_mode != LAWCAT_GATE_LOGITS && p->gate_mode != LAWCAT_GATE_LOGDECAY) return LAWCAT_ERR_INVALID_ARG;
  if (!(p->gate_tau > 0.f) || !(p->eps >= 0.f)) return LAWCAT_ERR_INVALID_ARG;
  if (p->normalize != 0 && p->normalize != 1) return LAWCAT_ERR_INVALID_ARG;
  if (p->mix_unshared != 0 && p->mix_unshared != 1) return LAWCAT_ERR_INVALID_ARG;
  if (p->chunk < 0) return LAWCAT_ERR_INVALID_ARG;
  if (!pow2_dim(p->d_k) || !pow2_dim(p->d_v)) return LAWCAT_ERR_UNSUPPORTED;
  if (p->conv_k < 1 || p->conv_k > 8) return LAWCAT_ERR_UNSUPPORTED;
  if (p->gate_dim != 1 && p->gate_dim != p->d_k) return LAWCAT_ERR_UNSUPPORTED;
  if ((long long)p->B * p->H > 0x7fffffffLL / 64) return LAWCAT_ERR_UNSUPPORTED;
  return LAWCAT_OK;
}

bool aligned16(const void* x) { return (reinterpret_cast<uintptr_t>(x) & 15u) == 0; }

// required pointers must be non-NULL, every given pointer 16-byte aligned
// (an empty problem, B*T == 0, has empty tensors whose pointers may be NULL)
template <size_t NR, size_t NO>
int check_ptrs(const void* const (&req)[NR], const void* const (&opt)[NO], bool empty = false) {
  for (const void* x : req)
    if ((!x && !empty) || !aligned16(x)) return LAWCAT_ERR_INVALID_ARG;
  for (const void* x : opt)
    if (x && !aligned16(x)) return LAWCAT_ERR_INVALID_ARG;
  return LAWCAT_OK;
}

size_t elems(const lawcat_params* p, int heads, int d) { return (size_t)p->B * (size_t)p->T * heads * d; }

}  // namespace

namespace lawcat {
int validate_params(const lawcat_params* p, bool need_T) { return check_params(p, need_T); }
}  // namespace lawcat

extern "C" size_t lawcat_workspace_bytes(const lawcat_params* p, int op);

namespace {
// whether the fused layer backward runs on the tensor-core kernels (fp32 features between its stages)
bool layer_bwd_tc(const lawcat_params& p) {
  return p.chunk != 1 && gla_tc_bwd_supported(p) && convmix_tc_fwd_supported(p) && convmix_tc_bwd_supported(p);
}

__global__ void widen_kernel(const bf16* __restrict__ x, float* __restrict__ y, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) y[i] = __bfloat162float(x[i]);
}
__global__ void narrow_kernel(const float* __restrict__ x, bf16* __restrict__ y, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) y[i] = __float2bfloat16_rn(x[i]);
}

// Scratch of the exact layer backward: the chain conv_fwd -> gla_fwd -> gla_bwd -> conv_bwd in fp32. bf16 tensors are
// widened to fp32 copies first and the four activation gradients narrowed at the end, so that no feature and no feature
// gradient is rounded to bf16 between the stages.
struct ExactBwdLayout {
  size_t in[10];    // q k v gate w_q w_k W dO cache_q cache_k  (fp32 copies; only for bf16 storage)
  size_t out[4];    // dq dk dv dgate (fp32; only for bf16 storage)
  size_t qd, kd, dqd, dkd, o, den, ws_g, ws_c, total;
};
ExactBwdLayout exact_bwd_layout(const lawcat_params* p) {
  ExactBwdLayout L{};
  lawcat_params p32 = *p;
  p32.dtype = LAWCAT_F32;
  const size_t n_in[10] = {elems(p, p->H, p->d_k), elems(p, p->H_kv, p->d_k), elems(p, p->H_kv, p->d_v),
                           elems(p, p->H, p->gate_dim), (size_t)p->H * p->d_k * p->conv_k,
                           (size_t)p->H_kv * p->d_k * p->conv_k, (size_t)(1 + p->mix_unshared) * p->H * p->d_k * p->d_k,
                           elems(p, p->H, p->d_v),
                           (size_t)p->B * (p->conv_k - 1) * p->H * p->d_k, (size_t)p->B * (p->conv_k - 1) * p->H_kv * p->d_k};
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes, 256); return o; };
  const bool widen = p->dtype == LAWCAT_BF16;
  for (int i = 0; i < 10; ++i) L.in[i] = take(widen ? 4 * n_in[i] : 0);
  for (int i = 0; i < 4; ++i) L.out[i] = take(widen ? 4 * n_in[i] : 0);
  L.qd = take(4 * n_in[0]); L.kd = take(4 * n_in[0]); L.dqd = take(4 * n_in[0]); L.dkd = take(4 * n_in[0]);
  L.o = take(4 * n_in[7]); L.den = take(4 * elems(p, p->H, 1));
  L.ws_g = take(lawcat_workspace_bytes(&p32, LAWCAT_OP_GLA_BWD));
  L.ws_c = take(lawcat_workspace_bytes(&p32, LAWCAT_OP_CONV_BWD));
  L.total = off;
  return L;
}

size_t layer_bwd_workspace(const lawcat_params* p) {
  if (layer_bwd_tc(*p)) {
    // fp32 features and their gradients between the stages, then the scratch of the attention and the conv backward
    return 4 * align_up(4 * elems(p, p->H, p->d_k), 256) + lawcat_workspace_bytes(p, LAWCAT_OP_GLA_BWD) +
           lawcat_workspace_bytes(p, LAWCAT_OP_CONV_BWD);
  }
  return exact_bwd_layout(p).total;
}
}  // namespace

extern "C" {

int lawcat_version(void) { return 100; }

const char* lawcat_status_string(int s) {
  switch (s) {
    case LAWCAT_OK: return "ok";
    case LAWCAT_ERR_INVALID_ARG: return "invalid argument";
    case LAWCAT_ERR_UNSUPPORTED: return "unsupported shape or option";
    case LAWCAT_ERR_CUDA: return "CUDA runtime error";
    case LAWCAT_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case LAWCAT_ERR_TIMEOUT: return "bounded device wait ran out";
    case LAWCAT_ERR_NUMERIC: return "numeric range violation";
    case LAWCAT_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

size_t lawcat_workspace_bytes(const lawcat_params* p, int op) {
  if (check_params(p, op != LAWCAT_OP_DECODE_STEP) != LAWCAT_OK) return 0;
  switch (op) {
    case LAWCAT_OP_CONV_BWD:
      return align_up(sizeof(float) * elems(p, p->H, p->d_k), 256) + align_up(sizeof(float) * elems(p, p->H_kv, p->d_k), 256);
    case LAWCAT_OP_GLA_BWD:
      if (gla_tc_bwd_supported(*p)) return gla_tc_bwd_workspace_bytes(*p);
      return align_up(sizeof(float) * elems(p, p->H, p->d_v), 256) + 2 * align_up(sizeof(float) * elems(p, p->H, 1), 256) +
             align_up(sizeof(float) * elems(p, p->H, p->d_k), 256);
    case LAWCAT_OP_LAYER_FWD:
      if (layer_tc_supported(*p)) return align_up(layer_tc_workspace_bytes(*p), 256);
      return 2 * align_up(sizeof(float) * elems(p, p->H, p->d_k), 256);
    case LAWCAT_OP_DECODE_STEP:
      return align_up(decode_workspace_bytes(*p), 256);
    case LAWCAT_OP_LAYER_BWD:
      return layer_bwd_workspace(p);
    default:
      return 0;
  }
}

int lawcat_conv_fwd(const lawcat_params* p, const void* q, const void* k, const void* w_q, const void* w_k,
                    const void* W, const void* cache_q, const void* cache_k, void* qdot, void* kdot, void* ws,
                    size_t ws_bytes, void* stream, int* dev_status) {
  (void)ws; (void)ws_bytes;
  int r = check_params(p, true);
  if (r) return r;
  const void* const req[] = {q, k, w_q, w_k, qdot, kdot};
  const void* const opt[] = {W, cache_q, cache_k};
  if ((r = check_ptrs(req, opt, (size_t)p->B * p->T == 0))) return r;
  Ctx c{p, (cudaStream_t)stream, dev_status};
  if (W) return launch_convmix_fwd(c, q, k, w_q, w_k, W, cache_q, cache_k, qdot, kdot, false, p->chunk == 1);
  if ((r = launch_conv_plain(c, q, w_q, cache_q, qdot, p->H))) return r;
  return launch_conv_plain(c, k, w_k, cache_k, kdot, p->H_kv);
}

size_t lawcat_gate_fn_workspace_bytes(const lawcat_params* p, int32_t d_model, int32_t rank) {
  if (check_params(p, true) != LAWCAT_OK || d_model <= 0 || rank <= 0) return 0;
  return align_up(gate_fn_workspace_bytes(*p, d_model, rank), 256);
}

int lawcat_gate_fn_fwd(const lawcat_params* p, int32_t d_model, int32_t rank, const void* x, const void* A1,
                       const void* A2, const void* bias, void* gate, void* ws, size_t ws_bytes, void* stream,
                       int* dev_status) {
  int r = check_params(p, true);
  if (r) return r;
  if (d_model <= 0 || rank <= 0) return LAWCAT_ERR_INVALID_ARG;
  if (d_model > 16384 || rank > 1024) return LAWCAT_ERR_UNSUPPORTED;
  if ((long long)p->B * p->T > 0x7fffffffLL) return LAWCAT_ERR_UNSUPPORTED;
  const bool empty = (size_t)p->B * p->T == 0;
  const void* const req[] = {x, gate};
  const void* const opt[] = {bias, ws};
  if ((r = check_ptrs(req, opt, empty))) return r;
  if (!A1 || !A2 || !aligned16(A1) || !aligned16(A2)) return LAWCAT_ERR_INVALID_ARG;
  const size_t need = lawcat_gate_fn_workspace_bytes(p, d_model, rank);
  if (need && !empty && (!ws || ws_bytes < need)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  Ctx c{p, (cudaStream_t)stream, dev_status};
  return launch_gate_fn(c, d_model, rank, x, A1, A2, bias, gate, ws);
}

int lawcat_conv_bwd(const lawcat_params* p, const void* q, const void* k, const void* w_q, const void* w_k,
                    const void* W, const void* cache_q, const void* cache_k, const void* d_qdot,
                    const void* d_kdot, void* dq, void* dk, float* dw_q, float* dw_k, float* dW, void* ws,
                    size_t ws_bytes, void* stream, int* dev_status) {
  int r = check_params(p, true);
  if (r) return r;
  const void* const req[] = {q, k, w_q, w_k, d_qdot, d_kdot};
  const void* const opt[] = {W, cache_q, cache_k, dq, dk, dw_q, dw_k, dW, ws};
  if ((r = check_ptrs(req, opt))) return r;
  if ((W == nullptr) != (dW == nullptr) && W == nullptr) return LAWCAT_ERR_INVALID_ARG;  // dW without W
  if (W) {
    const size_t need = lawcat_workspace_bytes(p, LAWCAT_OP_CONV_BWD);
    if (need && (!ws || ws_bytes < need)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  }
  Ctx c{p, (cudaStream_t)stream, dev_status};
  return launch_conv_bwd(c, q, k, w_q, w_k, W, cache_q, cache_k, d_qdot, d_kdot, dq, dk, dw_q, dw_k, dW, ws);
}

int lawcat_gla_fwd(const lawcat_params* p, const void* qdot, const void* kdot, const void* v, const void* gate,
                   const float* S0, const float* z0, void* o, float* den, float* S_T, float* z_T, void* ws,
                   size_t ws_bytes, void* stream, int* dev_status) {
  (void)ws; (void)ws_bytes;
  int r = check_params(p, true);
  if (r) return r;
  const void* const req[] = {qdot, kdot, v, gate, o};
  const void* const opt[] = {S0, z0, den, S_T, z_T};
  if ((r = check_ptrs(req, opt, (size_t)p->B * p->T == 0))) return r;
  Ctx c{p, (cudaStream_t)stream, dev_status};
  if ((size_t)p->B * p->T != 0 && gla_tc_supported(*p))  // chunkwise tensor-core kernel
    return launch_gla_fwd_tc(c, qdot, kdot, v, gate, S0, z0, o, den, S_T, z_T);
  return launch_gla_fwd_rec(c, qdot, kdot, false, v, gate, S0, z0, o, den, S_T, z_T);
}

int lawcat_gla_bwd(const lawcat_params* p, const void* qdot, const void* kdot, const void* v, const void* gate,
                   const float* S0, const float* z0, const void* o, const float* den, const void* dO,
                   void* d_qdot, void* d_kdot, void* dv, void* dgate, void* ws, size_t ws_bytes, void* stream,
                   int* dev_status) {
  int r = check_params(p, true);
  if (r) return r;
  const void* const req[] = {qdot, kdot, v, gate, dO, d_qdot, d_kdot, dv, dgate};
  const void* const opt[] = {S0, z0, o, den, ws};
  if ((r = check_ptrs(req, opt))) return r;
  const size_t need = lawcat_workspace_bytes(p, LAWCAT_OP_GLA_BWD);
  if (need && (!ws || ws_bytes < need)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  Ctx c{p, (cudaStream_t)stream, dev_status};
  if ((size_t)p->B * p->T != 0 && gla_tc_bwd_supported(*p))  // chunkwise tensor-core kernel
    return launch_gla_bwd_tc(c, qdot, kdot, v, gate, S0, z0, dO, d_qdot, d_kdot, dv, dgate, ws, false);
  return launch_gla_bwd_rec(c, qdot, kdot, v, gate, S0, z0, o, den, dO, d_qdot, d_kdot, dv, dgate, ws);
}

int lawcat_layer_fwd(const lawcat_params* p, const void* q, const void* k, const void* v, const void* gate,
                     const void* w_q, const void* w_k, const void* W, const void* cache_q_in,
                     const void* cache_k_in, const float* S0, const float* z0, void* o, void* cache_q_out,
                     void* cache_k_out, float* S_T, float* z_T, void* ws, size_t ws_bytes, void* stream,
                     int* dev_status) {
  int r = check_params(p, true);
  if (r) return r;
  const void* const req[] = {q, k, v, gate, w_q, w_k, W, o};
  const void* const opt[] = {cache_q_in, cache_k_in, S0, z0, cache_q_out, cache_k_out, S_T, z_T, ws};
  if ((r = check_ptrs(req, opt, (size_t)p->B * p->T == 0))) return r;
  if ((cache_q_out && cache_q_out == cache_q_in) || (cache_k_out && cache_k_out == cache_k_in))
    return LAWCAT_ERR_INVALID_ARG;
  const size_t need = lawcat_workspace_bytes(p, LAWCAT_OP_LAYER_FWD);
  if (need && (!ws || ws_bytes < need)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  Ctx c{p, (cudaStream_t)stream, dev_status};
  if (layer_tc_supported(*p)) {  // chunkwise tensor-core kernel
    // (the kernel also writes the conv caches after the last token)
    return launch_layer_tc(c, q, k, v, gate, w_q, w_k, W, cache_q_in, cache_k_in, S0, z0, o, cache_q_out, cache_k_out, S_T,
                           z_T, ws);
  }
  float* qdot = (float*)ws;
  float* kdot = (float*)((char*)ws + align_up(sizeof(float) * elems(p, p->H, p->d_k), 256));
  // The feature maps of Section 2 other than the softmax (1 + ELU, identity) on head width 64: tensor-core conv + mix +
  // phi into fp32 scratch, then the chunkwise tensor-core attention on those features.
  if ((size_t)p->B * p->T != 0 && (p->phi != LAWCAT_PHI_SOFTMAX || p->mix_unshared) && p->chunk != 1 &&
      convmix_tc_fwd_supported(*p) && gla_tc_supported(*p)) {
    if ((r = launch_convmix_tc_fwd(c, q, k, w_q, w_k, W, cache_q_in, cache_k_in, qdot, kdot, true))) return r;
    if ((r = launch_gla_fwd_tc(c, qdot, kdot, v, gate, S0, z0, o, nullptr, S_T, z_T, true))) return r;
    return launch_cache_out(c, q, k, cache_q_in, cache_k_in, cache_q_out, cache_k_out);
  }
  // exact path: conv + mix + phi into fp32 scratch, then the recurrent GLA
  if ((r = launch_convmix_fwd(c, q, k, w_q, w_k, W, cache_q_in, cache_k_in, qdot, kdot, true, true))) return r;
  if ((r = launch_gla_fwd_rec(c, qdot, kdot, true, v, gate, S0, z0, o, nullptr, S_T, z_T))) return r;
  return launch_cache_out(c, q, k, cache_q_in, cache_k_in, cache_q_out, cache_k_out);
}

size_t lawcat_layer_fwd_varlen_workspace_bytes(const lawcat_params* p, const int32_t* cu_seqlens, int nseq) {
  if (check_params(p, true) != LAWCAT_OK || !cu_seqlens || nseq < 0) return 0;
  size_t need = 0;
  for (int i = 0; i < nseq; ++i) {
    lawcat_params pi = *p;
    pi.B = 1;
    pi.T = cu_seqlens[i + 1] - cu_seqlens[i];
    if (pi.T <= 0) continue;
    const size_t n = lawcat_workspace_bytes(&pi, LAWCAT_OP_LAYER_FWD);
    if (n > need) need = n;
  }
  return need;
}

int lawcat_layer_fwd_varlen(const lawcat_params* p, const int32_t* cu_seqlens, int nseq, const void* q, const void* k,
                            const void* v, const void* gate, const void* w_q, const void* w_k, const void* W,
                            const void* cache_q_in, const void* cache_k_in, const float* S0, const float* z0, void* o,
                            void* cache_q_out, void* cache_k_out, float* S_T, float* z_T, void* ws, size_t ws_bytes,
                            void* stream, int* dev_status) {
  int r = check_params(p, true);
  if (r) return r;
  if (p->B != 1 || !cu_seqlens || nseq < 0) return LAWCAT_ERR_INVALID_ARG;
  if (cu_seqlens[0] != 0 || cu_seqlens[nseq] != p->T) return LAWCAT_ERR_INVALID_ARG;
  for (int i = 0; i < nseq; ++i)
    if (cu_seqlens[i + 1] < cu_seqlens[i]) return LAWCAT_ERR_INVALID_ARG;
  if (ws_bytes < lawcat_layer_fwd_varlen_workspace_bytes(p, cu_seqlens, nseq)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  const size_t es = p->dtype == LAWCAT_F32 ? 4 : 2;
  const size_t nS = (size_t)p->H * p->d_k * p->d_v, nz = (size_t)p->H * p->d_k;
  const size_t ncq = (size_t)(p->conv_k - 1) * p->H * p->d_k * es, nck = (size_t)(p->conv_k - 1) * p->H_kv * p->d_k * es;
  auto at = [](const void* base, size_t bytes) -> const void* { return base ? (const char*)base + bytes : nullptr; };
  auto atw = [](void* base, size_t bytes) -> void* { return base ? (char*)base + bytes : nullptr; };
  cudaStream_t st = (cudaStream_t)stream;
  for (int i = 0; i < nseq; ++i) {
    const size_t t0 = (size_t)cu_seqlens[i];
    lawcat_params pi = *p;
    pi.T = cu_seqlens[i + 1] - cu_seqlens[i];
    const float* S0i = S0 ? S0 + i * nS : nullptr;
    const float* z0i = z0 ? z0 + i * nz : nullptr;
    float* STi = S_T ? S_T + i * nS : nullptr;
    float* zTi = z_T ? z_T + i * nz : nullptr;
    if (pi.T == 0) {  // an empty sequence hands its state and caches through
      auto pass = [&](void* dst, const void* src, size_t bytes) -> bool {
        if (!dst || !bytes) return true;
        return (src ? cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) : cudaMemsetAsync(dst, 0, bytes, st)) == cudaSuccess;
      };
      if (!pass(STi, S0i, nS * 4) || !pass(zTi, z0i, nz * 4) || !pass(atw(cache_q_out, i * ncq), at(cache_q_in, i * ncq), ncq) ||
          !pass(atw(cache_k_out, i * nck), at(cache_k_in, i * nck), nck))
        return LAWCAT_ERR_CUDA;
      continue;
    }
    r = lawcat_layer_fwd(&pi, at(q, t0 * p->H * p->d_k * es), at(k, t0 * p->H_kv * p->d_k * es), at(v, t0 * p->H_kv * p->d_v * es),
                         at(gate, t0 * p->H * p->gate_dim * es), w_q, w_k, W, at(cache_q_in, i * ncq), at(cache_k_in, i * nck),
                         S0i, z0i, atw(o, t0 * p->H * p->d_v * es), atw(cache_q_out, i * ncq), atw(cache_k_out, i * nck), STi,
                         zTi, ws, ws_bytes, stream, dev_status);
    if (r) return r;
  }
  return LAWCAT_OK;
}

int lawcat_layer_bwd(const lawcat_params* p, const void* q, const void* k, const void* v, const void* gate,
                     const void* w_q, const void* w_k, const void* W, const void* cache_q, const void* cache_k,
                     const float* S0, const float* z0, const void* dO, void* dq, void* dk, void* dv, void* dgate,
                     float* dw_q, float* dw_k, float* dW, void* ws, size_t ws_bytes, void* stream, int* dev_status) {
  int r = check_params(p, true);
  if (r) return r;
  const void* const req[] = {q, k, v, gate, w_q, w_k, W, dO, dq, dk, dv, dgate, dw_q, dw_k, dW};
  const void* const opt[] = {cache_q, cache_k, S0, z0, ws};
  if ((r = check_ptrs(req, opt))) return r;
  const size_t need = lawcat_workspace_bytes(p, LAWCAT_OP_LAYER_BWD);
  if (need && (!ws || ws_bytes < need)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  Ctx c{p, (cudaStream_t)stream, dev_status};
  if ((size_t)p->B * p->T != 0 && layer_bwd_tc(*p)) {
    char* w = (char*)ws;
    const size_t nf = align_up(4 * elems(p, p->H, p->d_k), 256);
    void* qd = w; void* kd = w + nf; void* dqd = w + 2 * nf; void* dkd = w + 3 * nf;
    void* ws_g = w + 4 * nf;
    void* ws_c = (char*)ws_g + lawcat_workspace_bytes(p, LAWCAT_OP_GLA_BWD);
    // features recomputed in fp32, attention backward on them (it runs its own forward sweep), mix / softmax / conv backward
    if ((r = launch_convmix_tc_fwd(c, q, k, w_q, w_k, W, cache_q, cache_k, qd, kd, true))) return r;
    if ((r = launch_gla_bwd_tc(c, qd, kd, v, gate, S0, z0, dO, dqd, dkd, dv, dgate, ws_g, true))) return r;
    return launch_conv_bwd(c, q, k, w_q, w_k, W, cache_q, cache_k, dqd, dkd, dq, dk, dw_q, dw_k, dW, ws_c, true);
  }
  // exact kernels, the whole chain in fp32
  const ExactBwdLayout L = exact_bwd_layout(p);
  char* w = (char*)ws;
  lawcat_params p32 = *p;
  p32.dtype = LAWCAT_F32;
  p32.chunk = 1;
  Ctx c32{&p32, (cudaStream_t)stream, dev_status};
  const void* in[10] = {q, k, v, gate, w_q, w_k, W, dO, cache_q, cache_k};
  void* out[4] = {dq, dk, dv, dgate};
  const size_t n_in[10] = {elems(p, p->H, p->d_k), elems(p, p->H_kv, p->d_k), elems(p, p->H_kv, p->d_v),
                           elems(p, p->H, p->gate_dim), (size_t)p->H * p->d_k * p->conv_k,
                           (size_t)p->H_kv * p->d_k * p->conv_k, (size_t)(1 + p->mix_unshared) * p->H * p->d_k * p->d_k,
                           elems(p, p->H, p->d_v),
                           (size_t)p->B * (p->conv_k - 1) * p->H * p->d_k, (size_t)p->B * (p->conv_k - 1) * p->H_kv * p->d_k};
  const bool widen = p->dtype == LAWCAT_BF16;
  if (widen) {
    for (int i = 0; i < 10; ++i) {
      if (!in[i] || !n_in[i]) continue;
      LAWCAT_LAUNCH("widen", c.stream, widen_kernel<<<(unsigned)((n_in[i] + 255) / 256), 256, 0, c.stream>>>(
                                           (const bf16*)in[i], (float*)(w + L.in[i]), n_in[i]));
      LAWCAT_CHECK_LAUNCH();
      in[i] = w + L.in[i];
    }
    for (int i = 0; i < 4; ++i) out[i] = w + L.out[i];
  }
  if ((size_t)p->B * p->T != 0) {
    if ((r = launch_convmix_fwd(c32, in[0], in[1], in[4], in[5], in[6], in[8], in[9], w + L.qd, w + L.kd, false, true))) return r;
    if ((r = launch_gla_fwd_rec(c32, w + L.qd, w + L.kd, false, in[2], in[3], S0, z0, w + L.o, (float*)(w + L.den), nullptr, nullptr))) return r;
    if ((r = launch_gla_bwd_rec(c32, w + L.qd, w + L.kd, in[2], in[3], S0, z0, w + L.o, (const float*)(w + L.den), in[7],
                                w + L.dqd, w + L.dkd, out[2], out[3], w + L.ws_g)))
      return r;
  }
  if ((r = launch_conv_bwd(c32, in[0], in[1], in[4], in[5], in[6], in[8], in[9], w + L.dqd, w + L.dkd, out[0], out[1], dw_q,
                           dw_k, dW, w + L.ws_c, false)))
    return r;
  if (widen) {
    void* dst[4] = {dq, dk, dv, dgate};
    for (int i = 0; i < 4; ++i) {
      if (!n_in[i]) continue;
      LAWCAT_LAUNCH("narrow", c.stream, narrow_kernel<<<(unsigned)((n_in[i] + 255) / 256), 256, 0, c.stream>>>(
                                            (const float*)out[i], (bf16*)dst[i], n_in[i]));
      LAWCAT_CHECK_LAUNCH();
    }
  }
  return LAWCAT_OK;
}

int lawcat_decode_step(const lawcat_params* p, const void* q_t, const void* k_t, const void* v_t,
                       const void* gate_t, const void* w_q, const void* w_k, const void* W, float* S, float* z,
                       void* cache_q, void* cache_k, void* o_t, void* ws, size_t ws_bytes, void* stream,
                       int* dev_status) {
  int r = check_params(p, false);
  if (r) return r;
  const void* const req[] = {q_t, k_t, v_t, gate_t, w_q, w_k, W, S, z, o_t};
  const void* const opt[] = {cache_q, cache_k, ws};
  if ((r = check_ptrs(req, opt))) return r;
  if (p->conv_k > 1 && (!cache_q || !cache_k)) return LAWCAT_ERR_INVALID_ARG;
  const size_t need = lawcat_workspace_bytes(p, LAWCAT_OP_DECODE_STEP);
  if (need && (!ws || ws_bytes < need)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  Ctx c{p, (cudaStream_t)stream, dev_status};
  return launch_decode(c, q_t, k_t, v_t, gate_t, w_q, w_k, W, S, z, cache_q, cache_k, o_t, ws);
}

// ---- host-buffer variant of the layer forward ---------------------------------------------------------------------
// The sequence is cut into slices along T (per batch element); the copies of slice i+1 to the device, the layer on
// slice i (which starts from the state and conv caches slice i-1 left) and the copy of slice i-1's output back run
// on three streams, so that the step costs about its host-to-device copies alone.
constexpr int HOST_SLICE = 2048;  // tokens per slice (a multiple of the chunk)

struct HostStateSet { size_t S, z, cq, ck, bytes; };
static HostStateSet host_state_set(const lawcat_params* p) {
  const size_t es = p->dtype == LAWCAT_F32 ? 4 : 2;
  HostStateSet h;
  size_t o = 0;
  h.S = o; o += align_up(sizeof(float) * (size_t)p->H * p->d_k * p->d_v, 256);
  h.z = o; o += align_up(sizeof(float) * (size_t)p->H * p->d_k, 256);
  h.cq = o; o += align_up(es * (size_t)(p->conv_k - 1) * p->H * p->d_k, 256);
  h.ck = o; o += align_up(es * (size_t)(p->conv_k - 1) * p->H_kv * p->d_k, 256);
  h.bytes = o;
  return h;
}
static lawcat_params host_slice_params(const lawcat_params* p, int len) {
  lawcat_params ps = *p;
  ps.B = 1;
  ps.T = len;
  return ps;
}
// off[0..8]: q, k, v, gate, w_q, w_k, W, o, workspace; off[9]: two state sets (ping-pong between slices); off[10]: end
static size_t host_arena_layout(const lawcat_params* p, size_t off[11]) {
  const size_t es = p->dtype == LAWCAT_F32 ? 4 : 2;
  const lawcat_params ps = host_slice_params(p, p->T < HOST_SLICE ? p->T : HOST_SLICE);
  size_t ws = lawcat_workspace_bytes(p, LAWCAT_OP_LAYER_FWD);
  const size_t ws_slice = lawcat_workspace_bytes(&ps, LAWCAT_OP_LAYER_FWD);
  if (ws_slice > ws) ws = ws_slice;
  const size_t n[10] = {elems(p, p->H, p->d_k) * es,      // q
                        elems(p, p->H_kv, p->d_k) * es,   // k
                        elems(p, p->H_kv, p->d_v) * es,   // v
                        elems(p, p->H, p->gate_dim) * es, // gate
                        (size_t)p->H * p->d_k * p->conv_k * es, (size_t)p->H_kv * p->d_k * p->conv_k * es,
                        (size_t)(1 + p->mix_unshared) * p->H * p->d_k * p->d_k * es,  // w_q, w_k, W
                        elems(p, p->H, p->d_v) * es,      // o
                        ws, 2 * host_state_set(p).bytes};
  size_t o = 0;
  for (int i = 0; i < 10; ++i) {
    off[i] = o;
    o += align_up(n[i], 256);
  }
  off[10] = o;
  return o;
}

// copy streams and events of the host path, one set per device, created on first use and kept
struct HostPipe {
  std::mutex mu;  // held while a call enqueues: the events are shared by every caller on the device
  cudaStream_t in = nullptr, out = nullptr;
  std::vector<cudaEvent_t> ev;
  cudaEvent_t event(size_t i) {
    while (ev.size() <= i) {
      cudaEvent_t e;
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
      ev.push_back(e);
    }
    return ev[i];
  }
};
static HostPipe* host_pipe() {
  static std::mutex mu;
  static HostPipe pipes[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  HostPipe& hp = pipes[dev];
  if (!hp.in) {
    if (cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  }
  return &hp;
}

size_t lawcat_layer_fwd_host_arena_bytes(const lawcat_params* p) {
  if (check_params(p, true) != LAWCAT_OK) return 0;
  size_t off[11];
  return host_arena_layout(p, off);
}

int lawcat_layer_fwd_host(const lawcat_params* p, const void* h_q, const void* h_k, const void* h_v,
                          const void* h_gate, const void* h_w_q, const void* h_w_k, const void* h_W, void* h_o,
                          void* arena, size_t arena_bytes, void* stream) {
  int r = check_params(p, true);
  if (r) return r;
  if (!h_q || !h_k || !h_v || !h_gate || !h_w_q || !h_w_k || !h_W || !h_o || !arena || !aligned16(arena))
    return LAWCAT_ERR_INVALID_ARG;
  size_t off[11];
  if (arena_bytes < host_arena_layout(p, off)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  if (p->B * p->T == 0) return LAWCAT_OK;
  HostPipe* hp = host_pipe();
  if (!hp) return LAWCAT_ERR_CUDA;
  std::lock_guard<std::mutex> hold(hp->mu);
  char* a = (char*)arena;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t es = p->dtype == LAWCAT_F32 ? 4 : 2;
#define LAWCAT_HOST_TRY(x) do { if ((x) != cudaSuccess) return LAWCAT_ERR_CUDA; } while (0)
  size_t ne = 0;
  // both copy streams start behind whatever the caller's stream holds (an earlier call may still use the arena)
  cudaEvent_t e0 = hp->event(ne++);
  if (!e0) return LAWCAT_ERR_CUDA;
  LAWCAT_HOST_TRY(cudaEventRecord(e0, st));
  LAWCAT_HOST_TRY(cudaStreamWaitEvent(hp->in, e0, 0));
  LAWCAT_HOST_TRY(cudaStreamWaitEvent(hp->out, e0, 0));
  const void* wsrc[3] = {h_w_q, h_w_k, h_W};
  const size_t wnb[3] = {(size_t)p->H * p->d_k * p->conv_k * es, (size_t)p->H_kv * p->d_k * p->conv_k * es,
                         (size_t)(1 + p->mix_unshared) * p->H * p->d_k * p->d_k * es};
  for (int i = 0; i < 3; ++i)
    LAWCAT_HOST_TRY(cudaMemcpyAsync(a + off[4 + i], wsrc[i], wnb[i], cudaMemcpyHostToDevice, hp->in));
  const HostStateSet hs = host_state_set(p);
  // bytes per token of the four streams and of the output
  const size_t row[4] = {(size_t)p->H * p->d_k * es, (size_t)p->H_kv * p->d_k * es, (size_t)p->H_kv * p->d_v * es,
                         (size_t)p->H * p->gate_dim * es};
  const size_t orow = (size_t)p->H * p->d_v * es;
  const void* src[4] = {h_q, h_k, h_v, h_gate};
  for (int b = 0; b < p->B; ++b) {
    int set = 0;
    for (int t0 = 0; t0 < p->T; t0 += HOST_SLICE) {
      const int len = p->T - t0 < HOST_SLICE ? p->T - t0 : HOST_SLICE;
      const size_t tok = (size_t)b * p->T + t0;
      for (int i = 0; i < 4; ++i)
        LAWCAT_HOST_TRY(cudaMemcpyAsync(a + off[i] + tok * row[i], (const char*)src[i] + tok * row[i], (size_t)len * row[i],
                                        cudaMemcpyHostToDevice, hp->in));
      cudaEvent_t e_in = hp->event(ne++), e_done = hp->event(ne++);
      if (!e_in || !e_done) return LAWCAT_ERR_CUDA;
      LAWCAT_HOST_TRY(cudaEventRecord(e_in, hp->in));
      LAWCAT_HOST_TRY(cudaStreamWaitEvent(st, e_in, 0));
      const lawcat_params ps = host_slice_params(p, len);
      char* prev = a + off[9] + (size_t)(set ^ 1) * hs.bytes;
      char* next = a + off[9] + (size_t)set * hs.bytes;
      const bool first = t0 == 0, last = t0 + len >= p->T, cache = p->conv_k > 1;
      r = lawcat_layer_fwd(&ps, a + off[0] + tok * row[0], a + off[1] + tok * row[1], a + off[2] + tok * row[2],
                           a + off[3] + tok * row[3], a + off[4], a + off[5], a + off[6],
                           (first || !cache) ? nullptr : prev + hs.cq, (first || !cache) ? nullptr : prev + hs.ck,
                           first ? nullptr : (const float*)(prev + hs.S), first ? nullptr : (const float*)(prev + hs.z),
                           a + off[7] + tok * orow, (last || !cache) ? nullptr : next + hs.cq,
                           (last || !cache) ? nullptr : next + hs.ck, last ? nullptr : (float*)(next + hs.S),
                           last ? nullptr : (float*)(next + hs.z), a + off[8], off[9] - off[8], stream, nullptr);
      if (r) return r;
      LAWCAT_HOST_TRY(cudaEventRecord(e_done, st));
      LAWCAT_HOST_TRY(cudaStreamWaitEvent(hp->out, e_done, 0));
      LAWCAT_HOST_TRY(cudaMemcpyAsync((char*)h_o + tok * orow, a + off[7] + tok * orow, (size_t)len * orow,
                                      cudaMemcpyDeviceToHost, hp->out));
      set ^= 1;
    }
  }
  // the caller's stream ends behind the last copy back
  cudaEvent_t e_end = hp->event(ne++);
  if (!e_end) return LAWCAT_ERR_CUDA;
  LAWCAT_HOST_TRY(cudaEventRecord(e_end, hp->out));
  LAWCAT_HOST_TRY(cudaStreamWaitEvent(st, e_end, 0));
#undef LAWCAT_HOST_TRY
  return LAWCAT_OK;
}

}  // extern "C"
