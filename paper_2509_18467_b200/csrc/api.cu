// The C ABI: argument validation on the host, then dispatch to the kernels. Nothing here allocates or synchronizes.
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
    return launch_gla_bwd_tc(c, qdot, kdot, v, gate, S0, z0, dO, d_qdot, d_kdot, dv, dgate, ws);
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
    if ((r = launch_layer_tc(c, q, k, v, gate, w_q, w_k, W, cache_q_in, cache_k_in, S0, z0, o, S_T, z_T, ws))) return r;
    return launch_cache_out(c, q, k, cache_q_in, cache_k_in, cache_q_out, cache_k_out);
  }
  // exact path: conv + mix + phi into fp32 scratch, then the recurrent GLA
  float* qdot = (float*)ws;
  float* kdot = (float*)((char*)ws + align_up(sizeof(float) * elems(p, p->H, p->d_k), 256));
  if ((r = launch_convmix_fwd(c, q, k, w_q, w_k, W, cache_q_in, cache_k_in, qdot, kdot, true, true))) return r;
  if ((r = launch_gla_fwd_rec(c, qdot, kdot, true, v, gate, S0, z0, o, nullptr, S_T, z_T))) return r;
  return launch_cache_out(c, q, k, cache_q_in, cache_k_in, cache_q_out, cache_k_out);
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
static size_t host_arena_layout(const lawcat_params* p, size_t off[10]) {
  const size_t es = p->dtype == LAWCAT_F32 ? 4 : 2;
  const size_t n[9] = {elems(p, p->H, p->d_k) * es,      // q
                       elems(p, p->H_kv, p->d_k) * es,   // k
                       elems(p, p->H_kv, p->d_v) * es,   // v
                       elems(p, p->H, p->gate_dim) * es, // gate
                       (size_t)p->H * p->d_k * p->conv_k * es, (size_t)p->H_kv * p->d_k * p->conv_k * es,
                       (size_t)p->H * p->d_k * p->d_k * es,  // w_q, w_k, W
                       elems(p, p->H, p->d_v) * es,      // o
                       lawcat_workspace_bytes(p, LAWCAT_OP_LAYER_FWD)};
  size_t o = 0;
  for (int i = 0; i < 9; ++i) {
    off[i] = o;
    o += align_up(n[i], 256);
  }
  off[9] = o;
  return o;
}

size_t lawcat_layer_fwd_host_arena_bytes(const lawcat_params* p) {
  if (check_params(p, true) != LAWCAT_OK) return 0;
  size_t off[10];
  return host_arena_layout(p, off);
}

int lawcat_layer_fwd_host(const lawcat_params* p, const void* h_q, const void* h_k, const void* h_v,
                          const void* h_gate, const void* h_w_q, const void* h_w_k, const void* h_W, void* h_o,
                          void* arena, size_t arena_bytes, void* stream) {
  int r = check_params(p, true);
  if (r) return r;
  if (!h_q || !h_k || !h_v || !h_gate || !h_w_q || !h_w_k || !h_W || !h_o || !arena || !aligned16(arena))
    return LAWCAT_ERR_INVALID_ARG;
  size_t off[10];
  if (arena_bytes < host_arena_layout(p, off)) return LAWCAT_ERR_WORKSPACE_TOO_SMALL;
  char* a = (char*)arena;
  cudaStream_t st = (cudaStream_t)stream;
  const void* src[7] = {h_q, h_k, h_v, h_gate, h_w_q, h_w_k, h_W};
  const size_t es = p->dtype == LAWCAT_F32 ? 4 : 2;
  const size_t nb[7] = {elems(p, p->H, p->d_k) * es, elems(p, p->H_kv, p->d_k) * es, elems(p, p->H_kv, p->d_v) * es,
                        elems(p, p->H, p->gate_dim) * es, (size_t)p->H * p->d_k * p->conv_k * es,
                        (size_t)p->H_kv * p->d_k * p->conv_k * es, (size_t)p->H * p->d_k * p->d_k * es};
  for (int i = 0; i < 7; ++i)
    if (nb[i] && cudaMemcpyAsync(a + off[i], src[i], nb[i], cudaMemcpyHostToDevice, st) != cudaSuccess)
      return LAWCAT_ERR_CUDA;
  r = lawcat_layer_fwd(p, a + off[0], a + off[1], a + off[2], a + off[3], a + off[4], a + off[5], a + off[6], nullptr,
                       nullptr, nullptr, nullptr, a + off[7], nullptr, nullptr, nullptr, nullptr, a + off[8],
                       off[9] - off[8], stream, nullptr);
  if (r) return r;
  const size_t no = elems(p, p->H, p->d_v) * es;
  if (no && cudaMemcpyAsync(h_o, a + off[7], no, cudaMemcpyDeviceToHost, st) != cudaSuccess) return LAWCAT_ERR_CUDA;
  return LAWCAT_OK;
}

}  // extern "C"
