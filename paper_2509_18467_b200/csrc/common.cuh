// Shared device/host helpers of the LAWCAT CUDA library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lawcat.h"

namespace lawcat {

typedef __nv_bfloat16 bf16;

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<bf16>(const bf16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<bf16>(bf16* p, float v) { *p = __float2bfloat16_rn(v); }

// Log-decay of one gate entry (Section 4.2: sigmoid gate). LOGITS: logsigmoid(a) / tau, LOGDECAY: a itself.
__device__ __forceinline__ float log_decay(float a, int gate_mode, float inv_tau) {
  if (gate_mode == LAWCAT_GATE_LOGDECAY) return a;
  float ls = fminf(a, 0.f) - log1pf(expf(-fabsf(a)));
  return ls * inv_tau;
}
// d(log-decay)/d(gate entry)
__device__ __forceinline__ float log_decay_grad(float a, int gate_mode, float inv_tau) {
  if (gate_mode == LAWCAT_GATE_LOGDECAY) return 1.f;
  return (1.f - 1.f / (1.f + expf(-a))) * inv_tau;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- host-side launchers implemented in the .cu files (all return a lawcat_status) -------------------------------
struct Ctx {
  const lawcat_params* p;
  cudaStream_t stream;
  int* dev_status;
};

int launch_conv_plain(const Ctx& c, const void* x, const void* w, const void* cache, void* out, int NH);
// (exact: the fp32 CUDA-core kernel even where the tensor-core one applies)
int launch_convmix_fwd(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                       const void* cache_q, const void* cache_k, void* qdot, void* kdot, bool out_f32, bool exact);
// (grads_f32: d_qdot, d_kdot are fp32 scratch of the fused layer backward; only on the tensor-core path)
int launch_conv_bwd(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                    const void* cache_q, const void* cache_k, const void* d_qdot, const void* d_kdot, void* dq,
                    void* dk, float* dw_q, float* dw_k, float* dW, void* ws, bool grads_f32 = false);
int launch_cache_out(const Ctx& c, const void* q, const void* k, const void* cache_q_in, const void* cache_k_in,
                     void* cache_q_out, void* cache_k_out);
int launch_gla_fwd_rec(const Ctx& c, const void* qdot, const void* kdot, bool qk_f32, const void* v,
                       const void* gate, const float* S0, const float* z0, void* o, float* den, float* S_T,
                       float* z_T);
int launch_gla_bwd_rec(const Ctx& c, const void* qdot, const void* kdot, const void* v, const void* gate,
                       const float* S0, const float* z0, const void* o, const float* den, const void* dO,
                       void* d_qdot, void* d_kdot, void* dv, void* dgate, void* ws);
int launch_decode(const Ctx& c, const void* q_t, const void* k_t, const void* v_t, const void* gate_t,
                  const void* w_q, const void* w_k, const void* W, float* S, float* z, void* cache_q, void* cache_k,
                  void* o_t, void* ws);
size_t decode_workspace_bytes(const lawcat_params& p);

// Host-side check of a parameter block (api.cu): LAWCAT_OK, LAWCAT_ERR_INVALID_ARG or LAWCAT_ERR_UNSUPPORTED.
int validate_params(const lawcat_params* p, bool need_T);

// Chunkwise tensor-core layer forward (layer_tc.cu): whether it takes these parameters, and its launcher.
bool layer_tc_supported(const lawcat_params& p);
int layer_tc_segments(const lawcat_params& p);
size_t layer_tc_workspace_bytes(const lawcat_params& p);
int launch_layer_tc(const Ctx& c, const void* q, const void* k, const void* v, const void* gate, const void* w_q,
                    const void* w_k, const void* W, const void* cache_q_in, const void* cache_k_in, const float* S0,
                    const float* z0, void* o, void* cache_q_out, void* cache_k_out, float* S_T, float* z_T, void* ws);

// Chunkwise tensor-core GLA on given features and its backward (gla_tc.cu).
bool gla_tc_supported(const lawcat_params& p);
bool gla_tc_bwd_supported(const lawcat_params& p);
size_t gla_tc_bwd_workspace_bytes(const lawcat_params& p);
int launch_gla_fwd_tc(const Ctx& c, const void* qdot, const void* kdot, const void* v, const void* gate, const float* S0,
                      const float* z0, void* o, float* den, float* S_T, float* z_T, bool feat_f32 = false);
int launch_gla_bwd_tc(const Ctx& c, const void* qdot, const void* kdot, const void* v, const void* gate, const float* S0,
                      const float* z0, const void* dO, void* d_qdot, void* d_kdot, void* dv, void* dgate, void* ws,
                      bool feat_f32);

// Tensor-core conv -> mix -> softmax and the chain rule back through mix and softmax (convmix_tc.cu).
bool convmix_tc_fwd_supported(const lawcat_params& p);
bool convmix_tc_bwd_supported(const lawcat_params& p);
int launch_convmix_tc_fwd(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                          const void* cache_q, const void* cache_k, void* qdot, void* kdot, bool out_f32);
int launch_convmix_tc_bwd(const Ctx& c, const void* q, const void* k, const void* w_q, const void* w_k, const void* W,
                          const void* cache_q, const void* cache_k, const void* d_qdot, const void* d_kdot, bool grads_f32,
                          float* du_q, float* du_k, float* dW);

// The gate function in front of the layer: two consecutive low-rank linear layers producing the gate logits (gate_fn.cu).
bool gate_fn_tc_supported(const lawcat_params& p, int d_model, int rank);
size_t gate_fn_workspace_bytes(const lawcat_params& p, int d_model, int rank);
int launch_gate_fn(const Ctx& c, int d_model, int rank, const void* x, const void* A1, const void* A2, const void* bias,
                   void* gate, void* ws);

// Counts one kernel launch; while tracing is on it also brackets the launch with CUDA events on its stream.
struct LaunchScope {
  LaunchScope(const char* name, cudaStream_t s);
  ~LaunchScope();
  cudaStream_t stream;
  int idx;
};
#define LAWCAT_LAUNCH(name, strm, ...)       \
  do {                                       \
    ::lawcat::LaunchScope _ls(name, strm);   \
    __VA_ARGS__;                             \
  } while (0)

// Keeps the text of a CUDA runtime error (with the place that saw it) for lawcat_last_cuda_error(); per host thread.
void note_cuda_error(cudaError_t e, const char* file, int line);

#define LAWCAT_CHECK_LAUNCH()                                   \
  do {                                                          \
    const cudaError_t _e = cudaGetLastError();                  \
    if (_e != cudaSuccess) {                                    \
      ::lawcat::note_cuda_error(_e, __FILE__, __LINE__);        \
      return LAWCAT_ERR_CUDA;                                   \
    }                                                           \
  } while (0)

}  // namespace lawcat
