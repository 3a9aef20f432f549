// Layer forward for callers that cannot allocate device memory: the scratch lives in a fixed device array that is part
// of the loaded library image.
#include <mutex>

#include "common.cuh"

using namespace lawcat;

namespace {

// Scratch for the conv+mix+phi outputs (qdot and kdot in fp32). Every GPU that loads the library carries this array
// until the process exits, so it is kept modest.
constexpr size_t kScratchBytes = LAWCAT_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// In host code the array's name is only a handle of the symbol; the address a kernel can use has to be asked for, per
// device, while that device is current.
int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LAWCAT_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return LAWCAT_ERR_CUDA;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return LAWCAT_OK;
}

}  // namespace

extern "C" {

size_t lawcat_noalloc_scratch_bytes(void) { return kScratchBytes; }

int lawcat_layer_fwd_noalloc(const lawcat_params* p, const void* q, const void* k, const void* v, const void* gate,
                             const void* w_q, const void* w_k, const void* W, const void* cache_q_in,
                             const void* cache_k_in, const float* S0, const float* z0, void* o, void* cache_q_out,
                             void* cache_k_out, float* S_T, float* z_T, void* stream, int* dev_status) {
  if (!p) return LAWCAT_ERR_INVALID_ARG;
  const int bad = validate_params(p, true);  // invalid argument vs unsupported shape; nothing is enqueued
  if (bad) return bad;
  // the exact path's scratch: two fp32 tensors [B,T,H,d_k]
  // (the limit is tested by division, factor by factor: the element count itself could wrap around in 64 bits)
  const size_t max_elems = kScratchBytes / (2 * sizeof(float));
  size_t room = max_elems;
  for (const size_t f : {(size_t)p->H, (size_t)p->d_k, (size_t)p->B, (size_t)p->T}) {
    if (f != 0 && room / f == 0) return LAWCAT_ERR_TOO_LARGE;
    if (f != 0) room /= f;
  }
  const size_t half = align_up(sizeof(float) * (size_t)p->B * (size_t)p->T * p->H * p->d_k, 256);
  if (2 * half > kScratchBytes) return LAWCAT_ERR_TOO_LARGE;
  const void* const req[] = {w_q, w_k, W};
  for (const void* x : req)
    if (!x) return LAWCAT_ERR_INVALID_ARG;
  const bool empty = (size_t)p->B * p->T == 0;
  if (!empty && (!q || !k || !v || !gate || !o)) return LAWCAT_ERR_INVALID_ARG;
  const void* const all[] = {q, k, v, gate, w_q, w_k, W, cache_q_in, cache_k_in, S0, z0, o, cache_q_out, cache_k_out,
                             S_T, z_T};
  for (const void* x : all)
    if (reinterpret_cast<uintptr_t>(x) & 15u) return LAWCAT_ERR_INVALID_ARG;
  if ((cache_q_out && cache_q_out == cache_q_in) || (cache_k_out && cache_k_out == cache_k_in))
    return LAWCAT_ERR_INVALID_ARG;
  void* scratch = nullptr;
  int r = scratch_for_current_device(&scratch);
  if (r) return r;
  Ctx c{p, (cudaStream_t)stream, dev_status};
  float* qdot = (float*)scratch;
  float* kdot = (float*)((char*)scratch + half);
  if ((r = launch_convmix_fwd(c, q, k, w_q, w_k, W, cache_q_in, cache_k_in, qdot, kdot, true, true))) return r;
  if ((r = launch_gla_fwd_rec(c, qdot, kdot, true, v, gate, S0, z0, o, nullptr, S_T, z_T))) return r;
  return launch_cache_out(c, q, k, cache_q_in, cache_k_in, cache_q_out, cache_k_out);
}

}  // extern "C"
