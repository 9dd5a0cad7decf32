// Scaled Adam step for callers that cannot provide a workspace.
//
// scalify_scaled_adam_step needs a few bytes of scratch per tensor (the old scale words and
// the reciprocals of the new ones, which the update kernel reads while the scale words are
// being overwritten) plus a status word, and it takes them from a caller-allocated
// workspace.  Some callers have no way to allocate one: code that runs after the
// application has handed the whole device to its own memory pool, so that a further
// cudaMalloc fails; code on a latency-critical path, where cudaMalloc's implicit
// device-wide synchronisation is not acceptable; and plug-in style integrations that are
// only ever given the tensors themselves.  For them this file keeps the scratch in a
// fixed-size array that is part of the library image on every GPU that loads it.
#include <mutex>

#include "scalify_common.cuh"
#include "scalify_launch.h"

namespace scalify {

constexpr int kStaticAdamMaxTensors = 1024;
// header (status word) + 32 bytes per tensor + slack, see adam_ws_bytes()
constexpr size_t kStaticAdamBytes = kWsHeader + size_t(kStaticAdamMaxTensors) * 32 + 256;

// Lives in device memory of every GPU that loads the library, from load until exit (33 KB).
static __device__ __align__(256) unsigned char g_static_adam_scratch[kStaticAdamBytes];

// In host code the name above is only a handle for the runtime, not a device address: the
// address on the current device has to be asked for, once per device.
static std::mutex g_static_mutex;
static void* g_static_ptr[64] = {nullptr};

static int static_scratch_ptr(void** out) {
  int dev = 0;
  SCALIFY_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SCALIFY_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    SCALIFY_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_adam_scratch));
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return SCALIFY_OK;
}

}  // namespace scalify

using namespace scalify;

extern "C" int scalify_scaled_adam_step_static(int n_tensors, const scalify_array* grads, scalify_array* m,
                                               scalify_array* v, scalify_array* w, float lr, float beta1,
                                               float beta2, float eps, int64_t step, uint32_t* status_out,
                                               void* stream) {
  if (n_tensors < 0) return SCALIFY_ERR_VALUE;
  if (n_tensors == 0) return SCALIFY_OK;
  if (n_tensors > kStaticAdamMaxTensors) return SCALIFY_ERR_WORKSPACE;  // more tensors than the fixed scratch holds
  if (adam_ws_bytes(n_tensors) > kStaticAdamBytes) return SCALIFY_ERR_WORKSPACE;
  if (!grads || !m || !v || !w) return SCALIFY_ERR_NULL;
  if (step < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f) || !isfinite(lr))
    return SCALIFY_ERR_VALUE;
  int64_t numel[kStaticAdamMaxTensors];
  for (int i = 0; i < n_tensors; ++i) {
    int rc;
    if ((rc = check_array(&grads[i])) || (rc = check_array(&m[i])) || (rc = check_array(&v[i])) ||
        (rc = check_array(&w[i])))
      return rc;
    if (!m[i].scale || !v[i].scale || !w[i].scale) return SCALIFY_ERR_NULL;
    if (grads[i].dtype != grads[0].dtype || m[i].dtype != m[0].dtype || v[i].dtype != m[0].dtype ||
        w[i].dtype != w[0].dtype)
      return SCALIFY_ERR_DTYPE;
    if (!(m[i].dtype == SCALIFY_F16 || m[i].dtype == SCALIFY_F32) || !is_wide(w[i].dtype)) return SCALIFY_ERR_DTYPE;
    const int64_t n = contiguous_numel(&grads[i]);
    if (n < 0 || contiguous_numel(&m[i]) != n || contiguous_numel(&v[i]) != n || contiguous_numel(&w[i]) != n)
      return SCALIFY_ERR_SHAPE;
    if (m[i].scale == v[i].scale || m[i].scale == w[i].scale || v[i].scale == w[i].scale ||
        grads[i].scale == m[i].scale || grads[i].scale == v[i].scale || grads[i].scale == w[i].scale)
      return SCALIFY_ERR_ALIAS;
    numel[i] = n;
  }
  const void* words[kStaticAdamMaxTensors * 4];  // (on the stack: this call allocates nothing, on the host either)
  int rc = check_adam_scale_words(n_tensors, grads, m, v, w, nullptr, words);
  if (rc) return rc;
  void* scratch = nullptr;
  rc = static_scratch_ptr(&scratch);
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the previous call left: the status word has to start at zero
  SCALIFY_CUDA_TRY(cudaMemsetAsync(scratch, 0, kWsHeader, st));
  rc = launch_adam(n_tensors, grads, m, v, w, nullptr, numel, lr, beta1, beta2, eps, step, scratch, st);
  if (rc) return rc;
  if (status_out)
    SCALIFY_CUDA_TRY(cudaMemcpyAsync(status_out, scratch, sizeof(uint32_t), cudaMemcpyDeviceToDevice, st));
  return SCALIFY_OK;
}
