// C ABI entry points: argument validation and dispatch to the kernel launchers.
// Every check happens on the host before anything is enqueued.
#include <math.h>
#include <string.h>

#include <algorithm>

#include "scalify_common.cuh"
#include "scalify_launch.h"
#include <new>

namespace scalify {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }
int cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return SCALIFY_ERR_CUDA;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

int check_array(const scalify_array* a) {
  if (!a || !a->data) return SCALIFY_ERR_NULL;
  if (!valid_dtype(a->dtype)) return SCALIFY_ERR_DTYPE;
  if (a->ndim < 1 || a->ndim > 4) return SCALIFY_ERR_SHAPE;
  for (int i = 0; i < a->ndim; ++i)
    if (a->shape[i] < 0 || a->shape[i] > (int64_t(1) << 40)) return SCALIFY_ERR_SHAPE;
  if (a->stride[a->ndim - 1] != 1) return SCALIFY_ERR_ALIGNMENT;
  if (reinterpret_cast<uintptr_t>(a->data) % 16 != 0) return SCALIFY_ERR_ALIGNMENT;
  const int es = elem_size(a->dtype);
  for (int i = 0; i < a->ndim - 1; ++i) {
    if (a->stride[i] < 0) return SCALIFY_ERR_ALIGNMENT;
    if (a->shape[i] > 1 && (a->stride[i] * es) % 16 != 0) return SCALIFY_ERR_ALIGNMENT;
  }
#ifdef SCALIFY_DEBUG
  {
    // the bytes this array spans: every kernel access through the checked helpers must fall inside a registered span
    int64_t last = 0;
    bool empty = false;
    for (int i = 0; i < a->ndim; ++i) {
      if (a->shape[i] == 0) empty = true;
      else last += (a->shape[i] - 1) * a->stride[i];
    }
    if (!empty) dbg_register_range(a->data, static_cast<unsigned long long>(last + 1) * es);
  }
#endif
  return SCALIFY_OK;
}

int64_t contiguous_numel(const scalify_array* a) {
  int64_t n = 1;
  for (int i = a->ndim - 1; i >= 0; --i) {
    if (a->shape[i] != 1 && a->stride[i] != n) return -1;
    n *= a->shape[i];
  }
  return n;
}

static bool same_shape(const scalify_array* a, const scalify_array* b) {
  if (a->ndim != b->ndim) return false;
  for (int i = 0; i < a->ndim; ++i)
    if (a->shape[i] != b->shape[i]) return false;
  return true;
}

static bool valid_stat(int s) { return s == SCALIFY_STAT_NONE || s == SCALIFY_STAT_AMAX || s == SCALIFY_STAT_L2; }

// rows x cols view of a 2-D array (or 1-D as one row); row stride in elements
static int as_rows(const scalify_array* a, int64_t* rows, int64_t* cols, int64_t* ld) {
  if (a->ndim == 1) { *rows = 1; *cols = a->shape[0]; *ld = a->shape[0]; return SCALIFY_OK; }
  if (a->ndim == 2) { *rows = a->shape[0]; *cols = a->shape[1]; *ld = a->stride[0]; return SCALIFY_OK; }
  if (a->ndim == 3 && a->stride[0] == a->shape[1] * a->stride[1]) {
    *rows = a->shape[0] * a->shape[1]; *cols = a->shape[2]; *ld = a->stride[1];
    return SCALIFY_OK;
  }
  return SCALIFY_ERR_SHAPE;
}

}  // namespace scalify

using namespace scalify;

extern "C" {

int scalify_version(void) { return 100; }

int scalify_last_cuda_error(void) { return g_last_cuda_error; }

const char* scalify_status_string(int code) {
  switch (code) {
    case SCALIFY_OK: return "ok";
    case SCALIFY_ERR_NULL: return "a required pointer is NULL";
    case SCALIFY_ERR_DTYPE: return "dtype not valid for this argument";
    case SCALIFY_ERR_SHAPE: return "shapes inconsistent or out of range";
    case SCALIFY_ERR_ALIGNMENT: return "pointer or stride not 16-byte aligned, or innermost stride not 1";
    case SCALIFY_ERR_WORKSPACE: return "workspace missing or too small";
    case SCALIFY_ERR_UNSUPPORTED: return "combination not supported";
    case SCALIFY_ERR_CUDA: return "CUDA call failed (see scalify_last_cuda_error)";
    case SCALIFY_ERR_ALIAS: return "forbidden aliasing of scale words or buffers";
    case SCALIFY_ERR_VALUE: return "scalar argument out of range";
    default: return code > 0 ? "device status bits set" : "unknown error";
  }
}

size_t scalify_workspace_bytes(int op, int64_t d0, int64_t d1) {
  size_t n = kWsMin;
  const size_t stat_bytes = kWsHeader + size_t(sm_count()) * 8 * sizeof(double) + 256;
  switch (op) {
    case SCALIFY_OP_MATMUL: n = matmul_ws_bytes(d0, d1); break;
    case SCALIFY_OP_RESCALE:
    case SCALIFY_OP_STATISTIC:
      // one fp64 partial per block of the statistic pass over d0 elements (of at most 4 bytes)
      n = kWsHeader + size_t(statistic_blocks_wanted(d0 > 0 ? d0 : 0, 4)) * sizeof(double) + 256;
      break;
    case SCALIFY_OP_LAYERNORM_BWD: n = layernorm_bwd_ws_bytes(d0, d1); break;
    case SCALIFY_OP_ADAM: n = adam_ws_bytes(d0); break;
    case SCALIFY_OP_CROSS_ENTROPY: n = cross_entropy_ws_bytes(d0); break;
    case SCALIFY_OP_COLSUM: n = colsum_ws_bytes(d1); break;
    case SCALIFY_OP_MATMUL_SPLITK: n = matmul_splitk_ws_bytes(d0, d1); break;
    default: break;
  }
  if (n < stat_bytes) n = stat_bytes;
  return n < kWsMin ? kWsMin : n;
}

int scalify_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace) return SCALIFY_ERR_NULL;
  if (workspace_bytes < kWsMin || reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return SCALIFY_ERR_WORKSPACE;
  SCALIFY_CUDA_TRY(cudaMemsetAsync(workspace, 0, kWsHeader, static_cast<cudaStream_t>(stream)));
  return SCALIFY_OK;
}

int scalify_check_status(void* workspace, void* stream) {
  if (!workspace) return SCALIFY_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t bits = 0;
  SCALIFY_CUDA_TRY(cudaMemcpyAsync(&bits, workspace, sizeof(bits), cudaMemcpyDeviceToHost, st));
  SCALIFY_CUDA_TRY(cudaStreamSynchronize(st));
  if (bits) {
    SCALIFY_CUDA_TRY(cudaMemsetAsync(workspace, 0, sizeof(bits), st));
    SCALIFY_CUDA_TRY(cudaStreamSynchronize(st));
  }
  return static_cast<int>(bits & 0x7FFFFFFFu);
}

static int check_ws(void* ws, size_t bytes, size_t need) {
  if (!ws) return SCALIFY_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) % 256 != 0) return SCALIFY_ERR_WORKSPACE;
  if (bytes < need) return SCALIFY_ERR_WORKSPACE;
#ifdef SCALIFY_DEBUG
  dbg_register_range(ws, bytes);
#endif
  return SCALIFY_OK;
}

int scalify_statistic(const scalify_array* X, int stat, float* out_stat, void* workspace, size_t workspace_bytes,
                      void* stream) {
  int rc = check_array(X);
  if (rc) return rc;
  if (stat != SCALIFY_STAT_AMAX && stat != SCALIFY_STAT_L2) return SCALIFY_ERR_VALUE;
  const int64_t n = contiguous_numel(X);
  if (n < 0) return SCALIFY_ERR_SHAPE;
  rc = check_ws(workspace, workspace_bytes, kWsMin);
  if (rc) return rc;
  return launch_statistic(X->data, X->dtype, n, stat, workspace, workspace_bytes, out_stat,
                          static_cast<cudaStream_t>(stream));
}

int scalify_rescale(const scalify_array* X, int stat, const float* new_scale, const float* stat_in, scalify_array* Y,
                    void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_array(X);
  if (rc) return rc;
  rc = check_array(Y);
  if (rc) return rc;
  if (!valid_stat(stat)) return SCALIFY_ERR_VALUE;
  if (stat != SCALIFY_STAT_NONE && new_scale) return SCALIFY_ERR_VALUE;
  if (stat == SCALIFY_STAT_NONE && stat_in) return SCALIFY_ERR_VALUE;
  const int64_t n = contiguous_numel(X);
  if (n < 0 || contiguous_numel(Y) != n) return SCALIFY_ERR_SHAPE;
  if (Y->data == X->data && elem_size(X->dtype) != elem_size(Y->dtype)) return SCALIFY_ERR_ALIAS;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* status = workspace ? ws_view(workspace).status : nullptr;
  if (workspace && check_ws(workspace, workspace_bytes, kWsMin)) return SCALIFY_ERR_WORKSPACE;
  if (stat == SCALIFY_STAT_NONE) {
    if (new_scale) {
      if (Y->scale && Y->scale == X->scale) return SCALIFY_ERR_ALIAS;
      return launch_rebalance(X->data, X->dtype, Y->data, Y->dtype, n, X->scale, Y->scale, nullptr, new_scale,
                              kModeSet, status, st);
    }
    return launch_rebalance(X->data, X->dtype, Y->data, Y->dtype, n, X->scale, Y->scale, nullptr, nullptr, kModeCast,
                            status, st);
  }
  if (stat_in) {
    return launch_rebalance(X->data, X->dtype, Y->data, Y->dtype, n, X->scale, Y->scale, stat_in, nullptr,
                            kModeDynamic, status, st);
  }
  rc = check_ws(workspace, workspace_bytes, kWsMin);
  if (rc) return rc;
  // BF16 / F16 into an FP8 buffer of its own: the array is read once, the output written with the predicted
  // power of two, and a check launch repairs it if the prediction failed
  {
    const char* xb = static_cast<const char*>(X->data);
    const char* yb = static_cast<const char*>(Y->data);
    const bool disjoint = yb + n * elem_size(Y->dtype) <= xb || xb + n * elem_size(X->dtype) <= yb;
    if (disjoint && !(Y->scale && Y->scale == X->scale)) {
      rc = launch_rescale_predicted(X->data, X->dtype, Y->data, Y->dtype, n, stat, X->scale, Y->scale, workspace,
                                    workspace_bytes, st);
      if (rc <= 0) return rc;
    }
  }
  // one cooperative launch (statistic, grid barrier, rebalance); two launches where the device
  // cannot run a cooperative grid
  rc = launch_fused_rescale(X->data, X->dtype, Y->data, Y->dtype, n, stat, X->scale, Y->scale, workspace,
                            workspace_bytes, st);
  if (rc <= 0) return rc;
  rc = launch_statistic(X->data, X->dtype, n, stat, workspace, workspace_bytes, nullptr, st);
  if (rc) return rc;
  return launch_rebalance(X->data, X->dtype, Y->data, Y->dtype, n, X->scale, Y->scale, ws_view(workspace).stat,
                          nullptr, kModeDynamic, status, st);
}

int scalify_scaled_add(const scalify_array* A, const scalify_array* B, int subtract, scalify_array* Y, void* stream) {
  int rc = check_array(A);
  if (rc) return rc;
  rc = check_array(B);
  if (rc) return rc;
  rc = check_array(Y);
  if (rc) return rc;
  if (!is_wide(A->dtype) || B->dtype != A->dtype) return SCALIFY_ERR_DTYPE;
  const int64_t n = contiguous_numel(A);
  if (n < 0 || !same_shape(A, Y) || contiguous_numel(Y) != n) return SCALIFY_ERR_SHAPE;
  int broadcast = 0;
  const int64_t row_len = A->shape[A->ndim - 1];
  if (!same_shape(A, B)) {
    if (B->ndim == 1 && B->shape[0] == row_len) broadcast = 1;
    else return SCALIFY_ERR_SHAPE;
  } else if (contiguous_numel(B) != n) {
    return SCALIFY_ERR_SHAPE;
  }
  if (Y->scale && (Y->scale == A->scale || Y->scale == B->scale)) return SCALIFY_ERR_ALIAS;
  if (Y->data == A->data && elem_size(A->dtype) != elem_size(Y->dtype)) return SCALIFY_ERR_ALIAS;
  if (Y->data == B->data) return SCALIFY_ERR_ALIAS;
  return launch_add(A->data, B->data, A->dtype, Y->data, Y->dtype, n, row_len, broadcast, A->scale, B->scale, Y->scale,
                    subtract, static_cast<cudaStream_t>(stream));
}

int scalify_scaled_gelu(const scalify_array* X, int exact_erf, scalify_array* Y, void* stream) {
  int rc = check_array(X);
  if (rc) return rc;
  rc = check_array(Y);
  if (rc) return rc;
  if (!is_wide(X->dtype)) return SCALIFY_ERR_DTYPE;
  const int64_t n = contiguous_numel(X);
  if (n < 0 || contiguous_numel(Y) != n) return SCALIFY_ERR_SHAPE;
  if (Y->scale && Y->scale == X->scale) return SCALIFY_ERR_ALIAS;
  return launch_gelu(X->data, nullptr, X->dtype, Y->data, Y->dtype, n, X->scale, nullptr, Y->scale, exact_erf ? 1 : 0, 0,
                     static_cast<cudaStream_t>(stream));
}

int scalify_scaled_gelu_bwd(const scalify_array* G, const scalify_array* X, int exact_erf, scalify_array* dX,
                            void* stream) {
  int rc = check_array(G);
  if (rc) return rc;
  rc = check_array(X);
  if (rc) return rc;
  rc = check_array(dX);
  if (rc) return rc;
  if (!is_wide(X->dtype) || G->dtype != X->dtype) return SCALIFY_ERR_DTYPE;
  const int64_t n = contiguous_numel(X);
  if (n < 0 || contiguous_numel(G) != n || contiguous_numel(dX) != n) return SCALIFY_ERR_SHAPE;
  if (dX->scale && (dX->scale == X->scale || dX->scale == G->scale)) return SCALIFY_ERR_ALIAS;
  return launch_gelu(X->data, G->data, X->dtype, dX->data, dX->dtype, n, X->scale, G->scale, dX->scale,
                     exact_erf ? 1 : 0, 1, static_cast<cudaStream_t>(stream));
}

int scalify_scaled_layernorm(const scalify_array* X, const scalify_array* gamma, const scalify_array* beta, float eps,
                             int eps_inside_sqrt, scalify_array* Y, float* mean, float* rinv, void* stream) {
  int rc = check_array(X);
  if (rc) return rc;
  rc = check_array(Y);
  if (rc) return rc;
  if (!is_wide(X->dtype)) return SCALIFY_ERR_DTYPE;
  int64_t R, d, x_ld, Ry, dy, y_ld;
  if (as_rows(X, &R, &d, &x_ld) || as_rows(Y, &Ry, &dy, &y_ld) || R != Ry || d != dy) return SCALIFY_ERR_SHAPE;
  if (d < 1 || R > 0x7FFFFFFF || (d * elem_size(X->dtype)) % 16 != 0) return SCALIFY_ERR_SHAPE;
  if (!(eps >= 0.f)) return SCALIFY_ERR_VALUE;
  int gb_dt = SCALIFY_F32;
  if (gamma) {
    rc = check_array(gamma);
    if (rc) return rc;
    if (!is_wide(gamma->dtype) || gamma->ndim != 1 || gamma->shape[0] != d) return SCALIFY_ERR_SHAPE;
    gb_dt = gamma->dtype;
    if (beta) {
      rc = check_array(beta);
      if (rc) return rc;
      if (beta->dtype != gb_dt || beta->ndim != 1 || beta->shape[0] != d) return SCALIFY_ERR_SHAPE;
    }
  } else if (beta) {
    return SCALIFY_ERR_NULL;
  }
  if (R == 0) return SCALIFY_OK;
  return launch_layernorm_fwd(X->data, X->dtype, x_ld, Y->data, Y->dtype, y_ld, static_cast<int>(R), static_cast<int>(d),
                              gamma ? gamma->data : nullptr, beta ? beta->data : nullptr, gb_dt,
                              gamma ? gamma->scale : nullptr, beta ? beta->scale : nullptr, Y->scale, eps,
                              eps_inside_sqrt ? 1 : 0, mean, rinv, static_cast<cudaStream_t>(stream));
}

static int layernorm_bwd_impl(const scalify_array* G, const scalify_array* X, const scalify_array* gamma,
                              const float* mean, const float* rinv, float eps, int eps_inside_sqrt, int stat_dx,
                              const float* stat_in, scalify_array* dX, scalify_array* dXq, scalify_array* dgamma,
                              scalify_array* dbeta, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_array(G);
  if (rc) return rc;
  rc = check_array(X);
  if (rc) return rc;
  // dX == NULL with an FP8 dXq: the one-pass form of the dynamic rescale (the intermediate is not stored)
  const bool one_pass = dX == nullptr && dXq != nullptr && !stat_in;
  if (one_pass) {
    rc = check_array(dXq);
    if (rc) return rc;
    if (is_wide(dXq->dtype)) return SCALIFY_ERR_DTYPE;
    dX = dXq;  // shape, layout and scale word checks below apply to the array that is written
  }
  rc = check_array(dX);
  if (rc) return rc;
  if (!mean || !rinv) return SCALIFY_ERR_NULL;
  // the plain call keeps the un-rebalanced gradient in a wide format; the delayed one may round it once to FP8
  if (!is_wide(X->dtype) || G->dtype != X->dtype || (!stat_in && !one_pass && !is_wide(dX->dtype))) return SCALIFY_ERR_DTYPE;
  if (!valid_stat(stat_dx)) return SCALIFY_ERR_VALUE;
  int64_t R, d, x_ld, Rg, dg, g_ld, Rd, dd, dx_ld;
  if (as_rows(X, &R, &d, &x_ld) || as_rows(G, &Rg, &dg, &g_ld) || as_rows(dX, &Rd, &dd, &dx_ld)) return SCALIFY_ERR_SHAPE;
  if (R != Rg || d != dg || R != Rd || d != dd) return SCALIFY_ERR_SHAPE;
  if (d < 1 || R < 1 || R > 0x7FFFFFFF || (d * elem_size(X->dtype)) % 16 != 0) return SCALIFY_ERR_SHAPE;
  int gb_dt = SCALIFY_F32;
  if (gamma) {
    rc = check_array(gamma);
    if (rc) return rc;
    if (!is_wide(gamma->dtype) || gamma->ndim != 1 || gamma->shape[0] != d) return SCALIFY_ERR_SHAPE;
    gb_dt = gamma->dtype;
  }
  int dg_dt = SCALIFY_F32;
  if ((dgamma != nullptr) != (dbeta != nullptr)) return SCALIFY_ERR_NULL;
  if (dgamma) {
    rc = check_array(dgamma);
    if (rc) return rc;
    rc = check_array(dbeta);
    if (rc) return rc;
    if (!is_wide(dgamma->dtype) || dbeta->dtype != dgamma->dtype) return SCALIFY_ERR_DTYPE;
    if (dgamma->ndim != 1 || dgamma->shape[0] != d || dbeta->ndim != 1 || dbeta->shape[0] != d) return SCALIFY_ERR_SHAPE;
    dg_dt = dgamma->dtype;
  }
  if (one_pass) {
    if (stat_dx == SCALIFY_STAT_NONE) return SCALIFY_ERR_VALUE;
    if (contiguous_numel(dXq) != R * d) return SCALIFY_ERR_SHAPE;
  } else if (dXq) {
    rc = check_array(dXq);
    if (rc) return rc;
    if (stat_dx == SCALIFY_STAT_NONE) return SCALIFY_ERR_VALUE;
    if (contiguous_numel(dX) != R * d || contiguous_numel(dXq) != R * d) return SCALIFY_ERR_SHAPE;
    if (dXq->data == dX->data && elem_size(dXq->dtype) != elem_size(dX->dtype)) return SCALIFY_ERR_ALIAS;
  }
  if (dX->scale && (dX->scale == G->scale || dX->scale == X->scale || (gamma && dX->scale == gamma->scale)))
    return SCALIFY_ERR_ALIAS;
  rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_LAYERNORM_BWD, R, d));
  if (rc) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the un-rebalanced gradient needs a scale word for the rebalance pass; use a workspace slot if the caller has none
  float* dx_scale = dX->scale ? dX->scale : reinterpret_cast<float*>(static_cast<char*>(workspace) + 48);
  rc = launch_layernorm_bwd(G->data, g_ld, X->data, X->dtype, x_ld, dX->data, dX->dtype, dx_ld, static_cast<int>(R),
                            static_cast<int>(d), gamma ? gamma->data : nullptr, gb_dt, mean, rinv, eps,
                            eps_inside_sqrt ? 1 : 0, stat_dx, dgamma ? dgamma->data : nullptr,
                            dbeta ? dbeta->data : nullptr, dg_dt, G->scale, X->scale, gamma ? gamma->scale : nullptr,
                            dx_scale, dgamma ? dgamma->scale : nullptr, dbeta ? dbeta->scale : nullptr, stat_in,
                            one_pass ? 1 : 0, workspace, st);
  if (rc) return rc;
  if (dXq && !one_pass) {
    WsView v = ws_view(workspace);
    rc = launch_rebalance(dX->data, dX->dtype, dXq->data, dXq->dtype, R * d, dx_scale, dXq->scale, v.stat, nullptr,
                          kModeDynamic, v.status, st);
  }
  return rc;
}

int scalify_scaled_layernorm_bwd(const scalify_array* G, const scalify_array* X, const scalify_array* gamma,
                                 const float* mean, const float* rinv, float eps, int eps_inside_sqrt, int stat_dx,
                                 scalify_array* dX, scalify_array* dXq, scalify_array* dgamma, scalify_array* dbeta,
                                 void* workspace, size_t workspace_bytes, void* stream) {
  return layernorm_bwd_impl(G, X, gamma, mean, rinv, eps, eps_inside_sqrt, stat_dx, nullptr, dX, dXq, dgamma, dbeta,
                            workspace, workspace_bytes, stream);
}

int scalify_scaled_layernorm_bwd_delayed(const scalify_array* G, const scalify_array* X, const scalify_array* gamma,
                                         const float* mean, const float* rinv, float eps, int eps_inside_sqrt,
                                         const float* stat_in, int stat_dx, scalify_array* dX, scalify_array* dgamma,
                                         scalify_array* dbeta, void* workspace, size_t workspace_bytes, void* stream) {
  if (!stat_in) return SCALIFY_ERR_NULL;
  return layernorm_bwd_impl(G, X, gamma, mean, rinv, eps, eps_inside_sqrt, stat_dx, stat_in, dX, nullptr, dgamma, dbeta,
                            workspace, workspace_bytes, stream);
}

static int check_mx(const scalify_mx_array* a) {
  if (!a || !a->data || !a->sf) return SCALIFY_ERR_NULL;
  if (a->dtype != SCALIFY_E4M3 && a->dtype != SCALIFY_E5M2) return SCALIFY_ERR_DTYPE;
  if (a->rows < 1 || a->K < 128 || a->K % 128 != 0 || a->rows > 0x7FFFFFFF || a->K > 0x7FFFFFFF)
    return SCALIFY_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(a->data) % 16 != 0 || reinterpret_cast<uintptr_t>(a->sf) % 16 != 0)
    return SCALIFY_ERR_ALIGNMENT;
  if (a->transposed != 0 && a->transposed != 1) return SCALIFY_ERR_VALUE;
  if (a->transposed && a->rows % 16 != 0) return SCALIFY_ERR_ALIGNMENT;  // rows of the storage are `rows` bytes long
#ifdef SCALIFY_DEBUG
  dbg_register_range(a->data, static_cast<unsigned long long>(a->rows) * a->K);
  dbg_register_range(a->sf, mx_sf_bytes(a->rows, a->K));
#endif
  return SCALIFY_OK;
}

size_t scalify_mx_sf_bytes(int64_t rows, int64_t K) {
  if (rows < 1 || K < 128 || K % 128 != 0) return 0;
  return mx_sf_bytes(rows, K);
}

int scalify_mx_quantize(const scalify_array* X, scalify_mx_array* Y, uint32_t* status, void* stream) {
  int rc = check_array(X);
  if (rc) return rc;
  rc = check_mx(Y);
  if (rc) return rc;
  if (!is_wide(X->dtype)) return SCALIFY_ERR_DTYPE;
  if (Y->scale && Y->scale == X->scale) return SCALIFY_ERR_ALIAS;
  if (Y->transposed) {
    if (X->ndim != 2 || X->shape[0] != Y->K || X->shape[1] != Y->rows) return SCALIFY_ERR_SHAPE;
    return launch_mx_quantize_t(X->data, X->dtype, Y->rows, Y->K, X->stride[0], Y->data, Y->dtype, Y->sf, X->scale,
                                Y->scale, status, static_cast<cudaStream_t>(stream));
  }
  if (X->ndim != 2 || X->shape[0] != Y->rows || X->shape[1] != Y->K) return SCALIFY_ERR_SHAPE;
  return launch_mx_quantize(X->data, X->dtype, Y->rows, Y->K, X->stride[0], Y->data, Y->dtype, Y->sf, X->scale,
                            Y->scale, status, static_cast<cudaStream_t>(stream));
}

int scalify_mx_matmul(const scalify_mx_array* A, const scalify_mx_array* B, scalify_array* Y, int stat,
                      void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_mx(A);
  if (rc) return rc;
  rc = check_mx(B);
  if (rc) return rc;
  rc = check_array(Y);
  if (rc) return rc;
  if (!valid_stat(stat)) return SCALIFY_ERR_VALUE;
  if (!is_wide(Y->dtype)) return SCALIFY_ERR_DTYPE;
  if (A->K != B->K || Y->ndim != 2 || Y->shape[0] != A->rows || Y->shape[1] != B->rows) return SCALIFY_ERR_SHAPE;
  if (Y->scale && (Y->scale == A->scale || Y->scale == B->scale)) return SCALIFY_ERR_ALIAS;
  rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_MATMUL, A->rows, B->rows));
  if (rc) return rc;
  MxMatmulArgs a;
  a.A = A->data; a.a_dt = A->dtype; a.sfa = A->sf;
  a.B = B->data; a.b_dt = B->dtype; a.sfb = B->sf;
  a.Y = Y->data; a.y_dt = Y->dtype; a.ldy = Y->stride[0];
  a.M = static_cast<int>(A->rows); a.N = static_cast<int>(B->rows); a.K = static_cast<int>(A->K);
  a.a_scale = A->scale; a.b_scale = B->scale; a.y_scale = Y->scale;
  a.stat = stat;
  a.force_ncta = 0;
  a.transA = A->transposed;
  a.transB = B->transposed;
  return launch_mx_matmul(a, workspace, static_cast<cudaStream_t>(stream));
}

int scalify_scaled_colsum(const scalify_array* X, scalify_array* Y, void* workspace, size_t workspace_bytes,
                          void* stream) {
  int rc;
  if ((rc = check_array(X)) || (rc = check_array(Y))) return rc;
  if (!is_wide(Y->dtype)) return SCALIFY_ERR_DTYPE;
  if (X->ndim != 2 || Y->ndim != 1 || Y->shape[0] != X->shape[1]) return SCALIFY_ERR_SHAPE;
  const int64_t R = X->shape[0], N = X->shape[1];
  if (R < 1 || N < 1 || X->stride[0] < N) return SCALIFY_ERR_SHAPE;
  if (Y->scale && Y->scale == X->scale) return SCALIFY_ERR_ALIAS;
  rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_COLSUM, R, N));
  if (rc) return rc;
  return launch_colsum(X->data, X->dtype, X->stride[0], R, N, X->scale, Y->data, Y->dtype, Y->scale, workspace,
                       static_cast<cudaStream_t>(stream));
}

int scalify_scaled_cast_colsum(const scalify_array* X, scalify_array* C, scalify_array* Y, void* workspace,
                               size_t workspace_bytes, void* stream) {
  int rc;
  if ((rc = check_array(X)) || (rc = check_array(C)) || (rc = check_array(Y))) return rc;
  if ((X->dtype != SCALIFY_BF16 && X->dtype != SCALIFY_F16) || is_wide(C->dtype) || !is_wide(Y->dtype)) return SCALIFY_ERR_DTYPE;
  if (X->ndim != 2 || C->ndim != 2 || Y->ndim != 1 || Y->shape[0] != X->shape[1] || C->shape[0] != X->shape[0] ||
      C->shape[1] != X->shape[1])
    return SCALIFY_ERR_SHAPE;
  const int64_t R = X->shape[0], N = X->shape[1];
  if (R < 1 || N < 1 || X->stride[0] < N || C->stride[0] < N) return SCALIFY_ERR_SHAPE;
  if (C->data == X->data) return SCALIFY_ERR_ALIAS;
  if ((Y->scale && (Y->scale == X->scale || Y->scale == C->scale)) || (C->scale && C->scale == X->scale)) return SCALIFY_ERR_ALIAS;
  rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_COLSUM, R, N));
  if (rc) return rc;
  return launch_cast_colsum(X->data, X->dtype, X->stride[0], R, N, X->scale, C->data, C->dtype, C->stride[0], C->scale,
                            Y->data, Y->dtype, Y->scale, workspace, static_cast<cudaStream_t>(stream));
}

// [batch, heads, T, hd] view of a 2-D, 3-D or 4-D array: counts, rows, row / head / batch strides (elements)
struct HeadsView {
  int64_t batch, heads, rows, cols, ld, hs, bs;
};
static int as_heads(const scalify_array* a, HeadsView* v) {
  v->batch = 1; v->heads = 1; v->hs = 0; v->bs = 0;
  if (a->ndim == 2) { v->rows = a->shape[0]; v->cols = a->shape[1]; v->ld = a->stride[0]; return SCALIFY_OK; }
  if (a->ndim == 3) {
    v->heads = a->shape[0]; v->rows = a->shape[1]; v->cols = a->shape[2]; v->ld = a->stride[1]; v->hs = a->stride[0];
    return SCALIFY_OK;
  }
  if (a->ndim == 4) {
    v->batch = a->shape[0]; v->heads = a->shape[1]; v->rows = a->shape[2]; v->cols = a->shape[3];
    v->ld = a->stride[2]; v->hs = a->stride[1]; v->bs = a->stride[0];
    return SCALIFY_OK;
  }
  return SCALIFY_ERR_SHAPE;
}

int scalify_scaled_attention(const scalify_array* Q, const scalify_array* K, const scalify_array* V, float sm_scale,
                             int causal, scalify_array* O, scalify_array* S_dump, scalify_array* P_dump,
                             uint32_t* status, void* stream) {
  int rc;
  if ((rc = check_array(Q)) || (rc = check_array(K)) || (rc = check_array(V)) || (rc = check_array(O))) return rc;
  if (is_wide(Q->dtype) || is_wide(K->dtype) || is_wide(V->dtype) || !is_wide(O->dtype)) return SCALIFY_ERR_DTYPE;
  if (!isfinite(sm_scale)) return SCALIFY_ERR_VALUE;
  AttentionArgs a;
  HeadsView vq, vk, vv, vo;
  if ((rc = as_heads(Q, &vq)) || (rc = as_heads(K, &vk)) || (rc = as_heads(V, &vv)) || (rc = as_heads(O, &vo))) return rc;
  if (vq.batch != vk.batch || vq.batch != vv.batch || vq.batch != vo.batch || vq.heads != vk.heads ||
      vq.heads != vv.heads || vq.heads != vo.heads || vk.rows != vv.rows || vq.rows != vo.rows || vq.cols != vk.cols ||
      vq.cols != vv.cols || vq.cols != vo.cols)
    return SCALIFY_ERR_SHAPE;
  const int64_t tq = vq.rows, tk = vk.rows, hq = vq.batch * vq.heads;
  if (tq < 1 || tk < 1 || vq.heads < 1 || vq.batch < 1 || tq > 0x7FFFFFFF || tk > 0x7FFFFFFF || hq > 0x7FFFFFFF)
    return SCALIFY_ERR_SHAPE;
  if ((vq.cols != 64 && vq.cols != 128) || (causal && tk < tq)) return SCALIFY_ERR_UNSUPPORTED;
  a.q_ld = vq.ld; a.q_hs = vq.hs; a.q_bs = vq.bs; a.k_ld = vk.ld; a.k_hs = vk.hs; a.k_bs = vk.bs;
  a.v_ld = vv.ld; a.v_hs = vv.hs; a.v_bs = vv.bs; a.o_ld = vo.ld; a.o_hs = vo.hs; a.o_bs = vo.bs;
  if (O->scale && (O->scale == Q->scale || O->scale == K->scale || O->scale == V->scale)) return SCALIFY_ERR_ALIAS;
  a.S_dump = nullptr;
  a.P_dump = nullptr;
  if (S_dump) {
    if ((rc = check_array(S_dump))) return rc;
    if (S_dump->dtype != SCALIFY_BF16) return SCALIFY_ERR_DTYPE;
    if (contiguous_numel(S_dump) != hq * tq * tk || tk % 32 != 0) return SCALIFY_ERR_SHAPE;
    a.S_dump = S_dump->data;
  }
  if (P_dump) {
    if ((rc = check_array(P_dump))) return rc;
    if (P_dump->dtype != SCALIFY_E4M3) return SCALIFY_ERR_DTYPE;
    if (contiguous_numel(P_dump) != hq * tq * tk || tk % 32 != 0) return SCALIFY_ERR_SHAPE;
    a.P_dump = P_dump->data;
  }
  a.Q = Q->data; a.K = K->data; a.V = V->data;
  a.q_dt = Q->dtype; a.k_dt = K->dtype; a.v_dt = V->dtype;
  a.O = O->data; a.o_dt = O->dtype;
  a.batch = static_cast<int>(vq.batch); a.heads = static_cast<int>(vq.heads);
  a.Tq = static_cast<int>(tq); a.Tk = static_cast<int>(tk); a.hd = static_cast<int>(vq.cols);
  a.causal = causal ? 1 : 0;
  a.sm_scale = sm_scale;
  a.q_scale = Q->scale; a.k_scale = K->scale; a.v_scale = V->scale; a.o_scale = O->scale;
  a.status = status;
  return launch_attention(a, static_cast<cudaStream_t>(stream));
}

int scalify_scaled_attention_bwd(const scalify_array* Q, const scalify_array* K, const scalify_array* V,
                                 const scalify_array* P, const scalify_array* dO, float sm_scale, int causal,
                                 scalify_array* dS, scalify_array* dQ, scalify_array* dK, scalify_array* dV,
                                 scalify_array* dP_dump, uint32_t* status, void* stream) {
  int rc;
  if ((rc = check_array(Q)) || (rc = check_array(K)) || (rc = check_array(V)) || (rc = check_array(P)) ||
      (rc = check_array(dO)) || (rc = check_array(dS)) || (rc = check_array(dQ)) || (rc = check_array(dK)) ||
      (rc = check_array(dV)))
    return rc;
  if (is_wide(Q->dtype) || is_wide(K->dtype) || is_wide(V->dtype) || is_wide(dO->dtype)) return SCALIFY_ERR_DTYPE;
  if (P->dtype != SCALIFY_E4M3 || dS->dtype != SCALIFY_E5M2) return SCALIFY_ERR_DTYPE;
  if (!is_wide(dQ->dtype) || dK->dtype != dQ->dtype || dV->dtype != dQ->dtype) return SCALIFY_ERR_DTYPE;
  if (!dS->scale) return SCALIFY_ERR_NULL;  // the second launch reads dS_s from the device
  int ex = 0;
  if (!(sm_scale > 0.f) || !isfinite(sm_scale) || frexpf(sm_scale, &ex) != 0.5f) return SCALIFY_ERR_UNSUPPORTED;
  AttentionBwdArgs a;
  HeadsView vq, vk, vv, vdo, v1, v2, v3;
  if ((rc = as_heads(Q, &vq)) || (rc = as_heads(K, &vk)) || (rc = as_heads(V, &vv)) || (rc = as_heads(dO, &vdo)) ||
      (rc = as_heads(dQ, &v1)) || (rc = as_heads(dK, &v2)) || (rc = as_heads(dV, &v3)))
    return rc;
  const HeadsView* all[7] = {&vq, &vk, &vv, &vdo, &v1, &v2, &v3};
  for (int i = 1; i < 7; ++i)
    if (all[i]->batch != vq.batch || all[i]->heads != vq.heads || all[i]->cols != vq.cols) return SCALIFY_ERR_SHAPE;
  const int64_t tq = vq.rows, tk = vk.rows, hq = vq.batch * vq.heads;
  if (vv.rows != tk || vdo.rows != tq || v1.rows != tq || v2.rows != tk || v3.rows != tk) return SCALIFY_ERR_SHAPE;
  if (tq < 1 || tk < 1 || vq.heads < 1 || vq.batch < 1 || tq > 0x7FFFFFFF || tk > 0x7FFFFFFF || hq > 0x7FFFFFFF)
    return SCALIFY_ERR_SHAPE;
  if ((vq.cols != 64 && vq.cols != 128) || (causal && tk < tq)) return SCALIFY_ERR_UNSUPPORTED;
  a.q_ld = vq.ld; a.q_hs = vq.hs; a.q_bs = vq.bs; a.k_ld = vk.ld; a.k_hs = vk.hs; a.k_bs = vk.bs;
  a.v_ld = vv.ld; a.v_hs = vv.hs; a.v_bs = vv.bs; a.do_ld = vdo.ld; a.do_hs = vdo.hs; a.do_bs = vdo.bs;
  a.dq_ld = v1.ld; a.dq_hs = v1.hs; a.dq_bs = v1.bs; a.dk_ld = v2.ld; a.dk_hs = v2.hs; a.dk_bs = v2.bs;
  a.dv_ld = v3.ld; a.dv_hs = v3.hs; a.dv_bs = v3.bs;
  if (tk % 32 != 0) return SCALIFY_ERR_SHAPE;  // rows of P and dS are read and written in 32-byte pieces
  if (contiguous_numel(P) != hq * tq * tk || contiguous_numel(dS) != hq * tq * tk) return SCALIFY_ERR_SHAPE;
  const float* in_scales[5] = {Q->scale, K->scale, V->scale, P->scale, dO->scale};
  float* out_scales[4] = {dS->scale, dQ->scale, dK->scale, dV->scale};
  for (int o = 0; o < 4; ++o) {
    if (!out_scales[o]) continue;
    for (int i = 0; i < 5; ++i)
      if (out_scales[o] == in_scales[i]) return SCALIFY_ERR_ALIAS;
    for (int o2 = 0; o2 < o; ++o2)
      if (out_scales[o] == out_scales[o2]) return SCALIFY_ERR_ALIAS;
  }
  a.dP_dump = nullptr;
  if (dP_dump) {
    if ((rc = check_array(dP_dump))) return rc;
    if (dP_dump->dtype != SCALIFY_BF16) return SCALIFY_ERR_DTYPE;
    if (contiguous_numel(dP_dump) != hq * tq * tk) return SCALIFY_ERR_SHAPE;
    a.dP_dump = dP_dump->data;
  }
  a.Q = Q->data; a.K = K->data; a.V = V->data; a.dO = dO->data;
  a.q_dt = Q->dtype; a.k_dt = K->dtype; a.v_dt = V->dtype; a.do_dt = dO->dtype;
  a.P = P->data; a.dS = dS->data;
  a.dQ = dQ->data; a.dK = dK->data; a.dV = dV->data; a.g_dt = dQ->dtype;
  a.batch = static_cast<int>(vq.batch); a.heads = static_cast<int>(vq.heads);
  a.Tq = static_cast<int>(tq); a.Tk = static_cast<int>(tk); a.hd = static_cast<int>(vq.cols);
  a.causal = causal ? 1 : 0;
  a.sm_scale = sm_scale;
  a.q_scale = Q->scale; a.k_scale = K->scale; a.v_scale = V->scale; a.p_scale = P->scale; a.do_scale = dO->scale;
  a.ds_scale = dS->scale; a.dq_scale = dQ->scale; a.dk_scale = dK->scale; a.dv_scale = dV->scale;
  a.status = status;
  return launch_attention_bwd(a, static_cast<cudaStream_t>(stream));
}

static int adam_step_impl(int n_tensors, const scalify_array* grads, scalify_array* m, scalify_array* v,
                          scalify_array* w, const scalify_array* w_cast, float lr, float beta1, float beta2,
                          float eps, int64_t step, void* workspace, size_t workspace_bytes, void* stream) {
  if (n_tensors < 0) return SCALIFY_ERR_VALUE;
  if (n_tensors == 0) return SCALIFY_OK;
  if (!grads || !m || !v || !w) return SCALIFY_ERR_NULL;
  if (step < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f) || !isfinite(lr))
    return SCALIFY_ERR_VALUE;
  int rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_ADAM, n_tensors, 0));
  if (rc) return rc;
  int64_t stack_numel[64];
  int64_t* numel = stack_numel;
  int64_t* heap = nullptr;
  if (n_tensors > 64) {
    heap = new (std::nothrow) int64_t[n_tensors];
    if (!heap) return SCALIFY_ERR_VALUE;
    numel = heap;
  }
  rc = SCALIFY_OK;
  for (int i = 0; i < n_tensors && rc == SCALIFY_OK; ++i) {
    if ((rc = check_array(&grads[i])) || (rc = check_array(&m[i])) || (rc = check_array(&v[i])) ||
        (rc = check_array(&w[i])))
      break;
    if (!m[i].scale || !v[i].scale || !w[i].scale) { rc = SCALIFY_ERR_NULL; break; }
    if (grads[i].dtype != grads[0].dtype || m[i].dtype != m[0].dtype || v[i].dtype != m[0].dtype ||
        w[i].dtype != w[0].dtype) { rc = SCALIFY_ERR_DTYPE; break; }
    if (!(m[i].dtype == SCALIFY_F16 || m[i].dtype == SCALIFY_F32) || !is_wide(w[i].dtype)) { rc = SCALIFY_ERR_DTYPE; break; }
    const int64_t n = contiguous_numel(&grads[i]);
    if (n < 0 || contiguous_numel(&m[i]) != n || contiguous_numel(&v[i]) != n || contiguous_numel(&w[i]) != n) {
      rc = SCALIFY_ERR_SHAPE;
      break;
    }
    if (m[i].scale == v[i].scale || m[i].scale == w[i].scale || v[i].scale == w[i].scale ||
        grads[i].scale == m[i].scale || grads[i].scale == v[i].scale || grads[i].scale == w[i].scale) {
      rc = SCALIFY_ERR_ALIAS;
      break;
    }
    if (w_cast) {
      const scalify_array* c = &w_cast[i];
      if ((rc = check_array(c))) break;
      if (!c->scale) { rc = SCALIFY_ERR_NULL; break; }
      if (c->dtype == SCALIFY_F32 || c->dtype != w_cast[0].dtype || elem_size(c->dtype) >= elem_size(w[i].dtype)) {
        rc = SCALIFY_ERR_DTYPE;  // the copy is narrower than the weight it is cast from
        break;
      }
      if (contiguous_numel(c) != n) { rc = SCALIFY_ERR_SHAPE; break; }
      if (c->scale == m[i].scale || c->scale == v[i].scale || c->scale == w[i].scale || c->scale == grads[i].scale ||
          c->data == w[i].data) {
        rc = SCALIFY_ERR_ALIAS;
        break;
      }
    }
    numel[i] = n;
  }
  if (rc == SCALIFY_OK) {
    const void** words = new (std::nothrow) const void*[size_t(n_tensors) * 4];
    if (!words) rc = SCALIFY_ERR_VALUE;
    else rc = check_adam_scale_words(n_tensors, grads, m, v, w, w_cast, words);
    delete[] words;
  }
  if (rc == SCALIFY_OK)
    rc = launch_adam(n_tensors, grads, m, v, w, w_cast, numel, lr, beta1, beta2, eps, step, workspace,
                     static_cast<cudaStream_t>(stream));
  delete[] heap;
  return rc;
}

int scalify_scaled_adam_step(int n_tensors, const scalify_array* grads, scalify_array* m, scalify_array* v,
                             scalify_array* w, float lr, float beta1, float beta2, float eps, int64_t step,
                             void* workspace, size_t workspace_bytes, void* stream) {
  return adam_step_impl(n_tensors, grads, m, v, w, nullptr, lr, beta1, beta2, eps, step, workspace, workspace_bytes,
                        stream);
}

int scalify_scaled_adam_step_cast(int n_tensors, const scalify_array* grads, scalify_array* m, scalify_array* v,
                                  scalify_array* w, scalify_array* w_cast, float lr, float beta1, float beta2,
                                  float eps, int64_t step, void* workspace, size_t workspace_bytes, void* stream) {
  if (n_tensors > 0 && !w_cast) return SCALIFY_ERR_NULL;
  return adam_step_impl(n_tensors, grads, m, v, w, w_cast, lr, beta1, beta2, eps, step, workspace, workspace_bytes,
                        stream);
}

static int matmul_impl(const scalify_array* A, int transA, const scalify_array* B, int transB,
                       const scalify_array* bias, scalify_array* Y, int stat, scalify_array* Yq, float* stat_hint,
                       void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_array(A);
  if (rc) return rc;
  rc = check_array(B);
  if (rc) return rc;
  rc = check_array(Y);
  if (rc) return rc;
  // the plain call writes a 16- or 32-bit intermediate; with a bias the sum may also be cast straight to FP8
  if (!is_fp8(A->dtype) || !is_fp8(B->dtype) || (!bias && !is_wide(Y->dtype))) return SCALIFY_ERR_DTYPE;
  if (bias) {
    if ((rc = check_array(bias))) return rc;
    if (!is_wide(bias->dtype)) return SCALIFY_ERR_DTYPE;
    if (stat_hint) return SCALIFY_ERR_UNSUPPORTED;
    if (Y->scale && Y->scale == bias->scale) return SCALIFY_ERR_ALIAS;
  }
  if (!valid_stat(stat)) return SCALIFY_ERR_VALUE;
  if (A->ndim < 2 || A->ndim > 3 || B->ndim < 2 || Y->ndim != A->ndim || B->ndim > A->ndim) return SCALIFY_ERR_SHAPE;
  const int an = A->ndim, bn = B->ndim, yn = Y->ndim;
  const int64_t batch = an == 3 ? A->shape[0] : 1;
  const int64_t M = transA ? A->shape[an - 1] : A->shape[an - 2];
  const int64_t K = transA ? A->shape[an - 2] : A->shape[an - 1];
  const int64_t Kb = transB ? B->shape[bn - 1] : B->shape[bn - 2];
  const int64_t N = transB ? B->shape[bn - 2] : B->shape[bn - 1];
  if (K != Kb || K < 1 || M < 1 || N < 1 || batch < 1) return SCALIFY_ERR_SHAPE;
  if (Y->shape[yn - 2] != M || Y->shape[yn - 1] != N) return SCALIFY_ERR_SHAPE;
  if (bias && (bias->ndim != 1 || bias->shape[0] != N)) return SCALIFY_ERR_SHAPE;
  if (an == 3 && (Y->shape[0] != batch || (bn == 3 && B->shape[0] != batch))) return SCALIFY_ERR_SHAPE;
  if (M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF || batch > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
  if (Y->scale && (Y->scale == A->scale || Y->scale == B->scale)) return SCALIFY_ERR_ALIAS;
  rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_MATMUL, batch * M, N));
  if (rc) return rc;
  if (Yq) {
    rc = check_array(Yq);
    if (rc) return rc;
    if (stat == SCALIFY_STAT_NONE) return SCALIFY_ERR_VALUE;
    if (!same_shape(Y, Yq) || contiguous_numel(Y) != batch * M * N || contiguous_numel(Yq) != batch * M * N)
      return SCALIFY_ERR_SHAPE;
    if (Yq->data == Y->data && elem_size(Yq->dtype) != elem_size(Y->dtype)) return SCALIFY_ERR_ALIAS;
    if (Yq->scale && (Yq->scale == A->scale || Yq->scale == B->scale)) return SCALIFY_ERR_ALIAS;
  }
  MatmulArgs a{};
  a.A = A->data; a.a_dt = A->dtype; a.transA = transA ? 1 : 0; a.lda = A->stride[an - 2];
  a.a_bs = an == 3 ? A->stride[0] : 0;
  a.B = B->data; a.b_dt = B->dtype; a.transB = transB ? 1 : 0; a.ldb = B->stride[bn - 2];
  a.b_bs = bn == 3 ? B->stride[0] : 0;
  a.Y = Y->data; a.y_dt = Y->dtype; a.ldy = Y->stride[yn - 2]; a.y_bs = yn == 3 ? Y->stride[0] : 0;
  a.M = static_cast<int>(M); a.N = static_cast<int>(N); a.K = static_cast<int>(K); a.batch = static_cast<int>(batch);
  a.a_scale = A->scale; a.b_scale = B->scale;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the intermediate needs a scale word for the rebalance pass; use a workspace slot if the caller has none
  float* y_scale = Y->scale ? Y->scale : reinterpret_cast<float*>(static_cast<char*>(workspace) + 48);
  a.y_scale = y_scale;
  a.stat = stat;
  a.stat_in = nullptr;
  a.force_ncta = 0;
  a.alpha_override = 0.f;
  a.no_split = 0;
  a.bias = bias ? bias->data : nullptr;
  a.bias_dt = bias ? bias->dtype : 0;
  a.bias_scale = bias ? bias->scale : nullptr;
  a.stat_hint = nullptr;
  a.Yq = nullptr;
  a.q_dt = SCALIFY_E4M3;
  int took_spec = 0;
  a.took_spec = &took_spec;
  if (!stat_hint && !bias && Yq && stat == SCALIFY_STAT_AMAX && is_fp8(Yq->dtype) && Yq->data != Y->data &&
      (Y->dtype == SCALIFY_BF16 || Y->dtype == SCALIFY_F16) && N % 16 == 0) {
    // The exact dynamic rescale, predicted: the GEMM already writes Yq with the power of two of the statistic
    // this workspace saw last (header word at byte 56) and the check launch rebuilds Yq from Y only when this
    // call's statistic has another power of two.  Same bits as statistic + second pass, whatever the word holds.
    stat_hint = reinterpret_cast<float*>(static_cast<char*>(workspace) + 56);
    a.hint_optional = 1;
  }
  if (stat_hint) {
    // speculative rescale: 16-bit intermediate, FP8 result, AMAX (the statistic the GEMM gathers exactly)
    if (!Yq || stat != SCALIFY_STAT_AMAX) return SCALIFY_ERR_VALUE;
    if (!(Y->dtype == SCALIFY_BF16 || Y->dtype == SCALIFY_F16) || !is_fp8(Yq->dtype)) return SCALIFY_ERR_DTYPE;
    if (Yq->data == Y->data) return SCALIFY_ERR_ALIAS;
    a.stat_hint = stat_hint;
    a.Yq = Yq->data;
    a.q_dt = Yq->dtype;
  }
  if (a.lda < (transA ? M : K) || a.ldb < (transB ? K : N) || a.ldy < N) return SCALIFY_ERR_SHAPE;
  rc = launch_scaled_matmul(a, workspace, workspace_bytes, st);
  if (rc) return rc;
  if (Yq) {
    WsView v = ws_view(workspace);
    if (took_spec)
      rc = launch_rebalance_check(Y->data, Y->dtype, Yq->data, Yq->dtype, batch * M * N, y_scale, Yq->scale, v.stat,
                                  reinterpret_cast<const float*>(static_cast<char*>(workspace) + 52), stat_hint,
                                  v.status, st);
    else
      rc = launch_rebalance(Y->data, Y->dtype, Yq->data, Yq->dtype, batch * M * N, y_scale, Yq->scale, v.stat, nullptr,
                            kModeDynamic, v.status, st);
  }
  return rc;
}

// Y == NULL: only the rescaled FP8 output is stored (see the header).
static int matmul_fp8only_impl(const scalify_array* A, int transA, const scalify_array* B, int transB, int stat,
                               scalify_array* Yq, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_array(A);
  if (rc) return rc;
  if ((rc = check_array(B))) return rc;
  if (!Yq) return SCALIFY_ERR_NULL;
  if ((rc = check_array(Yq))) return rc;
  if (!is_fp8(A->dtype) || !is_fp8(B->dtype) || !is_fp8(Yq->dtype)) return SCALIFY_ERR_DTYPE;
  if (stat != SCALIFY_STAT_AMAX) return SCALIFY_ERR_VALUE;
  if (A->ndim < 2 || A->ndim > 3 || B->ndim < 2 || Yq->ndim != A->ndim || B->ndim > A->ndim) return SCALIFY_ERR_SHAPE;
  const int an = A->ndim, bn = B->ndim, yn = Yq->ndim;
  const int64_t batch = an == 3 ? A->shape[0] : 1;
  const int64_t M = transA ? A->shape[an - 1] : A->shape[an - 2];
  const int64_t K = transA ? A->shape[an - 2] : A->shape[an - 1];
  const int64_t Kb = transB ? B->shape[bn - 1] : B->shape[bn - 2];
  const int64_t N = transB ? B->shape[bn - 2] : B->shape[bn - 1];
  if (K != Kb || K < 1 || M < 1 || N < 1 || batch < 1) return SCALIFY_ERR_SHAPE;
  if (Yq->shape[yn - 2] != M || Yq->shape[yn - 1] != N || contiguous_numel(Yq) != batch * M * N) return SCALIFY_ERR_SHAPE;
  if (an == 3 && (Yq->shape[0] != batch || (bn == 3 && B->shape[0] != batch))) return SCALIFY_ERR_SHAPE;
  if (M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF || batch > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
  if (N % 16 != 0) return SCALIFY_ERR_ALIGNMENT;  // rows of the FP8 output are written by TMA: 16-byte row stride
  if (!Yq->scale) return SCALIFY_ERR_NULL;
  if (Yq->scale == A->scale || Yq->scale == B->scale) return SCALIFY_ERR_ALIAS;
  rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_MATMUL, batch * M, N));
  if (rc) return rc;
  MatmulArgs a{};
  a.A = A->data; a.a_dt = A->dtype; a.transA = transA ? 1 : 0; a.lda = A->stride[an - 2];
  a.a_bs = an == 3 ? A->stride[0] : 0;
  a.B = B->data; a.b_dt = B->dtype; a.transB = transB ? 1 : 0; a.ldb = B->stride[bn - 2];
  a.b_bs = bn == 3 ? B->stride[0] : 0;
  a.Y = nullptr; a.y_dt = SCALIFY_BF16; a.ldy = N; a.y_bs = yn == 3 ? M * N : 0;
  a.M = static_cast<int>(M); a.N = static_cast<int>(N); a.K = static_cast<int>(K); a.batch = static_cast<int>(batch);
  a.a_scale = A->scale; a.b_scale = B->scale;
  a.y_scale = reinterpret_cast<float*>(static_cast<char*>(workspace) + 48);  // scale of the intermediate that is not stored
  a.stat = SCALIFY_STAT_AMAX;
  a.no_split = 1;
  float* hint = reinterpret_cast<float*>(static_cast<char*>(workspace) + 56);
  a.stat_hint = hint; a.hint_out = hint;
  a.Yq = Yq->data; a.q_dt = Yq->dtype; a.yq_scale = Yq->scale;
  a.noy = 1;
  if (a.lda < (transA ? M : K) || a.ldb < (transB ? K : N)) return SCALIFY_ERR_SHAPE;
  return launch_scaled_matmul(a, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

int scalify_scaled_matmul(const scalify_array* A, int transA, const scalify_array* B, int transB, scalify_array* Y,
                          int stat, scalify_array* Yq, void* workspace, size_t workspace_bytes, void* stream) {
  if (!Y) return matmul_fp8only_impl(A, transA, B, transB, stat, Yq, workspace, workspace_bytes, stream);
  return matmul_impl(A, transA, B, transB, nullptr, Y, stat, Yq, nullptr, workspace, workspace_bytes, stream);
}

int scalify_scaled_matmul_bias(const scalify_array* A, int transA, const scalify_array* B, int transB,
                               const scalify_array* bias, scalify_array* Y, int stat, scalify_array* Yq,
                               void* workspace, size_t workspace_bytes, void* stream) {
  if (!bias) return SCALIFY_ERR_NULL;
  return matmul_impl(A, transA, B, transB, bias, Y, stat, Yq, nullptr, workspace, workspace_bytes, stream);
}

int scalify_scaled_matmul_speculative(const scalify_array* A, int transA, const scalify_array* B, int transB,
                                      scalify_array* Y, scalify_array* Yq, float* stat_hint, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  if (!stat_hint || !Yq) return SCALIFY_ERR_NULL;
  return matmul_impl(A, transA, B, transB, nullptr, Y, SCALIFY_STAT_AMAX, Yq, stat_hint, workspace, workspace_bytes, stream);
}

int scalify_scaled_matmul_delayed(const scalify_array* A, int transA, const scalify_array* B, int transB,
                                  const float* stat_in, scalify_array* Y, int stat, float* stat_out, void* workspace,
                                  size_t workspace_bytes, void* stream) {
  int rc = check_array(A);
  if (rc) return rc;
  rc = check_array(B);
  if (rc) return rc;
  rc = check_array(Y);
  if (rc) return rc;
  if (!stat_in) return SCALIFY_ERR_NULL;
  if (!is_fp8(A->dtype) || !is_fp8(B->dtype)) return SCALIFY_ERR_DTYPE;
  if (!valid_stat(stat)) return SCALIFY_ERR_VALUE;
  if (stat == SCALIFY_STAT_NONE && stat_out) return SCALIFY_ERR_VALUE;
  if (A->ndim < 2 || A->ndim > 3 || B->ndim < 2 || Y->ndim != A->ndim || B->ndim > A->ndim) return SCALIFY_ERR_SHAPE;
  const int an = A->ndim, bn = B->ndim, yn = Y->ndim;
  const int64_t batch = an == 3 ? A->shape[0] : 1;
  const int64_t M = transA ? A->shape[an - 1] : A->shape[an - 2];
  const int64_t K = transA ? A->shape[an - 2] : A->shape[an - 1];
  const int64_t Kb = transB ? B->shape[bn - 1] : B->shape[bn - 2];
  const int64_t N = transB ? B->shape[bn - 2] : B->shape[bn - 1];
  if (K != Kb || K < 1 || M < 1 || N < 1 || batch < 1) return SCALIFY_ERR_SHAPE;
  if (Y->shape[yn - 2] != M || Y->shape[yn - 1] != N) return SCALIFY_ERR_SHAPE;
  if (an == 3 && (Y->shape[0] != batch || (bn == 3 && B->shape[0] != batch))) return SCALIFY_ERR_SHAPE;
  if (M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF || batch > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
  if (Y->scale && (Y->scale == A->scale || Y->scale == B->scale)) return SCALIFY_ERR_ALIAS;
  rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_MATMUL, batch * M, N));
  if (rc) return rc;
  MatmulArgs a{};
  a.A = A->data; a.a_dt = A->dtype; a.transA = transA ? 1 : 0; a.lda = A->stride[an - 2];
  a.a_bs = an == 3 ? A->stride[0] : 0;
  a.B = B->data; a.b_dt = B->dtype; a.transB = transB ? 1 : 0; a.ldb = B->stride[bn - 2];
  a.b_bs = bn == 3 ? B->stride[0] : 0;
  a.Y = Y->data; a.y_dt = Y->dtype; a.ldy = Y->stride[yn - 2]; a.y_bs = yn == 3 ? Y->stride[0] : 0;
  a.M = static_cast<int>(M); a.N = static_cast<int>(N); a.K = static_cast<int>(K); a.batch = static_cast<int>(batch);
  a.a_scale = A->scale; a.b_scale = B->scale; a.y_scale = Y->scale;
  a.stat = stat;
  a.stat_in = stat_in;
  a.force_ncta = 0;
  a.alpha_override = 0.f;
  a.no_split = 0;
  a.bias = nullptr; a.bias_dt = 0; a.bias_scale = nullptr;
  a.stat_hint = nullptr;
  a.Yq = nullptr;
  a.q_dt = SCALIFY_E4M3;
  if (a.lda < (transA ? M : K) || a.ldb < (transB ? K : N) || a.ldy < N) return SCALIFY_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = launch_scaled_matmul(a, workspace, workspace_bytes, st);
  if (rc) return rc;
  // published only after the kernel has finished, so stat_out may be the word stat_in points to
  if (stat_out)
    SCALIFY_CUDA_TRY(cudaMemcpyAsync(stat_out, ws_view(workspace).stat, sizeof(float), cudaMemcpyDeviceToDevice, st));
  return SCALIFY_OK;
}

int scalify_debug_expire_wait(void* workspace, size_t workspace_bytes, uint32_t limit_us, uint32_t* waited_us,
                              void* stream) {
  int rc = check_ws(workspace, workspace_bytes, kWsMin);
  if (rc) return rc;
  if (limit_us < 1 || limit_us > 1000000u) return SCALIFY_ERR_VALUE;
  return launch_expire_wait(workspace, static_cast<unsigned long long>(limit_us) * 1000ull, waited_us,
                            static_cast<cudaStream_t>(stream));
}

int scalify_debug_bf16_round(const float* x, float* y, int64_t n, int two_wide, void* stream) {
  if (!x || !y) return SCALIFY_ERR_NULL;
  if (n < 1) return SCALIFY_ERR_SHAPE;
  return launch_bf16_round(x, y, n, two_wide ? 1 : 0, static_cast<cudaStream_t>(stream));
}

int scalify_debug_host_state_selftest(void) { return host_state_selftest(); }

int scalify_debug_bounds_report(uint64_t out[3], int reset_ranges, int64_t range_limit) {
  unsigned long long v[3] = {0, 0, 0};
  const int rc = debug_bounds_report(v, reset_ranges, range_limit);
  if (rc == SCALIFY_OK && out) { out[0] = v[0]; out[1] = v[1]; out[2] = v[2]; }
  return rc;
}

int scalify_debug_tensor_map_cache(uint64_t* hits, uint64_t* misses) {
  if (!hits || !misses) return SCALIFY_ERR_NULL;
  unsigned long long h = 0, m = 0;
  map_cache_counters(&h, &m);
  *hits = h;
  *misses = m;
  return SCALIFY_OK;
}

int scalify_debug_layernorm_plan(int64_t R, int64_t d, int x_dtype, int backward, int32_t plan[4]) {
  if (!plan) return SCALIFY_ERR_NULL;
  if (!is_wide(x_dtype)) return SCALIFY_ERR_DTYPE;
  if (R < 1 || d < 1 || R > 0x7FFFFFFF || d > 0x7FFFFFFF || (d * elem_size(x_dtype)) % 16 != 0) return SCALIFY_ERR_SHAPE;
  return layernorm_plan(R, d, x_dtype, backward, plan);
}

int scalify_scalar_mul_pow2(scalify_array* X, float c, void* stream) {
  if (!X || !X->scale) return SCALIFY_ERR_NULL;
  int ex;
  if (!(c > 0.f) || !isfinite(c) || frexpf(c, &ex) != 0.5f) return SCALIFY_ERR_UNSUPPORTED;
  return launch_scale_word_mul(X->scale, c, static_cast<cudaStream_t>(stream));
}

int scalify_scaled_embedding(const int64_t* ids, int64_t n, int64_t seq_len, const scalify_array* wte,
                             const scalify_array* wpe, scalify_array* Y, uint32_t* status, void* stream) {
  if (!ids) return SCALIFY_ERR_NULL;
  int rc = check_array(wte);
  if (rc) return rc;
  rc = check_array(Y);
  if (rc) return rc;
  if (!is_wide(wte->dtype) || wte->ndim != 2 || Y->ndim != 2) return SCALIFY_ERR_DTYPE;
  const int64_t vocab = wte->shape[0], d = wte->shape[1];
  if (n < 1 || seq_len < 1 || n % seq_len != 0 || d < 1 || d > 0x7FFFFFFF || seq_len > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
  if (Y->shape[0] != n || Y->shape[1] != d || contiguous_numel(wte) != vocab * d || contiguous_numel(Y) != n * d)
    return SCALIFY_ERR_SHAPE;
  if ((d * elem_size(wte->dtype)) % 16 != 0) return SCALIFY_ERR_SHAPE;
  if (wpe) {
    rc = check_array(wpe);
    if (rc) return rc;
    if (wpe->dtype != wte->dtype) return SCALIFY_ERR_DTYPE;
    if (wpe->ndim != 2 || wpe->shape[0] < seq_len || wpe->shape[1] != d || wpe->stride[0] != d) return SCALIFY_ERR_SHAPE;
  }
  if (Y->scale && (Y->scale == wte->scale || (wpe && Y->scale == wpe->scale))) return SCALIFY_ERR_ALIAS;
  return launch_embedding_fwd(reinterpret_cast<const long long*>(ids), n, static_cast<int>(seq_len), static_cast<int>(d),
                              vocab, wte->data, wpe ? wpe->data : nullptr, wte->dtype, wte->scale,
                              wpe ? wpe->scale : nullptr, Y->data, Y->dtype, Y->scale, status,
                              static_cast<cudaStream_t>(stream));
}

int scalify_scaled_embedding_bwd(const int64_t* ids, int64_t n, int64_t seq_len, const scalify_array* dY,
                                 scalify_array* dwte, scalify_array* dwpe, void* stream) {
  if (!ids) return SCALIFY_ERR_NULL;
  int rc = check_array(dY);
  if (rc) return rc;
  rc = check_array(dwte);
  if (rc) return rc;
  if (!is_wide(dY->dtype) || dwte->dtype != SCALIFY_F32) return SCALIFY_ERR_DTYPE;
  if (dY->ndim != 2 || dwte->ndim != 2) return SCALIFY_ERR_SHAPE;
  const int64_t d = dY->shape[1], vocab = dwte->shape[0];
  if (n < 1 || seq_len < 1 || n % seq_len != 0 || dY->shape[0] != n || dwte->shape[1] != d || d > 0x7FFFFFFF ||
      seq_len > 0x7FFFFFFF)
    return SCALIFY_ERR_SHAPE;
  if (contiguous_numel(dY) != n * d || contiguous_numel(dwte) != vocab * d) return SCALIFY_ERR_SHAPE;
  if ((d * elem_size(dY->dtype)) % 16 != 0) return SCALIFY_ERR_SHAPE;
  if (dwpe) {
    rc = check_array(dwpe);
    if (rc) return rc;
    if (dwpe->dtype != SCALIFY_F32) return SCALIFY_ERR_DTYPE;
    if (dwpe->ndim != 2 || dwpe->shape[0] != seq_len || dwpe->shape[1] != d || contiguous_numel(dwpe) != seq_len * d)
      return SCALIFY_ERR_SHAPE;
  }
  return launch_embedding_bwd(reinterpret_cast<const long long*>(ids), n, static_cast<int>(seq_len), static_cast<int>(d),
                              vocab, dY->data, dY->dtype, dY->scale, static_cast<float*>(dwte->data), dwte->scale,
                              dwpe ? static_cast<float*>(dwpe->data) : nullptr, dwpe ? dwpe->scale : nullptr,
                              static_cast<cudaStream_t>(stream));
}

int scalify_scaled_softmax(const scalify_array* S, int causal, scalify_array* P, void* stream) {
  int rc = check_array(S);
  if (rc) return rc;
  rc = check_array(P);
  if (rc) return rc;
  if (!is_wide(S->dtype)) return SCALIFY_ERR_DTYPE;
  if (S->ndim < 2 || !same_shape(S, P)) return SCALIFY_ERR_SHAPE;
  const int64_t Tq = S->shape[S->ndim - 2], Tk = S->shape[S->ndim - 1];
  const int64_t total = contiguous_numel(S);
  if (total < 1 || contiguous_numel(P) != total || Tk > 0x7FFFFFFF || Tq > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
  if ((Tk * elem_size(S->dtype)) % 16 != 0 || (causal && Tk < Tq)) return SCALIFY_ERR_SHAPE;
  if (P->scale && P->scale == S->scale) return SCALIFY_ERR_ALIAS;
  return launch_softmax_fwd(S->data, S->dtype, P->data, P->dtype, total / Tk, static_cast<int>(Tq), static_cast<int>(Tk),
                            causal ? 1 : 0, S->scale, P->scale, static_cast<cudaStream_t>(stream));
}

int scalify_scaled_softmax_bwd(const scalify_array* dP, const scalify_array* P, scalify_array* dS, void* stream) {
  int rc = check_array(dP);
  if (rc) return rc;
  rc = check_array(P);
  if (rc) return rc;
  rc = check_array(dS);
  if (rc) return rc;
  if (!is_wide(dP->dtype)) return SCALIFY_ERR_DTYPE;
  if (dP->ndim < 2 || !same_shape(dP, P) || !same_shape(dP, dS)) return SCALIFY_ERR_SHAPE;
  const int64_t Tk = dP->shape[dP->ndim - 1];
  const int64_t total = contiguous_numel(dP);
  if (total < 1 || contiguous_numel(P) != total || contiguous_numel(dS) != total || Tk > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
  if ((Tk * elem_size(dP->dtype)) % 16 != 0) return SCALIFY_ERR_SHAPE;
  if (dS->scale && (dS->scale == dP->scale || dS->scale == P->scale)) return SCALIFY_ERR_ALIAS;
  return launch_softmax_bwd(dP->data, dP->dtype, P->data, P->dtype, dS->data, dS->dtype, total / Tk, static_cast<int>(Tk),
                            dP->scale, P->scale, dS->scale, static_cast<cudaStream_t>(stream));
}

int scalify_scaled_cross_entropy(const scalify_array* logits, int64_t n_classes, const int64_t* targets, float* loss,
                                 scalify_array* dlogits, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_array(logits);
  if (rc) return rc;
  if (!targets || !loss) return SCALIFY_ERR_NULL;
  if (!is_wide(logits->dtype) || logits->ndim != 2) return SCALIFY_ERR_DTYPE;
  const int64_t n = logits->shape[0], ld = logits->shape[1];
  if (n < 1 || n_classes < 1 || n_classes > ld || n_classes > 0x7FFFFFFF || logits->stride[0] != ld) return SCALIFY_ERR_SHAPE;
  if (dlogits) {
    rc = check_array(dlogits);
    if (rc) return rc;
    if (!same_shape(logits, dlogits) || dlogits->stride[0] != ld) return SCALIFY_ERR_SHAPE;
    if (dlogits->scale && dlogits->scale == logits->scale) return SCALIFY_ERR_ALIAS;
  }
  rc = check_ws(workspace, workspace_bytes, scalify_workspace_bytes(SCALIFY_OP_CROSS_ENTROPY, n, 0));
  if (rc) return rc;
  return launch_cross_entropy(logits->data, logits->dtype, ld, static_cast<int>(n_classes),
                              reinterpret_cast<const long long*>(targets), n, logits->scale, loss,
                              dlogits ? dlogits->data : nullptr, dlogits ? dlogits->dtype : SCALIFY_F32,
                              dlogits ? dlogits->scale : nullptr, workspace, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
