// Scaled Adam step over a list of tensors (Sections 1, 3, 4; Table 3 row 4).
//
// Two launches per group of up to kAdamMaxTensors tensors:
//   1. adam_scales_kernel: one thread per tensor traces the static scale rules, keeps the old
//      scales and the reciprocals of the new ones in the workspace, and stores the new scale
//      words.  (Every block of the update kernel needs the OLD scales, so they cannot be
//      overwritten by the update kernel itself.)
//   2. adam_update_kernel: HBM-bound streaming update; a block takes chunks of
//      kAdamChunk elements, finds the owning tensor by binary search in a prefix table passed
//      by value, and moves 8 elements per thread access (8 B of FP8 gradient, 16 B of each
//      16-bit state, 32 B of fp32 master weight).
#include <algorithm>

#include "scalify_common.cuh"
#include "scalify_launch.h"

namespace scalify {

constexpr int kAdamMaxTensors = 160;
constexpr int kAdamThreads = 256;
constexpr int kAdamVec = 8;
constexpr int kAdamChunk = kAdamThreads * kAdamVec * 4;  // elements per block iteration

struct AdamTensorPtrs {
  const void* g;
  void* m;
  void* v;
  void* w;
  void* wc;  // optional compute copy of the updated weight (static cast of the stored value), or null
};

struct AdamTable {
  AdamTensorPtrs t[kAdamMaxTensors];
  long long n[kAdamMaxTensors];
  int chunk_start[kAdamMaxTensors + 1];  // prefix sum of ceil(n/kAdamChunk)
  int count;
  int wc_dt;  // dtype of the compute copies
};

struct AdamScalePtrs {
  const float* g[kAdamMaxTensors];
  float* m[kAdamMaxTensors];
  float* v[kAdamMaxTensors];
  float* w[kAdamMaxTensors];
  float* wc[kAdamMaxTensors];  // scale word of the compute copy, or null
  int count;
};

// per tensor, in the workspace: the old scales folded with the step's constants, and the
// reciprocals of the new scales (all scale factors are powers of two, so folding them is exact)
struct AdamFactors {
  float cm;      // b1 * m_s            m' = cm*m_d + cg*g_d          (value space)
  float cg;      // (1-b1) * g_s
  float cv;      // b2 * v_s            v' = cv*v_d + cg2*g_d^2
  float cg2;     // (1-b2) * g_s^2
  float inv_m2;  // 1 / m'_s
  float inv_v2;  // 1 / v'_s
  float cw;      // w_s / w'_s          w'_d = cw*w_d - cu * m' / (sqrt(v'/bc2) + eps)
  float cu;      // lr / bc1 / w'_s
};

struct AdamHyper {
  float lr, b1, b2, eps, one_m_b1, one_m_b2, inv_bc1, inv_bc2;
  // power-of-two scales of the scalar constants (Section 3.4: mantissa/exponent split)
  float p_b1, p_1mb1, p_b2, p_1mb2, p_lr, p_eps, p_bc1, p_bc2;
};

__global__ void adam_scales_kernel(AdamScalePtrs sp, AdamHyper h, AdamFactors* __restrict__ fac, uint32_t* status) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= sp.count) return;
  const float gs = load_scale(sp.g[i]);
  const float ms = *sp.m[i], vs = *sp.v[i], ws = *sp.w[i];
  if (!(is_pow2_scale(gs) && is_pow2_scale(ms) && is_pow2_scale(vs) && is_pow2_scale(ws)))
    atomicOr(status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
  // static rules on powers of two: mul -> product, add -> max, div -> ratio, sqrt -> floor of half exponent
  const float ms2 = fmaxf(h.p_b1 * ms, h.p_1mb1 * gs);
  const float vs2 = fmaxf(h.p_b2 * vs, h.p_1mb2 * gs * gs);
  const float den = fmaxf(p2_sqrt_floor(vs2 / h.p_bc2), h.p_eps);
  const float us = h.p_lr * (ms2 / h.p_bc1) / den;
  const float ws2 = fmaxf(ws, us);
  AdamFactors f;
  f.cm = h.b1 * ms;
  f.cg = h.one_m_b1 * gs;
  f.cv = h.b2 * vs;
  f.cg2 = h.one_m_b2 * gs * gs;
  f.inv_m2 = 1.0f / ms2;
  f.inv_v2 = 1.0f / vs2;
  f.cw = ws / ws2;
  f.cu = h.lr * h.inv_bc1 / ws2;
  fac[i] = f;
  *sp.m[i] = ms2;
  *sp.v[i] = vs2;
  *sp.w[i] = ws2;
  if (sp.wc[i]) *sp.wc[i] = ws2;  // a static cast keeps the scale (Appendix A)
}

// One element.  sqrt and the division use the hardware approximations (each within 2 ulp of fp32),
// far below the resolution of the FP16 / BF16 outputs and of the fp32 weight, whose update is a
// small correction; the kernel is otherwise limited by instruction issue, not by HBM.
__device__ __forceinline__ void adam_elem(float g, float& m, float& v, float& w, const AdamFactors& f,
                                          const AdamHyper& h) {
  const float m2 = fmaf(f.cm, m, f.cg * g);
  const float v2 = fmaf(f.cv, v, f.cg2 * (g * g));
  float root;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(root) : "f"(v2 * h.inv_bc2));
  const float upd = f.cu * __fdividef(m2, root + h.eps);
  w = fmaf(f.cw, w, -upd);
  m = m2 * f.inv_m2;
  v = v2 * f.inv_v2;
}

template <int GDT, int MVDT, int WDT>
__device__ __forceinline__ void adam_vec(const uint32_t* wg, uint32_t* wm, uint32_t* wv, uint32_t* ww,
                                         const AdamFactors& f, const AdamHyper& h) {
  float g[kAdamVec], m[kAdamVec], v[kAdamVec], w[kAdamVec];
  decode_vec<GDT, kAdamVec>(wg, g);
  decode_vec<MVDT, kAdamVec>(wm, m);
  decode_vec<MVDT, kAdamVec>(wv, v);
  decode_vec<WDT, kAdamVec>(ww, w);
#pragma unroll
  for (int e = 0; e < kAdamVec; ++e) adam_elem(g[e], m[e], v[e], w[e], f, h);
  encode_vec<MVDT, kAdamVec>(m, wm);
  encode_vec<MVDT, kAdamVec>(v, wv);
  encode_vec<WDT, kAdamVec>(w, ww);
}

// Compute copy of the updated weight: the STORED value (already rounded to WDT) converted to the
// copy's dtype, 8 elements -> 8 bytes (FP8) or 16 bytes (FP16 / BF16).
template <int WDT>
__device__ __forceinline__ void adam_cast_store(const uint32_t* ww, int dt, char* wcp, long long i) {
  float w[kAdamVec];
  decode_vec<WDT, kAdamVec>(ww, w);
  if (dt == SCALIFY_E4M3) {
    uint32_t o[2];
    encode_vec<SCALIFY_E4M3, kAdamVec>(w, o);
    st_raw<8>(wcp + i * 8, o);
  } else if (dt == SCALIFY_E5M2) {
    uint32_t o[2];
    encode_vec<SCALIFY_E5M2, kAdamVec>(w, o);
    st_raw<8>(wcp + i * 8, o);
  } else if (dt == SCALIFY_BF16) {
    uint32_t o[4];
    encode_vec<SCALIFY_BF16, kAdamVec>(w, o);
    st_raw<16>(wcp + i * 16, o);
  } else {
    uint32_t o[4];
    encode_vec<SCALIFY_F16, kAdamVec>(w, o);
    st_raw<16>(wcp + i * 16, o);
  }
}

template <int GDT, int MVDT, int WDT>
__global__ void __launch_bounds__(kAdamThreads) adam_update_kernel(const __grid_constant__ AdamTable tab,
                                                                   const AdamFactors* __restrict__ fac,
                                                                   AdamHyper h) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int GB = kAdamVec * ElemBytes<GDT>::v, MB = kAdamVec * ElemBytes<MVDT>::v,
                WB = kAdamVec * ElemBytes<WDT>::v;
  const int total_chunks = tab.chunk_start[tab.count];
  for (int chunk = blockIdx.x; chunk < total_chunks; chunk += gridDim.x) {
    // owning tensor: last index with chunk_start <= chunk
    int lo = 0, hi = tab.count - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (tab.chunk_start[mid] <= chunk) lo = mid; else hi = mid - 1;
    }
    const int ti = lo;
    const AdamFactors f = fac[ti];
    const long long n = tab.n[ti];
    const long long n_vec = n / kAdamVec;
    const long long vec0 = (long long)(chunk - tab.chunk_start[ti]) * (kAdamChunk / kAdamVec);
    const char* gp = static_cast<const char*>(tab.t[ti].g);
    char* mp = static_cast<char*>(tab.t[ti].m);
    char* vp = static_cast<char*>(tab.t[ti].v);
    char* wp = static_cast<char*>(tab.t[ti].w);
    char* wcp = static_cast<char*>(tab.t[ti].wc);
    uint32_t wg[4][GB / 4 > 0 ? GB / 4 : 1], wm[4][MB / 4], wv[4][MB / 4], ww[4][WB / 4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long i = vec0 + u * kAdamThreads + threadIdx.x;
      if (i < n_vec) {
        ld_raw_stream<GB>(gp + i * GB, wg[u]);
        ld_raw_stream<MB>(mp + i * MB, wm[u]);
        ld_raw_stream<MB>(vp + i * MB, wv[u]);
        ld_raw_stream<WB>(wp + i * WB, ww[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const long long i = vec0 + u * kAdamThreads + threadIdx.x;
      if (i < n_vec) {
        adam_vec<GDT, MVDT, WDT>(wg[u], wm[u], wv[u], ww[u], f, h);
        st_raw<MB>(mp + i * MB, wm[u]);
        st_raw<MB>(vp + i * MB, wv[u]);
        st_raw<WB>(wp + i * WB, ww[u]);
        if (wcp) adam_cast_store<WDT>(ww[u], tab.wc_dt, wcp, i);
      }
    }
    // ragged tail of the tensor (fewer than kAdamVec elements), done by its last chunk
    if (chunk == tab.chunk_start[ti + 1] - 1) {
      const long long i = n_vec * kAdamVec + threadIdx.x;
      if (i < n) {
        float mm = load_elem<MVDT>(mp, i), vv = load_elem<MVDT>(vp, i), ww = load_elem<WDT>(wp, i);
        adam_elem(load_elem<GDT>(gp, i), mm, vv, ww, f, h);
        store_elem<MVDT>(mp, i, mm);
        store_elem<MVDT>(vp, i, vv);
        store_elem<WDT>(wp, i, ww);
        if (wcp) {
          const float stored = round_through<WDT>(ww);
          if (tab.wc_dt == SCALIFY_E4M3) store_elem<SCALIFY_E4M3>(wcp, i, stored);
          else if (tab.wc_dt == SCALIFY_E5M2) store_elem<SCALIFY_E5M2>(wcp, i, stored);
          else if (tab.wc_dt == SCALIFY_BF16) store_elem<SCALIFY_BF16>(wcp, i, stored);
          else store_elem<SCALIFY_F16>(wcp, i, stored);
        }
      }
    }
  }
}

static float host_p2_floor_abs(double c) {
  if (c == 0.0) return 1.0f;
  int ex;
  frexp(fabs(c), &ex);
  return static_cast<float>(ldexp(1.0, ex - 1));
}

size_t adam_ws_bytes(int64_t n_tensors) { return kWsHeader + size_t(n_tensors) * sizeof(AdamFactors) + 256; }

int launch_adam(int n_tensors, const scalify_array* grads, scalify_array* m, scalify_array* v, scalify_array* w,
                const scalify_array* w_cast, const int64_t* numel, float lr, float beta1, float beta2, float eps, int64_t step, void* ws,
                cudaStream_t st) {
  WsView view = ws_view(ws);
  AdamFactors* fac_all = static_cast<AdamFactors*>(view.area);
  AdamHyper h;
  const double b1 = beta1, b2 = beta2;
  const double bc1 = 1.0 - pow(b1, static_cast<double>(step));
  const double bc2 = 1.0 - pow(b2, static_cast<double>(step));
  h.lr = lr; h.b1 = beta1; h.b2 = beta2; h.eps = eps;
  h.one_m_b1 = static_cast<float>(1.0 - b1);
  h.one_m_b2 = static_cast<float>(1.0 - b2);
  h.inv_bc1 = static_cast<float>(1.0 / bc1);
  h.inv_bc2 = static_cast<float>(1.0 / bc2);
  h.p_b1 = host_p2_floor_abs(b1); h.p_1mb1 = host_p2_floor_abs(1.0 - b1);
  h.p_b2 = host_p2_floor_abs(b2); h.p_1mb2 = host_p2_floor_abs(1.0 - b2);
  h.p_lr = host_p2_floor_abs(lr); h.p_eps = host_p2_floor_abs(eps);
  h.p_bc1 = host_p2_floor_abs(bc1); h.p_bc2 = host_p2_floor_abs(bc2);
  const int g_dt = grads[0].dtype, mv_dt = m[0].dtype, w_dt = w[0].dtype;
  for (int base = 0; base < n_tensors; base += kAdamMaxTensors) {
    const int cnt = (n_tensors - base < kAdamMaxTensors) ? n_tensors - base : kAdamMaxTensors;
    AdamTable tab;
    AdamScalePtrs sp;
    tab.count = cnt;
    tab.wc_dt = w_cast ? w_cast[0].dtype : SCALIFY_E4M3;
    sp.count = cnt;
    tab.chunk_start[0] = 0;
    for (int i = 0; i < cnt; ++i) {
      const int k = base + i;
      tab.t[i].g = grads[k].data; tab.t[i].m = m[k].data; tab.t[i].v = v[k].data; tab.t[i].w = w[k].data;
      tab.t[i].wc = w_cast ? w_cast[k].data : nullptr;
      sp.wc[i] = w_cast ? w_cast[k].scale : nullptr;
      tab.n[i] = numel[k];
      int64_t chunks = (numel[k] + kAdamChunk - 1) / kAdamChunk;
      if (chunks < 1) chunks = 1;
      if (tab.chunk_start[i] + chunks > (int64_t(1) << 30)) return SCALIFY_ERR_SHAPE;
      tab.chunk_start[i + 1] = tab.chunk_start[i] + static_cast<int>(chunks);
      sp.g[i] = grads[k].scale; sp.m[i] = m[k].scale; sp.v[i] = v[k].scale; sp.w[i] = w[k].scale;
    }
    AdamFactors* fac = fac_all + base;
    adam_scales_kernel<<<(cnt + 127) / 128, 128, 0, st>>>(sp, h, fac, view.status);
    SCALIFY_CUDA_TRY(cudaGetLastError());
    const int total = tab.chunk_start[cnt];
    // one chunk per block: the hardware scheduler balances the blocks over the SMs (measured
    // faster on B200 than a grid of 8 blocks per SM striding over the chunks)
    const int grid = total > 0 ? total : 1;
#define SCALIFY_ADAM_LAUNCH(G, MV, W) \
  adam_update_kernel<G, MV, W><<<grid, kAdamThreads, 0, st>>>(tab, fac, h)
    SCALIFY_DISPATCH_DTYPE(g_dt, GDT, {
      if (mv_dt == SCALIFY_F16) {
        if (w_dt == SCALIFY_F16) SCALIFY_ADAM_LAUNCH(GDT, SCALIFY_F16, SCALIFY_F16);
        else if (w_dt == SCALIFY_BF16) SCALIFY_ADAM_LAUNCH(GDT, SCALIFY_F16, SCALIFY_BF16);
        else SCALIFY_ADAM_LAUNCH(GDT, SCALIFY_F16, SCALIFY_F32);
      } else {
        if (w_dt == SCALIFY_F16) SCALIFY_ADAM_LAUNCH(GDT, SCALIFY_F32, SCALIFY_F16);
        else if (w_dt == SCALIFY_BF16) SCALIFY_ADAM_LAUNCH(GDT, SCALIFY_F32, SCALIFY_BF16);
        else SCALIFY_ADAM_LAUNCH(GDT, SCALIFY_F32, SCALIFY_F32);
      }
    });
#undef SCALIFY_ADAM_LAUNCH
    SCALIFY_CUDA_TRY(cudaGetLastError());
  }
  return SCALIFY_OK;
}

int check_adam_scale_words(int n_tensors, const scalify_array* grads, const scalify_array* m, const scalify_array* v,
                           const scalify_array* w, const scalify_array* w_cast, const void** scratch) {
  int k = 0;
  for (int i = 0; i < n_tensors; ++i) {
    scratch[k++] = m[i].scale;
    scratch[k++] = v[i].scale;
    scratch[k++] = w[i].scale;
    if (w_cast) scratch[k++] = w_cast[i].scale;
  }
  std::sort(scratch, scratch + k);
  for (int i = 1; i < k; ++i)
    if (scratch[i] == scratch[i - 1]) return SCALIFY_ERR_ALIAS;
  for (int i = 0; i < n_tensors; ++i)
    if (grads[i].scale && std::binary_search(scratch, scratch + k, static_cast<const void*>(grads[i].scale)))
      return SCALIFY_ERR_ALIAS;
  return SCALIFY_OK;
}

}  // namespace scalify
