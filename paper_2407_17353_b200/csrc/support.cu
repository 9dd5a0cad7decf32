// Support kernels of a GPT-style training step around the scaled matmuls: embedding lookup and
// its gradient, causal row softmax forward / backward, mean cross-entropy with its gradient.
// The paper gives no scale rule for these (Section 3.2.1 only says custom rules are possible for
// attention); the rules taken are stated with each kernel.  All arithmetic is fp32, every row is
// read once from HBM (cross-entropy re-reads its row from L1/L2).
#include "scalify_common.cuh"
#include "scalify_launch.h"

namespace scalify {

// ---------------------------------------------------------------------------------------------
// embedding: Y = wte[ids] + wpe[pos] through the add rule (Y_s = max of the two scales)
// ---------------------------------------------------------------------------------------------
template <int WDT, int YDT>
__global__ void __launch_bounds__(256) embedding_fwd_kernel(const long long* __restrict__ ids, long long n, int seq_len,
                                                            int d, long long vocab, const void* __restrict__ wte,
                                                            const void* __restrict__ wpe, const float* wte_scale,
                                                            const float* wpe_scale, void* __restrict__ Y, float* y_scale,
                                                            uint32_t* bad_index) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<WDT>::v;
  constexpr int OB = VEC * ElemBytes<YDT>::v;
  const float ts = load_scale(wte_scale), ps = wpe ? load_scale(wpe_scale) : 0.f;
  const float ys = fmaxf(ts, ps);
  const float ft = ts / ys, fp = ps / ys;
  const int n_vec = d / VEC;
  const long long total = n * n_vec;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += 256ll * gridDim.x) {
    const long long row = i / n_vec;
    const int c = static_cast<int>(i - row * n_vec);
    long long id = ids[row];
    if (id < 0 || id >= vocab) {  // out-of-range token: recorded, row of zeros from the table
      if (bad_index) atomicOr(bad_index, static_cast<uint32_t>(SCALIFY_DEV_BAD_INDEX));
      id = 0;
    }
    uint32_t w[4];
    float a[VEC], b[VEC];
    ld_raw<16>(static_cast<const char*>(wte) + (id * d) * ElemBytes<WDT>::v + c * 16ll, w);
    decode_vec<WDT, VEC>(w, a);
    if (wpe) {
      const int pos = static_cast<int>(row % seq_len);
      ld_raw<16>(static_cast<const char*>(wpe) + (static_cast<long long>(pos) * d) * ElemBytes<WDT>::v + c * 16ll, w);
      decode_vec<WDT, VEC>(w, b);
#pragma unroll
      for (int e = 0; e < VEC; ++e) a[e] = fmaf(b[e], fp, a[e] * ft);
    } else {
#pragma unroll
      for (int e = 0; e < VEC; ++e) a[e] *= ft;
    }
    uint32_t o[OB / 4];
    encode_vec<YDT, VEC>(a, o);
    st_raw<OB>(static_cast<char*>(Y) + (row * d) * ElemBytes<YDT>::v + static_cast<long long>(c) * OB, o);
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && y_scale) *y_scale = ys;
}

// dwte[v] += rows of dY with token v (fp32 atomics; the table must have been zeroed); scale unchanged
template <int GDT>
__global__ void __launch_bounds__(256) embedding_bwd_scatter_kernel(const long long* __restrict__ ids, long long n, int d,
                                                                    long long vocab, const void* __restrict__ dY,
                                                                    float* __restrict__ dwte) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<GDT>::v;
  const int n_vec = d / VEC;
  const long long total = n * n_vec;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += 256ll * gridDim.x) {
    const long long row = i / n_vec;
    const int c = static_cast<int>(i - row * n_vec);
    const long long id = ids[row];
    if (id < 0 || id >= vocab) continue;
    uint32_t w[4];
    float g[VEC];
    ld_raw_stream<16>(static_cast<const char*>(dY) + (row * d) * ElemBytes<GDT>::v + c * 16ll, w);
    decode_vec<GDT, VEC>(w, g);
    float* dst = dwte + id * d + static_cast<long long>(c) * VEC;
#pragma unroll
    for (int e = 0; e < VEC; ++e) atomicAdd(dst + e, g[e]);
  }
}

// dwpe[p] = sum over the B sequences of dY[b*T + p], divided by kf(B), scale dY_s*kf(B): fixed order
template <int GDT>
__global__ void __launch_bounds__(256) embedding_bwd_pos_kernel(long long n, int seq_len, int d,
                                                                const void* __restrict__ dY, float* __restrict__ dwpe,
                                                                const float* dy_scale, float* dwte_scale,
                                                                float* dwpe_scale) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<GDT>::v;
  const int n_vec = d / VEC;
  const int B = static_cast<int>(n / seq_len);
  const float f = kfactor(B);
  const long long total = static_cast<long long>(seq_len) * n_vec;
  if (dwpe) {
    for (long long i = blockIdx.x * 256ll + threadIdx.x; i < total; i += 256ll * gridDim.x) {
      const int pos = static_cast<int>(i / n_vec);
      const int c = static_cast<int>(i - static_cast<long long>(pos) * n_vec);
      float acc[VEC];
#pragma unroll
      for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
      for (int b = 0; b < B; ++b) {
        uint32_t w[4];
        float g[VEC];
        ld_raw<16>(static_cast<const char*>(dY) + ((static_cast<long long>(b) * seq_len + pos) * d) * ElemBytes<GDT>::v + c * 16ll, w);
        decode_vec<GDT, VEC>(w, g);
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] += g[e];
      }
      float* dst = dwpe + static_cast<long long>(pos) * d + c * VEC;
#pragma unroll
      for (int e = 0; e < VEC; ++e) dst[e] = acc[e] / f;
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    const float gs = load_scale(dy_scale);
    if (dwte_scale) *dwte_scale = gs;
    if (dwpe_scale) *dwpe_scale = gs * f;
  }
}

int launch_embedding_fwd(const long long* ids, long long n, int seq_len, int d, long long vocab, const void* wte,
                         const void* wpe, int w_dt, const float* wte_scale, const float* wpe_scale, void* Y, int y_dt,
                         float* y_scale, uint32_t* status, cudaStream_t st) {
  const long long total = n * (d * elem_size(w_dt) / 16);
  long long blocks = (total + 255) / 256;
  const long long cap = static_cast<long long>(sm_count()) * 8;
  const int grid = static_cast<int>(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
  SCALIFY_DISPATCH_WIDE(w_dt, WDT, SCALIFY_DISPATCH_DTYPE(y_dt, YDT,
      embedding_fwd_kernel<WDT, YDT><<<grid, 256, 0, st>>>(ids, n, seq_len, d, vocab, wte, wpe, wte_scale, wpe_scale, Y,
                                                           y_scale, status)));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

int launch_embedding_bwd(const long long* ids, long long n, int seq_len, int d, long long vocab, const void* dY, int g_dt,
                         const float* dy_scale, float* dwte, float* dwte_scale, float* dwpe, float* dwpe_scale,
                         cudaStream_t st) {
  SCALIFY_CUDA_TRY(cudaMemsetAsync(dwte, 0, static_cast<size_t>(vocab) * d * sizeof(float), st));
  const long long total = n * (d * elem_size(g_dt) / 16);
  long long blocks = (total + 255) / 256;
  const long long cap = static_cast<long long>(sm_count()) * 8;
  const int grid = static_cast<int>(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
  SCALIFY_DISPATCH_WIDE(g_dt, GDT, {
    embedding_bwd_scatter_kernel<GDT><<<grid, 256, 0, st>>>(ids, n, d, vocab, dY, dwte);
    embedding_bwd_pos_kernel<GDT><<<grid, 256, 0, st>>>(n, seq_len, d, dY, dwpe, dy_scale, dwte_scale, dwpe_scale);
  });
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// row softmax of the values S_d*S_s with optional causal mask; probabilities carry scale 1
// ---------------------------------------------------------------------------------------------
constexpr int kSmVpt = 8;  // 16-byte vectors per lane: rows up to 256 vectors (2048 16-bit elements)

template <int SDT, int PDT>
__global__ void __launch_bounds__(128) softmax_fwd_kernel(const void* __restrict__ S, void* __restrict__ P,
                                                          long long rows, int Tq, int Tk, int causal,
                                                          const float* s_scale, float* p_scale) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<SDT>::v;
  constexpr int OB = VEC * ElemBytes<PDT>::v;
  const int lane = threadIdx.x & 31;
  const long long warp = (blockIdx.x * 128ll + threadIdx.x) >> 5, n_warps = (gridDim.x * 128ll) >> 5;
  const int n_vec = Tk / VEC;
  const float sc2 = load_scale(s_scale) * 1.4426950408889634f;  // values in units of log2(e)
  for (long long row = warp; row < rows; row += n_warps) {
    const int i = static_cast<int>(row % Tq);
    const int lim = causal ? min(Tk, i + Tk - Tq + 1) : Tk;
    float x[kSmVpt][VEC];
    float mx = -INFINITY;
    const char* srow = static_cast<const char*>(S) + row * Tk * ElemBytes<SDT>::v;
#pragma unroll
    for (int v = 0; v < kSmVpt; ++v) {
      const int vi = lane + v * 32;
      if (vi < n_vec && vi * VEC < lim) {
        uint32_t w[4];
        ld_raw_stream<16>(srow + vi * 16ll, w);
        decode_vec<SDT, VEC>(w, x[v]);
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
          x[v][e] = (vi * VEC + e < lim) ? x[v][e] * sc2 : -INFINITY;
          mx = fmaxf(mx, x[v][e]);
        }
      } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e) x[v][e] = -INFINITY;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    float sum = 0.f;
#pragma unroll
    for (int v = 0; v < kSmVpt; ++v)
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        x[v][e] = exp2f(x[v][e] - mx);  // exp2f(-inf) = 0 for masked positions
        sum += x[v][e];
      }
    sum = warp_sum_f32(sum);
    const float inv = 1.0f / sum;
    char* prow = static_cast<char*>(P) + row * Tk * ElemBytes<PDT>::v;
#pragma unroll
    for (int v = 0; v < kSmVpt; ++v) {
      const int vi = lane + v * 32;
      if (vi < n_vec) {
        float o[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) o[e] = x[v][e] * inv;
        uint32_t ow[OB / 4];
        encode_vec<PDT, VEC>(o, ow);
        st_raw<OB>(prow + static_cast<long long>(vi) * OB, ow);
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && p_scale) *p_scale = 1.0f;
}

// dS = P*(dP - sum_j dP_j P_j), dS_s = dP_s * P_s
template <int GDT, int PDT, int ODT>
__global__ void __launch_bounds__(128) softmax_bwd_kernel(const void* __restrict__ dP, const void* __restrict__ P,
                                                          void* __restrict__ dS, long long rows, int Tk,
                                                          const float* dp_scale, const float* p_scale, float* ds_scale) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<GDT>::v;            // vector of the gradient dtype
  constexpr int PB = VEC * ElemBytes<PDT>::v, OB = VEC * ElemBytes<ODT>::v;
  const int lane = threadIdx.x & 31;
  const long long warp = (blockIdx.x * 128ll + threadIdx.x) >> 5, n_warps = (gridDim.x * 128ll) >> 5;
  const int n_vec = Tk / VEC;
  for (long long row = warp; row < rows; row += n_warps) {
    float g[kSmVpt][VEC], p[kSmVpt][VEC];
    float dot = 0.f;
    const char* grow = static_cast<const char*>(dP) + row * Tk * ElemBytes<GDT>::v;
    const char* prow = static_cast<const char*>(P) + row * Tk * ElemBytes<PDT>::v;
#pragma unroll
    for (int v = 0; v < kSmVpt; ++v) {
      const int vi = lane + v * 32;
      if (vi < n_vec) {
        uint32_t wg[4], wp[PB / 4];
        ld_raw_stream<16>(grow + vi * 16ll, wg);
        ld_raw_stream<PB>(prow + static_cast<long long>(vi) * PB, wp);
        decode_vec<GDT, VEC>(wg, g[v]);
        decode_vec<PDT, VEC>(wp, p[v]);
#pragma unroll
        for (int e = 0; e < VEC; ++e) dot = fmaf(g[v][e], p[v][e], dot);
      }
    }
    dot = warp_sum_f32(dot);
    char* orow = static_cast<char*>(dS) + row * Tk * ElemBytes<ODT>::v;
#pragma unroll
    for (int v = 0; v < kSmVpt; ++v) {
      const int vi = lane + v * 32;
      if (vi < n_vec) {
        float o[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) o[e] = p[v][e] * (g[v][e] - dot);
        uint32_t ow[OB / 4];
        encode_vec<ODT, VEC>(o, ow);
        st_raw<OB>(orow + static_cast<long long>(vi) * OB, ow);
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && ds_scale) *ds_scale = load_scale(dp_scale) * load_scale(p_scale);
}

static int rows_grid(long long rows, int rows_per_block) {
  long long need = (rows + rows_per_block - 1) / rows_per_block;
  const long long cap = static_cast<long long>(sm_count()) * 16;
  if (need < 1) need = 1;
  return static_cast<int>(need < cap ? need : cap);
}

int launch_softmax_fwd(const void* S, int s_dt, void* P, int p_dt, long long rows, int Tq, int Tk, int causal,
                       const float* s_scale, float* p_scale, cudaStream_t st) {
  if (Tk * elem_size(s_dt) / 16 > 32 * kSmVpt) return SCALIFY_ERR_UNSUPPORTED;
  const int grid = rows_grid(rows, 4);
  SCALIFY_DISPATCH_WIDE(s_dt, SDT, SCALIFY_DISPATCH_DTYPE(p_dt, PDT,
      softmax_fwd_kernel<SDT, PDT><<<grid, 128, 0, st>>>(S, P, rows, Tq, Tk, causal, s_scale, p_scale)));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

int launch_softmax_bwd(const void* dP, int g_dt, const void* P, int p_dt, void* dS, int o_dt, long long rows, int Tk,
                       const float* dp_scale, const float* p_scale, float* ds_scale, cudaStream_t st) {
  if (Tk * elem_size(g_dt) / 16 > 32 * kSmVpt) return SCALIFY_ERR_UNSUPPORTED;
  const int grid = rows_grid(rows, 4);
  // P: the probabilities as used in the forward (E4M3 matmul operand) or a 16-bit copy; dS: 16-bit or FP8
  if (!(p_dt == SCALIFY_E4M3 || p_dt == SCALIFY_BF16 || p_dt == SCALIFY_F16 || p_dt == SCALIFY_F32))
    return SCALIFY_ERR_UNSUPPORTED;
#define SCALIFY_SM_BWD(PD)                                                                                   \
  SCALIFY_DISPATCH_DTYPE(o_dt, ODT, softmax_bwd_kernel<GDT, PD, ODT><<<grid, 128, 0, st>>>(dP, P, dS, rows, Tk, \
                                                                                          dp_scale, p_scale, ds_scale))
  SCALIFY_DISPATCH_WIDE(g_dt, GDT, {
    if (p_dt == SCALIFY_E4M3) { SCALIFY_SM_BWD(SCALIFY_E4M3); }
    else if (p_dt == SCALIFY_BF16) { SCALIFY_SM_BWD(SCALIFY_BF16); }
    else if (p_dt == SCALIFY_F16) { SCALIFY_SM_BWD(SCALIFY_F16); }
    else { SCALIFY_SM_BWD(SCALIFY_F32); }
  });
#undef SCALIFY_SM_BWD
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// mean cross-entropy over n rows (logsumexp, Appendix B) and its gradient
// ---------------------------------------------------------------------------------------------
// One block per row; three sweeps over the row (max, sum of exponentials, gradient), the second and
// third served by L1/L2.  Per-row losses go to the workspace and are summed in row order.
template <int LDT, int GDT>
__global__ void __launch_bounds__(256) cross_entropy_kernel(const void* __restrict__ logits, long long ld, int n_classes,
                                                            const long long* __restrict__ targets, long long n,
                                                            const float* l_scale, void* __restrict__ dlogits,
                                                            float rem, float* __restrict__ row_loss,
                                                            uint32_t* bad_index) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  __shared__ float s_red[8];
  __shared__ float s_bcast;
  const float ls = load_scale(l_scale) * 1.4426950408889634f;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (long long row = blockIdx.x; row < n; row += gridDim.x) {
    const char* lrow = static_cast<const char*>(logits) + row * ld * ElemBytes<LDT>::v;
    float mx = -INFINITY;
    for (int j = threadIdx.x; j < n_classes; j += 256) mx = fmaxf(mx, load_elem<LDT>(lrow, j) * ls);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    __syncthreads();
    if (lane == 0) s_red[warp] = mx;
    __syncthreads();
    mx = s_red[0];
#pragma unroll
    for (int k = 1; k < 8; ++k) mx = fmaxf(mx, s_red[k]);
    float sum = 0.f;
    for (int j = threadIdx.x; j < n_classes; j += 256) sum += exp2f(load_elem<LDT>(lrow, j) * ls - mx);
    sum = warp_sum_f32(sum);
    __syncthreads();
    if (lane == 0) s_red[warp] = sum;
    __syncthreads();
    sum = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) sum += s_red[k];
    long long t = targets[row];
    if (t < 0 || t >= n_classes) {
      if (threadIdx.x == 0 && bad_index) atomicOr(bad_index, static_cast<uint32_t>(SCALIFY_DEV_BAD_INDEX));
      t = 0;
    }
    if (threadIdx.x == 0) {
      const float zt = load_elem<LDT>(lrow, t) * ls;
      // loss in natural-log units: ln(sum) + (mx - zt)*ln2
      row_loss[row] = logf(sum) + (mx - zt) * 0.6931471805599453f;
      s_bcast = rem / sum;
    }
    __syncthreads();
    if (dlogits) {
      const float k = s_bcast;
      char* grow = static_cast<char*>(dlogits) + row * ld * ElemBytes<GDT>::v;
      for (long long j = threadIdx.x; j < ld; j += 256) {
        float g = 0.f;
        if (j < n_classes) {
          g = exp2f(load_elem<LDT>(lrow, j) * ls - mx) * k;
          if (j == t) g -= rem;
        }
        store_elem<GDT>(grow, j, g);
      }
    }
  }
}

// The same with the row kept in shared memory (rows of up to 110 KB: a 50k-class row of 16-bit logits):
// one 16-byte-vector sweep over HBM, the other two over shared memory.
constexpr int kCeSmemMax = 110 * 1024;

// 2^x for x <= 0: the hardware approximation (2 ulp of fp32; results below 2^-126 flush to zero)
__device__ __forceinline__ float ce_exp2(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

__device__ __forceinline__ void ce_cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))),
               "l"(gmem_src)
               : "memory");
}

constexpr int kCeThreads = 512;

template <int LDT, int GDT>
__global__ void __launch_bounds__(kCeThreads, 2) cross_entropy_smem_kernel(const void* __restrict__ logits, long long ld,
                                                                    int n_classes, const long long* __restrict__ targets,
                                                                    long long n, const float* l_scale,
                                                                    void* __restrict__ dlogits, float rem,
                                                                    float* __restrict__ row_loss, uint32_t* bad_index) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<LDT>::v;
  constexpr int GB = VEC * ElemBytes<GDT>::v;
  extern __shared__ uint4 s_row[];
  // one array per reduction: a write is separated from the previous row's reads of the same array by the
  // barriers of the other reduction, so no barrier is needed in front of it
  __shared__ float s_max[kCeThreads / 32], s_sum[kCeThreads / 32];
  __shared__ float s_bcast;
  const float ls = load_scale(l_scale) * 1.4426950408889634f;  // positive: the maximum commutes with it
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nv_full = n_classes / VEC;               // vectors made of classes only
  const int n_part = n_classes - nv_full * VEC;      // classes in the one partial vector (0: none)
  const int nv = nv_full + (n_part ? 1 : 0);
  const int nv_ld = static_cast<int>(ld / VEC);      // vectors of the padded row (the gradient covers them all)
  // A row travels as 16-byte asynchronous copies straight into shared memory (about 100 KB in flight per
  // block for a 50k vocabulary, no registers held) and the three sweeps read it from there.  Every sweep
  // gives thread t the vectors t, t + 512, ...: a thread reads only what it copied itself, so the copies
  // need no barrier, and the last sweep refills each slot with the NEXT row's vector as soon as it has
  // read it - the next row loads behind this row's exponentials.
  auto row_ptr = [&](long long r) {
    return reinterpret_cast<const uint4*>(static_cast<const char*>(logits) + r * ld * ElemBytes<LDT>::v);
  };
  if (blockIdx.x < n) {
    const uint4* first = row_ptr(blockIdx.x);
    for (int v = threadIdx.x; v < nv; v += kCeThreads) ce_cp_async16(&s_row[v], first + v);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  for (long long row = blockIdx.x; row < n; row += gridDim.x) {
    const uint4* lrow = row_ptr(row);
    const long long next = row + gridDim.x;
    const uint4* nrow = row_ptr(next < n ? next : row);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    float mraw = -INFINITY;  // maximum of the data component
    for (int v = threadIdx.x; v < nv; v += kCeThreads) {
      const uint4 w = s_row[v];
      float f[VEC];
      decode_vec<LDT, VEC>(reinterpret_cast<const uint32_t*>(&w), f);
      if (v < nv_full) {
#pragma unroll
        for (int e = 0; e < VEC; ++e) mraw = fmaxf(mraw, f[e]);
      } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e)
          if (e < n_part) mraw = fmaxf(mraw, f[e]);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mraw = fmaxf(mraw, __shfl_xor_sync(0xFFFFFFFFu, mraw, o));
    if (lane == 0) s_max[warp] = mraw;
    __syncthreads();
    mraw = s_max[0];
#pragma unroll
    for (int k = 1; k < kCeThreads / 32; ++k) mraw = fmaxf(mraw, s_max[k]);
    const float mx = mraw * ls;
    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
    for (int v = threadIdx.x; v < nv; v += kCeThreads) {
      const uint4 w = s_row[v];
      float f[VEC];
      decode_vec<LDT, VEC>(reinterpret_cast<const uint32_t*>(&w), f);
      if (v < nv_full) {
#pragma unroll
        for (int e = 0; e < VEC; ++e) sum4[e & 3] += ce_exp2(fmaf(f[e], ls, -mx));
      } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e)
          if (e < n_part) sum4[e & 3] += ce_exp2(fmaf(f[e], ls, -mx));
      }
    }
    float sum = warp_sum_f32((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
    if (lane == 0) s_sum[warp] = sum;
    __syncthreads();
    sum = 0.f;
#pragma unroll
    for (int k = 0; k < kCeThreads / 32; ++k) sum += s_sum[k];
    long long t = targets[row];
    if (t < 0 || t >= n_classes) {
      if (threadIdx.x == 0 && bad_index) atomicOr(bad_index, static_cast<uint32_t>(SCALIFY_DEV_BAD_INDEX));
      t = 0;
    }
    if (threadIdx.x == 0) {
      const float zt = load_elem<LDT>(lrow, t) * ls;
      row_loss[row] = logf(sum) + (mx - zt) * 0.6931471805599453f;
      s_bcast = rem / sum;
    }
    __syncthreads();
    if (dlogits) {
      const float k = s_bcast;
      const int tv = static_cast<int>(t / VEC), te = static_cast<int>(t % VEC);
      char* grow = static_cast<char*>(dlogits) + row * ld * ElemBytes<GDT>::v;
      for (int v = threadIdx.x; v < nv_ld; v += kCeThreads) {
        float g[VEC];
        if (v < nv) {
          const uint4 w = s_row[v];
          if (next < n) ce_cp_async16(&s_row[v], nrow + v);
          float f[VEC];
          decode_vec<LDT, VEC>(reinterpret_cast<const uint32_t*>(&w), f);
#pragma unroll
          for (int e = 0; e < VEC; ++e) g[e] = ce_exp2(fmaf(f[e], ls, -mx)) * k;
          if (v >= nv_full) {
#pragma unroll
            for (int e = 0; e < VEC; ++e)
              if (e >= n_part) g[e] = 0.f;
          }
          if (v == tv) {
#pragma unroll
            for (int e = 0; e < VEC; ++e)
              if (e == te) g[e] -= rem;
          }
        } else {
#pragma unroll
          for (int e = 0; e < VEC; ++e) g[e] = 0.f;
        }
        uint32_t o[GB / 4 > 0 ? GB / 4 : 1];
        encode_vec<GDT, VEC>(g, o);
        st_raw_stream<GB>(grow + static_cast<long long>(v) * GB, o);
      }
      for (long long j = static_cast<long long>(nv_ld) * VEC + threadIdx.x; j < ld; j += kCeThreads) store_elem<GDT>(grow, j, 0.f);
    } else if (next < n) {
      for (int v = threadIdx.x; v < nv; v += kCeThreads) ce_cp_async16(&s_row[v], nrow + v);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
}

__global__ void __launch_bounds__(256) cross_entropy_finalize_kernel(const float* __restrict__ row_loss, long long n,
                                                                     float* loss, float* g_scale, float gs) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  __shared__ double s[8];
  double acc = 0.0;
  for (long long i = threadIdx.x; i < n; i += 256) acc += static_cast<double>(row_loss[i]);
  acc = warp_sum_f64(acc);
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int i = 0; i < 8; ++i) tot += s[i];
    *loss = static_cast<float>(tot / static_cast<double>(n));
    if (g_scale) *g_scale = gs;
  }
}

size_t cross_entropy_ws_bytes(int64_t n) { return kWsHeader + static_cast<size_t>(n) * sizeof(float) + 256; }

int launch_cross_entropy(const void* logits, int l_dt, long long ld, int n_classes, const long long* targets, long long n,
                         const float* l_scale, float* loss, void* dlogits, int g_dt, float* g_scale, void* ws,
                         cudaStream_t st) {
  WsView v = ws_view(ws);
  float* row_loss = static_cast<float*>(v.area);
  // 1/n = gs * rem with gs a power of two (rounded down) and rem in [1,2) kept in the data
  int ex;
  frexp(1.0 / static_cast<double>(n), &ex);
  const double gs = ldexp(1.0, ex - 1);
  const float rem = static_cast<float>((1.0 / static_cast<double>(n)) / gs);
  const long long cap = static_cast<long long>(sm_count()) * 8;
  const int grid = static_cast<int>(n < cap ? n : cap);
  const int les = elem_size(l_dt), lvec = 16 / les;
  const long long row_smem = static_cast<long long>((n_classes + lvec - 1) / lvec) * 16;
  // the vector path needs 16-byte-aligned rows on both sides and a gradient vector of at least 4 bytes
  const bool vec_ok = row_smem <= kCeSmemMax && (ld * les) % 16 == 0 && (!dlogits || (ld * elem_size(g_dt)) % 16 == 0) &&
                      lvec * elem_size(g_dt) >= 4 && reinterpret_cast<uintptr_t>(logits) % 16 == 0 &&
                      reinterpret_cast<uintptr_t>(dlogits) % 16 == 0;
  if (vec_ok) {
    const long long cap2 = static_cast<long long>(sm_count()) * 2;
    const int grid2 = static_cast<int>(n < cap2 ? n : cap2);
    SCALIFY_DISPATCH_WIDE(l_dt, LDT, SCALIFY_DISPATCH_DTYPE(g_dt, GDT, {
      auto kernel = cross_entropy_smem_kernel<LDT, GDT>;
      static DeviceOnce once;  // (one per instantiation: the attribute belongs to this kernel on this device)
      int rc_once = device_once(once, nullptr, [&](int*) {
        SCALIFY_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCeSmemMax));
        return int(SCALIFY_OK);
      });
      if (rc_once) return rc_once;
      kernel<<<grid2, kCeThreads, static_cast<size_t>(row_smem), st>>>(logits, ld, n_classes, targets, n, l_scale, dlogits, rem,
                                                               row_loss, v.status);
    }));
  } else {
    SCALIFY_DISPATCH_WIDE(l_dt, LDT, SCALIFY_DISPATCH_DTYPE(g_dt, GDT,
        cross_entropy_kernel<LDT, GDT><<<grid, 256, 0, st>>>(logits, ld, n_classes, targets, n, l_scale, dlogits, rem,
                                                             row_loss, v.status)));
  }
  SCALIFY_CUDA_TRY(cudaGetLastError());
  cross_entropy_finalize_kernel<<<1, 256, 0, st>>>(row_loss, n, loss, g_scale, static_cast<float>(gs));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// column sums of a scaled matrix (Section 3.2, the rule for a sum of R independent terms: the data
// component is divided by kf(R), the scale multiplied by it) - the bias gradient of a linear layer
// ---------------------------------------------------------------------------------------------
// Launch 1: a block is 32 vectors of columns wide and takes one slab of rows; its eight warps stride over
// the slab's rows (four rows in flight per thread), are added in warp order through shared memory, and
// leave one fp32 partial per column and slab.  Launch 2 adds the slabs in index order in fp64.
constexpr int kColSlabsMax = 64;  // the finish adds 8 x 8 slabs

// CDT >= 0: the fused cast (Appendix A: cast_on_backward of a gradient) - the input is also written to C in
// format CDT, and the sums are those of the values AS CAST, so that the result is what the cast followed by
// the column sums of its output gives.
template <int DT, int CDT = -1>
__global__ void __launch_bounds__(256) colsum_partial_kernel(const void* __restrict__ X, long long ld, long long R,
                                                             long long N, int slabs, float* __restrict__ part,
                                                             void* __restrict__ C = nullptr, long long ldc = 0) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<DT>::v;
  __shared__ float s_acc[8][32][VEC + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long n_vec = N / VEC;
  const int tail = static_cast<int>(N - n_vec * VEC);
  const long long vec = static_cast<long long>(blockIdx.x) * 32 + lane;  // vector of columns (n_vec: the ragged end)
  const long long rows_per_slab = (R + slabs - 1) / slabs;
  const long long r0 = blockIdx.y * rows_per_slab, r1 = min(R, r0 + rows_per_slab);
  float acc[VEC];
#pragma unroll
  for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
  if (vec < n_vec) {
    const char* base = static_cast<const char*>(X) + vec * 16;
    for (long long r = r0 + warp; r < r1; r += 32) {
      uint32_t w[4][4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
#pragma unroll
        for (int q = 0; q < 4; ++q) w[u][q] = 0u;  // zero bits decode to 0.0 in every format
        if (r + u * 8 < r1) ld_raw_stream<16>(base + (r + u * 8) * ld * ElemBytes<DT>::v, w[u]);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float f[VEC];
        decode_vec<DT, VEC>(w[u], f);
        if constexpr (CDT >= 0) {
          if (r + u * 8 < r1) {
            constexpr int CB = VEC * ElemBytes<CDT>::v;
            uint32_t cw[CB / 4];
            encode_vec<CDT, VEC>(f, cw);
            st_raw_stream<CB>(static_cast<char*>(C) + ((r + u * 8) * ldc + vec * VEC) * ElemBytes<CDT>::v, cw);
            decode_vec<CDT, VEC>(cw, f);   // the values as cast
          }
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] += f[e];
      }
    }
  } else if (vec == n_vec && tail > 0) {
    for (long long r = r0 + warp; r < r1; r += 8)
      for (int e = 0; e < tail; ++e) {
        float f = load_elem<DT>(X, r * ld + n_vec * VEC + e);
        if constexpr (CDT >= 0) {
          store_elem<CDT>(C, r * ldc + n_vec * VEC + e, f);
          f = round_through<CDT>(f);
        }
        acc[e] += f;
      }
  }
#pragma unroll
  for (int e = 0; e < VEC; ++e) s_acc[warp][lane][e] = acc[e];
  __syncthreads();
  // thread t adds the eight warps' values of (lane t / VEC... ) one column each: 32 * VEC columns per block
  for (int c = threadIdx.x; c < 32 * VEC; c += 256) {
    const int l = c / VEC, e = c % VEC;
    float sum = s_acc[0][l][e];
#pragma unroll
    for (int wv = 1; wv < 8; ++wv) sum += s_acc[wv][l][e];
    const long long col = (static_cast<long long>(blockIdx.x) * 32 + l) * VEC + e;
    if (col < N) part[static_cast<long long>(blockIdx.y) * N + col] = sum;
  }
}

// 32 columns per block; the eight warps each add eight slabs (index order, fp64), warp 0 adds the eight sums
template <int YDT>
__global__ void __launch_bounds__(256) colsum_finalize_kernel(const float* __restrict__ part, long long N, int slabs,
                                                              float inv_kf, float kf, void* __restrict__ Y,
                                                              const float* x_scale, float* y_scale, uint32_t* status,
                                                              float* c_scale = nullptr) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  __shared__ double s_sum[8][32];
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
  const long long col = static_cast<long long>(blockIdx.x) * 32 + lane;
  double sum = 0.0;
  if (col < N) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = (grp * 8 + u < slabs) ? part[static_cast<long long>(grp * 8 + u) * N + col] : 0.f;
#pragma unroll
    for (int u = 0; u < 8; ++u) sum += static_cast<double>(v[u]);
  }
  s_sum[grp][lane] = sum;
  __syncthreads();
  if (grp == 0 && col < N) {
    double tot = s_sum[0][lane];
#pragma unroll
    for (int g = 1; g < 8; ++g) tot += s_sum[g][lane];
    store_elem<YDT>(Y, col, static_cast<float>(tot * static_cast<double>(inv_kf)));
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    const float xs = load_scale(x_scale);
    if (y_scale) *y_scale = xs * kf;
    if (c_scale) *c_scale = xs;   // fused cast: the scale is unchanged
    if (!is_pow2_scale(xs) && status) atomicOr(status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
  }
}

static int colsum_slabs(long long R, long long N, int elem_bytes) {
  const long long gx = (N / (16 / elem_bytes) + 1 + 31) / 32;
  long long s = (static_cast<long long>(sm_count()) * 8 + gx - 1) / gx;   // about eight blocks per SM
  const long long by_rows = (R + 31) / 32;                                 // at least 32 rows per slab
  if (s > by_rows) s = by_rows;
  if (s > kColSlabsMax) s = kColSlabsMax;
  return static_cast<int>(s < 1 ? 1 : s);
}

size_t colsum_ws_bytes(int64_t N) { return kWsHeader + static_cast<size_t>(kColSlabsMax) * static_cast<size_t>(N) * sizeof(float) + 256; }

int launch_colsum(const void* X, int x_dt, long long ld, long long R, long long N, const float* x_scale, void* Y, int y_dt,
                  float* y_scale, void* ws, cudaStream_t st) {
  WsView v = ws_view(ws);
  float* part = static_cast<float*>(v.area);
  const int es = elem_size(x_dt);
  const int slabs = colsum_slabs(R, N, es);
  const long long gx = (N / (16 / es) + 1 + 31) / 32;
  if (gx > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
  const dim3 grid(static_cast<unsigned>(gx), static_cast<unsigned>(slabs));
  SCALIFY_DISPATCH_DTYPE(x_dt, DT, colsum_partial_kernel<DT><<<grid, 256, 0, st>>>(X, ld, R, N, slabs, part));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  const float kf = kfactor(R);
  SCALIFY_DISPATCH_WIDE(y_dt, YDT, colsum_finalize_kernel<YDT><<<static_cast<unsigned>((N + 31) / 32), 256, 0, st>>>(
                                       part, N, slabs, 1.0f / kf, kf, Y, x_scale, y_scale, v.status));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// Cast of a 16-bit matrix to FP8 fused with the column sums of the cast values (the bias gradient of a linear
// layer is the column sum of the E5M2 copy of the output gradient that the weight-gradient matmul reads).  The
// slabs are those the column sums of an FP8 matrix would get, and every column is added in the same order, so
// the sums equal those of scalify_scaled_colsum applied to the cast output bit for bit.
int launch_cast_colsum(const void* X, int x_dt, long long ld, long long R, long long N, const float* x_scale, void* C,
                       int c_dt, long long ldc, float* c_scale, void* Y, int y_dt, float* y_scale, void* ws,
                       cudaStream_t st) {
  WsView v = ws_view(ws);
  float* part = static_cast<float*>(v.area);
  const int slabs = colsum_slabs(R, N, 1);
  const long long gx = (N / 8 + 1 + 31) / 32;   // vectors of eight 16-bit columns
  if (gx > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
  const dim3 grid(static_cast<unsigned>(gx), static_cast<unsigned>(slabs));
#define SCALIFY_CCS(DT, CDT) colsum_partial_kernel<DT, CDT><<<grid, 256, 0, st>>>(X, ld, R, N, slabs, part, C, ldc)
  if (x_dt == SCALIFY_BF16) {
    if (c_dt == SCALIFY_E4M3) SCALIFY_CCS(SCALIFY_BF16, SCALIFY_E4M3); else SCALIFY_CCS(SCALIFY_BF16, SCALIFY_E5M2);
  } else {
    if (c_dt == SCALIFY_E4M3) SCALIFY_CCS(SCALIFY_F16, SCALIFY_E4M3); else SCALIFY_CCS(SCALIFY_F16, SCALIFY_E5M2);
  }
#undef SCALIFY_CCS
  SCALIFY_CUDA_TRY(cudaGetLastError());
  const float kf = kfactor(R);
  SCALIFY_DISPATCH_WIDE(y_dt, YDT, colsum_finalize_kernel<YDT><<<static_cast<unsigned>((N + 31) / 32), 256, 0, st>>>(
                                       part, N, slabs, 1.0f / kf, kf, Y, x_scale, y_scale, v.status, c_scale));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// Diagnostic: the fp32-pipe BF16 rounding used inside the attention kernels, applied to an array; the
// two-wide form takes the elements in pairs (a last odd element goes through the scalar form)
template <bool TWO_WIDE>
__global__ void __launch_bounds__(256) bf16_round_kernel(const float* __restrict__ x, float* __restrict__ y, long long n) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  const long long t0 = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x, step = static_cast<long long>(gridDim.x) * 256;
  if constexpr (TWO_WIDE) {
    for (long long i = t0; i < n / 2; i += step) {
      const float2 r = bf16_round_f32x2(make_float2(x[2 * i], x[2 * i + 1]));
      y[2 * i] = r.x;
      y[2 * i + 1] = r.y;
    }
    if ((n & 1) && t0 == 0) y[n - 1] = bf16_round_f32(x[n - 1]);
  } else {
    for (long long i = t0; i < n; i += step) y[i] = bf16_round_f32(x[i]);
  }
}

int launch_bf16_round(const float* x, float* y, long long n, int two_wide, cudaStream_t st) {
  const long long blocks = (n + 255) / 256;
  const unsigned grid = static_cast<unsigned>(blocks < 148 * 16 ? blocks : 148 * 16);
  if (two_wide) bf16_round_kernel<true><<<grid, 256, 0, st>>>(x, y, n);
  else bf16_round_kernel<false><<<grid, 256, 0, st>>>(x, y, n);
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// debug build: the table of registered byte ranges (host shadow, device copy) and its report
// ---------------------------------------------------------------------------------------------
#ifdef SCALIFY_DEBUG
}  // namespace scalify
#include <algorithm>
#include <mutex>
#include <vector>
namespace scalify {
static __device__ DbgTable g_dbg_storage;
namespace {
std::mutex g_dbg_mu;
std::vector<DbgSetPointerFn>& dbg_units() { static std::vector<DbgSetPointerFn> v; return v; }
std::vector<std::pair<unsigned long long, unsigned long long>> g_dbg_ranges;  // sorted, disjoint
bool g_dbg_pointers_set[64] = {};
long long g_dbg_limit = -1;  // self-test: cap on the length of every range registered from now on
}  // namespace

void dbg_add_translation_unit(DbgSetPointerFn fn) { dbg_units().push_back(fn); }

static cudaError_t dbg_upload() {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  DbgTable* dptr = nullptr;
  if ((e = cudaGetSymbolAddress(reinterpret_cast<void**>(&dptr), g_dbg_storage)) != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && !g_dbg_pointers_set[dev]) {
    for (DbgSetPointerFn fn : dbg_units())
      if ((e = fn(dptr)) != cudaSuccess) return e;
    g_dbg_pointers_set[dev] = true;
  }
  const int n = static_cast<int>(g_dbg_ranges.size());
  std::vector<unsigned long long> lo(n), hi(n);
  for (int i = 0; i < n; ++i) { lo[i] = g_dbg_ranges[i].first; hi[i] = g_dbg_ranges[i].second; }
  // synchronous copies: the debug build is not meant for stream capture or for timing
  if (n && (e = cudaMemcpy(dptr->lo, lo.data(), n * sizeof(unsigned long long), cudaMemcpyHostToDevice)) != cudaSuccess) return e;
  if (n && (e = cudaMemcpy(dptr->hi, hi.data(), n * sizeof(unsigned long long), cudaMemcpyHostToDevice)) != cudaSuccess) return e;
  return cudaMemcpy(&dptr->n, &n, sizeof(int), cudaMemcpyHostToDevice);
}

void dbg_register_range(const void* base, unsigned long long bytes) {
  if (!base || bytes == 0) return;
  std::lock_guard<std::mutex> lock(g_dbg_mu);
  if (g_dbg_limit >= 0 && bytes > static_cast<unsigned long long>(g_dbg_limit)) bytes = static_cast<unsigned long long>(g_dbg_limit);
  unsigned long long lo = reinterpret_cast<unsigned long long>(base), hi = lo + bytes;
  // already covered: nothing to do (the common case: the same buffers call after call)
  for (const auto& r : g_dbg_ranges)
    if (r.first <= lo && hi <= r.second) return;
  // merge with every range it touches, keep the list sorted and disjoint
  std::vector<std::pair<unsigned long long, unsigned long long>> out;
  for (const auto& r : g_dbg_ranges) {
    if (r.second < lo || hi < r.first) out.push_back(r);
    else { lo = std::min(lo, r.first); hi = std::max(hi, r.second); }
  }
  out.emplace_back(lo, hi);
  std::sort(out.begin(), out.end());
  if (static_cast<int>(out.size()) > kDbgMaxRanges) out.erase(out.begin(), out.begin() + (out.size() - kDbgMaxRanges));
  g_dbg_ranges.swap(out);
  (void)dbg_upload();
}

int debug_bounds_report(unsigned long long out[3], int reset_ranges, long long limit) {
  std::lock_guard<std::mutex> lock(g_dbg_mu);
  DbgTable* dptr = nullptr;
  SCALIFY_CUDA_TRY(cudaDeviceSynchronize());
  SCALIFY_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&dptr), g_dbg_storage));
  unsigned long long v[3] = {0, 0, 0};
  SCALIFY_CUDA_TRY(cudaMemcpy(v, &dptr->violations, sizeof(v), cudaMemcpyDeviceToHost));
  if (out) { out[0] = v[0]; out[1] = v[1]; out[2] = v[2]; }
  const unsigned long long zero[3] = {0, 0, 0};
  SCALIFY_CUDA_TRY(cudaMemcpy(&dptr->violations, zero, sizeof(zero), cudaMemcpyHostToDevice));
  g_dbg_limit = limit;
  if (reset_ranges) {
    g_dbg_ranges.clear();
    SCALIFY_CUDA_TRY(dbg_upload());
  }
  return SCALIFY_OK;
}
#else
int debug_bounds_report(unsigned long long*, int, long long) { return SCALIFY_ERR_UNSUPPORTED; }
#endif

}  // namespace scalify
