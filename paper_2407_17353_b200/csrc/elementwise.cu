// HBM-bound scaled elementwise kernels: statistic, rebalance / set_scaling /
// cast, scaled add, scaled GELU.  Every kernel moves 16-byte vectors of its
// widest operand per thread access, coalesced across the warp, with several
// independent accesses in flight per thread; the grid is a multiple of the SM
// count and strides over the array.
#include "scalify_common.cuh"
#include "scalify_launch.h"
#include <cooperative_groups.h>
namespace cg = cooperative_groups;

namespace scalify {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;

template <int A, int B> struct VecElems {
  static constexpr int big = ElemBytes<A>::v > ElemBytes<B>::v ? ElemBytes<A>::v : ElemBytes<B>::v;
  static constexpr int v = 16 / big;
};

// One tile per block.  Measured on B200 (256 MiB BF16 copy-shaped pass): 6240 GB/s, against 5640 GB/s
// for a grid capped at 8 blocks per SM that strides over the tiles - the hardware scheduler hands a
// new block to whichever SM finishes first, so no SM waits on a last partial round of the stride.
static int grid_all_tiles(int64_t n_vec) {
  int64_t tiles = (n_vec + int64_t(kThreads) * kUnroll - 1) / (int64_t(kThreads) * kUnroll);
  if (tiles < 1) tiles = 1;
  return static_cast<int>(tiles < 0x7FFFFFFF ? tiles : 0x7FFFFFFF);
}

static int grid_for(int64_t n_vec, int blocks_per_sm) {
  int64_t tiles = (n_vec + int64_t(kThreads) * kUnroll - 1) / (int64_t(kThreads) * kUnroll);
  int64_t cap = int64_t(sm_count()) * blocks_per_sm;
  if (tiles < 1) tiles = 1;
  return static_cast<int>(tiles < cap ? tiles : cap);
}

// ---------------------------------------------------------------------------------------------
// statistic of the data component (Section 3.3): AMAX or root mean square
// ---------------------------------------------------------------------------------------------
// Each block leaves one partial (AMAX: bit pattern of max|x|; L2: fp64 sum of squares) in
// `partials`; the block that draws the last ticket combines them in index order, so the result
// does not depend on scheduling.
template <int DT>
__global__ void __launch_bounds__(kThreads) statistic_kernel(const void* __restrict__ x, int64_t n, int stat,
                                                             double* __restrict__ partials, uint32_t* ticket,
                                                             float* stat_word, float* out_stat) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<DT>::v;
  constexpr int WORDS = 4;
  const int64_t n_vec = n / VEC;
  uint32_t amax = 0u;
  float ssq = 0.f;
  // every block reads one contiguous run of vectors; the runs differ by at most one vector
  const int64_t v0 = n_vec / gridDim.x * blockIdx.x + min(int64_t(blockIdx.x), int64_t(n_vec % gridDim.x));
  const int64_t v1 = v0 + n_vec / gridDim.x + (blockIdx.x < n_vec % gridDim.x ? 1 : 0);
  for (int64_t base = v0; base < v1; base += kThreads * kUnroll) {
    uint32_t w[kUnroll][WORDS];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < v1) ld_raw<16>(static_cast<const char*>(x) + i * 16, w[u]);
      else { w[u][0] = w[u][1] = w[u][2] = w[u][3] = 0u; }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float f[VEC];
      decode_vec<DT, VEC>(w[u], f);
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        amax = max(amax, abs_bits(f[e]));
        ssq = fmaf(f[e], f[e], ssq);
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < static_cast<int>(n - n_vec * VEC)) {
    float f = load_elem<DT>(x, n_vec * VEC + threadIdx.x);
    amax = max(amax, abs_bits(f));
    ssq = fmaf(f, f, ssq);
  }
  __shared__ double s_part[kThreads / 32];
  __shared__ bool s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double mine;
  if (stat == SCALIFY_STAT_AMAX) {
    amax = warp_max_u32(amax);
    mine = static_cast<double>(amax);
  } else {
    mine = warp_sum_f64(static_cast<double>(ssq));
  }
  if (lane == 0) s_part[warp] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot;
    if (stat == SCALIFY_STAT_AMAX) {
      uint32_t m = 0u;
      for (int i = 0; i < kThreads / 32; ++i) m = max(m, static_cast<uint32_t>(s_part[i]));
      tot = static_cast<double>(m);
    } else {
      tot = 0.0;
      for (int i = 0; i < kThreads / 32; ++i) tot += s_part[i];
    }
    partials[blockIdx.x] = tot;
    __threadfence();
    uint32_t t = atomicAdd(ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // fixed-order combination of the per-block partials
  double acc = 0.0;
  uint32_t accm = 0u;
  for (int i = threadIdx.x; i < static_cast<int>(gridDim.x); i += kThreads) {
    double p = __ldcg(&partials[i]);
    if (stat == SCALIFY_STAT_AMAX) accm = max(accm, static_cast<uint32_t>(p));
    else acc += p;
  }
  if (stat == SCALIFY_STAT_AMAX) {
    accm = warp_max_u32(accm);
    acc = static_cast<double>(accm);
  } else {
    acc = warp_sum_f64(acc);
  }
  __syncthreads();
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float result;
    if (stat == SCALIFY_STAT_AMAX) {
      uint32_t m = 0u;
      for (int i = 0; i < kThreads / 32; ++i) m = max(m, static_cast<uint32_t>(s_part[i]));
      result = __uint_as_float(m);
    } else {
      double tot = 0.0;
      for (int i = 0; i < kThreads / 32; ++i) tot += s_part[i];
      result = static_cast<float>(sqrt(tot / static_cast<double>(n)));
    }
    *stat_word = result;
    if (out_stat) *out_stat = result;
    *ticket = 0u;
  }
}

// Blocks wanted for a statistic over n elements of at most 4 bytes: about four tiles each (many
// more blocks than fit on the device at once, so the hardware scheduler balances them), at most 65536.
int64_t statistic_blocks_wanted(int64_t n, int elem_bytes) {
  const int64_t tiles = (n * elem_bytes / 16 + int64_t(kThreads) * kUnroll - 1) / (int64_t(kThreads) * kUnroll);
  int64_t blocks = (tiles + 3) / 4;
  const int64_t floor_blocks = int64_t(sm_count()) * 8;
  if (blocks < floor_blocks) blocks = tiles < floor_blocks ? (tiles > 0 ? tiles : 1) : floor_blocks;
  return blocks < 65536 ? blocks : 65536;
}

int launch_statistic(const void* x, int dtype, int64_t n, int stat, void* ws, size_t ws_bytes, float* out_stat,
                     cudaStream_t st) {
  WsView v = ws_view(ws);
  // one partial per block: a workspace smaller than scalify_workspace_bytes() asks for gets fewer blocks
  int64_t grid = statistic_blocks_wanted(n, elem_size(dtype));
  const int64_t room = static_cast<int64_t>((ws_bytes - kWsHeader) / sizeof(double));
  if (grid > room) grid = room;
  if (grid < 1) grid = 1;
  SCALIFY_DISPATCH_DTYPE(dtype, DT,
      statistic_kernel<DT><<<static_cast<int>(grid), kThreads, 0, st>>>(x, n, stat, static_cast<double*>(v.area),
                                                                       v.ticket, v.stat, out_stat));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// rebalance / set_scaling / cast (Sections 3.1, 3.3; Algorithm 4; Appendix A casts)
// ---------------------------------------------------------------------------------------------

template <int IN, int OUT>
__global__ void __launch_bounds__(kThreads) rebalance_kernel(const void* __restrict__ x, void* __restrict__ y,
                                                             int64_t n, const float* x_scale, float* y_scale,
                                                             const float* stat, const float* new_scale, int mode,
                                                             uint32_t* status) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = VecElems<IN, OUT>::v;
  constexpr int IB = VEC * ElemBytes<IN>::v, OB = VEC * ElemBytes<OUT>::v;
  const float xs = load_scale(x_scale);
  float factor = 1.0f, out_scale = xs;
  uint32_t flags = is_pow2_scale(xs) ? 0u : SCALIFY_DEV_BAD_SCALE;
  if (mode == kModeDynamic) {
    bool nonfinite;
    float r = rescale_factor(__ldg(stat), &nonfinite);
    factor = 1.0f / r;  // exact: r is a power of two
    out_scale = xs * r;
    if (nonfinite) flags |= SCALIFY_DEV_NONFINITE_STAT;
  } else if (mode == kModeSet) {
    float req = __ldg(new_scale);
    float ns = p2_floor(req);
    if (!(req > 0.f) || !is_pow2_scale(ns)) { flags |= SCALIFY_DEV_BAD_SCALE; ns = 1.0f; }
    factor = xs / ns;
    out_scale = ns;
  }
  const int64_t n_vec = n / VEC;
  const int64_t n_tiles = (n_vec + kThreads * kUnroll - 1) / (kThreads * kUnroll);
  // A dynamic rescale runs right after the kernel that produced (or measured) the data, whose most
  // recently touched part - the end of the array - is still in L2: walk the array from the end.
  const bool reverse = (mode == kModeDynamic);
  for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int64_t base = (reverse ? n_tiles - 1 - tile : tile) * (kThreads * kUnroll);
    uint32_t w[kUnroll][IB / 4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < n_vec) ld_raw_stream<IB>(static_cast<const char*>(x) + i * IB, w[u]);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < n_vec) {
        float f[VEC];
        decode_vec<IN, VEC>(w[u], f);
#pragma unroll
        for (int e = 0; e < VEC; ++e) f[e] *= factor;
        uint32_t o[OB / 4];
        encode_vec<OUT, VEC>(f, o);
        st_raw<OB>(static_cast<char*>(y) + i * OB, o);
      }
    }
  }
  if (blockIdx.x == 0) {
    int tail = static_cast<int>(n - n_vec * VEC);
    if (threadIdx.x < tail) {
      int64_t i = n_vec * VEC + threadIdx.x;
      store_elem<OUT>(y, i, load_elem<IN>(x, i) * factor);
    }
    if (threadIdx.x == 0) {
      if (y_scale) *y_scale = out_scale;
      if (flags && status) atomicOr(status, flags);
    }
  }
}

int launch_rebalance(const void* x, int in_dt, void* y, int out_dt, int64_t n, const float* x_scale, float* y_scale,
                     const float* stat, const float* new_scale, int mode, uint32_t* status, cudaStream_t st) {
  int big = elem_size(in_dt) > elem_size(out_dt) ? elem_size(in_dt) : elem_size(out_dt);
  int64_t n_vec = n / (16 / big);
  int grid = grid_all_tiles(n_vec);
  SCALIFY_DISPATCH_DTYPE(in_dt, IN, SCALIFY_DISPATCH_DTYPE(out_dt, OUT,
      rebalance_kernel<IN, OUT><<<grid, kThreads, 0, st>>>(x, y, n, x_scale, y_scale, stat, new_scale, mode, status)));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// check of a speculative rescale (Section 3.3: dynamic rescale; the producer already wrote the
// rebalanced array with a PREDICTED power of two)
// ---------------------------------------------------------------------------------------------
// If the power of two of the true statistic equals the predicted one, y already holds the exact
// result and only the scale word is written; otherwise the array is rebalanced from x as usual.
template <int IN, int OUT>
__global__ void __launch_bounds__(kThreads) rebalance_check_kernel(const void* __restrict__ x, void* __restrict__ y,
                                                                   int64_t n, const float* x_scale, float* y_scale,
                                                                   const float* stat, const float* r_pred,
                                                                   float* hint_out, uint32_t* status) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  // launched as a programmatic dependent of the GEMM: its blocks are resident when the GEMM ends and start here
  asm volatile("griddepcontrol.wait;" ::: "memory");
  constexpr int VEC = VecElems<IN, OUT>::v;
  constexpr int IB = VEC * ElemBytes<IN>::v, OB = VEC * ElemBytes<OUT>::v;
  // One thread per block reads the three words the grid before this one wrote (input scale, statistic, the power
  // of two it divided by) and hands them to the others: the loads are volatile, because a load through the
  // read-only path may be scheduled above the wait and then sees what the words held before.
  __shared__ float s_words[3];
  if (threadIdx.x == 0) {
    s_words[0] = load_scale_after_wait(x_scale);
    s_words[1] = *reinterpret_cast<const volatile float*>(stat);
    s_words[2] = *reinterpret_cast<const volatile float*>(r_pred);
  }
  __syncthreads();
  const float xs = s_words[0];
  const float s = s_words[1];
  bool nonfinite;
  const float r = rescale_factor(s, &nonfinite);
  const float rp = s_words[2];
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    uint32_t flags = is_pow2_scale(xs) ? 0u : SCALIFY_DEV_BAD_SCALE;
    if (nonfinite) flags |= SCALIFY_DEV_NONFINITE_STAT;
    if (y_scale) *y_scale = xs * r;
    if (hint_out) *hint_out = s;  // the prediction for the next call
    if (flags && status) atomicOr(status, flags);
  }
  if (r == rp) return;
  const float factor = 1.0f / r;  // exact: r is a power of two
  const int64_t n_vec = n / VEC;
  const int64_t n_tiles = (n_vec + kThreads * kUnroll - 1) / (kThreads * kUnroll);
  for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int64_t base = tile * (kThreads * kUnroll);
    uint32_t w[kUnroll][IB / 4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < n_vec) ld_raw_stream<IB>(static_cast<const char*>(x) + i * IB, w[u]);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < n_vec) {
        float f[VEC];
        decode_vec<IN, VEC>(w[u], f);
#pragma unroll
        for (int e = 0; e < VEC; ++e) f[e] *= factor;
        uint32_t o[OB / 4];
        encode_vec<OUT, VEC>(f, o);
        st_raw<OB>(static_cast<char*>(y) + i * OB, o);
      }
    }
  }
  if (blockIdx.x == 0) {
    const int tail = static_cast<int>(n - n_vec * VEC);
    if (threadIdx.x < tail) {
      int64_t i = n_vec * VEC + threadIdx.x;
      store_elem<OUT>(y, i, load_elem<IN>(x, i) * factor);
    }
  }
}

int launch_rebalance_check(const void* x, int in_dt, void* y, int out_dt, int64_t n, const float* x_scale,
                           float* y_scale, const float* stat, const float* r_pred, float* hint_out,
                           uint32_t* status, cudaStream_t st) {
  const int64_t n_vec = n / (16 / 2);
  const int grid = grid_for(n_vec, 8);  // small grid: in the expected case every block returns at once
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3(unsigned(grid));
  cfg.blockDim = dim3(kThreads);
  cfg.stream = st;
#define SCALIFY_RBC(IN, OUT)                                                                                     \
  SCALIFY_CUDA_TRY(cudaLaunchKernelEx(&cfg, rebalance_check_kernel<IN, OUT>, x, y, n, x_scale, y_scale, stat, r_pred, \
                                      hint_out, status))
  if (in_dt == SCALIFY_BF16) {
    if (out_dt == SCALIFY_E4M3) SCALIFY_RBC(SCALIFY_BF16, SCALIFY_E4M3); else SCALIFY_RBC(SCALIFY_BF16, SCALIFY_E5M2);
  } else {
    if (out_dt == SCALIFY_E4M3) SCALIFY_RBC(SCALIFY_F16, SCALIFY_E4M3); else SCALIFY_RBC(SCALIFY_F16, SCALIFY_E5M2);
  }
#undef SCALIFY_RBC
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// dynamic rescale with a predicted power of two (Section 3.3: statistic and rebalancing are separate
// primitives): the array is read ONCE
// ---------------------------------------------------------------------------------------------
// While the statistic is gathered (as statistic_kernel does: one partial per block, the block that draws the
// last ticket combines them in index order), the output is already written with the power of two of the
// statistic the workspace saw last (*hint, any content).  rebalance_check_kernel follows as a programmatic
// dependent: it writes the scale word and the next prediction and returns at once when this call's statistic
// has the predicted power of two; otherwise it rebalances from x as usual.  Either way every element is
// computed as cast(x / r) with the same r, so the result does not depend on the prediction.
template <int IN, int OUT>
__global__ void __launch_bounds__(kThreads) rescale_predict_kernel(const void* __restrict__ x, void* __restrict__ y,
                                                                   int64_t n, int stat, const float* hint,
                                                                   float* r_used, double* __restrict__ partials,
                                                                   uint32_t* ticket, float* stat_word) {
  bool nf;
  const float pred_r = rescale_factor(*reinterpret_cast<const volatile float*>(hint), &nf);
  if (blockIdx.x == 0 && threadIdx.x == 0) *r_used = pred_r;
  asm volatile("griddepcontrol.launch_dependents;");  // the dependent sets up while this grid runs
  const float factor = 1.0f / pred_r;  // exact: a power of two
  constexpr int VEC = VecElems<IN, OUT>::v;
  constexpr int IB = VEC * ElemBytes<IN>::v, OB = VEC * ElemBytes<OUT>::v;
  static_assert(ElemBytes<IN>::v == 2, "the packed maximum below is for 16-bit inputs");
  const int64_t n_vec = n / VEC;
  uint32_t amax = 0u, pmax = 0u;
  float ssq = 0.f;
  // every block takes one contiguous run of vectors; the runs differ by at most one vector
  const int64_t v0 = n_vec / gridDim.x * blockIdx.x + min(int64_t(blockIdx.x), int64_t(n_vec % gridDim.x));
  const int64_t v1 = v0 + n_vec / gridDim.x + (blockIdx.x < n_vec % gridDim.x ? 1 : 0);
  for (int64_t base = v0; base < v1; base += kThreads * kUnroll) {
    uint32_t w[kUnroll][IB / 4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t i = base + u * kThreads + threadIdx.x;
      if (i < v1) {
        ld_raw_stream<IB>(static_cast<const char*>(x) + i * IB, w[u]);
      } else {
#pragma unroll
        for (int q = 0; q < IB / 4; ++q) w[u][q] = 0u;
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int64_t i = base + u * kThreads + threadIdx.x;
      float f[VEC];
      decode_vec<IN, VEC>(w[u], f);
      if (stat == SCALIFY_STAT_AMAX) {
        // magnitudes compare as unsigned integers on the raw 16-bit patterns, two elements per instruction
#pragma unroll
        for (int q = 0; q < IB / 4; ++q) pmax = __vmaxu2(pmax, w[u][q] & 0x7FFF7FFFu);
      } else {
#pragma unroll
        for (int e = 0; e < VEC; ++e) ssq = fmaf(f[e], f[e], ssq);
      }
      if (i < v1) {
#pragma unroll
        for (int e = 0; e < VEC; ++e) f[e] *= factor;
        uint32_t o[OB / 4];
        encode_vec<OUT, VEC>(f, o);
        st_raw_stream<OB>(static_cast<char*>(y) + i * OB, o);
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < static_cast<int>(n - n_vec * VEC)) {
    const int64_t i = n_vec * VEC + threadIdx.x;
    const float f = load_elem<IN>(x, i);
    amax = max(amax, abs_bits(f));
    ssq = fmaf(f, f, ssq);
    store_elem<OUT>(y, i, f * factor);
  }
  {
    // the larger 16-bit pattern, widened to the fp32 bit pattern of the same value
    const uint32_t h = max(pmax & 0xFFFFu, pmax >> 16);
    const uint32_t wide = IN == SCALIFY_BF16 ? h << 16
                                             : __float_as_uint(__half2float(__ushort_as_half(static_cast<unsigned short>(h))));
    amax = max(amax, wide);
  }
  __shared__ double s_part[kThreads / 32];
  __shared__ bool s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double mine;
  if (stat == SCALIFY_STAT_AMAX) mine = static_cast<double>(warp_max_u32(amax));
  else mine = warp_sum_f64(static_cast<double>(ssq));
  if (lane == 0) s_part[warp] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot;
    if (stat == SCALIFY_STAT_AMAX) {
      uint32_t m = 0u;
      for (int i = 0; i < kThreads / 32; ++i) m = max(m, static_cast<uint32_t>(s_part[i]));
      tot = static_cast<double>(m);
    } else {
      tot = 0.0;
      for (int i = 0; i < kThreads / 32; ++i) tot += s_part[i];
    }
    partials[blockIdx.x] = tot;
    __threadfence();
    const uint32_t t = atomicAdd(ticket, 1u);
    s_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // fixed-order combination of the per-block partials
  double acc = 0.0;
  uint32_t accm = 0u;
  for (int i = threadIdx.x; i < static_cast<int>(gridDim.x); i += kThreads) {
    const double p = __ldcg(&partials[i]);
    if (stat == SCALIFY_STAT_AMAX) accm = max(accm, static_cast<uint32_t>(p));
    else acc += p;
  }
  if (stat == SCALIFY_STAT_AMAX) acc = static_cast<double>(warp_max_u32(accm));
  else acc = warp_sum_f64(acc);
  __syncthreads();
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float result;
    if (stat == SCALIFY_STAT_AMAX) {
      uint32_t m = 0u;
      for (int i = 0; i < kThreads / 32; ++i) m = max(m, static_cast<uint32_t>(s_part[i]));
      result = __uint_as_float(m);
    } else {
      double tot = 0.0;
      for (int i = 0; i < kThreads / 32; ++i) tot += s_part[i];
      result = static_cast<float>(sqrt(tot / static_cast<double>(n)));
    }
    *stat_word = result;
    *ticket = 0u;
  }
}

// Returns SCALIFY_OK after the two launches, or 1 if this pair of formats has no predicted form.
int launch_rescale_predicted(const void* x, int in_dt, void* y, int out_dt, int64_t n, int stat, const float* x_scale,
                             float* y_scale, void* ws, size_t ws_bytes, cudaStream_t st) {
  if ((in_dt != SCALIFY_BF16 && in_dt != SCALIFY_F16) || (out_dt != SCALIFY_E4M3 && out_dt != SCALIFY_E5M2)) return 1;
  WsView v = ws_view(ws);
  int64_t grid = statistic_blocks_wanted(n, elem_size(in_dt));
  const int64_t room = static_cast<int64_t>((ws_bytes - kWsHeader) / sizeof(double));
  if (grid > room) grid = room;
  if (grid < 1) grid = 1;
  float* hint = reinterpret_cast<float*>(static_cast<char*>(ws) + 56);
  float* r_used = reinterpret_cast<float*>(static_cast<char*>(ws) + 52);
#define SCALIFY_RP(IN, OUT)                                                                                     \
  rescale_predict_kernel<IN, OUT><<<static_cast<int>(grid), kThreads, 0, st>>>(x, y, n, stat, hint, r_used,     \
                                                                              static_cast<double*>(v.area),     \
                                                                              v.ticket, v.stat)
  if (in_dt == SCALIFY_BF16) {
    if (out_dt == SCALIFY_E4M3) SCALIFY_RP(SCALIFY_BF16, SCALIFY_E4M3); else SCALIFY_RP(SCALIFY_BF16, SCALIFY_E5M2);
  } else {
    if (out_dt == SCALIFY_E4M3) SCALIFY_RP(SCALIFY_F16, SCALIFY_E4M3); else SCALIFY_RP(SCALIFY_F16, SCALIFY_E5M2);
  }
#undef SCALIFY_RP
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return launch_rebalance_check(x, in_dt, y, out_dt, n, x_scale, y_scale, v.stat, r_used, hint, v.status, st);
}

// ---------------------------------------------------------------------------------------------
// dynamic rescale in one cooperative launch (Section 3.3): statistic, grid barrier, rebalance
// ---------------------------------------------------------------------------------------------
// Every block owns one contiguous run of vectors.  Phase 1 reads the run front to back with the
// default cache policy and leaves one partial per block; after the grid barrier every block
// combines all partials in index order (so all blocks hold the same statistic, bit for bit) and
// phase 2 walks its run back to front, so that what phase 1 touched last - still in L2 - is read
// first.  For arrays up to about the L2 size the second read never reaches HBM.
template <int IN, int OUT>
__global__ void __launch_bounds__(kThreads) fused_rescale_kernel(const void* x, void* y, int64_t n, int stat,
                                                                 const float* x_scale, float* y_scale,
                                                                 double* partials, float* stat_word,
                                                                 uint32_t* status, int one_block) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = VecElems<IN, OUT>::v;
  constexpr int IB = VEC * ElemBytes<IN>::v, OB = VEC * ElemBytes<OUT>::v;
  constexpr int kTile = kThreads * kUnroll;
  cg::grid_group grid = cg::this_grid();
  const int64_t n_vec = n / VEC;
  // one contiguous run of vectors per block; the runs differ by at most one vector
  const int64_t v0 = n_vec / gridDim.x * blockIdx.x + min(int64_t(blockIdx.x), int64_t(n_vec % gridDim.x));
  const int64_t v1 = v0 + n_vec / gridDim.x + (blockIdx.x < n_vec % gridDim.x ? 1 : 0);
  const int64_t n_chunks = (v1 - v0 + kTile - 1) / kTile;
  const int tail = static_cast<int>(n - n_vec * VEC);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __shared__ double s_part[kThreads / 32];

  uint32_t amax = 0u;
  float ssq = 0.f;
  for (int64_t chunk = 0; chunk < n_chunks; ++chunk) {
    const int64_t base = v0 + chunk * kTile;
    uint32_t w[kUnroll][IB / 4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < v1) {
        ld_raw<IB>(static_cast<const char*>(x) + i * IB, w[u]);
      } else {
#pragma unroll
        for (int q = 0; q < IB / 4; ++q) w[u][q] = 0u;
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float f[VEC];
      decode_vec<IN, VEC>(w[u], f);
#pragma unroll
      for (int e = 0; e < VEC; ++e) {
        amax = max(amax, abs_bits(f[e]));
        ssq = fmaf(f[e], f[e], ssq);
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < tail) {
    float f = load_elem<IN>(x, n_vec * VEC + threadIdx.x);
    amax = max(amax, abs_bits(f));
    ssq = fmaf(f, f, ssq);
  }
  double mine = (stat == SCALIFY_STAT_AMAX) ? static_cast<double>(warp_max_u32(amax))
                                            : warp_sum_f64(static_cast<double>(ssq));
  if (lane == 0) s_part[warp] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    if (stat == SCALIFY_STAT_AMAX) {
      for (int i = 0; i < kThreads / 32; ++i) tot = fmax(tot, s_part[i]);
    } else {
      for (int i = 0; i < kThreads / 32; ++i) tot += s_part[i];
    }
    partials[blockIdx.x] = tot;
  }
  // an array of one tile is launched as a single ordinary block (a cooperative launch costs several
  // microseconds more, which is most of the call for a bias or LayerNorm gradient)
  if (one_block) __syncthreads();
  else grid.sync();

  // the same fixed-order combination in every block
  double acc = 0.0;
  for (int i = threadIdx.x; i < static_cast<int>(gridDim.x); i += kThreads) {
    double p = __ldcg(&partials[i]);
    acc = (stat == SCALIFY_STAT_AMAX) ? fmax(acc, p) : acc + p;
  }
  if (stat == SCALIFY_STAT_AMAX) acc = static_cast<double>(warp_max_u32(static_cast<uint32_t>(acc)));
  else acc = warp_sum_f64(acc);
  __syncthreads();
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  double tot = 0.0;
  if (stat == SCALIFY_STAT_AMAX) {
    for (int i = 0; i < kThreads / 32; ++i) tot = fmax(tot, s_part[i]);
  } else {
    for (int i = 0; i < kThreads / 32; ++i) tot += s_part[i];
  }
  const float statistic = (stat == SCALIFY_STAT_AMAX) ? __uint_as_float(static_cast<uint32_t>(tot))
                                                      : static_cast<float>(sqrt(tot / static_cast<double>(n)));
  const float xs = load_scale(x_scale);
  bool nonfinite;
  const float r = rescale_factor(statistic, &nonfinite);
  const float factor = 1.0f / r;  // exact: r is a power of two

  for (int64_t chunk = n_chunks - 1; chunk >= 0; --chunk) {
    const int64_t base = v0 + chunk * kTile;
    uint32_t w[kUnroll][IB / 4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < v1) ld_raw_stream<IB>(static_cast<const char*>(x) + i * IB, w[u]);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < v1) {
        float f[VEC];
        decode_vec<IN, VEC>(w[u], f);
#pragma unroll
        for (int e = 0; e < VEC; ++e) f[e] *= factor;
        uint32_t o[OB / 4];
        encode_vec<OUT, VEC>(f, o);
        st_raw_stream<OB>(static_cast<char*>(y) + i * OB, o);
      }
    }
  }
  if (blockIdx.x == 0) {
    if (threadIdx.x < tail) {
      int64_t i = n_vec * VEC + threadIdx.x;
      store_elem<OUT>(y, i, load_elem<IN>(x, i) * factor);
    }
    if (threadIdx.x == 0) {
      uint32_t flags = is_pow2_scale(xs) ? 0u : SCALIFY_DEV_BAD_SCALE;
      if (nonfinite) flags |= SCALIFY_DEV_NONFINITE_STAT;
      *stat_word = statistic;
      if (y_scale) *y_scale = xs * r;
      if (flags && status) atomicOr(status, flags);
    }
  }
}

template <int IN, int OUT>
static int fused_rescale_blocks_per_sm() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (cached[dev] == 0) {
    int b = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, fused_rescale_kernel<IN, OUT>, kThreads, 0) != cudaSuccess)
      b = 0;
    cached[dev] = b > 0 ? b : -1;
  }
  return cached[dev] > 0 ? cached[dev] : 0;
}

// Returns SCALIFY_OK after a cooperative launch, 1 if the device cannot run one (the caller then
// takes the two-launch path), or an error code.
int launch_fused_rescale(const void* x, int in_dt, void* y, int out_dt, int64_t n, int stat, const float* x_scale,
                         float* y_scale, void* ws, size_t ws_bytes, cudaStream_t st) {
  WsView v = ws_view(ws);
  const int64_t room = static_cast<int64_t>((ws_bytes - kWsHeader) / sizeof(double));
  int big = elem_size(in_dt) > elem_size(out_dt) ? elem_size(in_dt) : elem_size(out_dt);
  int64_t n_vec = n / (16 / big);
  double* partials = static_cast<double*>(v.area);
  float* stat_word = v.stat;
  uint32_t* status = v.status;
  int one_block = 0;
  void* args[] = {&x, &y, &n, &stat, &x_scale, &y_scale, &partials, &stat_word, &status, &one_block};
  int rc = 1;
  SCALIFY_DISPATCH_DTYPE(in_dt, IN, SCALIFY_DISPATCH_DTYPE(out_dt, OUT, {
    if (grid_for(n_vec, 1) == 1 && room >= 1) {
      fused_rescale_kernel<IN, OUT><<<1, kThreads, 0, st>>>(x, y, n, stat, x_scale, y_scale, partials, stat_word, status, 1);
      SCALIFY_CUDA_TRY(cudaGetLastError());
      return SCALIFY_OK;
    }
    int per_sm = fused_rescale_blocks_per_sm<IN, OUT>();
    if (per_sm > 0) {
      int grid = grid_for(n_vec, per_sm < 8 ? per_sm : 8);
      if (grid > room) grid = static_cast<int>(room);
      cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fused_rescale_kernel<IN, OUT>),
                                                  dim3(grid), dim3(kThreads), args, 0, st);
      if (e == cudaSuccess) rc = SCALIFY_OK;
      else (void)cudaGetLastError();
    }
  }));
  return rc;
}

// ---------------------------------------------------------------------------------------------
// multiplication by a scalar constant that is a power of two (Section 3.4: a broadcast scalar
// splits into mantissa and exponent; with mantissa 1 only the scale word changes)
// ---------------------------------------------------------------------------------------------
__global__ void scale_word_mul_kernel(float* scale, float c) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  *scale = *scale * c;
}

int launch_scale_word_mul(float* scale, float c, cudaStream_t st) {
  scale_word_mul_kernel<<<1, 1, 0, st>>>(scale, c);
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// scaled add / subtract (Section 3.2, add rule)
// ---------------------------------------------------------------------------------------------
struct FastDiv {
  uint32_t d, magic, shift;
};
static FastDiv make_fastdiv(uint32_t d) {
  FastDiv f;
  f.d = d;
  if (d == 1) { f.magic = 0; f.shift = 0; return f; }
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;  // ceil(log2 d)
  uint64_t m = ((1ull << 32) * ((1ull << l) - d)) / d + 1;
  f.magic = static_cast<uint32_t>(m);
  f.shift = l;
  return f;
}
__device__ __forceinline__ uint32_t fastdiv(uint32_t n, FastDiv f) {
  if (f.d == 1) return n;
  uint32_t t = __umulhi(n, f.magic);
  return (t + ((n - t) >> 1)) >> (f.shift - 1);
}

template <int AB, int OUT>
__global__ void __launch_bounds__(kThreads) add_kernel(const void* __restrict__ a, const void* __restrict__ b,
                                                       void* __restrict__ y, int64_t n, int64_t row_len,
                                                       FastDiv row_vecs, int broadcast, const float* a_scale,
                                                       const float* b_scale, float* y_scale, float sign) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = VecElems<AB, OUT>::v;
  constexpr int IB = VEC * ElemBytes<AB>::v, OB = VEC * ElemBytes<OUT>::v;
  const float as = load_scale(a_scale), bs = load_scale(b_scale);
  // sqrt(as^2+bs^2) rounded down to a power of two is max(as,bs) for power-of-two operands
  const float ys = fmaxf(as, bs);
  const float fa = as / ys, fb = sign * (bs / ys);
  const int64_t n_vec = n / VEC;
  const int64_t stride = int64_t(gridDim.x) * kThreads * kUnroll;
  for (int64_t base = int64_t(blockIdx.x) * kThreads * kUnroll; base < n_vec; base += stride) {
    uint32_t wa[kUnroll][IB / 4], wb[kUnroll][IB / 4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < n_vec) {
        ld_raw_stream<IB>(static_cast<const char*>(a) + i * IB, wa[u]);
        if (broadcast) {
          uint32_t iv = static_cast<uint32_t>(i);
          uint32_t r = fastdiv(iv, row_vecs);
          uint32_t c = iv - r * row_vecs.d;
          ld_raw<IB>(static_cast<const char*>(b) + int64_t(c) * IB, wb[u]);
        } else {
          ld_raw_stream<IB>(static_cast<const char*>(b) + i * IB, wb[u]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < n_vec) {
        float fa_[VEC], fb_[VEC];
        decode_vec<AB, VEC>(wa[u], fa_);
        decode_vec<AB, VEC>(wb[u], fb_);
#pragma unroll
        for (int e = 0; e < VEC; ++e) fa_[e] = fmaf(fb_[e], fb, fa_[e] * fa);
        uint32_t o[OB / 4];
        encode_vec<OUT, VEC>(fa_, o);
        st_raw<OB>(static_cast<char*>(y) + i * OB, o);
      }
    }
  }
  if (blockIdx.x == 0) {
    int tail = static_cast<int>(n - n_vec * VEC);
    if (threadIdx.x < tail) {
      int64_t i = n_vec * VEC + threadIdx.x;
      float av = load_elem<AB>(a, i);
      float bv = load_elem<AB>(b, broadcast ? (i % row_len) : i);
      store_elem<OUT>(y, i, fmaf(bv, fb, av * fa));
    }
    if (threadIdx.x == 0 && y_scale) *y_scale = ys;
  }
}

int launch_add(const void* a, const void* b, int ab_dt, void* y, int out_dt, int64_t n, int64_t row_len, int broadcast,
               const float* a_scale, const float* b_scale, float* y_scale, int subtract, cudaStream_t st) {
  int big = elem_size(ab_dt) > elem_size(out_dt) ? elem_size(ab_dt) : elem_size(out_dt);
  int vec = 16 / big;
  int64_t n_vec = n / vec;
  if (broadcast && (row_len % vec != 0 || n_vec >= (int64_t(1) << 31))) return SCALIFY_ERR_UNSUPPORTED;
  FastDiv fd = make_fastdiv(static_cast<uint32_t>(broadcast ? row_len / vec : 1));
  int grid = grid_all_tiles(n_vec);
  float sign = subtract ? -1.0f : 1.0f;
  SCALIFY_DISPATCH_WIDE(ab_dt, AB, SCALIFY_DISPATCH_DTYPE(out_dt, OUT,
      add_kernel<AB, OUT><<<grid, kThreads, 0, st>>>(a, b, y, n, row_len, fd, broadcast, a_scale, b_scale, y_scale,
                                                     sign)));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// scaled GELU (Appendix C.1): f(x) = x*g(x)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float gelu_u(float x) { return 0.7978845608028654f * fmaf(0.044715f * x * x, x, x); }

// gate g(x): tanh form written as a logistic, 0.5*(1+tanh(u)) = 1/(1+exp(-2u)), and the erf form as
// 0.5*erfc(-x/sqrt2); both keep full relative accuracy where the gate is tiny
template <int EXACT>
__device__ __forceinline__ float gelu_gate(float x) {
  if constexpr (EXACT) return 0.5f * erfcf(-x * 0.7071067811865476f);
  else {
    // logistic of 2u through t = exp(-2|u|) in (0,1]: never overflows, and underflows gradually
    const float u = gelu_u(x);
    const float t = __expf(-2.0f * fabsf(u));
    const float r = __fdividef(1.0f, 1.0f + t);  // the approximate reciprocal (2 ulp of fp32) is far below the output's ulp
    return u >= 0.f ? r : t * r;
  }
}

template <int EXACT>
__device__ __forceinline__ float gelu_deriv(float x) {  // f'(x) = g + x*g'
  if constexpr (EXACT) {
    float g = 0.5f * erfcf(-x * 0.7071067811865476f);
    return fmaf(x, 0.3989422804014327f * __expf(-0.5f * x * x), g);
  } else {
    float g = gelu_gate<0>(x);
    float du = 0.7978845608028654f * fmaf(3.0f * 0.044715f * x, x, 1.0f);
    return fmaf(x, 2.0f * g * (1.0f - g) * du, g);
  }
}

template <int IN, int OUT, int EXACT, int BWD>
__global__ void __launch_bounds__(kThreads) gelu_kernel(const void* __restrict__ x, const void* __restrict__ g,
                                                        void* __restrict__ y, int64_t n, const float* x_scale,
                                                        const float* g_scale, float* y_scale) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = VecElems<IN, OUT>::v;
  constexpr int IB = VEC * ElemBytes<IN>::v, OB = VEC * ElemBytes<OUT>::v;
  const float xs = load_scale(x_scale);
  const int64_t n_vec = n / VEC;
  const int64_t stride = int64_t(gridDim.x) * kThreads * kUnroll;
  for (int64_t base = int64_t(blockIdx.x) * kThreads * kUnroll; base < n_vec; base += stride) {
    uint32_t wx[kUnroll][IB / 4], wg[kUnroll][IB / 4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < n_vec) {
        ld_raw_stream<IB>(static_cast<const char*>(x) + i * IB, wx[u]);
        if (BWD) ld_raw_stream<IB>(static_cast<const char*>(g) + i * IB, wg[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      int64_t i = base + u * kThreads + threadIdx.x;
      if (i < n_vec) {
        float fx[VEC], fg[VEC];
        decode_vec<IN, VEC>(wx[u], fx);
        if (BWD) decode_vec<IN, VEC>(wg[u], fg);
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
          float v = fx[e] * xs;
          fx[e] = BWD ? fg[e] * gelu_deriv<EXACT>(v) : fx[e] * gelu_gate<EXACT>(v);
        }
        uint32_t o[OB / 4];
        encode_vec<OUT, VEC>(fx, o);
        st_raw<OB>(static_cast<char*>(y) + i * OB, o);
      }
    }
  }
  if (blockIdx.x == 0) {
    int tail = static_cast<int>(n - n_vec * VEC);
    if (threadIdx.x < tail) {
      int64_t i = n_vec * VEC + threadIdx.x;
      float xd = load_elem<IN>(x, i);
      float v = xd * xs;
      store_elem<OUT>(y, i, BWD ? load_elem<IN>(g, i) * gelu_deriv<EXACT>(v) : xd * gelu_gate<EXACT>(v));
    }
    if (threadIdx.x == 0 && y_scale) *y_scale = BWD ? load_scale(g_scale) : xs;
  }
}

int launch_gelu(const void* x, const void* g, int in_dt, void* y, int out_dt, int64_t n, const float* x_scale,
                const float* g_scale, float* y_scale, int exact, int bwd, cudaStream_t st) {
  int big = elem_size(in_dt) > elem_size(out_dt) ? elem_size(in_dt) : elem_size(out_dt);
  int64_t n_vec = n / (16 / big);
  int grid = grid_all_tiles(n_vec);
#define SCALIFY_GELU_LAUNCH(EX, BW) \
  gelu_kernel<IN, OUT, EX, BW><<<grid, kThreads, 0, st>>>(x, g, y, n, x_scale, g_scale, y_scale)
  SCALIFY_DISPATCH_WIDE(in_dt, IN, SCALIFY_DISPATCH_DTYPE(out_dt, OUT, {
    if (exact) { if (bwd) SCALIFY_GELU_LAUNCH(1, 1); else SCALIFY_GELU_LAUNCH(1, 0); }
    else { if (bwd) SCALIFY_GELU_LAUNCH(0, 1); else SCALIFY_GELU_LAUNCH(0, 0); }
  }));
#undef SCALIFY_GELU_LAUNCH
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

}  // namespace scalify
