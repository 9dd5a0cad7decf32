// Scaled LayerNorm forward and backward (Section 3.2.1, Appendix C.2, Algorithm 5).
//
// HBM-bound: every element of X (and G) is read once and every output written once.  A row is
// owned by a team of TW warps (TW = 1, 2, 4 or 8, chosen so that a thread holds at most two
// 16-byte vectors of the row); the row stays in registers, so mean, variance and the normalised
// values come from one read.  Blocks of 256 threads hold 8/TW teams.  Rows are fetched ahead of
// use: the forward kernel stages each thread's vectors of the next four rows in shared memory
// with cp.async, the backward kernel keeps the raw words of the next row in registers.  gamma and beta for a thread's fixed
// columns are converted once and kept in registers.
#include "scalify_common.cuh"
#include "scalify_launch.h"

namespace scalify {

constexpr int kLnThreads = 256;
constexpr int kLnVpt = 2;  // 16-byte vectors per thread and row
constexpr int kLnFwdStages = 4;  // rows in flight per thread, forward
constexpr int kLnBwdStages = 3;  // rows (of X and G) in flight per team, backward

// Per-thread asynchronous 16-byte copies into shared memory: a thread stages the vectors of its own
// columns for the next kLnStages rows and later reads back only what it copied itself, so no
// barrier is involved; cp.async.wait_group is a hardware wait, not a spin.  This keeps several rows
// per thread in flight without holding them in registers.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
#ifdef SCALIFY_DEBUG
  if (!dbg_ok(gmem_src, 16)) { *static_cast<uint4*>(smem_dst) = make_uint4(0u, 0u, 0u, 0u); return; }
#endif
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))),
               "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))),
               "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int TW>
__device__ __forceinline__ void team_barrier(int team) {
  if constexpr (TW == 8) __syncthreads();
  else if constexpr (TW > 1) asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "r"(TW * 32) : "memory");
}

// Sum of (a, b) over the team.  `buf` alternates between two shared arrays from call to call, so a
// single barrier per call is enough (a warp can only overwrite an array after every warp of the
// team has passed the barrier of the following call, i.e. after they have read it).
template <int TW>
__device__ __forceinline__ void team_sum2(float& a, float& b, float (*smem)[8][2], int team, int& buf) {
  a = warp_sum_f32(a);
  b = warp_sum_f32(b);
  if constexpr (TW > 1) {
    const int lane = threadIdx.x & 31, wit = (threadIdx.x >> 5) % TW;
    float(*s)[2] = smem[buf] + team * TW;
    if (lane == 0) { s[wit][0] = a; s[wit][1] = b; }
    team_barrier<TW>(team);
    a = 0.f; b = 0.f;
#pragma unroll
    for (int w = 0; w < TW; ++w) { a += s[w][0]; b += s[w][1]; }
    buf ^= 1;
  }
}

template <int TW>
__device__ __forceinline__ float team_sum1(float a, float (*smem)[8][2], int team, int& buf) {
  a = warp_sum_f32(a);
  if constexpr (TW > 1) {
    const int lane = threadIdx.x & 31, wit = (threadIdx.x >> 5) % TW;
    float(*s)[2] = smem[buf] + team * TW;
    if (lane == 0) s[wit][0] = a;
    team_barrier<TW>(team);
    a = 0.f;
#pragma unroll
    for (int w = 0; w < TW; ++w) a += s[w][0];
    buf ^= 1;
  }
  return a;
}

// 1/(sqrt(var)+eps) or 1/sqrt(var+eps) with the hardware approximations (each within 2 ulp of
// fp32, far below the resolution of the 16-bit and 8-bit outputs)
__device__ __forceinline__ float inv_sigma(float var, float eps, int eps_inside) {
  float r;
  if (eps_inside) {
    asm("rsqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(var + eps));
  } else {
    float sroot;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(sroot) : "f"(var));
    r = __fdividef(1.0f, sroot + eps);
  }
  return r;
}

// gamma / beta vector of VEC elements starting at column c, as fp32 (dtype chosen at run time)
template <int VEC>
__device__ __forceinline__ void load_param_vec(const void* p, int dt, int c, float* f) {
  if (dt == SCALIFY_F32) {
    uint32_t w[VEC];
    ld_raw<VEC * 4>(static_cast<const char*>(p) + int64_t(c) * 4, w);
    decode_vec<SCALIFY_F32, VEC>(w, f);
  } else {
    uint32_t w[VEC / 2];
    ld_raw<VEC * 2>(static_cast<const char*>(p) + int64_t(c) * 2, w);
    if (dt == SCALIFY_BF16) decode_vec<SCALIFY_BF16, VEC>(w, f);
    else decode_vec<SCALIFY_F16, VEC>(w, f);
  }
}

// ---------------------------------------------------------------------------------------------
// forward
// ---------------------------------------------------------------------------------------------
template <int XDT, int YDT, int TW, int VPT>
__global__ void __launch_bounds__(kLnThreads) layernorm_fwd_kernel(
    const void* __restrict__ X, int64_t x_ld, void* __restrict__ Y, int64_t y_ld, int R, int d,
    const void* __restrict__ gamma, const void* __restrict__ beta, int gb_dt, const float* gamma_scale,
    const float* beta_scale, float* y_scale, float eps, int eps_inside, float* __restrict__ mean_out,
    float* __restrict__ rinv_out, int rows_per_team) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<XDT>::v;
  constexpr int OB = VEC * ElemBytes<YDT>::v;
  constexpr int TEAM = 32 * TW;
  constexpr int TPB = kLnThreads / TEAM;  // teams per block
  __shared__ float smem[2][8][2];
  const int n_vec = d / VEC;
  const int t = threadIdx.x % TEAM;
  const int team = threadIdx.x / TEAM;
  float ys = 1.0f, fg = 1.0f, fb = 0.0f;
  if (gamma) {
    const float gs = load_scale(gamma_scale), bs = beta ? load_scale(beta_scale) : 0.0f;
    ys = fmaxf(gs, bs);  // add rule on power-of-two scales
    fg = gs / ys;
    fb = bs / ys;
  }
  // this thread's columns: vectors t, t + TEAM, ...
  bool has[VPT];
#pragma unroll
  for (int v = 0; v < VPT; ++v) has[v] = (t + v * TEAM) < n_vec;
  const float inv_d = 1.0f / static_cast<float>(d);
  // a block owns TPB * rows_per_team consecutive rows; each iteration its teams take TPB adjacent rows
  constexpr int rows_per_iter = TPB;
  const int iters = rows_per_team;
  int buf = 0;
  extern __shared__ uint4 ln_stage[];  // [stage][v][thread]
  // (only rows of this block's own run are fetched: `mine` is false for the stages beyond it)
  auto issue = [&](int row, int slot, bool mine) {
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      if (mine && has[v] && row < R)
        cp_async16(&ln_stage[(slot * VPT + v) * kLnThreads + threadIdx.x],
                   static_cast<const char*>(X) + (int64_t(row) * x_ld) * ElemBytes<XDT>::v + int64_t(t + v * TEAM) * 16);
    }
    cp_async_commit();  // one group per row, even when empty, so that the group count stays uniform
  };
  const int first_row = blockIdx.x * (TPB * rows_per_team) + team;
  // gamma and beta go through shared memory once per block (all teams of a block use the same columns): the
  // whole block copies them as the oldest cp.async group, then the first rows follow
  uint4* gb_stage = ln_stage + kLnFwdStages * VPT * kLnThreads;  // [gamma | beta], raw bytes
  const int gb_bytes = d * (gb_dt == SCALIFY_F32 ? 4 : 2);
  if (gamma) {
    for (int idx = threadIdx.x; idx < gb_bytes / 16; idx += kLnThreads) {
      cp_async16(&gb_stage[idx], static_cast<const char*>(gamma) + idx * 16);
      if (beta) cp_async16(&gb_stage[gb_bytes / 16 + idx], static_cast<const char*>(beta) + idx * 16);
    }
  }
  cp_async_commit();
#pragma unroll
  for (int st = 0; st < kLnFwdStages; ++st) issue(first_row + st * rows_per_iter, st, st < iters);
  cp_async_wait<kLnFwdStages>();  // the parameter group has landed (this thread's part) ...
  __syncthreads();                // ... and everybody else's
  const void* gamma_s = gb_stage;
  const void* beta_s = reinterpret_cast<const char*>(gb_stage) + gb_bytes;
  float gam[VPT][VEC], bet[VPT][VEC];
#pragma unroll
  for (int v = 0; v < VPT; ++v) {
    const int vi = t + v * TEAM;
#pragma unroll
    for (int e = 0; e < VEC; ++e) { gam[v][e] = 1.0f; bet[v][e] = 0.0f; }
    if (has[v] && gamma) {
      load_param_vec<VEC>(gamma_s, gb_dt, vi * VEC, gam[v]);
      if (beta) {
        load_param_vec<VEC>(beta_s, gb_dt, vi * VEC, bet[v]);
#pragma unroll
        for (int e = 0; e < VEC; ++e) bet[v][e] *= fb;  // exact: fb is a power of two
      }
    }
  }
  int slot = 0;
  for (int it = 0; it < iters; ++it) {
    const int row = it * rows_per_iter + first_row;
    const bool live = row < R;
    float x[VPT][VEC];
    cp_async_wait<kLnFwdStages - 1>();  // the oldest row in flight has landed
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      if (has[v] && live) {
        const uint4 q4 = ln_stage[(slot * VPT + v) * kLnThreads + threadIdx.x];
        w[0] = q4.x; w[1] = q4.y; w[2] = q4.z; w[3] = q4.w;
      }
      decode_vec<XDT, VEC>(w, x[v]);
    }
    issue(row + kLnFwdStages * rows_per_iter, slot, it + kLnFwdStages < iters);  // refill the slot just read
    if (++slot == kLnFwdStages) slot = 0;
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v)
#pragma unroll
      for (int e = 0; e < VEC; ++e) s += x[v][e];  // absent vectors hold zeros
    const float mu = team_sum1<TW>(s, smem, team, buf) * inv_d;
    float q = 0.f;
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
      if (has[v]) {
#pragma unroll
        for (int e = 0; e < VEC; ++e) { x[v][e] -= mu; q = fmaf(x[v][e], x[v][e], q); }
      }
    }
    const float var = team_sum1<TW>(q, smem, team, buf) * inv_d;
    const float rinv = inv_sigma(var, eps, eps_inside);
    if (live) {
      if (t == 0) {
        if (mean_out) mean_out[row] = mu;
        if (rinv_out) rinv_out[row] = rinv;
      }
      const float rg = rinv * fg;  // exact: fg is a power of two
      char* yrow = static_cast<char*>(Y) + int64_t(row) * y_ld * ElemBytes<YDT>::v;
#pragma unroll
      for (int v = 0; v < VPT; ++v) {
        if (has[v]) {
          float o[VEC];
#pragma unroll
          for (int e = 0; e < VEC; ++e) o[e] = fmaf(x[v][e] * rg, gam[v][e], bet[v][e]);
          uint32_t ow[OB / 4];
          encode_vec<YDT, VEC>(o, ow);
          st_raw<OB>(yrow + int64_t(t + v * TEAM) * OB, ow);
        }
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && y_scale) *y_scale = ys;
}

static int ln_grid(int R, int teams_per_block, int blocks_per_sm) {
  int64_t need = (int64_t(R) + teams_per_block - 1) / teams_per_block;
  int64_t cap = int64_t(sm_count()) * blocks_per_sm;
  if (need < 1) need = 1;
  return static_cast<int>(need < cap ? need : cap);
}

// team width in warps so that a thread holds at most kLnVpt vectors; 0 if the row is too long
static int ln_team_warps(int d, int x_dt) {
  const int n_vec = d * elem_size(x_dt) / 16;
  for (int tw = 1; tw <= 8; tw *= 2)
    if (n_vec <= 32 * tw * kLnVpt) return tw;
  return 0;
}

// Launch shape of the forward kernel: team width, vectors per thread, rows each team walks, grid.
struct LnFwdPlan { int tw, vpt, rpt, grid; bool ok; };
static LnFwdPlan ln_fwd_plan(int R, int d, int x_dt) {
  LnFwdPlan p{};
  p.tw = ln_team_warps(d, x_dt);
  p.ok = p.tw != 0;
  if (!p.ok) return p;
  // rows of more than 64 vectors: four vectors per thread and a quarter of the warps per row (65..128 vectors:
  // one warp, no cross-warp step; up to 512 vectors: four warps, so a block works on two rows at a time)
  const int n_vec = d * elem_size(x_dt) / 16;
  const bool wide = n_vec > 64;
  if (wide) p.tw = n_vec <= 128 ? 1 : (n_vec <= 256 ? 2 : 4);
  p.vpt = wide ? 4 : 2;
  // Blocks are not persistent: each owns a short run of consecutive rows (6 per team) and the
  // hardware scheduler hands out the runs in address order.  Measured on B200 (131072 x 1024 BF16):
  // 90 us, against 104 us for a grid of 3 blocks per SM striding over the rows, and 101 us with 16
  // rows per team (fewer, longer blocks leave a larger partial last wave).
  const int tpb = 8 / p.tw;
  p.rpt = 6;
  while (p.rpt > 1 && (int64_t(R) + tpb * p.rpt - 1) / (tpb * p.rpt) < 4 * int64_t(sm_count())) --p.rpt;
  p.grid = static_cast<int>((int64_t(R) + tpb * p.rpt - 1) / (tpb * p.rpt));
  return p;
}

int launch_layernorm_fwd(const void* X, int x_dt, int64_t x_ld, void* Y, int y_dt, int64_t y_ld, int R, int d,
                         const void* gamma, const void* beta, int gb_dt, const float* gamma_scale,
                         const float* beta_scale, float* y_scale, float eps, int eps_inside, float* mean,
                         float* rinv, cudaStream_t st) {
  const LnFwdPlan plan = ln_fwd_plan(R, d, x_dt);
  if (!plan.ok) return SCALIFY_ERR_UNSUPPORTED;
  const int tw = plan.tw, rpt = plan.rpt, grid = plan.grid;
  const bool wide = plan.vpt == 4;
#define SCALIFY_LN_FWD(W, V)                                                                                   \
  do {                                                                                                         \
    /* row staging + gamma and beta (up to 4 bytes per element each) */                                       \
    constexpr int kSmemMax = kLnFwdStages * V * kLnThreads * 16 + 2 * (32 * W * V * 16 / 2) * 4;               \
    const int smem_bytes = kLnFwdStages * V * kLnThreads * 16 + 2 * d * 4;                                     \
    if (kSmemMax > 40 * 1024) { /* the kernel also has a little static shared memory */                       \
      static DeviceOnce once; /* per instantiation and device */                                               \
      int rc_once = device_once(once, nullptr, [&](int*) {                                                     \
        SCALIFY_CUDA_TRY(cudaFuncSetAttribute(layernorm_fwd_kernel<XDT, YDT, W, V>,                            \
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax));         \
        return int(SCALIFY_OK);                                                                                \
      });                                                                                                      \
      if (rc_once) return rc_once;                                                                             \
    }                                                                                                          \
    layernorm_fwd_kernel<XDT, YDT, W, V><<<grid, kLnThreads, smem_bytes, st>>>(                                     \
        X, x_ld, Y, y_ld, R, d, gamma, beta, gb_dt, gamma_scale, beta_scale, y_scale, eps, eps_inside, mean,   \
        rinv, rpt);                                                                                                \
  } while (0)
  SCALIFY_DISPATCH_WIDE(x_dt, XDT, SCALIFY_DISPATCH_DTYPE(y_dt, YDT, {
    if (wide) {
      switch (tw) {
        case 1: SCALIFY_LN_FWD(1, 4); break;
        case 2: SCALIFY_LN_FWD(2, 4); break;
        default: SCALIFY_LN_FWD(4, 4); break;
      }
    } else {
      switch (tw) {
        case 1: SCALIFY_LN_FWD(1, 2); break;
        case 2: SCALIFY_LN_FWD(2, 2); break;
        case 4: SCALIFY_LN_FWD(4, 2); break;
        default: SCALIFY_LN_FWD(8, 2); break;
      }
    }
  }));
#undef SCALIFY_LN_FWD
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// ---------------------------------------------------------------------------------------------
// backward (+ statistic of the stored input gradient, + per-block dgamma/dbeta partials)
// ---------------------------------------------------------------------------------------------
// ws layout (after the header): float dgamma_part[grid][d]; float dbeta_part[grid][d];
// double stat_part[grid].
// Packed two-wide fp32 arithmetic (one instruction for two lanes): the backward kernel is bound by instruction
// issue, not by bytes, so its per-element arithmetic runs on float2 pairs.
__device__ __forceinline__ float2 f2(float a, float b) { return make_float2(a, b); }
__device__ __forceinline__ float2 f2(float a) { return make_float2(a, a); }

// N elements of dtype DT held in raw words -> N/2 float2 pairs (element 2i in .x, 2i+1 in .y)
template <int DT, int N>
__device__ __forceinline__ void decode_pairs(const uint32_t* w, float2* f) {
  if constexpr (DT == SCALIFY_F32) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) f[i] = f2(__uint_as_float(w[2 * i]), __uint_as_float(w[2 * i + 1]));
  } else if constexpr (DT == SCALIFY_BF16) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) f[i] = f2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
  } else if constexpr (DT == SCALIFY_F16) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) f[i] = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
  } else {
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      f[2 * i] = fp8x2_to_float2(w[i], DT == SCALIFY_E5M2);
      f[2 * i + 1] = fp8x2_to_float2(w[i] >> 16, DT == SCALIFY_E5M2);
    }
  }
}

// N/2 float2 pairs -> N elements of dtype DT (round to nearest even; FP8 saturates)
template <int DT, int N>
__device__ __forceinline__ void encode_pairs(const float2* f, uint32_t* w) {
  if constexpr (DT == SCALIFY_F32) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) { w[2 * i] = __float_as_uint(f[i].x); w[2 * i + 1] = __float_as_uint(f[i].y); }
  } else if constexpr (DT == SCALIFY_BF16) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      __nv_bfloat162 t = __float22bfloat162_rn(f[i]);
      w[i] = *reinterpret_cast<uint32_t*>(&t);
    }
  } else if constexpr (DT == SCALIFY_F16) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      __half2 t = __float22half2_rn(f[i]);
      w[i] = *reinterpret_cast<uint32_t*>(&t);
    }
  } else {
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      const uint32_t lo = __nv_cvt_float2_to_fp8x2(f[2 * i], __NV_SATFINITE, DT == SCALIFY_E5M2 ? __NV_E5M2 : __NV_E4M3);
      const uint32_t hi = __nv_cvt_float2_to_fp8x2(f[2 * i + 1], __NV_SATFINITE, DT == SCALIFY_E5M2 ? __NV_E5M2 : __NV_E4M3);
      w[i] = (lo & 0xFFFFu) | (hi << 16);
    }
  }
}

// Sum of a pair (a.x, a.y are two independent quantities) over the team; same buffer discipline as team_sum2.
template <int TW>
__device__ __forceinline__ float2 team_sum_pair(float2 a, float (*smem)[8][2], int team, int& buf) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
    a = __fadd2_rn(a, f2(__shfl_xor_sync(0xFFFFFFFFu, a.x, o), __shfl_xor_sync(0xFFFFFFFFu, a.y, o)));
  if constexpr (TW > 1) {
    const int lane = threadIdx.x & 31, wit = (threadIdx.x >> 5) % TW;
    float2* s = reinterpret_cast<float2*>(smem[buf] + team * TW);
    if (lane == 0) s[wit] = a;
    team_barrier<TW>(team);
    a = s[0];
#pragma unroll
    for (int w = 1; w < TW; ++w) a = __fadd2_rn(a, s[w]);
    buf ^= 1;
  }
  return a;
}

// EXACT: the dynamic rescale of the plain call (values rounded through the intermediate format XDT, statistic of
// those rounded values, rebalanced output in DXDT) in ONE pass over the data: the output is written with a
// predicted power of two (that of the statistic word `pred.hint`, the statistic this workspace saw last), and a
// second launch of the same kernel (`pred.redo`) returns at once if this call's statistic has the same power of
// two and otherwise writes the output again with the right one.  The intermediate is never stored.
struct LnBwdPredict {
  const float* hint;       // statistic of the previous call (any content: a wrong prediction only costs the second pass)
  float* r_used;           // power of two the first launch divided by
  const float* stat_word;  // this call's statistic (read by the second launch)
  int redo;                // 0: first launch, 1: second launch
};

template <int XDT, int DXDT, int TW, bool EXACT>
__global__ void __launch_bounds__(kLnThreads, 2) layernorm_bwd_kernel(
    const void* __restrict__ G, int64_t g_ld, const void* __restrict__ X, int64_t x_ld, void* __restrict__ dX,
    int64_t dx_ld, int R, int d, const void* __restrict__ gamma, int gb_dt, const float* __restrict__ mean,
    const float* __restrict__ rinv_in, float eps, int eps_inside, int stat_arg, const float* __restrict__ stat_in,
    float* __restrict__ dgamma_part_arg, float* __restrict__ dbeta_part, double* __restrict__ stat_part,
    const LnBwdPredict pred) {
  int stat = stat_arg;
  float* dgamma_part = dgamma_part_arg;
  float exact_r = 1.0f;
  if constexpr (EXACT) {
    bool nf;
    if (pred.redo) {
      // everything this launch reads was written by the launches before it
      asm volatile("griddepcontrol.wait;" ::: "memory");
      exact_r = rescale_factor(*reinterpret_cast<const volatile float*>(pred.stat_word), &nf);
      if (exact_r == *reinterpret_cast<const volatile float*>(pred.r_used)) return;  // the prediction held
      stat = SCALIFY_STAT_NONE;   // statistic and column sums are already final
      dgamma_part = nullptr;
    } else {
      exact_r = rescale_factor(*reinterpret_cast<const volatile float*>(pred.hint), &nf);
      if (blockIdx.x == 0 && threadIdx.x == 0) *pred.r_used = exact_r;
    }
  }
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int VEC = 16 / ElemBytes<XDT>::v;
  constexpr int HP = VEC / 2;  // float2 pairs per vector
  constexpr int OB = VEC * ElemBytes<DXDT>::v;
  constexpr int TEAM = 32 * TW;
  constexpr int TPB = kLnThreads / TEAM;
  __shared__ __align__(16) float smem[2][8][2];
  // delayed rescale (Section 3.3): the gradient is stored already divided by r = p2_floor(earlier statistic)
  // and this step's statistic is that of the un-rebalanced fp32 values.  r is a power of two, so dividing the
  // three coefficients of the output expression by it gives the same bits as dividing the result, and the
  // statistic of the un-rebalanced values is the statistic of the stored-scale values times r (exactly).
  float inv_r = 1.0f, r_prev = 1.0f;
  if (!EXACT && stat_in) { bool nf; r_prev = rescale_factor(__ldg(stat_in), &nf); inv_r = 1.0f / r_prev; }
  const float2 exact_inv_r = f2(1.0f / exact_r);
  const int n_vec = d / VEC;
  const int t = threadIdx.x % TEAM;
  const int team = threadIdx.x / TEAM;
  const float inv_d = 1.0f / static_cast<float>(d);
  bool has[kLnVpt];
  float2 gam[kLnVpt][HP], acc_dg[kLnVpt][HP], acc_db[kLnVpt][HP];
#pragma unroll
  for (int v = 0; v < kLnVpt; ++v) {
    has[v] = (t + v * TEAM) < n_vec;
    float gf[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) gf[e] = 1.0f;
    if (has[v] && gamma) load_param_vec<VEC>(gamma, gb_dt, (t + v * TEAM) * VEC, gf);
#pragma unroll
    for (int h = 0; h < HP; ++h) { gam[v][h] = f2(gf[2 * h], gf[2 * h + 1]); acc_dg[v][h] = f2(0.f); acc_db[v][h] = f2(0.f); }
  }
  uint32_t amax = 0u;
  float2 ssq2 = f2(0.f);
  // the grid strides over the rows: at any moment its teams work on one dense stretch of X, G and dX (teams that
  // each walk their own contiguous run of rows measured 5 % slower)
  const int rows_per_iter = gridDim.x * TPB;
  const int iters = (R + rows_per_iter - 1) / rows_per_iter;
  int buf = 0;
  // Rows in flight: the next kLnBwdStages rows of X and G travel as cp.async copies into shared memory, every
  // thread copying and later reading only its own vectors (no barrier involved), so that enough bytes are in
  // flight per SM to cover the DRAM latency whatever the arithmetic of the current row is waiting for; the
  // row's mean and 1/sigma are fetched one row ahead into registers.  (Measured, 131072 x 1024 BF16: 139 us
  // against 150 us with one row prefetched in registers.  An earlier form that also staged mean and 1/sigma with
  // two 4-byte copies per thread was slower than either: 158 us.)
  extern __shared__ uint4 ln_bstage[];  // [stage][x | g][v][thread]
  float nmu = 0.f, nrinv = 0.f;
  const char* xcol = static_cast<const char*>(X) + int64_t(t) * 16;
  const char* gcol = static_cast<const char*>(G) + int64_t(t) * 16;
  const int64_t x_row_bytes = x_ld * ElemBytes<XDT>::v, g_row_bytes = g_ld * ElemBytes<XDT>::v;
  const int first_row = blockIdx.x * TPB + team;
  const int row_end = R;
  auto issue = [&](int row, int slot) {
    if (row < row_end) {
#pragma unroll
      for (int v = 0; v < kLnVpt; ++v) {
        if (has[v]) {
          cp_async16(&ln_bstage[((slot * 2 + 0) * kLnVpt + v) * kLnThreads + threadIdx.x],
                     xcol + row * x_row_bytes + v * (TEAM * 16));
          cp_async16(&ln_bstage[((slot * 2 + 1) * kLnVpt + v) * kLnThreads + threadIdx.x],
                     gcol + row * g_row_bytes + v * (TEAM * 16));
        }
      }
    }
    cp_async_commit();  // one group per row, even when empty, so that the group count stays uniform
  };
#pragma unroll
  for (int st = 0; st < kLnBwdStages; ++st) issue(first_row + st * rows_per_iter, st);
  if (first_row < row_end) { nmu = __ldg(&mean[first_row]); nrinv = __ldg(&rinv_in[first_row]); }
  int slot = 0;
  for (int it = 0; it < iters; ++it) {
    const int row = it * rows_per_iter + first_row;
    const bool live = row < row_end;
    float2 x[kLnVpt][HP], g[kLnVpt][HP];
    float mu = 0.f, rinv = 0.f;
    cp_async_wait<kLnBwdStages - 1>();  // the oldest row in flight has landed
    mu = live ? nmu : 0.f;
    rinv = live ? nrinv : 0.f;
    if (row + rows_per_iter < row_end) { nmu = __ldg(&mean[row + rows_per_iter]); nrinv = __ldg(&rinv_in[row + rows_per_iter]); }
#pragma unroll
    for (int v = 0; v < kLnVpt; ++v) {
      uint32_t wx[4] = {0u, 0u, 0u, 0u}, wg[4] = {0u, 0u, 0u, 0u};
      if (has[v] && live) {
        const uint4 qx = ln_bstage[((slot * 2 + 0) * kLnVpt + v) * kLnThreads + threadIdx.x];
        const uint4 qg = ln_bstage[((slot * 2 + 1) * kLnVpt + v) * kLnThreads + threadIdx.x];
        wx[0] = qx.x; wx[1] = qx.y; wx[2] = qx.z; wx[3] = qx.w;
        wg[0] = qg.x; wg[1] = qg.y; wg[2] = qg.z; wg[3] = qg.w;
      }
      decode_pairs<XDT, VEC>(wx, x[v]);
      decode_pairs<XDT, VEC>(wg, g[v]);
    }
    issue(row + kLnBwdStages * rows_per_iter, slot);  // refill the slot just read
    if (++slot == kLnBwdStages) slot = 0;
    // A row past the end (or an absent vector) holds zeros with rinv = 0: it adds exact zeros everywhere below,
    // so the arithmetic needs no predicates; only the stores are guarded.
    const float2 nmu2 = f2(-mu), rinv2 = f2(rinv);
    float2 m12 = f2(0.f), m22 = f2(0.f);
#pragma unroll
    for (int v = 0; v < kLnVpt; ++v) {
#pragma unroll
      for (int h = 0; h < HP; ++h) {
        const float2 n = __fmul2_rn(__fadd2_rn(x[v][h], nmu2), rinv2);
        acc_dg[v][h] = __ffma2_rn(g[v][h], n, acc_dg[v][h]);
        acc_db[v][h] = __fadd2_rn(acc_db[v][h], g[v][h]);
        const float2 gh = __fmul2_rn(g[v][h], gam[v][h]);
        x[v][h] = n;   // keep n
        g[v][h] = gh;  // keep ghat
        m12 = __fadd2_rn(m12, gh);
        m22 = __ffma2_rn(gh, n, m22);
      }
    }
    const float2 m = team_sum_pair<TW>(f2(m12.x + m12.y, m22.x + m22.y), smem, team, buf);
    const float m1 = m.x * inv_d, m2 = m.y * inv_d;
    // eps outside the root: dx = (ghat-m1)*rinv - n*m2/s with s = 1/rinv - eps (0 if s == 0)
    // eps inside the root:  dx = rinv*(ghat - m1 - n*m2)
    float c2;
    if (eps_inside) {
      c2 = rinv * m2;
    } else {
      const float s = __fdividef(1.0f, rinv) - eps;
      c2 = (s > 0.f) ? __fdividef(m2, s) : 0.f;
    }
    // coefficients at the stored scale (inv_r is 1 unless the rescale is delayed)
    const float2 k_g = f2(rinv * inv_r), k_n = f2(-c2 * inv_r), k_0 = f2(-m1 * rinv * inv_r);
    if (live) {
      char* orow = static_cast<char*>(dX) + int64_t(row) * dx_ld * ElemBytes<DXDT>::v + int64_t(t) * OB;
#pragma unroll
      for (int v = 0; v < kLnVpt; ++v) {
        if (has[v]) {
          float2 o[HP];
#pragma unroll
          for (int h = 0; h < HP; ++h) o[h] = __ffma2_rn(g[v][h], k_g, __ffma2_rn(x[v][h], k_n, k_0));
          uint32_t ow[OB / 4 > 0 ? OB / 4 : 1];
          if constexpr (EXACT) {
            // the value the plain call would have stored in the intermediate (one rounding to XDT), its
            // statistic, and the rebalanced output: an exact division by a power of two, then one rounding
            if constexpr (XDT != SCALIFY_F32) {
              uint32_t iw[4];
              encode_pairs<XDT, VEC>(o, iw);
              decode_pairs<XDT, VEC>(iw, o);
            }
            if (stat == SCALIFY_STAT_AMAX) {
#pragma unroll
              for (int h = 0; h < HP; ++h) amax = __vimax3_u32(amax, abs_bits(o[h].x), abs_bits(o[h].y));
            } else if (stat == SCALIFY_STAT_L2) {
#pragma unroll
              for (int h = 0; h < HP; ++h) ssq2 = __ffma2_rn(o[h], o[h], ssq2);
            }
            float2 q[HP];
#pragma unroll
            for (int h = 0; h < HP; ++h) q[h] = __fmul2_rn(o[h], exact_inv_r);
            encode_pairs<DXDT, VEC>(q, ow);
            st_raw<OB>(orow + v * (TEAM * OB), ow);
            continue;
          }
          encode_pairs<DXDT, VEC>(o, ow);
          st_raw<OB>(orow + v * (TEAM * OB), ow);
          if (stat == SCALIFY_STAT_AMAX) {
            // rounding is monotonic: the max of the stored values is the stored value of the max
#pragma unroll
            for (int h = 0; h < HP; ++h) amax = __vimax3_u32(amax, abs_bits(o[h].x), abs_bits(o[h].y));
          } else if (stat == SCALIFY_STAT_L2) {
            if (stat_in) {  // the unrounded values
#pragma unroll
              for (int h = 0; h < HP; ++h) ssq2 = __ffma2_rn(o[h], o[h], ssq2);
            } else {        // the values as stored
              float2 sv[HP];
              decode_pairs<DXDT, VEC>(ow, sv);
#pragma unroll
              for (int h = 0; h < HP; ++h) ssq2 = __ffma2_rn(sv[h], sv[h], ssq2);
            }
          }
        }
      }
    }
  }
  const float ssq = ssq2.x + ssq2.y;
  // per-block column partials of dgamma / dbeta: teams of a block own the same columns
  if (dgamma_part) {
    if constexpr (TPB > 1) {
      __shared__ float s_col[TPB][TEAM][VEC + 1];
#pragma unroll
      for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
        for (int v = 0; v < kLnVpt; ++v) {
          __syncthreads();
#pragma unroll
          for (int h = 0; h < HP; ++h) {
            const float2 a = pass ? acc_db[v][h] : acc_dg[v][h];
            s_col[team][t][2 * h] = a.x;
            s_col[team][t][2 * h + 1] = a.y;
          }
          __syncthreads();
          if (team == 0 && has[v]) {
            float* dst = (pass ? dbeta_part : dgamma_part) + int64_t(blockIdx.x) * d + (t + v * TEAM) * VEC;
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
              float sum = s_col[0][t][e];
#pragma unroll
              for (int tm = 1; tm < TPB; ++tm) sum += s_col[tm][t][e];
              dst[e] = sum;
            }
          }
        }
      }
    } else {
#pragma unroll
      for (int v = 0; v < kLnVpt; ++v) {
        if (has[v]) {
          float2* dg = reinterpret_cast<float2*>(dgamma_part + int64_t(blockIdx.x) * d + (t + v * TEAM) * VEC);
          float2* db = reinterpret_cast<float2*>(dbeta_part + int64_t(blockIdx.x) * d + (t + v * TEAM) * VEC);
#pragma unroll
          for (int h = 0; h < HP; ++h) { dg[h] = acc_dg[v][h]; db[h] = acc_db[v][h]; }
        }
      }
    }
  }
  if (stat != SCALIFY_STAT_NONE) {
    __shared__ double s_stat[kLnThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // AMAX: of the stored values (plain call) or of the un-rebalanced, unrounded ones (delayed: times r, exact)
    if (stat == SCALIFY_STAT_AMAX && !EXACT)  // (EXACT: the maximum is already that of the rounded intermediate values)
      amax = stat_in ? abs_bits(__uint_as_float(amax) * r_prev) : abs_bits(round_through<DXDT>(__uint_as_float(amax)));
    double mine = (stat == SCALIFY_STAT_AMAX)
                      ? static_cast<double>(warp_max_u32(amax))
                      : warp_sum_f64(static_cast<double>(ssq)) * (static_cast<double>(r_prev) * static_cast<double>(r_prev));
    if (lane == 0) s_stat[warp] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = s_stat[0];
      for (int i = 1; i < kLnThreads / 32; ++i)
        tot = (stat == SCALIFY_STAT_AMAX) ? fmax(tot, s_stat[i]) : tot + s_stat[i];
      stat_part[blockIdx.x] = tot;
    }
  }
}

// Combines the per-block partials in a fixed order: dgamma/dbeta columns (scaled by 1/kf(R)), the
// statistic word, and the propagated scale words.
template <int DGDT>
__global__ void __launch_bounds__(1024) layernorm_bwd_finalize_kernel(
    int nblocks, int R, int d, const float* __restrict__ dgamma_part, const float* __restrict__ dbeta_part,
    const double* __restrict__ stat_part, int stat, float* stat_word, void* __restrict__ dgamma,
    void* __restrict__ dbeta, const float* g_scale, const float* x_scale, const float* gamma_scale,
    float* dx_scale, float* dgamma_scale, float* dbeta_scale, const float* stat_in, uint32_t* status,
    float* exact_hint) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  // exact_hint != nullptr: the one-pass dynamic rescale.  The output scale carries the power of two of THIS
  // call's statistic (the second launch of the main kernel makes the data agree with it), and the statistic is
  // left in *exact_hint as the next call's prediction.
  // block = 8 columns (one 32-byte sector of a partial row) x 128 slices of the block list: 4 x as many
  // blocks as a 32-column layout, so the partials (a few MB in L2) are read by more SMs at once
  __shared__ float s_a[128][9], s_b[128][9];
  const float inv_kf = 1.0f / kfactor(R);
  const int pc = threadIdx.x & 7, slice = threadIdx.x >> 3;
  const int col = blockIdx.x * 8 + pc;
  const int cx = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (dgamma_part) {
    float a = 0.f, b = 0.f;
    if (col < d) {
      for (int i = slice; i < nblocks; i += 128) {
        a += dgamma_part[int64_t(i) * d + col];
        b += dbeta_part[int64_t(i) * d + col];
      }
    }
    s_a[slice][pc] = a;
    s_b[slice][pc] = b;
    __syncthreads();
#pragma unroll
    for (int off = 64; off > 0; off >>= 1) {  // fixed tree over the slices
      if (slice < off) {
        s_a[slice][pc] += s_a[slice + off][pc];
        s_b[slice][pc] += s_b[slice + off][pc];
      }
      __syncthreads();
    }
    if (slice == 0 && col < d) {
      store_elem<DGDT>(dgamma, col, s_a[0][pc] * inv_kf);
      store_elem<DGDT>(dbeta, col, s_b[0][pc] * inv_kf);
    }
  }
  if (blockIdx.x == 0 && warp == 1) {
    // delayed rescale: the factor the main kernel divided by.  Read before this step's statistic is
    // written, so the caller may keep both in the same word.
    float r_prev = 1.0f;
    if (stat_in) { bool nf; r_prev = rescale_factor(*stat_in, &nf); }
    __syncwarp();
    float result = 0.f;
    if (stat != SCALIFY_STAT_NONE) {
      double tot = 0.0;
      for (int i = cx; i < nblocks; i += 32) {
        double p = stat_part[i];
        tot = (stat == SCALIFY_STAT_AMAX) ? fmax(tot, p) : tot + p;
      }
      if (stat == SCALIFY_STAT_AMAX) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tot = fmax(tot, __shfl_xor_sync(0xFFFFFFFFu, tot, o));
      } else {
        tot = warp_sum_f64(tot);
      }
      if (cx == 0) {
        if (stat == SCALIFY_STAT_AMAX) result = __uint_as_float(static_cast<uint32_t>(tot));
        else result = static_cast<float>(sqrt(tot / (static_cast<double>(R) * static_cast<double>(d))));
        *stat_word = result;
      }
    }
    if (cx == 0) {
      const float gs = load_scale(g_scale), xs = load_scale(x_scale), gms = load_scale(gamma_scale);
      uint32_t flags = (is_pow2_scale(gs) && is_pow2_scale(xs) && is_pow2_scale(gms)) ? 0u : SCALIFY_DEV_BAD_SCALE;
      if (exact_hint) {
        bool nonfinite;
        r_prev = rescale_factor(result, &nonfinite);
        if (nonfinite) flags |= SCALIFY_DEV_NONFINITE_STAT;
        *exact_hint = result;
      }
      if (dx_scale) *dx_scale = gs * gms / xs * r_prev;
      if (dgamma_scale) *dgamma_scale = gs * kfactor(R);
      if (dbeta_scale) *dbeta_scale = gs * kfactor(R);
      if (flags && status) atomicOr(status, flags);
    }
  }
}

constexpr int kLnBwdBlocksPerSm = 2;

size_t layernorm_bwd_ws_bytes(int64_t R, int64_t d) {
  int64_t grid = int64_t(sm_count()) * kLnBwdBlocksPerSm;
  (void)R;
  return kWsHeader + size_t(grid) * size_t(d) * 8 + size_t(grid) * 8 + 256;
}

// Launch shape of the backward kernel: team width, grid (persistent) and the number of rows each team walks.
struct LnBwdPlan { int tw, grid, iters; bool ok; };
static LnBwdPlan ln_bwd_plan(int R, int d, int x_dt) {
  LnBwdPlan p{};
  p.tw = ln_team_warps(d, x_dt);
  p.ok = p.tw != 0;
  if (!p.ok) return p;
  p.grid = ln_grid(R, 8 / p.tw, kLnBwdBlocksPerSm);
  const int64_t rows_per_iter = int64_t(p.grid) * (8 / p.tw);
  p.iters = static_cast<int>((R + rows_per_iter - 1) / rows_per_iter);
  return p;
}

int layernorm_plan(int64_t R, int64_t d, int x_dt, int backward, int32_t out[4]) {
  if (backward) {
    const LnBwdPlan p = ln_bwd_plan(static_cast<int>(R), static_cast<int>(d), x_dt);
    if (!p.ok) return SCALIFY_ERR_UNSUPPORTED;
    out[0] = p.grid; out[1] = p.iters; out[2] = p.tw; out[3] = kLnBwdStages;
  } else {
    const LnFwdPlan p = ln_fwd_plan(static_cast<int>(R), static_cast<int>(d), x_dt);
    if (!p.ok) return SCALIFY_ERR_UNSUPPORTED;
    out[0] = p.grid; out[1] = p.rpt; out[2] = p.tw; out[3] = kLnFwdStages;
  }
  return SCALIFY_OK;
}

int launch_layernorm_bwd(const void* G, int64_t g_ld, const void* X, int x_dt, int64_t x_ld, void* dX, int dx_dt,
                         int64_t dx_ld, int R, int d, const void* gamma, int gb_dt, const float* mean,
                         const float* rinv, float eps, int eps_inside, int stat, void* dgamma, void* dbeta, int dg_dt,
                         const float* g_scale, const float* x_scale, const float* gamma_scale, float* dx_scale,
                         float* dgamma_scale, float* dbeta_scale, const float* stat_in, int exact, void* ws,
                         cudaStream_t st) {
  const LnBwdPlan plan = ln_bwd_plan(R, d, x_dt);
  if (!plan.ok) return SCALIFY_ERR_UNSUPPORTED;
  const int tw = plan.tw, grid = plan.grid;
  WsView v = ws_view(ws);
  float* dg_part = static_cast<float*>(v.area);
  float* db_part = dg_part + size_t(grid) * d;
  double* st_part = reinterpret_cast<double*>(db_part + size_t(grid) * d);
  float* dgp = dgamma ? dg_part : nullptr;
  float* dbp = dgamma ? db_part : nullptr;
  constexpr int kBwdSmem = kLnBwdStages * 2 * kLnVpt * kLnThreads * 16;
  if (exact) {
    // one-pass dynamic rescale: first launch with the predicted power of two, finalize (statistic, scale words,
    // next prediction), second launch as a programmatic dependent that returns at once if the prediction held
    if (dx_dt != SCALIFY_E4M3 && dx_dt != SCALIFY_E5M2) return SCALIFY_ERR_UNSUPPORTED;
    LnBwdPredict pred;
    pred.hint = reinterpret_cast<const float*>(static_cast<char*>(ws) + 56);
    pred.r_used = reinterpret_cast<float*>(static_cast<char*>(ws) + 52);
    pred.stat_word = v.stat;
    const int fgrid = dgamma ? (d + 7) / 8 : 1;
#define SCALIFY_LN_BWD_EXACT(W)                                                                                  \
  do {                                                                                                           \
    auto kernel = layernorm_bwd_kernel<XDT, DXDT, W, true>;                                                      \
    static DeviceOnce once; /* per instantiation and device */                                                   \
    int rc_once = device_once(once, nullptr, [&](int*) {                                                         \
      SCALIFY_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmem));     \
      return int(SCALIFY_OK);                                                                                    \
    });                                                                                                          \
    if (rc_once) return rc_once;                                                                                 \
    pred.redo = 0;                                                                                               \
    kernel<<<grid, kLnThreads, kBwdSmem, st>>>(G, g_ld, X, x_ld, dX, dx_ld, R, d, gamma, gb_dt, mean, rinv, eps, \
                                               eps_inside, stat, nullptr, dgp, dbp, st_part, pred);              \
    SCALIFY_CUDA_TRY(cudaGetLastError());                                                                        \
    SCALIFY_DISPATCH_WIDE(dg_dt, DGDT,                                                                           \
        layernorm_bwd_finalize_kernel<DGDT><<<fgrid, 1024, 0, st>>>(grid, R, d, dgp, dbp, st_part, stat, v.stat, \
            dgamma, dbeta, g_scale, x_scale, gamma_scale, dx_scale, dgamma_scale, dbeta_scale, nullptr, v.status, \
            reinterpret_cast<float*>(static_cast<char*>(ws) + 56)));                                             \
    SCALIFY_CUDA_TRY(cudaGetLastError());                                                                        \
    pred.redo = 1;                                                                                               \
    cudaLaunchConfig_t cfg = {};                                                                                 \
    cudaLaunchAttribute attr[1];                                                                                 \
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                             \
    attr[0].val.programmaticStreamSerializationAllowed = 1;                                                      \
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kLnThreads); cfg.dynamicSmemBytes = kBwdSmem; cfg.stream = st; \
    cfg.attrs = attr; cfg.numAttrs = 1;                                                                          \
    SCALIFY_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, G, g_ld, X, x_ld, dX, dx_ld, R, d, gamma, gb_dt, mean,     \
                                        rinv, eps, eps_inside, stat, static_cast<const float*>(nullptr), dgp,   \
                                        dbp, st_part, pred));                                                    \
  } while (0)
    SCALIFY_DISPATCH_WIDE(x_dt, XDT, {
      if (dx_dt == SCALIFY_E4M3) {
        constexpr int DXDT = SCALIFY_E4M3;
        switch (tw) {
          case 1: SCALIFY_LN_BWD_EXACT(1); break;
          case 2: SCALIFY_LN_BWD_EXACT(2); break;
          case 4: SCALIFY_LN_BWD_EXACT(4); break;
          default: SCALIFY_LN_BWD_EXACT(8); break;
        }
      } else {
        constexpr int DXDT = SCALIFY_E5M2;
        switch (tw) {
          case 1: SCALIFY_LN_BWD_EXACT(1); break;
          case 2: SCALIFY_LN_BWD_EXACT(2); break;
          case 4: SCALIFY_LN_BWD_EXACT(4); break;
          default: SCALIFY_LN_BWD_EXACT(8); break;
        }
      }
    });
#undef SCALIFY_LN_BWD_EXACT
    return SCALIFY_OK;
  }
#define SCALIFY_LN_BWD(W)                                                                                        \
  do {                                                                                                           \
    static DeviceOnce once; /* per instantiation and device */                                                   \
    int rc_once = device_once(once, nullptr, [&](int*) {                                                         \
      SCALIFY_CUDA_TRY(cudaFuncSetAttribute(layernorm_bwd_kernel<XDT, DXDT, W, false>,                           \
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, kBwdSmem));             \
      return int(SCALIFY_OK);                                                                                    \
    });                                                                                                          \
    if (rc_once) return rc_once;                                                                                 \
    layernorm_bwd_kernel<XDT, DXDT, W, false><<<grid, kLnThreads, kBwdSmem, st>>>(                               \
        G, g_ld, X, x_ld, dX, dx_ld, R, d, gamma, gb_dt, mean, rinv, eps, eps_inside, stat, stat_in, dgp, dbp,   \
        st_part, LnBwdPredict{});                                                                                \
  } while (0)
  SCALIFY_DISPATCH_WIDE(x_dt, XDT, SCALIFY_DISPATCH_DTYPE(dx_dt, DXDT, {
    switch (tw) {
      case 1: SCALIFY_LN_BWD(1); break;
      case 2: SCALIFY_LN_BWD(2); break;
      case 4: SCALIFY_LN_BWD(4); break;
      default: SCALIFY_LN_BWD(8); break;
    }
  }));
#undef SCALIFY_LN_BWD
  SCALIFY_CUDA_TRY(cudaGetLastError());
  const int fgrid = dgamma ? (d + 7) / 8 : 1;
  SCALIFY_DISPATCH_WIDE(dg_dt, DGDT,
      layernorm_bwd_finalize_kernel<DGDT><<<fgrid, 1024, 0, st>>>(grid, R, d, dgp, dbp, st_part, stat, v.stat, dgamma,
                                                                 dbeta, g_scale, x_scale, gamma_scale, dx_scale,
                                                                 dgamma_scale, dbeta_scale, stat_in, v.status, nullptr));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

}  // namespace scalify
