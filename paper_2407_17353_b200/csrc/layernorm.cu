// Scaled LayerNorm forward and backward (Section 3.2.1, Appendix C.2, Algorithm 5).
//
// HBM-bound: every element of X (and G) is read once and every output written once.  A row
// is owned by a team of WARPS warps; each thread keeps up to kMaxVpt 16-byte vectors of the
// row in registers, so mean, variance and the normalised values come from one read.  gamma
// and beta are re-read per row through L1 (they are a few KB).  Blocks stride over rows with
// a grid that is a multiple of the SM count.
#include "scalify_common.cuh"
#include "scalify_launch.h"

namespace scalify {

constexpr int kLnThreads = 128;  // 4 warps per block
constexpr int kMaxVpt = 4;       // 16-byte vectors per thread and row

template <int WARPS>
__device__ __forceinline__ void team_sum2(float& a, float& b, float* smem) {
  a = warp_sum_f32(a);
  b = warp_sum_f32(b);
  if constexpr (WARPS > 1) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();  // previous use of smem is over
    if (lane == 0) { smem[2 * warp] = a; smem[2 * warp + 1] = b; }
    __syncthreads();
    a = 0.f; b = 0.f;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) { a += smem[2 * w]; b += smem[2 * w + 1]; }
  }
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
template <int XDT, int YDT, int WARPS>
__global__ void __launch_bounds__(kLnThreads) layernorm_fwd_kernel(
    const void* __restrict__ X, int64_t x_ld, void* __restrict__ Y, int64_t y_ld, int R, int d,
    const void* __restrict__ gamma, const void* __restrict__ beta, int gb_dt, const float* gamma_scale,
    const float* beta_scale, float* y_scale, float eps, int eps_inside, float* __restrict__ mean_out,
    float* __restrict__ rinv_out) {
  constexpr int VEC = 16 / ElemBytes<XDT>::v;
  constexpr int OB = VEC * ElemBytes<YDT>::v;
  constexpr int TEAM = 32 * WARPS;
  constexpr int TEAMS_PER_BLOCK = kLnThreads / TEAM;
  __shared__ float smem[2 * (kLnThreads / 32)];
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
  const float inv_d = 1.0f / static_cast<float>(d);
  const int rows_per_iter = gridDim.x * TEAMS_PER_BLOCK;
  const int iters = (R + rows_per_iter - 1) / rows_per_iter;
  for (int it = 0; it < iters; ++it) {
    const int row = it * rows_per_iter + blockIdx.x * TEAMS_PER_BLOCK + team;
    const bool live = row < R;
    float x[kMaxVpt][VEC];
    const char* xrow = static_cast<const char*>(X) + int64_t(live ? row : 0) * x_ld * ElemBytes<XDT>::v;
#pragma unroll
    for (int v = 0; v < kMaxVpt; ++v) {
      const int vi = t + v * TEAM;
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      if (live && vi < n_vec) ld_raw_stream<16>(xrow + int64_t(vi) * 16, w);
      decode_vec<XDT, VEC>(w, x[v]);
    }
    float s = 0.f, dummy = 0.f;
#pragma unroll
    for (int v = 0; v < kMaxVpt; ++v)
#pragma unroll
      for (int e = 0; e < VEC; ++e) s += x[v][e];
    team_sum2<WARPS>(s, dummy, smem);
    const float mu = s * inv_d;
    float q = 0.f;
    dummy = 0.f;
#pragma unroll
    for (int v = 0; v < kMaxVpt; ++v) {
      const int vi = t + v * TEAM;
      if (vi < n_vec) {
#pragma unroll
        for (int e = 0; e < VEC; ++e) { float c = x[v][e] - mu; q = fmaf(c, c, q); }
      }
    }
    team_sum2<WARPS>(q, dummy, smem);
    const float var = q * inv_d;
    const float rinv = eps_inside ? 1.0f / sqrtf(var + eps) : 1.0f / (sqrtf(var) + eps);
    if (live) {
      if (t == 0) {
        if (mean_out) mean_out[row] = mu;
        if (rinv_out) rinv_out[row] = rinv;
      }
      char* yrow = static_cast<char*>(Y) + int64_t(row) * y_ld * ElemBytes<YDT>::v;
#pragma unroll
      for (int v = 0; v < kMaxVpt; ++v) {
        const int vi = t + v * TEAM;
        if (vi < n_vec) {
          float o[VEC];
#pragma unroll
          for (int e = 0; e < VEC; ++e) o[e] = (x[v][e] - mu) * rinv;
          if (gamma) {
            float g[VEC];
            load_param_vec<VEC>(gamma, gb_dt, vi * VEC, g);
#pragma unroll
            for (int e = 0; e < VEC; ++e) o[e] = o[e] * g[e] * fg;
            if (beta) {
              load_param_vec<VEC>(beta, gb_dt, vi * VEC, g);
#pragma unroll
              for (int e = 0; e < VEC; ++e) o[e] = fmaf(g[e], fb, o[e]);
            }
          }
          uint32_t ow[OB / 4];
          encode_vec<YDT, VEC>(o, ow);
          st_raw<OB>(yrow + int64_t(vi) * OB, ow);
        }
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && y_scale) *y_scale = ys;
}

int ln_grid(int R, int teams_per_block, int blocks_per_sm) {
  int64_t need = (int64_t(R) + teams_per_block - 1) / teams_per_block;
  int64_t cap = int64_t(sm_count()) * blocks_per_sm;
  if (need < 1) need = 1;
  return static_cast<int>(need < cap ? need : cap);
}

// chooses the team width; returns 0 if the row is too long for the register budget
static int ln_warps(int d, int x_dt) {
  int n_vec = d * elem_size(x_dt) / 16;
  if (n_vec <= 32 * kMaxVpt) return 1;
  if (n_vec <= 128 * kMaxVpt) return 4;
  return 0;
}

int launch_layernorm_fwd(const void* X, int x_dt, int64_t x_ld, void* Y, int y_dt, int64_t y_ld, int R, int d,
                         const void* gamma, const void* beta, int gb_dt, const float* gamma_scale,
                         const float* beta_scale, float* y_scale, float eps, int eps_inside, float* mean,
                         float* rinv, cudaStream_t st) {
  const int warps = ln_warps(d, x_dt);
  if (warps == 0) return SCALIFY_ERR_UNSUPPORTED;
  const int grid = ln_grid(R, 4 / warps, 12);
#define SCALIFY_LN_FWD(W)                                                                                      \
  layernorm_fwd_kernel<XDT, YDT, W><<<grid, kLnThreads, 0, st>>>(X, x_ld, Y, y_ld, R, d, gamma, beta, gb_dt,    \
                                                                 gamma_scale, beta_scale, y_scale, eps,         \
                                                                 eps_inside, mean, rinv)
  SCALIFY_DISPATCH_WIDE(x_dt, XDT, SCALIFY_DISPATCH_DTYPE(y_dt, YDT, {
    if (warps == 1) SCALIFY_LN_FWD(1); else SCALIFY_LN_FWD(4);
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
template <int WARPS> struct BwdCfg {
  static constexpr int threads = WARPS == 1 ? 256 : 128;  // WARPS == 1: eight one-warp teams per block
  static constexpr int min_blocks = WARPS == 1 ? 2 : 3;
};

template <int XDT, int DXDT, int WARPS>
__global__ void __launch_bounds__(BwdCfg<WARPS>::threads, BwdCfg<WARPS>::min_blocks) layernorm_bwd_kernel(
    const void* __restrict__ G, int64_t g_ld, const void* __restrict__ X, int64_t x_ld, void* __restrict__ dX,
    int64_t dx_ld, int R, int d, const void* __restrict__ gamma, int gb_dt, const float* __restrict__ mean,
    const float* __restrict__ rinv_in, float eps, int eps_inside, int stat, float* __restrict__ dgamma_part,
    float* __restrict__ dbeta_part, double* __restrict__ stat_part) {
  constexpr int VEC = 16 / ElemBytes<XDT>::v;
  constexpr int OB = VEC * ElemBytes<DXDT>::v;
  constexpr int TEAM = 32 * WARPS;
  constexpr int THREADS = BwdCfg<WARPS>::threads;
  constexpr int TEAMS_PER_BLOCK = THREADS / TEAM;
  __shared__ float smem[2 * (THREADS / 32)];
  const int n_vec = d / VEC;
  const int t = threadIdx.x % TEAM;
  const int team = threadIdx.x / TEAM;
  const float inv_d = 1.0f / static_cast<float>(d);
  float acc_dg[kMaxVpt][VEC], acc_db[kMaxVpt][VEC];
#pragma unroll
  for (int v = 0; v < kMaxVpt; ++v)
#pragma unroll
    for (int e = 0; e < VEC; ++e) { acc_dg[v][e] = 0.f; acc_db[v][e] = 0.f; }
  uint32_t amax = 0u;
  float ssq = 0.f;
  const int rows_per_iter = gridDim.x * TEAMS_PER_BLOCK;
  const int iters = (R + rows_per_iter - 1) / rows_per_iter;
  for (int it = 0; it < iters; ++it) {
    const int row = it * rows_per_iter + blockIdx.x * TEAMS_PER_BLOCK + team;
    const bool live = row < R;
    const int srow = live ? row : 0;
    float x[kMaxVpt][VEC], g[kMaxVpt][VEC];
    const char* xrow = static_cast<const char*>(X) + int64_t(srow) * x_ld * ElemBytes<XDT>::v;
    const char* grow = static_cast<const char*>(G) + int64_t(srow) * g_ld * ElemBytes<XDT>::v;
#pragma unroll
    for (int v = 0; v < kMaxVpt; ++v) {
      const int vi = t + v * TEAM;
      uint32_t wx[4] = {0u, 0u, 0u, 0u}, wg[4] = {0u, 0u, 0u, 0u};
      if (live && vi < n_vec) {
        ld_raw_stream<16>(xrow + int64_t(vi) * 16, wx);
        ld_raw_stream<16>(grow + int64_t(vi) * 16, wg);
      }
      decode_vec<XDT, VEC>(wx, x[v]);
      decode_vec<XDT, VEC>(wg, g[v]);
    }
    const float mu = __ldg(&mean[srow]);
    const float rinv = __ldg(&rinv_in[srow]);
    float m1 = 0.f, m2 = 0.f;
#pragma unroll
    for (int v = 0; v < kMaxVpt; ++v) {
      const int vi = t + v * TEAM;
      if (live && vi < n_vec) {
        float gam[VEC];
        if (gamma) load_param_vec<VEC>(gamma, gb_dt, vi * VEC, gam);
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
          const float n = (x[v][e] - mu) * rinv;
          acc_dg[v][e] = fmaf(g[v][e], n, acc_dg[v][e]);
          acc_db[v][e] += g[v][e];
          const float gh = gamma ? g[v][e] * gam[e] : g[v][e];
          x[v][e] = n;   // keep n
          g[v][e] = gh;  // keep ghat
          m1 += gh;
          m2 = fmaf(gh, n, m2);
        }
      }
    }
    team_sum2<WARPS>(m1, m2, smem);
    m1 *= inv_d;
    m2 *= inv_d;
    // eps outside the root: dx = (ghat-m1)*rinv - n*m2/s with s = 1/rinv - eps (0 if s == 0)
    // eps inside the root:  dx = rinv*(ghat - m1 - n*m2)
    float c2;
    if (eps_inside) {
      c2 = rinv * m2;
    } else {
      const float s = 1.0f / rinv - eps;
      c2 = (s > 0.f) ? m2 / s : 0.f;
    }
    if (live) {
      char* orow = static_cast<char*>(dX) + int64_t(row) * dx_ld * ElemBytes<DXDT>::v;
#pragma unroll
      for (int v = 0; v < kMaxVpt; ++v) {
        const int vi = t + v * TEAM;
        if (vi < n_vec) {
          float o[VEC];
#pragma unroll
          for (int e = 0; e < VEC; ++e) {
            o[e] = fmaf(-x[v][e], c2, (g[v][e] - m1) * rinv);
            const float stored = round_through<DXDT>(o[e]);
            amax = max(amax, abs_bits(stored));
            ssq = fmaf(stored, stored, ssq);
          }
          uint32_t ow[OB / 4];
          encode_vec<DXDT, VEC>(o, ow);
          st_raw<OB>(orow + int64_t(vi) * OB, ow);
        }
      }
    }
  }
  // per-block column partials of dgamma / dbeta
  if (dgamma_part) {
    if constexpr (WARPS == 1) {
      // the teams of a block own the same columns: combine them through shared memory in team order
      __shared__ float s_col[TEAMS_PER_BLOCK][32][VEC + 1];
#pragma unroll
      for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
        for (int v = 0; v < kMaxVpt; ++v) {
          const int vi = t + v * TEAM;
          __syncthreads();
#pragma unroll
          for (int e = 0; e < VEC; ++e) s_col[team][t][e] = pass ? acc_db[v][e] : acc_dg[v][e];
          __syncthreads();
          if (team == 0 && vi < n_vec) {
            float* dst = (pass ? dbeta_part : dgamma_part) + int64_t(blockIdx.x) * d + vi * VEC;
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
              float sum = s_col[0][t][e];
#pragma unroll
              for (int tm = 1; tm < TEAMS_PER_BLOCK; ++tm) sum += s_col[tm][t][e];
              dst[e] = sum;
            }
          }
        }
      }
    } else {
#pragma unroll
      for (int v = 0; v < kMaxVpt; ++v) {
        const int vi = t + v * TEAM;
        if (vi < n_vec) {
          float* dg = dgamma_part + int64_t(blockIdx.x) * d + vi * VEC;
          float* db = dbeta_part + int64_t(blockIdx.x) * d + vi * VEC;
#pragma unroll
          for (int e = 0; e < VEC; ++e) { dg[e] = acc_dg[v][e]; db[e] = acc_db[v][e]; }
        }
      }
    }
  }
  if (stat != SCALIFY_STAT_NONE) {
    __shared__ double s_stat[THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double mine = (stat == SCALIFY_STAT_AMAX) ? static_cast<double>(warp_max_u32(amax))
                                              : warp_sum_f64(static_cast<double>(ssq));
    if (lane == 0) s_stat[warp] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
      double tot = s_stat[0];
      for (int i = 1; i < THREADS / 32; ++i)
        tot = (stat == SCALIFY_STAT_AMAX) ? fmax(tot, s_stat[i]) : tot + s_stat[i];
      stat_part[blockIdx.x] = tot;
    }
  }
}

// Combines the per-block partials in block order: dgamma/dbeta columns (scaled by 1/kf(R)), the
// statistic word, and the propagated scale words.  Block = 32 columns x 8 slices of the block list.
template <int DGDT>
__global__ void __launch_bounds__(256) layernorm_bwd_finalize_kernel(
    int nblocks, int R, int d, const float* __restrict__ dgamma_part, const float* __restrict__ dbeta_part,
    const double* __restrict__ stat_part, int stat, float* stat_word, void* __restrict__ dgamma,
    void* __restrict__ dbeta, const float* g_scale, const float* x_scale, const float* gamma_scale,
    float* dx_scale, float* dgamma_scale, float* dbeta_scale, uint32_t* status) {
  __shared__ float s_a[8][33], s_b[8][33];
  const float inv_kf = 1.0f / kfactor(R);
  const int cx = threadIdx.x & 31, slice = threadIdx.x >> 5;
  const int col = blockIdx.x * 32 + cx;
  if (dgamma_part) {
    float a = 0.f, b = 0.f;
    if (col < d) {
      for (int i = slice; i < nblocks; i += 8) {
        a += dgamma_part[int64_t(i) * d + col];
        b += dbeta_part[int64_t(i) * d + col];
      }
    }
    s_a[slice][cx] = a;
    s_b[slice][cx] = b;
    __syncthreads();
    if (slice == 0 && col < d) {
      for (int k = 1; k < 8; ++k) { a += s_a[k][cx]; b += s_b[k][cx]; }
      store_elem<DGDT>(dgamma, col, a * inv_kf);
      store_elem<DGDT>(dbeta, col, b * inv_kf);
    }
  }
  if (blockIdx.x == 0 && slice == 1) {
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
        float result;
        if (stat == SCALIFY_STAT_AMAX) result = __uint_as_float(static_cast<uint32_t>(tot));
        else result = static_cast<float>(sqrt(tot / (static_cast<double>(R) * static_cast<double>(d))));
        *stat_word = result;
      }
    }
    if (cx == 0) {
      const float gs = load_scale(g_scale), xs = load_scale(x_scale), gms = load_scale(gamma_scale);
      uint32_t flags = (is_pow2_scale(gs) && is_pow2_scale(xs) && is_pow2_scale(gms)) ? 0u : SCALIFY_DEV_BAD_SCALE;
      if (dx_scale) *dx_scale = gs * gms / xs;
      if (dgamma_scale) *dgamma_scale = gs * kfactor(R);
      if (dbeta_scale) *dbeta_scale = gs * kfactor(R);
      if (flags && status) atomicOr(status, flags);
    }
  }
}

size_t layernorm_bwd_ws_bytes(int64_t R, int64_t d) {
  int64_t grid = int64_t(sm_count()) * 3;
  (void)R;
  return kWsHeader + size_t(grid) * size_t(d) * 8 + size_t(grid) * 8 + 256;
}

int launch_layernorm_bwd(const void* G, int64_t g_ld, const void* X, int x_dt, int64_t x_ld, void* dX, int dx_dt,
                         int64_t dx_ld, int R, int d, const void* gamma, int gb_dt, const float* mean,
                         const float* rinv, float eps, int eps_inside, int stat, void* dgamma, void* dbeta, int dg_dt,
                         const float* g_scale, const float* x_scale, const float* gamma_scale, float* dx_scale,
                         float* dgamma_scale, float* dbeta_scale, void* ws, cudaStream_t st) {
  const int warps = ln_warps(d, x_dt);
  if (warps == 0) return SCALIFY_ERR_UNSUPPORTED;
  const int grid = (warps == 1) ? ln_grid(R, 8, 2) : ln_grid(R, 1, 3);
  WsView v = ws_view(ws);
  float* dg_part = static_cast<float*>(v.area);
  float* db_part = dg_part + size_t(grid) * d;
  double* st_part = reinterpret_cast<double*>(db_part + size_t(grid) * d);
  float* dgp = dgamma ? dg_part : nullptr;
  float* dbp = dgamma ? db_part : nullptr;
#define SCALIFY_LN_BWD(W)                                                                                          \
  layernorm_bwd_kernel<XDT, DXDT, W><<<grid, BwdCfg<W>::threads, 0, st>>>(G, g_ld, X, x_ld, dX, dx_ld, R, d, gamma, gb_dt,  \
                                                                  mean, rinv, eps, eps_inside, stat, dgp, dbp,      \
                                                                  st_part)
  SCALIFY_DISPATCH_WIDE(x_dt, XDT, SCALIFY_DISPATCH_WIDE(dx_dt, DXDT, {
    if (warps == 1) SCALIFY_LN_BWD(1); else SCALIFY_LN_BWD(4);
  }));
#undef SCALIFY_LN_BWD
  SCALIFY_CUDA_TRY(cudaGetLastError());
  const int fgrid = dgamma ? (d + 31) / 32 : 1;
  SCALIFY_DISPATCH_WIDE(dg_dt, DGDT,
      layernorm_bwd_finalize_kernel<DGDT><<<fgrid, 256, 0, st>>>(grid, R, d, dgp, dbp, st_part, stat, v.stat, dgamma,
                                                                 dbeta, g_scale, x_scale, gamma_scale, dx_scale,
                                                                 dgamma_scale, dbeta_scale, v.status));
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

}  // namespace scalify
