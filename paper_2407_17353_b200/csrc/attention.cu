// Fused scaled attention forward (Section 3.2.1: attention is a place for a custom scale rule;
// the rule taken here is the composition the unfused path uses): for every head
//   S = Q K^T            scaled FP8 matmul, static rule:  S_s = Q_s K_s kf(hd),  S_d = bf16(acc / kf(hd))
//   P = softmax(S_d S_s c) on VALUES (c = 1/sqrt(hd) or any scalar), causal mask optional; the
//                        probabilities are bounded, carry scale 1 and are rounded to E4M3
//   O = P V              scaled FP8 matmul, static rule:  O_s = V_s kf(Tk),  O_d = acc / kf(Tk)
// in ONE kernel: neither S nor P ever reaches HBM (unless the caller asks for debug copies).
//
// One CTA per (head, block of 128 queries); 288 threads:
//   warps 0-7   two threads per query row (the TMEM lane of the row; each takes 64 of a block's 128
//               keys): read the score block from TMEM, softmax arithmetic, write the E4M3
//               probabilities as the A operand of the second matmul into shared memory (128-byte
//               swizzle), final read-out of O; the two partial (maximum, sum) pairs of a row are
//               combined once, between the sweeps
//   warp 8      one thread: TMA loads of Q, K, V tiles (64-byte swizzle) and all tcgen05.mma
// The softmax is the exact two-sweep form, not an online approximation of it: sweep A runs
// Q K^T over the key blocks and keeps the row maximum m and the sum l = sum exp(s - m)
// (moved to the new maximum whenever a 32-key chunk raises it); sweep B recomputes Q K^T, forms p = exp(s - m) / l, rounds it to
// E4M3 and accumulates P V in TMEM.  The probabilities are therefore the same normalised values
// the unfused path quantises, and O needs no rescaling.  Cost: the Q K^T work twice.
// The tensor core stays AHEAD of the row threads.  A row thread hands the score buffer back as soon as its
// last chunk of the block is in registers, and the issuing thread computes the scores of block b+1 BEFORE it
// waits for the probabilities of block b; two probability tiles in shared memory let the rows write block b+1
// while P V of block b runs; K / V tiles travel through a three-deep ring, fetched two blocks ahead.  (When the
// two sides took turns - one probability tile, buffer handed back after the arithmetic - 96 heads x 1024 x 64
// took 71 us; 57 us with the cheaper BF16 rounding below, 50 us with the hand-offs out of the way.  A form
// with ONE CTA of 16 row warps per SM and two score buffers in TMEM measured 67 us: two CTAs that drift apart
// fill each other's exp2 / conversion phases, sixteen warps released by the same barrier do not.)
// TMEM: 128 columns of scores + 64 columns of O (256 allocated, so two CTAs share an SM).
// Every mbarrier wait is bounded; on expiry the CTA records SCALIFY_DEV_TIMEOUT and leaves.
#include <cuda.h>

#include "scalify_common.cuh"
#include "scalify_launch.h"
#include "tcgen05_ptx.cuh"

namespace scalify {

constexpr int kAttQ = 128;     // queries per CTA
constexpr int kAttK = 128;     // keys per block
constexpr int kAttHd = 64;     // bytes per row of a Q, K or V tile: a head dimension of 128 travels as two such tiles
constexpr int kAttSmWarps = 8;   // softmax warps: two per TMEM lane quarter, each taking half of the key columns
constexpr int kAttThreads = 32 * (kAttSmWarps + 1);
constexpr int kAttTmemCols = 256;
constexpr uint32_t kAttOCol = 128;
constexpr int kAttKvStages = 3;
constexpr int kAttTileBytes = kAttK * kAttHd;  // 8 KB: a Q, K or V tile
// NH = head dimension / 64: every Q, K, V tile is NH column halves of 8 KB, one after the other
constexpr size_t att_smem(int nh) {
  return size_t(kAttTileBytes) * nh * (1 + 2 * kAttKvStages) /*Q, K ring, V ring*/ + 2 * kAttQ * kAttK /*two P tiles*/ +
         1024 + 256;
}

struct AttParams {
  int heads, h_inner, Tq, Tk, q_blocks;   // heads = batch x h_inner
  int causal;
  const float* q_scale; const float* k_scale;
  float sc_const;   // kf(hd) c log2(e); times Q_s K_s: scores' data component -> exponent in base 2
  float inv_kf_hd;  // 1 / kf(hd)
  float inv_kf_tk;  // 1 / kf(Tk)
  uint32_t idesc_s, idesc_pv;
  void* O; long long o_ld, o_hs, o_bs;
  void* S_dump; void* P_dump;
  const float* v_scale; float kf_tk; float* o_scale;
  uint32_t* status;
};

// 64-byte-swizzle shared-memory matrix descriptor (layout type 4): K-major tile of 64-byte rows
// (8-row atoms 512 B apart) or MN-major tile whose 64 MN-elements are one row (8 K-rows per atom).
__device__ __forceinline__ uint64_t make_smem_desc_sw64(uint32_t saddr, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= 4ull << 61;
  return d;
}

// 2^x for x <= 0 (and -inf): the hardware approximation (2 ulp of fp32, results below 2^-126 flush to 0),
// far finer than the E4M3 probabilities it feeds
// three-input maximum (one instruction on sm_100)
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

__device__ __forceinline__ float exp2_neg(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

template <int ODT, int NH>
__global__ void __launch_bounds__(kAttThreads, 2)
attention_fwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const AttParams p) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  constexpr int kTile = NH * kAttTileBytes;  // a Q, K or V tile: NH column halves of [128 rows][64 B]
  const uint32_t smem_q = base;
  const uint32_t smem_k = base + kTile;                              // kAttKvStages slots
  const uint32_t smem_v = base + (1 + kAttKvStages) * kTile;         // kAttKvStages slots
  const uint32_t smem_p = base + (1 + 2 * kAttKvStages) * kTile;     // 2 x 16 KB, 1024-byte aligned
  uint8_t* p_tiles = smem + (1 + 2 * kAttKvStages) * kTile;
  uint8_t* bar_mem = p_tiles + 2 * kAttQ * kAttK;
  const uint32_t bars = smem_p + 2 * kAttQ * kAttK;
  const uint32_t q_full = bars, kv_full = bars + 8 /*3*/, kv_empty = bars + 32 /*3*/, s_full = bars + 56,
                 s_empty = bars + 72, p_full = bars + 88 /*2*/, p_empty = bars + 104 /*2*/, o_full = bars + 120;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_mem + 128);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // query blocks in descending order within the launch: with a causal mask the late blocks have the most key
  // blocks, and starting them first leaves the short ones to fill the end of the launch
  const int qb = p.q_blocks - 1 - static_cast<int>(blockIdx.x / p.heads), head = blockIdx.x % p.heads;
  const int hh = head % p.h_inner, bb = head / p.h_inner;  // head inside its batch element, batch element
  const int q0 = qb * kAttQ;
  const int shift = p.Tk - p.Tq;  // causal: query i sees keys j <= i + shift
  int n_kb = (p.Tk + kAttK - 1) / kAttK;
  if (p.causal) n_kb = min(n_kb, (q0 + kAttQ - 1 + shift) / kAttK + 1);

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < kAttKvStages; ++s) { mbar_init(kv_full + 8 * s, 1); mbar_init(kv_empty + 8 * s, 1); }
    mbar_init(s_full, 1);
    mbar_init(s_empty, kAttSmWarps);
    for (int s = 0; s < 2; ++s) { mbar_init(p_full + 8 * s, kAttSmWarps); mbar_init(p_empty + 8 * s, 1); }
    mbar_init(o_full, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (blockIdx.x == 0) {
      const float vs = load_scale(p.v_scale);
      if (p.o_scale) *p.o_scale = vs * p.kf_tk;  // P carries scale 1
      if (!is_pow2_scale(vs) && p.status) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
    }
  }
  if (warp == kAttSmWarps) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kAttTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool timed_out = false;

  if (warp == kAttSmWarps) {
    // ------------------------------------------------------------ loads and MMAs (one thread)
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
      const int n_it = 2 * n_kb;  // iteration j: sweep A block j (K only), then sweep B block j - n_kb (K and V)
      // K (and V) tiles of iteration j into ring slot j % kAttKvStages
      auto issue_load = [&](int j) {
        const int slot = j % kAttKvStages, use = j / kAttKvStages;
        if (use >= 1 && !mbar_wait(kv_empty + 8 * slot, (use - 1) & 1, abort_flag)) { timed_out = true; return; }
        const bool sweep_b = j >= n_kb;
        const int kb = sweep_b ? j - n_kb : j;
        const uint32_t fb = kv_full + 8 * slot;
        mbar_expect_tx(fb, sweep_b ? 2 * kTile : kTile);
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          tma_load_4d(smem_k + slot * kTile + h * kAttTileBytes, &map_k, fb, h * kAttHd, kb * kAttK, hh, bb);
          if (sweep_b) tma_load_4d(smem_v + slot * kTile + h * kAttTileBytes, &map_v, fb, h * kAttHd, kb * kAttK, hh, bb);
        }
      };
      mbar_expect_tx(q_full, kTile);
#pragma unroll
      for (int h = 0; h < NH; ++h) tma_load_4d(smem_q + h * kAttTileBytes, &map_q, q_full, h * kAttHd, q0, hh, bb);
      issue_load(0);
      if (!timed_out && n_it > 1) issue_load(1);
      if (!timed_out && !mbar_wait(q_full, 0u, abort_flag)) timed_out = true;
      const uint64_t q_desc = make_smem_desc_sw64(smem_q, 512u);
      // scores of iteration j (the score buffer is free once the rows have taken iteration j - 1 to registers)
      auto issue_scores = [&](int j) {
        const int slot = j % kAttKvStages;
        if (!mbar_wait(kv_full + 8 * slot, (j / kAttKvStages) & 1, abort_flag)) { timed_out = true; return; }
        if (j >= 1 && !mbar_wait(s_empty, (j - 1) & 1, abort_flag)) { timed_out = true; return; }
        tc_fence_after();
        const uint64_t k_desc = make_smem_desc_sw64(smem_k + slot * kTile, 512u);
#pragma unroll
        for (int h = 0; h < NH; ++h)  // the contraction runs over the column halves ...
#pragma unroll
          for (int k = 0; k < kAttHd / 32; ++k)  // ... K = 32 bytes per MMA: +32 B on both K-major operands
            umma_f8(tmem_base, q_desc + static_cast<uint64_t>(h * (kAttTileBytes >> 4) + k * 2),
                    k_desc + static_cast<uint64_t>(h * (kAttTileBytes >> 4) + k * 2), p.idesc_s, (h | k) != 0 ? 1u : 0u);
        umma_commit(s_full);
        if (j < n_kb) umma_commit(kv_empty + 8 * slot);  // sweep A: the K tile is free after Q K^T
      };
      if (!timed_out) issue_scores(0);
      for (int it = 0; it < n_it && !timed_out; ++it) {
        // stay ahead of the rows: tiles two iterations ahead, scores one iteration ahead
        if (it + 2 < n_it) { issue_load(it + 2); if (timed_out) break; }
        if (it + 1 < n_it) { issue_scores(it + 1); if (timed_out) break; }
        if (it >= n_kb) {
          const int b = it - n_kb, pb = b & 1, slot = it % kAttKvStages;
          if (!mbar_wait(p_full + 8 * pb, (b >> 1) & 1, abort_flag)) { timed_out = true; break; }
          tc_fence_after();
          // P tile [128 queries][128 B of keys], K-major; V tile [128 keys][64 B]: the B operand in MN-major form,
          // 8-key atoms 512 B apart, 32 keys per MMA
          const uint64_t p_desc = make_smem_desc(smem_p + pb * (kAttQ * kAttK), 0u, 1024u);
          const uint64_t v_desc = make_smem_desc_sw64(smem_v + slot * kTile, 512u);
#pragma unroll
          for (int h = 0; h < NH; ++h)  // 64 columns of O per column half of V
#pragma unroll
            for (int k = 0; k < kAttK / 32; ++k)
              umma_f8(tmem_base + kAttOCol + h * kAttHd, p_desc + static_cast<uint64_t>(k * 2),
                      v_desc + static_cast<uint64_t>(h * (kAttTileBytes >> 4) + k * (32 * kAttHd / 16)), p.idesc_pv,
                      (b | k) != 0 ? 1u : 0u);
          umma_commit(p_empty + 8 * pb);
          umma_commit(kv_empty + 8 * slot);
        }
      }
      if (!timed_out) umma_commit(o_full);
      if (timed_out || *abort_flag) {
        // wait (bounded) for the copies still in flight before the CTA's shared memory goes away
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) {}
      }
    }
  } else {
    // ------------------------------------------------------------ softmax rows (one row per thread)
    const int quarter = warp & 3, half = warp >> 2;   // TMEM lane quarter; which 64 of a block's 128 keys
    const int r = quarter * 32 + lane;
    const int i = q0 + r;                     // query index
    const int lim = p.causal ? min(p.Tk, i + shift + 1) : p.Tk;  // keys [0, lim) are visible
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    constexpr int kChunks = kAttK / 32 / 2;   // 32-key chunks per thread and block
    const int c_first = half * kChunks;
    float m = -INFINITY, l = 0.f;
    const float sc2 = load_scale(p.q_scale) * load_scale(p.k_scale) * p.sc_const;
    long long dump_row = (static_cast<long long>(head) * p.Tq + i) * p.Tk;
    // x = data component of the score, rounded to BF16 like the unfused intermediate, in units of log2(e).
    // Dividing by kf(hd) only shifts the exponent, so it commutes with the rounding and is folded into sc3.
    const float sc3 = sc2 * p.inv_kf_hd;
    // The BF16 rounding (round to nearest even, as the unfused intermediate is rounded) runs on the fp32 pipe
    // (bf16_round_f32): the conversion unit is shared with exp2, and the integer form (four half-rate
    // instructions per element) made the integer pipe this kernel's busiest.
    const float2 sc3_2 = make_float2(sc3, sc3);
    // x[e] = rounded score times sc3 for the visible keys of a 32-key chunk, -inf for the others
    auto chunk_scores = [&](const uint32_t* acc_bits, int j0, float* x) {
#pragma unroll
      for (int e = 0; e < 32; e += 2) {
        const float2 v = __fmul2_rn(make_float2(bf16_round_f32(__uint_as_float(acc_bits[e])),
                                                bf16_round_f32(__uint_as_float(acc_bits[e + 1]))), sc3_2);
        x[e] = v.x;
        x[e + 1] = v.y;
      }
      if (j0 + 32 > lim) {  // the chunk crosses the end of this row's visible keys
#pragma unroll
        for (int e = 0; e < 32; ++e) x[e] = (j0 + e < lim) ? x[e] : -INFINITY;
      }
    };
    // Fast form for a positive scale (every real use): r[k] = the two rounded scores 2k, 2k+1 in accumulator
    // units (two-wide rounding, 1.5 instructions per element), -inf for hidden keys.  The scale is applied
    // inside the multiply-add that also subtracts the row maximum, and the row maximum is taken on the unscaled
    // values (scaling by a positive constant is monotone, so fl(max r * sc3) is the maximum of fl(r * sc3)).
    const bool pos_scale = sc3 > 0.f;
    auto chunk_rounded = [&](const uint32_t* acc_bits, int j0, float2* r2) {
#pragma unroll
      for (int k = 0; k < 16; ++k)
        r2[k] = bf16_round_f32x2(make_float2(__uint_as_float(acc_bits[2 * k]), __uint_as_float(acc_bits[2 * k + 1])));
      if (j0 + 32 > lim) {
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          r2[k].x = (j0 + 2 * k < lim) ? r2[k].x : -INFINITY;
          r2[k].y = (j0 + 2 * k + 1 < lim) ? r2[k].y : -INFINITY;
        }
      }
    };
    int it = 0;
    // sweep A: row maximum and sum of exponentials
    for (int kb = 0; kb < n_kb; ++kb, ++it) {
      if (!mbar_wait(s_full, it & 1, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      uint32_t acc[32];
#pragma unroll 1
      for (int c = c_first; c < c_first + kChunks; ++c) {
        tmem_ld32(t_row + c * 32, acc);
        tmem_ld_wait();
        if (c == c_first + kChunks - 1) {
          // the score block is in registers: hand the TMEM buffer back now, so that the tensor core computes the
          // next block's scores while this one is worked on (taking both chunks to registers first, to hand it
          // back a chunk earlier, costs a second CTA per SM its registers: 83 us against 54 us; issuing the next
          // chunk's read under this chunk's arithmetic changed nothing: 51.5 against 50.6 us)
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(s_empty);
        }
        // one pass per 32-key chunk: chunk maximum, then the running sum is moved to the new maximum
        if (pos_scale) {
          float2 r2[16];
          chunk_rounded(acc, kb * kAttK + c * 32, r2);
          float cm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // four independent chains
#pragma unroll
          for (int k = 0; k < 16; ++k) cm4[k & 3] = fmax3(cm4[k & 3], r2[k].x, r2[k].y);
          const float m_new = fmaxf(m, fmaxf(fmaxf(cm4[0], cm4[1]), fmaxf(cm4[2], cm4[3])) * sc3);
          if (m_new > -INFINITY) {
            const float2 nm2 = make_float2(-m_new, -m_new);
            float2 add2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
            for (int k = 0; k < 16; ++k) {
              const float2 a = __ffma2_rn(r2[k], sc3_2, nm2);  // -inf for hidden keys: 2^-inf = 0
              add2[k & 1] = __fadd2_rn(add2[k & 1], make_float2(exp2_neg(a.x), exp2_neg(a.y)));
            }
            l = l * exp2_neg(m - m_new) + ((add2[0].x + add2[0].y) + (add2[1].x + add2[1].y));  // and while nothing was seen
            m = m_new;
          }
        } else {
          float x[32];
          chunk_scores(acc, kb * kAttK + c * 32, x);
          float cm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int e = 0; e < 32; ++e) cm4[e & 3] = fmaxf(cm4[e & 3], x[e]);
          const float m_new = fmaxf(m, fmaxf(fmaxf(cm4[0], cm4[1]), fmaxf(cm4[2], cm4[3])));
          if (m_new > -INFINITY) {
            const float2 nm2 = make_float2(-m_new, -m_new);
            float2 add2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float2 a = __fadd2_rn(make_float2(x[e], x[e + 1]), nm2);
              add2[(e >> 1) & 1] = __fadd2_rn(add2[(e >> 1) & 1], make_float2(exp2_neg(a.x), exp2_neg(a.y)));
            }
            l = l * exp2_neg(m - m_new) + ((add2[0].x + add2[0].y) + (add2[1].x + add2[1].y));
            m = m_new;
          }
        }
        if (p.S_dump && i < p.Tq) {
          const int j0 = kb * kAttK + c * 32;
          if (j0 < p.Tk) {  // Tk is a multiple of 32 when a copy is requested
            float v[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(acc[e]) * p.inv_kf_hd;
            uint32_t o[16];
            encode_vec<SCALIFY_BF16, 32>(v, o);
            uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(p.S_dump) + (dump_row + j0) * 2);
#pragma unroll
            for (int q = 0; q < 4; ++q) dst[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
          }
        }
      }
    }
    // the two threads of a row (one per half of the key columns) combine their maxima and sums
    float2* part = reinterpret_cast<float2*>(p_tiles);  // [2][128], the P tiles are not in use yet
    part[half * kAttQ + r] = make_float2(m, l);
    asm volatile("bar.sync 1, %0;" ::"n"(32 * kAttSmWarps) : "memory");
    {
      const float2 a = part[r], b = part[kAttQ + r];
      m = fmaxf(a.x, b.x);
      l = (a.x > -INFINITY ? a.y * exp2_neg(a.x - m) : 0.f) + (b.x > -INFINITY ? b.y * exp2_neg(b.x - m) : 0.f);
    }
    asm volatile("bar.sync 1, %0;" ::"n"(32 * kAttSmWarps) : "memory");  // the tile may be overwritten from here on
    const float inv_l = 1.0f / l;
    // positive scale: the division by l moves into the exponent, p = 2^(r * sc3 - (m + log2 l)) in one
    // multiply-add and one exp2 per element (log2 to 2^-22 absolute: far finer than the E4M3 result)
    const float m_l = m + __log2f(l);
    // sweep B: probabilities -> E4M3 -> shared memory (A operand of P V)
    for (int kb = 0; kb < n_kb && !timed_out; ++kb, ++it) {
      if (!mbar_wait(s_full, it & 1, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      // P V of the block that used this probability tile last (two blocks ago) must have read it
      const int pb = kb & 1;
      if (kb >= 2 && !mbar_wait(p_empty + 8 * pb, ((kb >> 1) - 1) & 1, abort_flag)) { timed_out = true; break; }
      uint32_t acc[32];
#pragma unroll 1
      for (int c = c_first; c < c_first + kChunks; ++c) {
        tmem_ld32(t_row + c * 32, acc);
        tmem_ld_wait();
        if (c == c_first + kChunks - 1) {
          // the score block is in registers: hand the TMEM buffer back now (as in sweep A)
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(s_empty);
        }
        float pr[32];
        if (pos_scale) {
          float2 r2[16];
          chunk_rounded(acc, kb * kAttK + c * 32, r2);
          const float2 nml2 = make_float2(-m_l, -m_l);
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            const float2 a = __ffma2_rn(r2[k], sc3_2, nml2);
            pr[2 * k] = exp2_neg(a.x);
            pr[2 * k + 1] = exp2_neg(a.y);
          }
        } else {
          chunk_scores(acc, kb * kAttK + c * 32, pr);
          const float2 nm2 = make_float2(-m, -m), il2 = make_float2(inv_l, inv_l);
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float2 a = __fadd2_rn(make_float2(pr[e], pr[e + 1]), nm2);
            const float2 q = __fmul2_rn(make_float2(exp2_neg(a.x), exp2_neg(a.y)), il2);
            pr[e] = q.x;
            pr[e + 1] = q.y;
          }
        }
        uint32_t o[8];
        encode_vec<SCALIFY_E4M3, 32>(pr, o);
        // row r of the tile: 128 bytes = eight 16-byte pieces, piece index XOR (r % 8) (128-byte swizzle)
        uint4* row = reinterpret_cast<uint4*>(p_tiles + pb * (kAttQ * kAttK) + r * 128);
        row[(2 * c) ^ (r & 7)] = make_uint4(o[0], o[1], o[2], o[3]);
        row[(2 * c + 1) ^ (r & 7)] = make_uint4(o[4], o[5], o[6], o[7]);
        if (p.P_dump && i < p.Tq) {
          const int j0 = kb * kAttK + c * 32;
          if (j0 < p.Tk) {
            uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(p.P_dump) + dump_row + j0);
            dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full + 8 * pb);
    }
    // O: 64 fp32 columns of this row
    if (!timed_out && mbar_wait(o_full, 0u, abort_flag)) {
      tc_fence_after();
      constexpr int OSZ = ElemBytes<ODT>::v;
#pragma unroll 1
      for (int c = half; c < 2 * NH; c += 2) {  // 32 of the row's 64 * NH columns at a time
        uint32_t acc[32];
        tmem_ld32(t_row + kAttOCol + c * 32, acc);
        tmem_ld_wait();
        if (i < p.Tq) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(acc[e]) * p.inv_kf_tk;
          uint32_t o[32 * OSZ / 4];
          encode_vec<ODT, 32>(v, o);
          uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(p.O) +
                                                (static_cast<long long>(bb) * p.o_bs + static_cast<long long>(hh) * p.o_hs +
                                                 static_cast<long long>(i) * p.o_ld +
                                                 c * 32) * OSZ);
#pragma unroll
          for (int q = 0; q < 32 * OSZ / 16; ++q) dst[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
        }
      }
    } else {
      timed_out = true;
    }
  }

  if (timed_out && p.status) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_TIMEOUT));
  tc_fence_before();
  __syncthreads();
  if (warp == kAttSmWarps) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kAttTmemCols);
  }
}

int launch_attention(const AttentionArgs& a, cudaStream_t st) {
  CUtensorMap map_q, map_k, map_v;
  int rc = make_byte_map4(&map_q, a.Q, a.hd, a.Tq, a.heads, a.batch, a.q_ld, a.q_hs, a.q_bs, kAttHd, kAttQ);
  if (rc) return rc;
  rc = make_byte_map4(&map_k, a.K, a.hd, a.Tk, a.heads, a.batch, a.k_ld, a.k_hs, a.k_bs, kAttHd, kAttK);
  if (rc) return rc;
  rc = make_byte_map4(&map_v, a.V, a.hd, a.Tk, a.heads, a.batch, a.v_ld, a.v_hs, a.v_bs, kAttHd, kAttK);
  if (rc) return rc;
  AttParams p;
  p.heads = a.heads * a.batch; p.h_inner = a.heads; p.Tq = a.Tq; p.Tk = a.Tk;
  p.q_blocks = (a.Tq + kAttQ - 1) / kAttQ;
  p.causal = a.causal;
  p.inv_kf_hd = 1.0f / kfactor(a.hd);
  p.kf_tk = kfactor(a.Tk);
  p.inv_kf_tk = 1.0f / p.kf_tk;
  p.O = a.O; p.o_ld = a.o_ld; p.o_hs = a.o_hs; p.o_bs = a.o_bs;
  p.S_dump = a.S_dump; p.P_dump = a.P_dump;
  p.v_scale = a.v_scale; p.o_scale = a.o_scale;
  p.status = a.status;
  // scores: D fp32, A = Q, B = K (both K-major), N = 128, M = 128
  p.idesc_s = (1u << 4) | (uint32_t(a.q_dt == SCALIFY_E5M2) << 7) | (uint32_t(a.k_dt == SCALIFY_E5M2) << 10) |
              (uint32_t(kAttK >> 3) << 17) | (uint32_t(kAttQ >> 4) << 24);
  // P V: A = P (E4M3, K-major), B = V (MN-major: keys are the contraction), N = 64, M = 128
  p.idesc_pv = (1u << 4) | (uint32_t(a.v_dt == SCALIFY_E5M2) << 10) | (1u << 16) | (uint32_t(kAttHd >> 3) << 17) |
               (uint32_t(kAttQ >> 4) << 24);
  p.q_scale = a.q_scale; p.k_scale = a.k_scale;
  // kf(hd) and a power-of-two c only shift the exponent; the product with log2(e) rounds once, as in the
  // stand-alone softmax kernel
  p.sc_const = kfactor(a.hd) * a.sm_scale * 1.4426950408889634f;
  const long long ctas = static_cast<long long>(p.heads) * p.q_blocks;
  if (ctas > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
#define SCALIFY_ATT_LAUNCH(NH)                                                                                   \
  do {                                                                                                           \
    auto kernel = attention_fwd_kernel<ODT, NH>;                                                                 \
    static DeviceOnce once; /* one per instantiation: the attribute belongs to this kernel on this device */     \
    int rc_once = device_once(once, nullptr, [&](int*) {                                                         \
      SCALIFY_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,                 \
                                            int(att_smem(NH))));                                                 \
      return int(SCALIFY_OK);                                                                                    \
    });                                                                                                          \
    if (rc_once) return rc_once;                                                                                 \
    kernel<<<static_cast<unsigned>(ctas), kAttThreads, att_smem(NH), st>>>(map_q, map_k, map_v, p);              \
  } while (0)
  SCALIFY_DISPATCH_WIDE(a.o_dt, ODT, {
    if (a.hd == 64) SCALIFY_ATT_LAUNCH(1);
    else SCALIFY_ATT_LAUNCH(2);
  });
#undef SCALIFY_ATT_LAUNCH
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

}  // namespace scalify
