// Fused scaled attention backward (Section 3.2.1: attention is a place for a custom scale rule; the
// rule is the composition of the calls the unfused path makes).  With the probabilities P the forward
// pass used (E4M3, scale 1) and the gradient dO of its output:
//   dP = dO V^T          scaled FP8 matmul:  dP_s = dO_s V_s kf(hd),  dP_d = bf16(acc / kf(hd))
//   dS = P (dP - delta)  softmax backward on the data components, delta_i = sum_j dP_d[i,j] P_d[i,j];
//                        rounded to E5M2,  dS_s = dP_s P_s c   (c = the forward's power-of-two scalar)
//   dQ = dS K            scaled FP8 matmul:  dQ_s = dS_s K_s kf(Tk),  dQ_d = acc / kf(Tk)
//   dK = dS^T Q          scaled FP8 matmul:  dK_s = dS_s Q_s kf(Tq),  dK_d = acc / kf(Tq)
//   dV = P^T dO          scaled FP8 matmul:  dV_s = P_s dO_s kf(Tq),  dV_d = acc / kf(Tq)
// in two launches.  dP never reaches HBM; dS is written once (one byte per score) because the second
// launch contracts it over the queries.
//
// Launch 1, one CTA per (head, block of 128 queries), 288 threads, laid out like the forward kernel:
//   warps 0-7   two threads per query row (each takes 64 of a block's 128 keys): sweep A reads the dP block
//               from TMEM and the P tile from shared memory and accumulates delta; sweep B recomputes dP,
//               forms dS, rounds it to E5M2 and writes it as the A operand of dS K (128-byte swizzle) and to HBM
//   warp 8      one thread: TMA loads (dO once; V, P and in sweep B also K per key block) and all tcgen05.mma
//   TMEM: 128 columns of dP + 64 columns of dQ.
// Launch 2, one CTA per (head, block of 128 keys), 192 threads: a two-slot TMA ring of (P, dS, dO, Q) tiles,
// 64 queries each, over the queries that see the key block; P^T dO and dS^T Q read the P and dS tiles MN-major (the
// queries are the contraction), so no transposed copy exists; dV and dK accumulate in TMEM (64 columns
// each) and are read out once.
// Every mbarrier wait is bounded; on expiry the CTA records SCALIFY_DEV_TIMEOUT and leaves.
#include <cuda.h>

#include "scalify_common.cuh"
#include "scalify_launch.h"
#include "tcgen05_ptx.cuh"

namespace scalify {

constexpr int kBwQ = 128;      // queries per block
constexpr int kBwK = 128;      // keys per block
constexpr int kBwHd = 64;      // bytes per row of a Q, K, V or dO tile: a head dimension of 128 travels as two such tiles
constexpr int kBwTile = kBwK * kBwHd;        // 8 KB: one column half of a Q, K, V or dO tile
constexpr int kBwPTile = kBwQ * kBwK;        // 16 KB: a P or dS tile
constexpr int kBwSmWarps = 8;
constexpr int kBw1Threads = 32 * (kBwSmWarps + 1);
// NH = head dimension / 64 column halves per tile
__host__ __device__ constexpr int bw1_slot(int nh) { return 2 * nh * kBwTile + kBwPTile; }  // V, K, P of one key block
__host__ __device__ constexpr size_t bw1_smem(int nh) { return size_t(nh) * kBwTile + 2 * bw1_slot(nh) + kBwPTile + 1024 + 256; }
constexpr int kBw1TmemCols = 256;
constexpr uint32_t kBw1DqCol = 128;

struct AttBwdParams {
  int heads, h_inner, Tq, Tk, q_blocks, k_blocks;   // heads = batch x h_inner
  int causal;
  float inv_kf_hd, inv_kf_tk, inv_kf_tq;
  float kf_hd, kf_tk, kf_tq, sm_scale;
  uint32_t idesc_dp, idesc_dq, idesc_dv, idesc_dk;
  const float* q_scale; const float* k_scale; const float* v_scale; const float* p_scale; const float* do_scale;
  float* ds_scale; float* dq_scale; float* dk_scale; float* dv_scale;
  void* dS; void* dP_dump;
  void* dQ; long long dq_ld, dq_hs, dq_bs;
  void* dK; long long dk_ld, dk_hs, dk_bs;
  void* dV; long long dv_ld, dv_hs, dv_bs;
  uint32_t* status;
};

// 64-byte-swizzle shared-memory matrix descriptor (layout type 4): K-major tile of 64-byte rows
// (8-row atoms 512 B apart) or MN-major tile whose 64 MN-elements are one row (8 K-rows per atom).
__device__ __forceinline__ uint64_t bw_desc_sw64(uint32_t saddr, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= 4ull << 61;
  return d;
}

// Four E4M3 values of a word -> fp32: one conversion to two packed halves per pair (exact: E4M3 is a subset of
// FP16, subnormals included) and one widening per element - 1.5 instructions per element on the otherwise idle
// conversion path, against a shift, a mask and a multiply each with integer arithmetic.
__device__ __forceinline__ void e4m3x4_to_float(uint32_t w, float* f) {
  const float2 a = fp8x2_to_float2(w, 0);
  const float2 b = fp8x2_to_float2(w >> 16, 0);
  f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
}

// Two fp32 accumulators -> their BF16 roundings (round to nearest even, one conversion instruction for
// the pair: that pipe is idle in these kernels; the forward kernel's fp32 forms measured 90 us (scalar) and
// 86.6 us (two-wide), alternating the two 85.1 us, against 84.7 us here), widened back to fp32
__device__ __forceinline__ void bf16_round_pair(uint32_t a_bits, uint32_t b_bits, float& a, float& b) {
  uint32_t packed;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(packed) : "f"(__uint_as_float(b_bits)), "f"(__uint_as_float(a_bits)));
  a = __uint_as_float(packed << 16);
  b = __uint_as_float(packed & 0xFFFF0000u);
}

template <int GDT, int NH>
__global__ void __launch_bounds__(kBw1Threads, 2)
attention_bwd_dq_kernel(const __grid_constant__ CUtensorMap map_do, const __grid_constant__ CUtensorMap map_v,
                        const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_p,
                        const AttBwdParams p) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  constexpr int kTile = NH * kBwTile;         // a dO, V or K tile: NH column halves of [128 rows][64 B]
  constexpr int kBw1Slot = bw1_slot(NH);
  const uint32_t smem_do = base;
  const uint32_t smem_slot = base + kTile;                       // 2 slots: [V | K | P 16 KB]
  const uint32_t smem_ds = base + kTile + 2 * kBw1Slot;          // 16 KB, 1024-byte aligned
  uint8_t* slot_mem = smem + kTile;
  uint8_t* ds_tile = smem + kTile + 2 * kBw1Slot;
  uint8_t* bar_mem = ds_tile + kBwPTile;
  const uint32_t bars = smem_ds + kBwPTile;
  const uint32_t do_full = bars, kv_full = bars + 8 /*2*/, kv_empty = bars + 24 /*2*/, s_full = bars + 40,
                 s_empty = bars + 48, p_full = bars + 56, p_empty = bars + 64, o_full = bars + 72;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_mem + 80);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // long (late) query blocks first, as in the forward kernel
  const int qb = p.q_blocks - 1 - static_cast<int>(blockIdx.x / p.heads), head = blockIdx.x % p.heads;
  const int hh = head % p.h_inner, bb = head / p.h_inner;  // head inside its batch element, batch element
  const int q0 = qb * kBwQ;
  const int shift = p.Tk - p.Tq;  // causal: query i sees keys j <= i + shift
  int n_kb = p.k_blocks;
  if (p.causal) n_kb = min(n_kb, (q0 + kBwQ - 1 + shift) / kBwK + 1);

  if (threadIdx.x == 0) {
    mbar_init(do_full, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(kv_full + 8 * s, 1); mbar_init(kv_empty + 8 * s, 1 + kBwSmWarps); }
    mbar_init(s_full, 1);
    mbar_init(s_empty, kBwSmWarps);
    mbar_init(p_full, kBwSmWarps);
    mbar_init(p_empty, 1);
    mbar_init(o_full, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (blockIdx.x == 0) {
      const float dos = load_scale(p.do_scale), vs = load_scale(p.v_scale), ps = load_scale(p.p_scale),
                  ks = load_scale(p.k_scale);
      const float dss = dos * vs * p.kf_hd * ps * p.sm_scale;
      if (p.ds_scale) *p.ds_scale = dss;
      if (p.dq_scale) *p.dq_scale = dss * ks * p.kf_tk;
      if (!(is_pow2_scale(dos) && is_pow2_scale(vs) && is_pow2_scale(ps) && is_pow2_scale(ks)) && p.status)
        atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
    }
  }
  if (warp == kBwSmWarps) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kBw1TmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool timed_out = false;

  if (warp == kBwSmWarps) {
    // ------------------------------------------------------------ loads and MMAs (one thread)
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_do)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_v)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_k)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_p)) : "memory");
      const int n_it = 2 * n_kb;  // sweep A (V, P), sweep B (V, K, P)
      auto issue_load = [&](int it) {
        const int slot = it & 1, use = it >> 1;
        if (use >= 1 && !mbar_wait(kv_empty + 8 * slot, (use - 1) & 1, abort_flag)) { timed_out = true; return; }
        const bool sweep_b = it >= n_kb;
        const int kb = sweep_b ? it - n_kb : it;
        const uint32_t fb = kv_full + 8 * slot;
        const uint32_t s0 = smem_slot + slot * kBw1Slot;
        mbar_expect_tx(fb, (sweep_b ? 2 * kTile : kTile) + kBwPTile);
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          tma_load_4d(s0 + h * kBwTile, &map_v, fb, h * kBwHd, kb * kBwK, hh, bb);
          if (sweep_b) tma_load_4d(s0 + kTile + h * kBwTile, &map_k, fb, h * kBwHd, kb * kBwK, hh, bb);
        }
        tma_load_3d(s0 + 2 * kTile, &map_p, fb, kb * kBwK, q0, head);
      };
      mbar_expect_tx(do_full, kTile);
#pragma unroll
      for (int h = 0; h < NH; ++h) tma_load_4d(smem_do + h * kBwTile, &map_do, do_full, h * kBwHd, q0, hh, bb);
      issue_load(0);
      if (!timed_out && !mbar_wait(do_full, 0u, abort_flag)) timed_out = true;
      const uint64_t do_desc = bw_desc_sw64(smem_do, 512u);
      const uint64_t ds_desc = make_smem_desc(smem_ds, 0u, 1024u);
      for (int it = 0; it < n_it && !timed_out; ++it) {
        if (it + 1 < n_it) { issue_load(it + 1); if (timed_out) break; }
        const int slot = it & 1;
        if (!mbar_wait(kv_full + 8 * slot, (it >> 1) & 1, abort_flag)) { timed_out = true; break; }
        // the dP block in TMEM is free once the row threads have read the previous one
        if (it >= 1 && !mbar_wait(s_empty, (it - 1) & 1, abort_flag)) { timed_out = true; break; }
        tc_fence_after();
        const uint32_t s0 = smem_slot + slot * kBw1Slot;
        const uint64_t v_desc = bw_desc_sw64(s0, 512u);
#pragma unroll
        for (int h = 0; h < NH; ++h)  // dP = dO V^T over the column halves ...
#pragma unroll
          for (int k = 0; k < kBwHd / 32; ++k)  // ... both operands K-major, 32 bytes of hd per MMA
            umma_f8(tmem_base, do_desc + static_cast<uint64_t>(h * (kBwTile >> 4) + k * 2),
                    v_desc + static_cast<uint64_t>(h * (kBwTile >> 4) + k * 2), p.idesc_dp, (h | k) != 0 ? 1u : 0u);
        umma_commit(s_full);
        if (it < n_kb) {
          umma_commit(kv_empty + 8 * slot);  // sweep A: V is free after dO V^T (P: the row threads arrive)
        } else {
          const int b = it - n_kb;
          if (!mbar_wait(p_full, b & 1, abort_flag)) { timed_out = true; break; }
          tc_fence_after();
          // K tile [128 keys][64 B]: the B operand in MN-major form (keys are the contraction), 32 keys per MMA
          const uint64_t k_desc = bw_desc_sw64(s0 + kTile, 512u);
#pragma unroll
          for (int h = 0; h < NH; ++h)  // 64 columns of dQ per column half of K
#pragma unroll
            for (int k = 0; k < kBwK / 32; ++k)
              umma_f8(tmem_base + kBw1DqCol + h * kBwHd, ds_desc + static_cast<uint64_t>(k * 2),
                      k_desc + static_cast<uint64_t>(h * (kBwTile >> 4) + k * (32 * kBwHd / 16)), p.idesc_dq,
                      (b | k) != 0 ? 1u : 0u);
          umma_commit(p_empty);
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
    // ------------------------------------------------------------ query rows (two threads per row)
    const int quarter = warp & 3, half = warp >> 2;   // TMEM lane quarter; which 64 of a block's 128 keys
    const int r = quarter * 32 + lane;
    const int i = q0 + r;                     // query index
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    constexpr int kChunks = kBwK / 32 / 2;    // 32-key chunks per thread and block
    const int c_first = half * kChunks;
    const long long dump_row = (static_cast<long long>(head) * p.Tq + i) * p.Tk;
    // dP's data component: the accumulator rounded to BF16 and divided by kf(hd), a power of two, which
    // commutes with the rounding
    // this thread's 32 probabilities of chunk c: two 16-byte pieces of row r of the 128-byte-swizzled tile
    auto load_p = [&](const uint8_t* p_tile, int c, float* pf) {
      const uint4* row = reinterpret_cast<const uint4*>(p_tile + r * 128);
      const uint4 a = row[(2 * c) ^ (r & 7)], b = row[(2 * c + 1) ^ (r & 7)];
      e4m3x4_to_float(a.x, pf); e4m3x4_to_float(a.y, pf + 4); e4m3x4_to_float(a.z, pf + 8); e4m3x4_to_float(a.w, pf + 12);
      e4m3x4_to_float(b.x, pf + 16); e4m3x4_to_float(b.y, pf + 20); e4m3x4_to_float(b.z, pf + 24); e4m3x4_to_float(b.w, pf + 28);
    };
    float delta = 0.f;
    int it = 0;
    // sweep A: delta = sum over the keys of dP_d P_d
    for (int kb = 0; kb < n_kb; ++kb, ++it) {
      const int slot = it & 1;
      if (!mbar_wait(s_full, it & 1, abort_flag)) { timed_out = true; break; }
      if (!mbar_wait(kv_full + 8 * slot, (it >> 1) & 1, abort_flag)) { timed_out = true; break; }  // the P tile
      tc_fence_after();
      const uint8_t* p_tile = slot_mem + slot * kBw1Slot + 2 * kTile;
      uint32_t acc[32];
#pragma unroll 1
      for (int c = c_first; c < c_first + kChunks; ++c) {
        tmem_ld32(t_row + c * 32, acc);
        float pf[32];
        load_p(p_tile, c, pf);
        tmem_ld_wait();
        float2 d2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};  // four independent chains, two per instruction
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          float x0, x1;
          bf16_round_pair(acc[e], acc[e + 1], x0, x1);
          d2[(e >> 1) & 1] = __ffma2_rn(make_float2(x0, x1), make_float2(pf[e], pf[e + 1]), d2[(e >> 1) & 1]);
        }
        // (the division by kf(hd), a power of two, commutes with every rounding above: applied once per chunk)
        delta += ((d2[0].x + d2[0].y) + (d2[1].x + d2[1].y)) * p.inv_kf_hd;
        if (p.dP_dump && i < p.Tq) {
          const int j0 = kb * kBwK + c * 32;
          if (j0 < p.Tk) {  // Tk is a multiple of 32
            float v[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(acc[e]) * p.inv_kf_hd;
            uint32_t o[16];
            encode_vec<SCALIFY_BF16, 32>(v, o);
            uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(p.dP_dump) + (dump_row + j0) * 2);
#pragma unroll
            for (int q = 0; q < 4; ++q) dst[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { mbar_arrive(s_empty); mbar_arrive(kv_empty + 8 * slot); }
    }
    // the two threads of a row add their halves (always in the same order)
    float* part = reinterpret_cast<float*>(ds_tile);  // [2][128], the dS tile is not in use yet
    part[half * kBwQ + r] = delta;
    asm volatile("bar.sync 1, %0;" ::"n"(32 * kBwSmWarps) : "memory");
    delta = part[r] + part[kBwQ + r];
    asm volatile("bar.sync 1, %0;" ::"n"(32 * kBwSmWarps) : "memory");  // the tile may be overwritten from here on
    // sweep B: dS = P (dP - delta) -> E5M2 -> shared memory (A operand of dS K) and HBM
    for (int kb = 0; kb < n_kb && !timed_out; ++kb, ++it) {
      const int slot = it & 1;
      if (!mbar_wait(s_full, it & 1, abort_flag)) { timed_out = true; break; }
      if (!mbar_wait(kv_full + 8 * slot, (it >> 1) & 1, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      // the previous block's dS K must have read the tile before it is overwritten
      if (kb >= 1 && !mbar_wait(p_empty, (kb - 1) & 1, abort_flag)) { timed_out = true; break; }
      const uint8_t* p_tile = slot_mem + slot * kBw1Slot + 2 * kTile;
      uint32_t acc[32];
#pragma unroll 1
      for (int c = c_first; c < c_first + kChunks; ++c) {
        tmem_ld32(t_row + c * 32, acc);
        float pf[32];
        load_p(p_tile, c, pf);
        tmem_ld_wait();
        const float2 ik2 = make_float2(p.inv_kf_hd, p.inv_kf_hd), nd2 = make_float2(-delta, -delta);
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          float x0, x1;
          bf16_round_pair(acc[e], acc[e + 1], x0, x1);
          const float2 q = __fmul2_rn(make_float2(pf[e], pf[e + 1]), __ffma2_rn(make_float2(x0, x1), ik2, nd2));
          pf[e] = q.x;
          pf[e + 1] = q.y;
        }
        uint32_t o[8];
        encode_vec<SCALIFY_E5M2, 32>(pf, o);
        uint4* row = reinterpret_cast<uint4*>(ds_tile + r * 128);
        row[(2 * c) ^ (r & 7)] = make_uint4(o[0], o[1], o[2], o[3]);
        row[(2 * c + 1) ^ (r & 7)] = make_uint4(o[4], o[5], o[6], o[7]);
        if (i < p.Tq) {
          const int j0 = kb * kBwK + c * 32;
          if (j0 < p.Tk) {
            uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(p.dS) + dump_row + j0);
            dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { mbar_arrive(s_empty); mbar_arrive(p_full); mbar_arrive(kv_empty + 8 * slot); }
    }
    // dQ: 64 fp32 columns of this row, 32 per thread
    if (!timed_out && mbar_wait(o_full, 0u, abort_flag)) {
      tc_fence_after();
      constexpr int GSZ = ElemBytes<GDT>::v;
#pragma unroll 1
      for (int c = half; c < 2 * NH; c += 2) {  // 32 of the row's 64 * NH columns at a time
        uint32_t acc[32];
        tmem_ld32(t_row + kBw1DqCol + c * 32, acc);
        tmem_ld_wait();
        if (i < p.Tq) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(acc[e]) * p.inv_kf_tk;
          uint32_t o[32 * GSZ / 4];
          encode_vec<GDT, 32>(v, o);
          uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(p.dQ) +
                                                (static_cast<long long>(bb) * p.dq_bs + static_cast<long long>(hh) * p.dq_hs +
                                                 static_cast<long long>(i) * p.dq_ld +
                                                 c * 32) * GSZ);
#pragma unroll
          for (int q = 0; q < 32 * GSZ / 16; ++q) dst[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
        }
      }
    } else {
      timed_out = true;
    }
  }

  if (timed_out && p.status) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_TIMEOUT));
  tc_fence_before();
  __syncthreads();
  if (warp == kBwSmWarps) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kBw1TmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// launch 2: dV = P^T dO and dK = dS^T Q for one (head, block of 128 keys)
// ---------------------------------------------------------------------------------------------
constexpr int kBw2Threads = 192;   // warp 0: TMA, warp 1: MMA, warps 2-5: read-out
__host__ __device__ constexpr int bw2_stages(int nh) { return nh == 1 ? 2 : 3; }  // (a third slot for 128: at most two CTAs fit an SM then,
                                                              // as many as the 256 accumulator columns each allow)
constexpr int kBw2Q = 64;          // queries per ring slot: short slots, so that four CTAs fit an SM and their
                                   // prologues and read-outs overlap the others' loads
constexpr int kBw2PTile = kBw2Q * kBwK;    // 8 KB: 64 queries x 128 keys of P or dS
constexpr int kBw2Tile = kBw2Q * kBwHd;    // 4 KB: one column half of 64 rows of dO or Q
__host__ __device__ constexpr int bw2_stage(int nh) { return 2 * kBw2PTile + 2 * nh * kBw2Tile; }  // 24 KB / 32 KB
__host__ __device__ constexpr size_t bw2_smem(int nh) { return size_t(bw2_stages(nh)) * bw2_stage(nh) + 1024 + 256; }
// TMEM: dV in columns [0, 64 NH), dK in [64 NH, 128 NH)

template <int GDT, int NH>
__global__ void __launch_bounds__(kBw2Threads, 4)
attention_bwd_dkv_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_ds,
                         const __grid_constant__ CUtensorMap map_do, const __grid_constant__ CUtensorMap map_q,
                         const AttBwdParams p) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  constexpr int kBw2Stages = bw2_stages(NH), kBw2Stage = bw2_stage(NH), kBw2TmemCols = 128 * NH;
  constexpr int kTile2 = NH * kBw2Tile;  // a dO or Q tile of 64 rows: NH column halves
  uint8_t* bar_mem = smem + kBw2Stages * kBw2Stage;
  const uint32_t bars = base + kBw2Stages * kBw2Stage;
  const uint32_t full_bar = bars, empty_bar = bars + 8 * kBw2Stages, acc_full = bars + 16 * kBw2Stages;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_mem + 16 * kBw2Stages + 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // with a causal mask the early key blocks are seen by the most query blocks: they come first
  const int kb = static_cast<int>(blockIdx.x / p.heads), head = blockIdx.x % p.heads;
  const int hh = head % p.h_inner, bb = head / p.h_inner;
  const int shift = p.Tk - p.Tq;
  const int i_min = p.causal ? max(0, kb * kBwK - shift) / kBw2Q : 0;  // first 64-query step that sees a key of this block
  const int n_qb = (p.Tq + kBw2Q - 1) / kBw2Q - i_min;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kBw2Stages; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, 1); }
    mbar_init(acc_full, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (blockIdx.x == 0) {
      const float dss = load_scale(p.ds_scale), qs = load_scale(p.q_scale), ps = load_scale(p.p_scale),
                  dos = load_scale(p.do_scale);
      if (p.dk_scale) *p.dk_scale = dss * qs * p.kf_tq;
      if (p.dv_scale) *p.dv_scale = ps * dos * p.kf_tq;
      if (!is_pow2_scale(qs) && p.status) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
    }
  }
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kBw2TmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  bool timed_out = false;

  if (warp == 0) {
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_p)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_ds)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_do)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_q)) : "memory");
      for (int t = 0; t < n_qb; ++t) {
        const int stage = t % kBw2Stages, use = t / kBw2Stages;
        if (use >= 1 && !mbar_wait(empty_bar + 8 * stage, (use - 1) & 1, abort_flag)) { timed_out = true; break; }
        const uint32_t fb = full_bar + 8 * stage;
        const uint32_t s0 = base + stage * kBw2Stage;
        const int q0 = (i_min + t) * kBw2Q;
        mbar_expect_tx(fb, kBw2Stage);
        tma_load_3d(s0, &map_p, fb, kb * kBwK, q0, head);
        tma_load_3d(s0 + kBw2PTile, &map_ds, fb, kb * kBwK, q0, head);
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          tma_load_4d(s0 + 2 * kBw2PTile + h * kBw2Tile, &map_do, fb, h * kBwHd, q0, hh, bb);
          tma_load_4d(s0 + 2 * kBw2PTile + kTile2 + h * kBw2Tile, &map_q, fb, h * kBwHd, q0, hh, bb);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      for (int t = 0; t < n_qb; ++t) {
        const int stage = t % kBw2Stages, use = t / kBw2Stages;
        if (!mbar_wait(full_bar + 8 * stage, use & 1, abort_flag)) { timed_out = true; break; }
        tc_fence_after();
        const uint32_t s0 = base + stage * kBw2Stage;
        // P and dS tiles [64 queries][128 keys]: A operands in MN-major form (the keys are M, the queries the
        // contraction): 8-query atoms 1024 B apart, 32 queries (4096 B) per MMA.  dO and Q tiles [64 queries][64 B]:
        // B operands in MN-major form, 8-query atoms 512 B apart, 32 queries (2048 B) per MMA.
        const uint64_t p_desc = make_smem_desc(s0, 0u, 1024u);
        const uint64_t ds_desc = make_smem_desc(s0 + kBw2PTile, 0u, 1024u);
        const uint64_t do_desc = bw_desc_sw64(s0 + 2 * kBw2PTile, 512u);
        const uint64_t q_desc = bw_desc_sw64(s0 + 2 * kBw2PTile + kTile2, 512u);
#pragma unroll
        for (int h = 0; h < NH; ++h)  // 64 columns of dV per column half of dO
#pragma unroll
          for (int k = 0; k < kBw2Q / 32; ++k)
            umma_f8(tmem_base + h * kBwHd, p_desc + static_cast<uint64_t>(k * (32 * 128 / 16)),
                    do_desc + static_cast<uint64_t>(h * (kBw2Tile >> 4) + k * (32 * kBwHd / 16)), p.idesc_dv,
                    (t | k) != 0 ? 1u : 0u);
#pragma unroll
        for (int h = 0; h < NH; ++h)  // 64 columns of dK per column half of Q
#pragma unroll
          for (int k = 0; k < kBw2Q / 32; ++k)
            umma_f8(tmem_base + (NH + h) * kBwHd, ds_desc + static_cast<uint64_t>(k * (32 * 128 / 16)),
                    q_desc + static_cast<uint64_t>(h * (kBw2Tile >> 4) + k * (32 * kBwHd / 16)), p.idesc_dk,
                    (t | k) != 0 ? 1u : 0u);
        umma_commit(empty_bar + 8 * stage);
      }
      if (!timed_out) umma_commit(acc_full);
    }
  } else {
    // ------------------------------------------------------------ read-out: one key row per thread
    const int quarter = warp & 3;
    const int j = kb * kBwK + quarter * 32 + lane;  // key index
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
    if (mbar_wait(acc_full, 0u, abort_flag)) {
      tc_fence_after();
      constexpr int GSZ = ElemBytes<GDT>::v;
#pragma unroll 1
      for (int c = 0; c < 4 * NH; ++c) {  // dV: the first 64 NH columns, dK: the next 64 NH
        uint32_t acc[32];
        tmem_ld32(t_row + c * 32, acc);
        tmem_ld_wait();
        if (j < p.Tk) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(acc[e]) * p.inv_kf_tq;
          uint32_t o[32 * GSZ / 4];
          encode_vec<GDT, 32>(v, o);
          const bool is_dv = c < 2 * NH;
          char* out = is_dv ? static_cast<char*>(p.dV) : static_cast<char*>(p.dK);
          const long long hs = is_dv ? p.dv_hs : p.dk_hs, ld = is_dv ? p.dv_ld : p.dk_ld, bs = is_dv ? p.dv_bs : p.dk_bs;
          uint4* dst = reinterpret_cast<uint4*>(out + (static_cast<long long>(bb) * bs + static_cast<long long>(hh) * hs +
                                                       static_cast<long long>(j) * ld +
                                                       (c % (2 * NH)) * 32) * GSZ);
#pragma unroll
          for (int q = 0; q < 32 * GSZ / 16; ++q) dst[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
        }
      }
    } else {
      timed_out = true;
    }
  }

  if (timed_out && p.status) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_TIMEOUT));
  if (warp == 0 && lane == 0 && (timed_out || *abort_flag)) {
    // wait (bounded) for the copies still in flight before the CTA's shared memory goes away
    const unsigned long long t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) {}
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kBw2TmemCols);
  }
}

int launch_attention_bwd(const AttentionBwdArgs& a, cudaStream_t st) {
  CUtensorMap map_k, map_v, map_do, map_p;
  int rc;
  const int all_heads = a.heads * a.batch;
  if ((rc = make_byte_map4(&map_do, a.dO, a.hd, a.Tq, a.heads, a.batch, a.do_ld, a.do_hs, a.do_bs, kBwHd, kBwQ))) return rc;
  if ((rc = make_byte_map4(&map_k, a.K, a.hd, a.Tk, a.heads, a.batch, a.k_ld, a.k_hs, a.k_bs, kBwHd, kBwK))) return rc;
  if ((rc = make_byte_map4(&map_v, a.V, a.hd, a.Tk, a.heads, a.batch, a.v_ld, a.v_hs, a.v_bs, kBwHd, kBwK))) return rc;
  const uint64_t plane = static_cast<uint64_t>(a.Tq) * static_cast<uint64_t>(a.Tk);
  if ((rc = make_byte_map(&map_p, a.P, a.Tk, a.Tq, all_heads, a.Tk, plane, kBwK, kBwQ))) return rc;
  // launch 2 reads 64 queries per ring slot
  CUtensorMap map_p2, map_ds2, map_do2, map_q2;
  if ((rc = make_byte_map(&map_p2, a.P, a.Tk, a.Tq, all_heads, a.Tk, plane, kBwK, kBw2Q))) return rc;
  if ((rc = make_byte_map(&map_ds2, a.dS, a.Tk, a.Tq, all_heads, a.Tk, plane, kBwK, kBw2Q))) return rc;
  if ((rc = make_byte_map4(&map_do2, a.dO, a.hd, a.Tq, a.heads, a.batch, a.do_ld, a.do_hs, a.do_bs, kBwHd, kBw2Q))) return rc;
  if ((rc = make_byte_map4(&map_q2, a.Q, a.hd, a.Tq, a.heads, a.batch, a.q_ld, a.q_hs, a.q_bs, kBwHd, kBw2Q))) return rc;
  AttBwdParams p;
  p.heads = all_heads; p.h_inner = a.heads; p.Tq = a.Tq; p.Tk = a.Tk;
  p.q_blocks = (a.Tq + kBwQ - 1) / kBwQ;
  p.k_blocks = (a.Tk + kBwK - 1) / kBwK;
  p.causal = a.causal;
  p.kf_hd = kfactor(a.hd); p.kf_tk = kfactor(a.Tk); p.kf_tq = kfactor(a.Tq);
  p.inv_kf_hd = 1.0f / p.kf_hd; p.inv_kf_tk = 1.0f / p.kf_tk; p.inv_kf_tq = 1.0f / p.kf_tq;
  p.sm_scale = a.sm_scale;
  const uint32_t e5 = 1u;
  auto fmt = [](int dt) { return static_cast<uint32_t>(dt == SCALIFY_E5M2); };
  // dP = dO V^T: both K-major, N = 128, M = 128, fp32 accumulator
  p.idesc_dp = (1u << 4) | (fmt(a.do_dt) << 7) | (fmt(a.v_dt) << 10) | (uint32_t(kBwK >> 3) << 17) | (uint32_t(kBwQ >> 4) << 24);
  // dQ = dS K: A = dS (E5M2, K-major), B = K MN-major, N = 64
  p.idesc_dq = (1u << 4) | (e5 << 7) | (fmt(a.k_dt) << 10) | (1u << 16) | (uint32_t(kBwHd >> 3) << 17) | (uint32_t(kBwQ >> 4) << 24);
  // dV = P^T dO: A = P (E4M3) MN-major, B = dO MN-major, N = 64, M = 128 keys
  p.idesc_dv = (1u << 4) | (fmt(a.do_dt) << 10) | (1u << 15) | (1u << 16) | (uint32_t(kBwHd >> 3) << 17) | (uint32_t(kBwK >> 4) << 24);
  // dK = dS^T Q: A = dS (E5M2) MN-major, B = Q MN-major
  p.idesc_dk = (1u << 4) | (e5 << 7) | (fmt(a.q_dt) << 10) | (1u << 15) | (1u << 16) | (uint32_t(kBwHd >> 3) << 17) |
               (uint32_t(kBwK >> 4) << 24);
  p.q_scale = a.q_scale; p.k_scale = a.k_scale; p.v_scale = a.v_scale; p.p_scale = a.p_scale; p.do_scale = a.do_scale;
  p.ds_scale = a.ds_scale; p.dq_scale = a.dq_scale; p.dk_scale = a.dk_scale; p.dv_scale = a.dv_scale;
  p.dS = a.dS; p.dP_dump = a.dP_dump;
  p.dQ = a.dQ; p.dq_ld = a.dq_ld; p.dq_hs = a.dq_hs; p.dq_bs = a.dq_bs;
  p.dK = a.dK; p.dk_ld = a.dk_ld; p.dk_hs = a.dk_hs; p.dk_bs = a.dk_bs;
  p.dV = a.dV; p.dv_ld = a.dv_ld; p.dv_hs = a.dv_hs; p.dv_bs = a.dv_bs;
  p.status = a.status;
  const long long ctas1 = static_cast<long long>(p.heads) * p.q_blocks, ctas2 = static_cast<long long>(p.heads) * p.k_blocks;
  if (ctas1 > 0x7FFFFFFF || ctas2 > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
#define SCALIFY_ATT_BWD_LAUNCH(NH)                                                                               \
  do {                                                                                                           \
    auto k1 = attention_bwd_dq_kernel<GDT, NH>;                                                                  \
    auto k2 = attention_bwd_dkv_kernel<GDT, NH>;                                                                 \
    static DeviceOnce once; /* one per instantiation: the attributes belong to these kernels on this device */   \
    int rc_once = device_once(once, nullptr, [&](int*) {                                                         \
      SCALIFY_CUDA_TRY(cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bw1_smem(NH)))); \
      SCALIFY_CUDA_TRY(cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bw2_smem(NH)))); \
      return int(SCALIFY_OK);                                                                                    \
    });                                                                                                          \
    if (rc_once) return rc_once;                                                                                 \
    k1<<<static_cast<unsigned>(ctas1), kBw1Threads, bw1_smem(NH), st>>>(map_do, map_v, map_k, map_p, p);         \
    SCALIFY_CUDA_TRY(cudaGetLastError());                                                                        \
    k2<<<static_cast<unsigned>(ctas2), kBw2Threads, bw2_smem(NH), st>>>(map_p2, map_ds2, map_do2, map_q2, p);    \
  } while (0)
  SCALIFY_DISPATCH_WIDE(a.g_dt, GDT, {
    if (a.hd == 64) SCALIFY_ATT_BWD_LAUNCH(1);
    else SCALIFY_ATT_BWD_LAUNCH(2);
  });
#undef SCALIFY_ATT_BWD_LAUNCH
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

}  // namespace scalify
