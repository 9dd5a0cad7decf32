// Scaled FP8 matmul for sm_100a (Section 3.2 matmul rule; Appendix A mixed E4M3/E5M2 operands,
// higher-precision output):  Y_d = (op(A)_d . op(B)_d) / kf(K),  Y_s = A_s * B_s * kf(K).
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0      TMA producer: cp.async.bulk.tensor tiles of A and B into a kStages-deep ring of
//               128-byte-swizzled shared-memory buffers, completion on mbarriers
//   warp 1      MMA issuer: one thread issues tcgen05.mma (kind::f8f6f4, fp32 accumulate) from
//               shared-memory descriptors into a TMEM accumulator; tcgen05.commit releases ring
//               slots and publishes finished accumulators
//   warps 2-9   epilogue: tcgen05.ld of the accumulator (two accumulators of 256 TMEM columns, so
//               the epilogue of tile i overlaps the main loop of tile i+1), multiply by the exact
//               power of two 1/kf(K), round once to the output type, 16-byte stores, and the
//               statistic of the stored values (AMAX: warp-shuffle max + one atomicMax on the
//               fp32 bit pattern per warp; L2: per-warp partial sums in fixed slots)
// Tile 128 x 256 x 128 (one 128-byte swizzle row of FP8 per K block, four K=32 MMAs per block).
// Operands may be K-major (row-major [rows, K]) or MN-major (row-major [K, rows]); the layout is
// expressed in the shared-memory descriptors and the instruction descriptor, not by copying.
// Every wait on an mbarrier is bounded; on expiry the CTA records SCALIFY_DEV_TIMEOUT, drains
// its own copies in flight, frees its TMEM and returns.
#include <cuda.h>
#include <string.h>

#include <mutex>

#include "scalify_common.cuh"
#include "scalify_launch.h"
#include "tcgen05_ptx.cuh"

namespace scalify {

constexpr int kBM = 128;   // rows of the output tile per CTA
constexpr int kBN = 256;   // columns of the output tile
constexpr int kBK = 128;   // FP8 elements = bytes per K block (one 128-byte swizzle row)
constexpr int kUmmaK = 32;
constexpr int kAccStages = 2;
constexpr int kEpiWarps = 8;                 // two warps per TMEM lane quarter, each taking half of the columns
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;
constexpr int kTmemCols = kAccStages * kBN;  // 512
constexpr int kGroupM = 16;                  // m-tiles per rasterisation group
constexpr int kMxSfWarps = 4;                // block-scaled kernel: one warp per TMEM lane quarter writes the exponents
constexpr int kMxGemmThreads = kGemmThreads + 32 * kMxSfWarps;

// NCTA = 1: one CTA computes a 128 x 256 tile (tcgen05 cta_group::1).
// NCTA = 2: a cluster of two CTAs on an SM pair computes a 256 x 256 tile (cta_group::2): each
//           CTA stages its own 128 rows of A and its own 128-column half of B, the leader CTA
//           issues the MMAs, which read both CTAs' shared memory and write both CTAs' TMEM.
//           Per SM this halves the shared-memory traffic of B, the limiter of the 1-CTA form.
// MX: block-scaled operands (one E8M0 exponent per 32 elements of K, Section 2's block-scale
//     generalisation).  The MMAs read the exponents from tensor memory: TMEM holds ONE 256-column
//     accumulator and, behind it, one 16-column exponent buffer per ring slot (A: 4 columns, B: 8).
//     Four extra warps, one per TMEM lane quarter, read the exponent tiles of a K block (512 B for
//     the 128 rows of A, 2 x 512 B for the 256 rows of B) from L2, 16 bytes per lane, and write
//     them into the slot's buffer with tcgen05.st; they wait for the slot on the same "empty"
//     barrier as the TMA producer and arrive on the same "full" barrier as the TMA bytes, so the
//     MMA thread issues exactly what the per-tensor kernel's does.  In the two-CTA form every CTA
//     holds the exponents of its own 128 rows of A and of ALL 256 rows of B (each CTA multiplies
//     its rows of A with the whole B tile).
template <int NCTA, bool MX = false> struct GemmCfg {
  static constexpr int kTileM = kBM * NCTA;
  static constexpr int kBRows = kBN / NCTA;          // B rows (columns of the output) staged per CTA
  static constexpr int kABytes = kBM * kBK;          // 16 KB
  static constexpr int kBBytes = kBRows * kBK;       // 32 KB / 16 KB
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStages = NCTA == 1 ? 3 : 5;
  static constexpr int kAcc = MX ? 1 : kAccStages;   // accumulators in TMEM
  // Epilogue staging: 8 KB per warp = one tile (32 rows x 32 columns) per chunk of a 16-bit output, so that a
  // warp never waits for the TMA store of an earlier chunk of the same accumulator (two tiles for fp32 output).
  static constexpr int kEpiWarpBytes = 8192;
  static constexpr int kEpiBytes = kEpiWarps * kEpiWarpBytes;
  static constexpr size_t kSmem = size_t(kStages) * kStageBytes + kEpiBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};
// MX: TMEM columns of the exponents: one buffer of 16 columns per ring slot (A: 4 columns at +0, B: 8 columns at +4)
constexpr uint32_t kSfaTmemCol = 256;
constexpr uint32_t kMxSfCols = 16;

struct GemmParams {
  int M, N, K, batch;
  int tiles_m, tiles_n;
  int a_mn_major, b_mn_major;  // 0: K-major (row-major [rows,K]); 1: MN-major (row-major [K,rows])
  int b_batched;               // 0: one 2-D B shared by every batch
  uint32_t idesc;
  float alpha;                 // 1/kf(K)
  float kf;
  void* Y;
  long long ldy, y_batch_stride;  // elements
  const float* a_scale;
  const float* b_scale;
  float* y_scale;
  int stat;
  const float* stat_in;  // delayed rescale: statistic of an earlier step (device), or NULL
  // AMAX: every epilogue warp takes an atomicMax of the fp32 bit pattern on a scratch word; the CTA that
  // draws the last ticket moves the result to the statistic word and leaves scratch and ticket at zero for
  // the next launch.  Nothing is zeroed from the host and nothing depends on the launch's position in a
  // sequence, so a recorded launch can be replayed from a CUDA graph.
  float* stat_word;
  uint32_t* amax_scratch;
  uint32_t* ticket;
  double* l2_partials;   // L2: [tiles][4]
  uint32_t* status;
  // Speculative rescale (SPEC kernels): besides Y, the epilogue writes Yq = fp8(stored Y / r_pred) with
  // r_pred = p2_floor(*stat_hint); a later check compares r_pred with the power of two of the true statistic.
  const float* stat_hint;
  int q_dt;          // SCALIFY_E4M3 or SCALIFY_E5M2
  float* r_pred_out; // the r_pred this launch used (read by the check kernel)
  // FP8-only form (NOY kernels: no 16-bit intermediate is stored).  The CTA that draws the last ticket also
  // publishes what the check launch publishes otherwise: the FP8 output's scale word and the prediction for the
  // next call.  redo != 0 marks the repair launch that follows every such GEMM: its CTAs return at once when
  // the power of two of the statistic equals the predicted one, and otherwise compute the product again with
  // the statistic itself as the "prediction".
  float* yq_scale;
  float* hint_out;
  int redo;
  // BIAS kernels: Y = A B + bias by the add rule, rounded once: Y_s = max(A_s B_s kf(K), bias_s)
  const void* bias;  // [N], F16 / BF16 / F32
  int bias_dt;
  const float* bias_scale;
  // MX only: block exponents in tiles of 128 rows x 4 K-blocks (512 B each), tile (r, k) at
  // ((r * K/128) + k) * 512, byte (row % 32) * 16 + (row / 32 % 4) * 4 + (block % 4)
  const uint8_t* sfa;
  const uint8_t* sfb;
};

__device__ __forceinline__ void tile_coords(const GemmParams& p, int tile, int& b, int& mt, int& nt) {
  const int per_batch = p.tiles_m * p.tiles_n;
  b = tile / per_batch;
  const int t = tile - b * per_batch;
  const int group_sz = kGroupM * p.tiles_n;
  const int group = t / group_sz;
  const int first_m = group * kGroupM;
  const int gm = min(p.tiles_m - first_m, kGroupM);
  const int r = t - group * group_sz;
  mt = first_m + r % gm;
  nt = r / gm;
}

// map_sfa is the map of the speculative FP8 output in the SPEC form (map_sfb is not used).
template <int OUT, int NCTA, bool MX, bool SPEC = false, bool BIAS = false, bool NOY = false>
__device__ __forceinline__ void gemm_body(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_y,
                                          const CUtensorMap& map_sfa, const CUtensorMap& map_sfb, const GemmParams& p) {
  static_assert(!SPEC || (!MX && ElemBytes<OUT>::v == 2), "speculative FP8 output: per-tensor kernel, 16-bit Y");
  static_assert(!BIAS || (!MX && !SPEC), "bias: per-tensor kernel only");
  static_assert(!NOY || SPEC, "the FP8-only form is a speculative form");
  using C = GemmCfg<NCTA, MX>;
  constexpr int kStages = C::kStages;
  constexpr int kAcc = C::kAcc;
  if constexpr (NOY) {
    if (p.redo) {
      // repair launch: the GEMM before it has finished (and so has everything it wrote) once this returns
      asm volatile("griddepcontrol.wait;" ::: "memory");
      bool nf0;
      const float r_true = rescale_factor(*reinterpret_cast<const volatile float*>(p.stat_word), &nf0);
      if (r_true == *reinterpret_cast<const volatile float*>(p.r_pred_out)) return;  // the same words for every thread
    }
  }
  asm volatile("griddepcontrol.launch_dependents;");  // a dependent grid may set up while this one runs
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  const uint32_t smem_a = base;
  const uint32_t smem_b = base + kStages * C::kABytes;
  uint8_t* epi_mem = smem + kStages * C::kStageBytes;  // 8 KB per epilogue warp, 1024-byte aligned
  uint8_t* bar_mem = epi_mem + C::kEpiBytes;
  const uint32_t bars = base + kStages * C::kStageBytes + C::kEpiBytes;
  const uint32_t full_bar = bars;                         // kStages x 8 B
  const uint32_t empty_bar = bars + 8 * kStages;          // kStages x 8 B
  const uint32_t acc_full_bar = bars + 16 * kStages;      // kAccStages x 8 B
  const uint32_t acc_empty_bar = acc_full_bar + 8 * kAccStages;
  const uint32_t drain_bar = acc_empty_bar + 8 * kAccStages;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_mem + 16 * kStages + 16 * kAccStages + 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = (NCTA == 2) ? cluster_ctarank() : 0u;  // position in the CTA pair; 0 = leader
  const int unit = blockIdx.x / NCTA;                          // CTA (NCTA=1) or cluster (NCTA=2) index
  const int num_units = gridDim.x / NCTA;
  const int num_kb = (p.K + kBK - 1) / kBK;
  const int num_tiles = p.tiles_m * p.tiles_n * p.batch;

  if (threadIdx.x == 0) {
    // MX: besides the producer's arrival (with the byte count), one arrival per exponent warp of every CTA of the pair
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar + 8 * s, MX ? 1 + kMxSfWarps * NCTA : 1); mbar_init(empty_bar + 8 * s, 1); }
    for (int s = 0; s < kAccStages; ++s) {
      mbar_init(acc_full_bar + 8 * s, 1);
      mbar_init(acc_empty_bar + 8 * s, kEpiWarps * NCTA);  // one arrival per epilogue warp of every CTA of the pair
    }
    mbar_init(drain_bar, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
  tc_fence_before();
  __syncthreads();
  if constexpr (NCTA == 2) cluster_sync_all();  // the peer's barriers exist before anything signals them
  tc_fence_after();
  // Everything above touches no global memory: launched as a programmatic dependent, the grid may set up
  // while the kernel before it in the stream drains; from here on that kernel's writes are needed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x == 0) {
    if (blockIdx.x == 0) {
      float r = 1.0f;
      bool nf = false;
      // (volatile: the word may have been written by the grid this one depends on; a read-only-path load could be
      // scheduled above the wait)
      if (p.stat_in) r = rescale_factor(*reinterpret_cast<const volatile float*>(p.stat_in), &nf);
      float ys = load_scale_after_wait(p.a_scale) * load_scale_after_wait(p.b_scale) * p.kf * r;
      if constexpr (BIAS) ys = fmaxf(ys, load_scale_after_wait(p.bias_scale));  // add rule for powers of two
      if (p.y_scale) *p.y_scale = ys;
      if constexpr (SPEC) {
        bool nf2;
        if (!(NOY && p.redo)) *p.r_pred_out = rescale_factor(*reinterpret_cast<const volatile float*>(p.stat_hint), &nf2);
      }
      if (nf && p.status) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_NONFINITE_STAT));
    }
    if (blockIdx.x == 0 && p.status) {
      bool bad = !is_pow2_scale(load_scale_after_wait(p.a_scale)) || !is_pow2_scale(load_scale_after_wait(p.b_scale));
      if constexpr (BIAS) bad = bad || !is_pow2_scale(load_scale_after_wait(p.bias_scale));
      if (bad) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
    }
  }
  const uint32_t tmem_base = *tmem_slot;
  bool timed_out = false;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_y)) : "memory");
      uint32_t stage = 0, phase = 0;
      long long issued = 0;
      for (int tile = unit; tile < num_tiles && !timed_out; tile += num_units) {
        int b, mt, nt;
        tile_coords(p, tile, b, mt, nt);
        const int m0 = mt * C::kTileM + static_cast<int>(rank) * kBM;
        const int n0 = nt * kBN + static_cast<int>(rank) * C::kBRows * (NCTA - 1);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag)) { timed_out = true; break; }
          const int k0 = kb * kBK;
          const uint32_t sa = smem_a + stage * C::kABytes, sb = smem_b + stage * C::kBBytes;
          const int bb = p.b_batched ? b : 0;
          if constexpr (NCTA == 1) {
            const uint32_t fb = full_bar + 8 * stage;
            mbar_expect_tx(fb, C::kABytes + C::kBBytes);
            if (p.a_mn_major) tma_load_3d(sa, &map_a, fb, m0, k0, b);
            else tma_load_3d(sa, &map_a, fb, k0, m0, b);
            if (p.b_mn_major) {
              tma_load_3d(sb, &map_b, fb, n0, k0, bb);
              tma_load_3d(sb + kBK * 128, &map_b, fb, n0 + 128, k0, bb);
            } else {
              tma_load_3d(sb, &map_b, fb, k0, n0, bb);
            }
          } else {
            // both CTAs' copies are counted on the LEADER's full barrier, which expects the bytes of the pair
            const uint32_t fb = map_to_cta(full_bar + 8 * stage, 0u);
            if (rank == 0u) mbar_expect_tx(full_bar + 8 * stage, 2 * (C::kABytes + C::kBBytes));
            if (p.a_mn_major) tma_load_3d_pair(sa, &map_a, fb, m0, k0, b);
            else tma_load_3d_pair(sa, &map_a, fb, k0, m0, b);
            if (p.b_mn_major) tma_load_3d_pair(sb, &map_b, fb, n0, k0, bb);
            else tma_load_3d_pair(sb, &map_b, fb, k0, n0, bb);
          }
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if ((timed_out || *abort_flag) && rank == 0u) {
        // drain: every copy signals a full barrier of this CTA; wait (bounded) for the most recent use of
        // each ring slot so that no copy is in flight when the CTA (pair) exits
        const int pending = issued < kStages ? static_cast<int>(issued) : kStages;
        uint32_t s = stage, ph = phase;
        for (int i = 0; i < pending; ++i) {
          if (s == 0) { s = kStages - 1; ph ^= 1u; } else { --s; }
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(full_bar + 8 * s, ph) && global_timer_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0u) {
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      const uint32_t a_lbo = 0u, a_sbo = 1024u;
      const uint32_t b_lbo = (p.b_mn_major && NCTA == 1) ? kBK * 128u : 0u, b_sbo = 1024u;
      const uint32_t a_step = p.a_mn_major ? (kUmmaK * 128u) : kUmmaK;  // bytes per K=32 step
      const uint32_t b_step = p.b_mn_major ? (kUmmaK * 128u) : kUmmaK;
      // The issuing thread is alone on its scheduler slot and every instruction between two MMAs is exposed
      // latency, so everything that does not change is computed once: descriptors of ring slot 0 (a later
      // slot or K step only adds to the 14-bit address field, which cannot carry: shared memory ends below
      // 2^18 bytes), and the four instruction descriptors of a K block.
      const uint64_t a_desc0 = make_smem_desc(smem_a, a_lbo, a_sbo);
      const uint64_t b_desc0 = make_smem_desc(smem_b, b_lbo, b_sbo);
      constexpr uint32_t kAStageInc = C::kABytes >> 4, kBStageInc = C::kBBytes >> 4;
      const uint32_t a_k_inc = a_step >> 4, b_k_inc = b_step >> 4;
      uint32_t idesc_k[kBK / kUmmaK];
#pragma unroll
      for (int k = 0; k < kBK / kUmmaK; ++k)  // MX: scale-factor ids = exponent byte k of each row's word (bits 29-30: A, 4-5: B)
        idesc_k[k] = MX ? (p.idesc | (uint32_t(k) << 29) | (uint32_t(k) << 4)) : p.idesc;
      for (int tile = unit; tile < num_tiles && !timed_out; tile += num_units) {
        if (!mbar_wait(acc_empty_bar + 8 * acc, acc_phase ^ 1u, abort_flag)) { timed_out = true; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kBN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag)) { timed_out = true; break; }
          tc_fence_after();
          const uint64_t ad0 = a_desc0 + static_cast<uint64_t>(stage * kAStageInc);
          const uint64_t bd0 = b_desc0 + static_cast<uint64_t>(stage * kBStageInc);
          // MX: the slot's exponents are in tensor memory (the "full" barrier also counts the exponent warps)
          const uint32_t sf_col = tmem_base + kSfaTmemCol + stage * kMxSfCols;
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            const uint64_t ad = ad0 + static_cast<uint64_t>(k * a_k_inc);
            const uint64_t bd = bd0 + static_cast<uint64_t>(k * b_k_inc);
            const uint32_t accumulate = (kb | k) != 0 ? 1u : 0u;
            if constexpr (MX) {
              if constexpr (NCTA == 1) umma_mxf8(d_tmem, ad, bd, idesc_k[k], accumulate, sf_col, sf_col + 4);
              else umma_mxf8_pair(d_tmem, ad, bd, idesc_k[k], accumulate, sf_col, sf_col + 4);
            } else if constexpr (NCTA == 1) {
              umma_f8(d_tmem, ad, bd, idesc_k[k], accumulate);
            } else {
              umma_f8_pair(d_tmem, ad, bd, idesc_k[k], accumulate);
            }
          }
          // slot free (in both CTAs) once these MMAs have read it
          if constexpr (NCTA == 1) umma_commit(empty_bar + 8 * stage);
          else umma_commit_pair(empty_bar + 8 * stage);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (timed_out) break;
        // accumulator complete (in both CTAs)
        if constexpr (NCTA == 1) umma_commit(acc_full_bar + 8 * acc);
        else umma_commit_pair(acc_full_bar + 8 * acc);
        if (++acc == kAcc) { acc = 0; acc_phase ^= 1u; }
      }
      if (timed_out || *abort_flag) {
        // all MMAs issued so far must retire before TMEM is freed
        if constexpr (NCTA == 1) umma_commit(drain_bar);
        else umma_commit_pair(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0u) && global_timer_ns() - t0 < kWaitLimitNs) {}
      }
    }
  } else if (MX && warp >= 2 + kEpiWarps) {
    // ---------------------------------------------------------------- exponent warps (block-scaled kernel)
    // One warp per TMEM lane quarter.  A 512-byte exponent tile is 16 bytes per row % 32 (byte (row / 32) * 4 +
    // block), which is what lane (row % 32) of EVERY quarter must hold in four consecutive columns: each warp
    // reads the tile with one 16-byte load per lane (from L2: the four warps and the peer CTA read the same
    // bytes) and stores it into its own quarter of the ring slot's exponent buffer.  The loads of the next three
    // K blocks are in flight while the current three are stored.
    const int q = warp & 3;
    const uint32_t t_sf = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + kSfaTmemCol;
    uint32_t stage = 0, phase = 0;
    for (int tile = unit; tile < num_tiles && !timed_out; tile += num_units) {
      int b, mt, nt;
      tile_coords(p, tile, b, mt, nt);
      const uint4* ta = reinterpret_cast<const uint4*>(p.sfa) +
                        (static_cast<size_t>(NCTA == 2 ? 2 * mt + static_cast<int>(rank) : mt) * num_kb) * 32 + lane;
      const uint4* tb0 = reinterpret_cast<const uint4*>(p.sfb) + (static_cast<size_t>(2 * nt) * num_kb) * 32 + lane;
      const uint4* tb1 = reinterpret_cast<const uint4*>(p.sfb) + (static_cast<size_t>(2 * nt + 1) * num_kb) * 32 + lane;
      constexpr int kG = 3;  // K blocks per group of loads (registers: two groups of 12 per block)
      uint4 va[kG], vb0[kG], vb1[kG], na[kG], nb0[kG], nb1[kG];
      auto load_group = [&](int kb0, uint4 (&xa)[kG], uint4 (&xb0)[kG], uint4 (&xb1)[kG]) {
#pragma unroll
        for (int j = 0; j < kG; ++j) {
          if (kb0 + j < num_kb) {
            ld_raw<16>(ta + (kb0 + j) * 32, reinterpret_cast<uint32_t*>(&xa[j]));
            ld_raw<16>(tb0 + (kb0 + j) * 32, reinterpret_cast<uint32_t*>(&xb0[j]));
            ld_raw<16>(tb1 + (kb0 + j) * 32, reinterpret_cast<uint32_t*>(&xb1[j]));
          }
        }
      };
      load_group(0, va, vb0, vb1);
      for (int kb0 = 0; kb0 < num_kb && !timed_out; kb0 += kG) {
        if (kb0 + kG < num_kb) load_group(kb0 + kG, na, nb0, nb1);
#pragma unroll
        for (int j = 0; j < kG; ++j) {
          if (kb0 + j < num_kb && !timed_out) {
            // the MMAs that read this slot (operands and exponents) one ring revolution ago have completed
            if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag)) {
              timed_out = true;
            } else {
              tc_fence_after();
              const uint32_t col = t_sf + stage * kMxSfCols;
              tmem_st4(col, va[j]);
              tmem_st4(col + 4u, vb0[j]);
              tmem_st4(col + 8u, vb1[j]);
              tmem_st_wait();
              tc_fence_before();
              __syncwarp();
              if (lane == 0) {
                if constexpr (NCTA == 1) mbar_arrive(full_bar + 8 * stage);
                else mbar_arrive_cluster(map_to_cta(full_bar + 8 * stage, 0u));  // the leader issues the MMAs
              }
              if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
          }
        }
#pragma unroll
        for (int j = 0; j < kG; ++j) { va[j] = na[j]; vb0[j] = nb0[j]; vb1[j] = nb1[j]; }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue (warps 2..9)
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int half = (warp - 2) / 4;              // which half of the tile's columns this warp handles
    constexpr int kChunksPerWarp = (kBN / 32) / (kEpiWarps / 4);
    uint32_t acc = 0, acc_phase = 0;
    uint32_t amax_bits = 0u;
    constexpr int OSZ = ElemBytes<OUT>::v;
    // delayed rescale (Section 3.3): the data are written already divided by r = p2_floor(earlier
    // statistic); this step's statistic is taken on the un-rebalanced fp32 values
    float r_prev = 1.0f;
    if (p.stat_in) { bool nf; r_prev = rescale_factor(*reinterpret_cast<const volatile float*>(p.stat_in), &nf); }
    float alpha = p.alpha * (1.0f / r_prev);  // exact: both are powers of two
    float beta = 0.f;
    if constexpr (BIAS) {
      // both terms are brought to the output scale max(A_s B_s kf(K), bias_s): exact power-of-two factors
      const float ab_s = load_scale_after_wait(p.a_scale) * load_scale_after_wait(p.b_scale) * p.kf;
      const float b_s = load_scale_after_wait(p.bias_scale);
      const float ys = fmaxf(ab_s, b_s);
      alpha *= ab_s / ys;
      beta = b_s / ys;
    }
    for (int tile = unit; tile < num_tiles; tile += num_units) {
      int b, mt, nt;
      tile_coords(p, tile, b, mt, nt);
      if (!mbar_wait(acc_full_bar + 8 * acc, acc_phase, abort_flag)) { timed_out = true; break; }
      tc_fence_after();
      const int n0 = nt * kBN;
      float ssq = 0.f;
      const int c_first = half * kChunksPerWarp;
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kBN + c_first * 32;
      // chunks of this warp that lie inside the matrix (warp-uniform)
      const int n_chunks = max(0, min(kChunksPerWarp, (p.N - n0 + 31) / 32 - c_first));
      float bias_reg[kChunksPerWarp];
      if constexpr (BIAS) {
#pragma unroll
        for (int c = 0; c < kChunksPerWarp; ++c) {
          const int col = n0 + (c_first + c) * 32 + lane;
          float bv = 0.f;
          if (col < p.N) {
            if (p.bias_dt == SCALIFY_F32) bv = load_elem<SCALIFY_F32>(p.bias, col);
            else if (p.bias_dt == SCALIFY_BF16) bv = load_elem<SCALIFY_BF16>(p.bias, col);
            else bv = load_elem<SCALIFY_F16>(p.bias, col);
          }
          bias_reg[c] = bv * beta;
        }
      }
      // One 32-column chunk of this thread's row in two steps: scale + statistic + round (convert), then store.
      constexpr int CPR = 32 * OSZ / 16;              // 16-byte pieces per row: 2 (FP8), 4 (16-bit), 8 (F32)
      constexpr int kTileBytes = 32 * 32 * OSZ;
      // staging tiles per warp: 4, 4 or 2; with the speculative output 2 of Y (4 KB) and 2 FP8 tiles behind them
      // (the FP8-only form stages no 16-bit tile and uses four FP8 tiles)
      constexpr int NBUF = NOY ? 4 : SPEC ? 2 : (C::kEpiWarpBytes / kTileBytes > 4 ? 4 : C::kEpiWarpBytes / kTileBytes);
      float inv_r_pred = 1.0f;
      // (a plain load: in the FP8-only form the word is rewritten at the end of this very kernel)
      if constexpr (SPEC) { bool nf2; inv_r_pred = 1.0f / rescale_factor(*reinterpret_cast<const volatile float*>(p.stat_hint), &nf2); }
      auto convert = [&](const uint32_t* acc_regs, uint32_t* o, int c) {
        float v[32];
        if constexpr (BIAS) {
          // lane l holds the (scaled) bias of column l of each of this warp's chunks; every lane needs all 32
          static_assert(!BIAS || kChunksPerWarp == 4, "four chunks per warp");
          const float mine = c == 0 ? bias_reg[0] : (c == 1 ? bias_reg[1] : (c == 2 ? bias_reg[2] : bias_reg[3]));
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            v[i] = fmaf(__uint_as_float(acc_regs[i]), alpha, __shfl_sync(0xFFFFFFFFu, mine, i));
            amax_bits = max(amax_bits, abs_bits(v[i]));
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            v[i] = __uint_as_float(acc_regs[i]) * alpha;
            amax_bits = max(amax_bits, abs_bits(v[i]));
          }
        }
        if (p.stat == SCALIFY_STAT_L2) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float s = p.stat_in ? v[i] : round_through<OUT>(v[i]);
            ssq = fmaf(s, s, ssq);
          }
        }
        encode_vec<OUT, 32>(v, o);
      };
      // speculative FP8 copy of a chunk: the STORED 16-bit values divided by the predicted power of two
      auto convert_q = [&](const uint32_t* o, uint32_t* oq) {
        float vr[32];
        decode_vec<OUT, 32>(o, vr);
#pragma unroll
        for (int i = 0; i < 32; ++i) vr[i] *= inv_r_pred;
        if (p.q_dt == SCALIFY_E4M3) encode_vec<SCALIFY_E4M3, 32>(vr, oq);
        else encode_vec<SCALIFY_E5M2, 32>(vr, oq);
      };
      // Each lane holds 32 consecutive columns of ONE row.  The warp writes the chunk (32 rows x 32 columns)
      // into a shared-memory tile in the swizzle pattern TMA uses for rows of this width, and one lane hands
      // the tile to a TMA store, which writes whole row segments and clips rows >= M and columns >= N.
      // (stage_chunk fills the tile; issue_chunk hands it to TMA)
      auto stage_chunk = [&](const uint32_t* o, int c) {
        if constexpr (!NOY) {
          uint8_t* tile_b = epi_mem + (warp - 2) * C::kEpiWarpBytes + (c % NBUF) * kTileBytes;
          uint4* tile = reinterpret_cast<uint4*>(tile_b);
#pragma unroll
          for (int j = 0; j < CPR; ++j)
            tile[lane * CPR + (j ^ ((lane / (8 / CPR)) % CPR))] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        }
        if constexpr (SPEC) {
          uint8_t* tile_q = epi_mem + (warp - 2) * C::kEpiWarpBytes + 4096 + (c % NBUF) * 1024;
          uint32_t oq[8];
          convert_q(o, oq);
          uint4* tq = reinterpret_cast<uint4*>(tile_q);  // 32 rows x 32 B, 32-byte swizzle: piece XOR (row / 4) % 2
          tq[lane * 2 + (0 ^ ((lane >> 2) & 1))] = make_uint4(oq[0], oq[1], oq[2], oq[3]);
          tq[lane * 2 + (1 ^ ((lane >> 2) & 1))] = make_uint4(oq[4], oq[5], oq[6], oq[7]);
        }
      };
      auto issue_chunk = [&](int c) {  // lane 0, after fence_async_smem + __syncwarp
        const int col0 = n0 + (c_first + c) * 32;
        const int row0 = mt * C::kTileM + static_cast<int>(rank) * kBM + q * 32;
        if constexpr (!NOY) {
          uint8_t* tile_b = epi_mem + (warp - 2) * C::kEpiWarpBytes + (c % NBUF) * kTileBytes;
          tma_store_3d(&map_y, smem_u32(tile_b), col0, row0, b);
        }
        if constexpr (SPEC) {
          uint8_t* tile_q = epi_mem + (warp - 2) * C::kEpiWarpBytes + 4096 + (c % NBUF) * 1024;
          tma_store_3d(&map_sfa, smem_u32(tile_q), col0, row0, b);
        }
      };
      auto store = [&](const uint32_t* o, int c) {
        if (lane == 0) bulk_wait_read<NBUF - 1>();      // the tile's previous store has read it
        __syncwarp();
        stage_chunk(o, c);
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          issue_chunk(c);
          bulk_commit();
        }
      };
      auto release_accumulator = [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if constexpr (NCTA == 1) mbar_arrive(acc_empty_bar + 8 * acc);
          else mbar_arrive_cluster(map_to_cta(acc_empty_bar + 8 * acc, 0u));  // the leader issues the next MMAs
        }
      };
      uint32_t ra[32], rb[32];
      if constexpr (kAcc == 1 && OSZ <= 2) {
        // A single accumulator: the next tile's MMAs wait for this read-out.  The staging area holds all of
        // a warp's chunks (NBUF == kChunksPerWarp), so every chunk is converted straight into its tile, the
        // accumulator is handed back, and only then the TMA stores are issued.
        static_assert(NBUF >= kChunksPerWarp, "staging must hold every chunk of a warp");
        uint32_t o[32 * OSZ / 4];
        if (lane == 0) bulk_wait_read<0>();  // the previous tile's stores have read the staging area
        __syncwarp();
        if (n_chunks > 0) tmem_ld32(t_addr, ra);
#pragma unroll 1
        for (int c = 0; c < n_chunks; c += 2) {
          tmem_ld_wait();
          if (c + 1 < n_chunks) tmem_ld32(t_addr + (c + 1) * 32, rb);
          convert(ra, o, c);
          stage_chunk(o, c);
          if (c + 1 < n_chunks) {
            tmem_ld_wait();
            if (c + 2 < n_chunks) tmem_ld32(t_addr + (c + 2) * 32, ra);
            convert(rb, o, c + 1);
            stage_chunk(o, c + 1);
          }
        }
        release_accumulator();
        fence_async_smem();
        __syncwarp();
        if (lane == 0 && n_chunks > 0) {
          for (int c = 0; c < n_chunks; ++c) issue_chunk(c);
          bulk_commit();
        }
      } else {
        // The TMEM load of the next chunk is in flight while the current chunk is processed.
        uint32_t o[32 * OSZ / 4];
        if (n_chunks > 0) tmem_ld32(t_addr, ra);
#pragma unroll 1
        for (int c = 0; c < n_chunks; c += 2) {
          tmem_ld_wait();
          if (c + 1 < n_chunks) tmem_ld32(t_addr + (c + 1) * 32, rb);
          convert(ra, o, c);
          store(o, c);
          if (c + 1 < n_chunks) {
            tmem_ld_wait();
            if (c + 2 < n_chunks) tmem_ld32(t_addr + (c + 2) * 32, ra);
            convert(rb, o, c + 1);
            store(o, c + 1);
          }
        }
        release_accumulator();
      }
      if (p.stat == SCALIFY_STAT_L2) {
        const double s = warp_sum_f64(static_cast<double>(ssq)) * (double(r_prev) * double(r_prev));
        if (lane == 0) p.l2_partials[((static_cast<long long>(tile) * NCTA + rank) * 4 + q) * 2 + half] = s;
      }
      if (++acc == kAcc) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_all();  // every store of this warp has completed
    if (p.stat == SCALIFY_STAT_AMAX) {
      // rounding is monotonic, so the max of the stored values is the stored value of the max
      if (p.stat_in) amax_bits = abs_bits(__uint_as_float(amax_bits) * r_prev);  // un-rebalanced, unrounded
      else amax_bits = abs_bits(round_through<OUT>(__uint_as_float(amax_bits)));
      amax_bits = warp_max_u32(amax_bits);
      if (lane == 0 && amax_bits != 0u) atomicMax(p.amax_scratch, amax_bits);
    }
  }

  if (timed_out && p.status) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_TIMEOUT));
  tc_fence_before();
  __syncthreads();
  if (p.stat == SCALIFY_STAT_AMAX && threadIdx.x == 0) {
    // publish: the last CTA to get here has everybody's maxima in the scratch word
    __threadfence();
    if (atomicAdd(p.ticket, 1u) == gridDim.x - 1) {
      __threadfence();
      const float stat_now = __uint_as_float(atomicExch(p.amax_scratch, 0u));
      *p.stat_word = stat_now;
      *p.ticket = 0u;
      if constexpr (NOY) {
        bool nfq;
        const float r_true = rescale_factor(stat_now, &nfq);
        const float ys = load_scale_after_wait(p.a_scale) * load_scale_after_wait(p.b_scale) * p.kf;
        if (p.yq_scale) *p.yq_scale = ys * r_true;
        if (p.hint_out) *p.hint_out = stat_now;  // every CTA has read the old prediction: all passed the ticket
        if (nfq && p.status) atomicOr(p.status, static_cast<uint32_t>(SCALIFY_DEV_NONFINITE_STAT));
      }
    }
  }
  if constexpr (NCTA == 2) cluster_sync_all();  // neither CTA leaves while the other may still touch its memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int OUT, int NCTA>
__global__ void __launch_bounds__(kGemmThreads, 1)
scaled_matmul_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __grid_constant__ CUtensorMap map_y, const GemmParams p) {
  gemm_body<OUT, NCTA, false>(map_a, map_b, map_y, map_a, map_a, p);
}

// The same kernel with a bias vector added in the epilogue (add rule, one rounding).
template <int OUT, int NCTA>
__global__ void __launch_bounds__(kGemmThreads, 1)
scaled_matmul_bias_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                          const __grid_constant__ CUtensorMap map_y, const GemmParams p) {
  gemm_body<OUT, NCTA, false, false, true>(map_a, map_b, map_y, map_a, map_a, p);
}

// The same kernel that also writes the FP8 output quantised with a PREDICTED rescale factor.
template <int OUT, int NCTA>
__global__ void __launch_bounds__(kGemmThreads, 1)
scaled_matmul_spec_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                          const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_q,
                          const GemmParams p) {
  gemm_body<OUT, NCTA, false, true>(map_a, map_b, map_y, map_q, map_q, p);
}

// The speculative kernel without the 16-bit intermediate: only the FP8 output is stored (map_y is not used).
template <int OUT, int NCTA>
__global__ void __launch_bounds__(kGemmThreads, 1)
scaled_matmul_fp8only_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                             const __grid_constant__ CUtensorMap map_q, const GemmParams p) {
  gemm_body<OUT, NCTA, false, true, false, true>(map_a, map_b, map_q, map_q, map_q, p);
}

// Block-scaled operands (E8M0 exponent per 32 elements of K), K-major A [M,K] and B [N,K].
template <int OUT, int NCTA>
__global__ void __launch_bounds__(kMxGemmThreads, 1)
mx_matmul_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_y, const GemmParams p) {
  gemm_body<OUT, NCTA, true>(map_a, map_b, map_y, map_a, map_a, p);
}

// Diagnostic: one thread waits, with the GEMM's bounded-wait routine and a short limit, on an
// mbarrier that nothing ever arrives at; the wait must give up, record SCALIFY_DEV_TIMEOUT and let
// the kernel finish normally (this is the path a lost copy or a lost MMA completion would take).
__global__ void expire_wait_kernel(uint32_t* status, unsigned long long limit_ns, uint32_t* waited_us) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    const uint32_t b = smem_u32(&bar);
    mbar_init(b, 1);
    abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const unsigned long long t0 = global_timer_ns();
    const bool ok = mbar_wait(b, 0u, &abort_flag, limit_ns);
    if (waited_us) *waited_us = static_cast<uint32_t>((global_timer_ns() - t0) / 1000ull);
    if (!ok && status) atomicOr(status, static_cast<uint32_t>(SCALIFY_DEV_TIMEOUT));
  }
}

int launch_expire_wait(void* ws, unsigned long long limit_ns, uint32_t* waited_us, cudaStream_t st) {
  expire_wait_kernel<<<1, 32, 0, st>>>(ws_view(ws).status, limit_ns, waited_us);
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

// Sums the per-warp partial sums of squares in slot order and leaves sqrt(mean) in the statistic word.
__global__ void __launch_bounds__(256) gemm_l2_finalize_kernel(const double* __restrict__ partials, int n_slots,
                                                               double count, float* stat_word) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  __shared__ double s[8];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n_slots; i += 256) acc += partials[i];
  acc = warp_sum_f64(acc);
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int i = 0; i < 8; ++i) tot += s[i];
    *stat_word = static_cast<float>(sqrt(tot / count));
  }
}

// Split contraction: the partial products [splits][M][ldp] (fp32, not yet divided by kf(K)) are added in split
// order, scaled, rounded once to the output format and written; the statistic of the stored values goes
// through one partial per block and the block that draws the last ticket (index order: scheduling does not
// change the result).
template <int OUT>
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float* __restrict__ part, long long ldp, long long plane,
                                                            int splits, int M, int N, void* __restrict__ Y, long long ldy,
                                                            float alpha, int stat, const float* a_scale,
                                                            const float* b_scale, float* y_scale, float kf,
                                                            double* __restrict__ partials, uint32_t* ticket,
                                                            float* stat_word) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int OSZ = ElemBytes<OUT>::v;
  const long long nvr = ldp / 4, total = static_cast<long long>(M) * nvr;
  const long long idx = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
  uint32_t amax = 0u;
  float ssq = 0.f;
  if (idx < total) {
    const long long row = idx / nvr;
    const int col = static_cast<int>(idx % nvr) * 4;
    const float4* src = reinterpret_cast<const float4*>(part + row * ldp + col);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < splits; s0 += 4) {  // four loads in flight, added in split order
      float4 t[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        t[u] = (s0 + u < splits)
                   ? __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(src) + (s0 + u) * plane))
                   : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 4; ++u) { acc.x += t[u].x; acc.y += t[u].y; acc.z += t[u].z; acc.w += t[u].w; }
    }
    float v[4] = {acc.x * alpha, acc.y * alpha, acc.z * alpha, acc.w * alpha};
    uint32_t o[OSZ];  // 4 elements: 4 * OSZ bytes
    encode_vec<OUT, 4>(v, o);
    char* dst = static_cast<char*>(Y) + (row * ldy + col) * OSZ;
    if (col + 4 <= N) {
      st_raw<4 * OSZ>(dst, o);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (col + e < N) store_elem<OUT>(Y, row * ldy + col + e, v[e]);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (col + e < N) {
        const float sv = round_through<OUT>(v[e]);  // the value as stored
        amax = max(amax, abs_bits(sv));
        ssq = fmaf(sv, sv, ssq);
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && y_scale) *y_scale = load_scale(a_scale) * load_scale(b_scale) * kf;
  if (stat == SCALIFY_STAT_NONE) return;
  __shared__ double s_part[8];
  __shared__ bool s_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double mine = (stat == SCALIFY_STAT_AMAX) ? static_cast<double>(warp_max_u32(amax))
                                            : warp_sum_f64(static_cast<double>(ssq));
  if (lane == 0) s_part[warp] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int i = 0; i < 8; ++i) tot = (stat == SCALIFY_STAT_AMAX) ? fmax(tot, s_part[i]) : tot + s_part[i];
    partials[blockIdx.x] = tot;
    __threadfence();
    s_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  double acc = 0.0;
  for (int i = threadIdx.x; i < static_cast<int>(gridDim.x); i += 256) {
    const double pv = __ldcg(&partials[i]);
    acc = (stat == SCALIFY_STAT_AMAX) ? fmax(acc, pv) : acc + pv;
  }
  acc = (stat == SCALIFY_STAT_AMAX) ? static_cast<double>(warp_max_u32(static_cast<uint32_t>(acc))) : warp_sum_f64(acc);
  __syncthreads();
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int i = 0; i < 8; ++i) tot = (stat == SCALIFY_STAT_AMAX) ? fmax(tot, s_part[i]) : tot + s_part[i];
    *stat_word = (stat == SCALIFY_STAT_AMAX) ? __uint_as_float(static_cast<uint32_t>(tot))
                                             : static_cast<float>(sqrt(tot / (static_cast<double>(M) * N)));
    *ticket = 0u;
  }
}

// Region of the workspace after the header that is left to per-block statistic partials before the split-K
// partial products begin
constexpr size_t kSplitStatBytes = 65536 * sizeof(double);

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Encoded tensor maps are kept: a training step calls the same matmuls on the same buffers over and over, and
// encoding is host work (about a microsecond per map, three to five maps per call).  The key is everything the
// encoder is given; a tensor map describes addresses and a layout, not the memory's contents, so it stays valid
// for as long as that key describes what the caller passes.  256 entries, hashed, overwritten on collision.
struct MapKey {
  uint64_t ptr, dims[5], strides[4];
  uint32_t box[5], estr[5], dtype, rank, interleave, swizzle, promo, oob;
};
struct MapCache {
  static constexpr int kEntries = 256;
  std::mutex mu;
  bool used[kEntries] = {};
  MapKey keys[kEntries];
  CUtensorMap maps[kEntries];
  unsigned long long hits = 0, misses = 0;
};
static MapCache g_map_cache;

int encode_tiled_cached(MapCache& cache, EncodeTiledFn fn, CUtensorMap* map, CUtensorMapDataType dt, cuuint32_t rank,
                        void* ptr, const cuuint64_t* dims, const cuuint64_t* strides, const cuuint32_t* box,
                        const cuuint32_t* estr, CUtensorMapInterleave il, CUtensorMapSwizzle sw,
                        CUtensorMapL2promotion promo, CUtensorMapFloatOOBfill oob) {
  MapKey k;
  memset(&k, 0, sizeof(k));
  k.ptr = reinterpret_cast<uint64_t>(ptr);
  for (cuuint32_t i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; k.estr[i] = estr[i]; }
  for (cuuint32_t i = 0; i + 1 < rank; ++i) k.strides[i] = strides[i];
  k.dtype = static_cast<uint32_t>(dt); k.rank = rank; k.interleave = static_cast<uint32_t>(il);
  k.swizzle = static_cast<uint32_t>(sw); k.promo = static_cast<uint32_t>(promo); k.oob = static_cast<uint32_t>(oob);
  uint64_t h = 1469598103934665603ull;  // FNV-1a over the key
  const unsigned char* b = reinterpret_cast<const unsigned char*>(&k);
  for (size_t i = 0; i < sizeof(k); ++i) { h ^= b[i]; h *= 1099511628211ull; }
  const int slot = static_cast<int>((h ^ (h >> 29)) % MapCache::kEntries);
  std::lock_guard<std::mutex> lock(cache.mu);
  if (cache.used[slot] && memcmp(&cache.keys[slot], &k, sizeof(k)) == 0) {
    *map = cache.maps[slot];
    ++cache.hits;
    return SCALIFY_OK;
  }
  CUresult r = fn(map, dt, rank, ptr, dims, strides, box, estr, il, sw, promo, oob);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error(static_cast<int>(r));
    return SCALIFY_ERR_CUDA;
  }
  cache.keys[slot] = k;
  cache.maps[slot] = *map;
  cache.used[slot] = true;
  ++cache.misses;
  return SCALIFY_OK;
}

// Self-test of the two pieces of host state above, without a GPU: the per-device one-time set-up is driven with
// made-up device numbers, the tensor-map cache with a stand-in for the driver's encoder that counts its calls.
static int g_fake_encodes = 0;
static CUresult fake_encode(CUtensorMap* m, CUtensorMapDataType, cuuint32_t rank, void* p, const cuuint64_t* dims,
                            const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                            CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill) {
  ++g_fake_encodes;
  memset(m, 0, sizeof(*m));
  uint64_t tag = reinterpret_cast<uint64_t>(p) ^ (dims[0] << 20) ^ rank;
  memcpy(m, &tag, sizeof(tag));
  return CUDA_SUCCESS;
}
int host_state_selftest() {
  // (1) per-device once: devices 0, 1, 0, 2, 1, 63 -> four set-ups, each device keeps its own value
  DeviceOnce once;
  int runs = 0, v = -1;
  const int order[6] = {0, 1, 0, 2, 1, 63};
  for (int i = 0; i < 6; ++i) {
    const int dev = order[i];
    if (device_once_at(once, dev, &v, [&](int* val) { ++runs; *val = 100 + dev; return int(SCALIFY_OK); })) return 1;
    if (v != 100 + dev) return 2;
  }
  if (runs != 4) return 3;
  if (device_once_at(once, 64, &v, [&](int*) { return int(SCALIFY_OK); }) != SCALIFY_ERR_UNSUPPORTED) return 4;
  // a set-up that fails is not remembered as done
  int tries = 0;
  if (device_once_at(once, 5, &v, [&](int*) { ++tries; return int(SCALIFY_ERR_CUDA); }) != SCALIFY_ERR_CUDA) return 5;
  if (device_once_at(once, 5, &v, [&](int* val) { ++tries; *val = 7; return int(SCALIFY_OK); }) || v != 7 || tries != 2) return 6;
  // (2) tensor-map cache
  MapCache* cache = new MapCache();
  g_fake_encodes = 0;
  cuuint64_t dims[3] = {4096, 128, 1}, strides[2] = {4096, 4096 * 128};
  cuuint32_t box[3] = {128, 128, 1}, estr[3] = {1, 1, 1};
  CUtensorMap a, b, c;
  char* base = reinterpret_cast<char*>(0x100000);
  int bad = 0;
  auto enc = [&](CUtensorMap* m, void* p, cuuint64_t d0) {
    dims[0] = d0;
    return encode_tiled_cached(*cache, fake_encode, m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, p, dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  };
  bad |= enc(&a, base, 4096);             // miss
  bad |= enc(&b, base, 4096);             // hit: same bytes, no second encode
  if (bad || g_fake_encodes != 1 || memcmp(&a, &b, sizeof(a)) != 0) { delete cache; return 7; }
  bad |= enc(&c, base + 4096, 4096);      // another pointer: miss
  bad |= enc(&c, base, 8192);             // another extent: miss
  if (bad || g_fake_encodes != 3 || memcmp(&a, &c, sizeof(a)) == 0) { delete cache; return 8; }
  for (int i = 0; i < 2000; ++i) bad |= enc(&c, base + 16 * i, 4096);   // more keys than entries: still correct
  bad |= enc(&b, base, 4096);
  if (bad || memcmp(&a, &b, sizeof(a)) != 0) { delete cache; return 9; }
  const bool counted = cache->hits + cache->misses == 2005 && cache->misses == static_cast<unsigned long long>(g_fake_encodes);
  delete cache;
  return counted ? 0 : 10;
}

void map_cache_counters(unsigned long long* hits, unsigned long long* misses) {
  std::lock_guard<std::mutex> lock(g_map_cache.mu);
  *hits = g_map_cache.hits;
  *misses = g_map_cache.misses;
}

// Tensor map over a row-major byte matrix [batch][rows][inner] with row stride ld and batch
// stride bs (bytes); box = [1][box_rows][128].
static int make_map(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t rows, uint64_t batch, uint64_t ld,
                    uint64_t bs, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return SCALIFY_ERR_CUDA;
  cuuint64_t dims[3] = {inner, rows, batch};
  cuuint64_t strides[2] = {ld, bs ? bs : ld * rows};
  cuuint32_t box[3] = {128u, box_rows, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  return encode_tiled_cached(g_map_cache, fn, map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(ptr), dims, strides,
                             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// Tensor map over a row-major byte matrix [batch][rows][inner] with a box of [1][box_rows][box_inner]
// bytes and a 32 / 64 / 128-byte swizzle (box_inner equal to the swizzle width).
int make_byte_map(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t rows, uint64_t batch, uint64_t ld,
                  uint64_t bs, uint32_t box_inner, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return SCALIFY_ERR_CUDA;
  cuuint64_t dims[3] = {inner, rows, batch};
  cuuint64_t strides[2] = {ld, bs ? bs : ld * rows};
  cuuint32_t box[3] = {box_inner, box_rows, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  const CUtensorMapSwizzle sw = box_inner == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                              : box_inner == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
  return encode_tiled_cached(g_map_cache, fn, map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(ptr), dims, strides,
                             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// The same for [batch][heads][rows][inner] views (attention operands): box = one tile of one head
int make_byte_map4(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t rows, uint64_t heads, uint64_t batch,
                   uint64_t ld, uint64_t hs, uint64_t bs, uint32_t box_inner, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return SCALIFY_ERR_CUDA;
  cuuint64_t dims[4] = {inner, rows, heads, batch};
  const uint64_t hs_eff = hs ? hs : ld * rows;
  cuuint64_t strides[3] = {ld, hs_eff, bs ? bs : hs_eff * heads};
  cuuint32_t box[4] = {box_inner, box_rows, 1u, 1u};
  cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUtensorMapSwizzle sw = box_inner == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                              : box_inner == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
  return encode_tiled_cached(g_map_cache, fn, map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(ptr), dims, strides,
                             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// Tensor map of the output [batch][M][N] (row stride ld, batch stride bs, in elements of `es` bytes) for the
// epilogue's stores: box 32 columns x 32 rows, swizzle equal to the width of a box row (32 / 64 / 128 bytes).
static int make_map_y(CUtensorMap* map, const void* ptr, int es, uint64_t N, uint64_t M, uint64_t batch, uint64_t ld,
                      uint64_t bs) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return SCALIFY_ERR_CUDA;
  cuuint64_t dims[3] = {N, M, batch};
  cuuint64_t strides[2] = {ld * es, (bs ? bs : ld * M) * es};
  cuuint32_t box[3] = {32u, 32u, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  const CUtensorMapDataType dt = es == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                               : es == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32;
  const CUtensorMapSwizzle sw = es == 1 ? CU_TENSOR_MAP_SWIZZLE_32B
                              : es == 2 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
  return encode_tiled_cached(g_map_cache, fn, map, dt, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

size_t matmul_splitk_ws_bytes(int64_t rows, int64_t cols) {
  const size_t base = matmul_ws_bytes(rows, cols);
  // the most parts launch_scaled_matmul would cut a product of this output size into (none for a large output)
  const int ncta = rows > kBM ? 2 : 1;
  const int64_t out_tiles = ((rows + kBM * ncta - 1) / (kBM * ncta)) * ((cols + kBN - 1) / kBN);
  int64_t splits = (ncta == 2 ? sm_count() / 2 : sm_count()) / (out_tiles > 0 ? out_tiles : 1);
  if (splits > 16) splits = 16;
  if (splits < 3) return base;
  const size_t ldp = static_cast<size_t>((cols + 3) / 4 * 4);
  const size_t n = kWsHeader + kSplitStatBytes + static_cast<size_t>(splits) * static_cast<size_t>(rows) * ldp * sizeof(float) + 256;
  return n > base ? n : base;
}

size_t matmul_ws_bytes(int64_t rows, int64_t cols) {
  int64_t tiles = ((rows + kBM - 1) / kBM + 8) * ((cols + kBN - 1) / kBN);
  return kWsHeader + size_t(tiles) * 8 * sizeof(double) + 256;
}

template <int OUT, int NCTA, bool SPEC, bool BIAS, bool NOY = false>
struct GemmKernelOf {
  static auto get() { return scaled_matmul_kernel<OUT, NCTA>; }
};
template <int OUT, int NCTA>
struct GemmKernelOf<OUT, NCTA, true, false, true> {
  static auto get() { return scaled_matmul_fp8only_kernel<OUT, NCTA>; }
};
template <int OUT, int NCTA>
struct GemmKernelOf<OUT, NCTA, true, false, false> {
  static auto get() { return scaled_matmul_spec_kernel<OUT, NCTA>; }
};
template <int OUT, int NCTA>
struct GemmKernelOf<OUT, NCTA, false, true, false> {
  static auto get() { return scaled_matmul_bias_kernel<OUT, NCTA>; }
};

template <int OUT, int NCTA, bool SPEC = false, bool BIAS = false, bool NOY = false>
static int launch_variant(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_y,
                          const CUtensorMap& map_q, const GemmParams& p, long long tiles,
                          cudaStream_t st) {
  using C = GemmCfg<NCTA>;
  auto kernel = GemmKernelOf<OUT, NCTA, SPEC, BIAS, NOY>::get();
  // per device: the dynamic shared-memory limit of this kernel and the number of CTA pairs that fit the GPU
  static DeviceOnce once;
  int max_clusters = 0;
  int rc_once = device_once(once, &max_clusters, [&](int* clusters) {
    SCALIFY_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(C::kSmem)));
    if (NCTA == 2) {
      cudaLaunchConfig_t qc = {};
      qc.gridDim = dim3(unsigned(sm_count() / 2 * 2));
      qc.blockDim = dim3(kGemmThreads);
      qc.dynamicSmemBytes = C::kSmem;
      cudaLaunchAttribute qa[1];
      qa[0].id = cudaLaunchAttributeClusterDimension;
      qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
      qc.attrs = qa;
      qc.numAttrs = 1;
      int n = 0;
      SCALIFY_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, kernel, &qc));
      if (n < 1) return int(SCALIFY_ERR_UNSUPPORTED);
      *clusters = n;
    }
    return int(SCALIFY_OK);
  });
  if (rc_once) return rc_once;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attrs[2];
  attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the prologue may overlap the grid before it
  attrs[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = 1;
  if (NCTA == 2) {
    const long long units = tiles < max_clusters ? tiles : max_clusters;
    cfg.gridDim = dim3(unsigned(units * 2));
    attrs[1].id = cudaLaunchAttributeClusterDimension;
    attrs[1].val.clusterDim.x = 2; attrs[1].val.clusterDim.y = 1; attrs[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  } else {
    cfg.gridDim = dim3(unsigned(tiles < sm_count() ? tiles : sm_count()));
  }
  cfg.blockDim = dim3(kGemmThreads);
  cfg.dynamicSmemBytes = C::kSmem;
  cfg.stream = st;
  if constexpr (NOY) SCALIFY_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, map_a, map_b, map_q, p));
  else if constexpr (SPEC) SCALIFY_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, map_a, map_b, map_y, map_q, p));
  else SCALIFY_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, map_a, map_b, map_y, p));
  return SCALIFY_OK;
}

int launch_scaled_matmul(const MatmulArgs& a, void* ws, size_t ws_bytes, cudaStream_t st) {
  WsView v = ws_view(ws);
  // two-CTA tiles (256 rows) whenever there is more than one 128-row tile of output
  const int ncta = (a.M > kBM && a.force_ncta != 1) ? 2 : 1;
  const int tile_m = kBM * ncta;
  // A product with few output tiles and a long contraction (a weight gradient) leaves most SMs idle: its K
  // range is cut into `splits` parts that run as one batched call writing fp32 partial products into the
  // workspace (when the caller's workspace has the room), and a second launch adds them in split order.
  if (a.took_spec) *a.took_spec = 0;
  if (!a.no_split && a.batch == 1 && !a.stat_in && (!a.stat_hint || a.hint_optional) && !a.noy && !a.bias &&
      a.K >= 2048) {
    const long long out_tiles = static_cast<long long>((a.M + tile_m - 1) / tile_m) * ((a.N + kBN - 1) / kBN);
    const long long units = ncta == 2 ? sm_count() / 2 : sm_count();
    int splits = static_cast<int>(units / out_tiles);
    if (splits > a.K / 512) splits = a.K / 512;
    if (splits > 16) splits = 16;
    while (splits >= 3 && a.K % (splits * kBK) != 0) --splits;
    const long long ldp = (static_cast<long long>(a.N) + 3) / 4 * 4;
    const size_t need = kWsHeader + kSplitStatBytes + static_cast<size_t>(splits) * a.M * ldp * sizeof(float);
    const long long red_blocks = (static_cast<long long>(a.M) * (ldp / 4) + 255) / 256;
    if (splits >= 3 && ws_bytes >= need && red_blocks <= 65536) {  // (two parts measured no faster than one launch)
      float* part = reinterpret_cast<float*>(static_cast<char*>(v.area) + kSplitStatBytes);
      MatmulArgs pa = a;
      pa.stat_hint = nullptr; pa.Yq = nullptr; pa.hint_optional = 0; pa.took_spec = nullptr;
      const int Kc = a.K / splits;
      pa.K = Kc;
      pa.batch = splits;
      pa.a_bs = a.transA ? static_cast<int64_t>(Kc) * a.lda : Kc;
      pa.b_bs = a.transB ? Kc : static_cast<int64_t>(Kc) * a.ldb;
      pa.Y = part; pa.y_dt = SCALIFY_F32; pa.ldy = ldp; pa.y_bs = static_cast<int64_t>(a.M) * ldp;
      pa.y_scale = nullptr;
      pa.stat = SCALIFY_STAT_NONE;
      pa.alpha_override = 1.0f;
      pa.no_split = 1;
      int rc2 = launch_scaled_matmul(pa, ws, ws_bytes, st);
      if (rc2) return rc2;
      const float kf = kfactor(a.K);
      SCALIFY_DISPATCH_WIDE(a.y_dt, OUT, splitk_reduce_kernel<OUT><<<static_cast<unsigned>(red_blocks), 256, 0, st>>>(
                                             part, ldp, static_cast<long long>(a.M) * ldp, splits, a.M, a.N, a.Y, a.ldy,
                                             1.0f / kf, a.stat, a.a_scale, a.b_scale, a.y_scale, kf,
                                             static_cast<double*>(v.area), v.ticket, v.stat));
      SCALIFY_CUDA_TRY(cudaGetLastError());
      return SCALIFY_OK;
    }
  }
  const uint32_t b_box_rows = ncta == 2 ? kBN / 2 : kBN;
  CUtensorMap map_a, map_b, map_y;
  // A is logically [M,K]; stored [M,K] (K-major) or, with transA, [K,M] (MN-major).
  int rc;
  if (!a.transA) rc = make_map(&map_a, a.A, a.K, a.M, a.batch, a.lda, a.a_bs, kBM);
  else rc = make_map(&map_a, a.A, a.M, a.K, a.batch, a.lda, a.a_bs, kBK);
  if (rc) return rc;
  // B is logically [K,N]; stored [K,N] (MN-major) or, with transB, [N,K] (K-major).
  const int b_batched = a.b_bs != 0 ? 1 : 0;
  const int b_batch = b_batched ? a.batch : 1;
  if (a.transB) rc = make_map(&map_b, a.B, a.K, a.N, b_batch, a.ldb, a.b_bs, b_box_rows);
  else rc = make_map(&map_b, a.B, a.N, a.K, b_batch, a.ldb, a.b_bs, kBK);
  if (rc) return rc;

  if (!a.noy) {
    rc = make_map_y(&map_y, a.Y, elem_size(a.y_dt), a.N, a.M, a.batch, a.ldy, a.y_bs);
    if (rc) return rc;
  }

  GemmParams p;
  p.M = a.M; p.N = a.N; p.K = a.K; p.batch = a.batch;
  p.tiles_m = (a.M + tile_m - 1) / tile_m;
  p.tiles_n = (a.N + kBN - 1) / kBN;
  p.a_mn_major = a.transA ? 1 : 0;
  p.b_mn_major = a.transB ? 0 : 1;
  p.b_batched = b_batched;
  // instruction descriptor (kind::f8f6f4): D fp32, A/B formats (0 = E4M3, 1 = E5M2), operand
  // majorness (0 = K-major), N >> 3, M >> 4 (M counts the rows of the whole CTA pair)
  p.idesc = (1u << 4) | (uint32_t(a.a_dt == SCALIFY_E5M2) << 7) | (uint32_t(a.b_dt == SCALIFY_E5M2) << 10) |
            (uint32_t(p.a_mn_major) << 15) | (uint32_t(p.b_mn_major) << 16) | (uint32_t(kBN >> 3) << 17) |
            (uint32_t(tile_m >> 4) << 24);
  p.kf = kfactor(a.K);
  p.alpha = a.alpha_override != 0.f ? a.alpha_override : 1.0f / p.kf;
  p.Y = a.Y; p.ldy = a.ldy; p.y_batch_stride = a.y_bs;
  p.a_scale = a.a_scale; p.b_scale = a.b_scale; p.y_scale = a.y_scale;
  p.stat = a.stat;
  p.stat_in = a.stat_in;
  p.stat_word = v.stat;
  p.amax_scratch = reinterpret_cast<uint32_t*>(v.stat) + 1;
  p.ticket = v.ticket;
  p.l2_partials = static_cast<double*>(v.area);
  p.status = v.status;
  p.sfa = nullptr;
  p.sfb = nullptr;
  p.stat_hint = a.stat_hint;
  p.q_dt = a.q_dt;
  p.bias = a.bias; p.bias_dt = a.bias_dt; p.bias_scale = a.bias_scale;
  p.r_pred_out = reinterpret_cast<float*>(static_cast<char*>(ws) + 52);  // header word read by the check kernel
  p.yq_scale = a.yq_scale; p.hint_out = a.hint_out; p.redo = 0;
  const long long tiles = static_cast<long long>(p.tiles_m) * p.tiles_n * p.batch;
  if (tiles > (1ll << 30)) return SCALIFY_ERR_SHAPE;
  if (a.stat_hint && a.noy) {
    // FP8 output only, then the repair launch (its CTAs return at once when the prediction held)
    CUtensorMap map_q;
    rc = make_map_y(&map_q, a.Yq, 1, a.N, a.M, a.batch, a.ldy, a.y_bs);
    if (rc) return rc;
    for (int pass = 0; pass < 2 && !rc; ++pass) {
      p.redo = pass;
      if (pass) p.stat_hint = v.stat;  // the statistic the first launch left is the exact "prediction"
      if (a.y_dt == SCALIFY_BF16) {
        if (ncta == 2) rc = launch_variant<SCALIFY_BF16, 2, true, false, true>(map_a, map_b, map_q, map_q, p, tiles, st);
        else rc = launch_variant<SCALIFY_BF16, 1, true, false, true>(map_a, map_b, map_q, map_q, p, tiles, st);
      } else {
        if (ncta == 2) rc = launch_variant<SCALIFY_F16, 2, true, false, true>(map_a, map_b, map_q, map_q, p, tiles, st);
        else rc = launch_variant<SCALIFY_F16, 1, true, false, true>(map_a, map_b, map_q, map_q, p, tiles, st);
      }
    }
    if (a.took_spec) *a.took_spec = 1;
  } else if (a.stat_hint) {
    if (a.took_spec) *a.took_spec = 1;
    // speculative FP8 output next to the 16-bit intermediate
    CUtensorMap map_q;
    rc = make_map_y(&map_q, a.Yq, 1, a.N, a.M, a.batch, a.ldy, a.y_bs);
    if (rc) return rc;
    if (a.y_dt == SCALIFY_BF16) {
      if (ncta == 2) rc = launch_variant<SCALIFY_BF16, 2, true>(map_a, map_b, map_y, map_q, p, tiles, st);
      else rc = launch_variant<SCALIFY_BF16, 1, true>(map_a, map_b, map_y, map_q, p, tiles, st);
    } else {
      if (ncta == 2) rc = launch_variant<SCALIFY_F16, 2, true>(map_a, map_b, map_y, map_q, p, tiles, st);
      else rc = launch_variant<SCALIFY_F16, 1, true>(map_a, map_b, map_y, map_q, p, tiles, st);
    }
  } else if (a.bias) {
    SCALIFY_DISPATCH_DTYPE(a.y_dt, OUT, {
      if (ncta == 2) rc = launch_variant<OUT, 2, false, true>(map_a, map_b, map_y, map_a, p, tiles, st);
      else rc = launch_variant<OUT, 1, false, true>(map_a, map_b, map_y, map_a, p, tiles, st);
    });
  } else {
    SCALIFY_DISPATCH_DTYPE(a.y_dt, OUT, {
      if (ncta == 2) rc = launch_variant<OUT, 2>(map_a, map_b, map_y, map_a, p, tiles, st);
      else rc = launch_variant<OUT, 1>(map_a, map_b, map_y, map_a, p, tiles, st);
    });
  }
  if (rc) return rc;
  if (a.stat == SCALIFY_STAT_L2) {
    gemm_l2_finalize_kernel<<<1, 256, 0, st>>>(p.l2_partials, static_cast<int>(tiles * ncta * 8),
                                               double(a.M) * double(a.N) * double(a.batch), v.stat);
    SCALIFY_CUDA_TRY(cudaGetLastError());
  }
  return SCALIFY_OK;
}

template <int OUT, int NCTA>
static int launch_mx_variant(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_y,
                             const GemmParams& p, long long tiles, cudaStream_t st) {
  using C = GemmCfg<NCTA, true>;
  auto kernel = mx_matmul_kernel<OUT, NCTA>;
  cudaLaunchAttribute attrs[1];
  attrs[0].id = cudaLaunchAttributeClusterDimension;
  attrs[0].val.clusterDim.x = 2; attrs[0].val.clusterDim.y = 1; attrs[0].val.clusterDim.z = 1;
  static DeviceOnce once;  // per device, like the per-tensor kernel
  int max_clusters = 0;
  int rc_once = device_once(once, &max_clusters, [&](int* clusters) {
    SCALIFY_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(C::kSmem)));
    if (NCTA == 2) {
      cudaLaunchConfig_t qc = {};
      qc.gridDim = dim3(unsigned(sm_count() / 2 * 2));
      qc.blockDim = dim3(kMxGemmThreads);
      qc.dynamicSmemBytes = C::kSmem;
      qc.attrs = attrs;
      qc.numAttrs = 1;
      int n = 0;
      SCALIFY_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, kernel, &qc));
      if (n < 1) return int(SCALIFY_ERR_UNSUPPORTED);
      *clusters = n;
    }
    return int(SCALIFY_OK);
  });
  if (rc_once) return rc_once;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute run_attrs[2];
  run_attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the prologue may overlap the grid before it
  run_attrs[0].val.programmaticStreamSerializationAllowed = 1;
  run_attrs[1] = attrs[0];
  cfg.attrs = run_attrs;
  if (NCTA == 2) {
    const long long units = tiles < max_clusters ? tiles : max_clusters;
    cfg.gridDim = dim3(unsigned(units * 2));
    cfg.numAttrs = 2;
  } else {
    cfg.gridDim = dim3(unsigned(tiles < sm_count() ? tiles : sm_count()));
    cfg.numAttrs = 1;
  }
  cfg.blockDim = dim3(kMxGemmThreads);
  cfg.dynamicSmemBytes = C::kSmem;
  cfg.stream = st;
  SCALIFY_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, map_a, map_b, map_y, p));
  return SCALIFY_OK;
}

int launch_mx_matmul(const MxMatmulArgs& a, void* ws, cudaStream_t st) {
  WsView v = ws_view(ws);
  const int ncta = (a.M > kBM && a.force_ncta != 1) ? 2 : 1;
  const int tile_m = kBM * ncta;
  CUtensorMap map_a, map_b, map_y;
  // K-major operand [rows, K]: box of 128 (or 256) rows x 128 bytes of K; transposed operand [K, rows]: box of
  // 128 K-rows x 128 bytes of rows, consumed MN-major (as the per-tensor kernel does for transA / plain B)
  int rc;
  if (!a.transA) rc = make_map(&map_a, a.A, a.K, a.M, 1, a.K, 0, kBM);
  else rc = make_map(&map_a, a.A, a.M, a.K, 1, a.M, 0, kBK);
  if (rc) return rc;
  if (!a.transB) rc = make_map(&map_b, a.B, a.K, a.N, 1, a.K, 0, ncta == 2 ? kBN / 2 : kBN);
  else rc = make_map(&map_b, a.B, a.N, a.K, 1, a.N, 0, kBK);
  if (rc) return rc;
  rc = make_map_y(&map_y, a.Y, elem_size(a.y_dt), a.N, a.M, 1, a.ldy, 0);
  if (rc) return rc;
  GemmParams p;
  p.M = a.M; p.N = a.N; p.K = a.K; p.batch = 1;
  p.tiles_m = (a.M + tile_m - 1) / tile_m;
  p.tiles_n = (a.N + kBN - 1) / kBN;
  p.a_mn_major = a.transA ? 1 : 0;
  p.b_mn_major = a.transB ? 1 : 0;
  p.b_batched = 0;
  // block-scaled instruction descriptor (kind::mxf8f6f4): scale-factor ids in bits 4-5 (B) and 29-30 (A)
  // are filled in per MMA; A/B formats, operand majorness (0 = K-major), N >> 3, E8M0 exponents (bit 23),
  // M >> 4 (M counts the rows of the whole CTA pair)
  p.idesc = (uint32_t(a.a_dt == SCALIFY_E5M2) << 7) | (uint32_t(a.b_dt == SCALIFY_E5M2) << 10) |
            (uint32_t(p.a_mn_major) << 15) | (uint32_t(p.b_mn_major) << 16) |
            (uint32_t(kBN >> 3) << 17) | (1u << 23) | (uint32_t(tile_m >> 4) << 24);
  p.kf = kfactor(a.K);
  p.alpha = 1.0f / p.kf;
  p.Y = a.Y; p.ldy = a.ldy; p.y_batch_stride = 0;
  p.a_scale = a.a_scale; p.b_scale = a.b_scale; p.y_scale = a.y_scale;
  p.stat = a.stat;
  p.stat_in = nullptr;
  p.stat_word = v.stat;
  p.amax_scratch = reinterpret_cast<uint32_t*>(v.stat) + 1;
  p.ticket = v.ticket;
  p.l2_partials = static_cast<double*>(v.area);
  p.status = v.status;
  p.sfa = a.sfa;
  p.bias = nullptr; p.bias_dt = 0; p.bias_scale = nullptr;
  p.sfb = a.sfb;
  p.stat_hint = nullptr;
  p.q_dt = SCALIFY_E4M3;
  p.r_pred_out = nullptr;
  p.yq_scale = nullptr; p.hint_out = nullptr; p.redo = 0;
  const long long tiles = static_cast<long long>(p.tiles_m) * p.tiles_n;
  if (tiles > (1ll << 30)) return SCALIFY_ERR_SHAPE;
  SCALIFY_DISPATCH_WIDE(a.y_dt, OUT, {
    if (ncta == 2) rc = launch_mx_variant<OUT, 2>(map_a, map_b, map_y, p, tiles, st);
    else rc = launch_mx_variant<OUT, 1>(map_a, map_b, map_y, p, tiles, st);
  });
  if (rc) return rc;
  if (a.stat == SCALIFY_STAT_L2) {
    gemm_l2_finalize_kernel<<<1, 256, 0, st>>>(p.l2_partials, static_cast<int>(tiles * ncta * 8),
                                               double(a.M) * double(a.N), v.stat);
    SCALIFY_CUDA_TRY(cudaGetLastError());
  }
  return SCALIFY_OK;
}

}  // namespace scalify
