// Block-scale quantisation (Section 2: the scale component generalised to block formats; E8M0
// exponents as in the OCP micro-scaling formats): FP8 elements plus one E8M0 exponent per 32
// consecutive elements of a row, written in the tile order the block-scaled MMA consumes.
//
// HBM-bound: a thread holds 32 bytes of input (16 elements of a 16-bit format: two lanes share a
// block; 8 fp32 elements: four lanes), the block maximum comes from one or two shuffles, every lane
// rounds its elements once and stores them, and one lane keeps the exponent byte.
#include "scalify_common.cuh"
#include "scalify_launch.h"

namespace scalify {

constexpr int kMxThreads = 256;
constexpr int kMxBlock = 32;   // elements that share an exponent
constexpr int kMxUnroll = 4;   // loads in flight per thread (32 bytes each)

// 32 bytes that are read once: one 256-bit load where the address allows it
__device__ __forceinline__ void mx_load32(const void* p, bool aligned32, uint32_t* w) {
  if (aligned32) {
    asm volatile("ld.global.cs.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
  } else {
    ld_raw_stream<32>(p, w);
  }
}

// Exponent storage: tiles of 128 rows x 4 blocks (128 elements of K), 512 bytes each, tile (r, k)
// at ((r * K/128) + k) * 512; inside a tile row `row`, block `blk` sit at byte
// (row % 32) * 16 + (row / 32) * 4 + blk.  Rows are padded up to a multiple of 256 so that a
// 256-row operand tile of the matmul never reads past the buffer.
size_t mx_sf_bytes(int64_t rows, int64_t K) {
  const int64_t padded = (rows + 255) / 256 * 256;
  return static_cast<size_t>(padded / 128) * static_cast<size_t>(K / 128) * 512;
}

// One thread block quantises a tile of 128 rows x 128 elements of K: exactly one 512-byte exponent
// tile, which is assembled in shared memory and written with 16-byte stores.  With 16-bit input a
// warp covers four rows (4 x 8 pieces of 16 elements) per step, the eight warps 32 rows, four steps the
// tile; with fp32 input half as many.  All of a thread's loads of four steps are issued before their
// first use.
template <int IN, int ELEM>
__global__ void __launch_bounds__(kMxThreads) mx_quantize_kernel(const void* __restrict__ X, int64_t ldx, int64_t rows,
                                                                 int64_t K, void* __restrict__ data,
                                                                 uint8_t* __restrict__ sf, const float* x_scale,
                                                                 float* y_scale, uint32_t* status) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int LE = 32 / ElemBytes<IN>::v;       // elements per thread: 16 or 8
  constexpr int kPieces = 128 / LE;               // threads per 128-element row segment: 8 or 16
  constexpr int kLanesPerBlock = kMxBlock / LE;   // 2 or 4
  constexpr int kRowsPerStep = kMxThreads / kPieces;
  constexpr int kGroups = 128 / kRowsPerStep / kMxUnroll;
  constexpr int kEmax = ELEM == SCALIFY_E4M3 ? 8 : 15;
  __shared__ __align__(16) uint8_t s_sf[512];
  const int64_t k_tile = blockIdx.x, r_tile = blockIdx.y;
  const int piece = threadIdx.x % kPieces;
  const int row_in_step = threadIdx.x / kPieces;
  const int64_t col0 = k_tile * 128 + piece * LE;
  const bool aligned32 = ((reinterpret_cast<uintptr_t>(X) | static_cast<uintptr_t>(ldx * ElemBytes<IN>::v)) & 31) == 0;
#pragma unroll
  for (int g = 0; g < kGroups; ++g) {
    uint32_t w[kMxUnroll][8];
#pragma unroll
    for (int u = 0; u < kMxUnroll; ++u) {
      const int64_t row = r_tile * 128 + (g * kMxUnroll + u) * kRowsPerStep + row_in_step;
#pragma unroll
      for (int q = 0; q < 8; ++q) w[u][q] = 0u;
      if (row < rows)
        mx_load32(static_cast<const char*>(X) + (row * ldx + col0) * ElemBytes<IN>::v, aligned32, w[u]);
    }
#pragma unroll
    for (int u = 0; u < kMxUnroll; ++u) {
      const int lrow = (g * kMxUnroll + u) * kRowsPerStep + row_in_step;  // row inside the tile
      const int64_t row = r_tile * 128 + lrow;
      float f[LE];
      decode_vec<IN, LE>(w[u], f);
      uint32_t amax = 0u;
      if constexpr (ElemBytes<IN>::v == 2) {
        // the 15 magnitude bits of a 16-bit float order like the magnitudes: maximum on the packed halves,
        // widened to the fp32 pattern afterwards (exact)
        uint32_t m2 = 0u;
#pragma unroll
        for (int q = 0; q < 8; ++q) m2 = __vmaxu2(m2, w[u][q] & 0x7FFF7FFFu);
        amax = max(m2 & 0xFFFFu, m2 >> 16);
      } else {
#pragma unroll
        for (int e = 0; e < LE; ++e) amax = max(amax, abs_bits(f[e]));
      }
#pragma unroll
      for (int m = 1; m < kLanesPerBlock; m <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, m));
      if constexpr (IN == SCALIFY_BF16) amax <<= 16;
      if constexpr (IN == SCALIFY_F16)
        amax = __float_as_uint(__half2float(__ushort_as_half(static_cast<unsigned short>(amax))));
      // shared exponent: floor(log2(amax)) - emax of the element format; 0 for a block whose maximum is
      // zero, infinite or NaN (abs_bits orders NaN above infinity, so one comparison covers both)
      int e = 0;
      if (amax != 0u && amax < 0x7F800000u) {
        int ex = static_cast<int>(amax >> 23) - 127;              // normal numbers
        if ((amax >> 23) == 0u) ex = -127 - __clz(amax << 9);      // fp32 subnormal: leading one of the mantissa
        e = ex - kEmax;
        e = max(-127, min(127, e));
      }
      if (row < rows) {
        // multiply by 2^-e, exactly: 2^-127 is the subnormal 0x00400000, every other factor is normal
        const uint32_t field = static_cast<uint32_t>(127 - e);
        const float s = __uint_as_float(field ? field << 23 : 0x00400000u);
#pragma unroll
        for (int t = 0; t < LE; ++t) f[t] *= s;
        uint32_t o[LE / 4];
        encode_vec<ELEM, LE>(f, o);
        st_raw<LE>(static_cast<char*>(data) + row * K + col0, o);
      }
      if (piece % kLanesPerBlock == 0)
        s_sf[(lrow & 31) * 16 + (lrow >> 5) * 4 + piece / kLanesPerBlock] = static_cast<uint8_t>(e + 127);
    }
  }
  __syncthreads();
  if (threadIdx.x < 32)
    reinterpret_cast<uint4*>(sf + (r_tile * gridDim.x + k_tile) * 512)[threadIdx.x] =
        reinterpret_cast<const uint4*>(s_sf)[threadIdx.x];
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
    const float xs = load_scale(x_scale);
    if (y_scale) *y_scale = xs;  // the tensor-wide scale is untouched: the exponents belong to the data
    if (!is_pow2_scale(xs) && status) atomicOr(status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
  }
}

// The same quantisation for an operand stored TRANSPOSED: X and the data are [K, rows] (row-major, `rows`
// contiguous), and a block is 32 consecutive elements of K = 32 consecutive ROWS of the storage at one column.
// This is the form a backward matmul needs (the contraction runs over the dimension that is not contiguous in the
// forward tensors); the matmul then consumes the data MN-major, so no transposed copy exists.  The exponent tiles
// are the same as for the plain form: tile (r, k) holds operand rows r*128..+127 (columns of the storage here)
// and the four blocks of K-rows k*128..+127.
// One thread block of 512 threads quantises 128 K-rows x 128 columns (one exponent tile).  Warp w takes the
// 32 K-rows of block w / 4 and the 32 columns of quarter w % 4; a lane takes 4 rows x 8 columns, the column
// maxima of the eight lanes that share a column come from three shuffles.  The raw words stay in registers
// and are decoded twice (once for the maxima, once for the scaling): the small per-thread state is what
// keeps enough blocks on an SM to cover the load latency.
constexpr int kMxTThreads = 512;
#ifndef SCALIFY_MXT_BLOCKS
#define SCALIFY_MXT_BLOCKS 3
#endif
template <int IN, int ELEM>
__global__ void __launch_bounds__(kMxTThreads, ElemBytes<IN>::v == 4 ? 2 : SCALIFY_MXT_BLOCKS) mx_quantize_t_kernel(
    const void* __restrict__ X, int64_t ldx, int64_t rows, int64_t K, void* __restrict__ data, int64_t ldd,
    uint8_t* __restrict__ sf, const float* x_scale, float* y_scale, uint32_t* status) {
  asm volatile("griddepcontrol.launch_dependents;");  // a programmatic dependent may set up while this grid runs
  constexpr int ES = ElemBytes<IN>::v;
  constexpr int kEmax = ELEM == SCALIFY_E4M3 ? 8 : 15;
  __shared__ __align__(16) uint8_t s_sf[512];
  // consecutive blocks walk along the contiguous axis of the storage (operand rows), as the plain form's do
  const int64_t k_tile = blockIdx.y, r_tile = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blk = warp >> 2, quarter = warp & 3;
  const int cg = lane & 3, rq = lane >> 2;
  const int64_t col0 = r_tile * 128 + quarter * 32 + cg * 8;         // first of this lane's 8 columns (operand rows)
  const int64_t krow0 = k_tile * 128 + blk * 32 + rq * 4;            // first of this lane's 4 K-rows
  const bool in_cols = col0 < rows;                                   // rows is a multiple of 8: whole vector or nothing
  uint32_t w[4][8 * ES / 4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
#pragma unroll
    for (int q = 0; q < 8 * ES / 4; ++q) w[r][q] = 0u;
    if (in_cols) ld_raw_stream<8 * ES>(static_cast<const char*>(X) + ((krow0 + r) * ldx + col0) * ES, w[r]);
  }
  // Column maxima over the block's 32 K-rows as a butterfly over the eight lanes that share the columns: each
  // exchange halves the number of columns a lane still carries, so that lane rq ends with the complete maximum
  // of column rq alone and computes ONE exponent.  Magnitudes are compared as unsigned integers on the raw bit
  // patterns (monotone for every input format; 16-bit inputs two columns per word).
  const bool b2 = (lane & 16) != 0, b1 = (lane & 8) != 0, b0 = (lane & 4) != 0;
  uint32_t amax;  // fp32 bit pattern of |x| max of column rq
  if constexpr (ES == 2) {
    uint32_t pm[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int q = 0; q < 4; ++q) pm[q] = __vmaxu2(pm[q], w[r][q] & 0x7FFF7FFFu);
    uint32_t k0 = b2 ? pm[2] : pm[0], k1 = b2 ? pm[3] : pm[1];
    k0 = __vmaxu2(k0, __shfl_xor_sync(0xFFFFFFFFu, b2 ? pm[0] : pm[2], 16));
    k1 = __vmaxu2(k1, __shfl_xor_sync(0xFFFFFFFFu, b2 ? pm[1] : pm[3], 16));
    uint32_t k = __vmaxu2(b1 ? k1 : k0, __shfl_xor_sync(0xFFFFFFFFu, b1 ? k0 : k1, 8));
    k = __vmaxu2(k, __shfl_xor_sync(0xFFFFFFFFu, k, 4));
    const uint32_t own = b0 ? (k >> 16) : (k & 0xFFFFu);
    if constexpr (IN == SCALIFY_BF16) amax = own << 16;
    else amax = __float_as_uint(__half2float(__ushort_as_half(static_cast<unsigned short>(own))));
  } else {
    uint32_t cm[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) cm[c] = 0u;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 8; ++c) cm[c] = max(cm[c], w[r][c] & 0x7FFFFFFFu);
    uint32_t a4[4], a2[2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      a4[i] = max(b2 ? cm[4 + i] : cm[i], __shfl_xor_sync(0xFFFFFFFFu, b2 ? cm[i] : cm[4 + i], 16));
#pragma unroll
    for (int i = 0; i < 2; ++i)
      a2[i] = max(b1 ? a4[2 + i] : a4[i], __shfl_xor_sync(0xFFFFFFFFu, b1 ? a4[i] : a4[2 + i], 8));
    amax = max(b0 ? a2[1] : a2[0], __shfl_xor_sync(0xFFFFFFFFu, b0 ? a2[0] : a2[1], 4));
  }
  // shared exponent: floor(log2(amax)) - emax of the element format; 0 for a block whose maximum is zero,
  // infinite or NaN
  int e = 0;
  if (amax != 0u && amax < 0x7F800000u) {
    int ex = static_cast<int>(amax >> 23) - 127;
    if ((amax >> 23) == 0u) ex = -127 - __clz(amax << 9);
    e = max(-127, min(127, ex - kEmax));
  }
  // the eight exponent bytes of the lane's columns, gathered by the reverse butterfly (byte c = column c)
  uint32_t ebytes[2];
  {
    uint32_t v = static_cast<uint32_t>(e + 127), o;
    o = __shfl_xor_sync(0xFFFFFFFFu, v, 4);
    v = b0 ? (o | (v << 8)) : (v | (o << 8));
    o = __shfl_xor_sync(0xFFFFFFFFu, v, 8);
    v = b1 ? (o | (v << 16)) : (v | (o << 16));
    o = __shfl_xor_sync(0xFFFFFFFFu, v, 16);
    ebytes[0] = b2 ? o : v;
    ebytes[1] = b2 ? v : o;
  }
  float sc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    // 2^-e exactly: e <= 127 - emax (a finite maximum has an exponent of at most 127), so the field 127 - e of
    // the power of two is never zero
    const uint32_t byte = (ebytes[c >> 2] >> (8 * (c & 3))) & 0xFFu;
    sc[c] = __uint_as_float((254u - byte) << 23);
  }
  if (in_cols) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      float g[8];
      decode_vec<IN, 8>(w[r], g);
#pragma unroll
      for (int c = 0; c < 8; ++c) g[c] *= sc[c];
      uint32_t o[2];
      encode_vec<ELEM, 8>(g, o);
      st_raw<8>(static_cast<char*>(data) + (krow0 + r) * ldd + col0, o);
    }
  }
  if (rq == 0) {
    // operand row m = quarter*32 + cg*8 + c of the tile, block blk: byte (m % 32) * 16 + (m / 32) * 4 + blk
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int m = quarter * 32 + cg * 8 + c;
      s_sf[(m & 31) * 16 + (m >> 5) * 4 + blk] = static_cast<uint8_t>((ebytes[c >> 2] >> (8 * (c & 3))) & 0xFFu);
    }
  }
  __syncthreads();
  if (threadIdx.x < 32)
    reinterpret_cast<uint4*>(sf + (r_tile * (K >> 7) + k_tile) * 512)[threadIdx.x] =
        reinterpret_cast<const uint4*>(s_sf)[threadIdx.x];
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
    const float xs = load_scale(x_scale);
    if (y_scale) *y_scale = xs;
    if (!is_pow2_scale(xs) && status) atomicOr(status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
  }
}

int launch_mx_quantize_t(const void* X, int x_dt, int64_t rows, int64_t K, int64_t ldx, void* data, int elem_dt,
                         uint8_t* sf, const float* x_scale, float* y_scale, uint32_t* status, cudaStream_t st) {
  const int64_t r_tiles = (rows + 255) / 256 * 2;  // 128-row tiles of the operand, padding rows included
  if (K / 128 > 65535) return SCALIFY_ERR_SHAPE;
  const dim3 grid(static_cast<unsigned>(r_tiles), static_cast<unsigned>(K / 128));
#define SCALIFY_MXT_LAUNCH(ELEM) \
  mx_quantize_t_kernel<IN, ELEM><<<grid, kMxTThreads, 0, st>>>(X, ldx, rows, K, data, rows, sf, x_scale, y_scale, status)
  SCALIFY_DISPATCH_WIDE(x_dt, IN, {
    if (elem_dt == SCALIFY_E4M3) SCALIFY_MXT_LAUNCH(SCALIFY_E4M3);
    else SCALIFY_MXT_LAUNCH(SCALIFY_E5M2);
  });
#undef SCALIFY_MXT_LAUNCH
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

int launch_mx_quantize(const void* X, int x_dt, int64_t rows, int64_t K, int64_t ldx, void* data, int elem_dt,
                       uint8_t* sf, const float* x_scale, float* y_scale, uint32_t* status, cudaStream_t st) {
  const int64_t r_tiles = (rows + 255) / 256 * 2;  // 128-row tiles, padding rows included
  if (r_tiles > 65535) return SCALIFY_ERR_SHAPE;
  const dim3 grid(static_cast<unsigned>(K / 128), static_cast<unsigned>(r_tiles));
#define SCALIFY_MX_LAUNCH(ELEM) \
  mx_quantize_kernel<IN, ELEM><<<grid, kMxThreads, 0, st>>>(X, ldx, rows, K, data, sf, x_scale, y_scale, status)
  SCALIFY_DISPATCH_WIDE(x_dt, IN, {
    if (elem_dt == SCALIFY_E4M3) SCALIFY_MX_LAUNCH(SCALIFY_E4M3);
    else SCALIFY_MX_LAUNCH(SCALIFY_E5M2);
  });
#undef SCALIFY_MX_LAUNCH
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

}  // namespace scalify
