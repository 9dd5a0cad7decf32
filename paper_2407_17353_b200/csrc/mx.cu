// Block-scale quantisation (Section 2: the scale component generalised to block formats; E8M0
// exponents as in the OCP micro-scaling formats): FP8 elements plus one E8M0 exponent per 32
// consecutive elements of a row, written in the tile order the block-scaled MMA consumes.
//
// HBM-bound: four lanes share a block (8 elements = one 16-byte vector of 16-bit input per lane),
// the block maximum comes from two shuffles, every lane rounds its 8 elements once and stores
// 8 bytes, and one lane stores the exponent byte.  One block of 256 threads covers 64 blocks of
// 32 elements; the grid holds one such piece per thread block.
#include "scalify_common.cuh"
#include "scalify_launch.h"

namespace scalify {

constexpr int kMxThreads = 256;
constexpr int kMxBlock = 32;   // elements that share an exponent
constexpr int kMxLaneElems = 8;

// Exponent storage: tiles of 128 rows x 4 blocks (128 elements of K), 512 bytes each, tile (r, k)
// at ((r * K/128) + k) * 512; inside a tile row `row`, block `blk` sit at byte
// (row % 32) * 16 + (row / 32) * 4 + blk.  Rows are padded up to a multiple of 256 so that a
// 256-row operand tile of the matmul never reads past the buffer.
size_t mx_sf_bytes(int64_t rows, int64_t K) {
  const int64_t padded = (rows + 255) / 256 * 256;
  return static_cast<size_t>(padded / 128) * static_cast<size_t>(K / 128) * 512;
}

__device__ __forceinline__ int64_t mx_sf_offset(int64_t row, int64_t blk, int64_t k_tiles) {
  return ((row >> 7) * k_tiles + (blk >> 2)) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + (blk & 3);
}

template <int IN, int ELEM>
__global__ void __launch_bounds__(kMxThreads) mx_quantize_kernel(const void* __restrict__ X, int64_t ldx, int64_t rows,
                                                                 int64_t K, void* __restrict__ data,
                                                                 uint8_t* __restrict__ sf, const float* x_scale,
                                                                 float* y_scale, uint32_t* status) {
  constexpr int IB = kMxLaneElems * ElemBytes<IN>::v;  // 16 (16-bit input) or 32 (fp32 input)
  constexpr int kEmax = ELEM == SCALIFY_E4M3 ? 8 : 15;
  const int64_t lanes_per_row = K / kMxLaneElems;
  const int64_t k_tiles = K / 128;
  const int64_t padded_rows = (rows + 255) / 256 * 256;
  const int64_t total = padded_rows * lanes_per_row;
  const int64_t i = int64_t(blockIdx.x) * kMxThreads + threadIdx.x;
  // rows and K/8 are such that a group of four lanes never straddles the end (K % 32 == 0)
  const bool in_range = i < total;
  const int64_t row = in_range ? i / lanes_per_row : 0;
  const int64_t piece = in_range ? i - row * lanes_per_row : 0;
  const bool real = in_range && row < rows;
  float f[kMxLaneElems];
#pragma unroll
  for (int e = 0; e < kMxLaneElems; ++e) f[e] = 0.f;
  if (real) {
    uint32_t w[IB / 4];
    ld_raw_stream<IB>(static_cast<const char*>(X) + (row * ldx + piece * kMxLaneElems) * ElemBytes<IN>::v, w);
    decode_vec<IN, kMxLaneElems>(w, f);
  }
  uint32_t amax = 0u;
#pragma unroll
  for (int e = 0; e < kMxLaneElems; ++e) amax = max(amax, abs_bits(f[e]));
  amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
  amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
  // shared exponent: floor(log2(amax)) - emax of the element format; 0 for a block whose maximum is zero,
  // infinite or NaN (abs_bits orders NaN above infinity, so one comparison covers both)
  int e = 0;
  if (amax != 0u && amax < 0x7F800000u) {
    int ex = static_cast<int>(amax >> 23) - 127;              // normal numbers
    if ((amax >> 23) == 0u) ex = -127 - __clz(amax << 9);      // fp32 subnormal: leading one of the mantissa
    e = ex - kEmax;
    e = max(-127, min(127, e));
  }
  if (real) {
    // multiply by 2^-e exactly (two steps keep the factor a normal fp32 for every e in [-127, 127])
    const int h = (-e) / 2;
    const float s1 = __uint_as_float(static_cast<uint32_t>(h + 127) << 23);
    const float s2 = __uint_as_float(static_cast<uint32_t>((-e - h) + 127) << 23);
#pragma unroll
    for (int t = 0; t < kMxLaneElems; ++t) f[t] = f[t] * s1 * s2;
    uint32_t o[2];
    encode_vec<ELEM, kMxLaneElems>(f, o);
    st_raw<8>(static_cast<char*>(data) + row * K + piece * kMxLaneElems, o);
  }
  if (in_range && (piece & 3) == 0) sf[mx_sf_offset(row, piece >> 2, k_tiles)] = static_cast<uint8_t>(e + 127);
  if (i == 0) {
    const float xs = load_scale(x_scale);
    if (y_scale) *y_scale = xs;  // the tensor-wide scale is untouched: the exponents belong to the data
    if (!is_pow2_scale(xs) && status) atomicOr(status, static_cast<uint32_t>(SCALIFY_DEV_BAD_SCALE));
  }
}

int launch_mx_quantize(const void* X, int x_dt, int64_t rows, int64_t K, int64_t ldx, void* data, int elem_dt,
                       uint8_t* sf, const float* x_scale, float* y_scale, uint32_t* status, cudaStream_t st) {
  const int64_t padded_rows = (rows + 255) / 256 * 256;
  const int64_t total = padded_rows * (K / kMxLaneElems);
  const int64_t grid = (total + kMxThreads - 1) / kMxThreads;
  if (grid > 0x7FFFFFFF) return SCALIFY_ERR_SHAPE;
#define SCALIFY_MX_LAUNCH(ELEM)                                                                              \
  mx_quantize_kernel<IN, ELEM><<<static_cast<unsigned>(grid), kMxThreads, 0, st>>>(X, ldx, rows, K, data, sf, \
                                                                                  x_scale, y_scale, status)
  SCALIFY_DISPATCH_WIDE(x_dt, IN, {
    if (elem_dt == SCALIFY_E4M3) SCALIFY_MX_LAUNCH(SCALIFY_E4M3);
    else SCALIFY_MX_LAUNCH(SCALIFY_E5M2);
  });
#undef SCALIFY_MX_LAUNCH
  SCALIFY_CUDA_TRY(cudaGetLastError());
  return SCALIFY_OK;
}

}  // namespace scalify
