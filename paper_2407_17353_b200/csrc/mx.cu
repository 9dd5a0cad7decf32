// Block-scale quantisation (Section 2: the scale component generalised to block formats; E8M0
// exponents as in the OCP micro-scaling formats): FP8 elements plus one E8M0 exponent per 32
// consecutive elements of a row, written in the tile order the block-scaled MMA consumes.
//
// HBM-bound: four lanes share a block (8 elements = one 16-byte vector of 16-bit input per lane),
// the block maximum comes from two shuffles, every lane rounds its 8 elements once and stores
// 8 bytes, and one lane keeps the exponent byte.
#include "scalify_common.cuh"
#include "scalify_launch.h"

namespace scalify {

constexpr int kMxThreads = 256;
constexpr int kMxBlock = 32;   // elements that share an exponent
constexpr int kMxLaneElems = 8;
constexpr int kMxUnroll = 4;   // loads in flight per thread

// Exponent storage: tiles of 128 rows x 4 blocks (128 elements of K), 512 bytes each, tile (r, k)
// at ((r * K/128) + k) * 512; inside a tile row `row`, block `blk` sit at byte
// (row % 32) * 16 + (row / 32) * 4 + blk.  Rows are padded up to a multiple of 256 so that a
// 256-row operand tile of the matmul never reads past the buffer.
size_t mx_sf_bytes(int64_t rows, int64_t K) {
  const int64_t padded = (rows + 255) / 256 * 256;
  return static_cast<size_t>(padded / 128) * static_cast<size_t>(K / 128) * 512;
}

// One thread block quantises a tile of 128 rows x 128 elements of K: exactly one 512-byte exponent
// tile, which is assembled in shared memory and written with 16-byte stores.  A warp covers two rows
// (2 x 16 pieces of 8 elements) per step, the eight warps 16 rows, eight steps the tile; all of a
// thread's loads of four steps are issued before their first use.
template <int IN, int ELEM>
__global__ void __launch_bounds__(kMxThreads) mx_quantize_kernel(const void* __restrict__ X, int64_t ldx, int64_t rows,
                                                                 int64_t K, void* __restrict__ data,
                                                                 uint8_t* __restrict__ sf, const float* x_scale,
                                                                 float* y_scale, uint32_t* status) {
  constexpr int IB = kMxLaneElems * ElemBytes<IN>::v;  // 16 (16-bit input) or 32 (fp32 input)
  constexpr int kEmax = ELEM == SCALIFY_E4M3 ? 8 : 15;
  __shared__ __align__(16) uint8_t s_sf[512];
  const int64_t k_tile = blockIdx.x, r_tile = blockIdx.y;
  const int piece = threadIdx.x & 15;        // 8-element piece of the 128-element row segment
  const int row_in_step = threadIdx.x >> 4;  // 0..15
  const int64_t col0 = k_tile * 128 + piece * kMxLaneElems;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    uint32_t w[kMxUnroll][IB / 4];
#pragma unroll
    for (int u = 0; u < kMxUnroll; ++u) {
      const int64_t row = r_tile * 128 + (half * kMxUnroll + u) * 16 + row_in_step;
#pragma unroll
      for (int q = 0; q < IB / 4; ++q) w[u][q] = 0u;
      if (row < rows) ld_raw_stream<IB>(static_cast<const char*>(X) + (row * ldx + col0) * ElemBytes<IN>::v, w[u]);
    }
#pragma unroll
    for (int u = 0; u < kMxUnroll; ++u) {
      const int lrow = (half * kMxUnroll + u) * 16 + row_in_step;  // row inside the tile
      const int64_t row = r_tile * 128 + lrow;
      float f[kMxLaneElems];
      decode_vec<IN, kMxLaneElems>(w[u], f);
      uint32_t amax = 0u;
#pragma unroll
      for (int e = 0; e < kMxLaneElems; ++e) amax = max(amax, abs_bits(f[e]));
      amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
      amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
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
        // multiply by 2^-e exactly (two steps keep each factor a normal fp32 for every e in [-127, 127])
        const int h = (-e) / 2;
        const float s1 = __uint_as_float(static_cast<uint32_t>(h + 127) << 23);
        const float s2 = __uint_as_float(static_cast<uint32_t>((-e - h) + 127) << 23);
#pragma unroll
        for (int t = 0; t < kMxLaneElems; ++t) f[t] = f[t] * s1 * s2;
        uint32_t o[2];
        encode_vec<ELEM, kMxLaneElems>(f, o);
        st_raw<8>(static_cast<char*>(data) + row * K + col0, o);
      }
      if ((piece & 3) == 0) s_sf[(lrow & 31) * 16 + (lrow >> 5) * 4 + (piece >> 2)] = static_cast<uint8_t>(e + 127);
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
