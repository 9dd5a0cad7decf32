// Shared device/host helpers of the scaled-array kernels: number-format
// conversion, power-of-two arithmetic on fp32 bit patterns, workspace header
// layout and argument validation.
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <stdint.h>

#include <mutex>

#include "scalify.h"

namespace scalify {

// ---------------------------------------------------------------- workspace header
// byte 0   : uint32 status bits (SCALIFY_DEV_*)
// byte 16  : fp32 statistic word (bit pattern is also used for atomicMax)
// byte 20  : scratch word of the matmul's fused AMAX (atomicMax target; zero between launches)
// byte 32  : uint32 ticket of the "last block finishes" reductions (self-resetting)
// byte 48  : fp32 scale word of an output whose caller passed no scale pointer
// byte 52  : fp32 rescale factor a speculative matmul predicted
// byte 56  : fp32 AMAX of the last matmul + FP8 rescale on this workspace (the next call's prediction)
// byte 64  : (Adam) not used
// byte 256 : operation-specific area
constexpr size_t kWsStatus = 0;
constexpr size_t kWsStat = 16;
constexpr size_t kWsTicket = 32;
constexpr size_t kWsHeader = 256;
constexpr size_t kWsMin = 4096;

struct WsView {
  uint32_t* status;
  float* stat;
  uint32_t* ticket;
  void* area;
};

inline WsView ws_view(void* ws) {
  char* p = static_cast<char*>(ws);
  return WsView{reinterpret_cast<uint32_t*>(p + kWsStatus), reinterpret_cast<float*>(p + kWsStat),
                reinterpret_cast<uint32_t*>(p + kWsTicket), p + kWsHeader};
}

// ---------------------------------------------------------------- programmatic dependent launch
// Every kernel of the library begins with `griddepcontrol.launch_dependents`, so a grid that follows it in
// the stream AND was launched as a programmatic dependent (the matmul kernels are: their prologue of barrier
// set-up, TMEM allocation and cluster synchronisation touches no global memory) may be scheduled while it
// still runs.  Such a dependent executes `griddepcontrol.wait` before its first access to global memory;
// only from there on are the writes of the grid before it complete and visible.  For an ordinary launch
// both instructions do nothing.

// ---------------------------------------------------------------- host side helpers
inline int elem_size(int dt) { return dt <= SCALIFY_E5M2 ? 1 : (dt == SCALIFY_F32 ? 4 : 2); }
inline bool valid_dtype(int dt) { return dt >= SCALIFY_E4M3 && dt <= SCALIFY_F32; }
inline bool is_fp8(int dt) { return dt == SCALIFY_E4M3 || dt == SCALIFY_E5M2; }
inline bool is_wide(int dt) { return dt == SCALIFY_F16 || dt == SCALIFY_BF16 || dt == SCALIFY_F32; }

// Total element count of a contiguous array, or -1 if it is not contiguous / malformed.
int64_t contiguous_numel(const scalify_array* a);
// Checks pointer, dtype, ndim, innermost stride and 16-byte alignment of data and outer strides.
int check_array(const scalify_array* a);
int sm_count();
void set_last_cuda_error(int e);
int cuda_fail(cudaError_t e);

// One-time set-up of a kernel PER DEVICE.  Function attributes (the dynamic shared-memory limit) and occupancy
// figures belong to a device, not to the process: a process that uses the library on a second GPU has to set
// them again there.  `fn(int* value)` runs once per device, with that device current, under a lock (so two host
// threads cannot both believe the other did it); `value` is what it computed for that device (e.g. the number
// of co-resident clusters), handed back on every later call.
constexpr int kMaxDevices = 64;
struct DeviceOnce {
  std::mutex mu;
  bool done[kMaxDevices] = {};
  int value[kMaxDevices] = {};
};
template <class Fn>
inline int device_once_at(DeviceOnce& o, int dev, int* value_out, Fn fn) {
  if (dev < 0 || dev >= kMaxDevices) return SCALIFY_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(o.mu);
  if (!o.done[dev]) {
    int rc = fn(&o.value[dev]);
    if (rc) return rc;
    o.done[dev] = true;
  }
  if (value_out) *value_out = o.value[dev];
  return SCALIFY_OK;
}
template <class Fn>
inline int device_once(DeviceOnce& o, int* value_out, Fn fn) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SCALIFY_ERR_CUDA;
  return device_once_at(o, dev, value_out, fn);
}

#define SCALIFY_CUDA_TRY(expr)                               \
  do {                                                       \
    cudaError_t e__ = (expr);                                \
    if (e__ != cudaSuccess) return ::scalify::cuda_fail(e__); \
  } while (0)

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// scale word or 1 (Section 3.1: an unscaled array unbundles to (x, 1))
// A scale word is usually written by the kernel just before this one.  In an ordinary launch the read-only path
// is right for it (every thread of thousands of blocks reads the same word: it has to be served by the L1s).
__device__ __forceinline__ float load_scale(const float* s) { return s ? __ldg(s) : 1.0f; }
// In a kernel launched as a PROGRAMMATIC DEPENDENT, after its `griddepcontrol.wait`: a load through the read-only
// path counts as invariant and may be scheduled above the wait, where it would see the word's previous content;
// this one is volatile (use it from few threads: it goes to the L2 every time).
__device__ __forceinline__ float load_scale_after_wait(const float* s) {
  return s ? *reinterpret_cast<const volatile float*>(s) : 1.0f;
}

__device__ __forceinline__ bool is_pow2_scale(float s) {
  uint32_t b = __float_as_uint(s);
  uint32_t e = b >> 23;  // sign must be 0, so e is the exponent field
  return (b & 0x807FFFFFu) == 0u && e >= 1u && e <= 253u;
}

// largest power of two <= x for a normal positive fp32 (Section 3.2: scales round down)
__device__ __forceinline__ float p2_floor(float x) { return __uint_as_float(__float_as_uint(x) & 0x7F800000u); }

// Rebalancing factor of a dynamic rescale: r = p2_floor(stat), or 1 when the statistic cannot
// define a scale (zero, subnormal, Inf, NaN).  `nonfinite` reports Inf/NaN.
__device__ __forceinline__ float rescale_factor(float stat, bool* nonfinite) {
  uint32_t b = __float_as_uint(stat) & 0x7FFFFFFFu;
  uint32_t e = b >> 23;
  *nonfinite = (e == 255u);
  if (e == 0u || e == 255u) return 1.0f;
  return __uint_as_float(b & 0x7F800000u);
}

// sqrt(K) rounded down to a power of two: 2^(floor(log2 K) div 2)
__host__ __device__ __forceinline__ float kfactor(long long K) {
  int l = 0;
  while ((1ll << (l + 1)) <= K) ++l;
  int e = l / 2;
  float f = 1.0f;
  for (int i = 0; i < e; ++i) f *= 2.0f;
  return f;
}

// p2_floor(sqrt(s)) for a power of two s: halve the exponent, rounding toward -inf
__device__ __forceinline__ float p2_sqrt_floor(float s) {
  int e = static_cast<int>((__float_as_uint(s) >> 23) & 0xFFu) - 127;
  int h = (e >= 0) ? (e / 2) : -((-e + 1) / 2);
  return __uint_as_float(static_cast<uint32_t>(h + 127) << 23);
}

template <int DT> struct ElemBytes { static constexpr int v = (DT <= SCALIFY_E5M2) ? 1 : (DT == SCALIFY_F32 ? 4 : 2); };

// ---- vector load of N consecutive elements (N*size bytes, naturally aligned) into fp32
// ---------------------------------------------------------------------------------------------
// Debug build (-DSCALIFY_DEBUG): every global access that goes through the helpers below (vector loads and
// stores, the asynchronous row copies, the scalar tail accesses) is checked against the byte ranges of the
// arrays the host has registered (every scalify_array an entry point validates).  An access outside all of
// them is counted, its address recorded, and SKIPPED (a load yields zeros), so nothing faults.  The table
// lives in one translation unit; every other one holds a pointer to it that the host sets before first use.
// ---------------------------------------------------------------------------------------------
#ifdef SCALIFY_DEBUG
constexpr int kDbgMaxRanges = 4096;
struct DbgTable {
  unsigned long long lo[kDbgMaxRanges], hi[kDbgMaxRanges];  // sorted by lo, disjoint
  int n;
  unsigned long long violations, first_addr, first_bytes;
};
static __device__ DbgTable* g_dbg_table = nullptr;
__device__ __forceinline__ bool dbg_ok(const void* p, int bytes) {
  const DbgTable* t = g_dbg_table;
  if (!t || !__isGlobal(p)) return true;  // (the helpers also read parameters staged in shared memory)
  const unsigned long long a = reinterpret_cast<unsigned long long>(p);
  int l = 0, r = t->n;  // last range whose lo <= a
  while (l < r) {
    const int m = (l + r) >> 1;
    if (t->lo[m] <= a) l = m + 1; else r = m;
  }
  if (l > 0 && a + static_cast<unsigned long long>(bytes) <= t->hi[l - 1]) return true;
  DbgTable* w = g_dbg_table;
  if (atomicAdd(&w->violations, 1ull) == 0ull) { w->first_addr = a; w->first_bytes = static_cast<unsigned long long>(bytes); }
  return false;
}
// host side (support.cu): registration of a translation unit's pointer, of an array's byte range, report
typedef cudaError_t (*DbgSetPointerFn)(DbgTable*);
void dbg_add_translation_unit(DbgSetPointerFn fn);
void dbg_register_range(const void* base, unsigned long long bytes);
namespace {
struct DbgTranslationUnit {
  DbgTranslationUnit() {
    dbg_add_translation_unit([](DbgTable* t) { return cudaMemcpyToSymbol(g_dbg_table, &t, sizeof(t)); });
  }
} g_dbg_translation_unit;
}  // namespace
#define SCALIFY_DBG_CHECK_LOAD(p, bytes, words)                      \
  if (!dbg_ok(p, bytes)) {                                          \
    for (int dbg_i = 0; dbg_i < (words); ++dbg_i) w[dbg_i] = 0u;    \
    return;                                                         \
  }
#define SCALIFY_DBG_CHECK_STORE(p, bytes) \
  if (!dbg_ok(p, bytes)) return;
#else
#define SCALIFY_DBG_CHECK_LOAD(p, bytes, words)
#define SCALIFY_DBG_CHECK_STORE(p, bytes)
#endif

template <int BYTES> struct RawVec;
template <> struct RawVec<4> { uint32_t w[1]; };
template <> struct RawVec<8> { uint32_t w[2]; };
template <> struct RawVec<16> { uint32_t w[4]; };
template <> struct RawVec<32> { uint32_t w[8]; };
template <> struct RawVec<2> { uint16_t h; };

template <int BYTES>
__device__ __forceinline__ void ld_raw(const void* p, uint32_t* w) {
  SCALIFY_DBG_CHECK_LOAD(p, BYTES, BYTES / 4)
  if constexpr (BYTES == 16) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
  } else if constexpr (BYTES == 32) {
    uint4 v0 = reinterpret_cast<const uint4*>(p)[0];
    uint4 v1 = reinterpret_cast<const uint4*>(p)[1];
    w[0] = v0.x; w[1] = v0.y; w[2] = v0.z; w[3] = v0.w;
    w[4] = v1.x; w[5] = v1.y; w[6] = v1.z; w[7] = v1.w;
  } else if constexpr (BYTES == 8) {
    uint2 v = *reinterpret_cast<const uint2*>(p);
    w[0] = v.x; w[1] = v.y;
  } else {
    static_assert(BYTES == 4, "unsupported vector width");
    w[0] = *reinterpret_cast<const uint32_t*>(p);
  }
}

template <int BYTES>
__device__ __forceinline__ void st_raw(void* p, const uint32_t* w) {
  SCALIFY_DBG_CHECK_STORE(p, BYTES)
  if constexpr (BYTES == 16) {
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  } else if constexpr (BYTES == 32) {
    reinterpret_cast<uint4*>(p)[0] = make_uint4(w[0], w[1], w[2], w[3]);
    reinterpret_cast<uint4*>(p)[1] = make_uint4(w[4], w[5], w[6], w[7]);
  } else if constexpr (BYTES == 8) {
    *reinterpret_cast<uint2*>(p) = make_uint2(w[0], w[1]);
  } else {
    static_assert(BYTES == 4, "unsupported vector width");
    *reinterpret_cast<uint32_t*>(p) = w[0];
  }
}

// streaming variants (read-once / write-once data: do not keep in L1)
template <int BYTES>
__device__ __forceinline__ void ld_raw_stream(const void* p, uint32_t* w) {
  SCALIFY_DBG_CHECK_LOAD(p, BYTES, BYTES / 4)
  if constexpr (BYTES == 16) {
    uint4 v = __ldcs(reinterpret_cast<const uint4*>(p));
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
  } else if constexpr (BYTES == 32) {
    uint4 v0 = __ldcs(reinterpret_cast<const uint4*>(p));
    uint4 v1 = __ldcs(reinterpret_cast<const uint4*>(p) + 1);
    w[0] = v0.x; w[1] = v0.y; w[2] = v0.z; w[3] = v0.w;
    w[4] = v1.x; w[5] = v1.y; w[6] = v1.z; w[7] = v1.w;
  } else if constexpr (BYTES == 8) {
    uint2 v = __ldcs(reinterpret_cast<const uint2*>(p));
    w[0] = v.x; w[1] = v.y;
  } else {
    w[0] = __ldcs(reinterpret_cast<const uint32_t*>(p));
  }
}

template <int BYTES>
__device__ __forceinline__ void st_raw_stream(void* p, const uint32_t* w) {
  SCALIFY_DBG_CHECK_STORE(p, BYTES)
  if constexpr (BYTES == 16) {
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
  } else if constexpr (BYTES == 32) {
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
    __stcs(reinterpret_cast<uint4*>(p) + 1, make_uint4(w[4], w[5], w[6], w[7]));
  } else if constexpr (BYTES == 8) {
    __stcs(reinterpret_cast<uint2*>(p), make_uint2(w[0], w[1]));
  } else {
    __stcs(reinterpret_cast<uint32_t*>(p), w[0]);
  }
}

// ---- element decode: raw words -> floats
__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

__device__ __forceinline__ float2 fp8x2_to_float2(uint32_t two, int is_e5m2) {
  __half2_raw hr = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(two & 0xFFFFu),
                                              is_e5m2 ? __NV_E5M2 : __NV_E4M3);
  return __half22float2(*reinterpret_cast<__half2*>(&hr));
}

// Decode N elements of dtype DT held in raw words.
template <int DT, int N>
__device__ __forceinline__ void decode_vec(const uint32_t* w, float* f) {
  if constexpr (DT == SCALIFY_F32) {
#pragma unroll
    for (int i = 0; i < N; ++i) f[i] = __uint_as_float(w[i]);
  } else if constexpr (DT == SCALIFY_BF16) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  } else if constexpr (DT == SCALIFY_F16) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      float2 t = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
      f[2 * i] = t.x;
      f[2 * i + 1] = t.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      float2 a = fp8x2_to_float2(w[i], DT == SCALIFY_E5M2);
      float2 b = fp8x2_to_float2(w[i] >> 16, DT == SCALIFY_E5M2);
      f[4 * i] = a.x; f[4 * i + 1] = a.y; f[4 * i + 2] = b.x; f[4 * i + 3] = b.y;
    }
  }
}

// Encode N floats to dtype DT (round to nearest even; FP8 saturates to max finite).
template <int DT, int N>
__device__ __forceinline__ void encode_vec(const float* f, uint32_t* w) {
  if constexpr (DT == SCALIFY_F32) {
#pragma unroll
    for (int i = 0; i < N; ++i) w[i] = __float_as_uint(f[i]);
  } else if constexpr (DT == SCALIFY_BF16) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      __nv_bfloat162 t = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&t);
    }
  } else if constexpr (DT == SCALIFY_F16) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      __half2 t = __floats2half2_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&t);
    }
  } else {
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(f[4 * i], f[4 * i + 1]), __NV_SATFINITE,
                                             DT == SCALIFY_E5M2 ? __NV_E5M2 : __NV_E4M3);
      uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(f[4 * i + 2], f[4 * i + 3]), __NV_SATFINITE,
                                             DT == SCALIFY_E5M2 ? __NV_E5M2 : __NV_E4M3);
      w[i] = (lo & 0xFFFFu) | (hi << 16);
    }
  }
}

// Round a float to dtype DT and back (the value that will be stored).
template <int DT>
__device__ __forceinline__ float round_through(float x) {
  if constexpr (DT == SCALIFY_F32) return x;
  else if constexpr (DT == SCALIFY_BF16) return __bfloat162float(__float2bfloat16_rn(x));
  else if constexpr (DT == SCALIFY_F16) return __half2float(__float2half_rn(x));
  else {
    uint32_t two = __nv_cvt_float2_to_fp8x2(make_float2(x, 0.f), __NV_SATFINITE,
                                            DT == SCALIFY_E5M2 ? __NV_E5M2 : __NV_E4M3);
    return fp8x2_to_float2(two, DT == SCALIFY_E5M2).x;
  }
}

// fp32 -> the nearest BF16 value (ties to even), returned as fp32, computed on the fp32 pipe: Veltkamp's split
// with the constant 2^16 + 1,   c = x (2^16 + 1);  hi = c - (c - x),   leaves exactly the upper 8 significand
// bits of x rounded to nearest even.  Exact for every normal x below 2^111 (checked on the GPU against the
// integer formula for all 2^32 bit patterns; zero stays zero; subnormal inputs are not covered).  It replaces
// four half-rate integer instructions, or a conversion instruction plus unpacking, in the attention kernels.
// The three operations must remain three separately rounded operations: the scalar intrinsics are documented
// never to be contracted into a multiply-add.  (The two-wide forms are NOT safe here: the same sequence written
// with mul.rn.f32x2 / sub.rn.f32x2 came out fused on this toolchain and returned x unrounded.)
__device__ __forceinline__ float bf16_round_f32(float x) {
  const float c = __fmul_rn(x, 65537.0f);
  const float d = __fsub_rn(c, x);
  return __fsub_rn(c, d);
}

// The same rounding for two values at once on the two-wide fp32 instructions.  Each of the three steps is
// written as a fused multiply-add with a non-trivial addend (65536 x + x = 65537 x rounded once; c - x and
// c - d as (-1) * v + c), so that there is no separate multiply for the toolchain to contract into the
// subtraction that follows: a multiply-add cannot be merged with another operation.
__device__ __forceinline__ float2 bf16_round_f32x2(float2 x) {
  const float2 k = make_float2(65536.0f, 65536.0f), neg = make_float2(-1.0f, -1.0f);
  const float2 c = __ffma2_rn(x, k, x);
  const float2 d = __ffma2_rn(x, neg, c);
  return __ffma2_rn(d, neg, c);
}

// scalar load/store for ragged tails
template <int DT>
__device__ __forceinline__ float load_elem(const void* p, int64_t i) {
#ifdef SCALIFY_DEBUG
  if (!dbg_ok(static_cast<const char*>(p) + i * ElemBytes<DT>::v, ElemBytes<DT>::v)) return 0.f;
#endif
  if constexpr (DT == SCALIFY_F32) return static_cast<const float*>(p)[i];
  else if constexpr (DT == SCALIFY_BF16) return bf16_bits_to_float(static_cast<const uint16_t*>(p)[i]);
  else if constexpr (DT == SCALIFY_F16) return __half2float(static_cast<const __half*>(p)[i]);
  else return fp8x2_to_float2(static_cast<const uint8_t*>(p)[i], DT == SCALIFY_E5M2).x;
}

template <int DT>
__device__ __forceinline__ void store_elem(void* p, int64_t i, float x) {
#ifdef SCALIFY_DEBUG
  if (!dbg_ok(static_cast<char*>(p) + i * ElemBytes<DT>::v, ElemBytes<DT>::v)) return;
#endif
  if constexpr (DT == SCALIFY_F32) static_cast<float*>(p)[i] = x;
  else if constexpr (DT == SCALIFY_BF16) static_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(x);
  else if constexpr (DT == SCALIFY_F16) static_cast<__half*>(p)[i] = __float2half_rn(x);
  else {
    uint32_t two = __nv_cvt_float2_to_fp8x2(make_float2(x, 0.f), __NV_SATFINITE,
                                            DT == SCALIFY_E5M2 ? __NV_E5M2 : __NV_E4M3);
    static_cast<uint8_t*>(p)[i] = static_cast<uint8_t>(two & 0xFFu);
  }
}

// |x| as an unsigned integer: ordering of the bit patterns is the ordering of
// the magnitudes, and NaN patterns sort above infinity, so an integer max
// propagates NaN.
__device__ __forceinline__ uint32_t abs_bits(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

#endif  // __CUDACC__

// dtype dispatch: calls F.template operator()<DT>() for a runtime dtype
#define SCALIFY_DISPATCH_DTYPE(dt, NAME, ...)                                  \
  switch (dt) {                                                                \
    case SCALIFY_E4M3: { constexpr int NAME = SCALIFY_E4M3; __VA_ARGS__; } break; \
    case SCALIFY_E5M2: { constexpr int NAME = SCALIFY_E5M2; __VA_ARGS__; } break; \
    case SCALIFY_F16: { constexpr int NAME = SCALIFY_F16; __VA_ARGS__; } break;   \
    case SCALIFY_BF16: { constexpr int NAME = SCALIFY_BF16; __VA_ARGS__; } break; \
    default: { constexpr int NAME = SCALIFY_F32; __VA_ARGS__; } break;            \
  }

#define SCALIFY_DISPATCH_WIDE(dt, NAME, ...)                                   \
  switch (dt) {                                                                \
    case SCALIFY_F16: { constexpr int NAME = SCALIFY_F16; __VA_ARGS__; } break;   \
    case SCALIFY_BF16: { constexpr int NAME = SCALIFY_BF16; __VA_ARGS__; } break; \
    default: { constexpr int NAME = SCALIFY_F32; __VA_ARGS__; } break;            \
  }

}  // namespace scalify
