// Shared host/device helpers of libqbert: workspace layout, status word, error text.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "qbert.h"

namespace qb {

// ---- workspace layout (device memory owned by the caller) ------------------------------------
// [0]   int32  status   first device-side error, never cleared by a kernel
// [4]   int32  detail   where a bounded wait gave up (role << 16 | stage), diagnostics only
// [16]  uint32 act_absmax_bits   bit pattern of max|x| of the last qb_quantize_act
// [256] uint32 range_hi_enc[G], uint32 range_lo_inv[G]   ordered encodings of per-group max / min
constexpr size_t kWsStatusOff = 0;
constexpr size_t kWsDetailOff = 4;
constexpr size_t kWsActMaxOff = 16;
constexpr size_t kWsRangeOff = 256;
constexpr size_t kWsMinBytes = 256;

struct WsHeader {
  int32_t status;
  int32_t detail;
  uint32_t pad[2];
  uint32_t act_absmax_bits;
};

inline size_t ws_bytes_needed(int groups) {
  size_t b = kWsRangeOff + (groups > 0 ? size_t(groups) * 8 : 0);
  return (b + 255) / 256 * 256;
}

// ---- host-side error plumbing ------------------------------------------------------------------
void set_last_error(const char* fmt, ...);
qb_status cuda_fail(cudaError_t e, const char* what);
// QB_OK if the current device is sm_100; caches the answer and the SM count per device.
qb_status require_sm100(int* sm_count);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool valid_bits(int b) { return b == 2 || b == 3 || b == 4 || b == 8; }

#define QB_CUDA_TRY(expr)                                   \
  do {                                                      \
    cudaError_t e__ = (expr);                               \
    if (e__ != cudaSuccess) return qb::cuda_fail(e__, #expr); \
  } while (0)

// ---- device-side helpers -----------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ void report_status(void* ws, int32_t code, int32_t detail = 0) {
  WsHeader* h = reinterpret_cast<WsHeader*>(ws);
  if (atomicCAS(&h->status, 0, code) == 0) h->detail = detail;
}

// Monotone map from float bit patterns to unsigned integers (so that integer atomicMax orders floats).
// Written as integer PTX on the register: as C++ the compiler may turn the sign-bit operations into
// floating-point negation, which does not keep the bit pattern of a NaN (and the NaN would then sort
// below the finite values instead of above them).
__device__ __forceinline__ uint32_t float_to_ordered(float f) {
  uint32_t o;
  asm("{\n\t.reg .b32 t, m;\n\tmov.b32 t, %1;\n\tshr.s32 m, t, 31;\n\tor.b32 m, m, 0x80000000;\n\txor.b32 %0, t, m;\n\t}"
      : "=r"(o)
      : "f"(f));
  return o;
}
__device__ __forceinline__ float ordered_to_float(uint32_t e) {
  uint32_t b = (e & 0x80000000u) ? (e & 0x7fffffffu) : ~e;
  return __uint_as_float(b);
}
// 16-byte load with an L2 eviction-priority policy (createpolicy).  The two-pass quantizers use it: the
// first pass asks L2 to keep a fraction of what it reads (the second pass reads the same tensor next),
// the second pass marks its reads as the first to go.
__device__ __forceinline__ float4 ldg_policy(const float4* p, uint64_t policy) {
  float4 v;
  asm volatile("ld.global.nc.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "l"(p), "l"(policy));
  return v;
}
__device__ __forceinline__ uint64_t policy_evict_last(float fraction) {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, %1;" : "=l"(pol) : "f"(fraction));
  return pol;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

// Share of a first pass's input that L2 is asked to keep: all of it up to 96 MB (what the 126 MB L2 holds
// of a stream besides what the second pass writes), else 96 MB worth.
inline float l2_keep_fraction(double input_bytes) {
  const double keep = 96.0 * 1048576.0;
  return input_bytes <= keep ? 1.0f : (float)(keep / input_bytes);
}

#endif

}  // namespace qb
