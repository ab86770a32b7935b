// qb_quantize_act: per-tensor 8-bit activation quantizer (Table 1 caption: 8-bit activations;
// Appendix A's uniform quantizer on the symmetric range [-a, a], a = max|x|).
//
// Kernel 1  act_absmax_kernel    grid-stride float4 loads, max of |x| bit patterns (monotone as
//                                unsigned integers, and NaN/Inf sort above every finite value),
//                                warp reduce + one atomicMax per block into the workspace.
// Kernel 2  act_quantize_kernel  one warp per row: x * (127/a), round half to even, clamp, four
//                                codes packed per 32-bit store, int32 row sum by warp reduction.
// Both kernels are HBM-bound: 4 B read per element in each, 1 B written in the second.
#include "common.cuh"

namespace qb {

constexpr int kActThreads = 256;

__global__ void __launch_bounds__(kActThreads)
act_absmax_kernel(const float4* __restrict__ x, int64_t n4, uint32_t* __restrict__ out_bits) {
  uint32_t m = 0;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  // four independent 16-byte loads in flight per thread
  for (; i + 3 * stride < n4; i += 4 * stride) {
    float4 a = __ldg(x + i), b = __ldg(x + i + stride), c = __ldg(x + i + 2 * stride),
           d = __ldg(x + i + 3 * stride);
#define QB_ABSMAX4(v)                                            \
  m = max(m, __float_as_uint(v.x) & 0x7fffffffu);                \
  m = max(m, __float_as_uint(v.y) & 0x7fffffffu);                \
  m = max(m, __float_as_uint(v.z) & 0x7fffffffu);                \
  m = max(m, __float_as_uint(v.w) & 0x7fffffffu);
    QB_ABSMAX4(a) QB_ABSMAX4(b) QB_ABSMAX4(c) QB_ABSMAX4(d)
  }
  for (; i < n4; i += stride) {
    float4 a = __ldg(x + i);
    QB_ABSMAX4(a)
  }
#undef QB_ABSMAX4
  m = __reduce_max_sync(0xffffffffu, m);
  __shared__ uint32_t warp_max[kActThreads / 32];
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    uint32_t v = threadIdx.x < kActThreads / 32 ? warp_max[threadIdx.x] : 0u;
    v = __reduce_max_sync(0xffffffffu, v);
    if (threadIdx.x == 0 && v != 0u) atomicMax(out_bits, v);
  }
}

__device__ __forceinline__ int quant_code(float v, float inv) {
  int q = __float2int_rn(__fmul_rn(v, inv));
  return min(max(q, -127), 127);
}

__global__ void __launch_bounds__(kActThreads)
act_quantize_kernel(const float* __restrict__ x, int64_t M, int64_t K, int8_t* __restrict__ xq,
                    float* __restrict__ act_scale, int32_t* __restrict__ rowsum, void* ws,
                    const uint32_t* __restrict__ absmax_bits) {
  const uint32_t mb = *absmax_bits;
  float s = 1.0f, inv = 0.0f;
  if (mb >= 0x7f800000u) {  // NaN or Inf somewhere in the tensor
    if (blockIdx.x == 0 && threadIdx.x == 0) report_status(ws, QB_ERR_NONFINITE);
  } else {
    const float a = __uint_as_float(mb);
    const float s1 = __fdiv_rn(a, 127.0f);
    const float inv1 = __fdiv_rn(127.0f, a);
    if (a > 0.0f && inv1 <= 3.402823466e38f) {
      s = s1;
      inv = inv1;
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *act_scale = s;

  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  const int64_t k4 = K >> 2;  // float4 per row
  for (int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); row < M; row += warps) {
    const float4* src = reinterpret_cast<const float4*>(x + row * K);
    uint32_t* dst = reinterpret_cast<uint32_t*>(xq + row * K);
    int sum = 0;
#pragma unroll 4
    for (int64_t c = lane; c < k4; c += 32) {
      const float4 v = __ldg(src + c);
      const int q0 = quant_code(v.x, inv), q1 = quant_code(v.y, inv), q2 = quant_code(v.z, inv),
                q3 = quant_code(v.w, inv);
      sum += (q0 + q1) + (q2 + q3);
      dst[c] = (uint32_t)(q0 & 0xff) | ((uint32_t)(q1 & 0xff) << 8) | ((uint32_t)(q2 & 0xff) << 16) |
               ((uint32_t)(q3 & 0xff) << 24);
    }
    sum = __reduce_add_sync(0xffffffffu, sum);
    if (lane == 0) rowsum[row] = sum;
  }
}

qb_status launch_quantize_act(const float* x, int64_t M, int64_t K, int8_t* xq, float* act_scale,
                              int32_t* rowsum, void* ws, uint32_t* absmax_slot, int sm_count,
                              cudaStream_t stream) {
  QB_CUDA_TRY(cudaMemsetAsync(absmax_slot, 0, sizeof(uint32_t), stream));
  const int64_t n4 = M * K / 4;
  int64_t blocks1 = (n4 + (int64_t)kActThreads * 4 - 1) / ((int64_t)kActThreads * 4);
  const int64_t cap = (int64_t)sm_count * 8;
  if (blocks1 > cap) blocks1 = cap;
  if (blocks1 < 1) blocks1 = 1;
  act_absmax_kernel<<<(unsigned)blocks1, kActThreads, 0, stream>>>(reinterpret_cast<const float4*>(x), n4,
                                                                   absmax_slot);
  QB_CUDA_TRY(cudaGetLastError());
  const int warps_per_block = kActThreads / 32;
  int64_t blocks2 = (M + warps_per_block - 1) / warps_per_block;
  if (blocks2 > cap) blocks2 = cap;
  act_quantize_kernel<<<(unsigned)blocks2, kActThreads, 0, stream>>>(x, M, K, xq, act_scale, rowsum, ws,
                                                                     absmax_slot);
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}

}  // namespace qb

extern "C" qb_status qb_quantize_act(const float* x, int64_t M, int64_t K, int8_t* xq, float* act_scale,
                                     int32_t* rowsum, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!x || !xq || !act_scale || !rowsum || M <= 0 || K <= 0 || M > QB_MAX_MN || K > QB_MAX_K) {
    qb::set_last_error("qb_quantize_act: null pointer or size out of range (M=%lld K=%lld)", (long long)M,
                       (long long)K);
    return QB_ERR_INVALID;
  }
  if (K % 128 != 0 || !qb::aligned16(x) || !qb::aligned16(xq)) {
    qb::set_last_error("qb_quantize_act: K must be a multiple of 128 and x, xq 16-byte aligned");
    return QB_ERR_ALIGN;
  }
  if (!ws || ws_bytes < qb::ws_bytes_needed(0)) {
    qb::set_last_error("qb_quantize_act: workspace null or too small");
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  uint32_t* slot = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + qb::kWsActMaxOff);
  return qb::launch_quantize_act(x, M, K, xq, act_scale, rowsum, ws, slot, sms, (cudaStream_t)cuda_stream);
}
