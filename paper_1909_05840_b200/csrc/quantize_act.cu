// qb_quantize_act(_batch): per-tensor 8-bit activation quantizer (Table 1 caption: 8-bit activations;
// Appendix A's uniform quantizer on the symmetric range [-a, a], a = max|x|), for one tensor or a
// batch of tensors in one pair of launches.
//
// Kernel 1  act_absmax_kernel    each block belongs to one tensor; block-stride float4 loads, max of
//                                |x| bit patterns (monotone as unsigned integers, and NaN/Inf sort
//                                above every finite value), warp reduce + one atomicMax per block
//                                into the tensor's slot of the workspace.
// Kernel 2  act_quantize_kernel  one warp per row (rows of all tensors form one sequence):
//                                x * (127/a), round half to even, clamp, four codes packed per 32-bit
//                                store, int32 row sum by warp reduction.
// Both kernels are HBM-bound: 4 B read per element in each, 1 B written in the second.
#include <algorithm>
#include <cstring>

#include "common.cuh"

namespace qb {

constexpr int kActThreads = 256;
constexpr int kMaxActBatch = 64;  // tensors per launch (descriptors travel as kernel parameters, 4 KB)

struct ActItem {
  const float* x;
  int8_t* xq;
  float* act_scale;
  int32_t* rowsum;
  int64_t M, K;
  int64_t row_begin;    // index of the tensor's first row in the launch's row sequence
  int32_t block_begin;  // first block of kernel 1 that works on this tensor
  int32_t blocks;       // number of such blocks
};

struct ActBatch {
  ActItem item[kMaxActBatch];
  uint32_t* absmax_bits;  // [count] slots in the workspace
  void* ws;
  int64_t rows_total;
  int32_t count;
  float keep_fraction;  // share of the launch's input that L2 is asked to keep between the two passes
};

__global__ void __launch_bounds__(kActThreads)
act_absmax_kernel(const __grid_constant__ ActBatch b) {
  int it = 0;
  while (it + 1 < b.count && (int)blockIdx.x >= b.item[it + 1].block_begin) ++it;
  const ActItem& t = b.item[it];
  const float4* __restrict__ x = reinterpret_cast<const float4*>(t.x);
  const int64_t n4 = t.M * t.K / 4;
  uint32_t m = 0;
  const uint64_t pol = policy_evict_last(b.keep_fraction);
  const int64_t stride = (int64_t)t.blocks * blockDim.x;
  int64_t i = (int64_t)((int)blockIdx.x - t.block_begin) * blockDim.x + threadIdx.x;
  // four independent 16-byte loads in flight per thread
  for (; i + 3 * stride < n4; i += 4 * stride) {
    float4 a = ldg_policy(x + i, pol), bb = ldg_policy(x + i + stride, pol), c = ldg_policy(x + i + 2 * stride, pol),
           d = ldg_policy(x + i + 3 * stride, pol);
#define QB_ABSMAX4(v)                                            \
  m = max(m, __float_as_uint(v.x) & 0x7fffffffu);                \
  m = max(m, __float_as_uint(v.y) & 0x7fffffffu);                \
  m = max(m, __float_as_uint(v.z) & 0x7fffffffu);                \
  m = max(m, __float_as_uint(v.w) & 0x7fffffffu);
    QB_ABSMAX4(a) QB_ABSMAX4(bb) QB_ABSMAX4(c) QB_ABSMAX4(d)
  }
  for (; i < n4; i += stride) {
    float4 a = ldg_policy(x + i, pol);
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
    if (threadIdx.x == 0 && v != 0u) atomicMax(b.absmax_bits + it, v);
  }
}

__device__ __forceinline__ int quant_code(float v, float inv) {
  int q = __float2int_rn(__fmul_rn(v, inv));
  return min(max(q, -127), 127);
}

// scale and reciprocal of a tensor from the bit pattern of its max|x|; false if NaN/Inf was seen
__device__ __forceinline__ bool act_scales(uint32_t mb, float* s, float* inv) {
  *s = 1.0f;
  *inv = 0.0f;
  if (mb >= 0x7f800000u) return false;
  const float a = __uint_as_float(mb);
  const float s1 = __fdiv_rn(a, 127.0f);
  const float inv1 = __fdiv_rn(127.0f, a);
  if (a > 0.0f && inv1 <= 3.402823466e38f) {
    *s = s1;
    *inv = inv1;
  }
  return true;
}

__global__ void __launch_bounds__(kActThreads, 8)  // eight blocks per SM resident: the grid is one full wave
act_quantize_kernel(const __grid_constant__ ActBatch b) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  int it = 0;
  int cur = -1;
  float inv = 0.0f;
  const uint64_t pol = policy_evict_first();
  for (int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); row < b.rows_total; row += warps) {
    while (it + 1 < b.count && row >= b.item[it + 1].row_begin) ++it;
    const ActItem& t = b.item[it];
    if (it != cur) {  // warp-uniform: first row of this warp in tensor `it`
      cur = it;
      float s;
      const bool finite = act_scales(b.absmax_bits[it], &s, &inv);
      if (row == t.row_begin && lane == 0) {  // exactly one warp sees the tensor's first row
        *t.act_scale = s;
        if (!finite) report_status(b.ws, QB_ERR_NONFINITE);
      }
    }
    const int64_t r = row - t.row_begin;
    const int64_t k4 = t.K >> 2;  // float4 per row
    const float4* src = reinterpret_cast<const float4*>(t.x + r * t.K);
    uint32_t* dst = reinterpret_cast<uint32_t*>(t.xq + r * t.K);
    int sum = 0;
#pragma unroll 4
    for (int64_t c = lane; c < k4; c += 32) {
      const float4 v = ldg_policy(src + c, pol);
      const int q0 = quant_code(v.x, inv), q1 = quant_code(v.y, inv), q2 = quant_code(v.z, inv),
                q3 = quant_code(v.w, inv);
      sum += (q0 + q1) + (q2 + q3);
      dst[c] = (uint32_t)(q0 & 0xff) | ((uint32_t)(q1 & 0xff) << 8) | ((uint32_t)(q2 & 0xff) << 16) |
               ((uint32_t)(q3 & 0xff) << 24);
    }
    sum = __reduce_add_sync(0xffffffffu, sum);
    if (lane == 0) t.rowsum[r] = sum;
  }
}

// One pair of launches over `count` tensors (<= kMaxActBatch).  `absmax_slots` has room for `count` words.
static qb_status launch_act_batch(const qb_act_desc* d, int count, void* ws, uint32_t* absmax_slots, int sm_count,
                                  cudaStream_t stream) {
  ActBatch b;
  memset(&b, 0, sizeof(b));
  b.count = count;
  b.ws = ws;
  b.absmax_bits = absmax_slots;
  const int64_t cap = (int64_t)sm_count * 8;  // one full wave of either kernel (eight blocks per SM)
  int64_t total4 = 0;
  for (int i = 0; i < count; ++i) total4 += d[i].M * d[i].K / 4;
  // Tensors with the longest rows first: kernel 2 hands rows to warps round-robin, and a long row met
  // at the end of a warp's list would be the launch's tail.  Slot i of `absmax_slots` stays with the
  // i-th tensor of this order; nothing outside the two kernels reads the slots.
  int ord[kMaxActBatch];
  for (int i = 0; i < count; ++i) ord[i] = i;
  std::stable_sort(ord, ord + count, [&](int a, int c) { return d[a].K > d[c].K; });
  int64_t rows = 0;
  int blocks1 = 0;
  for (int i = 0; i < count; ++i) {
    const qb_act_desc& q = d[ord[i]];
    ActItem& t = b.item[i];
    t.x = q.x;
    t.xq = q.xq;
    t.act_scale = q.act_scale;
    t.rowsum = q.rowsum;
    t.M = q.M;
    t.K = q.K;
    t.row_begin = rows;
    rows += q.M;
    // blocks of kernel 1 in proportion to the tensor's size (rounded down, so that the launch never
    // exceeds one wave: a block of a second wave would run alone for as long as the whole first wave),
    // each thread >= 4 loads when possible
    const int64_t n4 = q.M * q.K / 4;
    int64_t want = (n4 + (int64_t)kActThreads * 4 - 1) / ((int64_t)kActThreads * 4);
    const int64_t avail = cap - count > 0 ? cap - count : 0;  // one block per tensor is set aside
    const int64_t share = 1 + avail * n4 / total4;
    if (want > share) want = share;
    if (want < 1) want = 1;
    t.block_begin = blocks1;
    t.blocks = (int32_t)want;
    blocks1 += (int)want;
  }
  b.rows_total = rows;
  b.keep_fraction = l2_keep_fraction(16.0 * (double)total4);
  QB_CUDA_TRY(cudaMemsetAsync(absmax_slots, 0, sizeof(uint32_t) * (size_t)count, stream));
  act_absmax_kernel<<<(unsigned)blocks1, kActThreads, 0, stream>>>(b);
  QB_CUDA_TRY(cudaGetLastError());
  const int warps_per_block = kActThreads / 32;
  int64_t blocks2 = (rows + warps_per_block - 1) / warps_per_block;
  if (blocks2 > cap) blocks2 = cap;
  act_quantize_kernel<<<(unsigned)blocks2, kActThreads, 0, stream>>>(b);
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}

static qb_status validate_act(const char* who, const float* x, int64_t M, int64_t K, const int8_t* xq,
                              const float* act_scale, const int32_t* rowsum) {
  if (!x || !xq || !act_scale || !rowsum || M <= 0 || K <= 0 || M > QB_MAX_MN || K > QB_MAX_K) {
    set_last_error("%s: null pointer or size out of range (M=%lld K=%lld)", who, (long long)M, (long long)K);
    return QB_ERR_INVALID;
  }
  if (K % 128 != 0 || !aligned16(x) || !aligned16(xq)) {
    set_last_error("%s: K must be a multiple of 128 and x, xq 16-byte aligned", who);
    return QB_ERR_ALIGN;
  }
  return QB_OK;
}

}  // namespace qb

extern "C" qb_status qb_quantize_act(const float* x, int64_t M, int64_t K, int8_t* xq, float* act_scale,
                                     int32_t* rowsum, void* ws, size_t ws_bytes, void* cuda_stream) {
  qb_status st = qb::validate_act("qb_quantize_act", x, M, K, xq, act_scale, rowsum);
  if (st != QB_OK) return st;
  if (!ws || ws_bytes < qb::ws_bytes_needed(0)) {
    qb::set_last_error("qb_quantize_act: workspace null or too small");
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  uint32_t* slot = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + qb::kWsActMaxOff);
  const qb_act_desc d{x, M, K, xq, act_scale, rowsum};
  return qb::launch_act_batch(&d, 1, ws, slot, sms, (cudaStream_t)cuda_stream);
}

extern "C" qb_status qb_quantize_act_batch(const qb_act_desc* descs, int32_t count, void* ws, size_t ws_bytes,
                                           void* cuda_stream) {
  if (!descs || count <= 0) {
    qb::set_last_error("qb_quantize_act_batch: descs null or count <= 0");
    return QB_ERR_INVALID;
  }
  for (int i = 0; i < count; ++i) {
    qb_status st = qb::validate_act("qb_quantize_act_batch", descs[i].x, descs[i].M, descs[i].K, descs[i].xq,
                                    descs[i].act_scale, descs[i].rowsum);
    if (st != QB_OK) return st;
  }
  // max-abs slots of a launch: the head of the range area of the workspace
  if (!ws || ws_bytes < qb::kWsRangeOff + sizeof(uint32_t) * (size_t)qb::kMaxActBatch) {
    qb::set_last_error("qb_quantize_act_batch: workspace null or smaller than %zu bytes",
                       qb::kWsRangeOff + sizeof(uint32_t) * (size_t)qb::kMaxActBatch);
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  uint32_t* slots = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + qb::kWsRangeOff);
  for (int i = 0; i < count; i += qb::kMaxActBatch) {
    const int n = count - i < qb::kMaxActBatch ? count - i : qb::kMaxActBatch;
    st = qb::launch_act_batch(descs + i, n, ws, slots, sms, (cudaStream_t)cuda_stream);
    if (st != QB_OK) return st;
  }
  return QB_OK;
}

extern "C" int32_t qb_quantize_act_launch_count(int32_t count) {
  if (count <= 0) return 0;
  return 2 * ((count + qb::kMaxActBatch - 1) / qb::kMaxActBatch);
}
