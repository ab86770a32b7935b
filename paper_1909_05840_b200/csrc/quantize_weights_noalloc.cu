// qb_quantize_pack_weights_noalloc: the group-wise weight quantizer and packer for callers that
// cannot hand the library a workspace.
//
// Who needs this: code that runs where device allocation is off the table -- inside a region whose
// memory pool is frozen, in a plug-in that is given tensors but no allocator, or in a
// latency-critical serving loop where cudaMalloc (which synchronises the device) is forbidden.
// Such callers still own the input matrix and the three outputs, but have nowhere to put the few
// kilobytes of per-group min/max scratch the quantizer needs between its two kernels.
//
// The scratch therefore lives inside the library image: one file-scope device array, present on
// every GPU that loads libqbert until the process exits.  It has room for the status word and the
// ranges of at most QB_NOALLOC_MAX_GROUPS groups; larger group counts are refused on the host.
// The array is shared by every call and keeps whatever the last call left in it, so each call
// clears the parts that must start at zero, and two calls that overlap on the GPU (different
// streams, or the same stream from two threads without ordering) would race on it.
#include <atomic>

#include "common.cuh"

namespace qb {

// defined in quantize_weights.cu
qb_status launch_quantize_pack_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                       const float* range_lo, const float* range_hi, uint32_t* packed,
                                       float* delta, float* q0, void* ws, int sm_count, cudaStream_t stream);

constexpr size_t kNoAllocScratchBytes = kWsRangeOff + 8 * (size_t)QB_NOALLOC_MAX_GROUPS;

// Same layout as a caller-provided workspace: status word at offset 0, encoded ranges at kWsRangeOff.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel can
// use: the device address is looked up once per device, with that device current.
static qb_status noalloc_scratch_ptr(void** out) {
  constexpr int kMaxDev = 64;
  static std::atomic<void*> cached[kMaxDev] = {};  // two threads may look the address up at once: both find the same value
  int dev = 0;
  QB_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDev) {
    set_last_error("device ordinal %d out of range", dev);
    return QB_ERR_CUDA;
  }
  void* p = cached[dev].load(std::memory_order_acquire);
  if (p == nullptr) {
    cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(g_noalloc_scratch)");
    if (p == nullptr) {
      set_last_error("cudaGetSymbolAddress returned a null address for the built-in scratch");
      return QB_ERR_CUDA;
    }
    cached[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return QB_OK;
}

}  // namespace qb

extern "C" qb_status qb_quantize_pack_weights_noalloc(const float* w, int64_t N, int64_t K, int bits, int groups,
                                                      const float* range_lo, const float* range_hi,
                                                      uint32_t* packed, float* delta, float* q0,
                                                      int32_t* status_out, void* cuda_stream) {
  if (!w || !packed || !delta || !q0 || N <= 0 || K <= 0 || N > QB_MAX_MN || K > QB_MAX_K ||
      !qb::valid_bits(bits) || groups < 1 || N % groups != 0 || ((range_lo == nullptr) != (range_hi == nullptr))) {
    qb::set_last_error("qb_quantize_pack_weights_noalloc: invalid argument (N=%lld K=%lld bits=%d groups=%d)",
                       (long long)N, (long long)K, bits, groups);
    return QB_ERR_INVALID;
  }
  if (groups > QB_NOALLOC_MAX_GROUPS) {
    qb::set_last_error("qb_quantize_pack_weights_noalloc: groups=%d exceeds QB_NOALLOC_MAX_GROUPS=%d, the capacity "
                       "of the built-in scratch; use qb_quantize_pack_weights with a workspace instead",
                       groups, (int)QB_NOALLOC_MAX_GROUPS);
    return QB_ERR_WORKSPACE;
  }
  if (K % 128 != 0 || !qb::aligned16(w) || !qb::aligned16(packed)) {
    qb::set_last_error("qb_quantize_pack_weights_noalloc: K must be a multiple of 128 and w, packed 16-byte aligned");
    return QB_ERR_ALIGN;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  void* scratch = nullptr;
  st = qb::noalloc_scratch_ptr(&scratch);
  if (st != QB_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  // the status word is sticky inside one call only: start it at zero (the ranges are cleared by the launcher)
  QB_CUDA_TRY(cudaMemsetAsync(scratch, 0, qb::kWsRangeOff, stream));
  st = qb::launch_quantize_pack_weights(w, N, K, bits, groups, range_lo, range_hi, packed, delta, q0, scratch, sms,
                                        stream);
  if (st != QB_OK) return st;
  if (status_out != nullptr)
    QB_CUDA_TRY(cudaMemcpyAsync(status_out, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream));
  return QB_OK;
}
