// Host-side plumbing of libqbert: version, status text, workspace helpers, device check.
#include <cstdarg>
#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace qb {

static thread_local char g_last_error[512] = "";

void set_last_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
  va_end(ap);
}

qb_status cuda_fail(cudaError_t e, const char* what) {
  set_last_error("CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
  return QB_ERR_CUDA;
}

qb_status require_sm100(int* sm_count) {
  constexpr int kMaxDev = 64;
  static int cached_major[kMaxDev];  // 0 = unknown
  static int cached_sms[kMaxDev];
  int dev = 0;
  QB_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDev) {
    set_last_error("device ordinal %d out of range", dev);
    return QB_ERR_CUDA;
  }
  if (cached_major[dev] == 0) {
    int major = 0, sms = 0;
    QB_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    QB_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    cached_sms[dev] = sms;
    cached_major[dev] = major;
  }
  if (cached_major[dev] != 10) {
    set_last_error("libqbert needs an sm_100 device (B200); device %d has compute capability %d.x", dev,
                   cached_major[dev]);
    return QB_ERR_CUDA;
  }
  if (sm_count) *sm_count = cached_sms[dev];
  return QB_OK;
}

}  // namespace qb

extern "C" {

int qb_version(void) { return 100; }

const char* qb_status_string(qb_status s) {
  switch (s) {
    case QB_OK: return "QB_OK";
    case QB_ERR_INVALID: return "QB_ERR_INVALID";
    case QB_ERR_ALIGN: return "QB_ERR_ALIGN";
    case QB_ERR_WORKSPACE: return "QB_ERR_WORKSPACE";
    case QB_ERR_CUDA: return "QB_ERR_CUDA";
    case QB_ERR_NONFINITE: return "QB_ERR_NONFINITE";
    case QB_ERR_TIMEOUT: return "QB_ERR_TIMEOUT";
    default: return "QB_ERR_UNKNOWN";
  }
}

const char* qb_last_error(void) { return qb::g_last_error; }

size_t qb_packed_words(int64_t N, int64_t K, int bits) {
  if (N <= 0 || K <= 0 || !qb::valid_bits(bits) || (K * bits) % 32 != 0) return 0;
  return (size_t)(N * K * bits / 32);
}

size_t qb_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits, int groups) {
  (void)M; (void)N; (void)K; (void)bits;
  return qb::ws_bytes_needed(groups);
}

qb_status qb_workspace_init(void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!ws || ws_bytes < qb::kWsMinBytes) {
    qb::set_last_error("workspace is null or smaller than %zu bytes", qb::kWsMinBytes);
    return QB_ERR_WORKSPACE;
  }
  QB_CUDA_TRY(cudaMemsetAsync(ws, 0, ws_bytes, (cudaStream_t)cuda_stream));
  return QB_OK;
}

qb_status qb_read_status(const void* ws, void* cuda_stream) {
  if (!ws) {
    qb::set_last_error("workspace is null");
    return QB_ERR_WORKSPACE;
  }
  int32_t st = 0;
  QB_CUDA_TRY(cudaMemcpyAsync(&st, ws, sizeof(st), cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream));
  QB_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
  return (qb_status)st;
}

}  // extern "C"
