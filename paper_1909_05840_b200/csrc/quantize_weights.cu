// qb_quantize_pack_weights: group-wise uniform quantizer Q (Section 3.3, Appendix A) and dense
// k-bit packing (Table 1 counts exactly k bits per weight).
//
// The matrix is walked in "units" of 128 consecutive elements of one row (one float4 per lane,
// fully coalesced; K % 128 == 0 so a unit never crosses a row).  Each warp owns a contiguous run
// of units, so it crosses few group boundaries.
//
// Kernel 1  weight_range_kernel  running min/max per lane, warp reduction when the group changes,
//                                atomicMax on order-preserving integer encodings in the workspace
//                                (block-level merge of the final partials first).
// Kernel 2  weight_pack_kernel   re-reads the unit (from L2 for BERT-sized matrices), computes four
//                                codes per lane, and assembles the unit's 4k output words with warp
//                                shuffles so that the stores are contiguous 16k-byte runs.
#include "common.cuh"

namespace qb {

constexpr int kWqThreads = 256;
constexpr int kWqWarps = kWqThreads / 32;

struct WeightWalk {
  int64_t units_total;     // N * K / 128
  int units_per_row;       // K / 128
  int rows_per_group;      // R
  int64_t units_per_warp;  // contiguous run per warp
};

__device__ __forceinline__ void flush_range(uint32_t* __restrict__ hi_enc, uint32_t* __restrict__ lo_inv,
                                            int g, float lo, float hi) {
  // all lanes call; lane 0 publishes
  const uint32_t e_hi = __reduce_max_sync(0xffffffffu, float_to_ordered(hi));
  const uint32_t e_lo = __reduce_max_sync(0xffffffffu, ~float_to_ordered(lo));
  if ((threadIdx.x & 31) == 0) {
    atomicMax(hi_enc + g, e_hi);
    atomicMax(lo_inv + g, e_lo);
  }
}

__global__ void __launch_bounds__(kWqThreads)
weight_range_kernel(const float4* __restrict__ w, WeightWalk walk, int groups, uint32_t* __restrict__ hi_enc,
                    uint32_t* __restrict__ lo_inv, void* ws) {
  const int lane = threadIdx.x & 31;
  const int warp_in_block = threadIdx.x >> 5;
  const int64_t gwarp = (int64_t)blockIdx.x * kWqWarps + warp_in_block;
  int64_t u = gwarp * walk.units_per_warp;
  int64_t u_end = u + walk.units_per_warp;
  if (u_end > walk.units_total) u_end = walk.units_total;

  __shared__ int s_group[kWqWarps];
  __shared__ uint32_t s_hi[kWqWarps], s_lo[kWqWarps];

  const float kInf = __int_as_float(0x7f800000);
  float lo = kInf, hi = -kInf;
  uint32_t absmax = 0;
  int cur_g = -1;
  if (u < u_end) {
    int64_t row = u / walk.units_per_row;
    int col_unit = (int)(u - row * walk.units_per_row);
    int g = (int)(row / walk.rows_per_group);
    int row_in_group = (int)(row - (int64_t)g * walk.rows_per_group);
    cur_g = g;
    while (u < u_end) {
      float4 v[4];
      const int nload = (int)min((int64_t)4, u_end - u);
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (j < nload) v[j] = __ldg(w + (u + j) * 32 + lane);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (j < nload) {
          if (g != cur_g) {  // warp-uniform
            flush_range(hi_enc, lo_inv, cur_g, lo, hi);
            cur_g = g;
            lo = kInf;
            hi = -kInf;
          }
          lo = fminf(fminf(lo, v[j].x), fminf(v[j].y, fminf(v[j].z, v[j].w)));
          hi = fmaxf(fmaxf(hi, v[j].x), fmaxf(v[j].y, fmaxf(v[j].z, v[j].w)));
          absmax = max(absmax, max(max(__float_as_uint(v[j].x) << 1, __float_as_uint(v[j].y) << 1),
                                   max(__float_as_uint(v[j].z) << 1, __float_as_uint(v[j].w) << 1)));
          // advance (row, group) counters by one unit
          if (++col_unit == walk.units_per_row) {
            col_unit = 0;
            if (++row_in_group == walk.rows_per_group) {
              row_in_group = 0;
              ++g;
            }
          }
        }
      }
      u += nload;
    }
  }
  // NaN / Inf: exponent all ones survives the shift as >= 0xff000000
  absmax = __reduce_max_sync(0xffffffffu, absmax);
  if (lane == 0 && absmax >= 0xff000000u) report_status(ws, QB_ERR_NONFINITE);

  // final partial of each warp: merge equal groups inside the block, then one pair of atomics each
  const uint32_t e_hi = __reduce_max_sync(0xffffffffu, float_to_ordered(hi));
  const uint32_t e_lo = __reduce_max_sync(0xffffffffu, ~float_to_ordered(lo));
  if (lane == 0) {
    s_group[warp_in_block] = cur_g;
    s_hi[warp_in_block] = e_hi;
    s_lo[warp_in_block] = e_lo;
  }
  __syncthreads();
  if (threadIdx.x < kWqWarps) {
    const int my_g = s_group[threadIdx.x];
    bool leader = my_g >= 0;
    for (int j = 0; j < (int)threadIdx.x; ++j) leader = leader && (s_group[j] != my_g);
    if (leader) {
      uint32_t mh = s_hi[threadIdx.x], ml = s_lo[threadIdx.x];
      for (int j = threadIdx.x + 1; j < kWqWarps; ++j)
        if (s_group[j] == my_g) {
          mh = max(mh, s_hi[j]);
          ml = max(ml, s_lo[j]);
        }
      atomicMax(hi_enc + my_g, mh);
      atomicMax(lo_inv + my_g, ml);
    }
  }
}

struct GroupParams {
  float lo, hi, inv;
};

// Range of group g -> (q0, qmax, 1/Delta); lane-uniform.  Also publishes Delta and q0 once.
__device__ __forceinline__ GroupParams load_group(int g, int bits_levels, const uint32_t* __restrict__ hi_enc,
                                                  const uint32_t* __restrict__ lo_inv,
                                                  const float* __restrict__ range_lo,
                                                  const float* __restrict__ range_hi, float* __restrict__ delta,
                                                  float* __restrict__ q0, bool publish, void* ws) {
  GroupParams p;
  if (range_lo != nullptr) {
    p.lo = __ldg(range_lo + g);
    p.hi = __ldg(range_hi + g);
    const bool bad = !(fabsf(p.lo) <= 3.402823466e38f) || !(fabsf(p.hi) <= 3.402823466e38f) || p.hi < p.lo;
    if (bad) {
      if (publish) report_status(ws, QB_ERR_NONFINITE);
      p.lo = 0.0f;
      p.hi = 0.0f;
    }
  } else {
    p.hi = ordered_to_float(hi_enc[g]);
    p.lo = ordered_to_float(~lo_inv[g]);
  }
  float d = __fdiv_rn(__fsub_rn(p.hi, p.lo), (float)bits_levels);
  float inv = __fdiv_rn(1.0f, d);
  if (!(d > 0.0f) || !(inv <= 3.402823466e38f)) {  // constant group
    d = 1.0f;
    inv = 1.0f;
    p.hi = p.lo;
  }
  p.inv = inv;
  if (publish) {
    delta[g] = d;
    q0[g] = p.lo;
  }
  return p;
}

template <int BITS>
__global__ void __launch_bounds__(kWqThreads)
weight_pack_kernel(const float4* __restrict__ w, WeightWalk walk, const uint32_t* __restrict__ hi_enc,
                   const uint32_t* __restrict__ lo_inv, const float* __restrict__ range_lo,
                   const float* __restrict__ range_hi, uint32_t* __restrict__ packed,
                   float* __restrict__ delta, float* __restrict__ q0, void* ws) {
  constexpr int L = (1 << BITS) - 1;
  constexpr int F = 4 * BITS;          // bits contributed by one lane (four codes)
  constexpr int WORDS = 4 * BITS;      // output words per unit of 128 codes
  constexpr int NSRC = BITS == 8 ? 1 : (BITS == 4 ? 2 : 4);
  const int lane = threadIdx.x & 31;
  const int64_t gwarp = (int64_t)blockIdx.x * kWqWarps + (threadIdx.x >> 5);
  int64_t u = gwarp * walk.units_per_warp;
  int64_t u_end = u + walk.units_per_warp;
  if (u_end > walk.units_total) u_end = walk.units_total;
  if (u >= u_end) return;

  int64_t row = u / walk.units_per_row;
  int col_unit = (int)(u - row * walk.units_per_row);
  int g = (int)(row / walk.rows_per_group);
  int row_in_group = (int)(row - (int64_t)g * walk.rows_per_group);
  int cur_g = -1;
  GroupParams gp{0.f, 0.f, 1.f};

  // which lanes feed output word `lane` of a unit (stream bits [32*lane, 32*lane + 32))
  const int first_src = (32 * lane) / F;

  while (u < u_end) {
    float4 v[4];
    const int nload = (int)min((int64_t)4, u_end - u);
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (j < nload) v[j] = __ldg(w + (u + j) * 32 + lane);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (j < nload) {
        if (g != cur_g) {  // warp-uniform
          cur_g = g;
          // the warp that handles the first unit of the group publishes Delta and q0
          const bool publish = lane == 0 && row_in_group == 0 && col_unit == 0;
          gp = load_group(g, L, hi_enc, lo_inv, range_lo, range_hi, delta, q0, publish, ws);
        }
        const float e[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
        uint32_t field = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float xc = fminf(fmaxf(e[i], gp.lo), gp.hi);            // Clamp(X, q0, qmax)
          const float t = __fmul_rn(__fsub_rn(xc, gp.lo), gp.inv);      // (X' - q0) * (1/Delta)
          int c = __float2int_rn(t);                                    // round half to even
          c = min(max(c, 0), L);
          field |= (uint32_t)c << (BITS * i);
        }
        // word `lane` of this unit collects the fields that overlap its 32 bits
        uint32_t word = 0;
#pragma unroll
        for (int s = 0; s < NSRC; ++s) {
          const int src = first_src + s;
          const uint32_t f = __shfl_sync(0xffffffffu, field, src & 31);
          const int off = src * F - 32 * lane;  // position of that field relative to the word
          if (off >= 0) {
            if (off < 32) word |= f << off;
          } else {
            word |= f >> (-off);
          }
        }
        if (lane < WORDS) packed[(u + j) * WORDS + lane] = word;
        if (++col_unit == walk.units_per_row) {
          col_unit = 0;
          if (++row_in_group == walk.rows_per_group) {
            row_in_group = 0;
            ++g;
          }
        }
      }
    }
    u += nload;
  }
}

qb_status launch_quantize_pack_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                       const float* range_lo, const float* range_hi, uint32_t* packed,
                                       float* delta, float* q0, void* ws, int sm_count, cudaStream_t stream) {
  uint32_t* hi_enc = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + kWsRangeOff);
  uint32_t* lo_inv = hi_enc + groups;
  QB_CUDA_TRY(cudaMemsetAsync(hi_enc, 0, sizeof(uint32_t) * 2 * (size_t)groups, stream));

  WeightWalk walk;
  walk.units_total = N * K / 128;
  walk.units_per_row = (int)(K / 128);
  walk.rows_per_group = (int)(N / groups);
  const int64_t max_warps = (int64_t)sm_count * 32;  // 4 blocks of 8 warps per SM
  int64_t upw = (walk.units_total + max_warps - 1) / max_warps;
  if (upw < 4) upw = 4;
  walk.units_per_warp = upw;
  const int64_t warps = (walk.units_total + upw - 1) / upw;
  const unsigned blocks = (unsigned)((warps + kWqWarps - 1) / kWqWarps);

  const float4* w4 = reinterpret_cast<const float4*>(w);
  weight_range_kernel<<<blocks, kWqThreads, 0, stream>>>(w4, walk, groups, hi_enc, lo_inv, ws);
  QB_CUDA_TRY(cudaGetLastError());
  switch (bits) {
#define QB_PACK_CASE(B)                                                                                      \
  case B:                                                                                                    \
    weight_pack_kernel<B><<<blocks, kWqThreads, 0, stream>>>(w4, walk, hi_enc, lo_inv, range_lo, range_hi,   \
                                                             packed, delta, q0, ws);                         \
    break;
    QB_PACK_CASE(2) QB_PACK_CASE(3) QB_PACK_CASE(4) QB_PACK_CASE(8)
#undef QB_PACK_CASE
    default: return QB_ERR_INVALID;
  }
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}

}  // namespace qb

extern "C" qb_status qb_quantize_pack_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                              const float* range_lo, const float* range_hi, uint32_t* packed,
                                              float* delta, float* q0, void* ws, size_t ws_bytes,
                                              void* cuda_stream) {
  if (!w || !packed || !delta || !q0 || N <= 0 || K <= 0 || N > QB_MAX_MN || K > QB_MAX_K ||
      !qb::valid_bits(bits) || groups < 1 || N % groups != 0 || ((range_lo == nullptr) != (range_hi == nullptr))) {
    qb::set_last_error("qb_quantize_pack_weights: invalid argument (N=%lld K=%lld bits=%d groups=%d)",
                       (long long)N, (long long)K, bits, groups);
    return QB_ERR_INVALID;
  }
  if (K % 128 != 0 || !qb::aligned16(w) || !qb::aligned16(packed)) {
    qb::set_last_error("qb_quantize_pack_weights: K must be a multiple of 128 and w, packed 16-byte aligned");
    return QB_ERR_ALIGN;
  }
  if (!ws || ws_bytes < qb::ws_bytes_needed(groups)) {
    qb::set_last_error("qb_quantize_pack_weights: workspace null or smaller than %zu bytes",
                       qb::ws_bytes_needed(groups));
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  return qb::launch_quantize_pack_weights(w, N, K, bits, groups, range_lo, range_hi, packed, delta, q0, ws, sms,
                                          (cudaStream_t)cuda_stream);
}
