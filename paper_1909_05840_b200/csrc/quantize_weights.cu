// qb_quantize_pack_weights(_batch): group-wise uniform quantizer Q (Section 3.3, Appendix A) and dense
// k-bit packing (Table 1 counts exactly k bits per weight), for one matrix or a batch of matrices of
// the same bit width in one pair of launches.
//
// The matrices of a launch are walked as one sequence of "units" of 128 consecutive elements of one
// row (one float4 per lane, fully coalesced; K % 128 == 0 so a unit never crosses a row).  Each warp
// owns a contiguous run of units, so it crosses few group (and matrix) boundaries.
//
// Kernel 1  weight_range_kernel  running min/max per lane, warp reduction when the group changes,
//                                atomicMax on order-preserving integer encodings in the workspace
//                                (block-level merge of the final partials first).
// Kernel 2  weight_pack_kernel   re-reads the unit (from L2 for BERT-sized matrices), computes four
//                                codes per lane, and assembles the unit's 4k output words with warp
//                                shuffles so that the stores are contiguous 16k-byte runs.
#include <algorithm>
#include <cstring>
#include <vector>

#include "common.cuh"

namespace qb {

constexpr int kWqThreads = 256;
constexpr int kWqWarps = kWqThreads / 32;
constexpr int kMaxWeightBatch = 32;  // matrices per launch (descriptors travel as kernel parameters)

struct WeightItem {
  const float4* w;
  uint32_t* packed;
  float* delta;
  float* q0;
  const float* range_lo;
  const float* range_hi;
  int64_t unit_begin;      // index of the matrix's first unit in the launch
  int64_t units;           // N * K / 128
  int32_t units_per_row;   // K / 128
  int32_t rows_per_group;  // R
  int32_t group_begin;     // index of the matrix's first group in the launch's range tables
  int32_t pad;
};

struct WeightBatch {
  WeightItem item[kMaxWeightBatch];
  uint32_t* hi_enc;        // [groups of the launch] encoded maxima
  uint32_t* lo_inv;        // [groups of the launch] inverted encoded minima
  void* ws;
  int64_t units_total;
  int64_t units_per_warp;  // contiguous run per warp
  int32_t count;
};

// Position of a warp in the launch's unit sequence.
struct UnitWalk {
  int it;             // matrix
  int64_t u_local;    // unit inside the matrix
  int col_unit;       // unit inside the row
  int row_in_group;
  int g;              // group, numbered over the whole launch
  __device__ __forceinline__ void seek(const WeightBatch& b, int64_t u) {
    it = 0;
    while (it + 1 < b.count && u >= b.item[it + 1].unit_begin) ++it;
    enter(b, u - b.item[it].unit_begin);
  }
  __device__ __forceinline__ void enter(const WeightBatch& b, int64_t local) {
    const WeightItem& m = b.item[it];
    u_local = local;
    const int64_t row = local / m.units_per_row;
    col_unit = (int)(local - row * m.units_per_row);
    const int gl = (int)(row / m.rows_per_group);
    row_in_group = (int)(row - (int64_t)gl * m.rows_per_group);
    g = m.group_begin + gl;
  }
  // one unit forward; moves to the next matrix at the end of this one
  __device__ __forceinline__ void advance(const WeightBatch& b) {
    const WeightItem& m = b.item[it];
    ++u_local;
    if (++col_unit == m.units_per_row) {
      col_unit = 0;
      if (++row_in_group == m.rows_per_group) {
        row_in_group = 0;
        ++g;
      }
    }
    if (u_local == m.units && it + 1 < b.count) {
      ++it;
      enter(b, 0);
    }
  }
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
weight_range_kernel(const __grid_constant__ WeightBatch b) {
  const int lane = threadIdx.x & 31;
  const int warp_in_block = threadIdx.x >> 5;
  const int64_t gwarp = (int64_t)blockIdx.x * kWqWarps + warp_in_block;
  int64_t u = gwarp * b.units_per_warp;
  int64_t u_end = u + b.units_per_warp;
  if (u_end > b.units_total) u_end = b.units_total;

  __shared__ int s_group[kWqWarps];
  __shared__ uint32_t s_hi[kWqWarps], s_lo[kWqWarps];

  const float kInf = __int_as_float(0x7f800000);
  float lo = kInf, hi = -kInf;
  uint32_t absmax = 0;
  int cur_g = -1;
  if (u < u_end) {
    UnitWalk pos;
    pos.seek(b, u);
    cur_g = pos.g;
    while (u < u_end) {
      // up to four units of the current matrix in flight
      const WeightItem& m = b.item[pos.it];
      const int nload = (int)min(min((int64_t)4, u_end - u), m.units - pos.u_local);
      float4 v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (j < nload) v[j] = __ldg(m.w + (pos.u_local + j) * 32 + lane);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (j < nload) {
          if (pos.g != cur_g) {  // warp-uniform
            flush_range(b.hi_enc, b.lo_inv, cur_g, lo, hi);
            cur_g = pos.g;
            lo = kInf;
            hi = -kInf;
          }
          lo = fminf(fminf(lo, v[j].x), fminf(v[j].y, fminf(v[j].z, v[j].w)));
          hi = fmaxf(fmaxf(hi, v[j].x), fmaxf(v[j].y, fmaxf(v[j].z, v[j].w)));
          absmax = max(absmax, max(max(__float_as_uint(v[j].x) << 1, __float_as_uint(v[j].y) << 1),
                                   max(__float_as_uint(v[j].z) << 1, __float_as_uint(v[j].w) << 1)));
          pos.advance(b);
        }
      }
      u += nload;
    }
  }
  // NaN / Inf: exponent all ones survives the shift as >= 0xff000000
  absmax = __reduce_max_sync(0xffffffffu, absmax);
  if (lane == 0 && absmax >= 0xff000000u) report_status(b.ws, QB_ERR_NONFINITE);

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
      atomicMax(b.hi_enc + my_g, mh);
      atomicMax(b.lo_inv + my_g, ml);
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
weight_pack_kernel(const __grid_constant__ WeightBatch b) {
  constexpr int L = (1 << BITS) - 1;
  constexpr int F = 4 * BITS;          // bits contributed by one lane (four codes)
  constexpr int WORDS = 4 * BITS;      // output words per unit of 128 codes
  constexpr int NSRC = BITS == 8 ? 1 : (BITS == 4 ? 2 : 4);
  const int lane = threadIdx.x & 31;
  const int64_t gwarp = (int64_t)blockIdx.x * kWqWarps + (threadIdx.x >> 5);
  int64_t u = gwarp * b.units_per_warp;
  int64_t u_end = u + b.units_per_warp;
  if (u_end > b.units_total) u_end = b.units_total;
  if (u >= u_end) return;

  UnitWalk pos;
  pos.seek(b, u);
  int cur_g = -1;
  GroupParams gp{0.f, 0.f, 1.f};

  // which lanes feed output word `lane` of a unit (stream bits [32*lane, 32*lane + 32))
  const int first_src = (32 * lane) / F;

  while (u < u_end) {
    const WeightItem& m = b.item[pos.it];
    const int nload = (int)min(min((int64_t)4, u_end - u), m.units - pos.u_local);
    float4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (j < nload) v[j] = __ldg(m.w + (pos.u_local + j) * 32 + lane);
    uint32_t* const out_base = m.packed + pos.u_local * WORDS;
    const int group_begin = m.group_begin;
    const float* const rlo = m.range_lo;
    const float* const rhi = m.range_hi;
    float* const dl = m.delta;
    float* const qz = m.q0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (j < nload) {
        if (pos.g != cur_g) {  // warp-uniform
          cur_g = pos.g;
          // the warp that handles the first unit of the group publishes Delta and q0
          const bool publish = lane == 0 && pos.row_in_group == 0 && pos.col_unit == 0;
          const int gl = cur_g - group_begin;
          gp = load_group(gl, L, b.hi_enc + group_begin, b.lo_inv + group_begin, rlo, rhi, dl, qz, publish, b.ws);
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
        if (lane < WORDS) out_base[j * WORDS + lane] = word;
        pos.advance(b);
      }
    }
    u += nload;
  }
}

struct HostWeight {
  const float* w;
  int64_t N, K;
  int groups;
  const float* range_lo;
  const float* range_hi;
  uint32_t* packed;
  float* delta;
  float* q0;
};

// One pair of launches over `count` matrices (<= kMaxWeightBatch) of the same bit width.  Their range
// tables sit back to back in the workspace: maxima at ws + kWsRangeOff, inverted minima after them.
static qb_status launch_weight_batch(const HostWeight* m, int count, int bits, void* ws, int sm_count,
                                     cudaStream_t stream) {
  WeightBatch b;
  memset(&b, 0, sizeof(b));
  int total_groups = 0;
  int64_t units = 0;
  for (int i = 0; i < count; ++i) {
    WeightItem& it = b.item[i];
    it.w = reinterpret_cast<const float4*>(m[i].w);
    it.packed = m[i].packed;
    it.delta = m[i].delta;
    it.q0 = m[i].q0;
    it.range_lo = m[i].range_lo;
    it.range_hi = m[i].range_hi;
    it.unit_begin = units;
    it.units = m[i].N * m[i].K / 128;
    it.units_per_row = (int32_t)(m[i].K / 128);
    it.rows_per_group = (int32_t)(m[i].N / m[i].groups);
    it.group_begin = total_groups;
    units += it.units;
    total_groups += m[i].groups;
  }
  b.count = count;
  b.ws = ws;
  b.hi_enc = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + kWsRangeOff);
  b.lo_inv = b.hi_enc + total_groups;
  b.units_total = units;
  QB_CUDA_TRY(cudaMemsetAsync(b.hi_enc, 0, sizeof(uint32_t) * 2 * (size_t)total_groups, stream));

  const int64_t max_warps = (int64_t)sm_count * 32;  // 4 blocks of 8 warps per SM
  int64_t upw = (units + max_warps - 1) / max_warps;
  if (upw < 4) upw = 4;
  b.units_per_warp = upw;
  const int64_t warps = (units + upw - 1) / upw;
  const unsigned blocks = (unsigned)((warps + kWqWarps - 1) / kWqWarps);

  weight_range_kernel<<<blocks, kWqThreads, 0, stream>>>(b);
  QB_CUDA_TRY(cudaGetLastError());
  switch (bits) {
    case 2: weight_pack_kernel<2><<<blocks, kWqThreads, 0, stream>>>(b); break;
    case 3: weight_pack_kernel<3><<<blocks, kWqThreads, 0, stream>>>(b); break;
    case 4: weight_pack_kernel<4><<<blocks, kWqThreads, 0, stream>>>(b); break;
    case 8: weight_pack_kernel<8><<<blocks, kWqThreads, 0, stream>>>(b); break;
    default: return QB_ERR_INVALID;
  }
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}

qb_status launch_quantize_pack_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                       const float* range_lo, const float* range_hi, uint32_t* packed,
                                       float* delta, float* q0, void* ws, int sm_count, cudaStream_t stream) {
  const HostWeight m{w, N, K, groups, range_lo, range_hi, packed, delta, q0};
  return launch_weight_batch(&m, 1, bits, ws, sm_count, stream);
}

static qb_status validate_weight(const char* who, const float* w, int64_t N, int64_t K, int bits, int groups,
                                 const float* range_lo, const float* range_hi, const uint32_t* packed,
                                 const float* delta, const float* q0) {
  if (!w || !packed || !delta || !q0 || N <= 0 || K <= 0 || N > QB_MAX_MN || K > QB_MAX_K || !valid_bits(bits) ||
      groups < 1 || N % groups != 0 || ((range_lo == nullptr) != (range_hi == nullptr))) {
    set_last_error("%s: invalid argument (N=%lld K=%lld bits=%d groups=%d)", who, (long long)N, (long long)K, bits,
                   groups);
    return QB_ERR_INVALID;
  }
  if (K % 128 != 0 || !aligned16(w) || !aligned16(packed)) {
    set_last_error("%s: K must be a multiple of 128 and w, packed 16-byte aligned", who);
    return QB_ERR_ALIGN;
  }
  return QB_OK;
}

}  // namespace qb

extern "C" qb_status qb_quantize_pack_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                              const float* range_lo, const float* range_hi, uint32_t* packed,
                                              float* delta, float* q0, void* ws, size_t ws_bytes,
                                              void* cuda_stream) {
  qb_status st = qb::validate_weight("qb_quantize_pack_weights", w, N, K, bits, groups, range_lo, range_hi, packed,
                                     delta, q0);
  if (st != QB_OK) return st;
  if (!ws || ws_bytes < qb::ws_bytes_needed(groups)) {
    qb::set_last_error("qb_quantize_pack_weights: workspace null or smaller than %zu bytes",
                       qb::ws_bytes_needed(groups));
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  return qb::launch_quantize_pack_weights(w, N, K, bits, groups, range_lo, range_hi, packed, delta, q0, ws, sms,
                                          (cudaStream_t)cuda_stream);
}

extern "C" qb_status qb_quantize_pack_weights_batch(const qb_weight_desc* descs, int32_t count, void* ws,
                                                    size_t ws_bytes, void* cuda_stream) {
  if (!descs || count <= 0) {
    qb::set_last_error("qb_quantize_pack_weights_batch: descs null or count <= 0");
    return QB_ERR_INVALID;
  }
  int64_t total_groups = 0;
  for (int i = 0; i < count; ++i) {
    const qb_weight_desc& d = descs[i];
    qb_status st = qb::validate_weight("qb_quantize_pack_weights_batch", d.w, d.N, d.K, d.bits, d.groups, d.range_lo,
                                       d.range_hi, d.packed, d.delta, d.q0);
    if (st != QB_OK) return st;
    total_groups += d.groups;
  }
  if (total_groups > (1 << 24) || !ws || ws_bytes < qb::ws_bytes_needed((int)total_groups)) {
    qb::set_last_error("qb_quantize_pack_weights_batch: workspace null or smaller than %zu bytes (sum of groups %lld)",
                       qb::ws_bytes_needed((int)total_groups), (long long)total_groups);
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  // launches: same bit width, at most kMaxWeightBatch matrices each; the range tables of a launch
  // reuse the head of the workspace (launches on one stream run in order)
  std::vector<int> order(count);
  for (int i = 0; i < count; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return descs[a].bits < descs[b].bits; });
  int i = 0;
  while (i < count) {
    qb::HostWeight m[qb::kMaxWeightBatch];
    int n = 0;
    const int bits = descs[order[i]].bits;
    while (i < count && n < qb::kMaxWeightBatch && descs[order[i]].bits == bits) {
      const qb_weight_desc& d = descs[order[i]];
      m[n++] = qb::HostWeight{d.w, d.N, d.K, d.groups, d.range_lo, d.range_hi, d.packed, d.delta, d.q0};
      ++i;
    }
    st = qb::launch_weight_batch(m, n, bits, ws, sms, (cudaStream_t)cuda_stream);
    if (st != QB_OK) return st;
  }
  return QB_OK;
}
