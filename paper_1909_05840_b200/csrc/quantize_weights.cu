// qb_quantize_pack_weights(_batch): group-wise uniform quantizer Q (Section 3.3, Appendix A) and dense
// k-bit packing (Table 1 counts exactly k bits per weight), for one matrix or a batch of matrices.
//
// Two paths, chosen per matrix on the host:
//   weight_regs_kernel   one read of W; any bit widths in one launch.  With the group's own [min, max]: groups
//                        of up to 288 units stay in the registers of one CTA between the range and the
//                        rounding, groups of up to 2,304 units in those of a thread-block cluster.  With
//                        caller-supplied ranges: groups of any size (nothing to reduce).
//   two passes           own ranges of larger groups (a range per tensor, say), below.
//
// Two-pass path, first pass: the matrices of a launch are walked as one sequence of "units" of 128
// consecutive elements of one row (one float4 per lane, fully coalesced; K % 128 == 0 so a unit never
// crosses a row).  Each warp owns a contiguous run of units, so it crosses few group (and matrix)
// boundaries: weight_range_kernel keeps a running min/max per lane, reduces over the warp when the group
// changes and publishes with atomicMax on order-preserving integer encodings in the workspace (block-level
// merge of the final partials first).  Second pass: weight_regs_kernel in its supplied-ranges form, reading
// those encodings (the matrix comes from L2 as far as L2 holds it).
#include <algorithm>
#include <atomic>
#include <cstring>
#include <vector>

#include "common.cuh"
#include "ptx.cuh"

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
  float keep_fraction;     // share of the input that L2 is asked to keep between the range pass and the next
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
  const uint64_t pol = policy_evict_last(b.keep_fraction);
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
        if (j < nload) v[j] = ldg_policy(m.w + (pos.u_local + j) * 32 + lane, pol);
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

// Range [lo, hi] of group g -> (q0, qmax, 1/Delta); lane-uniform.  Publishes Delta and q0 if asked.
// A caller-supplied range must be finite and ordered; a constant group gets Delta = 1, all codes 0.
__device__ __forceinline__ GroupParams finish_group(float lo, float hi, bool from_caller, int bits_levels, int g,
                                                    float* __restrict__ delta, float* __restrict__ q0,
                                                    bool publish, void* ws) {
  GroupParams p;
  p.lo = lo;
  p.hi = hi;
  if (from_caller) {
    const bool bad = !(fabsf(p.lo) <= 3.402823466e38f) || !(fabsf(p.hi) <= 3.402823466e38f) || p.hi < p.lo;
    if (bad) {
      if (publish) report_status(ws, QB_ERR_NONFINITE);
      p.lo = 0.0f;
      p.hi = 0.0f;
    }
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

// Delta of a finished group as finish_group publishes it (a constant group comes back with hi == lo: Delta = 1).
__device__ __forceinline__ float group_step(const GroupParams& gp, int bits_levels) {
  const float d = __fdiv_rn(__fsub_rn(gp.hi, gp.lo), (float)bits_levels);
  return d > 0.0f ? d : 1.0f;
}

// ---- straight-through backward (quantization-aware fine-tuning) ----------------------------------------
// Backward (straight-through estimator): the gradient passes where Clamp passes X (lo_g <= x <= hi_g).
__global__ void __launch_bounds__(256)
ste_backward_kernel(const float4* __restrict__ grad_q, const float4* __restrict__ w, int64_t n4, int64_t k4,
                    int64_t rows_per_group, const float* __restrict__ lo, const float* __restrict__ hi,
                    float4* __restrict__ grad_w) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const int64_t g = (i / k4) / rows_per_group;
    const float l = __ldg(lo + g), h = __ldg(hi + g);
    const float4 x = __ldg(w + i);
    float4 gq = __ldg(grad_q + i);
    gq.x = (x.x >= l && x.x <= h) ? gq.x : 0.0f;
    gq.y = (x.y >= l && x.y <= h) ? gq.y : 0.0f;
    gq.z = (x.z >= l && x.z <= h) ? gq.z : 0.0f;
    gq.w = (x.w >= l && x.w <= h) ? gq.w : 0.0f;
    grad_w[i] = gq;
  }
}

// ---- register-resident path ---------------------------------------------------------------------------
// Groups of up to 288 units (36,864 weights: all of BERT's matrices at 128 groups, and anything finer) are
// read from HBM once and stay in registers between the range and the rounding: 16 warps per CTA, one CTA
// per SM, every thread holds up to 18 float4 (one warp: 18 consecutive units, 9 KB, all loads in flight at
// once).  A matrix is served in one of two shapes:
//   * teams: a group is cut into contiguous slices over W = 1, 2, 4, 8 or 16 warps (the smallest W whose
//     slices fit), the team agrees on the range through shared memory and a named barrier;
//   * several groups per warp (groups of at most 9 units: one range per output row, say): a warp holds as
//     many whole consecutive groups as fit and reduces them one after the other.
// A CTA item is 16 warps' worth of consecutive groups of one matrix; the items of all matrices of a launch
// (largest items first, any mix of bit widths: the width is a field of the matrix) form one list that the
// CTAs stride over, so a mixed-precision stack is one launch.  Codes go through a 768-byte staging area per
// warp in blocks of six units: the 4k-bit fields laid down in element order are the packed stream for
// k = 2, 4, 8 (copied out with 16-byte stores) and are regrouped (eight 12-bit fields -> three words) for
// k = 3.  The kernel's other forms (template parameters, below): a thread-block cluster per group for
// groups of up to 2,304 units; fp32 Q(w) instead of packed words (fake quantization); supplied ranges
// (the caller's, or the range pass's for groups too large for a cluster), where nothing is reduced and
// the rounding clamps.
constexpr int kRgUnits = 18;                       // float4 per thread
constexpr int kRgBlock = 6;                        // units per staging block
constexpr int kRgWarps = 16;
constexpr int kRgThreads = 32 * kRgWarps;
constexpr int kRgMaxGroupUnits = kRgUnits * kRgWarps;  // 288
constexpr int kRgMaxBatch = 96;                    // matrices per launch

struct RegsItem {
  const float4* w;
  uint32_t* packed;
  float* delta;
  float* q0;
  int32_t ug;               // units per group
  int32_t groups;
  int32_t item_begin;       // first CTA item of this matrix in the launch's list
  int32_t groups_per_item;  // (16 / W) * groups_per_warp
  int16_t team_warps;       // W
  int16_t groups_per_warp;  // > 1 only with W = 1
  int16_t slice_units;      // units per warp of a team: ceil(ug / W)
  int16_t bits;
  const float* range_lo;    // caller-supplied ranges (the kernel that clamps), else null
  const float* range_hi;
  int32_t chunks;           // supplied ranges only: a group of more than 288 units is cut into this many items
  int32_t encoded;          // supplied ranges are the range pass's order-preserving encodings (max, inverted min)
};

struct RegsBatch {
  RegsItem item[kRgMaxBatch];
  void* ws;
  int32_t total_items;
  int32_t count;
};

// What one warp holds of a CTA item.
struct RegsSlice {
  const float4* src;  // first unit of the slice (+ lane)
  int32_t n;          // units held (0: nothing to do)
  int32_t it;         // matrix
  int32_t first_group;
  int32_t ng;         // groups (several-groups shape), 0 or 1 (teams)
  int32_t first_unit; // of the slice inside its group (teams)
};

__device__ __forceinline__ float min3_nan(float a, float b, float c) {
  float d;
  asm("min.NaN.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max3_nan(float a, float b, float c) {
  float d;
  asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Four codes of one float4 as a 4k-bit field in the low bits of the result (k < 8: bits from 22 up are
// left over from the rounding constant and are dropped by the narrow store that follows).
template <int BITS, bool CLAMP>
__device__ __forceinline__ uint32_t quant_field_open(float4 v, const float lo, const float inv, const float hi) {
  constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it rounds to an integer, half to even
  if (CLAMP) {  // Clamp(X, q0, qmax): a caller's range may leave weights outside
    v.x = fminf(fmaxf(v.x, lo), hi);
    v.y = fminf(fmaxf(v.y, lo), hi);
    v.z = fminf(fmaxf(v.z, lo), hi);
    v.w = fminf(fmaxf(v.w, lo), hi);
  }
  // Two lanes of fp32 per instruction (sub, mul, then the rounding add).  The add is written as a fused
  // multiply-add with 1.0: a packed mul followed by a packed add gets contracted into one fused operation,
  // which rounds the exact product instead of the rounded one and lands on the other side of a tie.
  uint32_t b0, b1, b2, b3;
  asm("{\n\t.reg .b64 p0, p1, l2, i2, m2, o2;\n\t"
      "mov.b64 p0, {%4, %5};\n\tmov.b64 p1, {%6, %7};\n\t"
      "mov.b64 l2, {%8, %8};\n\tmov.b64 i2, {%9, %9};\n\tmov.b64 m2, {%10, %10};\n\tmov.b64 o2, {%11, %11};\n\t"
      "sub.rn.f32x2 p0, p0, l2;\n\tsub.rn.f32x2 p1, p1, l2;\n\t"
      "mul.rn.f32x2 p0, p0, i2;\n\tmul.rn.f32x2 p1, p1, i2;\n\t"
      "fma.rn.f32x2 p0, p0, o2, m2;\n\tfma.rn.f32x2 p1, p1, o2, m2;\n\t"
      "mov.b64 {%0, %1}, p0;\n\tmov.b64 {%2, %3}, p1;\n\t}"
      : "=r"(b0), "=r"(b1), "=r"(b2), "=r"(b3)
      : "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "f"(lo), "f"(inv), "f"(kMagic), "f"(1.0f));
  if constexpr (BITS == 8) {
    return __byte_perm(__byte_perm(b0, b1, 0x0040), __byte_perm(b2, b3, 0x0040), 0x5410);
  } else {
    return b0 + (b1 << BITS) + (b2 << (2 * BITS)) + (b3 << (3 * BITS));
  }
}

// Parameters of the group a warp is rounding: q0, 1/Delta, and Delta (fake quantization only).
struct RgGroup {
  float lo, inv, d, hi;  // hi: the kernel that clamps only
};
// Several groups per warp: lane gi holds the parameters of the warp's group gi.
__device__ __forceinline__ void rg_next_group(RgGroup& cur, const RgGroup& mine, int& gi, int& next_start, const int ug) {
  cur.lo = __shfl_sync(0xffffffffu, mine.lo, gi);
  cur.inv = __shfl_sync(0xffffffffu, mine.inv, gi);
  cur.d = __shfl_sync(0xffffffffu, mine.d, gi);
  cur.hi = __shfl_sync(0xffffffffu, mine.hi, gi);
  ++gi;
  next_start += ug;
}

// One staging block (units BLK * 6 ... of the slice): fields into the warp's staging area, then out.
template <int BITS, int BLK, bool MULTI, bool CLAMP>
__device__ __forceinline__ void regs_pack_block(float4 (&v)[kRgUnits], const int n, RgGroup& cur, const RgGroup& mine,
                                                int& gi, int& next_start, const int ug, uint8_t* stg,
                                                uint32_t* __restrict__ out, const int lane,
                                                const float4* __restrict__ next_src, const int next_n) {
#pragma unroll
  for (int jj = 0; jj < kRgBlock; ++jj) {
    const int j = BLK * kRgBlock + jj;
    if (j < n) {
      if (MULTI) {
        if (j == next_start) rg_next_group(cur, mine, gi, next_start, ug);  // warp-uniform: the warp's next group begins
      }
      const uint32_t f = quant_field_open<BITS, CLAMP>(v[j], cur.lo, cur.inv, cur.hi);
      const int fi = jj * 32 + lane;  // field index = element index / 4 inside the block
      if (BITS == 8) reinterpret_cast<uint32_t*>(stg)[fi] = f;
      if (BITS == 4 || BITS == 3) reinterpret_cast<uint16_t*>(stg)[fi] = (uint16_t)f;
      if (BITS == 2) stg[fi] = (uint8_t)f;
    }
  }
  // the registers of this block are free: the same units of the warp's next slice start their way here
#pragma unroll
  for (int jj = 0; jj < kRgBlock; ++jj) {
    const int j = BLK * kRgBlock + jj;
    if (j < next_n) v[j] = __ldg(next_src + j * 32);
  }
  __syncwarp();
  const int nu = min(kRgBlock, n - BLK * kRgBlock);
  uint32_t* const o = out + BLK * kRgBlock * 4 * BITS;
  if (BITS == 3) {
    // 32 codes = eight 12-bit fields held in 16-bit cells -> three words; four such items per unit
    if (lane < 4 * nu) {
      const uint4 q = reinterpret_cast<const uint4*>(stg)[lane];
      const uint32_t f0 = q.x & 0xffffu, f1 = q.x >> 16, f2 = q.y & 0xffffu, f3 = q.y >> 16;
      const uint32_t f4 = q.z & 0xffffu, f5 = q.z >> 16, f6 = q.w & 0xffffu, f7 = q.w >> 16;
      uint32_t* o3 = o + lane * 3;
      o3[0] = f0 | (f1 << 12) | (f2 << 24);
      o3[1] = (f2 >> 8) | (f3 << 4) | (f4 << 16) | (f5 << 28);
      o3[2] = (f5 >> 4) | (f6 << 8) | (f7 << 20);
    }
  } else {
    const int n16 = nu * BITS;  // 16 * BITS bytes per unit
    const uint4* pk = reinterpret_cast<const uint4*>(stg);
    uint4* o4 = reinterpret_cast<uint4*>(o);
#pragma unroll
    for (int r = 0; r < (kRgBlock * BITS + 31) / 32; ++r) {
      const int i = r * 32 + lane;
      if (i < n16) o4[i] = pk[i];
    }
  }
  __syncwarp();  // the staging area is free again
}

// Fake quantization (Appendix A, forward of the fine-tuning step): Q(w) = Delta * code + q0 as fp32, written
// where the packed words would go.  code = (t + 1.5 * 2^23) - 1.5 * 2^23 is the rounded product as a float
// (exact), then one fused multiply-add; packed two lanes wide like the rounding itself.
template <bool CLAMP>
__device__ __forceinline__ float4 fake_quant4(float4 v, const RgGroup& g) {
  constexpr float kMagic = 12582912.0f;
  float4 q;
  if (CLAMP) {
    v.x = fminf(fmaxf(v.x, g.lo), g.hi);
    v.y = fminf(fmaxf(v.y, g.lo), g.hi);
    v.z = fminf(fmaxf(v.z, g.lo), g.hi);
    v.w = fminf(fmaxf(v.w, g.lo), g.hi);
  }
  asm("{\n\t.reg .b64 p0, p1, l2, i2, m2, o2, d2;\n\t"
      "mov.b64 p0, {%4, %5};\n\tmov.b64 p1, {%6, %7};\n\t"
      "mov.b64 l2, {%8, %8};\n\tmov.b64 i2, {%9, %9};\n\tmov.b64 m2, {%10, %10};\n\tmov.b64 o2, {%11, %11};\n\t"
      "mov.b64 d2, {%12, %12};\n\t"
      "sub.rn.f32x2 p0, p0, l2;\n\tsub.rn.f32x2 p1, p1, l2;\n\t"
      "mul.rn.f32x2 p0, p0, i2;\n\tmul.rn.f32x2 p1, p1, i2;\n\t"
      "fma.rn.f32x2 p0, p0, o2, m2;\n\tfma.rn.f32x2 p1, p1, o2, m2;\n\t"
      "sub.rn.f32x2 p0, p0, m2;\n\tsub.rn.f32x2 p1, p1, m2;\n\t"
      "fma.rn.f32x2 p0, d2, p0, l2;\n\tfma.rn.f32x2 p1, d2, p1, l2;\n\t"
      "mov.b64 {%0, %1}, p0;\n\tmov.b64 {%2, %3}, p1;\n\t}"
      : "=f"(q.x), "=f"(q.y), "=f"(q.z), "=f"(q.w)
      : "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "f"(g.lo), "f"(g.inv), "f"(kMagic), "f"(1.0f), "f"(g.d));
  return q;
}

template <int BLK, bool MULTI, bool CLAMP>
__device__ __forceinline__ void regs_fake_block(float4 (&v)[kRgUnits], const int n, RgGroup& cur, const RgGroup& mine,
                                                int& gi, int& next_start, const int ug, float4* __restrict__ out,
                                                const float4* __restrict__ next_src, const int next_n) {
#pragma unroll
  for (int jj = 0; jj < kRgBlock; ++jj) {
    const int j = BLK * kRgBlock + jj;
    if (j < n) {
      if (MULTI) {
        if (j == next_start) rg_next_group(cur, mine, gi, next_start, ug);
      }
      out[j * 32] = fake_quant4<CLAMP>(v[j], cur);
    }
    if (j < next_n) v[j] = __ldg(next_src + j * 32);
  }
}

template <int BLK, bool MULTI, bool FAKE, bool CLAMP>
__device__ __forceinline__ void regs_pack_block_any(const int bits, float4 (&v)[kRgUnits], const int n, RgGroup& cur,
                                                    const RgGroup& mine, int& gi, int& next_start, const int ug,
                                                    uint8_t* stg, uint32_t* __restrict__ out, const int lane,
                                                    const float4* __restrict__ next_src, const int next_n) {
  if (BLK * kRgBlock >= n) {  // nothing of this slice here: only the next slice's loads
#pragma unroll
    for (int jj = 0; jj < kRgBlock; ++jj) {
      const int j = BLK * kRgBlock + jj;
      if (j < next_n) v[j] = __ldg(next_src + j * 32);
    }
    return;
  }
  if (FAKE) {
    regs_fake_block<BLK, MULTI, CLAMP>(v, n, cur, mine, gi, next_start, ug, reinterpret_cast<float4*>(out) + lane, next_src, next_n);
    return;
  }
  switch (bits) {  // CTA-uniform
    case 2: regs_pack_block<2, BLK, MULTI, CLAMP>(v, n, cur, mine, gi, next_start, ug, stg, out, lane, next_src, next_n); break;
    case 3: regs_pack_block<3, BLK, MULTI, CLAMP>(v, n, cur, mine, gi, next_start, ug, stg, out, lane, next_src, next_n); break;
    case 4: regs_pack_block<4, BLK, MULTI, CLAMP>(v, n, cur, mine, gi, next_start, ug, stg, out, lane, next_src, next_n); break;
    default: regs_pack_block<8, BLK, MULTI, CLAMP>(v, n, cur, mine, gi, next_start, ug, stg, out, lane, next_src, next_n); break;
  }
}

template <bool CLUSTER>
__device__ __forceinline__ RegsSlice regs_slice(const RegsBatch& b, const int id, int& it, const int warp,
                                                const int lane, const int crank) {
  RegsSlice s;
  s.n = 0;
  s.it = it;
  s.src = nullptr;
  s.first_group = 0;
  s.ng = 0;
  s.first_unit = 0;
  if (id >= b.total_items) return s;
  while (it + 1 < b.count && id >= b.item[it + 1].item_begin) ++it;
  const RegsItem& m = b.item[it];
  s.it = it;
  if (CLUSTER) {
    // one group per cluster item, cut into slices over the 16 warps of each of the cluster's CTAs
    s.first_group = id - m.item_begin;
    s.ng = 1;
    s.first_unit = (crank * kRgWarps + warp) * m.slice_units;
    s.n = min(max(m.ug - s.first_unit, 0), (int)m.slice_units);
  } else {
    const int W = m.team_warps;
    const int team = warp / W, tw = warp - team * W;
    if (m.chunks > 1) {
      // caller-supplied ranges, a group larger than a CTA's registers: no reduction ties the group together,
      // so it is cut into items of 288 units
      const int local = id - m.item_begin;
      s.first_group = local / m.chunks;
      s.ng = 1;
      s.first_unit = (local - s.first_group * m.chunks) * kRgMaxGroupUnits + warp * kRgUnits;
      s.n = min(max(m.ug - s.first_unit, 0), kRgUnits);
      s.src = m.w + ((int64_t)s.first_group * m.ug + s.first_unit) * 32 + lane;
      return s;
    }
    s.first_group = (id - m.item_begin) * m.groups_per_item + team * m.groups_per_warp;
    s.ng = min(max(m.groups - s.first_group, 0), (int)m.groups_per_warp);
    if (s.ng > 0) {
      if (m.groups_per_warp > 1) {
        s.n = s.ng * m.ug;
      } else {
        s.first_unit = tw * m.slice_units;
        s.n = min(max(m.ug - s.first_unit, 0), (int)m.slice_units);
      }
    }
  }
  s.src = m.w + ((int64_t)s.first_group * m.ug + s.first_unit) * 32 + lane;
  return s;
}

__device__ __forceinline__ uint32_t cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}

// CLUSTER = false: the kernel described above.  CLUSTER = true: groups of 289 to 2,304 units; a thread-block
// cluster of 2 to 8 CTAs (the launch's cluster size) holds one group, every CTA reduces its 16 slices,
// writes its range into every CTA's shared memory and the cluster's barrier publishes them.  Every CTA of a
// cluster runs the same number of items, so the barriers pair up; the last one also keeps a CTA's shared
// memory alive until no peer writes to it any more.
// Supplied range of group g: the caller's floats, or the encodings the range pass of the two-pass path left.
__device__ __forceinline__ GroupParams supplied_group(const RegsItem& m, int g, int L, bool publish, void* ws) {
  if (m.encoded) {
    const float lo = ordered_to_float(~__ldg(reinterpret_cast<const uint32_t*>(m.range_lo) + g));
    const float hi = ordered_to_float(__ldg(reinterpret_cast<const uint32_t*>(m.range_hi) + g));
    return finish_group(lo, hi, false, L, g, m.delta, m.q0, publish, ws);
  }
  return finish_group(__ldg(m.range_lo + g), __ldg(m.range_hi + g), true, L, g, m.delta, m.q0, publish, ws);
}

// FAKE: the fp32 fake-quantized matrix is written instead of packed words (`packed` of the item points to it).
// CLAMP: the ranges are supplied (`range_lo`, `range_hi` of the item: the caller's, or what the range pass of
// the two-pass path found): no reduction and no exchange, the weights are clamped into the range, and the pass
// over the registers only looks for NaN and Inf.
template <bool CLUSTER, bool FAKE, bool CLAMP>
__global__ void __launch_bounds__(kRgThreads, 1)
weight_regs_kernel(const __grid_constant__ RegsBatch b) {
  __shared__ __align__(16) uint8_t s_stage[kRgWarps][kRgBlock * 128];
  __shared__ uint32_t s_hi[2][kRgWarps], s_lo[2][kRgWarps];
  __shared__ uint32_t x_hi[2][8], x_lo[2][8];  // CLUSTER: the ranges of the cluster's CTAs
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* const stg = s_stage[warp];
  const float kInf = __int_as_float(0x7f800000);
  const int csize = CLUSTER ? (int)cluster_size() : 1;
  const int crank = CLUSTER ? (int)ptx::cluster_ctarank() : 0;
  const int id0 = (int)blockIdx.x / csize, stride = (int)gridDim.x / csize;  // items go to clusters
  int it = 0, prev_it = 0;
  float4 v[kRgUnits];
  RegsSlice s = regs_slice<CLUSTER>(b, id0, it, warp, lane, crank);
#pragma unroll
  for (int j = 0; j < kRgUnits; ++j)
    if (j < s.n) v[j] = __ldg(s.src + j * 32);
  for (int id = id0, round = 0; id < b.total_items; id += stride, ++round) {
    const RegsItem& m = b.item[s.it];
    // The exchange buffers below are double-buffered per run of items with the same teams; when the
    // matrix (and with it, possibly, the team size) changes, every warp of the CTA passes here first.
    if (!CLUSTER && s.it != prev_it) __syncthreads();
    prev_it = s.it;
    const int n = s.n;
    // the warp's slice of the CTA's next item: its loads are issued as the registers come free below
    const RegsSlice nx = regs_slice<CLUSTER>(b, id + stride, it, warp, lane, crank);
    const int W = m.team_warps;
    const int bits = m.bits;
    const int L = (1 << bits) - 1;
    // first output word of the slice: 4k packed words per unit, or the unit's 128 floats
    uint32_t* const out = m.packed + ((int64_t)s.first_group * m.ug + s.first_unit) * (FAKE ? 128 : 4 * bits);
    if (!CLUSTER && m.groups_per_warp > 1) {
      // ---- several whole groups in this warp ----
      const int ug = m.ug;
      float lo = kInf, hi = -kInf;
      uint32_t my_hi = 0, my_lo = 0;
      int end = ug, gi = 0;
#pragma unroll
      for (int j = 0; j < kRgUnits; ++j) {
        if (j < n) {
          lo = min3_nan(min3_nan(lo, v[j].x, v[j].y), v[j].z, v[j].w);
          hi = max3_nan(max3_nan(hi, v[j].x, v[j].y), v[j].z, v[j].w);
          if (!CLAMP && j + 1 == end) {  // warp-uniform
            const uint32_t e_hi = __reduce_max_sync(0xffffffffu, float_to_ordered(hi));
            const uint32_t e_lo = __reduce_max_sync(0xffffffffu, ~float_to_ordered(lo));
            if (lane == gi) {
              my_hi = e_hi;
              my_lo = e_lo;
            }
            ++gi;
            end += ug;
            lo = kInf;
            hi = -kInf;
          }
        }
      }
      // lane i finishes group i of the warp
      RgGroup mine{0.0f, 1.0f, 1.0f, 0.0f};
      if (CLAMP) {
        // hi / lo hold this lane's running extremes over all of the warp's groups: NaN or Inf anywhere shows
        if (__any_sync(0xffffffffu, !(fabsf(hi) <= 3.402823466e38f && fabsf(lo) <= 3.402823466e38f)) && lane == 0 && n > 0)
          report_status(b.ws, QB_ERR_NONFINITE);
      }
      if (lane < s.ng) {
        GroupParams gp;
        if (CLAMP) {
          gp = supplied_group(m, s.first_group + lane, L, true, b.ws);
        } else {
          const float g_hi = ordered_to_float(my_hi);
          const float g_lo = ordered_to_float(~my_lo);
          if (!(fabsf(g_hi) <= 3.402823466e38f && fabsf(g_lo) <= 3.402823466e38f)) report_status(b.ws, QB_ERR_NONFINITE);
          gp = finish_group(g_lo, g_hi, false, L, s.first_group + lane, m.delta, m.q0, true, b.ws);
        }
        mine.lo = gp.lo;
        mine.inv = gp.inv;
        mine.d = group_step(gp, L);
        mine.hi = gp.hi;
      }
      RgGroup cur{0.0f, 1.0f, 1.0f, 0.0f};
      int next_start = 0;
      gi = 0;
      regs_pack_block_any<0, true, FAKE, CLAMP>(bits, v, n, cur, mine, gi, next_start, ug, stg, out, lane, nx.src, nx.n);
      regs_pack_block_any<1, true, FAKE, CLAMP>(bits, v, n, cur, mine, gi, next_start, ug, stg, out, lane, nx.src, nx.n);
      regs_pack_block_any<2, true, FAKE, CLAMP>(bits, v, n, cur, mine, gi, next_start, ug, stg, out, lane, nx.src, nx.n);
    } else if (s.ng > 0) {
      // ---- a slice of one group (team-uniform: every warp of the team is here) ----
      float lo = kInf, hi = -kInf;
#pragma unroll
      for (int j = 0; j < kRgUnits; ++j) {
        if (j < n) {
          lo = min3_nan(min3_nan(lo, v[j].x, v[j].y), v[j].z, v[j].w);
          hi = max3_nan(max3_nan(hi, v[j].x, v[j].y), v[j].z, v[j].w);
        }
      }
      // NaN anywhere makes hi NaN (encoded above every number); Inf shows as hi = +Inf or lo = -Inf
      uint32_t e_hi = 0, e_lo = 0;
      if (!CLAMP) {
        e_hi = __reduce_max_sync(0xffffffffu, float_to_ordered(hi));
        e_lo = __reduce_max_sync(0xffffffffu, ~float_to_ordered(lo));
      }
      if (CLAMP) {
        if (__any_sync(0xffffffffu, !(fabsf(hi) <= 3.402823466e38f && fabsf(lo) <= 3.402823466e38f)) && lane == 0 && n > 0)
          report_status(b.ws, QB_ERR_NONFINITE);
      } else if (CLUSTER) {
        const int flip = round & 1;
        if (lane == 0) {
          s_hi[flip][warp] = e_hi;
          s_lo[flip][warp] = e_lo;
        }
        __syncthreads();
        e_hi = __reduce_max_sync(0xffffffffu, lane < kRgWarps ? s_hi[flip][lane] : 0u);
        e_lo = __reduce_max_sync(0xffffffffu, lane < kRgWarps ? s_lo[flip][lane] : 0u);
        if (warp == 0 && lane < csize) {  // this CTA's range into slot `crank` of CTA `lane`
          st_cluster_u32(ptx::map_to_cta(ptx::smem_u32(&x_hi[flip][crank]), (uint32_t)lane), e_hi);
          st_cluster_u32(ptx::map_to_cta(ptx::smem_u32(&x_lo[flip][crank]), (uint32_t)lane), e_lo);
        }
        ptx::cluster_sync_all();
        e_hi = __reduce_max_sync(0xffffffffu, lane < csize ? x_hi[flip][lane] : 0u);
        e_lo = __reduce_max_sync(0xffffffffu, lane < csize ? x_lo[flip][lane] : 0u);
      } else if (W > 1) {
        const int flip = round & 1;
        const int team0 = warp - (warp % W);  // first warp of the team
        if (lane == 0) {
          s_hi[flip][warp] = e_hi;
          s_lo[flip][warp] = e_lo;
        }
        asm volatile("bar.sync %0, %1;" ::"r"(1 + team0 / W), "r"(32 * W) : "memory");
        const uint32_t vh = lane < W ? s_hi[flip][team0 + lane] : 0u;
        const uint32_t vl = lane < W ? s_lo[flip][team0 + lane] : 0u;
        e_hi = __reduce_max_sync(0xffffffffu, vh);
        e_lo = __reduce_max_sync(0xffffffffu, vl);
      }
      const bool publish = s.first_unit == 0 && lane == 0;
      GroupParams gp;
      if (CLAMP) {
        gp = supplied_group(m, s.first_group, L, publish, b.ws);
      } else {
        const float g_hi = ordered_to_float(e_hi);
        const float g_lo = ordered_to_float(~e_lo);
        if (publish && !(fabsf(g_hi) <= 3.402823466e38f && fabsf(g_lo) <= 3.402823466e38f))
          report_status(b.ws, QB_ERR_NONFINITE);
        gp = finish_group(g_lo, g_hi, false, L, s.first_group, m.delta, m.q0, publish, b.ws);
      }
      RgGroup cur{gp.lo, gp.inv, group_step(gp, L), gp.hi};
      const RgGroup mine{0.0f, 1.0f, 1.0f, 0.0f};
      int gi = 0, next_start = -1;
      regs_pack_block_any<0, false, FAKE, CLAMP>(bits, v, n, cur, mine, gi, next_start, 0, stg, out, lane, nx.src, nx.n);
      regs_pack_block_any<1, false, FAKE, CLAMP>(bits, v, n, cur, mine, gi, next_start, 0, stg, out, lane, nx.src, nx.n);
      regs_pack_block_any<2, false, FAKE, CLAMP>(bits, v, n, cur, mine, gi, next_start, 0, stg, out, lane, nx.src, nx.n);
    } else {
      // nothing of this item here (a last item with fewer groups than teams): only the next slice's loads
#pragma unroll
      for (int j = 0; j < kRgUnits; ++j)
        if (j < nx.n) v[j] = __ldg(nx.src + j * 32);
    }
    s = nx;
  }
  if (CLUSTER) ptx::cluster_sync_all();
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
  int bits;
};

static qb_status launch_regs_single(const HostWeight* m, int count, bool ranged, void* ws, int sm_count,
                                    cudaStream_t stream, bool fake, bool encoded);

// Two-pass path (own ranges over groups too large for a cluster): one pair of launches over `count`
// matrices (<= kMaxWeightBatch).  Their range tables sit back to back in the workspace: maxima at
// ws + kWsRangeOff, inverted minima after them.  The second pass is the register-resident kernel in its
// supplied-ranges form, reading those tables.
static qb_status launch_two_pass(const HostWeight* m, int count, void* ws, int sm_count, cudaStream_t stream,
                                 bool fake = false) {
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
  b.keep_fraction = l2_keep_fraction(512.0 * (double)units);
  QB_CUDA_TRY(cudaMemsetAsync(b.hi_enc, 0, sizeof(uint32_t) * 2 * (size_t)total_groups, stream));

  const int64_t max_warps = (int64_t)sm_count * 32;  // 4 blocks of 8 warps per SM
  int64_t upw = (units + max_warps - 1) / max_warps;
  if (upw < 4) upw = 4;
  b.units_per_warp = upw;
  const int64_t warps = (units + upw - 1) / upw;
  const unsigned blocks = (unsigned)((warps + kWqWarps - 1) / kWqWarps);

  weight_range_kernel<<<blocks, kWqThreads, 0, stream>>>(b);
  QB_CUDA_TRY(cudaGetLastError());
  HostWeight second[kMaxWeightBatch];
  for (int i = 0; i < count; ++i) {
    second[i] = m[i];
    second[i].range_lo = reinterpret_cast<const float*>(b.lo_inv + b.item[i].group_begin);
    second[i].range_hi = reinterpret_cast<const float*>(b.hi_enc + b.item[i].group_begin);
  }
  return launch_regs_single(second, count, true, ws, sm_count, stream, fake, true);
}

static inline int64_t group_units(const HostWeight& h) { return (h.N / h.groups) * (h.K / 128); }

// Does a matrix take the register-resident path?  With its own ranges: groups of at most 288 units in one
// CTA, up to 2,304 in a cluster of up to 8 CTAs.  With the caller's ranges: always (nothing to reduce).
constexpr int kRgMaxCluster = 8;
static inline int regs_cluster_size(const HostWeight& h) {
  if (h.range_lo != nullptr) return 1;
  return (int)((group_units(h) + kRgMaxGroupUnits - 1) / kRgMaxGroupUnits);
}
static inline bool regs_eligible(const HostWeight& h) {
  return h.range_lo != nullptr || group_units(h) <= (int64_t)kRgMaxGroupUnits * kRgMaxCluster;
}

// Clusters of `cl` CTAs that can be resident at once (asked once per device and cluster size).
static qb_status regs_max_clusters(int cl, int* out) {
  static std::atomic<int> cached[64][kRgMaxCluster + 1] = {};
  int dev = 0;
  QB_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) {
    set_last_error("device ordinal %d out of range", dev);
    return QB_ERR_CUDA;
  }
  int n = cached[dev][cl].load(std::memory_order_acquire);
  if (n == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cl * 64u);
    cfg.blockDim = dim3(kRgThreads);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)cl;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    QB_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, weight_regs_kernel<true, false, false>, &cfg));
    if (n < 1) {
      set_last_error("no cluster of %d CTAs fits the device", cl);
      return QB_ERR_CUDA;
    }
    cached[dev][cl].store(n, std::memory_order_release);
  }
  *out = n;
  return QB_OK;
}

// Matrices whose groups need a cluster of `cl` CTAs (289 to 2,304 units per group), any bit widths: one
// group per cluster item.
static qb_status launch_regs_cluster(const HostWeight* m, int count, int cl, void* ws, cudaStream_t stream, bool fake) {
  int max_clusters = 0;
  qb_status st = regs_max_clusters(cl, &max_clusters);
  if (st != QB_OK) return st;
  for (int first = 0; first < count; first += kRgMaxBatch) {
    const int n = std::min(kRgMaxBatch, count - first);
    RegsBatch b;
    memset(&b, 0, sizeof(b));
    int items = 0;
    for (int i = 0; i < n; ++i) {
      const HostWeight& h = m[first + i];
      RegsItem& it = b.item[i];
      const int ug = (int)group_units(h);
      it.w = reinterpret_cast<const float4*>(h.w);
      it.packed = h.packed;
      it.delta = h.delta;
      it.q0 = h.q0;
      it.ug = ug;
      it.groups = h.groups;
      it.item_begin = items;
      it.groups_per_item = 1;
      it.team_warps = (int16_t)kRgWarps;
      it.groups_per_warp = 1;
      it.slice_units = (int16_t)((ug + kRgWarps * cl - 1) / (kRgWarps * cl));
      it.bits = (int16_t)h.bits;
      items += h.groups;
    }
    b.ws = ws;
    b.total_items = items;
    b.count = n;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(std::min(items, max_clusters) * cl));
    cfg.blockDim = dim3(kRgThreads);
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)cl;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (fake)
      QB_CUDA_TRY(cudaLaunchKernelEx(&cfg, weight_regs_kernel<true, true, false>, b));
    else
      QB_CUDA_TRY(cudaLaunchKernelEx(&cfg, weight_regs_kernel<true, false, false>, b));
  }
  return QB_OK;
}

// Matrices served by single CTAs (own ranges with groups of at most 288 units, or the caller's ranges with
// groups of any size: `ranged`), any bit widths: launches of up to kRgMaxBatch matrices, inside a launch
// the matrices with the largest CTA items first.
static qb_status launch_regs_single(const HostWeight* m, int count, bool ranged, void* ws, int sm_count,
                                    cudaStream_t stream, bool fake, bool encoded) {
  struct Shape {
    int idx, W, gpw, slice, gpi, chunks;
    int64_t item_units;
  };
  std::vector<Shape> sh(count);
  for (int i = 0; i < count; ++i) {
    const int64_t ug = group_units(m[i]);
    Shape& s = sh[i];
    s.idx = i;
    s.chunks = 1;
    if (ug > kRgMaxGroupUnits) {  // `ranged` only: the group is cut into items of 288 units
      s.W = kRgWarps;
      s.gpw = 1;
      s.slice = kRgUnits;
      s.gpi = 1;
      s.chunks = (int)((ug + kRgMaxGroupUnits - 1) / kRgMaxGroupUnits);
      s.item_units = kRgMaxGroupUnits;
      continue;
    }
    s.W = 1;
    while (s.W * kRgUnits < ug) s.W *= 2;
    s.gpw = s.W == 1 ? std::max(1, kRgUnits / (int)ug) : 1;
    s.slice = ((int)ug + s.W - 1) / s.W;
    s.gpi = (kRgWarps / s.W) * s.gpw;
    s.item_units = (int64_t)std::min(s.gpi, m[i].groups) * ug;
  }
  std::stable_sort(sh.begin(), sh.end(), [](const Shape& a, const Shape& b) { return a.item_units > b.item_units; });
  for (int first = 0; first < count; first += kRgMaxBatch) {
    const int n = std::min(kRgMaxBatch, count - first);
    RegsBatch b;
    memset(&b, 0, sizeof(b));
    int64_t items = 0;
    for (int i = 0; i < n; ++i) {
      const Shape& s = sh[first + i];
      const HostWeight& h = m[s.idx];
      RegsItem& it = b.item[i];
      it.w = reinterpret_cast<const float4*>(h.w);
      it.packed = h.packed;
      it.delta = h.delta;
      it.q0 = h.q0;
      it.ug = (int32_t)group_units(h);
      it.groups = h.groups;
      it.item_begin = (int32_t)items;
      it.groups_per_item = s.gpi;
      it.team_warps = (int16_t)s.W;
      it.groups_per_warp = (int16_t)s.gpw;
      it.slice_units = (int16_t)s.slice;
      it.bits = (int16_t)h.bits;
      it.range_lo = h.range_lo;
      it.range_hi = h.range_hi;
      it.chunks = s.chunks;
      it.encoded = encoded ? 1 : 0;
      items += s.chunks > 1 ? (int64_t)h.groups * s.chunks : (h.groups + s.gpi - 1) / s.gpi;
    }
    if (items > 0x7fffffff) {
      set_last_error("weight batch too large for one launch (%lld items)", (long long)items);
      return QB_ERR_INVALID;
    }
    b.ws = ws;
    b.total_items = (int32_t)items;
    b.count = n;
    const unsigned grid = (unsigned)std::min<int64_t>(items, sm_count);
    if (ranged) {
      if (fake)
        weight_regs_kernel<false, true, true><<<grid, kRgThreads, 0, stream>>>(b);
      else
        weight_regs_kernel<false, false, true><<<grid, kRgThreads, 0, stream>>>(b);
    } else {
      if (fake)
        weight_regs_kernel<false, true, false><<<grid, kRgThreads, 0, stream>>>(b);
      else
        weight_regs_kernel<false, false, false><<<grid, kRgThreads, 0, stream>>>(b);
    }
    QB_CUDA_TRY(cudaGetLastError());
  }
  return QB_OK;
}

// Register-resident path over any number of eligible matrices of any bit widths.  Matrices whose groups
// need a cluster go to launches of their cluster size, matrices with caller-supplied ranges to launches of
// the kernel that clamps.
static qb_status launch_regs(const HostWeight* m_all, int count_all, void* ws, int sm_count, cudaStream_t stream,
                             bool fake = false) {
  std::vector<HostWeight> single, ranged, clustered[kRgMaxCluster + 1];
  for (int i = 0; i < count_all; ++i) {
    if (m_all[i].range_lo != nullptr) {
      ranged.push_back(m_all[i]);
      continue;
    }
    const int cl = regs_cluster_size(m_all[i]);
    (cl <= 1 ? single : clustered[cl]).push_back(m_all[i]);
  }
  for (int cl = 2; cl <= kRgMaxCluster; ++cl) {
    if (clustered[cl].empty()) continue;
    qb_status st = launch_regs_cluster(clustered[cl].data(), (int)clustered[cl].size(), cl, ws, stream, fake);
    if (st != QB_OK) return st;
  }
  if (!ranged.empty()) {
    qb_status st = launch_regs_single(ranged.data(), (int)ranged.size(), true, ws, sm_count, stream, fake, false);
    if (st != QB_OK) return st;
  }
  if (single.empty()) return QB_OK;
  return launch_regs_single(single.data(), (int)single.size(), false, ws, sm_count, stream, fake, false);
}

// One pair of launches of the two-pass path: matrices of one bit width (<= kMaxWeightBatch).
struct WeightJob {
  HostWeight m[kMaxWeightBatch];
  int n;
  int bits;
};

static void plan_weight_batch(const HostWeight* m, int count, int bits, std::vector<WeightJob>& jobs) {
  WeightJob j;
  j.n = count;
  j.bits = bits;
  for (int i = 0; i < count; ++i) j.m[i] = m[i];
  jobs.push_back(j);
}

// The two-pass jobs of a call, one after the other (they share the range tables at the head of the workspace).
static qb_status run_weight_jobs(const std::vector<WeightJob>& jobs, void* ws, int sm_count, cudaStream_t stream) {
  for (const WeightJob& j : jobs) {
    qb_status st = launch_two_pass(j.m, j.n, ws, sm_count, stream);
    if (st != QB_OK) return st;
  }
  return QB_OK;
}

static qb_status launch_weight_batch(const HostWeight* m, int count, int bits, void* ws, int sm_count,
                                     cudaStream_t stream) {
  std::vector<HostWeight> regs, rest;
  for (int i = 0; i < count; ++i) (regs_eligible(m[i]) ? regs : rest).push_back(m[i]);
  if (!regs.empty()) {
    qb_status st = launch_regs(regs.data(), (int)regs.size(), ws, sm_count, stream);
    if (st != QB_OK) return st;
  }
  if (rest.empty()) return QB_OK;
  std::vector<WeightJob> jobs;
  for (size_t i = 0; i < rest.size(); i += kMaxWeightBatch)
    plan_weight_batch(rest.data() + i, (int)std::min<size_t>(kMaxWeightBatch, rest.size() - i), bits, jobs);
  return run_weight_jobs(jobs, ws, sm_count, stream);
}

// Fake quantization of one matrix: the register-resident kernel where the groups fit it, else the two passes.
static qb_status launch_fake_quantize(const float* w, int64_t N, int64_t K, int bits, int groups,
                                      const float* range_lo, const float* range_hi, float* wq, float* delta,
                                      float* q0, void* ws, int sm_count, cudaStream_t stream) {
  // `packed` of the descriptor points to the fp32 output
  const HostWeight h{w, N, K, groups, range_lo, range_hi, reinterpret_cast<uint32_t*>(wq), delta, q0, bits};
  if (regs_eligible(h)) return launch_regs(&h, 1, ws, sm_count, stream, true);
  return launch_two_pass(&h, 1, ws, sm_count, stream, true);
}

qb_status launch_quantize_pack_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                       const float* range_lo, const float* range_hi, uint32_t* packed,
                                       float* delta, float* q0, void* ws, int sm_count, cudaStream_t stream) {
  const HostWeight m{w, N, K, groups, range_lo, range_hi, packed, delta, q0, bits};
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

namespace qb {

// The launch plan of a batch: the matrices of the register-resident path, and the jobs of the others.
static void plan_batch(const qb_weight_desc* descs, int count, std::vector<HostWeight>& regs,
                       std::vector<WeightJob>& jobs) {
  // Matrices that fit the register-resident path (see regs_eligible): all bit widths in the same launches.
  // The others (own ranges over groups too large for a cluster) take the two passes: launches of one bit
  // width, at most kMaxWeightBatch matrices each; the range tables of a launch reuse the head of the
  // workspace (launches on one stream run in order).
  std::vector<int> order;
  for (int i = 0; i < count; ++i) {
    const qb_weight_desc& d = descs[i];
    const HostWeight h{d.w, d.N, d.K, d.groups, d.range_lo, d.range_hi, d.packed, d.delta, d.q0, d.bits};
    if (regs_eligible(h))
      regs.push_back(h);
    else
      order.push_back(i);
  }
  const int rest = (int)order.size();
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return descs[a].bits < descs[b].bits; });
  int i = 0;
  while (i < rest) {
    HostWeight m[kMaxWeightBatch];
    int n = 0;
    const int bits = descs[order[i]].bits;
    while (i < rest && n < kMaxWeightBatch && descs[order[i]].bits == bits) {
      const qb_weight_desc& d = descs[order[i]];
      m[n++] = HostWeight{d.w, d.N, d.K, d.groups, d.range_lo, d.range_hi, d.packed, d.delta, d.q0, d.bits};
      ++i;
    }
    plan_weight_batch(m, n, bits, jobs);
  }
}

}  // namespace qb

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
  std::vector<qb::HostWeight> regs;
  std::vector<qb::WeightJob> jobs;
  qb::plan_batch(descs, count, regs, jobs);
  if (!regs.empty()) {
    st = qb::launch_regs(regs.data(), (int)regs.size(), ws, sms, (cudaStream_t)cuda_stream);
    if (st != QB_OK) return st;
  }
  if (jobs.empty()) return QB_OK;
  return qb::run_weight_jobs(jobs, ws, sms, (cudaStream_t)cuda_stream);
}

extern "C" int32_t qb_quantize_pack_weights_launch_count(const qb_weight_desc* descs, int32_t count) {
  if (!descs || count <= 0) return 0;
  for (int i = 0; i < count; ++i) {
    const qb_weight_desc& d = descs[i];
    if (d.N <= 0 || d.K <= 0 || d.groups < 1 || d.N % d.groups != 0 || d.K % 128 != 0) return 0;
  }
  std::vector<qb::HostWeight> regs;
  std::vector<qb::WeightJob> jobs;
  qb::plan_batch(descs, count, regs, jobs);
  int per_cluster[qb::kRgMaxCluster + 1] = {};
  int ranged = 0;
  for (const qb::HostWeight& h : regs) {
    if (h.range_lo != nullptr)
      ++ranged;
    else
      ++per_cluster[std::max(1, qb::regs_cluster_size(h))];
  }
  int32_t n = (ranged + qb::kRgMaxBatch - 1) / qb::kRgMaxBatch;
  for (int cl = 1; cl <= qb::kRgMaxCluster; ++cl) n += (per_cluster[cl] + qb::kRgMaxBatch - 1) / qb::kRgMaxBatch;
  n += 2 * (int32_t)jobs.size();
  return n;
}

extern "C" qb_status qb_fake_quantize_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                              const float* range_lo, const float* range_hi, float* wq, float* delta,
                                              float* q0, void* ws, size_t ws_bytes, void* cuda_stream) {
  qb_status st = qb::validate_weight("qb_fake_quantize_weights", w, N, K, bits, groups, range_lo, range_hi,
                                     reinterpret_cast<const uint32_t*>(wq), delta, q0);
  if (st != QB_OK) return st;
  if (!ws || ws_bytes < qb::ws_bytes_needed(groups)) {
    qb::set_last_error("qb_fake_quantize_weights: workspace null or smaller than %zu bytes",
                       qb::ws_bytes_needed(groups));
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  return qb::launch_fake_quantize(w, N, K, bits, groups, range_lo, range_hi, wq, delta, q0, ws, sms,
                                  (cudaStream_t)cuda_stream);
}

extern "C" qb_status qb_fake_quantize_weights_batch(const qb_weight_desc* descs, int32_t count, void* ws,
                                                    size_t ws_bytes, void* cuda_stream) {
  if (!descs || count <= 0) {
    qb::set_last_error("qb_fake_quantize_weights_batch: descs null or count <= 0");
    return QB_ERR_INVALID;
  }
  int64_t total_groups = 0;
  for (int i = 0; i < count; ++i) {
    const qb_weight_desc& d = descs[i];
    qb_status st = qb::validate_weight("qb_fake_quantize_weights_batch", d.w, d.N, d.K, d.bits, d.groups, d.range_lo,
                                       d.range_hi, d.packed, d.delta, d.q0);
    if (st != QB_OK) return st;
    total_groups += d.groups;
  }
  if (total_groups > (1 << 24) || !ws || ws_bytes < qb::ws_bytes_needed((int)total_groups)) {
    qb::set_last_error("qb_fake_quantize_weights_batch: workspace null or smaller than %zu bytes (sum of groups %lld)",
                       qb::ws_bytes_needed((int)total_groups), (long long)total_groups);
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  std::vector<qb::HostWeight> regs, rest;
  for (int i = 0; i < count; ++i) {
    const qb_weight_desc& d = descs[i];
    const qb::HostWeight h{d.w, d.N, d.K, d.groups, d.range_lo, d.range_hi, d.packed, d.delta, d.q0, d.bits};
    (qb::regs_eligible(h) ? regs : rest).push_back(h);
  }
  if (!regs.empty()) {
    st = qb::launch_regs(regs.data(), (int)regs.size(), ws, sms, (cudaStream_t)cuda_stream, true);
    if (st != QB_OK) return st;
  }
  for (size_t i = 0; i < rest.size(); i += qb::kMaxWeightBatch) {  // own ranges over groups beyond a cluster: two passes
    st = qb::launch_two_pass(rest.data() + i, (int)std::min<size_t>(qb::kMaxWeightBatch, rest.size() - i), ws, sms,
                             (cudaStream_t)cuda_stream, true);
    if (st != QB_OK) return st;
  }
  return QB_OK;
}

extern "C" qb_status qb_ste_backward(const float* grad_wq, const float* w, int64_t N, int64_t K, int groups,
                                     const float* range_lo, const float* range_hi, float* grad_w,
                                     void* cuda_stream) {
  if (!grad_wq || !w || !grad_w || N <= 0 || K <= 0 || N > QB_MAX_MN || K > QB_MAX_K || groups < 1 ||
      N % groups != 0 || ((range_lo == nullptr) != (range_hi == nullptr))) {
    qb::set_last_error("qb_ste_backward: invalid argument (N=%lld K=%lld groups=%d)", (long long)N, (long long)K,
                       groups);
    return QB_ERR_INVALID;
  }
  if (K % 128 != 0 || !qb::aligned16(grad_wq) || !qb::aligned16(w) || !qb::aligned16(grad_w)) {
    qb::set_last_error("qb_ste_backward: K must be a multiple of 128 and grad_wq, w, grad_w 16-byte aligned");
    return QB_ERR_ALIGN;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  if (range_lo == nullptr) {  // the group's own [min, max]: every element is inside, the gradient passes unchanged
    if (grad_w != grad_wq)
      QB_CUDA_TRY(cudaMemcpyAsync(grad_w, grad_wq, sizeof(float) * (size_t)N * (size_t)K, cudaMemcpyDeviceToDevice,
                                  stream));
    return QB_OK;
  }
  const int64_t n4 = N * K / 4;
  int64_t blocks = (n4 + 256 * 4 - 1) / (256 * 4);
  if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
  qb::ste_backward_kernel<<<(unsigned)blocks, 256, 0, stream>>>(
      reinterpret_cast<const float4*>(grad_wq), reinterpret_cast<const float4*>(w), n4, K / 4, N / groups, range_lo,
      range_hi, reinterpret_cast<float4*>(grad_w));
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}
