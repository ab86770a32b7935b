// qb_quantize_embedding, qb_embedding_lookup: group-wise quantized embedding tables (Section 5.1 and the
// appendix on mixed-precision embedding: the embedding dimensions are bucketed into groups, 4-bit word
// and 8-bit position embedding) and the lookup that dequantizes the rows it gathers.
//
// The table stays in lookup order, E[v][d], so that a token's row of codes is one contiguous run of
// D*k/8 bytes; a group is therefore a block of D/G consecutive COLUMNS over all V rows.
//
// One thread owns four consecutive columns (blockDim = D/4, a warp = 128 columns = one packing unit):
//   emb_range_kernel   blocks stride over the rows; per-thread running min / max of its four columns,
//                      one atomicMax per column and block on order-preserving encodings in the workspace
//   emb_pack_kernel    every thread reduces the column ranges of its columns' groups (a few loads, once),
//                      then blocks stride over the rows: four codes per thread, the unit's 4k words
//                      assembled with warp shuffles, contiguous stores
//   emb_lookup_kernel  blocks stride over the tokens: the thread's 4k-bit field of the row, four fused
//                      multiply-adds with its columns' (Delta, q0), one float4 store (or add-and-store)
// All three are HBM-bound streams: 4 B, 4 B + k/8 B per table element, and k/8 B + 4 B per looked-up element.
#include "common.cuh"

namespace qb {

constexpr int kEmbMaxD = 4096;  // blockDim = D/4 <= 1024

__device__ __forceinline__ bool finite_f(float x) { return fabsf(x) <= 3.402823466e38f; }

// blockDim = (D/4) * slots: thread (slot, q) owns columns 4q..4q+3 of the rows slot, slot + slots, ... of the
// block's share; the slots of a block are merged in shared memory, so that few blocks (two per SM) with
// many loads in flight each take the place of many blocks that would queue on the same 2 D atomics.
__global__ void emb_range_kernel(const float4* __restrict__ e, int64_t V, int d4, int slots, float keep_fraction,
                                 uint32_t* __restrict__ col_hi, uint32_t* __restrict__ col_lo_inv, void* ws) {
  const uint64_t pol = policy_evict_last(keep_fraction);
  extern __shared__ uint32_t emb_smem[];  // [slots][2][4 * d4] encoded maxima / inverted minima
  const int q = threadIdx.x % d4, slot = threadIdx.x / d4;
  const float kInf = __int_as_float(0x7f800000);
  float lo[4] = {kInf, kInf, kInf, kInf}, hi[4] = {-kInf, -kInf, -kInf, -kInf};
  bool bad = false;
  const int64_t step = (int64_t)gridDim.x * slots;
  int64_t r = (int64_t)blockIdx.x * slots + slot;
  for (; r + 3 * step < V; r += 4 * step) {  // four rows in flight per thread
    float4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = ldg_policy(e + (r + j * step) * d4 + q, pol);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float x[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        bad = bad || !finite_f(x[i]);
        lo[i] = fminf(lo[i], x[i]);
        hi[i] = fmaxf(hi[i], x[i]);
      }
    }
  }
  for (; r < V; r += step) {
    const float4 v = ldg_policy(e + r * d4 + q, pol);
    const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      bad = bad || !finite_f(x[i]);
      lo[i] = fminf(lo[i], x[i]);
      hi[i] = fmaxf(hi[i], x[i]);
    }
  }
  if (bad) report_status(ws, QB_ERR_NONFINITE);
  const int D = 4 * d4;
  uint32_t* mine = emb_smem + (size_t)slot * 2 * D;
#pragma unroll
  for (int i = 0; i < 4; ++i) {  // a thread that saw no row contributes the neutral encodings of -inf / +inf
    mine[4 * q + i] = float_to_ordered(hi[i]);
    mine[D + 4 * q + i] = ~float_to_ordered(lo[i]);
  }
  __syncthreads();
  if (slot == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t eh = 0, el = 0;
      for (int s2 = 0; s2 < slots; ++s2) {
        eh = max(eh, emb_smem[(size_t)s2 * 2 * D + 4 * q + i]);
        el = max(el, emb_smem[(size_t)s2 * 2 * D + D + 4 * q + i]);
      }
      // the slots in the workspace only ever grow: skip the atomic when it cannot change anything
      if (eh > __ldcg(col_hi + 4 * q + i)) atomicMax(col_hi + 4 * q + i, eh);
      if (el > __ldcg(col_lo_inv + 4 * q + i)) atomicMax(col_lo_inv + 4 * q + i, el);
    }
  }
}

struct ColParams {
  float lo[4], hi[4], inv[4], d[4];
};

// Range of the group of column c (the reduced ranges of its D/G columns) -> q0, qmax, 1/Delta, Delta.
__device__ __forceinline__ void column_params(int c, int cols_per_group, int levels, const uint32_t* __restrict__ col_hi,
                                              const uint32_t* __restrict__ col_lo_inv, float* lo, float* hi,
                                              float* inv, float* d) {
  const int c0 = (c / cols_per_group) * cols_per_group;
  uint32_t eh = 0, el = 0;
  for (int j = 0; j < cols_per_group; ++j) {
    eh = max(eh, col_hi[c0 + j]);
    el = max(el, col_lo_inv[c0 + j]);
  }
  float l = ordered_to_float(~el), h = ordered_to_float(eh);
  if (!(finite_f(l) && finite_f(h))) {  // a non-finite table was reported by the range pass; stay in bounds
    l = 0.0f;
    h = 0.0f;
  }
  float dl = __fdiv_rn(__fsub_rn(h, l), (float)levels);
  float iv = __fdiv_rn(1.0f, dl);
  if (!(dl > 0.0f) || !(iv <= 3.402823466e38f)) {  // constant group
    dl = 1.0f;
    iv = 1.0f;
    h = l;
  }
  *lo = l;
  *hi = h;
  *inv = iv;
  *d = dl;
}

template <int BITS>
__global__ void emb_pack_kernel(const float4* __restrict__ e, int64_t V, int d4, int cols_per_group,
                                const uint32_t* __restrict__ col_hi, const uint32_t* __restrict__ col_lo_inv,
                                uint32_t* __restrict__ packed, float* __restrict__ delta, float* __restrict__ q0) {
  constexpr int L = (1 << BITS) - 1;
  constexpr int F = 4 * BITS;      // bits contributed by one thread (four codes)
  constexpr int WORDS = 4 * BITS;  // output words per unit of 128 codes
  constexpr int NSRC = BITS == 8 ? 1 : (BITS == 4 ? 2 : 4);
  const int q = threadIdx.x, lane = threadIdx.x & 31, unit = threadIdx.x >> 5;
  const uint64_t pol = policy_evict_first();
  ColParams p;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int c = 4 * q + i;
    column_params(c, cols_per_group, L, col_hi, col_lo_inv, &p.lo[i], &p.hi[i], &p.inv[i], &p.d[i]);
    if (blockIdx.x == 0 && c % cols_per_group == 0) {  // first column of a group publishes Delta and q0
      delta[c / cols_per_group] = p.d[i];
      q0[c / cols_per_group] = p.lo[i];
    }
  }
  const int first_src = (32 * lane) / F;  // lanes whose fields overlap output word `lane` of the unit
  const int64_t words_per_row = (int64_t)d4 * 4 * BITS / 32;
  auto pack_row = [&](int64_t r, const float4 v) {
    const float x[4] = {v.x, v.y, v.z, v.w};
    uint32_t field = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float xc = fminf(fmaxf(x[i], p.lo[i]), p.hi[i]);        // Clamp(X, q0, qmax)
      const float t = __fmul_rn(__fsub_rn(xc, p.lo[i]), p.inv[i]);  // (X' - q0) * (1/Delta)
      int c = __float2int_rn(t);                                    // round half to even
      c = min(max(c, 0), L);
      field |= (uint32_t)c << (BITS * i);
    }
    uint32_t word = 0;
#pragma unroll
    for (int s = 0; s < NSRC; ++s) {
      const int src = first_src + s;
      const uint32_t f = __shfl_sync(0xffffffffu, field, src & 31);
      const int off = src * F - 32 * lane;
      if (off >= 0) {
        if (off < 32) word |= f << off;
      } else {
        word |= f >> (-off);
      }
    }
    if (lane < WORDS) packed[r * words_per_row + unit * WORDS + lane] = word;
  };
  int64_t r = blockIdx.x;
  const int64_t step = gridDim.x;
  for (; r + 3 * step < V; r += 4 * step) {  // four rows in flight
    float4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = ldg_policy(e + (r + j * step) * d4 + q, pol);
#pragma unroll
    for (int j = 0; j < 4; ++j) pack_row(r + j * step, v[j]);
  }
  for (; r < V; r += step) pack_row(r, ldg_policy(e + r * d4 + q, pol));
}

template <int BITS>
__global__ void emb_lookup_kernel(const int32_t* __restrict__ ids, int64_t T, const uint32_t* __restrict__ packed,
                                  int64_t V, int d4, int cols_per_group, const float* __restrict__ delta,
                                  const float* __restrict__ q0, int accumulate, float4* __restrict__ out, void* ws) {
  constexpr uint32_t kMask = BITS == 8 ? 0xFFFFFFFFu : ((1u << (4 * BITS)) - 1u);
  const int q = threadIdx.x;
  float d[4], z[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int g = (4 * q + i) / cols_per_group;
    d[i] = __ldg(delta + g);
    z[i] = __ldg(q0 + g);
  }
  const int64_t words_per_row = (int64_t)d4 * 4 * BITS / 32;
  const int bit = 4 * q * BITS;  // position of this thread's field in the row's bit stream
  const int wi = bit >> 5, sh = bit & 31;
  for (int64_t t = blockIdx.x; t < T; t += gridDim.x) {
    const int id = __ldg(ids + t);
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (id >= 0 && id < V) {
      const uint32_t* row = packed + (int64_t)id * words_per_row;
      uint32_t f = __ldg(row + wi);
      if (BITS == 3 && sh + 12 > 32)
        f = __funnelshift_r(f, __ldg(row + wi + 1), sh);
      else
        f >>= sh;
      f &= kMask;
      constexpr uint32_t cm = (1u << BITS) - 1u;
      r.x = __fmaf_rn(d[0], (float)(f & cm), z[0]);
      r.y = __fmaf_rn(d[1], (float)((f >> BITS) & cm), z[1]);
      r.z = __fmaf_rn(d[2], (float)((f >> (2 * BITS)) & cm), z[2]);
      r.w = __fmaf_rn(d[3], (float)((f >> (3 * BITS)) & cm), z[3]);
    } else if (q == 0) {
      report_status(ws, QB_ERR_INVALID, (int)t);
    }
    float4* o = out + t * d4 + q;
    if (accumulate) {
      const float4 a = *o;
      r.x = __fadd_rn(a.x, r.x);
      r.y = __fadd_rn(a.y, r.y);
      r.z = __fadd_rn(a.z, r.z);
      r.w = __fadd_rn(a.w, r.w);
    }
    *o = r;
  }
}

static qb_status validate_embedding(const char* who, int64_t V, int64_t D, int bits, int groups) {
  if (V <= 0 || D <= 0 || V > QB_MAX_MN || D > kEmbMaxD || !valid_bits(bits) || groups < 1 || D % groups != 0) {
    set_last_error("%s: invalid argument (V=%lld D=%lld bits=%d groups=%d; D <= %d)", who, (long long)V, (long long)D,
                   bits, groups, kEmbMaxD);
    return QB_ERR_INVALID;
  }
  if (D % 128 != 0) {
    set_last_error("%s: D must be a multiple of 128", who);
    return QB_ERR_ALIGN;
  }
  return QB_OK;
}

}  // namespace qb

extern "C" qb_status qb_quantize_embedding(const float* table, int64_t V, int64_t D, int bits, int groups,
                                           uint32_t* packed, float* delta, float* q0, void* ws, size_t ws_bytes,
                                           void* cuda_stream) {
  if (!table || !packed || !delta || !q0) {
    qb::set_last_error("qb_quantize_embedding: null pointer");
    return QB_ERR_INVALID;
  }
  qb_status st = qb::validate_embedding("qb_quantize_embedding", V, D, bits, groups);
  if (st != QB_OK) return st;
  if (!qb::aligned16(table) || !qb::aligned16(packed)) {
    qb::set_last_error("qb_quantize_embedding: table and packed must be 16-byte aligned");
    return QB_ERR_ALIGN;
  }
  if (!ws || ws_bytes < qb::ws_bytes_needed((int)D)) {
    qb::set_last_error("qb_quantize_embedding: workspace null or smaller than %zu bytes (8 bytes per column)",
                       qb::ws_bytes_needed((int)D));
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  uint32_t* col_hi = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + qb::kWsRangeOff);
  uint32_t* col_lo = col_hi + D;
  QB_CUDA_TRY(cudaMemsetAsync(col_hi, 0, sizeof(uint32_t) * 2 * (size_t)D, stream));
  const int threads = (int)(D / 4);
  int per_sm = 2048 / threads;
  if (per_sm > 8) per_sm = 8;
  if (per_sm < 1) per_sm = 1;
  int64_t blocks = (int64_t)sms * per_sm;
  if (blocks > V) blocks = V;
  const float4* e4 = reinterpret_cast<const float4*>(table);
  {
    int slots = 1024 / threads;  // rows a block reads side by side
    if (slots > 4) slots = 4;
    int64_t rblocks = (int64_t)sms * 2;
    if (rblocks * slots > V) rblocks = (V + slots - 1) / slots;
    // slots * D <= 4096 columns (blockDim <= 1024 threads of four columns each): at most 32 KB
    const size_t smem = (size_t)slots * 2 * (size_t)D * sizeof(uint32_t);
    qb::emb_range_kernel<<<(unsigned)rblocks, threads * slots, smem, stream>>>(e4, V, threads, slots, qb::l2_keep_fraction(4.0 * (double)V * (double)D), col_hi, col_lo, ws);
    QB_CUDA_TRY(cudaGetLastError());
  }
  const int cpg = (int)(D / groups);
  switch (bits) {
    case 2: qb::emb_pack_kernel<2><<<(unsigned)blocks, threads, 0, stream>>>(e4, V, threads, cpg, col_hi, col_lo, packed, delta, q0); break;
    case 3: qb::emb_pack_kernel<3><<<(unsigned)blocks, threads, 0, stream>>>(e4, V, threads, cpg, col_hi, col_lo, packed, delta, q0); break;
    case 4: qb::emb_pack_kernel<4><<<(unsigned)blocks, threads, 0, stream>>>(e4, V, threads, cpg, col_hi, col_lo, packed, delta, q0); break;
    default: qb::emb_pack_kernel<8><<<(unsigned)blocks, threads, 0, stream>>>(e4, V, threads, cpg, col_hi, col_lo, packed, delta, q0); break;
  }
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}

extern "C" qb_status qb_embedding_lookup(const int32_t* ids, int64_t T, const uint32_t* packed, const float* delta,
                                         const float* q0, int64_t V, int64_t D, int bits, int groups,
                                         int accumulate, float* out, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!ids || !packed || !delta || !q0 || !out || T <= 0 || T > QB_MAX_MN) {
    qb::set_last_error("qb_embedding_lookup: null pointer or T out of range (T=%lld)", (long long)T);
    return QB_ERR_INVALID;
  }
  qb_status st = qb::validate_embedding("qb_embedding_lookup", V, D, bits, groups);
  if (st != QB_OK) return st;
  if (!qb::aligned16(packed) || !qb::aligned16(out)) {
    qb::set_last_error("qb_embedding_lookup: packed and out must be 16-byte aligned");
    return QB_ERR_ALIGN;
  }
  if (!ws || ws_bytes < qb::kWsMinBytes) {
    qb::set_last_error("qb_embedding_lookup: workspace null or too small");
    return QB_ERR_WORKSPACE;
  }
  int sms = 0;
  st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  const int threads = (int)(D / 4);
  int per_sm = 2048 / threads;
  if (per_sm > 8) per_sm = 8;
  if (per_sm < 1) per_sm = 1;
  int64_t blocks = (int64_t)sms * per_sm;
  if (blocks > T) blocks = T;
  const int cpg = (int)(D / groups);
  float4* o4 = reinterpret_cast<float4*>(out);
  const int acc = accumulate ? 1 : 0;
  switch (bits) {
    case 2: qb::emb_lookup_kernel<2><<<(unsigned)blocks, threads, 0, stream>>>(ids, T, packed, V, threads, cpg, delta, q0, acc, o4, ws); break;
    case 3: qb::emb_lookup_kernel<3><<<(unsigned)blocks, threads, 0, stream>>>(ids, T, packed, V, threads, cpg, delta, q0, acc, o4, ws); break;
    case 4: qb::emb_lookup_kernel<4><<<(unsigned)blocks, threads, 0, stream>>>(ids, T, packed, V, threads, cpg, delta, q0, acc, o4, ws); break;
    default: qb::emb_lookup_kernel<8><<<(unsigned)blocks, threads, 0, stream>>>(ids, T, packed, V, threads, cpg, delta, q0, acc, o4, ws); break;
  }
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}
