// CPU oracle for the group-wise k-bit quantized linear layer of Q-BERT.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
// CUDA library is checked against.  It shares no source, header, table or
// helper with the CUDA path, and nothing in the product path may call it.
//
// Every function follows one passage of the paper and is written as the
// plain loop that passage describes: no blocking, no fusion, no intrinsics.
// fp32 arithmetic is written one IEEE-754 operation at a time (compile with
// -ffp-contract=off) so that a GPU kernel using round-to-nearest single
// operations reproduces it bit for bit.
//
// Readings taken where the paper is silent (each is listed with its reason in
// the design notes of the repository):
//   * quantization range of a group = its exact [min, max]      (Appendix A)
//   * round operator = IEEE round-half-to-even                  (Appendix A)
//   * (X' - q0) / Delta evaluated as (X' - q0) * (1 / Delta)    (Appendix A)
//   * constant group (max == min): Delta := 1, every code 0
//   * activations: dynamic per-tensor max-abs, signed 8 bit in [-127, 127]
//     (Table 1 caption only says "8-bits activation")
//   * packing: dense little-endian bit stream, exactly k bits per weight
//     (Table 1 sizes require k bits per weight, also for k = 3)
//
// Parity pins: every function below is pinned by the CPU tests against
// brute force, closed forms or invariants that do not call it (see tests).
// "parity unpinned": none in this file.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>

#if defined(_OPENMP)
#include <omp.h>
#endif

extern "C" {

enum { QO_OK = 0, QO_ERR_INVALID = -1, QO_ERR_NONFINITE = -5 };

int qo_num_threads(void) {
#if defined(_OPENMP)
  return omp_get_max_threads();
#else
  return 1;
#endif
}

static int qo_valid_bits(int bits) { return bits == 2 || bits == 3 || bits == 4 || bits == 8; }

// ---------------------------------------------------------------------------
// Section 3.3 (group-wise quantization) + Appendix A (uniform quantizer).
// W is [N][K] row-major, one row per output neuron.  Group g owns the R = N/G
// consecutive rows [g*R, (g+1)*R) and has its own range [q0, qmax].
//   X'  = Clamp(X, q0, qmax)
//   X^I = round((X' - q0) / Delta),  Delta = (qmax - q0) / (2^k - 1)
// Codes are unsigned integers in {0 .. 2^k - 1} (Section 3.1).
// If range_lo / range_hi are non-null they give the caller's [q0, qmax] per
// group (Appendix A allows a sub-interval of [min, max]); otherwise the exact
// min and max of the group are used.
// ---------------------------------------------------------------------------
int qo_quantize_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                        const float* range_lo, const float* range_hi,
                        uint8_t* codes, float* delta, float* q0) {
  if (!w || !codes || !delta || !q0 || N <= 0 || K <= 0 || groups < 1 || !qo_valid_bits(bits) ||
      N % groups != 0)
    return QO_ERR_INVALID;
  const int64_t R = N / groups;
  const int L = (1 << bits) - 1;
  int status = QO_OK;
#pragma omp parallel for schedule(static)
  for (int64_t g = 0; g < groups; ++g) {
    float lo = std::numeric_limits<float>::infinity();
    float hi = -std::numeric_limits<float>::infinity();
    bool finite = true;
    for (int64_t n = g * R; n < (g + 1) * R; ++n)
      for (int64_t k = 0; k < K; ++k) {
        const float v = w[n * K + k];
        if (!std::isfinite(v)) finite = false;
        if (v < lo) lo = v;
        if (v > hi) hi = v;
      }
    if (range_lo && range_hi) {
      lo = range_lo[g];
      hi = range_hi[g];
      if (!std::isfinite(lo) || !std::isfinite(hi) || hi < lo) finite = false;
    }
    if (!finite) {
#pragma omp atomic write
      status = QO_ERR_NONFINITE;
      delta[g] = 1.0f;
      q0[g] = 0.0f;
      for (int64_t n = g * R; n < (g + 1) * R; ++n)
        for (int64_t k = 0; k < K; ++k) codes[n * K + k] = 0;
      continue;
    }
    float d = (hi - lo) / (float)L;  // Delta, one IEEE division
    float inv = 1.0f / d;            // one IEEE division
    if (!(d > 0.0f) || !std::isfinite(inv)) {  // constant group (or a range too small to divide)
      d = 1.0f;
      inv = 1.0f;
      hi = lo;
    }
    delta[g] = d;
    q0[g] = lo;
    for (int64_t n = g * R; n < (g + 1) * R; ++n)
      for (int64_t k = 0; k < K; ++k) {
        float x = w[n * K + k];
        x = x < lo ? lo : x;  // Clamp(X, q0, qmax)
        x = x > hi ? hi : x;
        const float t = (x - lo) * inv;      // subtract, then multiply
        int u = (int)std::nearbyintf(t);     // round half to even
        u = u < 0 ? 0 : (u > L ? L : u);
        codes[n * K + k] = (uint8_t)u;
      }
  }
  return status;
}

// Appendix A, third line: Q(X) = Delta * X^I + q0, as one fused multiply-add.
void qo_dequantize_weights(const uint8_t* codes, int64_t N, int64_t K, int groups,
                           const float* delta, const float* q0, float* wq) {
  const int64_t R = N / groups;
  for (int64_t n = 0; n < N; ++n) {
    const int64_t g = n / R;
    for (int64_t k = 0; k < K; ++k)
      wq[n * K + k] = std::fmaf(delta[g], (float)codes[n * K + k], q0[g]);
  }
}

// ---------------------------------------------------------------------------
// Packed storage (Table 1 counts exactly k bits per weight).  Row n is a
// little-endian bit stream: code j occupies stream bits [k*j, k*j + k); the
// stream is stored as little-endian 32-bit words, K*k/32 words per row.
// Requires K*k % 32 == 0.
// ---------------------------------------------------------------------------
int qo_pack(const uint8_t* codes, int64_t N, int64_t K, int bits, uint32_t* words) {
  if (!qo_valid_bits(bits) || (K * bits) % 32 != 0) return QO_ERR_INVALID;
  const int64_t wpr = K * bits / 32;
  for (int64_t i = 0; i < N * wpr; ++i) words[i] = 0u;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t j = 0; j < K; ++j)
      for (int b = 0; b < bits; ++b) {
        const int64_t pos = (int64_t)bits * j + b;  // bit position in the row's stream
        if ((codes[n * K + j] >> b) & 1u) words[n * wpr + pos / 32] |= (1u << (pos % 32));
      }
  return QO_OK;
}

int qo_unpack(const uint32_t* words, int64_t N, int64_t K, int bits, uint8_t* codes) {
  if (!qo_valid_bits(bits) || (K * bits) % 32 != 0) return QO_ERR_INVALID;
  const int64_t wpr = K * bits / 32;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t j = 0; j < K; ++j) {
      unsigned u = 0;
      for (int b = 0; b < bits; ++b) {
        const int64_t pos = (int64_t)bits * j + b;
        u |= ((words[n * wpr + pos / 32] >> (pos % 32)) & 1u) << b;
      }
      codes[n * K + j] = (uint8_t)u;
    }
  return QO_OK;
}

// ---------------------------------------------------------------------------
// 8-bit activations (Table 1 caption).  Per-tensor, dynamic: a = max|x|,
// scale s = a/127, codes xq = clamp(round(x * (127/a)), -127, 127).  This is
// the Appendix A quantizer on the symmetric range [-a, a] with 255 points and
// the codes shifted by -127.  rowsum[m] = sum_k xq[m][k] (needed to carry the
// weights' offset q0 through the integer product).
// ---------------------------------------------------------------------------
int qo_quantize_act(const float* x, int64_t M, int64_t K, int8_t* xq, float* scale,
                    int32_t* rowsum) {
  if (!x || !xq || !scale || !rowsum || M <= 0 || K <= 0) return QO_ERR_INVALID;
  float a = 0.0f;
  bool finite = true;
  for (int64_t i = 0; i < M * K; ++i) {
    const float v = std::fabs(x[i]);
    if (!std::isfinite(v)) finite = false;
    if (v > a) a = v;
  }
  if (!finite) {
    *scale = 1.0f;
    for (int64_t i = 0; i < M * K; ++i) xq[i] = 0;
    for (int64_t m = 0; m < M; ++m) rowsum[m] = 0;
    return QO_ERR_NONFINITE;
  }
  float s = a / 127.0f;
  float inv = 127.0f / a;
  if (!(a > 0.0f) || !std::isfinite(inv)) {  // all-zero tensor
    s = 1.0f;
    inv = 0.0f;
  }
  *scale = s;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    int32_t sum = 0;
    for (int64_t k = 0; k < K; ++k) {
      int q = (int)std::nearbyintf(x[m * K + k] * inv);
      q = q < -127 ? -127 : (q > 127 ? 127 : q);
      xq[m * K + k] = (int8_t)q;
      sum += q;
    }
    rowsum[m] = sum;
  }
  return QO_OK;
}

// ---------------------------------------------------------------------------
// Appendix A, inference: "integer arithmetic for the matrix multiplication
// with X^I".  acc[m][n] = sum_k xq[m][k] * u[n][k], plain triple loop.
// acc64 (optional) receives the same sums in 64-bit, to prove no overflow.
// ---------------------------------------------------------------------------
void qo_int_gemm(const int8_t* xq, const uint8_t* codes, int64_t M, int64_t N, int64_t K,
                 int32_t* acc, int64_t* acc64) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      int32_t s = 0;
      int64_t s64 = 0;
      for (int64_t k = 0; k < K; ++k) {
        const int32_t p = (int32_t)xq[m * K + k] * (int32_t)codes[n * K + k];
        s += p;
        s64 += p;
      }
      acc[m * N + n] = s;
      if (acc64) acc64[m * N + n] = s64;
    }
}

// ---------------------------------------------------------------------------
// Appendix A, "gathered dequantization".  With Q(w) = Delta*u + q0 and
// x ~ s*xq, sum_k x*Q(w) = s*Delta_g*acc + s*q0_g*rowsum.  Evaluated in fp32
// about the centre code c = 2^(k-1), which keeps the two terms small when
// rowsum is large:
//   Ac = acc - c*rowsum            (int32, exact)
//   zc = fma(Delta_g, c, q0_g)     (value of code c)
//   alpha = s*Delta_g ; beta = s*zc
//   y = fma(alpha, float(Ac), fma(beta, float(rowsum), bias))
// bias may be null (treated as 0).
// ---------------------------------------------------------------------------
void qo_dequant_epilogue(const int32_t* acc, const int32_t* rowsum, float act_scale,
                         const float* delta, const float* q0, const float* bias, int64_t M,
                         int64_t N, int bits, int groups, float* y) {
  const int64_t R = N / groups;
  const int32_t c = 1 << (bits - 1);
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      const int64_t g = n / R;
      const int32_t Ac = acc[m * N + n] - c * rowsum[m];
      const float zc = std::fmaf(delta[g], (float)c, q0[g]);
      const float alpha = act_scale * delta[g];
      const float beta = act_scale * zc;
      const float b = bias ? bias[n] : 0.0f;
      y[m * N + n] = std::fmaf(alpha, (float)Ac, std::fmaf(beta, (float)rowsum[m], b));
    }
}

// The same linear layer straight from the definitions, in double precision:
// y[m][n] = sum_k (s*xq[m][k]) * Q(w)[n][k] + bias[n], Q(w) = Delta*u + q0.
// Used by the tests to bound the fp32 epilogue's rounding; never a gate for
// the GPU.
void qo_linear_fp64(const int8_t* xq, float act_scale, const uint8_t* codes, const float* delta,
                    const float* q0, const float* bias, int64_t M, int64_t N, int64_t K,
                    int groups, double* y) {
  const int64_t R = N / groups;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      const int64_t g = n / R;
      double s = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        const double xv = (double)act_scale * (double)xq[m * K + k];
        const double wv = (double)delta[g] * (double)codes[n * K + k] + (double)q0[g];
        s += xv * wv;
      }
      y[m * N + n] = s + (bias ? (double)bias[n] : 0.0);
    }
}

// Narrow output (the paper keeps the activations between layers at 8 bits, Table 1 caption, so a
// linear's fp32 result is an intermediate that the next operation narrows): the fp32 result of the
// dequantizing epilogue rounded to bfloat16 (8 significant bits, the exponent range of fp32), round to
// nearest, ties to the value whose last kept bit is 0.  Written as the definition: the two neighbours
// of y that bfloat16 can represent are found by dropping the 16 low bits (towards zero) and by one
// step of the kept field away from zero; the nearer one in exact arithmetic (double holds both
// differences exactly) is taken.  Inputs must be finite; a result that would overflow becomes
// infinity, as the step away from zero yields that bit pattern.
void qo_round_bf16(const float* y, int64_t n, uint16_t* out) {
  for (int64_t i = 0; i < n; ++i) {
    uint32_t u;
    std::memcpy(&u, &y[i], 4);
    const uint32_t lo_bits = u & 0xFFFF0000u;    // towards zero
    const uint32_t hi_bits = lo_bits + 0x10000u;  // one step away from zero (same sign bit)
    float lo, hi;
    std::memcpy(&lo, &lo_bits, 4);
    std::memcpy(&hi, &hi_bits, 4);
    const double d_lo = std::fabs((double)y[i] - (double)lo);
    const bool hi_finite = ((hi_bits >> 23) & 0xFFu) != 0xFFu;
    // distance to the upper neighbour; when that neighbour is infinity the value it stands for is
    // 2^128 (the next step of the same grid)
    const double hi_val = hi_finite ? (double)hi : std::ldexp((u >> 31) ? -1.0 : 1.0, 128);
    const double d_hi = std::fabs(hi_val - (double)y[i]);
    uint32_t r;
    if (d_lo < d_hi) r = lo_bits;
    else if (d_hi < d_lo) r = hi_bits;
    else r = ((lo_bits >> 16) & 1u) == 0u ? lo_bits : hi_bits;  // tie: last kept bit 0
    out[i] = (uint16_t)(r >> 16);
  }
}

// Backward pass of the quantizer for quantization-aware fine-tuning (Section 3.1 and Appendix A: the
// straight-through estimator is used for the gradient of X).  Q is Clamp followed by rounding onto the
// grid; the estimator treats the rounding as the identity, so the gradient of the loss with respect
// to X is the gradient with respect to Q(X) where Clamp passes X through (q0 <= X <= qmax of its
// group, both ends included) and zero where Clamp holds X at an end of the range.  With the default
// range [min, max] of the group every element is inside and the gradient passes unchanged.
// lo, hi: per group, [G]; rows of W are grouped as in qo_quantize_weights.
void qo_ste_backward(const float* grad_q, const float* w, int64_t N, int64_t K, int groups, const float* lo,
                     const float* hi, float* grad_w) {
  const int64_t R = N / groups;
  for (int64_t n = 0; n < N; ++n) {
    const int64_t g = n / R;
    for (int64_t k = 0; k < K; ++k) {
      const float x = w[n * K + k];
      grad_w[n * K + k] = (x >= lo[g] && x <= hi[g]) ? grad_q[n * K + k] : 0.0f;
    }
  }
}

// ---------------------------------------------------------------------------
// Embedding tables (Section 5.1 and the appendix on mixed-precision embedding: the 768 output
// neurons of the word and position embedding layers are bucketed into 128 groups; 4-bit word and
// 8-bit position embedding).  The table is stored as it is looked up, E[v][d] (one row per
// vocabulary entry or position, D embedding dimensions), so a group is a block of D / G consecutive
// COLUMNS over all V rows.  Per group the quantizer is Appendix A's Q with the group's exact
// [min, max], as in qo_quantize_weights; codes[v][d] in {0 .. 2^k - 1}.
// ---------------------------------------------------------------------------
int qo_quantize_embedding(const float* e, int64_t V, int64_t D, int bits, int groups, uint8_t* codes,
                          float* delta, float* q0) {
  if (!e || !codes || !delta || !q0 || V <= 0 || D <= 0 || groups < 1 || !qo_valid_bits(bits) || D % groups != 0)
    return QO_ERR_INVALID;
  const int64_t C = D / groups;  // columns per group
  const int L = (1 << bits) - 1;
  int status = QO_OK;
  for (int64_t g = 0; g < groups; ++g) {
    float lo = std::numeric_limits<float>::infinity();
    float hi = -std::numeric_limits<float>::infinity();
    bool finite = true;
    for (int64_t v = 0; v < V; ++v)
      for (int64_t d = g * C; d < (g + 1) * C; ++d) {
        const float x = e[v * D + d];
        if (!std::isfinite(x)) finite = false;
        if (x < lo) lo = x;
        if (x > hi) hi = x;
      }
    if (!finite) {
      status = QO_ERR_NONFINITE;
      delta[g] = 1.0f;
      q0[g] = 0.0f;
      for (int64_t v = 0; v < V; ++v)
        for (int64_t d = g * C; d < (g + 1) * C; ++d) codes[v * D + d] = 0;
      continue;
    }
    float dl = (hi - lo) / (float)L;
    float inv = 1.0f / dl;
    if (!(dl > 0.0f) || !std::isfinite(inv)) {  // constant group
      dl = 1.0f;
      inv = 1.0f;
      hi = lo;
    }
    delta[g] = dl;
    q0[g] = lo;
    for (int64_t v = 0; v < V; ++v)
      for (int64_t d = g * C; d < (g + 1) * C; ++d) {
        float x = e[v * D + d];
        x = x < lo ? lo : x;
        x = x > hi ? hi : x;
        const float t = (x - lo) * inv;
        int u = (int)std::nearbyintf(t);
        u = u < 0 ? 0 : (u > L ? L : u);
        codes[v * D + d] = (uint8_t)u;
      }
  }
  return status;
}

// Dequantizing lookup: out[t][d] (+)= Q(E)[ids[t]][d] = Delta_g * code + q0_g, g = d / (D / G).
// With `accumulate` the value is added to what out already holds (one fp32 addition), which is how
// the word and the position embedding of a token are summed.  ids must lie in [0, V).
int qo_embedding_lookup(const int32_t* ids, int64_t T, const uint8_t* codes, int64_t V, int64_t D, int groups,
                        const float* delta, const float* q0, int accumulate, float* out) {
  const int64_t C = D / groups;
  for (int64_t t = 0; t < T; ++t) {
    if (ids[t] < 0 || ids[t] >= V) return QO_ERR_INVALID;
    for (int64_t d = 0; d < D; ++d) {
      const int64_t g = d / C;
      const float q = std::fmaf(delta[g], (float)codes[(int64_t)ids[t] * D + d], q0[g]);
      out[t * D + d] = accumulate ? out[t * D + d] + q : q;
    }
  }
  return QO_OK;
}

// Re-quantized output: the fp32 result of a linear narrowed back to the 8-bit activation format that
// the next linear consumes (Table 1 caption: 8-bit activations throughout), with a scale s_out that the
// caller supplies (a static, calibrated activation scale).  It is qo_quantize_act's grid with a given
// step instead of the tensor's own maximum: code = clamp(round_half_even(y * (1 / s_out)), -127, 127);
// values beyond 127 * s_out saturate.  s_out must be finite and positive.
int qo_requantize_i8(const float* y, int64_t n, float s_out, int8_t* out) {
  if (!(s_out > 0.0f) || !std::isfinite(s_out)) return QO_ERR_INVALID;
  const float inv = 1.0f / s_out;  // one IEEE division
  for (int64_t i = 0; i < n; ++i) {
    const float t = y[i] * inv;
    int c = (int)std::nearbyintf(t < -128.0f ? -128.0f : (t > 128.0f ? 128.0f : t));
    c = c < -127 ? -127 : (c > 127 ? 127 : c);
    out[i] = (int8_t)c;
  }
  return QO_OK;
}

// Row sums of int8 codes (the rank-1 offset term of the next linear's epilogue needs them).
void qo_rowsum_i8(const int8_t* xq, int64_t M, int64_t K, int32_t* rowsum) {
  for (int64_t m = 0; m < M; ++m) {
    int32_t s = 0;
    for (int64_t k = 0; k < K; ++k) s += xq[m * K + k];
    rowsum[m] = s;
  }
}

// ---------------------------------------------------------------------------
// Section 3.2, Eq. 2: sensitivity of encoder layer i from the top Hessian eigenvalues lambda_i measured
// on `samples` portions of the training data (the caller supplies them; the power iteration that finds
// them is not part of this library):
//     Omega_i = |mean(lambda_i)| + std(lambda_i)
// and the paragraph after it: the layers are sorted by Omega in descending order and the order decides
// the precision relative to the other layers.
// Readings: std is the standard deviation of the empirical distribution of the given samples (divide by
// the number of samples, not by one less); equal Omega keep the lower layer index first; the paper gives
// no rule from rank to bit width, so the caller supplies `budget`, the bit width for rank 0 (most
// sensitive), rank 1, ...; `reverse` deals the budget from the least sensitive layer instead (the
// "MP-rev" ablation of the appendix).
// lambda: [layers][samples] fp64.  Outputs: omega [layers], order [layers] (order[r] = layer of rank r),
// bits [layers].  All arithmetic in fp64, sums taken in index order.
int qo_sensitivity_bits(const double* lambda, int layers, int samples, const int* budget, int reverse,
                        double* omega, int* order, int* bits) {
  if (layers < 1 || samples < 1) return QO_ERR_INVALID;
  for (int r = 0; r < layers; ++r)
    if (!qo_valid_bits(budget[r])) return QO_ERR_INVALID;
  for (int i = 0; i < layers; ++i) {
    const double* l = lambda + (int64_t)i * samples;
    double sum = 0.0;
    for (int s = 0; s < samples; ++s) {
      if (!std::isfinite(l[s])) return QO_ERR_NONFINITE;
      sum += l[s];
    }
    const double mean = sum / (double)samples;
    double sq = 0.0;
    for (int s = 0; s < samples; ++s) {
      const double d = l[s] - mean;
      sq += d * d;
    }
    omega[i] = std::fabs(mean) + std::sqrt(sq / (double)samples);
  }
  // descending order by repeated selection of the largest remaining Omega; ties: lower index first
  for (int i = 0; i < layers; ++i) order[i] = -1;
  for (int r = 0; r < layers; ++r) {
    int best = -1;
    for (int i = 0; i < layers; ++i) {
      bool taken = false;
      for (int q = 0; q < r; ++q) taken = taken || order[q] == i;
      if (taken) continue;
      if (best < 0 || omega[i] > omega[best]) best = i;
    }
    order[r] = best;
  }
  for (int r = 0; r < layers; ++r) bits[order[r]] = budget[reverse ? layers - 1 - r : r];
  return QO_OK;
}

}  // extern "C"
