/*
 * libqbert — group-wise k-bit quantized transformer linear layers on NVIDIA B200 (sm_100a).
 *
 * The library implements the inference path of Q-BERT ("Hessian Based Ultra Low Precision
 * Quantization of BERT"): weights quantized by the paper's uniform quantizer Q with one range
 * per group of output neurons, 8-bit activations, an integer matrix product on the integer
 * codes and one dequantization at the end.
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - Pure C ABI.  Pointers marked "dev" are CUDA device pointers on the current device, pointers
 *    marked "host" are ordinary host pointers.  The caller owns every buffer; the library keeps no
 *    pointer after a call returns and allocates no device memory.
 *  - All device work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *    legacy default stream) and is asynchronous with respect to the host.
 *  - Argument errors are detected on the host, before anything is launched, and returned as a
 *    negative qb_status.  Conditions only the device can see (a non-finite input, a bounded wait
 *    that expired) are recorded in the status word at the head of the workspace `ws` (first error
 *    wins, it is never cleared by a kernel) and read back with qb_read_status.  After such a
 *    condition the outputs of that call are unspecified, but every write stays in bounds.
 *  - Matrices are row-major.  X is [M][K] (tokens x input features), W is [N][K] (output neurons x
 *    input features, the orientation of W in y = W x of Section 3.3), Y is [M][N].
 *  - bits (k) is one of 2, 3, 4, 8.  `groups` (G) splits the N rows of W into G blocks of
 *    R = N / G consecutive rows; N % G must be 0.  K must be a multiple of 128.
 *  - There is no CPU fallback: on a device that is not sm_100 every compute call returns
 *    QB_ERR_CUDA.
 */
#ifndef QBERT_H_
#define QBERT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t qb_status;

enum {
  QB_OK = 0,
  QB_ERR_INVALID = -1,   /* null pointer, bits not in {2,3,4,8}, G < 1, N % G != 0, size <= 0 or too large */
  QB_ERR_ALIGN = -2,     /* pointer not 16-byte aligned, or K not a multiple of 128 */
  QB_ERR_WORKSPACE = -3, /* workspace pointer null or smaller than qb_workspace_bytes() */
  QB_ERR_CUDA = -4,      /* CUDA runtime / driver error or unsupported device; text in qb_last_error() */
  QB_ERR_NONFINITE = -5, /* status word only: NaN or Inf met while reducing a range */
  QB_ERR_TIMEOUT = -6    /* status word only: a bounded device-side wait expired */
};

/* Largest sizes accepted (int32 accumulators stay exact: 127 * 255 * K < 2^31). */
#define QB_MAX_K 65536
#define QB_MAX_MN (1 << 24)

int qb_version(void);
const char* qb_status_string(qb_status s);
/* Text of the last error raised on the calling thread ("" if none).  Host pointer, valid until the
 * next failing call on this thread. */
const char* qb_last_error(void);

/* Number of 32-bit words of the packed form of an [N][K] matrix at `bits` bits per weight:
 * N * K * bits / 32 (Table 1 counts exactly k bits per weight).  0 on invalid arguments. */
size_t qb_packed_words(int64_t N, int64_t K, int bits);

/* Bytes of workspace any call on a problem of this size needs (>= 256).  Pass 0 for dimensions a
 * call does not have.  The workspace is device memory owned by the caller; one workspace may serve
 * consecutive calls on one stream.  It must be zeroed once with qb_workspace_init before first use. */
size_t qb_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits, int groups);

/* Zero the workspace (status word included) on the stream. */
qb_status qb_workspace_init(void* ws /*dev*/, size_t ws_bytes, void* cuda_stream);

/* Synchronize the stream and return the status word of the workspace: QB_OK, QB_ERR_NONFINITE or
 * QB_ERR_TIMEOUT (or QB_ERR_CUDA if the copy itself failed). */
qb_status qb_read_status(const void* ws /*dev*/, void* cuda_stream);

/*
 * 8-bit activation quantizer (Table 1 caption: every quantized model uses 8-bit activations).
 * The paper gives no further detail; this is Appendix A's uniform quantizer on the symmetric
 * per-tensor range [-a, a], a = max|x|, with 255 points and the codes shifted to [-127, 127]:
 *     act_scale = a / 127,   xq = clamp(round_half_even(x * (127 / a)), -127, 127),
 *     rowsum[m] = sum_k xq[m][k].
 * An all-zero tensor gives act_scale = 1 and zero codes.
 *   x         dev, fp32 [M][K], 16-byte aligned          (read)
 *   xq        dev, int8 [M][K], 16-byte aligned          (written)
 *   act_scale dev, fp32 [1]                              (written)
 *   rowsum    dev, int32 [M]                             (written)
 * Two kernels: a grid-wide max-abs reduction into the workspace, then round/clamp/store.
 */
qb_status qb_quantize_act(const float* x, int64_t M, int64_t K, int8_t* xq, float* act_scale,
                          int32_t* rowsum, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Group-wise weight quantizer and packer (Section 3.3 group-wise quantization; Appendix A):
 * for each group g of R = N / G consecutive rows, q0 = min, qmax = max over the group,
 *     Delta = (qmax - q0) / (2^k - 1),
 *     code  = clamp(round_half_even((clamp(w, q0, qmax) - q0) * (1 / Delta)), 0, 2^k - 1).
 * A constant group gets Delta = 1 and zero codes.  Codes are packed densely: row n is a
 * little-endian bit stream with code j in bits [k*j, k*j + k), stored as K*k/32 uint32 words.
 * G = 1 is the paper's layer-wise ("DirectQ") setting, G = N one range per output neuron.
 *   w        dev, fp32 [N][K], 16-byte aligned           (read)
 *   packed   dev, uint32 [N][K*bits/32], 16-byte aligned (written)
 *   delta,q0 dev, fp32 [G]                               (written)
 *   range_lo, range_hi: dev fp32 [G] or both NULL.  When given they replace the group's min and
 *            max (Appendix A: the range "can be a subinterval of [min, max]"); values outside are
 *            clamped.  They must be finite with range_lo <= range_hi.
 * One kernel (the weights are read once and stay in registers between the range and the rounding)
 * when the range is the group's own and the groups have at most 294,912 weights each (groups above
 * 36,864 weights are held by a thread-block cluster), and always with caller-supplied ranges
 * (nothing is reduced then); otherwise two kernels: per-group min/max reduction into the workspace,
 * then round/clamp/pack.
 */
qb_status qb_quantize_pack_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                   const float* range_lo, const float* range_hi, uint32_t* packed,
                                   float* delta, float* q0, void* ws, size_t ws_bytes,
                                   void* cuda_stream);

/* One tensor of qb_quantize_act_batch: the arguments of qb_quantize_act. */
typedef struct {
  const float* x;
  int64_t M, K;
  int8_t* xq;
  float* act_scale;
  int32_t* rowsum;
} qb_act_desc;

/* One matrix of qb_quantize_pack_weights_batch: the arguments of qb_quantize_pack_weights. */
typedef struct {
  const float* w;
  int64_t N, K;
  int32_t bits, groups;
  const float* range_lo; /* may be NULL (then range_hi too) */
  const float* range_hi;
  uint32_t* packed;
  float* delta;
  float* q0;
} qb_weight_desc;

/*
 * The two quantizers over a whole stack of linears (the inputs and weight matrices of the encoder
 * layers, Section 3.3 / Table 1 caption) in one pair of launches per call instead of one pair per
 * tensor: BERT's matrices are a few MB each, so single launches are bound by launch latency, not by
 * memory bandwidth.  `descs` is a HOST array; every element is validated before anything is launched;
 * each result equals the single call on the same arguments bit for bit.  Each activation tensor keeps
 * its own scale (per-tensor quantization).  Weight matrices of different bit widths may be mixed:
 * all matrices that take the single-kernel path of qb_quantize_pack_weights go into one launch per 96
 * matrices, whatever their widths (a mixed-precision stack is one launch), separately for groups that
 * fit one thread block, for each cluster size, and for caller-supplied ranges.  The others get a pair
 * of launches per bit width and 32 matrices.  Everything is enqueued on `cuda_stream`; the call
 * creates no host or device object.
 * Workspace: qb_workspace_bytes(0, 0, 0, 0, G) bytes with G = max(32, sum of `groups` over the batch).
 */
qb_status qb_quantize_act_batch(const qb_act_desc* descs /*host*/, int32_t count, void* ws, size_t ws_bytes,
                                void* cuda_stream);
qb_status qb_quantize_pack_weights_batch(const qb_weight_desc* descs /*host*/, int32_t count, void* ws,
                                         size_t ws_bytes, void* cuda_stream);

/*
 * The same quantizer and packer for callers that have no workspace to give.  (The paper has no
 * counterpart; this entry point exists for the library's users.)
 *
 * Some callers cannot allocate device memory at the point where they need this call: a plug-in that
 * receives tensors but no allocator, code running while its memory pool is frozen, a serving loop in
 * which cudaMalloc is banned because it stalls the whole device.  For them the per-group min/max
 * scratch that normally sits in the caller's workspace is a fixed array inside the library, held on
 * every GPU that loads it until the process ends (256 + 8 * QB_NOALLOC_MAX_GROUPS bytes).  The call
 * itself allocates and frees nothing.
 *
 *  - Arguments and results are those of qb_quantize_pack_weights, minus the workspace.  `groups` may
 *    not exceed QB_NOALLOC_MAX_GROUPS; a larger value returns QB_ERR_WORKSPACE and launches nothing.
 *  - status_out: dev int32 [1] or NULL.  When given, it receives this call's device status word
 *    (QB_OK, or QB_ERR_NONFINITE for a NaN or Inf weight or an unordered or non-finite supplied range)
 *    by a 4-byte device-to-device copy enqueued after the kernels.
 *  - The first call on each device looks up the array's device address.  Make that first call
 *    outside any stream capture.
 *  - Every call uses the same array and finds the previous call's contents in it; the call clears
 *    what it needs to be zero.  Calls that may run on the GPU at the same time (two streams, two
 *    host threads) race on the array: order them on one stream or with events.
 */
#define QB_NOALLOC_MAX_GROUPS 4096
qb_status qb_quantize_pack_weights_noalloc(const float* w, int64_t N, int64_t K, int bits, int groups,
                                           const float* range_lo, const float* range_hi, uint32_t* packed,
                                           float* delta, float* q0, int32_t* status_out, void* cuda_stream);

/*
 * Quantized linear layer (Appendix A: "integer arithmetic for the matrix multiplication with X^I,
 * and then followed by a gathered dequantization operation").
 *     acc[m][n] = sum_k xq[m][k] * code[n][k]                       (int32, exact)
 *     y[m][n]   = act_scale * (Delta_g * acc + q0_g * rowsum[m]) + bias[n],   g = n / R
 * The dequantization is evaluated in fp32 about the centre code c = 2^(k-1):
 *     Ac = acc - c * rowsum[m];  zc = fma(Delta_g, c, q0_g);  alpha = act_scale * Delta_g;
 *     beta = act_scale * zc;     y = fma(alpha, (float)Ac, fma(beta, (float)rowsum[m], bias[n])).
 * Packed codes are expanded to 8 bits in shared memory (Section 4: low-bit values are loaded and
 * cast to 8 bits in the execution units) and multiplied on the tensor cores.
 *   xq, act_scale, rowsum: dev, as written by qb_quantize_act         (read)
 *   packed, delta, q0:     dev, as written by qb_quantize_pack_weights (read)
 *   bias     dev fp32 [N] or NULL                                     (read)
 *   y        dev fp32 [M][N]                                          (written)
 *   acc_out  dev int32 [M][N] or NULL: the accumulators acc[m][n]     (written)
 * xq and packed must be 16-byte aligned.
 */
qb_status qb_gemm(const int8_t* xq, const float* act_scale, const int32_t* rowsum,
                  const uint32_t* packed, const float* delta, const float* q0, const float* bias,
                  int64_t M, int64_t N, int64_t K, int bits, int groups, float* y, int32_t* acc_out,
                  void* ws, size_t ws_bytes, void* cuda_stream);

/* One linear of a stack: the arguments of qb_gemm. */
typedef struct {
  const int8_t* xq;
  const float* act_scale;
  const int32_t* rowsum;
  const uint32_t* packed;
  const float* delta;
  const float* q0;
  const float* bias; /* may be NULL */
  int64_t M, N, K;
  int32_t bits, groups;
  float* y;
} qb_linear_desc;

/*
 * Encoder-layer linear stack with per-layer bit widths (the appendix tables "Bits setting for
 * 2/3-bit / 2/4-bit Q-BERT MP" give one weight bit width per encoder layer; the Hessian-based
 * assignment that produces them is an input here).  `descs` is a HOST array of `count`
 * descriptors, e.g. four per encoder layer in the order QKV, attention output, FFN1, FFN2; each is
 * an independent problem with its own input, and the result of each equals qb_gemm on the same
 * arguments bit for bit.  All descriptors are validated before anything is launched.
 * Up to 48 descriptors share one launch.  A large stack is cut into launches by bit width; a stack
 * that mixes bit widths and is small (fewer than 16 tiles of 128 x 128 per SM in all: a mixed-precision
 * stack at a few hundred tokens) goes out as launches that mix bit widths, so that the whole stack pays
 * one start-up and one drain.  All launches are enqueued on `cuda_stream`, in order; the call uses no
 * other stream, creates no host or device object, and may be captured into a CUDA graph.
 */
qb_status qb_layer_linears(const qb_linear_desc* descs /*host*/, int32_t count, void* ws,
                           size_t ws_bytes, void* cuda_stream);

/*
 * How many kernel launches qb_quantize_act_batch issues for `count` tensors (two per 64 tensors); host
 * arithmetic, no GPU work.  (No counterpart in the paper; for callers that count or budget launches.)
 */
int32_t qb_quantize_act_launch_count(int32_t count);

/*
 * How many kernel launches qb_quantize_pack_weights_batch issues for these matrices: host arithmetic on
 * the descriptors only (shapes, groups, bit widths, whether ranges are supplied), no GPU work.  (No
 * counterpart in the paper; for callers that count or budget launches.)  Returns 0 for a null or
 * empty batch or a descriptor with impossible shapes.
 */
int32_t qb_quantize_pack_weights_launch_count(const qb_weight_desc* descs /*host*/, int32_t count);

/*
 * How many GEMM kernel launches qb_layer_linears (and its narrow-output forms) issue for this stack: host
 * arithmetic on the descriptors only (bit widths, shapes), no GPU work.  (No counterpart in the paper; it
 * lets a caller that counts or budgets launches, e.g. a benchmark, ask the library instead of guessing.)
 *   descs   host array of `count` descriptors; only M, N, K and bits are read
 * Returns 0 for a null or empty stack.
 */
int32_t qb_layer_linears_launch_count(const qb_linear_desc* descs /*host*/, int32_t count);

/*
 * Narrow-output forms of qb_gemm and qb_layer_linears.  The paper keeps the activations between
 * layers at 8 bits (Table 1 caption: every quantized model uses 8-bit activations), so the fp32
 * result of a linear is an intermediate that the next operation narrows again; writing it as
 * bfloat16 halves the bytes of the write that bounds the K <= 1024 linears.
 *     y[m][n] = bf16( the fp32 value qb_gemm writes for the same arguments )
 * with round to nearest, ties to even, on the finished fp32 value (one extra rounding, after the
 * epilogue of Appendix A has been evaluated exactly as in qb_gemm).
 *   y   dev bfloat16 [M][N], as 16-bit patterns                     (written)
 * Everything else as for qb_gemm; there is no accumulator export.  In qb_layer_linears_bf16 the
 * `y` field of every descriptor points to such a bfloat16 array (cast to float*); each result equals
 * qb_gemm_bf16 on the same arguments bit for bit.
 */
qb_status qb_gemm_bf16(const int8_t* xq, const float* act_scale, const int32_t* rowsum,
                       const uint32_t* packed, const float* delta, const float* q0, const float* bias,
                       int64_t M, int64_t N, int64_t K, int bits, int groups, uint16_t* y, void* ws,
                       size_t ws_bytes, void* cuda_stream);
qb_status qb_layer_linears_bf16(const qb_linear_desc* descs /*host*/, int32_t count, void* ws,
                                size_t ws_bytes, void* cuda_stream);

/*
 * Re-quantized output: the result of a linear written directly in the 8-bit activation format that the
 * next linear reads (Table 1 caption: 8-bit activations throughout), so that no fp32 tensor and no
 * separate activation-quantizer pass lie between two linears.  The output grid has a step the caller
 * supplies (a static, calibrated scale; the dynamic per-tensor maximum of qb_quantize_act cannot be
 * known before the product is finished):
 *     yq[m][n] = clamp(round_half_even(y[m][n] * (1 / *out_scale)), -127, 127),
 * y the fp32 value qb_gemm writes for the same arguments.  Values beyond 127 * out_scale saturate.
 *   out_scale dev fp32 [1], finite and > 0; it is the act_scale of the consuming linear   (read)
 *   yq        dev int8 [M][N]                                                              (written)
 * qb_rowsum_i8 gives the row sums the consuming linear also needs: rowsum[m] = sum_k xq[m][k]
 * (xq dev int8 [M][K], 16-byte aligned, K a multiple of 128; rowsum dev int32 [M]).
 */
qb_status qb_gemm_i8(const int8_t* xq, const float* act_scale, const int32_t* rowsum,
                     const uint32_t* packed, const float* delta, const float* q0, const float* bias,
                     int64_t M, int64_t N, int64_t K, int bits, int groups, const float* out_scale,
                     int8_t* yq, void* ws, size_t ws_bytes, void* cuda_stream);
qb_status qb_rowsum_i8(const int8_t* xq, int64_t M, int64_t K, int32_t* rowsum, void* cuda_stream);
/* Stack form of qb_gemm_i8: `y` of descriptor i points to int8 [M][N] (cast to float*) and
 * out_scales[i] (HOST array of `count` dev pointers) is its output scale; grouping and side-by-side
 * launches as in qb_layer_linears; each result equals qb_gemm_i8 on the same arguments bit for bit. */
qb_status qb_layer_linears_i8(const qb_linear_desc* descs /*host*/, const float* const* out_scales /*host*/,
                              int32_t count, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Quantization-aware fine-tuning (Section 3.1: gradients pass through Q by the straight-through
 * estimator; Appendix A: forward and backward of the quantization process).
 *
 * Forward ("fake quantization"): the quantizer of qb_quantize_pack_weights, but the result is the
 * dequantized tensor Q(W) = Delta_g * code + q0_g in fp32 (one fused multiply-add per element, on the
 * codes and the Delta, q0 that qb_quantize_pack_weights computes for the same arguments).
 *   w        dev fp32 [N][K], 16-byte aligned                     (read)
 *   wq       dev fp32 [N][K], 16-byte aligned                     (written)
 *   delta,q0 dev fp32 [G]                                         (written)
 *   range_lo, range_hi: dev fp32 [G] or both NULL, as for qb_quantize_pack_weights.
 * One kernel (W read once) in the cases where qb_quantize_pack_weights takes one; otherwise two:
 * per-group min/max reduction into the workspace, then round/clamp/dequantize.
 *
 * Backward: grad_w = grad_wq where Clamp passes the weight through (range_lo[g] <= w <= range_hi[g],
 * both ends included), 0 where Clamp holds it at an end of the range; the rounding is treated as the
 * identity.  With range_lo = range_hi = NULL (the group's own [min, max]) every weight is inside
 * and the call copies grad_wq to grad_w (nothing is done if they are the same buffer).
 *   grad_wq  dev fp32 [N][K], gradient with respect to Q(W)       (read)
 *   w        dev fp32 [N][K], the weights that were quantized     (read)
 *   grad_w   dev fp32 [N][K]                                      (written; may alias grad_wq)
 * All three 16-byte aligned.  No workspace, no device-side status.
 */
qb_status qb_fake_quantize_weights(const float* w, int64_t N, int64_t K, int bits, int groups,
                                   const float* range_lo, const float* range_hi, float* wq, float* delta,
                                   float* q0, void* ws, size_t ws_bytes, void* cuda_stream);
qb_status qb_ste_backward(const float* grad_wq, const float* w, int64_t N, int64_t K, int groups,
                          const float* range_lo, const float* range_hi, float* grad_w, void* cuda_stream);

/*
 * qb_fake_quantize_weights over a stack of matrices (the weights of all encoder layers, once per
 * fine-tuning step) in as few launches as qb_quantize_pack_weights_batch takes: `descs` is a HOST array of
 * qb_weight_desc whose `packed` field points to the fp32 output Q(W) [N][K] (cast to uint32_t*), bit
 * widths may differ from matrix to matrix; every element is validated before anything is launched; each
 * result equals the single call on the same arguments bit for bit.
 * Workspace: qb_workspace_bytes(0, 0, 0, 0, G) bytes with G = max(32, sum of `groups` over the batch).
 */
qb_status qb_fake_quantize_weights_batch(const qb_weight_desc* descs /*host*/, int32_t count, void* ws,
                                         size_t ws_bytes, void* cuda_stream);

/*
 * Group-wise quantized embedding tables (Section 5.1: embedding quantized separately from the
 * encoder, word and position embedding at their own precisions; appendix on mixed-precision
 * embedding: the embedding dimensions are bucketed into 128 groups, 4-bit word and 8-bit position
 * embedding).  The table is kept in lookup order, E[v][d] with one row per vocabulary entry or
 * position, so a group is a block of D / G consecutive COLUMNS over all V rows; per group the
 * quantizer is the one of qb_quantize_pack_weights (exact [min, max] of the group, Appendix A).
 * Row v of `packed` is the dense little-endian bit stream of its D codes, D*k/32 words.
 *   table    dev fp32 [V][D], 16-byte aligned                     (read)
 *   packed   dev uint32 [V][D*bits/32], 16-byte aligned           (written)
 *   delta,q0 dev fp32 [G]                                         (written)
 * D must be a multiple of 128, at most 4096, and divisible by G.  The workspace must hold
 * qb_workspace_bytes(0, 0, 0, 0, D) bytes (8 per column).  Two kernels: per-column min/max into the
 * workspace, then round/clamp/pack.
 *
 * qb_embedding_lookup gathers and dequantizes: out[t][d] = Delta_g * code[ids[t]][d] + q0_g (one fused
 * multiply-add), g = d / (D / G); with accumulate != 0 that value is added to what `out` holds (one
 * fp32 addition), which sums the word and the position embedding of a token in two calls.
 *   ids      dev int32 [T], each in [0, V)                        (read)
 *   out      dev fp32 [T][D], 16-byte aligned                     (written, or read and written)
 * An id outside [0, V) writes zeros for that token and records QB_ERR_INVALID in the status word of `ws`.
 */
qb_status qb_quantize_embedding(const float* table, int64_t V, int64_t D, int bits, int groups,
                                uint32_t* packed, float* delta, float* q0, void* ws, size_t ws_bytes,
                                void* cuda_stream);
qb_status qb_embedding_lookup(const int32_t* ids, int64_t T, const uint32_t* packed, const float* delta,
                              const float* q0, int64_t V, int64_t D, int bits, int groups, int accumulate,
                              float* out, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Mixed-precision assignment from Hessian spectra (Section 3.2, Eq. 2 and the paragraph after it).
 * Host-only: no GPU work, no stream, all pointers are HOST pointers.
 *
 *   Omega_i = | mean(lambda_i) | + std(lambda_i)
 *
 * where lambda_i are the top eigenvalues of the Hessian of encoder layer i measured on `samples`
 * portions of the training data (the caller computes them; the power iteration is not part of this
 * library).  The layers are sorted by Omega in descending order (equal Omega: lower layer first) and
 * the layer of rank r receives budget_bits[r].  The paper fixes the ordering but no rule from rank to
 * bit width, so the budget is the caller's (e.g. six 3s then six 2s for the 2/3-bit mixed setting of
 * a 12-layer encoder).  std is the standard deviation of the empirical distribution of the samples
 * (divisor `samples`).  All arithmetic in fp64, sums in index order.
 *   lambda       host fp64 [layers][samples]                         (read)
 *   budget_bits  host int32 [layers], each in {2,3,4,8}; entry r is the width for rank r (read)
 *   reverse      0: as above; != 0: rank r receives budget_bits[layers-1-r] (the appendix's
 *                "MP-rev" ablation: fewest bits to the most sensitive layer)
 *   omega_out    host fp64 [layers] or NULL                          (written)
 *   order_out    host int32 [layers] or NULL: order_out[r] = layer of rank r   (written)
 *   bits_out     host int32 [layers]: bit width per layer, ready for qb_linear_desc.bits (written)
 * Returns QB_ERR_INVALID for null pointers, sizes < 1 or a budget entry outside {2,3,4,8};
 * QB_ERR_NONFINITE if a sample is NaN or Inf (nothing is written then).
 */
qb_status qb_sensitivity_bits(const double* lambda, int32_t layers, int32_t samples, const int32_t* budget_bits,
                              int32_t reverse, double* omega_out, int32_t* order_out, int32_t* bits_out);

/*
 * Diagnostic: the rate the tensor cores sustain for the GEMM's own instruction (tcgen05.mma kind::i8,
 * s8 x s8 -> s32, 128 x `tokens` x 32) with both operands resident in shared memory, no global
 * traffic, four K blocks in flight, one CTA per SM on the default stream.  (No counterpart in the
 * paper; it gives the denominator for the tensor-bound shapes of qb_gemm.)
 *   tokens    128 or 256 (the N of the instruction)
 *   k_blocks  K blocks of 128 per CTA (8 .. 2^22); the run lasts about k_blocks * 0.3 us
 *   tops_out  host, receives 1e-12 * 2*128*tokens*128*k_blocks*SMs / elapsed seconds
 *   cycles_per_kblock_out  host or NULL, SM cycles per K block (four instructions) on the slowest SM
 * Synchronizes the device.  Returns QB_ERR_TIMEOUT if a bounded wait expired.
 */
qb_status qb_probe_i8_mma(int32_t tokens, int32_t k_blocks, double* tops_out, double* cycles_per_kblock_out);

/*
 * Self-test of the bounded waits.  (No counterpart in the paper: every wait of the GEMM kernels on an
 * mbarrier is bounded so that a fault elsewhere cannot hang the GPU; this call shows the bound working.)
 * One small kernel waits, with the GEMM's own wait routines, on a barrier at which nothing ever arrives.
 * After `limit_cycles` SM cycles (1e3 .. 2e9; 2e6 is about a millisecond) the waits give up, the kernel
 * records QB_ERR_TIMEOUT in the status word of `ws` and returns normally; the context stays usable.
 *   ws                 dev, >= 256 bytes: its status word receives QB_ERR_TIMEOUT (sticky, as everywhere)
 *   waited_cycles_out  dev uint64 [2] or NULL: cycles each of the two waiting warps spent before giving up
 * Enqueued on `cuda_stream`; read the outcome with qb_read_status.
 */
qb_status qb_probe_wait_limit(void* ws, size_t ws_bytes, int64_t limit_cycles, uint64_t* waited_cycles_out,
                              void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* QBERT_H_ */
