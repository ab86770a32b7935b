// qb_gemm: integer matrix product on the quantization codes followed by one dequantization
// (Appendix A), for weights stored at k in {2,3,4,8} bits per code.
//
// Orientation.  The tensor-core product is computed transposed, D[n][m] = sum_k Wc[n][k] * xq[m][k]:
//   * the 128 rows of the MMA's A operand are 128 output neurons (weight rows), expanded from the
//     packed k-bit words to signed 8-bit values in shared memory (Section 4: low-bit values are
//     loaded and cast to 8 bits for execution);
//   * the MMA's B operand is a tile of BT tokens (128 or 256) of the int8 activations, staged by TMA;
//   * the int32 accumulator tile lives in tensor memory: TMEM lane = output neuron, column = token.
// With this orientation the per-neuron dequantization constants are per-thread registers in the
// epilogue and, for a fixed token, the 32 lanes of a warp hold 32 consecutive outputs of one row of
// Y, so every store instruction writes one full 128-byte line.
//
// Codes are fed to the MMA recentred and pre-scaled, v = (code - 2^(k-1)) << (8-k), as s8.  The
// shift makes the expansion a mask and an xor per word; the epilogue shifts the exact int32 sum
// back.  |sum| <= 127 * 128 * K < 2^31 for K <= 65536.
//
// One persistent CTA per SM, 28 warps, roles on warpgroup boundaries (registers are moved between the
// warpgroups with setmaxnreg):
//   warp 0        TMA producer for the token tiles               (one lane)
//   warp 1        tcgen05.mma issuer, owns the TMEM allocation   (one lane)
//   warps 2..3    idle (they complete the warpgroup that gives its registers away)
//   warps 4..19   weight expanders in four teams of four warps; team g fills the K blocks whose
//                 running index is g mod 4, thread r of a team owns weight row r of the tile
//   warps 20..27  epilogue: TMEM -> registers -> fp32 -> shared memory -> TMA store; two warps per
//                 TMEM lane quarter, each taking every other chunk of 32 tokens
// Large launches run as CTA pairs (clusters of two, tcgen05 cta_group::2): the tile is 256 neurons x 256
// tokens, each CTA expands its own 128 weight rows and stages its own 128 tokens, the pair's first CTA
// issues one MMA for both.  That halves the token bytes each SM pulls from L2 and writes to and reads from
// shared memory per MMA, and lets the ring be five K blocks deep instead of three.  No load is multicast.
// One launch serves up to kMaxProblems independent linears that share the token tile: their tiles form
// one list that the CTAs (or pairs) walk, so the start-up and the drain of the pipeline are paid once
// per launch, not once per linear.  The bit width is a template argument, or (BITS = 0, small stacks
// that mix widths) a field of every problem that the expanders and the epilogue read per tile.
// Shared-memory ring of kStages stages (16 KB expanded weights + the CTA's token rows x 128 B each,
// 128-byte swizzle, K block of 128), two accumulator tiles in TMEM so the epilogue of tile i overlaps
// the MMAs of tile i+1.  Every wait is bounded: on expiry the CTA records QB_ERR_TIMEOUT and leaves
// through the normal exit path (TMEM freed).
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <type_traits>
#include <vector>

#include "common.cuh"
#include "mbar_wait.cuh"
#include "ptx.cuh"

namespace qb {

// Roles sit on warpgroup boundaries (four consecutive warps) so that registers can be moved between them
// with setmaxnreg: warpgroup 0 holds the two single-thread roles (and two idle warps) and gives its
// registers away, warpgroups 1-4 are the expander teams, warpgroups 5-6 the epilogue.
// Four expander teams: at K = 4096 an expander iteration is about 1,500 busy cycles, so three teams only
// just keep up with the 512 cycles the tensor cores need per K block (config 3's K = 4096 GEMM: 95 -> 84 us
// with the fourth team).
constexpr int kExpandTeams = 4;     // teams of 128 expander threads
constexpr int kEpilogueWarps = 8;
constexpr int kFirstExpandWarp = 4;
constexpr int kFirstEpilogueWarp = kFirstExpandWarp + 4 * kExpandTeams;
constexpr int kEpilogueThread0 = 32 * kFirstEpilogueWarp;
constexpr int kGemmThreads = kEpilogueThread0 + 32 * kEpilogueWarps;
// Registers per thread: the launch gives every thread kRegsLaunch (65,536 / 896 rounded down to a multiple
// of 8); the shares below add up to at most kGemmThreads * kRegsLaunch, which setmaxnreg.inc needs in order
// not to wait forever.
constexpr int kRegsLaunch = 72;
constexpr int kRegsLight = 56;      // producer / issuer warpgroup
constexpr int kRegsExpand = 64;
constexpr int kRegsEpilogue = 96;
static_assert(128 * kRegsLight + 128 * kExpandTeams * kRegsExpand + 32 * kEpilogueWarps * kRegsEpilogue <=
                  kGemmThreads * kRegsLaunch,
              "register shares exceed what the launch allocates");
static_assert(kGemmThreads * kRegsLaunch <= 65536, "launch allocation exceeds the register file");
constexpr int kTileN = 128;          // output neurons per tile (MMA M)
constexpr int kBlockK = 128;         // K elements (= bytes) per pipeline stage
constexpr int kWBytes = kTileN * kBlockK;

constexpr int kMaxProblems = 48;
constexpr int kMaxOrder = 4096;   // entries of the explicit tile visiting order (when it is used)
constexpr uint16_t kNoTile = 0xFFFF;  // linears per launch (all in kernel-parameter space, no device table)

// One linear of a launch.
struct Problem {
  const float* act_scale;
  const int32_t* rowsum;
  const uint32_t* packed;
  const float* delta;
  const float* q0;
  const float* bias;
  void* y;           // fp32 [M][N], or bfloat16 / int8 [M][N] in the narrow-output kernels
  const float* out_scale;  // int8 output only: dev [1], step of the output grid
  int32_t* acc_out;
  int32_t M, N, K;
  int32_t rows_per_group;
  int32_t n_tiles, m_tiles;
  int32_t tile_begin;  // index of this problem's first tile in the launch's tile list
  int32_t tma_store;   // 1: Y rows are 16-byte aligned, the epilogue stores through TMA
  int32_t bits;        // bit width of this problem's codes (read by the kernels that mix bit widths)
};

struct GroupedParams {
  CUtensorMap tmx[kMaxProblems];  // int8 activations, box 128 B x BT tokens, 128-byte swizzle
  CUtensorMap tmy[kMaxProblems];  // outputs (fp32 or bfloat16), box 32 neurons x 32 tokens
  Problem prob[kMaxProblems];
  void* ws;
  int32_t count;
  int32_t total_tiles;
  // Visiting order.  Position p is visited by CTA p % gridDim.x.  Without `use_order` position p is tile
  // p; with it, order[p] is the tile (or kNoTile): the host balances tiles of unequal length (K) over
  // the CTAs instead of dealing them round-robin.
  int32_t total_positions;
  int32_t use_order;
  uint16_t order[kMaxOrder];
  uint8_t order_prob[kMaxOrder];  // with `order`: the problem that owns order[p] (spares every role the search)
};

// BT: tokens per tile (the N of the MMA).  CG: CTAs that share one MMA (1, or 2 = a CTA pair of a cluster:
// the tile is then 256 neurons x BT tokens, each CTA expands its own 128 weight rows, loads its own half
// of the token tile and drains its own half of the accumulator).
template <int BT, int CG>
struct GemmCfg {
  static constexpr int kXRows = BT / CG;             // token rows this CTA stages per K block
  static constexpr int kXBytes = kXRows * kBlockK;
  static constexpr int kStageBytes = kWBytes + kXBytes;
  static constexpr int kStages = (kStageBytes == 48 * 1024) ? 3 : 5;
  static constexpr int kTmemCols = 2 * BT;
  static constexpr int kBarBytes = 256 + 2 * 256 * 4;  // barriers + two row-sum tiles
  static constexpr int kOutStageBytes = kEpilogueWarps * 2 * 32 * 32 * 4;  // per epilogue warp: two buffers of 32 tokens x 32 neurons fp32
  static constexpr int kSmemBytes = kStages * kStageBytes + kOutStageBytes + kBarBytes;
};

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, groups of
// 8 rows 1024 bytes apart.  Fields: start address >> 4 (bits 0-13), leading byte offset >> 4 (16-29,
// unused for swizzled K-major, set to 1), stride byte offset >> 4 (32-45), descriptor version 1
// (bits 46-47), layout type 2 = SWIZZLE_128B (bits 61-63).
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor for kind::i8: D = s32 (bits 4-5 = 2), A = s8 (bits 7-9 = 1), B = s8
// (bits 10-12 = 1), both operands K-major (bits 15, 16 = 0), N >> 3 in bits 17-22, M >> 4 in 24-28.
__host__ __device__ constexpr uint32_t make_idesc_i8(int mma_m, int mma_n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(mma_n >> 3) << 17) | ((uint32_t)(mma_m >> 4) << 24);
}

// Expand one item of 32 consecutive codes (BITS packed 32-bit words) to 32 signed bytes
// v = (code - 2^(BITS-1)) << (8-BITS), returned as 8 words (word j = codes 4j..4j+3).
template <int BITS>
__device__ __forceinline__ void expand_item(const uint32_t* in, uint32_t (&out)[8]) {
  if constexpr (BITS == 8) {
#pragma unroll
    for (int i = 0; i < 8; ++i) out[i] = in[i] ^ 0x80808080u;
  } else if constexpr (BITS == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t w = in[i];
      const uint32_t even = ((w << 4) & 0xF0F0F0F0u) ^ 0x80808080u;  // codes 0,2,4,6 of this word
      const uint32_t odd = (w & 0xF0F0F0F0u) ^ 0x80808080u;          // codes 1,3,5,7
      out[2 * i] = __byte_perm(even, odd, 0x5140);                    // codes 0,1,2,3
      out[2 * i + 1] = __byte_perm(even, odd, 0x7362);                // codes 4,5,6,7
    }
  } else if constexpr (BITS == 2) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const uint32_t w = in[i];
      const uint32_t t0 = ((w << 6) & 0xC0C0C0C0u) ^ 0x80808080u;  // codes 0,4,8,12
      const uint32_t t1 = ((w << 4) & 0xC0C0C0C0u) ^ 0x80808080u;  // codes 1,5,9,13
      const uint32_t t2 = ((w << 2) & 0xC0C0C0C0u) ^ 0x80808080u;  // codes 2,6,10,14
      const uint32_t t3 = (w & 0xC0C0C0C0u) ^ 0x80808080u;         // codes 3,7,11,15
      const uint32_t a_lo = __byte_perm(t0, t1, 0x5140);           // codes 0,1,4,5
      const uint32_t b_lo = __byte_perm(t2, t3, 0x5140);           // codes 2,3,6,7
      const uint32_t a_hi = __byte_perm(t0, t1, 0x7362);           // codes 8,9,12,13
      const uint32_t b_hi = __byte_perm(t2, t3, 0x7362);           // codes 10,11,14,15
      out[4 * i] = __byte_perm(a_lo, b_lo, 0x5410);                // codes 0..3
      out[4 * i + 1] = __byte_perm(a_lo, b_lo, 0x7632);            // codes 4..7
      out[4 * i + 2] = __byte_perm(a_hi, b_hi, 0x5410);            // codes 8..11
      out[4 * i + 3] = __byte_perm(a_hi, b_hi, 0x7632);            // codes 12..15
    }
  } else {  // BITS == 3: 32 codes = 96 bits = 3 words; 4 codes = 12 bits per output word
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int bit = 12 * j;
      const int wi = bit >> 5, sh = bit & 31;
      uint32_t f;
      if (sh + 12 > 32)
        f = __funnelshift_r(in[wi], in[wi + 1], sh);
      else
        f = in[wi] >> sh;
      out[j] = 0x80808080u ^ ((f << 5) & 0x000000E0u) ^ ((f << 10) & 0x0000E000u) ^ ((f << 15) & 0x00E00000u) ^
               ((f << 20) & 0xE0000000u);
    }
  }
}

// Load one item (32 codes = BITS words, 4*BITS bytes) with the widest aligned access.
template <int BITS>
__device__ __forceinline__ void load_item(const uint32_t* __restrict__ src, uint32_t* dst) {
  if constexpr (BITS == 8) {
    const uint4 a = __ldg(reinterpret_cast<const uint4*>(src));
    const uint4 b = __ldg(reinterpret_cast<const uint4*>(src) + 1);
    dst[0] = a.x; dst[1] = a.y; dst[2] = a.z; dst[3] = a.w;
    dst[4] = b.x; dst[5] = b.y; dst[6] = b.z; dst[7] = b.w;
  } else if constexpr (BITS == 4) {
    const uint4 a = __ldg(reinterpret_cast<const uint4*>(src));
    dst[0] = a.x; dst[1] = a.y; dst[2] = a.z; dst[3] = a.w;
  } else if constexpr (BITS == 2) {
    const uint2 a = __ldg(reinterpret_cast<const uint2*>(src));
    dst[0] = a.x; dst[1] = a.y;
  } else {
    dst[0] = __ldg(src); dst[1] = __ldg(src + 1); dst[2] = __ldg(src + 2);
  }
}

// A role's walk over the tiles of its CTA (or CTA pair): positions g, g + G, ... of the visiting order, g the
// index of the CTA group and G their number.
struct TileCursor {
  int p;   // position
  int t;   // tile at that position
  int pi;  // problem that owns tile t
  int stride;  // CTA groups in the launch
  // `cg`: CTAs per group (1 or 2); the CTAs of a group walk the same tiles
  __device__ __forceinline__ void start(int cg = 1) {
    stride = (int)gridDim.x / cg;
    p = (int)blockIdx.x / cg - stride;
    t = 0;
    pi = 0;
  }
  // move to the CTA's next tile; false when there is none
  __device__ __forceinline__ bool next(const GroupedParams& gp) {
    for (;;) {
      p += stride;
      if (p >= gp.total_positions) return false;
      if (!gp.use_order) {
        t = p;
        break;
      }
      const uint16_t e = gp.order[p];
      if (e != kNoTile) {
        t = (int)e;
        pi = (int)gp.order_prob[p];
        return true;
      }
    }
    // the problem that owns tile t: the last one whose first tile is <= t
    int lo = 0, hi = gp.count - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (t >= gp.prob[mid].tile_begin) lo = mid;
      else hi = mid - 1;
    }
    pi = lo;
    return true;
  }
};

// Barrier over the four warps of an expander team (named barriers 2..) that also ORs a predicate over them.
__device__ __forceinline__ bool team_sync_or(bool pred, int bar_id) {
  uint32_t res;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, %2, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(res)
      : "r"((uint32_t)pred), "r"(bar_id)
      : "memory");
  return res != 0;
}

// Barrier over the epilogue warps (named barrier 1) that also ORs a predicate over them.
__device__ __forceinline__ bool epilogue_sync_or(bool pred) {
  uint32_t res;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(res)
      : "r"((uint32_t)pred), "n"(32 * kEpilogueWarps)
      : "memory");
  return res != 0;
}

// OUT selects what the epilogue writes: the fp32 result; that result rounded to bfloat16 (round to nearest
// even), Y bfloat16 [M][N]; or that result re-quantized to the 8-bit activation grid of step *out_scale,
// clamp(round_half_even(y * (1 / out_scale)), -127, 127), Y int8 [M][N].
enum { kOutF32 = 0, kOutBf16 = 1, kOutI8 = 2 };
template <int BT, int BITS, int OUT, int CG>
__global__ void __launch_bounds__(kGemmThreads, 1)
qb_gemm_kernel(const __grid_constant__ GroupedParams gp) {
  using Cfg = GemmCfg<BT, CG>;
  constexpr int kStages = Cfg::kStages;
  // CG == 2: this CTA's rank in its pair (rank 0 issues the MMAs for both and owns the barriers the issuer
  // waits on); the pair's tile is 2 * kTileN neurons x BT tokens, rank r owns neurons 128 r .. 128 r + 127
  // and stages token rows (BT / 2) r .. of the tile
  const uint32_t cta_rank = CG == 2 ? ptx::cluster_ctarank() : 0u;
  constexpr int kGroupN = kTileN * CG;  // neurons per tile of the CTA group
  // 128-byte swizzle patterns repeat every 1024 bytes: stage bases must be 1024-byte aligned.  The
  // kernel has no static shared memory, so the dynamic segment starts at offset 0 of the CTA's window.
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t smem_base = ptx::smem_u32(smem);
  if ((smem_base & 1023u) != 0u) {  // never expected; leave without touching anything
    if (threadIdx.x == 0) report_status(gp.ws, QB_ERR_CUDA, (int)smem_base);
    return;
  }
  // after the ring: fp32 output staging for the TMA stores (1024-byte aligned), then barriers
  float* out_stage = reinterpret_cast<float*>(smem + kStages * Cfg::kStageBytes);
  const uint32_t bar_base = smem_base + kStages * Cfg::kStageBytes + Cfg::kOutStageBytes;
  uint8_t* bar_ptr = smem + kStages * Cfg::kStageBytes + Cfg::kOutStageBytes;
  // one "full" barrier per stage: the TMA producer's expect-tx arrival (+ the bytes) and one arrival per
  // warp of the expander team that filled the weights; the issuer then needs a single wait per K block
  auto full = [&](int s) { return bar_base + 8u * s; };
  auto empty = [&](int s) { return bar_base + 8u * (2 * kStages + s); };
  auto acc_full = [&](int a) { return bar_base + 8u * (3 * kStages + a); };
  auto acc_empty = [&](int a) { return bar_base + 8u * (3 * kStages + 2 + a); };
  const uint32_t drain_bar = bar_base + 8u * (3 * kStages + 4);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 8 * (3 * kStages + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* rs_tile = reinterpret_cast<float*>(bar_ptr + 256);  // [2][256] row sums of a tile's tokens, as fp32
  auto stage_w = [&](int s) { return smem_base + s * Cfg::kStageBytes; };
  auto stage_x = [&](int s) { return smem_base + s * Cfg::kStageBytes + kWBytes; };

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full(s), 1 + 4 * CG);  // the producer's expect-tx arrival + the expander warps of every CTA of the group
      ptx::mbar_init(empty(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(acc_full(a), 1);
      ptx::mbar_init(acc_empty(a), kEpilogueWarps * CG);  // one arrival per epilogue warp of the group
    }
    ptx::mbar_init(drain_bar, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc_cg<CG>(ptx::smem_u32(tmem_slot), Cfg::kTmemCols);
    ptx::tmem_relinquish_cg<CG>();
  }
  ptx::tcgen05_fence_before_sync();
  __syncthreads();
  // a pair: no arrival or copy may reach the other CTA's barriers before it has initialised them
  if constexpr (CG == 2) ptx::cluster_sync_all();
  ptx::tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // the barriers the MMA issuer waits on live in the group's first CTA
  auto full_lead = [&](int s) { return CG == 2 ? ptx::map_to_cta(full(s), 0) : full(s); };
  auto acc_empty_lead = [&](int a) { return CG == 2 ? ptx::map_to_cta(acc_empty(a), 0) : acc_empty(a); };

  bool timed_out = false;
  int where = 0;

  // Each warpgroup first sets its register share: the light warpgroup (and the expanders, a little) hand
  // registers to the epilogue warps.
  if (warp < kFirstExpandWarp) {
  ptx::setmaxnreg_dec<kRegsLight>();
  if (warp == 0) {
    // ---------------- TMA producer: token tiles -------------------------------------------------
    if (ptx::elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      // The token tiles are first touched in DRAM by several CTAs at about the same time, and the
      // ring holds only a few K blocks: L2 prefetches run kL2Ahead blocks ahead of the loads (into the
      // CTA's next tile when the current one ends) so that the loads themselves hit L2.  Only for long K
      // (more than kL2MinBlocks K blocks per tile): there the loads of a tile are what the tensor cores
      // wait for (K = 4096 GEMM of config 3: 84 against 86 us); for short K the token tile was fetched
      // moments ago by the CTAs on the neighbouring neuron tiles, and the prefetch instructions only take
      // the TMA unit's time (16 linears of config 3: 1,241 -> 1,208 us without them).
      constexpr int kL2Ahead = 8;
      constexpr int kL2MinBlocks = 8;
      TileCursor c;
      c.start(CG);
      bool have = c.next(gp);
      constexpr int kMyRow0 = 0;
      const int row_off = (int)cta_rank * Cfg::kXRows + kMyRow0;  // this CTA's rows inside the token tile
      // Narrow token tiles are what launches with few tokens use: there every packed weight is read once,
      // straight from DRAM, and the expanders' register prefetch alone does not keep enough bytes in flight
      // (a K block of 2-bit weights is 4 KB).  The producer therefore asks L2 for a tile's whole block of
      // packed rows (contiguous in memory) one tile ahead of its use.
      auto prefetch_weights = [&](const TileCursor& tc) {
        if constexpr (BT == 128) {
          const Problem& pw = gp.prob[tc.pi];
          const int n0 = ((tc.t - pw.tile_begin) % pw.n_tiles) * kGroupN + (int)cta_rank * kTileN;
          const int rows = min(kTileN, pw.N - n0);
          const uint32_t row_bytes = (uint32_t)(pw.K / 8 * (BITS ? BITS : pw.bits));
          if (rows > 0) ptx::bulk_prefetch_l2(reinterpret_cast<const uint8_t*>(pw.packed) + (size_t)n0 * row_bytes, (uint32_t)rows * row_bytes);
        }
      };
      if (have) {
        const Problem& pr = gp.prob[c.pi];
        const int m0 = ((c.t - pr.tile_begin) / pr.n_tiles) * BT + row_off;
        prefetch_weights(c);
        if (pr.K / kBlockK > kL2MinBlocks)
          for (int kb = 0; kb < kL2Ahead && kb < pr.K / kBlockK; ++kb) ptx::tma_prefetch_l2_2d(&gp.tmx[c.pi], kb * kBlockK, m0);
      }
      while (have && !timed_out) {
        const Problem& pr = gp.prob[c.pi];
        const int m0 = ((c.t - pr.tile_begin) / pr.n_tiles) * BT + row_off;
        const int k_blocks = pr.K / kBlockK;
        const CUtensorMap* tm = &gp.tmx[c.pi];
        // the CTA's next tile, for prefetches that run past the end of this one
        TileCursor nx = c;
        const bool have_nx = nx.next(gp);
        const CUtensorMap* tm_nx = nullptr;
        int m0_nx = 0, kblocks_nx = 0;
        if (have_nx) {
          const Problem& pn = gp.prob[nx.pi];
          prefetch_weights(nx);
          tm_nx = &gp.tmx[nx.pi];
          m0_nx = ((nx.t - pn.tile_begin) / pn.n_tiles) * BT + row_off;
          kblocks_nx = pn.K / kBlockK;
        }
        for (int kb = 0; kb < k_blocks; ++kb) {
          const int ahead = kb + kL2Ahead;
          if (ahead < k_blocks) {
            if (k_blocks > kL2MinBlocks) ptx::tma_prefetch_l2_2d(tm, ahead * kBlockK, m0);
          } else if (tm_nx != nullptr && kblocks_nx > kL2MinBlocks && ahead - k_blocks < kblocks_nx &&
                     ahead - k_blocks < kL2Ahead) {
            ptx::tma_prefetch_l2_2d(tm_nx, (ahead - k_blocks) * kBlockK, m0_nx);
          }
          if (!wait_barrier_relaxed(empty(stage), phase ^ 1u, abort_flag)) {
            timed_out = true;
            where = (0 << 16) | stage;
            break;
          }
          if constexpr (CG == 2) {
            // the first CTA announces the bytes of both halves; each CTA's copy completes on that barrier
            if (cta_rank == 0) ptx::mbar_arrive_expect_tx(full(stage), CG * Cfg::kXBytes);
            ptx::tma_load_2d_pair(stage_x(stage), tm, full_lead(stage), kb * kBlockK, m0);
          } else {
            ptx::mbar_arrive_expect_tx(full(stage), Cfg::kXBytes);
            ptx::tma_load_2d(stage_x(stage), tm, full(stage), kb * kBlockK, m0);
          }
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        c = nx;
        have = have_nx;
      }
      if (timed_out) {
        // let copies already in flight land before the CTA's shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 400000ll) {
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (of a pair: in its first CTA only) -------------------------------
    if (cta_rank == 0 && ptx::elect_one()) {
      // This one thread must issue a K block's work in well under the 512 cycles the tensor cores need
      // for it, and every instruction here is long-latency and serial.  So: one barrier wait per K
      // block, and the loop is unrolled over the ring so that barrier addresses and both operand
      // descriptors of a stage are compile-time offsets from loop-invariant values.
      constexpr uint32_t idesc = make_idesc_i8(kGroupN, BT);
      const uint64_t a_desc0 = make_kmajor_sw128_desc(stage_w(0));
      const uint64_t b_desc0 = make_kmajor_sw128_desc(stage_x(0));
      constexpr uint32_t kStageDescStep = Cfg::kStageBytes >> 4;  // start-address field counts 16-byte units
      uint32_t phase = 0;
      int it = 0, kb = 0, k_blocks = 0, a = 0;
      uint32_t d_tmem = 0;
      TileCursor c;
      c.start(CG);
      bool active = c.next(gp);
      while (active) {
#pragma unroll
        for (int stage = 0; stage < kStages; ++stage) {
          if (active) {
            if (kb == 0) {  // first K block of a tile: its problem, and a free accumulator
              k_blocks = gp.prob[c.pi].K / kBlockK;
              a = it & 1;
              const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
              if (!wait_barrier(acc_empty(a), aphase ^ 1u, abort_flag)) {
                timed_out = true;
                where = (1 << 16) | 0x100 | a;
                active = false;
              }
              d_tmem = tmem_base + (uint32_t)(a * BT);
            }
            if (active && !wait_barrier(full(stage), phase, abort_flag)) {
              timed_out = true;
              where = (1 << 16) | stage;
              active = false;
            }
            if (active) {
              ptx::tcgen05_fence_after_sync();
              const uint64_t a_desc = a_desc0 + (uint64_t)(stage * kStageDescStep);
              const uint64_t b_desc = b_desc0 + (uint64_t)(stage * kStageDescStep);
#pragma unroll
              for (int j = 0; j < kBlockK / 32; ++j)  // 32 bytes of K per instruction: +2 in the address field
                ptx::mma_i8_ss_cg<CG>(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, j != 0 ? 1u : (kb != 0 ? 1u : 0u));
              ptx::mma_commit_cg<CG>(empty(stage));
              if (++kb == k_blocks) {  // tile done: hand the accumulator to the epilogue
                ptx::mma_commit_cg<CG>(acc_full(a));
                kb = 0;
                ++it;
                active = c.next(gp);
              }
            }
          }
        }
        phase ^= 1u;
      }
      if (timed_out) {
        // wait (bounded) for the MMAs already issued before tensor memory is freed
        ptx::mma_commit_cg<CG>(drain_bar);
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(drain_bar, 0) && clock64() - t0 < 400000000ll) {
        }
      }
    }
  }
  // (warps 2 and 3 of warpgroup 0 have nothing to do but to give their registers away)
  } else if (warp < kFirstEpilogueWarp) {
    ptx::setmaxnreg_dec<kRegsExpand>();
    // ---------------- weight expanders ------------------------------------------------------------
    // A K block of the tile is 128 rows x 4 items of 32 codes.  Thread i of a team takes items
    // i, i+128, i+256, i+384: piece i%4 of rows i/4 + 32j.  Four neighbouring lanes read one row's
    // 16*BITS contiguous bytes, so a warp-wide load touches 8 rows instead of 32.
    // The K blocks of all tiles of this CTA form one sequence; team g takes those with index g mod 4.
    const int team = (warp - kFirstExpandWarp) >> 2;
    const int i_team = (threadIdx.x - 32 * kFirstExpandWarp) & 127;
    const int piece = i_team & 3;
    const int row0 = i_team >> 2;
    // fetch cursor: tile, K block inside it, and the tile's weight rows
    TileCursor c;
    c.start(CG);
    int ld_kb = team;
    int ld_kblocks = 0, ld_n0 = 0, ld_N = 0, ld_wpr = 0, ld_bits = BITS;
    const uint32_t* ld_packed = nullptr;
    bool ld_done = !c.next(gp);
    auto enter_tile = [&]() {  // fields of the tile the cursor stands on
      const Problem& pr = gp.prob[c.pi];
      ld_kblocks = pr.K / kBlockK;
      ld_n0 = ((c.t - pr.tile_begin) % pr.n_tiles) * kGroupN + (int)cta_rank * kTileN;
      ld_N = pr.N;
      if constexpr (BITS == 0) ld_bits = pr.bits;  // a launch that mixes bit widths: the tile's own
      ld_wpr = pr.K / 32 * ld_bits;
      ld_packed = pr.packed;
    };
    auto normalize = [&]() {  // carry ld_kb over tile ends
      while (!ld_done && ld_kb >= ld_kblocks) {
        ld_kb -= ld_kblocks;
        if (!c.next(gp)) {
          ld_done = true;
        } else {
          enter_tile();
        }
      }
    };
    if (!ld_done) {
      enter_tile();
      normalize();
    }
    // Register prefetch of the packed words, one team-iteration (four K blocks) ahead.  kW: words per item of 32 codes
    // (the bit width; 8, the largest, when the launch mixes widths: every buffer then carries its own width).
    constexpr int kW = BITS ? BITS : 8;
    constexpr int kPrefetch = 1;
    uint32_t pre[kPrefetch][4 * kW];
    int pre_bits[kPrefetch];
    bool pre_valid[kPrefetch];
    auto load_rows = [&](auto width, uint32_t* nxt) {
      constexpr int B = decltype(width)::value;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int n = ld_n0 + row0 + 32 * j;
        if (n < ld_N) {
          load_item<B>(ld_packed + (size_t)n * ld_wpr + ld_kb * (4 * B) + piece * B, nxt + j * kW);
        } else {
          // rows past N: their accumulators are never stored, any operand value will do
#pragma unroll
          for (int w = 0; w < B; ++w) nxt[j * kW + w] = 0u;
        }
      }
    };
    auto load_next = [&](uint32_t* nxt, int& nxt_bits) -> bool {
      if (ld_done) return false;
      nxt_bits = ld_bits;
      if constexpr (BITS != 0) {
        load_rows(std::integral_constant<int, BITS ? BITS : 8>(), nxt);
      } else {
        switch (ld_bits) {  // the same for every thread of the CTA
          case 2: load_rows(std::integral_constant<int, 2>(), nxt); break;
          case 3: load_rows(std::integral_constant<int, 3>(), nxt); break;
          case 4: load_rows(std::integral_constant<int, 4>(), nxt); break;
          default: load_rows(std::integral_constant<int, 8>(), nxt); break;
        }
      }
      ld_kb += kExpandTeams;
      normalize();
      return true;
    };
    auto expand_rows = [&](auto width, const uint32_t* words, uint8_t* stage_ptr) {
      constexpr int B = decltype(width)::value;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int row = row0 + 32 * j;
        uint32_t out[8];
        expand_item<B>(words + j * kW, out);
        // the item is 16-byte chunks 2*piece and 2*piece+1 of the row; 128-byte swizzle: chunk ^ (row % 8)
        uint8_t* row_ptr = stage_ptr + row * 128;
        *reinterpret_cast<uint4*>(row_ptr + (((2 * piece) ^ (row & 7)) << 4)) = make_uint4(out[0], out[1], out[2], out[3]);
        *reinterpret_cast<uint4*>(row_ptr + (((2 * piece + 1) ^ (row & 7)) << 4)) = make_uint4(out[4], out[5], out[6], out[7]);
      }
    };
#pragma unroll
    for (int d = 0; d < kPrefetch; ++d) pre_valid[d] = load_next(pre[d], pre_bits[d]);
    int stage = team % kStages;
    uint32_t phase = (uint32_t)(team / kStages) & 1u;
    while (pre_valid[0]) {
      uint32_t cur[4 * kW];
      const int cur_bits = pre_bits[0];
#pragma unroll
      for (int i = 0; i < 4 * kW; ++i) cur[i] = pre[0][i];
#pragma unroll
      for (int d = 0; d + 1 < kPrefetch; ++d) {
        pre_valid[d] = pre_valid[d + 1];
        pre_bits[d] = pre_bits[d + 1];
#pragma unroll
        for (int i = 0; i < 4 * kW; ++i) pre[d][i] = pre[d + 1][i];
      }
      // the team's first warp polls the stage's barrier, the other three are parked at the team's named
      // barrier, which also makes the decision to give up the same in all four
      const bool got = (warp & 3) != 0 || wait_barrier_warp(empty(stage), phase ^ 1u, abort_flag);
      if (team_sync_or(!got, 2 + team)) {
        timed_out = true;
        where = (2 << 16) | stage;
        break;
      }
      uint8_t* stage_ptr = smem + stage * Cfg::kStageBytes;
      if constexpr (BITS != 0) {
        expand_rows(std::integral_constant<int, BITS ? BITS : 8>(), cur, stage_ptr);
      } else {
        switch (cur_bits) {
          case 2: expand_rows(std::integral_constant<int, 2>(), cur, stage_ptr); break;
          case 3: expand_rows(std::integral_constant<int, 3>(), cur, stage_ptr); break;
          case 4: expand_rows(std::integral_constant<int, 4>(), cur, stage_ptr); break;
          default: expand_rows(std::integral_constant<int, 8>(), cur, stage_ptr); break;
        }
      }
      ptx::fence_proxy_async_smem();  // every lane: its own stores -> visible to the tensor cores
      __syncwarp();
      if (lane == 0) {
        if (CG == 2 && cta_rank != 0) ptx::mbar_arrive_remote(full_lead(stage));
        else ptx::mbar_arrive(full(stage));
      }
      // the next fetch goes out after the proxy fence, not before it: the fence waits for the thread's loads
      // in flight, and a fetch issued first would put its whole latency into every K block
      pre_valid[kPrefetch - 1] = load_next(pre[kPrefetch - 1], pre_bits[kPrefetch - 1]);
      stage += kExpandTeams;
      while (stage >= kStages) {
        stage -= kStages;
        phase ^= 1u;
      }
    }
  } else {
    ptx::setmaxnreg_inc<kRegsEpilogue>();
    // ---------------- epilogue --------------------------------------------------------------------
    // Two warps per TMEM lane quarter; the warps of a quarter take alternate chunks of 32 tokens.  Per tile:
    // wait for the accumulator, then for every chunk: tcgen05.ld, convert and two fused multiply-adds per
    // output, 32 x 32 tile into shared memory, one TMA store.  The accumulator is handed back to the issuer as soon as the warp's last
    // chunk is in registers.  The next tile's dequantization constants and row sums are fetched while
    // this tile drains.
    const int ew = warp - kFirstEpilogueWarp;
    const int quarter = warp & 3;              // TMEM lanes this warp may access: 32*quarter ..
    const int half = ew >> 2;                  // which of the quarter's two warps
    const int r = quarter * 32 + lane;         // output neuron inside the CTA's 128 rows
    const int e = threadIdx.x - kEpilogueThread0;  // 0..255: the token whose row sum this thread stages
    float* const warp_bufs = out_stage + ew * (2 * 32 * 32);
    int out_flip = 0;

    // per-tile values: the tile being drained, and the CTA's next tile (prefetched)
    // `fetch` only issues the loads; the arithmetic on them (`finish`) comes when the tile's turn has come,
    // so that the warp does not wait for a tile's constants while it could drain the one before.
    struct TileVals {
      int pi, n_base, m0;
      int bits;                   // bit width of the tile's codes
      float s_a, dlt, z;          // as loaded: activation scale, the neuron's group step and offset
      int32_t rs_i;               // row sum of token m0 + e, 0 past M
      float alpha, beta, b, rs;   // after finish(); rs as fp32 (exact: |rowsum| < 2^24)
    };
    auto finish = [&](TileVals& tv) {
      const float zc = __fmaf_rn(tv.dlt, (float)(1 << (tv.bits - 1)), tv.z);
      tv.alpha = __fmul_rn(tv.s_a, tv.dlt);
      tv.beta = __fmul_rn(tv.s_a, zc);
      tv.rs = (float)tv.rs_i;
    };
    auto fetch = [&](const TileCursor& tc, TileVals& tv) {
      const Problem& pr = gp.prob[tc.pi];
      const int local = tc.t - pr.tile_begin;
      tv.pi = tc.pi;
      tv.bits = BITS ? BITS : pr.bits;
      tv.n_base = (local % pr.n_tiles) * kGroupN + (int)cta_rank * kTileN;
      tv.m0 = (local / pr.n_tiles) * BT;
      const int n = tv.n_base + r;
      tv.s_a = tv.dlt = tv.z = tv.b = 0.f;  // neurons past N: alpha = beta = b = 0, never stored
      if (n < pr.N) {
        tv.s_a = __ldg(pr.act_scale);
        const int g = n / pr.rows_per_group;
        tv.dlt = __ldg(pr.delta + g);
        tv.z = __ldg(pr.q0 + g);
        tv.b = pr.bias ? __ldg(pr.bias + n) : 0.0f;
      }
      tv.rs_i = (e < BT && tv.m0 + e < pr.M) ? __ldg(pr.rowsum + tv.m0 + e) : 0;
    };

    TileCursor c;
    c.start(CG);
    bool have = c.next(gp);
    TileVals cur;
    if (have) {
      fetch(c, cur);
      finish(cur);
      if (e < BT) rs_tile[e] = cur.rs;  // accumulator 0's row sums; published by the barrier below
    }
    for (int it = 0; have; ++it) {
      const Problem& pr = gp.prob[cur.pi];
      const CUtensorMap* tmy = &gp.tmy[cur.pi];
      const int pM = pr.M, pN = pr.N;
      const int a = it & 1;
      const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
      const int n_base = cur.n_base, m0 = cur.m0;
      const int n = n_base + r;
      const bool nvalid = n < pN;
      const bool tma_store = pr.tma_store != 0;
      const float alpha = cur.alpha, beta = cur.beta, b = cur.b;
      const int sh = 8 - cur.bits;           // the tensor cores were fed (code - c) << sh
      const int c_code = 1 << (cur.bits - 1);
      float* const y_ptr = reinterpret_cast<float*>(pr.y);
      uint16_t* const y16_ptr = reinterpret_cast<uint16_t*>(pr.y);
      int8_t* const y8_ptr = reinterpret_cast<int8_t*>(pr.y);
      float out_inv = 0.0f;
      if constexpr (OUT == kOutI8) out_inv = __fdiv_rn(1.0f, __ldg(pr.out_scale));
      int32_t* const acc_ptr = pr.acc_out;

      // one warp polls the accumulator's barrier; the others are parked at the named barrier below (a
      // polling warp spends issue slots, a parked one none)
      const bool ok = ew != 0 || wait_barrier_warp(acc_full(a), aphase, abort_flag);
      // One barrier over the epilogue warps per tile: it publishes the row sums staged for this tile and
      // makes the decision to give up the same in all eight warps (a warp that left alone would leave
      // the others waiting at this barrier).
      if (epilogue_sync_or(!ok)) {
        timed_out = true;
        where = (3 << 16) | a;
        break;
      }
      ptx::tcgen05_fence_after_sync();

      // the CTA's next tile: its constants are fetched now and used after this tile's chunks
      TileCursor nx = c;
      const bool have_nx = nx.next(gp);
      TileVals nxt;
      if (have_nx) fetch(nx, nxt);

      const uint32_t t_base = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * BT);
      const int n_chunks = min(BT / 32, (pM - m0 + 31) / 32);  // chunks of 32 tokens, warp-uniform
      const int x0 = n_base + quarter * 32;
      const float* const rs_a = rs_tile + a * 256;

      auto release_acc = [&]() {  // this warp has read all it needs from the accumulator
        ptx::tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          if (CG == 2 && cta_rank != 0) ptx::mbar_arrive_remote(acc_empty_lead(a));
          else ptx::mbar_arrive(acc_empty(a));
        }
      };
      auto process = [&](uint32_t (&v)[32], int ch) {
        const int mc = m0 + ch * 32;
        const float4* rs4 = reinterpret_cast<const float4*>(rs_a + ch * 32);
        float* buf = warp_bufs + (out_flip & 1) * (32 * 32);  // alternate between the warp's two staging buffers
        ++out_flip;
        if (tma_store) {
          // 32 tokens x 32 neurons of this warp -> shared memory [token][neuron] -> one TMA store.
          // Lanes write consecutive words of a row: conflict-free.  Rows past M and neurons past N
          // are clipped by the tensor map.  All 32 results are formed first (in the registers that held
          // the accumulators): y = fma(alpha, (float)Ac, fma(beta, rowsum, b)) with Ac = v >> sh.
          float yv[32];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float4 rv = rs4[q];  // same address in every lane: one broadcast read
            const float rsv[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int ac = ((int)v[4 * q + i]) >> sh;
              yv[4 * q + i] = __fmaf_rn(alpha, (float)ac, __fmaf_rn(beta, rsv[i], b));
            }
          }
          if (lane == 0) ptx::tma_store_wait_read1();  // the store before last (same buffer) has read it
          __syncwarp();
          if constexpr (OUT == kOutBf16) {  // rows of 32 bfloat16 (64 bytes): the first half of the fp32 buffer
            uint16_t* buf16 = reinterpret_cast<uint16_t*>(buf);
#pragma unroll
            for (int j = 0; j < 32; ++j) buf16[j * 32 + lane] = __bfloat16_as_ushort(__float2bfloat16_rn(yv[j]));
          } else if constexpr (OUT == kOutI8) {  // rows of 32 codes (32 bytes): the first quarter of the buffer
            int8_t* buf8 = reinterpret_cast<int8_t*>(buf);
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int q = __float2int_rn(__fmul_rn(yv[j], out_inv));
              buf8[j * 32 + lane] = (int8_t)min(max(q, -127), 127);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) buf[j * 32 + lane] = yv[j];
          }
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0 && x0 < pN) {
            ptx::tma_store_2d(tmy, ptx::smem_u32(buf), x0, mc);
            ptx::tma_store_commit();
          }
        }
        if (!tma_store || acc_ptr != nullptr) {
          float* yrow = y_ptr + (size_t)mc * pN + n;
          uint16_t* yrow16 = y16_ptr + (size_t)mc * pN + n;
          int8_t* yrow8 = y8_ptr + (size_t)mc * pN + n;
          int32_t* arow = acc_ptr ? acc_ptr + (size_t)mc * pN + n : nullptr;
          const int rows = min(32, pM - mc);  // warp-uniform
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float4 rv = rs4[q];
            const float rs[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int j = 4 * q + i;
              const int ac = ((int)v[j]) >> sh;
              if (nvalid && j < rows) {
                if (!tma_store) {
                  const float yv = __fmaf_rn(alpha, (float)ac, __fmaf_rn(beta, rs[i], b));
                  if constexpr (OUT == kOutBf16)
                    yrow16[(size_t)j * pN] = __bfloat16_as_ushort(__float2bfloat16_rn(yv));
                  else if constexpr (OUT == kOutI8)
                    yrow8[(size_t)j * pN] = (int8_t)min(max(__float2int_rn(__fmul_rn(yv, out_inv)), -127), 127);
                  else
                    yrow[(size_t)j * pN] = yv;
                }
                if (arow) arow[(size_t)j * pN] = ac + c_code * __float2int_rn(rs[i]);
              }
            }
          }
        }
      };

      // the warp's chunks: half, half + 2, ...
      if (half >= n_chunks) release_acc();
#pragma unroll 1
      for (int ch = half; ch < n_chunks; ch += kEpilogueWarps / 4) {
        uint32_t v[32];
        ptx::tmem_ld_32x32b_x32(t_base + (uint32_t)(ch * 32), v);
        ptx::tmem_ld_wait();
        ptx::tmem_ld_regs_ready(v);
        if (ch + kEpilogueWarps / 4 >= n_chunks) release_acc();  // the warp's last chunk is in registers
        process(v, ch);
      }
      // stage the next tile's row sums for the other accumulator (its previous readers all passed this
      // tile's barrier) and move on
      if (have_nx) {
        finish(nxt);
        if (e < BT) rs_tile[(a ^ 1) * 256 + e] = nxt.rs;
      }
      c = nx;
      cur = nxt;
      have = have_nx;
    }
  }

  if (warp >= kFirstEpilogueWarp && lane == 0) ptx::tma_store_wait_read0();  // staging buffers still in use
  if (timed_out) {
    *abort_flag = 1;
    report_status(gp.ws, QB_ERR_TIMEOUT, where);
  }
  // ---------------- teardown ----------------------------------------------------------------------
  ptx::tcgen05_fence_before_sync();
  __syncthreads();
  // a pair: the other CTA's MMAs write this CTA's tensor memory and its roles arrive on this CTA's barriers;
  // neither CTA may free anything or exit before both are done
  if constexpr (CG == 2) ptx::cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    ptx::tcgen05_fence_after_sync();
    ptx::tmem_dealloc_cg<CG>(tmem_base, Cfg::kTmemCols);
  }
}

// ---- host side -----------------------------------------------------------------------------------
// 1 (default): launches with enough 256 x 256 tiles run as CTA pairs; 0: single-CTA tiles everywhere.
// Read once from the environment (QBERT_PAIR=0 switches the pairs off, for comparisons).
static const int g_pair_mode = [] {
  const char* e = std::getenv("QBERT_PAIR");
  return (e && e[0] == '0') ? 0 : 1;
}();

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static qb_status get_encode_fn(EncodeTiledFn* out) {
  static EncodeTiledFn cached = nullptr;
  if (!cached) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    QB_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (qres != cudaDriverEntryPointSuccess || !fn) {
      set_last_error("cuTensorMapEncodeTiled not available from the driver");
      return QB_ERR_CUDA;
    }
    cached = reinterpret_cast<EncodeTiledFn>(fn);
  }
  *out = cached;
  return QB_OK;
}

// int8 activations [M][K], K contiguous; box = 128 bytes of K x `box_rows` tokens, 128-byte swizzle.
static qb_status make_x_tensormap(CUtensorMap* tm, const int8_t* xq, int64_t M, int64_t K, int box_rows) {
  EncodeTiledFn encode = nullptr;
  qb_status st = get_encode_fn(&encode);
  if (st != QB_OK) return st;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)K};
  const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows};
  const cuuint32_t elem[2] = {1, 1};
  CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(xq), dims, strides, box, elem,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_error("cuTensorMapEncodeTiled failed with CUresult %d (M=%lld K=%lld)", (int)r, (long long)M,
                   (long long)K);
    return QB_ERR_CUDA;
  }
  return QB_OK;
}

// Outputs [M][N] (fp32 or bfloat16), N contiguous; box = 32 neurons x 32 tokens, no swizzle (plain row-major
// in smem).
static qb_status make_y_tensormap(CUtensorMap* tm, void* y, int64_t M, int64_t N, int out) {
  const int esize = out == kOutF32 ? 4 : (out == kOutBf16 ? 2 : 1);
  const CUtensorMapDataType dtype = out == kOutF32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                   : (out == kOutBf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                                      : CU_TENSOR_MAP_DATA_TYPE_UINT8);
  EncodeTiledFn encode = nullptr;
  qb_status st = get_encode_fn(&encode);
  if (st != QB_OK) return st;
  const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)N * esize};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t elem[2] = {1, 1};
  CUresult r = encode(tm, dtype, 2, y, dims, strides,
                      box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
                      CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_error("cuTensorMapEncodeTiled (outputs) failed with CUresult %d (M=%lld N=%lld)", (int)r, (long long)M,
                   (long long)N);
    return QB_ERR_CUDA;
  }
  return QB_OK;
}

// `grid` CTAs; with CG == 2 they are launched as clusters of two (grid is even).
template <int BT, int BITS, int OUT, int CG>
static qb_status launch_group_inst(const GroupedParams& gp, int grid, cudaStream_t stream) {
  using Cfg = GemmCfg<BT, CG>;
  auto kernel = qb_gemm_kernel<BT, BITS, OUT, CG>;
  static std::atomic<bool> attr_set[64] = {};
  int dev = 0;
  QB_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
    QB_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
    if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(kGemmThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CG;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = CG == 2 ? 1 : 0;
  QB_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, gp));
  return QB_OK;
}

template <int BT, int OUT, int CG>
static qb_status launch_group_bits(int bits, const GroupedParams& gp, int grid, cudaStream_t stream) {
  switch (bits) {
    case 2: return launch_group_inst<BT, 2, OUT, CG>(gp, grid, stream);
    case 3: return launch_group_inst<BT, 3, OUT, CG>(gp, grid, stream);
    case 4: return launch_group_inst<BT, 4, OUT, CG>(gp, grid, stream);
    case 8: return launch_group_inst<BT, 8, OUT, CG>(gp, grid, stream);
    default: return QB_ERR_INVALID;
  }
}

// Token-tile width for a launch: 256 tokens unless every problem has at most 128 or the launch is too
// small to give every SM a 256-token tile.  The 128-wide instruction takes as long as the 256-wide one
// (measured with qb_probe_i8_mma: 498 vs 512 cycles per K block), so narrow tiles halve the tensor rate
// and double the weight expansion per token; they pay only when SMs would otherwise idle.
// `cg_out`: CTAs per tile.  A launch with at least one 256 x 256 tile per pair of SMs runs as CTA pairs: each
// CTA then stages half of the token tile (half the L2 and shared-memory traffic per MMA) and the ring is
// five K blocks deep instead of three.
static int choose_token_tile(const qb_linear_desc* d, const int* idx, int count, int sm_count, int* cg_out) {
  bool wide = false;
  int64_t tiles256 = 0, tiles_pair = 0;
  for (int i = 0; i < count; ++i) {
    if (d[idx[i]].M > 128) wide = true;
    tiles256 += ((d[idx[i]].N + kTileN - 1) / kTileN) * ((d[idx[i]].M + 255) / 256);
    tiles_pair += ((d[idx[i]].N + 2 * kTileN - 1) / (2 * kTileN)) * ((d[idx[i]].M + 255) / 256);
  }
  *cg_out = 1;
  if (wide && sm_count >= 2 && tiles_pair >= sm_count / 2 && g_pair_mode != 0) {
    *cg_out = 2;
    return 256;
  }
  // a launch that cannot give every SM a 256-token tile uses 128-token tiles: twice the CTAs at work,
  // half the epilogue per tile
  if (wide && tiles256 >= sm_count) return 256;
  return 128;
}

static qb_status validate_gemm(const int8_t* xq, const float* act_scale, const int32_t* rowsum,
                               const uint32_t* packed, const float* delta, const float* q0, int64_t M, int64_t N,
                               int64_t K, int bits, int groups, const void* y, const void* ws, size_t ws_bytes) {
  if (!xq || !act_scale || !rowsum || !packed || !delta || !q0 || !y || M <= 0 || N <= 0 || K <= 0 ||
      M > QB_MAX_MN || N > QB_MAX_MN || K > QB_MAX_K || !valid_bits(bits) || groups < 1 || N % groups != 0) {
    set_last_error("qb_gemm: invalid argument (M=%lld N=%lld K=%lld bits=%d groups=%d)", (long long)M,
                   (long long)N, (long long)K, bits, groups);
    return QB_ERR_INVALID;
  }
  if (K % 128 != 0 || !aligned16(xq) || !aligned16(packed)) {
    set_last_error("qb_gemm: K must be a multiple of 128 and xq, packed 16-byte aligned");
    return QB_ERR_ALIGN;
  }
  if (!ws || ws_bytes < kWsMinBytes) {
    set_last_error("qb_gemm: workspace null or too small");
    return QB_ERR_WORKSPACE;
  }
  return QB_OK;
}

// One launch over descriptors d[idx[0..count)] (count <= kMaxProblems), all with the same bit width, on at
// most `max_ctas` CTAs.
static qb_status launch_group(const qb_linear_desc* d, const int* idx, int count, int32_t* acc_out, void* ws,
                              int max_ctas, cudaStream_t stream, int out,
                              const float* const* out_scales = nullptr) {
  const int sm_count = max_ctas;
  int bits = d[idx[0]].bits;  // 0: the launch mixes bit widths (every problem carries its own)
  for (int i = 1; i < count; ++i)
    if (d[idx[i]].bits != bits) bits = 0;
  int cg = 1;
  int bt = choose_token_tile(d, idx, count, sm_count, &cg);
  if (bits == 0) {  // mixed widths: built for small stacks only (128-token tiles, single CTAs)
    cg = 1;
    bt = 128;
  }
  const int group_n = kTileN * cg;
  GroupedParams gp;
  memset(&gp, 0, sizeof(gp));
  gp.ws = ws;
  gp.count = count;
  int tile = 0;
  for (int i = 0; i < count; ++i) {
    const qb_linear_desc& q = d[idx[i]];
    qb_status st = make_x_tensormap(&gp.tmx[i], q.xq, q.M, q.K, bt / cg);
    if (st != QB_OK) return st;
    // Y rows 16-byte aligned: the epilogue stages tiles in shared memory and stores them with TMA
    const bool tma_store = (q.N % (out == kOutF32 ? 4 : (out == kOutBf16 ? 8 : 16)) == 0) && aligned16(q.y);
    if (tma_store) {
      st = make_y_tensormap(&gp.tmy[i], q.y, q.M, q.N, out);
      if (st != QB_OK) return st;
    } else {
      gp.tmy[i] = gp.tmx[i];  // unused by the kernel
    }
    Problem& p = gp.prob[i];
    p.act_scale = q.act_scale;
    p.rowsum = q.rowsum;
    p.packed = q.packed;
    p.delta = q.delta;
    p.q0 = q.q0;
    p.bias = q.bias;
    p.y = q.y;
    p.out_scale = out_scales ? out_scales[idx[i]] : nullptr;
    p.acc_out = acc_out;
    p.M = (int32_t)q.M;
    p.N = (int32_t)q.N;
    p.K = (int32_t)q.K;
    p.rows_per_group = (int32_t)(q.N / q.groups);
    p.n_tiles = (int32_t)((q.N + group_n - 1) / group_n);
    p.m_tiles = (int32_t)((q.M + bt - 1) / bt);
    p.tile_begin = tile;
    p.tma_store = tma_store ? 1 : 0;
    p.bits = q.bits;
    tile += p.n_tiles * p.m_tiles;
  }
  gp.total_tiles = tile;
  const int max_groups = sm_count / cg;
  const int grid = tile < max_groups ? tile : max_groups;  // CTA groups
  gp.total_positions = tile;
  gp.use_order = 0;
  // Tiles of different problems differ in length (K blocks).  When the launch is small enough for the
  // table, deal the tiles longest first to the least loaded CTA instead of round-robin.
  {
    bool uniform = bits != 0;
    for (int i = 1; i < count; ++i) uniform = uniform && gp.prob[i].K == gp.prob[0].K;
    if (!uniform && tile <= kMaxOrder && tile < (int)kNoTile) {
      constexpr int kEpilogueCost = 5;  // a tile's fixed cost in units of one K block
      std::vector<int> ids(tile), cost(tile);
      for (int i = 0, t = 0; i < count; ++i)
        for (int j = 0; j < gp.prob[i].n_tiles * gp.prob[i].m_tiles; ++j, ++t) {
          ids[t] = t;
          // measured at M = 128: a K block of 3-bit weights takes about 1.2 times, of 8-bit weights about 1.4
          // times as long as one of 2- or 4-bit weights
          cost[t] = (gp.prob[i].K / kBlockK + kEpilogueCost) * (gp.prob[i].bits == 3 ? 12 : (gp.prob[i].bits == 8 ? 14 : 10));
        }
      std::stable_sort(ids.begin(), ids.end(), [&](int a, int b) { return cost[a] > cost[b]; });
      std::vector<std::vector<int>> lists(grid);
      std::vector<long long> load(grid, 0);
      size_t max_len = 0;
      for (int t : ids) {
        int best = 0;
        for (int c = 1; c < grid; ++c)
          if (load[c] < load[best]) best = c;
        lists[best].push_back(t);
        load[best] += cost[t];
        if (lists[best].size() > max_len) max_len = lists[best].size();
      }
      if (max_len * (size_t)grid <= (size_t)kMaxOrder) {
        // Each CTA visits its own list shortest tile first: the short tile's epilogue then runs under the
        // long tile's main loop and the launch's first weight reads are spread over more tiles (measured
        // on a 6-linear mixed stack at M = 128: 5 % less than longest first).
        for (size_t i = 0; i < max_len; ++i)
          for (int c = 0; c < grid; ++c)
            gp.order[i * grid + c] = i < lists[c].size() ? (uint16_t)lists[c][lists[c].size() - 1 - i] : kNoTile;
        // the owner of every listed tile, so that the kernel's roles need not search for it at every tile
        for (int q = 0; q < (int)(max_len * grid); ++q) {
          if (gp.order[q] == kNoTile) continue;
          int pi = 0;
          while (pi + 1 < count && (int)gp.order[q] >= gp.prob[pi + 1].tile_begin) ++pi;
          gp.order_prob[q] = (uint8_t)pi;
        }
        gp.total_positions = (int32_t)(max_len * grid);
        gp.use_order = 1;
      }
    }
  }
  if (bits == 0) {
    if (out == kOutBf16) return launch_group_inst<128, 0, kOutBf16, 1>(gp, grid, stream);
    if (out == kOutI8) return launch_group_inst<128, 0, kOutI8, 1>(gp, grid, stream);
    return launch_group_inst<128, 0, kOutF32, 1>(gp, grid, stream);
  }
  if (cg == 2) {
    if (out == kOutBf16) return launch_group_bits<256, kOutBf16, 2>(bits, gp, 2 * grid, stream);
    if (out == kOutI8) return launch_group_bits<256, kOutI8, 2>(bits, gp, 2 * grid, stream);
    return launch_group_bits<256, kOutF32, 2>(bits, gp, 2 * grid, stream);
  }
  if (out == kOutBf16)
    return bt == 256 ? launch_group_bits<256, kOutBf16, 1>(bits, gp, grid, stream)
                     : launch_group_bits<128, kOutBf16, 1>(bits, gp, grid, stream);
  if (out == kOutI8)
    return bt == 256 ? launch_group_bits<256, kOutI8, 1>(bits, gp, grid, stream)
                     : launch_group_bits<128, kOutI8, 1>(bits, gp, grid, stream);
  return bt == 256 ? launch_group_bits<256, kOutF32, 1>(bits, gp, grid, stream)
                   : launch_group_bits<128, kOutF32, 1>(bits, gp, grid, stream);
}

struct StackGroup {
  int begin, count;
};
// The launches of a stack.  `order` lists the descriptors, every group is a run of `order` that one launch
// serves (at most kMaxProblems linears and 2^30 tiles).  A small stack (fewer than 16 tiles of 128 x 128
// per SM in all: a mixed-precision stack at small M) is cut in stack order only, longest K first inside a
// launch, and its launches mix bit widths: one launch, one tile list, one start-up and one drain for all
// of it.  A large stack is sorted by bit width (every launch then has its bit width compiled in), longest
// K first.
static void plan_stack(const qb_linear_desc* d, int count, int sm_count, std::vector<int>& order,
                       std::vector<StackGroup>& groups) {
  groups.clear();
  order.resize(count);
  for (int i = 0; i < count; ++i) order[i] = i;
  int64_t all_tiles = 0;
  bool mixed = false;
  for (int i = 0; i < count; ++i) {
    all_tiles += ((d[i].N + kTileN - 1) / kTileN) * ((d[i].M + 127) / 128);
    mixed = mixed || d[i].bits != d[0].bits;
  }
  const bool small = mixed && all_tiles < (int64_t)16 * sm_count;
  if (!small) {
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
      if (d[a].bits != d[b].bits) return d[a].bits < d[b].bits;
      return d[a].K > d[b].K;
    });
  }
  int i = 0;
  while (i < count) {
    int j = i;
    int64_t tiles = 0;
    while (j < count && j - i < kMaxProblems && (small || d[order[j]].bits == d[order[i]].bits)) {
      const int64_t t = ((d[order[j]].N + kTileN - 1) / kTileN) * ((d[order[j]].M + 127) / 128);
      if (j > i && tiles + t > (1 << 30)) break;
      tiles += t;
      ++j;
    }
    if (small)  // longest K first inside the launch: its tiles go out first
      std::stable_sort(order.begin() + i, order.begin() + j, [&](int a, int b) { return d[a].K > d[b].K; });
    groups.push_back({i, j - i});
    i = j;
  }
}

static qb_status launch_stack(const qb_linear_desc* d, int count, void* ws, int sm_count, cudaStream_t stream,
                              int out, const float* const* out_scales = nullptr) {
  std::vector<int> order;
  std::vector<StackGroup> groups;
  plan_stack(d, count, sm_count, order, groups);
  for (const StackGroup& g : groups) {
    qb_status st = launch_group(d, order.data() + g.begin, g.count, nullptr, ws, sm_count, stream, out, out_scales);
    if (st != QB_OK) return st;
  }
  return QB_OK;
}

}  // namespace qb

// fp32 or bfloat16 output: `y` is float* or uint16_t* (bfloat16 bit patterns) accordingly
static qb_status gemm_entry(const int8_t* xq, const float* act_scale, const int32_t* rowsum, const uint32_t* packed,
                            const float* delta, const float* q0, const float* bias, int64_t M, int64_t N, int64_t K,
                            int bits, int groups, void* y, int32_t* acc_out, void* ws, size_t ws_bytes,
                            void* cuda_stream, int out, const float* out_scale = nullptr) {
  qb_status st = qb::validate_gemm(xq, act_scale, rowsum, packed, delta, q0, M, N, K, bits, groups, y, ws, ws_bytes);
  if (st != QB_OK) return st;
  int sms = 0;
  st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  qb_linear_desc d;
  d.xq = xq;
  d.act_scale = act_scale;
  d.rowsum = rowsum;
  d.packed = packed;
  d.delta = delta;
  d.q0 = q0;
  d.bias = bias;
  d.M = M;
  d.N = N;
  d.K = K;
  d.bits = bits;
  d.groups = groups;
  d.y = static_cast<float*>(y);
  const int idx = 0;
  return qb::launch_group(&d, &idx, 1, acc_out, ws, sms, (cudaStream_t)cuda_stream, out, out_scale ? &out_scale : nullptr);
}

static qb_status stack_entry(const char* who, const qb_linear_desc* descs, int32_t count, void* ws, size_t ws_bytes,
                             void* cuda_stream, int out, const float* const* out_scales = nullptr) {
  if (!descs || count <= 0) {
    qb::set_last_error("%s: descs null or count <= 0", who);
    return QB_ERR_INVALID;
  }
  for (int i = 0; i < count; ++i) {
    const qb_linear_desc& d = descs[i];
    qb_status st = qb::validate_gemm(d.xq, d.act_scale, d.rowsum, d.packed, d.delta, d.q0, d.M, d.N, d.K, d.bits,
                                     d.groups, d.y, ws, ws_bytes);
    if (st != QB_OK) return st;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  return qb::launch_stack(descs, count, ws, sms, (cudaStream_t)cuda_stream, out, out_scales);
}

extern "C" qb_status qb_gemm(const int8_t* xq, const float* act_scale, const int32_t* rowsum,
                             const uint32_t* packed, const float* delta, const float* q0, const float* bias,
                             int64_t M, int64_t N, int64_t K, int bits, int groups, float* y, int32_t* acc_out,
                             void* ws, size_t ws_bytes, void* cuda_stream) {
  return gemm_entry(xq, act_scale, rowsum, packed, delta, q0, bias, M, N, K, bits, groups, y, acc_out, ws, ws_bytes,
                    cuda_stream, qb::kOutF32);
}

extern "C" qb_status qb_gemm_bf16(const int8_t* xq, const float* act_scale, const int32_t* rowsum,
                                  const uint32_t* packed, const float* delta, const float* q0, const float* bias,
                                  int64_t M, int64_t N, int64_t K, int bits, int groups, uint16_t* y, void* ws,
                                  size_t ws_bytes, void* cuda_stream) {
  return gemm_entry(xq, act_scale, rowsum, packed, delta, q0, bias, M, N, K, bits, groups, y, nullptr, ws, ws_bytes,
                    cuda_stream, qb::kOutBf16);
}

extern "C" qb_status qb_gemm_i8(const int8_t* xq, const float* act_scale, const int32_t* rowsum,
                                const uint32_t* packed, const float* delta, const float* q0, const float* bias,
                                int64_t M, int64_t N, int64_t K, int bits, int groups, const float* out_scale,
                                int8_t* yq, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!out_scale) {
    qb::set_last_error("qb_gemm_i8: out_scale is null");
    return QB_ERR_INVALID;
  }
  return gemm_entry(xq, act_scale, rowsum, packed, delta, q0, bias, M, N, K, bits, groups, yq, nullptr, ws, ws_bytes,
                    cuda_stream, qb::kOutI8, out_scale);
}

namespace qb {
// one warp per row, 16 codes per lane and load
__global__ void __launch_bounds__(256) rowsum_i8_kernel(const int4* __restrict__ xq, int64_t M, int64_t k16,
                                                        int32_t* __restrict__ rowsum) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * 8;
  for (int64_t m = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); m < M; m += warps) {
    int s = 0;
    for (int64_t c = lane; c < k16; c += 32) {
      const int4 v = __ldg(xq + m * k16 + c);
      s = __dp4a(v.x, 0x01010101, s);
      s = __dp4a(v.y, 0x01010101, s);
      s = __dp4a(v.z, 0x01010101, s);
      s = __dp4a(v.w, 0x01010101, s);
    }
    s = __reduce_add_sync(0xffffffffu, s);
    if (lane == 0) rowsum[m] = s;
  }
}
}  // namespace qb

extern "C" qb_status qb_rowsum_i8(const int8_t* xq, int64_t M, int64_t K, int32_t* rowsum, void* cuda_stream) {
  if (!xq || !rowsum || M <= 0 || K <= 0 || M > QB_MAX_MN || K > QB_MAX_K) {
    qb::set_last_error("qb_rowsum_i8: null pointer or size out of range (M=%lld K=%lld)", (long long)M, (long long)K);
    return QB_ERR_INVALID;
  }
  if (K % 128 != 0 || !qb::aligned16(xq)) {
    qb::set_last_error("qb_rowsum_i8: K must be a multiple of 128 and xq 16-byte aligned");
    return QB_ERR_ALIGN;
  }
  int sms = 0;
  qb_status st = qb::require_sm100(&sms);
  if (st != QB_OK) return st;
  int64_t blocks = (M + 7) / 8;
  if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
  qb::rowsum_i8_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(reinterpret_cast<const int4*>(xq), M,
                                                                                K / 16, rowsum);
  QB_CUDA_TRY(cudaGetLastError());
  return QB_OK;
}

extern "C" int32_t qb_layer_linears_launch_count(const qb_linear_desc* descs, int32_t count) {
  if (!descs || count <= 0) return 0;
  std::vector<int> order;
  std::vector<qb::StackGroup> groups;
  int sms = 148;
  qb::require_sm100(&sms);  // without a device: the plan for a 148-SM part
  qb::plan_stack(descs, count, sms, order, groups);
  return (int32_t)groups.size();
}

extern "C" qb_status qb_layer_linears(const qb_linear_desc* descs, int32_t count, void* ws, size_t ws_bytes,
                                      void* cuda_stream) {
  return stack_entry("qb_layer_linears", descs, count, ws, ws_bytes, cuda_stream, qb::kOutF32);
}

extern "C" qb_status qb_layer_linears_bf16(const qb_linear_desc* descs, int32_t count, void* ws, size_t ws_bytes,
                                           void* cuda_stream) {
  return stack_entry("qb_layer_linears_bf16", descs, count, ws, ws_bytes, cuda_stream, qb::kOutBf16);
}

extern "C" qb_status qb_layer_linears_i8(const qb_linear_desc* descs, const float* const* out_scales, int32_t count,
                                         void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!out_scales) {
    qb::set_last_error("qb_layer_linears_i8: out_scales is null");
    return QB_ERR_INVALID;
  }
  for (int i = 0; i < count; ++i)
    if (!out_scales[i]) {
      qb::set_last_error("qb_layer_linears_i8: out_scales[%d] is null", i);
      return QB_ERR_INVALID;
    }
  return stack_entry("qb_layer_linears_i8", descs, count, ws, ws_bytes, cuda_stream, qb::kOutI8, out_scales);
}
