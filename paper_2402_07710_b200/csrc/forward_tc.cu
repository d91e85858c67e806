// Tensor-core forward for f16 / bf16 features on sm_100a: output-stationary implicit GEMM.
//
// Algorithm 2 (Sec. III-C.3) per 128-row output tile:  D_tile = sum_k A_{tile,k} * W_k, where row r of
// A_{tile,k} is the input row feeding output row r of the tile through kernel offset k (zeros where there
// is none).  The contraction runs on tcgen05.mma with the fp32 accumulator of every tile of the CTA
// resident in TMEM until all offsets are summed, so each output row is written exactly once, offsets in
// ascending order, and nothing is accumulated through atomics.  The paper's computeConv kernel stages one
// output channel's weights in shared memory and lets one thread own an (output row, output channel) pair;
// here a CTA owns whole rows, W_k is staged per step by TMA, and (tile, offset)
// blocks without any input row are skipped (the tile plan groups rows with equal offset sets to make such
// blocks common).
//
// One persistent CTA per SM takes its share of the tiles from the kernel map's schedule (heaviest tiles
// first, dealt serpentine), up to 512 / COUT of them per round; one pipeline step = one (tile, offset)
// block, or, for rows shorter than 128 bytes, up to four offsets of one tile (see Cfg).  The CTA runs up to
// two gather -> MMA pipelines side by side; each owns a fixed subset of the CTA's tiles (so the MMAs of an
// accumulator come from one thread, in offset order), its own ring of stages with their barriers, eight
// producer warps, one issuer warp and one W loader warp.  A stage holds the gathered rows and the W_k of its
// step; only the shapes whose weights are too large for that keep W_k in slots of their own (see Cfg).
// The kernel waits for the grid before it in the stream (programmatic dependent launch) only when its step
// list is built: the set-up reads nothing but the kernel map.
//   producer warps   16-byte cp.async copies of the gathered feature rows into the swizzled K-major A
//                    tile (rows a block lacks are skipped and masked out of the MMA); a copy engine
//                    arrival on the stage's mbarrier replaces any wait for the data.
//   issuer warps     one per pipeline; the warp runs in lockstep and an elected lane issues tcgen05.mma and
//                    the commits that release stages.  The first issuer warp owns TMEM.
//   W loader warps   one per pipeline; lane 0 issues the TMA loads of W_k into the swizzled MN-major B tiles.
// After the last step all warps run the epilogue: tcgen05.ld of the accumulators, conversion, staging
// through shared memory, full-line stores.
// Every wait on an mbarrier is bounded (poll count and wall time); when a bound is hit the CTA raises a
// status bit, stops waiting, lets its copies in flight land, frees TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace spconv {
namespace {

constexpr int kMaxPipes = 2;                     // independent gather -> MMA pipelines per CTA (fewer when the A ring is short)
constexpr int kGroupWarps = 8;                   // producer warps of one pipeline (they share a step's rows)
constexpr int kGroupThreads = 32 * kGroupWarps;
constexpr int kMaxAStages = 12;                  // most stages a CTA's rings hold in all
#ifndef SPCONV_X_INSTAGE_MIN
#define SPCONV_X_INSTAGE_MIN 3
#endif
constexpr int kInStageMin = SPCONV_X_INSTAGE_MIN;                   // a stage carries its W_k where at least this many stages per pipeline fit
constexpr int kGroupMaxCin = 64;                 // widest input rows that take several offsets per step
// Shapes that take several offsets per step: short rows always; 128-byte rows (two offsets) only where two such stages per pipeline fit.
constexpr bool grouped_shape(int cin, int cout) { return cin <= kGroupMaxCin && (cin < 64 || cout <= 64); }
constexpr int kMaxGroup = 32;                    // tiles a CTA keeps in TMEM at once (<= 512 / COUT)
constexpr uint32_t kSpinLimit = 1u << 24;        // polls per wait, and
constexpr uint64_t kWaitLimitNs = 250ull * 1000 * 1000;  // wall-time bound per wait (0.25 s) unless a test shortens it
constexpr int kMaxSmem = 227 * 1024;             // largest dynamic shared memory a CTA may request on sm_100
constexpr int kStagingPitch = 64 * 2 + 16;       // epilogue staging row: 64 columns of 16 bits + one 16-byte pad

// GROUPED (rows shorter than 128 bytes, kernel volume <= 32): a step takes up to kSub offsets of its tile at once.
// The stage's A tile is 128 rows x 128 bytes whatever the row length, offset s of the step fills the byte columns
// [s * row bytes, (s + 1) * row bytes) of it, and the stage carries kSub W_k; the issuer runs one group of MMAs
// per offset, each with that offset's row mask.  A step then costs its fixed price (barrier hand-over, polls,
// commit) once per 128 bytes of gathered row instead of once per 32 or 64.
template <int CIN, int COUT, bool GROUPED = false>
struct Cfg {
  static constexpr bool kGrouped = GROUPED;
  static constexpr int kARowBytes = CIN * 2;
  // The A tile of a grouped stage is one or two 128-byte-wide panels; a panel holds 128 / row bytes offsets side by
  // side.  Two panels (up to four offsets for 64-byte rows, two for 128-byte rows) where two such stages per pipeline
  // fit with their W_k, else one panel.
  static constexpr int kSubPerPanel = kARowBytes <= 128 ? 128 / kARowBytes : 1;
  static constexpr int kSubWide = 2 * kSubPerPanel < 4 ? 2 * kSubPerPanel : 4;
  static constexpr int kWBytesOne = CIN * COUT * 2 < 1024 ? 1024 : CIN * COUT * 2;
  static constexpr int kWideStage = ((kSubWide + kSubPerPanel - 1) / kSubPerPanel) * kTileRows * 128 + kSubWide * kWBytesOne;
  static constexpr bool kWideFits = ((kMaxSmem - 1024 - 12 * 1024) / kWideStage) / kMaxPipes >= 2;
  static constexpr int kSub = GROUPED ? (kWideFits ? kSubWide : kSubPerPanel) : 1;          // offsets per step
  static_assert(!GROUPED || (kARowBytes <= 128 && kSub <= 4), "grouping is for rows of at most 128 bytes");
  static constexpr int kASpan = GROUPED ? 128 : (kARowBytes < 128 ? kARowBytes : 128);      // swizzle span of A (bytes)
  static constexpr int kAPanelBytes = kTileRows * kASpan;
  static constexpr int kAPanelsGrouped = (kSub + kSubPerPanel - 1) / kSubPerPanel;
  // (grouped) byte position of offset s of a step inside the A tile, before the row and chunk terms
  __host__ __device__ static constexpr int sub_offset(int s) { return (s / kSubPerPanel) * kAPanelBytes + (s % kSubPerPanel) * kARowBytes; }
  static constexpr int kABytes = GROUPED ? kAPanelsGrouped * kTileRows * 128 : kTileRows * kARowBytes;   // A tile of a stage
  static constexpr int kAChunksPerRow = kARowBytes / 16;
  static constexpr int kWRowBytes = COUT * 2;
  static constexpr int kWSpan = kWRowBytes < 128 ? kWRowBytes : 128;      // swizzle span of B (bytes)
  static constexpr int kWPanels = kWRowBytes / kWSpan;
  static constexpr int kWPanelBytes = CIN * kWSpan;
  static constexpr int kWBytesRaw = CIN * kWRowBytes;
  static constexpr int kWBytes = kWBytesRaw < 1024 ? 1024 : kWBytesRaw;   // one W_k in shared memory
  static constexpr int kWSlotBytes = kSub * kWBytes;                       // W region of a stage / one W slot
  // Every pipeline has its own ring of stages.  Where enough stages per pipeline fit with W_k inside them, a stage
  // holds the gathered rows AND the weights of its step (kWInStage): one barrier says both are there and one
  // commit frees both, so the issuer polls once and commits once per step; W_k is then fetched once per step,
  // which costs nothing measurable (it comes from L2, and a pipeline rarely has two tiles with the same offset).
  // Otherwise W_k lives in slots of its own that are filled once per offset: private to a pipeline when that
  // fits (kWStagesPer each); shared by the pipelines for the largest weights, which every issuer then has to
  // wait for and release (kSharedW); and if even that does not fit there is one pipeline.
  static constexpr int kAvail = kMaxSmem - 1024 - 12 * 1024;
  static constexpr int kInStageFit = kAvail / (kABytes + kWSlotBytes);
  static constexpr bool kWInStage = kMaxPipes > 1 && kInStageFit / kMaxPipes >= (GROUPED ? 2 : kInStageMin);
  static constexpr int kWSlotsPrivate = kWBytes >= 16384 ? 2 : (kWBytes >= 8192 ? 3 : 4);
  static constexpr int kWSlotsShared = kWBytes >= 32768 ? 2 : 4;
  static constexpr bool kPrivateFits = kWInStage || kMaxPipes * (kWSlotsPrivate * kWSlotBytes + 2 * kABytes) <= kAvail;
  static constexpr bool kSharedW = !kPrivateFits && kMaxPipes > 1 && kMaxPipes * 2 * kABytes + kWSlotsShared * kWSlotBytes <= kAvail;
  static constexpr int kPipes = (kPrivateFits || kSharedW) ? kMaxPipes : 1;
  static constexpr int kWLoaders = kSharedW ? 1 : kPipes;
  static constexpr int kProducerWarps = kPipes * kGroupWarps;
  static constexpr int kThreads = 32 * (kProducerWarps + kPipes + kWLoaders);   // producers, one MMA issuer warp per pipeline, W loader warps
  static constexpr int kInStagePer = kInStageFit / kPipes < kMaxAStages / kPipes ? kInStageFit / kPipes : kMaxAStages / kPipes;
  static constexpr int kWStagesPer = kSharedW ? kWSlotsShared : kWSlotsPrivate;   // depth of the W ring an issuer sees (not kWInStage)
  static constexpr int kWStagesRing = kSharedW ? kWSlotsShared : kPipes * kWSlotsPrivate;
  static constexpr int kBudget = kAvail - kWStagesRing * kWSlotBytes;
  static constexpr int kStagesFit = kBudget / kABytes >= kMaxAStages ? kMaxAStages : kBudget / kABytes;
  static constexpr int kStagesPer = kWInStage ? kInStagePer : kStagesFit / kPipes;   // ring depth of one pipeline
  static constexpr int kStages = kStagesPer * kPipes;                     // stages in all
  static constexpr int kWStages = kWInStage ? kStages : kWStagesRing;     // W slots in all (kWInStage: slot s belongs to stage s)
  static constexpr int kKSteps = CIN / 16;                                // UMMA_K = 16 for 16-bit inputs
  static constexpr int kMaxTilesInTmem = 512 / COUT < kMaxGroup ? 512 / COUT : kMaxGroup;
  static_assert(kStagesPer >= 2 && kProducerWarps >= 4, "A ring too shallow");
  // the epilogue staging area (32 rows per warp) reuses the A and W rings once the main loop is over
  static constexpr int kEpiFit = (kStages * kABytes + kWStages * kWSlotBytes) / (32 * kStagingPitch);
  static_assert(!GROUPED || kWInStage, "grouped steps carry their W_k in the stage");
  static constexpr int kEpilogueWarps = ((kEpiFit >= kThreads / 32 ? kThreads / 32 : kEpiFit) / 4) * 4;   // all warps help once their role is done
  static_assert(kEpilogueWarps >= 4, "staging does not fit the rings");
};

__host__ __device__ constexpr uint32_t layout_type_of_span(int span) { return span == 128 ? 2u : span == 64 ? 4u : 6u; }

struct Smem {  // fixed-size part that follows the A and W rings
  unsigned long long full_a[kMaxAStages], empty_a[kMaxAStages], full_w[kMaxPipes * 4], empty_w[kMaxPipes * 4], accum_full, drain;
  uint32_t stage_absent[kMaxAStages][4][4];   // per A stage and offset of the step: 128-bit mask of the tile rows that were not gathered (16-byte aligned)
  uint32_t tmem_base;
  int n_steps;
  int n_own[kMaxPipes];   // steps of each pipeline
  int abort_flag;
  int tile[kMaxGroup];
  uint32_t mask[kMaxGroup][kMaskWordsMax];
};

// ------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking polls.  mbar_test_wait3 issues three of them back to back so that their latencies overlap.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void mbar_test_wait3(uint32_t bar0, uint32_t par0, uint32_t bar1, uint32_t par1, uint32_t bar2, uint32_t par2,
                                                uint32_t& ok0, uint32_t& ok1, uint32_t& ok2) {
  asm volatile(
      "{\n\t.reg .pred p0, p1, p2;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p0, [%3], %4;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p1, [%5], %6;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p2, [%7], %8;\n\t"
      "selp.u32 %0, 1, 0, p0;\n\t"
      "selp.u32 %1, 1, 0, p1;\n\t"
      "selp.u32 %2, 1, 0, p2;\n\t}"
      : "=r"(ok0), "=r"(ok1), "=r"(ok2)
      : "r"(bar0), "r"(par0), "r"(bar1), "r"(par1), "r"(bar2), "r"(par2)
      : "memory");
}
// What every bounded wait of a CTA needs: the CTA's give-up flag, the kernel map's status words, the time limit.
struct WaitCtx {
  volatile int* abort_flag;
  uint32_t* diag;
  uint64_t limit_ns;
};
// Bounded wait: at most kSpinLimit polls and at most limit_ns of wall time.  Returns false when a
// bound was hit or another thread of the CTA already gave up.
// `where` identifies the wait (role << 24 | detail); the first wait of the CTA that gives up records it in
// the kernel map's status words 1 (code) and 2 (CTA + 1), first writer wins, for post-mortem reading.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& ctx, uint32_t where) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*ctx.abort_flag) return false;
    if ((it & 63u) == 63u && global_timer_ns() - t0 > ctx.limit_ns) break;
  }
  if (atomicExch(const_cast<int*>(ctx.abort_flag), 1) == 0) {
    atomicCAS(ctx.diag + 1, 0u, where | 0x80000000u);
    atomicCAS(ctx.diag + 2, 0u, blockIdx.x + 1u);
  }
  return false;
}
// Warp-wide bounded wait: lane 0 polls, the other lanes take its verdict (they are ordered behind lane 0's
// acquire by the warp-level synchronisation of the shuffle).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const WaitCtx& ctx, uint32_t where) {
  bool ok = true;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, ctx, where);
  return __shfl_sync(0xffffffffu, int(ok), 0) != 0;
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

// Shared-memory matrix descriptor of tcgen05.mma (version 1, base offset 0), split into its two words:
// bits 0-13 start address >> 4, 16-29 leading byte offset >> 4 | 32-45 stride byte offset >> 4, 46 version,
// 61-63 swizzle mode.
__host__ __device__ constexpr uint64_t make_smem_desc_hi(uint32_t sbo_bytes, uint32_t layout_type) {
  return ((uint64_t((sbo_bytes >> 4) & 0x3FFFu) << 32) | (uint64_t(1) << 46) | (uint64_t(layout_type) << 61)) >> 32;
}
__device__ __forceinline__ uint32_t make_smem_desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
// tcgen05.mma with each descriptor given as (low word, high word) and a 128-bit mask of accumulator lanes
// (tile rows) that must not be updated.
__device__ __forceinline__ void umma_f16_masked(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                uint32_t idesc, const uint4& lanes_off, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, {%7, %8, %9, %10}, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(lanes_off.x), "r"(lanes_off.y),
        "r"(lanes_off.z), "r"(lanes_off.w)
      : "memory");
}
// True in exactly one lane of the (converged) warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16_zero(uint32_t taddr, uint32_t z) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
      ::"r"(taddr), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack2(float lo, float hi, int is_bf16) {
  if (is_bf16) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
  }
  __half2 t = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Section timing for development builds (-DSPCONV_TC_PROFILE): cycle sums of the first round, written to
// slots 8-15 of the CTA's timeline record: 8 steps of pipeline 0 | steps of the last pipeline << 32,
// 9-12 issuer 0 (barrier waits; fences + MMAs + stage commit; offset-group ends; whole loop), 13 W loader
// waits, 14-15 producer warp 0 (stage waits; everything else).  Compiled out otherwise.
#ifdef SPCONV_TC_PROFILE
#define SPCONV_PROF_T(var) const long long var = clock64()
#define SPCONV_PROF_ADD(acc, a, b) acc += (b) - (a)
#else
#define SPCONV_PROF_T(var)
#define SPCONV_PROF_ADD(acc, a, b)
#endif

// Step list entry: bits 0-4 tile slot g, bits 5-11 offset k, bit 12 first step of its offset in its pipeline, bit 13
// last, bits 14-15 the pipeline.
constexpr uint32_t kStepFirst = 1u << 12, kStepLast = 1u << 13, kStepIssuerShift = 14;

template <int CIN, int COUT, bool GROUPED>
__global__ void __launch_bounds__((Cfg<CIN, COUT, GROUPED>::kThreads), 1)
k_forward_tc(const __grid_constant__ CUtensorMap w_map, const uint8_t* __restrict__ feats,
             const int32_t* __restrict__ tile_nbr, const uint8_t* __restrict__ tile_crow, const int32_t* __restrict__ tile_rows,
             const uint32_t* __restrict__ tile_mask, const uint32_t* __restrict__ tile_absent,
             const int32_t* __restrict__ sorted_tiles, uint8_t* __restrict__ out,
             int n_tiles, int kvol, int mask_words, int G, int n_rounds, uint32_t tmem_cols, uint32_t idesc, int is_bf16,
             uint32_t* __restrict__ status, unsigned long long* __restrict__ timeline, long long feat_lines, int strict_order,
             unsigned long long wait_limit_ns, int withhold_first_w) {
  using C = Cfg<CIN, COUT, GROUPED>;
  extern __shared__ uint8_t smem_raw[];
  // Swizzled operand tiles need 1024-byte aligned bases.
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* a_ring = smem;
  uint8_t* w_ring = a_ring + C::kStages * C::kABytes;
  Smem* sm = reinterpret_cast<Smem*>(w_ring + C::kWStages * C::kWSlotBytes);
  uint32_t* step_blk = reinterpret_cast<uint32_t*>(sm + 1);                         // [kvol * kMaxTilesInTmem]: tile * kvol + offset
  uint16_t* steps = reinterpret_cast<uint16_t*>(step_blk + kvol * C::kMaxTilesInTmem);  // [kvol * kMaxTilesInTmem]
  uint16_t* own_steps = steps + kvol * C::kMaxTilesInTmem;                              // [kPipes][kvol * kMaxTilesInTmem]: a pipeline's steps

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sm->abort_flag;
  const WaitCtx wctx{abort_flag, status, wait_limit_ns};
  // Optional per-CTA timeline (diagnostics): globaltimer stamps when a buffer is installed.
  auto stamp = [&](int slot) { if (timeline != nullptr) timeline[size_t(blockIdx.x) * 16 + slot] = global_timer_ns(); };
  if (tid == 0) stamp(0);

  if (tid == 0) {
    for (int s = 0; s < C::kStages; ++s) { mbar_init(smem_u32(&sm->full_a[s]), kGroupThreads + (C::kWInStage ? 1 : 0)); mbar_init(smem_u32(&sm->empty_a[s]), 1); }
    for (int s = 0; s < (C::kWInStage ? 0 : C::kWStages); ++s) { mbar_init(smem_u32(&sm->full_w[s]), 1); mbar_init(smem_u32(&sm->empty_w[s]), C::kSharedW ? C::kPipes : 1); }
    mbar_init(smem_u32(&sm->accum_full), C::kPipes);
    mbar_init(smem_u32(&sm->drain), C::kPipes);
    sm->abort_flag = 0;
    sm->n_steps = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == C::kProducerWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm->tmem_base)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Programmatic dependent launch: the kernel that follows in the stream may be scheduled as soon as SMs have
  // room, and its CTAs then set up while this grid's slowest CTAs finish.  Setting up reads only the kernel
  // map, which is complete before a handle exists (the build returns after the device has reported the tile
  // plan done); features, weights and output rows may be the work of whatever precedes this grid in the
  // stream, so nothing touches them before griddepcontrol.wait below, where the first round's step list is
  // ready.  Without the launch attribute both instructions do nothing.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // strict_order: the launch was enqueued together with the map's own build, so the map is read only behind it too.
  if (strict_order) asm volatile("griddepcontrol.wait;" ::: "memory");
  // The input rows are requested into L2 (a request only: no data reaches the SM, so it does not matter that the
  // preceding grid may still be writing them).  After a layer that has just written them this does nothing;
  // rows that come from device memory are then on their way while the CTAs set up and wait.
  for (long long i = (long long)blockIdx.x * C::kThreads + tid; i < feat_lines; i += (long long)gridDim.x * C::kThreads)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(feats + i * 128));

  // Running ring positions over all rounds.  Each role advances only what it uses itself, always by the
  // same amounts: the producers a_step (steps of their own pipeline), an issuer its stage / W slot, the W loader w_group.
  uint32_t a_step = 0, w_group = 0, accum_uses = 0;
  uint32_t mma_stage = 0, mma_phase = 0, mma_wslot = 0, mma_wphase = 0;

  for (int round = 0; round < n_rounds; ++round) {
    // ---- this CTA's tiles of the round (schedule: heaviest tiles first, dealt serpentine over the CTAs)
    if (tid < kMaxGroup) {
      int t = -1;
      uint32_t words[kMaskWordsMax];
#pragma unroll
      for (int w = 0; w < kMaskWordsMax; ++w) words[w] = 0u;
      if (tid < G) {
        const int j = round * G + tid;
        const long long p = (long long)j * gridDim.x + ((j & 1) ? int(gridDim.x) - 1 - int(blockIdx.x) : int(blockIdx.x));
        if (p < n_tiles) {   // schedule record: tile index, then its offset mask words
          const int32_t* rec = sorted_tiles + size_t(p) * (1 + mask_words);
          t = rec[0];
#pragma unroll
          for (int w = 0; w < kMaskWordsMax; ++w) if (w < mask_words) words[w] = uint32_t(rec[1 + w]);
        }
      }
      sm->tile[tid] = t;
#pragma unroll
      for (int w = 0; w < kMaskWordsMax; ++w) sm->mask[tid][w] = words[w];
    }
    if (round == 0) tc_fence_before();
    __syncthreads();
    if (round == 0) tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    // Output rows of this warp's first two epilogue tiles, fetched now so that the epilogue does not wait for them.
    int early_row[2] = {-1, -1};
    if (warp < C::kEpilogueWarps) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int g = (warp >> 2) + u * (C::kEpilogueWarps / 4);
        const int t = g < G ? sm->tile[g] : -1;
        if (t >= 0) early_row[u] = __ldg(tile_rows + size_t(t) * kTileRows + (warp & 3) * 32 + lane);
      }
    }
    if (tid == 0 && round == 0) stamp(1);
    // ---- every MMA accumulates (rows a block lacks are masked, not zeroed), so the accumulators start at zero
    constexpr int kZeroWarp0 = C::kProducerWarps >= 8 ? 4 : 0;   // four warps, one per TMEM lane quarter (warp 0 also builds the step list)
    if (warp >= kZeroWarp0 && warp < kZeroWarp0 + 4) {
      const uint32_t z = 0u;
      for (int c0 = 0; c0 < G * COUT; c0 += 16)
        tmem_st16_zero(tmem_base + (uint32_t((warp & 3) * 32) << 16) + uint32_t(c0), z);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      tc_fence_before();
    }
    // ---- ordered step list, offset-major: for every offset the tiles that have it; every tile (and so every
    // step) belongs to one pipeline, and each pipeline also gets the list of its own steps.  One lane per
    // offset: it counts the tiles that have the offset, a warp scan turns the counts into list positions,
    // and the lane writes its offset's entries (work proportional to the tiles of the CTA, not to the offsets).
    if (warp == 0) {
      int cnt = 0;
      int own_cnt[C::kPipes];
#pragma unroll
      for (int p = 0; p < C::kPipes; ++p) own_cnt[p] = 0;
      const int own_stride = kvol * C::kMaxTilesInTmem;
      // Tiles come heaviest first; each goes to the pipeline with the least work so far (two bits per tile).
      // A CTA is as slow as its busier pipeline, so this split matters as much as the split across CTAs.
      uint64_t assign = 0;
      {
        int load[C::kPipes];
#pragma unroll
        for (int p = 0; p < C::kPipes; ++p) load[p] = 0;
        // lane g weighs tile g (its steps) once; the sequential part below takes the weights by shuffle
        int my_weight = 0;
        if (lane < G) {
          for (int w = 0; w < mask_words; ++w) my_weight += __popc(sm->mask[lane][w]);
          my_weight = (my_weight + C::kSub - 1) / C::kSub;
        }
        for (int g = 0; g < G; ++g) {
          const int c = __shfl_sync(0xffffffffu, my_weight, g);
          int best = 0, best_load = load[0];
#pragma unroll
          for (int p = 1; p < C::kPipes; ++p)
            if (load[p] < best_load) { best = p; best_load = load[p]; }
#pragma unroll
          for (int p = 0; p < C::kPipes; ++p) load[p] += (p == best) ? c : 0;
          assign |= uint64_t(best) << (2 * g);
        }
      }
      auto pipe_of = [&](int g) { return int((assign >> (2 * g)) & 3u); };
      auto excl_scan = [&](int v, int& total) {
        int incl = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) { const int t = __shfl_up_sync(0xffffffffu, incl, off); if (lane >= off) incl += t; }
        total = __shfl_sync(0xffffffffu, incl, 31);
        return incl - v;
      };
      if constexpr (C::kGrouped) {
        // Tile-major lists, one per pipeline: lane g owns tile slot g and writes its steps, each step up to kSub
        // of the tile's offsets in ascending order.  Step word: bits 0-4 tile slot, 5-7 offsets in the step - 1,
        // then six bits per offset.  (The greedy split above weighs a tile by its offsets; steps follow it closely.)
        uint32_t* gsteps = reinterpret_cast<uint32_t*>(step_blk);   // [kPipes][own_stride]
        const int g = lane;
        const uint32_t mk = g < G ? sm->mask[g][0] : 0u;
        const int nst = (__popc(mk) + C::kSub - 1) / C::kSub;
        const int pg = g < G ? pipe_of(g) : -1;
        int my_start = 0, all = 0;
#pragma unroll
        for (int p = 0; p < C::kPipes; ++p) {
          int total = 0;
          const int st = excl_scan(pg == p ? nst : 0, total);
          if (pg == p) my_start = st;
          own_cnt[p] = total;
          all += total;
        }
        uint32_t rest = mk;
        int at = my_start;
        while (rest != 0u) {
          uint32_t word = uint32_t(g);
          int c = 0;
#pragma unroll
          for (int sidx = 0; sidx < C::kSub; ++sidx) {
            if (rest == 0u) break;
            const uint32_t k = uint32_t(__ffs(int(rest)) - 1);
            rest &= rest - 1u;
            word |= k << (8 + 6 * sidx);
            ++c;
          }
          word |= uint32_t(c - 1) << 5;
          gsteps[pg * own_stride + at++] = word;
        }
        cnt = all;
      } else
      for (int w = 0; w < mask_words; ++w) {
        const int k = 32 * w + lane;
        int c = 0;
        int cp[C::kPipes];
#pragma unroll
        for (int p = 0; p < C::kPipes; ++p) cp[p] = 0;
        for (int g = 0; g < G; ++g) {
          const int bit = int((sm->mask[g][w] >> lane) & 1u);
          const int pg = pipe_of(g);
          c += bit;
#pragma unroll
          for (int p = 0; p < C::kPipes; ++p) cp[p] += (pg == p) ? bit : 0;
        }
        int total = 0;
        const int start = cnt + excl_scan(c, total);
        int startp[C::kPipes], totalp[C::kPipes];
#pragma unroll
        for (int p = 0; p < C::kPipes; ++p) startp[p] = own_cnt[p] + excl_scan(cp[p], totalp[p]);
        int j = 0;
        int seenp[C::kPipes];
#pragma unroll
        for (int p = 0; p < C::kPipes; ++p) seenp[p] = 0;
        for (int g = 0; g < G; ++g) {
          if (!((sm->mask[g][w] >> lane) & 1u)) continue;
          const int pg = pipe_of(g), at = start + j;
          // first / last: among the steps of this offset that belong to the same pipeline (its W slot's life)
          bool first = false, last = false;
#pragma unroll
          for (int p = 0; p < C::kPipes; ++p)
            if (pg == p) {
              first = seenp[p] == 0;
              last = seenp[p] == cp[p] - 1;
              ++seenp[p];
              own_steps[p * own_stride + startp[p]++] = uint16_t(at);
            }
          steps[at] = uint16_t(uint32_t(g) | (uint32_t(k) << 5) | (first ? kStepFirst : 0u) | (last ? kStepLast : 0u) |
                               (uint32_t(pg) << kStepIssuerShift));
          step_blk[at] = uint32_t(sm->tile[g]) * uint32_t(kvol) + uint32_t(k);
          ++j;
        }
        cnt += total;
#pragma unroll
        for (int p = 0; p < C::kPipes; ++p) own_cnt[p] += totalp[p];
      }
      if (lane == 0) {
        sm->n_steps = cnt;
#pragma unroll
        for (int p = 0; p < C::kPipes; ++p) sm->n_own[p] = own_cnt[p];
      }
    }
    __syncthreads();
    const int n_steps = sm->n_steps;
    // The compacted block lists of all of this round's steps are requested into L2 now, so that the producers'
    // index fetches a few steps ahead of the copies find them there even when the kernel map is cold.
    if constexpr (C::kGrouped) {   // (tile slot, offset) pairs straight from the masks
      for (int i = tid; i < G * 32; i += C::kThreads) {   // one thread per (tile slot, offset): the six lines of its block
        const int g = i >> 5, k = i & 31;
        if (!((sm->mask[g][0] >> k) & 1u)) continue;
        const size_t blk = size_t(sm->tile[g]) * size_t(kvol) + size_t(k);
#pragma unroll
        for (int part = 0; part < 4; ++part) asm volatile("prefetch.global.L2 [%0];" ::"l"(tile_nbr + blk * kTileRows + part * 32));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(tile_crow + blk * kTileRows));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(tile_absent + blk * 4));
      }
    } else
    for (int i = tid; i < n_steps * 6; i += C::kThreads) {
      const size_t blk = step_blk[i / 6];
      const int part = i % 6;
      const void* line = part < 4 ? static_cast<const void*>(tile_nbr + blk * kTileRows + part * 32)
                       : part == 4 ? static_cast<const void*>(tile_crow + blk * kTileRows)
                                   : static_cast<const void*>(tile_absent + blk * 4);
      asm volatile("prefetch.global.L2 [%0];" ::"l"(line));
    }
    if (tid == 0 && round == 0) stamp(2);
    if (round == 0) asm volatile("griddepcontrol.wait;" ::: "memory");

    // =============================== epilogue (every warp that has staging room, once its role is done) ===============================
    auto run_epilogue = [&](bool ok) {
      if (ok) { ok = mbar_wait_warp(smem_u32(&sm->accum_full), accum_uses & 1u, wctx, 2u << 24); ++accum_uses; }
      tc_fence_after();
      if (tid == 0 && round == 0) stamp(4);
      if (ok) {
        // Warps w, w + 4, ... share TMEM lane quarter w % 4 and take the tiles round-robin.  A warp stages 32 rows of at
        // most 64 columns in shared memory (the A ring is idle now) and writes them out as full lines.
        uint8_t* stg = a_ring + warp * (32 * kStagingPitch);
        const int quarter = warp & 3;
        int visit = 0;
        for (int g = warp >> 2; g < G && warp < C::kEpilogueWarps; g += C::kEpilogueWarps / 4, ++visit) {
          const int t = sm->tile[g];
          if (t < 0) continue;
          bool any = false;
          for (int w = 0; w < kMaskWordsMax; ++w) any |= sm->mask[g][w] != 0u;
          // output row of TMEM lane 32 * quarter + lane
          const int my_row = visit == 0 ? early_row[0] : visit == 1 ? early_row[1] : tile_rows[size_t(t) * kTileRows + quarter * 32 + lane];
#pragma unroll
          for (int h = 0; h < COUT; h += 64) {
            constexpr int kCols = COUT < 64 ? COUT : 64;
#pragma unroll
            for (int c0 = 0; c0 < kCols; c0 += 16) {
              uint32_t v[16];
              if (any) {
                tmem_ld16(tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(g * COUT + h + c0), v);
                tmem_ld_wait();
              } else {
#pragma unroll
                for (int z = 0; z < 16; ++z) v[z] = 0u;
              }
              uint4 lo, hi;
              lo.x = pack2(__uint_as_float(v[0]), __uint_as_float(v[1]), is_bf16);
              lo.y = pack2(__uint_as_float(v[2]), __uint_as_float(v[3]), is_bf16);
              lo.z = pack2(__uint_as_float(v[4]), __uint_as_float(v[5]), is_bf16);
              lo.w = pack2(__uint_as_float(v[6]), __uint_as_float(v[7]), is_bf16);
              hi.x = pack2(__uint_as_float(v[8]), __uint_as_float(v[9]), is_bf16);
              hi.y = pack2(__uint_as_float(v[10]), __uint_as_float(v[11]), is_bf16);
              hi.z = pack2(__uint_as_float(v[12]), __uint_as_float(v[13]), is_bf16);
              hi.w = pack2(__uint_as_float(v[14]), __uint_as_float(v[15]), is_bf16);
              *reinterpret_cast<uint4*>(stg + lane * kStagingPitch + c0 * 2) = lo;
              *reinterpret_cast<uint4*>(stg + lane * kStagingPitch + c0 * 2 + 16) = hi;
            }
            __syncwarp();
            constexpr int kLanesPerRow = kCols / 8, kRowsPerInst = 32 / kLanesPerRow;
#pragma unroll
            for (int it = 0; it < kLanesPerRow; ++it) {
              const int sub = it * kRowsPerInst + lane / kLanesPerRow, chunk = lane % kLanesPerRow;
              const int orow = __shfl_sync(0xffffffffu, my_row, sub);
              const uint4 val = *reinterpret_cast<const uint4*>(stg + sub * kStagingPitch + chunk * 16);
              if (orow >= 0) *reinterpret_cast<uint4*>(out + size_t(orow) * (COUT * 2) + h * 2 + chunk * 16) = val;
            }
            __syncwarp();
          }
        }
      }
      // the staging writes went through the generic proxy; the next round's copies into the ring must see them done
      fence_proxy_async();
      tc_fence_before();
      if (tid == 0 && round == 0) stamp(5);
    };

    if (warp < C::kProducerWarps) {
      // =============================== gather producers ===============================
      // The producer warps of pipeline p fill the steps of p's tiles, in order, into p's own ring of kStagesPer
      // stages; within the pipeline fills and releases both happen in step order.
      // Only rows that exist are copied: a block's input rows come compacted (tile_nbr) with the tile row each
      // one feeds (tile_crow); warp w of the group takes the entries 16w..16w+15 and has nothing to do when the
      // block has fewer.  A feature row is copied by kCPR consecutive lanes (16 bytes each, cp.async), so a warp
      // instruction moves 32 / kCPR rows; lane group gq owns the kEPG consecutive entries
      // 16w + gq * kEPG .. + kEPG - 1 and loads their indices itself with one vector load each for rows and
      // positions (no shuffles on the copy path).  The entries are fetched kIdxDepth steps ahead into a
      // register ring that is indexed statically: the step loop is unrolled kIdxDepth times and slot d is
      // refilled right after step i0 + d has used it.  Tile rows that are not written keep stale data: the MMA
      // is told not to update their accumulator lanes (stage_absent).  No thread waits for its data: the copy
      // engine arrives on the stage's barrier when the thread's copies have landed.
      bool ok = true;
      constexpr int kCPR = C::kAChunksPerRow, kRPI = 32 / kCPR, kRows = kTileRows / kGroupWarps;
      constexpr int kEPG = kRows / kRPI;    // entries per lane group and step: 1, 2, 4, 8 or 16
      constexpr int kIdxDepth = kEPG >= 16 ? 2 : 4;
      static_assert(kEPG >= 1 && kEPG <= 16 && kEPG * kRPI == kRows && (kEPG < 4 || kEPG % 4 == 0), "entry split");
      constexpr int kRowWords = (kEPG + 3) / 4;
      // grouped: a warp takes one offset of a step and kTileRows / (kGroupWarps / kSub) of its entries
      constexpr int kEnt = C::kGrouped ? (kTileRows / (kGroupWarps / C::kSub)) / kRPI : kEPG;   // entries a lane group copies per step
      static_assert(!C::kGrouped || kEnt == 4 || kEnt == 8, "grouped entry split");
      constexpr int kEntWords = C::kGrouped ? kEnt / 4 : kRowWords;
      struct Entries { int idx[kEnt]; uint32_t rows[kEntWords]; uint32_t blk; };   // grouped: blk holds the step word
      Entries q[kIdxDepth];
      const int gq = lane / kCPR, chunk = lane % kCPR;
      const int pipe = warp / kGroupWarps, wg = warp % kGroupWarps;
      const uint16_t* own = own_steps + pipe * (kvol * C::kMaxTilesInTmem);
      const int n_own = sm->n_own[pipe];
      const uint32_t* gsteps = reinterpret_cast<const uint32_t*>(step_blk) + pipe * (kvol * C::kMaxTilesInTmem);
      const int my_sub = wg % C::kSub, my_range = wg / C::kSub;   // (grouped) this warp's offset of a step and its range of entries
      const int my_sub_offset = C::sub_offset(my_sub);
      static_assert(!C::kGrouped || kGroupWarps % C::kSub == 0, "grouped entry split");
      auto fetch = [&](int m, Entries& en) {
#pragma unroll
        for (int j = 0; j < kEnt; ++j) en.idx[j] = -1;
#pragma unroll
        for (int j = 0; j < kEntWords; ++j) en.rows[j] = 0u;
        en.blk = 0u;
        if (m >= n_own) return;
        if constexpr (C::kGrouped) {
          // A warp takes one offset of the step (its index modulo kSub) and a contiguous range of that offset's
          // entries, four per lane group: one vector load each for rows and positions, as for 128-byte rows.
          const uint32_t word = gsteps[m];
          en.blk = word;
          const int n_sub = int((word >> 5) & 7u) + 1;
          if (my_sub < n_sub) {
            const size_t at = (size_t(sm->tile[word & 31u]) * size_t(kvol) + ((word >> (8 + 6 * my_sub)) & 63u)) * kTileRows +
                              size_t(my_range * (kTileRows / (kGroupWarps / C::kSub)) + gq * kEnt);
#pragma unroll
            for (int v4 = 0; v4 < kEnt / 4; ++v4) {
              const int4 v = __ldg(reinterpret_cast<const int4*>(tile_nbr + at) + v4);
              en.idx[4 * v4] = v.x; en.idx[4 * v4 + 1] = v.y; en.idx[4 * v4 + 2] = v.z; en.idx[4 * v4 + 3] = v.w;
              en.rows[v4] = __ldg(reinterpret_cast<const uint32_t*>(tile_crow + at) + v4);
            }
          }
          return;
        }
        en.blk = step_blk[own[m]];
        const size_t at = size_t(en.blk) * kTileRows + wg * kRows + gq * kEPG;
        if constexpr (kEPG == 1) {
          en.idx[0] = __ldg(tile_nbr + at);
          en.rows[0] = __ldg(tile_crow + at);
        } else if constexpr (kEPG == 2) {
          const int2 v = __ldg(reinterpret_cast<const int2*>(tile_nbr + at));
          en.idx[0] = v.x; en.idx[1] = v.y;
          en.rows[0] = __ldg(reinterpret_cast<const unsigned short*>(tile_crow + at));
        } else {
#pragma unroll
          for (int v4 = 0; v4 < kEPG / 4; ++v4) {
            const int4 v = __ldg(reinterpret_cast<const int4*>(tile_nbr + at) + v4);
            en.idx[4 * v4] = v.x; en.idx[4 * v4 + 1] = v.y; en.idx[4 * v4 + 2] = v.z; en.idx[4 * v4 + 3] = v.w;
            en.rows[v4] = __ldg(reinterpret_cast<const uint32_t*>(tile_crow + at) + v4);
          }
        }
      };
#pragma unroll
      for (int d = 0; d < kIdxDepth; ++d) fetch(d, q[d]);
      const int panel = (chunk * 16) / C::kASpan, within = (chunk * 16) % C::kASpan;
      const uint8_t* feats_lane = feats + chunk * 16;
      const uint32_t a_lane0 = smem_u32(a_ring) + panel * C::kAPanelBytes;
      const bool mask_thread = wg == kGroupWarps - 1 && lane == 0;   // the group's last warp has the fewest rows to copy
      [[maybe_unused]] long long pc_wait = 0, pc_copy = 0, pc_rest = 0;
      for (int m0 = 0; m0 < n_own && ok; m0 += kIdxDepth) {
#pragma unroll
        for (int d = 0; d < kIdxDepth; ++d) {
          const int m = m0 + d;
          if (m >= n_own || !ok) continue;
          const uint32_t s = a_step + uint32_t(m);
          const uint32_t stage = uint32_t(pipe * C::kStagesPer) + s % uint32_t(C::kStagesPer);
          const uint32_t parity = ((s / uint32_t(C::kStagesPer)) & 1u) ^ 1u;
          SPCONV_PROF_T(c0);
          // every lane polls (one warp instruction, no divergence); measured faster than one lane plus a broadcast
          if (!__all_sync(0xffffffffu, mbar_test_wait(smem_u32(&sm->empty_a[stage]), parity))) {
            ok = mbar_wait_warp(smem_u32(&sm->empty_a[stage]), parity, wctx, (1u << 24) | uint32_t(m));
            if (!ok) continue;
          }
          SPCONV_PROF_T(c1);
          const Entries& en = q[d];
          if constexpr (C::kGrouped) {
            // this warp's offset of the step fills byte columns [my_sub * row bytes, ...) of the tile rows
            const uint32_t a_base = smem_u32(a_ring) + stage * uint32_t(C::kABytes);
#pragma unroll
            for (int e = 0; e < kEnt; ++e) {
              const uint32_t row = (en.rows[e / 4] >> (8 * (e % 4))) & 0xFFu;
              uint32_t off = row * 128u + uint32_t(my_sub_offset + chunk * 16);
              off ^= ((off >> 7) & 7u) << 4;
              if (en.idx[e] >= 0) cp_async_16(a_base + off, feats_lane + size_t(en.idx[e]) * C::kARowBytes, 16u);
            }
            SPCONV_PROF_T(c2);
            // the group's last warp also brings the row masks of the step's offsets, one lane each
            const uint32_t word = en.blk;
            if (wg == kGroupWarps - 1 && lane <= int((word >> 5) & 7u)) {
              const size_t blk = size_t(sm->tile[word & 31u]) * size_t(kvol) + ((word >> (8 + 6 * lane)) & 63u);
              cp_async_16(smem_u32(&sm->stage_absent[stage][lane][0]), tile_absent + blk * 4, 16u);
            }
            cp_async_arrive_noinc(smem_u32(&sm->full_a[stage]));
            fetch(m + kIdxDepth, q[d]);
            SPCONV_PROF_T(c3);
            SPCONV_PROF_ADD(pc_wait, c0, c1); SPCONV_PROF_ADD(pc_copy, c1, c2); SPCONV_PROF_ADD(pc_rest, c2, c3);
            continue;
          }
          if (__any_sync(0xffffffffu, en.idx[0] >= 0)) {
            const uint32_t a_base = a_lane0 + stage * uint32_t(C::kABytes);
#pragma unroll
            for (int j = 0; j < kEPG; ++j) {
              const uint32_t row = (en.rows[j / 4] >> (8 * (j % 4))) & 0xFFu;
              uint32_t off = row * uint32_t(C::kASpan) + uint32_t(within);
              off ^= ((off >> 7) & uint32_t(C::kASpan / 16 - 1)) << 4;
              if (en.idx[j] >= 0) cp_async_16(a_base + off, feats_lane + size_t(en.idx[j]) * C::kARowBytes, 16u);
            }
          }
          SPCONV_PROF_T(c2);
          if (mask_thread) cp_async_16(smem_u32(&sm->stage_absent[stage][0][0]), tile_absent + size_t(en.blk) * 4, 16u);
          cp_async_arrive_noinc(smem_u32(&sm->full_a[stage]));
          fetch(m + kIdxDepth, q[d]);
          SPCONV_PROF_T(c3);
          SPCONV_PROF_ADD(pc_wait, c0, c1); SPCONV_PROF_ADD(pc_copy, c1, c2); SPCONV_PROF_ADD(pc_rest, c2, c3);
        }
      }
#ifdef SPCONV_TC_PROFILE
      if (tid == 0 && round == 0 && timeline != nullptr) {
        unsigned long long* tl = timeline + size_t(blockIdx.x) * 16;
        tl[14] = pc_wait; tl[15] = pc_copy + pc_rest;
      }
#endif
      a_step += uint32_t(n_own);
      if (tid == 0 && round == 0) stamp(3);
      run_epilogue(ok);
    } else if (warp < C::kProducerWarps + C::kPipes) {
      // =============================== MMA issuers ===============================
      // Issuing a step costs its warp several hundred cycles around the MMAs themselves (barrier polls,
      // commits) during which the tensor pipe would idle, so the CTA runs kPipes pipelines side by side: every
      // tile belongs to one of them (bits 14+ of the step word), whose issuer warp takes the tile's steps in
      // offset order, and one warp's waits overlap the other's MMAs.  The pipelines share nothing but TMEM and
      // the tensor pipe: each has its own A ring and its own ring of W slots with their barriers (a pipeline loads
      // W_k only for the offsets its tiles have).  That matters beyond speed: a parity wait is only meaningful for
      // a waiter that sees every phase of its barrier, and a warp that skips another pipeline's steps on a shared
      // ring does not.
      // The whole warp runs the loop in lockstep and only the tcgen05 instructions are predicated on the
      // elected lane: ring positions, phases and descriptors then stay warp-uniform values (uniform registers,
      // which is where the MMA instruction takes its operands from) instead of one diverged lane's private ones.
      {
        const uint32_t me = uint32_t(warp - C::kProducerWarps);
        const bool leader = elect_one();
        bool ok = true;
        constexpr uint32_t kAHi = uint32_t(make_smem_desc_hi(8u * C::kASpan, layout_type_of_span(C::kASpan)));
        constexpr uint32_t kBHi = uint32_t(make_smem_desc_hi(8u * C::kWSpan, layout_type_of_span(C::kWSpan)));
        const uint32_t a_lo0 = make_smem_desc_lo(smem_u32(a_ring + me * uint32_t(C::kStagesPer) * C::kABytes), 16u);
        const uint32_t w_first = C::kSharedW ? 0u : me * uint32_t(C::kWInStage ? C::kStagesPer : C::kWStagesPer);   // first W slot this issuer uses
        const uint32_t b_lo0 = make_smem_desc_lo(smem_u32(w_ring + w_first * C::kWSlotBytes), uint32_t(C::kWPanelBytes));
        const uint32_t full_a0 = smem_u32(&sm->full_a[me * C::kStagesPer]), empty_a0 = smem_u32(&sm->empty_a[me * C::kStagesPer]);
        const uint32_t full_w0 = smem_u32(&sm->full_w[w_first]), empty_w0 = smem_u32(&sm->empty_w[w_first]);
        // Private W slots: the issuer walks its own steps.  Shared W slots: it walks all steps, because it has to
        // wait for and release the slot of every offset group, also of groups none of its tiles take part in (its
        // arrival for one use of a slot can then never overtake another issuer's arrival for the use before);
        // a group ends where the offset of the next step differs.
        const uint16_t* own = own_steps + me * (kvol * C::kMaxTilesInTmem);
        const int n_walk = C::kSharedW ? n_steps : sm->n_own[me];
        auto step_at = [&](int m) { return uint32_t(C::kSharedW ? steps[m] : steps[own[m]]); };
        uint32_t e_next = (!C::kGrouped && n_walk > 0) ? step_at(0) : 0u;
        bool w_known = false;     // (shared slots) this issuer has already seen the current group's slot loaded
        [[maybe_unused]] long long mc_wait = 0, mc_work = 0, mc_all = 0;
        SPCONV_PROF_T(mbegin);
        if constexpr (C::kGrouped) {
          // One step = up to kSub offsets of one tile: for each, CIN / 16 MMAs on its byte columns of the A tile with
          // its own W_k (sub-slot of the stage) and its own row mask.
          const uint32_t* gsteps = reinterpret_cast<const uint32_t*>(step_blk) + me * (kvol * C::kMaxTilesInTmem);
          uint32_t word_next = n_walk > 0 ? gsteps[0] : 0u;
          for (int m = 0; m < n_walk; ++m) {
            const uint32_t word = word_next;
            word_next = gsteps[m + 1 < n_walk ? m + 1 : m];
            const uint32_t g = word & 31u;
            const int n_sub = int((word >> 5) & 7u) + 1;
            SPCONV_PROF_T(m0);
            ok = mbar_wait(full_a0 + mma_stage * 8u, mma_phase, wctx, (4u << 24) | uint32_t(m));
            if (!ok) break;
            SPCONV_PROF_T(m1);
            fence_proxy_async();
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + mma_stage * uint32_t(C::kABytes >> 4);
            const uint32_t b_lo = b_lo0 + mma_stage * uint32_t(C::kWSlotBytes >> 4);
            const uint32_t d_tmem = tmem_base + g * COUT;
            uint4 absent[C::kSub];
#pragma unroll
            for (int sidx = 0; sidx < C::kSub; ++sidx)
              asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(absent[sidx].x), "=r"(absent[sidx].y), "=r"(absent[sidx].z), "=r"(absent[sidx].w) : "r"(smem_u32(&sm->stage_absent[me * C::kStagesPer + mma_stage][sidx][0])) : "memory");
            if (leader) {
#pragma unroll
              for (int sidx = 0; sidx < C::kSub; ++sidx) {
                if (sidx >= n_sub) break;
#pragma unroll
                for (int j = 0; j < C::kKSteps; ++j) {
                  const uint32_t a_off = uint32_t(C::sub_offset(sidx) + j * 32) >> 4;
                  const uint32_t b_off = (uint32_t(sidx) * C::kWBytes + uint32_t(j) * 16u * C::kWSpan) >> 4;
                  umma_f16_masked(d_tmem, a_lo + a_off, kAHi, b_lo + b_off, kBHi, idesc, absent[sidx], 1u);
                }
              }
              umma_commit(empty_a0 + mma_stage * 8u);   // the stage, rows and weights, is free once these MMAs have read it
            }
            if (++mma_stage == uint32_t(C::kStagesPer)) { mma_stage = 0; mma_phase ^= 1u; }
            SPCONV_PROF_T(m2);
            SPCONV_PROF_ADD(mc_wait, m0, m1); SPCONV_PROF_ADD(mc_work, m1, m2);
          }
        } else
        for (int m = 0; m < n_walk; ++m) {
          const uint32_t e = e_next;
          e_next = step_at(m + 1 < n_walk ? m + 1 : m);
          const uint32_t g = e & 31u;
          if constexpr (C::kSharedW) {
            const bool group_ends = m + 1 == n_walk || ((e_next >> 5) & 127u) != ((e >> 5) & 127u);
            const bool mine = (e >> kStepIssuerShift) == me;
            if ((mine || group_ends) && !w_known) {
              ok = mbar_wait(full_w0 + mma_wslot * 8u, mma_wphase, wctx, (3u << 24) | uint32_t(m));
              if (!ok) break;
              w_known = true;
            }
            if (!mine) {
              if (group_ends) {
                if (leader) umma_commit(empty_w0 + mma_wslot * 8u);   // covers this issuer's MMAs of the group (possibly none)
                if (++mma_wslot == uint32_t(C::kWStagesPer)) { mma_wslot = 0; mma_wphase ^= 1u; }
                w_known = false;
              }
              continue;
            }
          }
          const bool w_done = C::kWInStage ? false : C::kSharedW ? (m + 1 == n_walk || ((e_next >> 5) & 127u) != ((e >> 5) & 127u)) : (e & kStepLast) != 0u;
          SPCONV_PROF_T(m0);
          if (!C::kSharedW && !C::kWInStage && (e & kStepFirst)) {
            ok = mbar_wait(full_w0 + mma_wslot * 8u, mma_wphase, wctx, (3u << 24) | uint32_t(m));
            if (!ok) break;
          }
          ok = mbar_wait(full_a0 + mma_stage * 8u, mma_phase, wctx, (4u << 24) | uint32_t(m));
          if (!ok) break;
          SPCONV_PROF_T(m1);
          fence_proxy_async();   // the rows were written by cp.async; the MMA reads them through the async proxy
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + mma_stage * uint32_t(C::kABytes >> 4);
          const uint32_t b_lo = b_lo0 + (C::kWInStage ? mma_stage : mma_wslot) * uint32_t(C::kWBytes >> 4);   // kWInStage: the stage's own W slot
          const uint32_t d_tmem = tmem_base + g * COUT;
          uint4 absent;
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(absent.x), "=r"(absent.y), "=r"(absent.z), "=r"(absent.w) : "r"(smem_u32(&sm->stage_absent[me * C::kStagesPer + mma_stage][0][0])) : "memory");
          if (leader) {
#pragma unroll
            for (int j = 0; j < C::kKSteps; ++j) {
              const uint32_t a_off = (uint32_t((j * 32) / C::kASpan) * C::kAPanelBytes + uint32_t((j * 32) % C::kASpan)) >> 4;
              const uint32_t b_off = (uint32_t(j) * 16u * C::kWSpan) >> 4;
              umma_f16_masked(d_tmem, a_lo + a_off, kAHi, b_lo + b_off, kBHi, idesc, absent, 1u);
            }
            umma_commit(empty_a0 + mma_stage * 8u);   // the stage is free once these MMAs have read it
            if (w_done) umma_commit(empty_w0 + mma_wslot * 8u);   // and so is the W slot after the offset's last step
          }
          if (++mma_stage == uint32_t(C::kStagesPer)) { mma_stage = 0; mma_phase ^= 1u; }
          if (w_done) {
            if (++mma_wslot == uint32_t(C::kWStagesPer)) { mma_wslot = 0; mma_wphase ^= 1u; }
            w_known = false;
          }
          SPCONV_PROF_T(m2);
          SPCONV_PROF_ADD(mc_wait, m0, m1); SPCONV_PROF_ADD(mc_work, m1, m2);
        }
#ifdef SPCONV_TC_PROFILE
        if (leader && me == 0 && round == 0 && timeline != nullptr) {
          SPCONV_PROF_T(mend);
          SPCONV_PROF_ADD(mc_all, mbegin, mend);
          unsigned long long* tl = timeline + size_t(blockIdx.x) * 16;
          tl[8] = (unsigned long long)(sm->n_own[0]) | ((unsigned long long)(sm->n_own[C::kPipes - 1]) << 32);
          tl[9] = mc_wait; tl[10] = mc_work; tl[12] = mc_all;
        }
#endif
        if (leader && ok) umma_commit(smem_u32(&sm->accum_full));   // every issuer arrives, with or without steps
        if (leader && me == 0 && round == 0) stamp(6);
        __syncwarp();
        run_epilogue(ok);
      }
    } else {
      // =============================== W loaders (TMA) ===============================
      // One warp per pipeline: W_k for every offset the pipeline's tiles have, into the pipeline's own slots.
      bool loader_ok = true;
      if (lane == 0) {
        const uint32_t me = uint32_t(warp - C::kProducerWarps - C::kPipes);
        const uint16_t* own = own_steps + me * (kvol * C::kMaxTilesInTmem);
        const int n_walk = C::kSharedW ? n_steps : sm->n_own[me];
        bool ok = true;
        int k_prev = -1;
        [[maybe_unused]] long long wc_wait = 0;
        if constexpr (C::kGrouped) {
          const uint32_t* gsteps = reinterpret_cast<const uint32_t*>(step_blk) + me * (kvol * C::kMaxTilesInTmem);
          for (int m = 0; m < n_walk && ok; ++m) {
            const uint32_t word = gsteps[m];
            const int n_sub = int((word >> 5) & 7u) + 1;
            const uint32_t wslot = me * uint32_t(C::kStagesPer) + w_group % uint32_t(C::kStagesPer), wuse = w_group / uint32_t(C::kStagesPer);
            ok = mbar_wait(smem_u32(&sm->empty_a[wslot]), (wuse & 1u) ^ 1u, wctx, (5u << 24) | uint32_t(m));
            if (!ok) break;
            const uint32_t bar = smem_u32(&sm->full_a[wslot]);
            const uint32_t dst = smem_u32(w_ring + wslot * C::kWSlotBytes);
            if (withhold_first_w && blockIdx.x == 0 && me == 0 && m == 0 && round == 0) { ++w_group; continue; }   // test hook, see launch()
            mbar_arrive_expect_tx(bar, uint32_t(n_sub * C::kWBytesRaw));
            for (int sidx = 0; sidx < n_sub; ++sidx) {
              const int k = int((word >> (8 + 6 * sidx)) & 63u);
#pragma unroll
              for (int p = 0; p < C::kWPanels; ++p) tma_load_2d(dst + sidx * C::kWBytes + p * C::kWPanelBytes, &w_map, bar, p * 64, k * CIN);
            }
            ++w_group;
          }
        } else
        for (int m = 0; m < n_walk && ok; ++m) {
          const uint32_t e = C::kSharedW ? steps[m] : steps[own[m]];
          const int k = (e >> 5) & 127u;
          const bool group_starts = C::kWInStage ? true : C::kSharedW ? k != k_prev : (e & kStepFirst) != 0u;
          k_prev = k;
          if (!group_starts) continue;
          SPCONV_PROF_T(w0);
          // kWInStage: W_k goes into the stage of the step itself, behind the same two barriers as its rows
          const uint32_t depth = uint32_t(C::kWInStage ? C::kStagesPer : C::kWStagesPer);
          const uint32_t wslot = (C::kSharedW ? 0u : me * depth) + w_group % depth, wuse = w_group / depth;
          ok = mbar_wait(smem_u32(C::kWInStage ? &sm->empty_a[wslot] : &sm->empty_w[wslot]), (wuse & 1u) ^ 1u, wctx, (5u << 24) | uint32_t(m));
          if (!ok) break;
          SPCONV_PROF_T(w1);
          SPCONV_PROF_ADD(wc_wait, w0, w1);
          const uint32_t bar = smem_u32(C::kWInStage ? &sm->full_a[wslot] : &sm->full_w[wslot]);
          const uint32_t dst = smem_u32(w_ring + wslot * C::kWSlotBytes);
          if (withhold_first_w && blockIdx.x == 0 && me == 0 && m == 0 && round == 0) { ++w_group; continue; }   // test hook, see launch()
          mbar_arrive_expect_tx(bar, uint32_t(C::kWBytesRaw));
#pragma unroll
          for (int p = 0; p < C::kWPanels; ++p) tma_load_2d(dst + p * C::kWPanelBytes, &w_map, bar, p * 64, k * CIN);
          ++w_group;
        }
        if (me == 0 && round == 0) stamp(7);
#ifdef SPCONV_TC_PROFILE
        if (me == 0 && round == 0 && timeline != nullptr) timeline[size_t(blockIdx.x) * 16 + 13] = wc_wait;
#endif
        loader_ok = ok;
      }
      loader_ok = __shfl_sync(0xffffffffu, int(loader_ok), 0) != 0;
      run_epilogue(loader_ok);
    }
    __syncthreads();  // tiles, masks, steps and the accumulators are reused by the next round
    if (sm->abort_flag) break;
  }

  // ---- teardown
  if (sm->abort_flag) {
    // A wait gave up.  Bulk copies already issued still write into this CTA's shared memory and signal its
    // barriers; they depend on nothing the CTA does, so give them time to land before the CTA exits.
    for (int i = 0; i < 100; ++i) __nanosleep(1000);
  }
  if (warp >= C::kProducerWarps && warp < C::kProducerWarps + C::kPipes && sm->abort_flag) {
    // Give MMAs that may still be in flight a bounded chance to finish before TMEM is released (the commit
    // has to come from the lane that issued them).
    __syncwarp();
    if (elect_one()) umma_commit(smem_u32(&sm->drain));
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
      if (mbar_try_wait(smem_u32(&sm->drain), 0u)) break;
      if ((it & 63u) == 63u && global_timer_ns() - t0 > wait_limit_ns) break;
    }
  }
  if (warp < C::kProducerWarps) cp_async_wait_all();
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && sm->abort_flag) atomicOr(status, kDevPipeTimeout);
  if (warp == C::kProducerWarps) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sm->tmem_base), "r"(tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ host side
unsigned long long* g_timeline = nullptr;  // diagnostics only, see set_forward_tc_timeline

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode_fn() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
    (void)cudaGetLastError();
  });
  return fn;
}

// Test hook: SPCONV_TC_MAX_CTAS=<n> caps the grid so that small inputs exercise many tiles per CTA and
// several rounds.  Unset (or 0) means one CTA per SM.
int max_ctas_override() {
  static const int v = [] {
    const char* e = std::getenv("SPCONV_TC_MAX_CTAS");
    return e != nullptr ? std::atoi(e) : 0;
  }();
  return v;
}

// Test hook for the kernel's give-up path (spconv_test_hook, SPCONV_HOOK_PIPE_WAIT_LIMIT_US): a positive value
// shortens the wall-time bound of every wait to that many microseconds and makes CTA 0's first W loader withhold the
// weights of its first step, so that the wait for that step's stage runs out, the CTA gives up, frees what it holds
// and the launch reports SPCONV_ERR_PIPE_TIMEOUT through the status word -- nothing faults and nothing waits without
// a bound.  0: the ordinary limit, nothing withheld.
std::atomic<long long> g_test_wait_limit_us{0};
long long test_wait_limit_us() { return g_test_wait_limit_us.load(std::memory_order_relaxed); }

template <int CIN, int COUT, bool GROUPED>
size_t smem_bytes_for(int kvol) {
  using C = Cfg<CIN, COUT, GROUPED>;
  return 1024 + size_t(C::kStages) * C::kABytes + size_t(C::kWStages) * C::kWSlotBytes + sizeof(Smem) +
         size_t(kvol) * C::kMaxTilesInTmem * (sizeof(uint16_t) * (1 + C::kPipes) + sizeof(uint32_t)) + 64;
}

template <int CIN, int COUT, bool GROUPED>
int launch(const void* feats, const void* w, const spconv_kmap* km, void* out, spconv_dtype_t dtype, cudaStream_t stream, bool strict_order) {
  using C = Cfg<CIN, COUT, GROUPED>;
  EncodeFn encode = get_encode_fn();
  if (!encode) return SPCONV_ERR_CUDA;
  const int kvol = km->kvol;
  const CUtensorMapDataType dt = dtype == SPCONV_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
  const cuuint32_t estr[2] = {1, 1};
  auto swizzle_of = [](int span) {
    return span == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : span == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  };

  // W as a 2-D tensor [kvol * CIN rows][COUT columns]; one box = one W_k panel of <= 64 columns.  The encoded
  // map of the last weights pointer is kept per thread and layer shape: a network calls the same layer again
  // and again, and the encoding is a driver call on the launch path.
  struct CachedMap { const void* w = nullptr; int kvol = 0; int dt = -1; CUtensorMap map; };
  thread_local CachedMap cached;
  if (cached.w != w || cached.kvol != kvol || cached.dt != int(dtype)) {
    CUtensorMap& wmap = cached.map;
    const cuuint64_t dims[2] = {cuuint64_t(COUT), cuuint64_t(kvol) * CIN};
    const cuuint64_t strides[1] = {cuuint64_t(COUT) * 2};
    const cuuint32_t box[2] = {cuuint32_t(COUT < 64 ? COUT : 64), cuuint32_t(CIN)};
    if (encode(&wmap, dt, 2, const_cast<void*>(w), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(C::kWSpan),
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      cached.w = nullptr;
      return SPCONV_ERR_CUDA;
    }
    cached.w = w; cached.kvol = kvol; cached.dt = int(dtype);
  }
  const CUtensorMap& wmap = cached.map;
  static int num_sms[64] = {0};
  const int dev = km->device;
  if (dev < 0 || dev >= 64) return SPCONV_ERR_INVALID_ARG;
  if (num_sms[dev] == 0) {
    int v = 0;
    SPCONV_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev));
    num_sms[dev] = v;
  }
  const size_t smem = smem_bytes_for<CIN, COUT, GROUPED>(kvol);
  if (smem > size_t(kMaxSmem)) return SPCONV_ERR_TOO_LARGE;
  static bool attr_set[64] = {false};
  if (!attr_set[dev]) {
    SPCONV_CUDA_TRY(cudaFuncSetAttribute(k_forward_tc<CIN, COUT, GROUPED>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
    attr_set[dev] = true;
  }
  const int n_tiles = km->n_tiles;
  const int max_ctas = max_ctas_override() > 0 ? max_ctas_override() : num_sms[dev];
  const int grid = n_tiles < max_ctas ? n_tiles : max_ctas;

  // Instruction descriptor: fp32 accumulate, A K-major, B MN-major, M = 128, N = COUT.
  const uint32_t fmt = dtype == SPCONV_BF16 ? 1u : 0u;
  const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | (0u << 15) | (1u << 16) | (uint32_t(COUT >> 3) << 17) |
                         (uint32_t(kTileRows >> 4) << 24);

  // Tiles per CTA and round: as few rounds as TMEM allows, tiles spread evenly over them.
  const int rounds = (n_tiles + grid * C::kMaxTilesInTmem - 1) / (grid * C::kMaxTilesInTmem);
  const int G = (n_tiles + grid * rounds - 1) / (grid * rounds);
  uint32_t cols = 32;
  while (cols < uint32_t(G * COUT)) cols <<= 1;

  // Input rows the kernel requests into L2 up front, in 128-byte lines: all of them up to 32 MB.
  const long long feat_bytes = (long long)km->n_in * C::kARowBytes;
  const long long feat_lines = std::min<long long>(feat_bytes, 32ll << 20) / 128;
  const unsigned long long wait_limit_ns = test_wait_limit_us() > 0 ? (unsigned long long)test_wait_limit_us() * 1000ull : kWaitLimitNs;
  const int withhold_first_w = test_wait_limit_us() > 0 ? 1 : 0;

  cudaLaunchConfig_t config = {};
  config.gridDim = dim3(unsigned(grid));
  config.blockDim = dim3(unsigned(C::kThreads));
  // Always the SM's whole shared memory, whatever the layout needs: one CTA per SM by construction.  The kernel
  // allocates TMEM and lets its dependents start before it waits for its predecessors, so a second resident CTA (of
  // this or of the next grid) could hold TMEM columns that a CTA waiting in tcgen05.alloc needs.
  config.dynamicSmemBytes = kMaxSmem;
  config.stream = stream;
  cudaLaunchAttribute attribute[1];
  attribute[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see the kernel's griddepcontrol instructions
  attribute[0].val.programmaticStreamSerializationAllowed = 1;
  config.attrs = attribute;
  config.numAttrs = 1;
  SPCONV_CUDA_TRY(cudaLaunchKernelEx(&config, k_forward_tc<CIN, COUT, GROUPED>, wmap, static_cast<const uint8_t*>(feats), km->d.tile_nbr,
                                     km->d.tile_crow, km->d.tile_rows, km->d.tile_mask, km->d.tile_absent, km->d.sorted_tiles,
                                     static_cast<uint8_t*>(out), n_tiles, kvol, km->mask_words, G, rounds, cols, idesc,
                                     dtype == SPCONV_BF16 ? 1 : 0, km->d.status, g_timeline, feat_lines, strict_order ? 1 : 0, wait_limit_ns,
                                     withhold_first_w));
  SPCONV_CUDA_TRY(cudaGetLastError());
  return SPCONV_OK;
}

template <int CIN>
int dispatch_cout(const void* feats, const void* w, const spconv_kmap* km, void* out, int cout, spconv_dtype_t dtype,
                  cudaStream_t stream, bool strict_order, bool single) {
  if (single) {
    switch (cout) {
      case 16: return launch<CIN, 16, false>(feats, w, km, out, dtype, stream, strict_order);
      case 32: return launch<CIN, 32, false>(feats, w, km, out, dtype, stream, strict_order);
      case 64: return launch<CIN, 64, false>(feats, w, km, out, dtype, stream, strict_order);
      case 128: return launch<CIN, 128, false>(feats, w, km, out, dtype, stream, strict_order);
    }
    return SPCONV_ERR_INVALID_ARG;
  }
  switch (cout) {
    case 16: return (grouped_shape(CIN, 16) && km->kvol <= 32) ? launch<CIN, 16, grouped_shape(CIN, 16)>(feats, w, km, out, dtype, stream, strict_order)
                                                                  : launch<CIN, 16, false>(feats, w, km, out, dtype, stream, strict_order);
    case 32: return (grouped_shape(CIN, 32) && km->kvol <= 32) ? launch<CIN, 32, grouped_shape(CIN, 32)>(feats, w, km, out, dtype, stream, strict_order)
                                                                  : launch<CIN, 32, false>(feats, w, km, out, dtype, stream, strict_order);
    case 64: return (grouped_shape(CIN, 64) && km->kvol <= 32) ? launch<CIN, 64, grouped_shape(CIN, 64)>(feats, w, km, out, dtype, stream, strict_order)
                                                                  : launch<CIN, 64, false>(feats, w, km, out, dtype, stream, strict_order);
    case 128: return (grouped_shape(CIN, 128) && km->kvol <= 32) ? launch<CIN, 128, grouped_shape(CIN, 128)>(feats, w, km, out, dtype, stream, strict_order)
                                                                  : launch<CIN, 128, false>(feats, w, km, out, dtype, stream, strict_order);
  }
  return SPCONV_ERR_INVALID_ARG;
}

}  // namespace

void set_forward_tc_test_wait_limit_us(long long us) { g_test_wait_limit_us.store(us > 0 ? us : 0, std::memory_order_relaxed); }

// Diagnostics: install (or clear, with nullptr) a device buffer of 16 * gridDim uint64 that the
// tensor-core kernel fills with per-CTA globaltimer stamps: 0 start, 1 set-up done, 2 step list built,
// 3 gather issue done, 4 accumulators complete, 5 epilogue done, 6 MMA issue done, 7 W loads issued (first round).
void set_forward_tc_timeline(unsigned long long* buf) { g_timeline = buf; }

bool forward_tc_supported(int cin, int cout, spconv_dtype_t dtype) {
  auto okc = [](int c) { return c == 16 || c == 32 || c == 64 || c == 128; };
  return (dtype == SPCONV_F16 || dtype == SPCONV_BF16) && okc(cin) && okc(cout);
}

int forward_tc(const void* feats, const void* w, const spconv_kmap* km, void* out, int cin, int cout,
               spconv_dtype_t dtype, cudaStream_t stream, bool strict_order, bool one_offset_per_step) {
  if (!forward_tc_supported(cin, cout, dtype) || km->kvol > 128) return SPCONV_ERR_INVALID_ARG;
  if (km->n_out == 0) return SPCONV_OK;
  switch (cin) {
    case 16: return dispatch_cout<16>(feats, w, km, out, cout, dtype, stream, strict_order, one_offset_per_step);
    case 32: return dispatch_cout<32>(feats, w, km, out, cout, dtype, stream, strict_order, one_offset_per_step);
    case 64: return dispatch_cout<64>(feats, w, km, out, cout, dtype, stream, strict_order, one_offset_per_step);
    case 128: return dispatch_cout<128>(feats, w, km, out, cout, dtype, stream, strict_order, one_offset_per_step);
  }
  return SPCONV_ERR_INVALID_ARG;
}

}  // namespace spconv
