// QK4PV8 prefill (Algorithm 1 lines 6-20) for sm_100a.
//
// A work item is one 128-row query tile of one q head; its KV blocks (128 keys) are visited from the last
// visible block down to block 0 (Section 4.1).  One persistent CTA per SM walks a static list of work items
// (struct TileWalk) and keeps its pipeline running across item boundaries.  Roles (512 threads):
//   warp 0       producer: K codes (tensor map, 64B swizzle), K scale factors and Delta_S (bulk copies)
//                and V (tensor map, 128B swizzle) into rings of 4 (K) and 3 (V) stages; in the paged
//                variant (template parameter PAGED, entry point mpfa_prefill_paged) every tile half is
//                one bulk copy of a 64-token page slab, found through the page table;
//   warp 2       paged variant only: re-tiles the pages' row-major K scales for tcgen05.cp and un-swizzles
//                their Delta_S rows (idle otherwise; it also owns the tensor-memory allocation);
//   warp 1       Q K^T issuer: per block a rank-one BF16 MMA seeds S with 1 x Delta_S
//                (Eq. 11) and two block-scaled FP4 MMAs (K = 64 each) accumulate Q K^T into
//                the same TMEM columns;
//   warp 3       P V issuer: four FP8 MMAs per block (A = P_hat from TMEM, B = V from
//                shared memory, MN-major) accumulate P V into O;
//   warps 4-7    softmax of the even-numbered blocks of the traversal;
//   warps 8-11   softmax of the odd-numbered blocks.  One thread per row:
//                the whole 128-column row is read into registers once; mask, row maximum,
//                running maximum handed from one group to the other through shared memory
//                (only the maximum is loop-carried, so the exponentials of block t overlap
//                the maximum pass and exponentials of block t+1), 2^(lam S - lam m), row sum
//                from the unquantized P, P -> E4M3 at the fixed scale 448 written to its own
//                32 TMEM columns (Algorithm 1 lines 11-14).  The score buffer is handed back to
//                the MMA warp as soon as the row is in registers, so Q K^T runs two blocks
//                ahead of P V and a softmax group never waits for its next scores;
//   warps 12-15  correction + epilogue.  Even blocks accumulate into O0, odd blocks into O1,
//                so the rescale of an accumulator (Eq. 6, by alpha_t * alpha_{t-1}, only when
//                some row's maximum moved) has a whole block of slack instead of sitting
//                between two dependent MMAs; the epilogue adds the two accumulators
//                (the older one times the last alpha) and writes O / (448 l) * v_scale as BF16.
// Tensor memory (512 columns): S [0,128) O0 [128,256) O1 [256,384), P_hat0 [384,416)
// P_hat1 [416,448), scale factors of two query tiles [448,464) and of two K blocks [464,472) [472,480).
// Register budget is moved between the roles with setmaxnreg (72 for warps 0-3, 168 for the softmax warps,
// 104 for the correction warps, whose epilogue holds two accumulator chunks at once).
// Template parameter EW: the compensation-placement ablation (mpfa_prefill_variant): no seed MMA, Delta_S added
// element by element by the softmax threads.
//
// Every mbarrier wait is bounded; on expiry the CTA raises MPFA_DEV_TIMEOUT in
// *device_status, all roles leave their loops, outstanding TMA copies are drained and
// tensor memory is released.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "prefill_common.cuh"

namespace mpfa {
namespace {

constexpr int KSTAGES = 4;
constexpr int VSTAGES = 3;
constexpr int NTHREADS = 512;
// setmaxnreg only moves registers inside the pool the CTA got at launch (512 threads x the 128 registers of the
// launch bound); a request beyond the pool would block forever, so the split is checked here.
#ifndef MPFA_REGS_UTIL_PAGED
#define MPFA_REGS_UTIL_PAGED 64
#define MPFA_REGS_CORR_PAGED 112
#endif
#ifndef MPFA_REGS_SOFTMAX
#define MPFA_REGS_SOFTMAX 168
#define MPFA_REGS_UTIL 72
#define MPFA_REGS_CORR 104
#endif
constexpr int REGS_SOFTMAX = MPFA_REGS_SOFTMAX;
// measured (16K / 64K TFLOPS, utility / softmax / correction): 56/168/120 1325 / 1418, 72/168/104 1339 / 1447,
// 72/160/112 1335 / 1447, 64/168/112 1307 / 1423, 80/160/104 1310 / 1435, 96/160/88 1302 / 1427, 152 for the softmax
// warps 1243 / 1318 (their row spills); the paged variant's producer and re-tiling warps need a few more (measured on the
// config-2 shape from pages: 56/120 1217, 64/112 1223, 72/104 1211, 80/96 1172, 88/88 1173 TFLOPS)
template <bool PAGED> constexpr int REGS_UTIL = PAGED ? MPFA_REGS_UTIL_PAGED : MPFA_REGS_UTIL;
template <bool PAGED> constexpr int REGS_CORR = PAGED ? MPFA_REGS_CORR_PAGED : MPFA_REGS_CORR;
static_assert(4 * REGS_UTIL<false> + 8 * REGS_SOFTMAX + 4 * REGS_CORR<false> <= 16 * 128, "register pool");
static_assert(4 * REGS_UTIL<true> + 8 * REGS_SOFTMAX + 4 * REGS_CORR<true> <= 16 * 128, "register pool");
// the utility and correction warps give registers back (setmaxnreg.dec: the target must not exceed the 128 of the
// launch, or the instruction is illegal), the softmax warps take them (setmaxnreg.inc: not below 128)
static_assert(REGS_UTIL<false> <= 128 && REGS_UTIL<true> <= 128 && REGS_CORR<false> <= 128 && REGS_CORR<true> <= 128 &&
              REGS_UTIL<false> >= 24 && REGS_UTIL<true> >= 24 && REGS_CORR<false> >= 24 && REGS_CORR<true> >= 24 &&
              REGS_SOFTMAX >= 128 && REGS_SOFTMAX <= 255, "setmaxnreg direction");
static_assert(REGS_SOFTMAX % 8 == 0 && REGS_UTIL<false> % 8 == 0 && REGS_CORR<false> % 8 == 0 && REGS_UTIL<true> % 8 == 0 &&
              REGS_CORR<true> % 8 == 0, "setmaxnreg granularity");

enum {
  BAR_Q_FULL = 0,                       // [2] query tile of work item i in buffer i & 1
  BAR_Q_EMPTY = 2,                      // [2] every Q K^T MMA of that work item has completed
  BAR_K_FULL = 4,
  BAR_K_EMPTY = BAR_K_FULL + KSTAGES,
  BAR_V_FULL = BAR_K_EMPTY + KSTAGES,
  BAR_V_EMPTY = BAR_V_FULL + VSTAGES,
  BAR_S_FULL = BAR_V_EMPTY + VSTAGES,   // [2] scores of block t in TMEM (one buffer, one barrier per
                                        //     softmax group so that each group's first wait is on phase 0)
  BAR_S_EMPTY = BAR_S_FULL + 2,         // scores read into registers, buffer free for block t+1
  BAR_P_FULL = BAR_S_EMPTY + 1,         // [2] P_hat of block t written
  BAR_P_EMPTY = BAR_P_FULL + 2,         // [2] P V of block t has consumed P_hat
  BAR_M_FULL = BAR_P_EMPTY + 2,         // [2] running maximum and alpha of block t published
  BAR_O_FULL = BAR_M_FULL + 2,          // [2] P V of block t accumulated into O[t & 1]
  BAR_O_READY = BAR_O_FULL + 2,         // [2] O[t & 1] rescaled for block t
  BAR_L_FULL = BAR_O_READY + 2,         // [4] row sums of the u-th item that has KV blocks (T > 0), slot u & 3.  The
                                        //     softmax warps can be at most three (one-block) such items ahead of the
                                        //     epilogue - P_hat of block c needs P V of block c-2, which needs the
                                        //     correction warps - so a slot is never two phases ahead of its reader.
                                        //     Items without blocks stay out of the ring: nothing bounds how many of
                                        //     them the softmax warps could run through
  BAR_O_FREE = BAR_L_FULL + 4,          // the epilogue has read both accumulators (phase = items with T > 0)
  BAR_SF_READY = BAR_O_FREE + 1,        // [KSTAGES] paged source only: scales and Delta_S of the stage re-tiled
  NUM_BARS = BAR_SF_READY + KSTAGES
};
static_assert(NUM_BARS <= 64, "barrier table");
// Shared-memory layout.  PVK selects the operands of the second MMA (mpfa_prefill_variant): 0 = the method (FP8);
// 1 = the NVFP4 + BF16 precision assignment: V tiles are BF16 (32 KB, three stages), P is handed to the second MMA
// through shared memory as a K-major BF16 A operand (2 x 32 KB), and the K ring has two stages to make room;
// 2 = the NVFP4 + NVFP4 assignment: V tiles are channel-major FP4 (8 KB + 1 KB of block scales), P goes through
// shared memory as a K-major FP4 A operand (2 x 8 KB) with its block scales (2 x 1 KB).
template <int PVK>
struct Lay {
  static constexpr bool PVB = PVK == 1, PV4 = PVK == 2;
  // ring depths measured on the product kernel (16K / 64K TFLOPS, K / V stages): 4/3 1340 / 1446, 6/3 1342 / 1452, 4/4
  // 1325 / 1464, 3/3 1329 / 1450, 2/3 within 1 % of 4/3, but 4/2 and 3/2 894 / 822: a V stage is held from its load until
  // the P V MMA of its block, which the late hand-over of P-hat issues a block later.  The BF16 variant therefore gives
  // up K stages, not V stages, to make room for its 32 KB tiles.
  static constexpr int KST = PVB ? 2 : KSTAGES;
  static constexpr int VST = VSTAGES;
  static constexpr uint32_t V_BYTES = PVB ? 32768u : (PV4 ? 8192u : 16384u);
  static constexpr uint32_t OFF_Q = 0;                               // 2 tiles (the next tile's queries are prefetched)
  static constexpr uint32_t OFF_K = OFF_Q + 2 * 8192;
  static constexpr uint32_t OFF_V = OFF_K + KST * 8192;
  static constexpr uint32_t OFF_DELTA = OFF_V + VST * V_BYTES;
  static constexpr uint32_t OFF_ONES = OFF_DELTA + KST * 4096;
  static constexpr uint32_t OFF_SFQ = OFF_ONES + 4096;
  static constexpr uint32_t OFF_SFK = OFF_SFQ + 2 * 1024;
  static constexpr uint32_t OFF_ALPHA = OFF_SFK + KST * 1024;   // alpha[2][128]
  static constexpr uint32_t OFF_M = OFF_ALPHA + 2 * 128 * 4;        // running maximum after block t, [t & 1][128]
  static constexpr uint32_t OFF_L = OFF_M + 2 * 128 * 4;            // final (l, m) of the two softmax groups, [item & 3][2][2][128]
  static constexpr uint32_t OFF_BAR = OFF_L + 4 * 4 * 128 * 4;
  static constexpr uint32_t OFF_MISC = OFF_BAR + 64 * 8;            // tmem base, abort flag (NUM_BARS <= 64)
  // paged source only: per K stage the two pages' scale bytes (2 x 512) and Delta_S rows (2 x 128) as stored
  static constexpr uint32_t RAW_STAGE = 1280;
  static constexpr uint32_t OFF_RAW = (OFF_MISC + 16 + 127) & ~127u;
  static constexpr uint32_t OFF_PS = (OFF_MISC + 16 + 1023) & ~1023u;   // PVB / PV4 only: P of the two softmax groups
  static constexpr uint32_t PS_BYTES = PVB ? 32768u : 8192u;
  static constexpr uint32_t OFF_SFP = OFF_PS + 2 * PS_BYTES;            // PV4 only: block scales of P, [group][2 atoms]
  static constexpr uint32_t OFF_SFV = OFF_SFP + 2 * 1024;               // PV4 only: block scales of V, [stage][2 atoms]
  static constexpr uint32_t SMEM_BYTES =
      (PVB ? OFF_PS + 2 * PS_BYTES : (PV4 ? OFF_SFV + VST * 1024 : OFF_MISC + 16)) + 1024;   // + slack for the 1024-byte alignment
  static constexpr uint32_t SMEM_BYTES_PAGED = OFF_RAW + KST * RAW_STAGE + 1024;
};
static_assert(Lay<1>::SMEM_BYTES <= 227 * 1024 && Lay<2>::SMEM_BYTES <= 227 * 1024 && Lay<0>::SMEM_BYTES_PAGED <= 227 * 1024, "shared memory");

constexpr uint32_t TM_S = 0, TM_O0 = 128, TM_O1 = 256, TM_P0 = 384, TM_P1 = 416, TM_SFQ = 448 /* 2 x 8 */,
                   TM_SFK0 = 464, TM_SFK1 = 472;
// NVFP4 + NVFP4 variant only: block scales of P (per softmax group) and of V (per block parity)
constexpr uint32_t TM_SFP0 = 480, TM_SFP1 = 488, TM_SFV0 = 496, TM_SFV1 = 504;
constexpr uint32_t TMEM_COLS = 512;

// Optional timeline capture for tuning (compiled in only with -DMPFA_TRACE): one CTA records
// clock64() at fixed points of every role, [role][block][event].
#ifdef MPFA_TRACE
__device__ long long *g_trace = nullptr;
__device__ int g_trace_cta = 0;
#define TR_INIT() long long *tr_buf = ((int)blockIdx.x == g_trace_cta && lane == 0) ? g_trace : nullptr
#define TR(role, t, ev)                                                              \
  do {                                                                               \
    if (tr_buf && (t) < 256) tr_buf[((role) * 256 + (t)) * 8 + (ev)] = clock64();    \
  } while (0)
#else
#define TR_INIT() do {} while (0)
#define TR(role, t, ev) do {} while (0)
#endif

// One work item: a 128-row query tile of one q head.
struct Tile {
  int b, hq, hk, qt, row0, T;   // T: KV blocks to visit
  int nkv, nq;                  // keys and queries of this item's request
};

// The list of work items of this CTA.  Items are ordered by length (latest query tile first; all heads of a
// tile adjacent, so the G heads of a kv head stream the same K/V through L2 together) and dealt to the CTAs
// boustrophedon: round r goes 0..n-1, round r+1 goes n-1..0.  For a causal 16K problem on 148 CTAs the
// heaviest CTA gets 0.15 % more blocks than the mean (plain round-robin: 7 %).
struct TileWalk {
  int round;   // everything else is read from the kernel parameters (constant bank), not kept in registers
  __device__ __forceinline__ void init() { round = 0; }
  template <bool PAGED>
  __device__ __forceinline__ bool next(const PrefillParams &pp, const PagedSrc &pg, Tile &t) {
    const int c = (round & 1) ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x;
    const int i = round * (int)gridDim.x + c;
    ++round;
    if (i >= pp.n_items) return false;
    const int n_heads = pp.B * pp.H_q;
    t.qt = pp.nq_tiles - 1 - i / n_heads;
    const int h = i % n_heads;
    t.b = h / pp.H_q;
    t.hq = h % pp.H_q;
    t.hk = t.hq / (pp.H_q / pp.H_kv);
    t.row0 = t.qt * TILE;
    const int n_q = (PAGED && pg.q_lens) ? min(pg.q_lens[t.b], pp.N_q) : pp.N_q;
    const int last_row = min(n_q - 1, t.row0 + TILE - 1);
    // a length beyond what the page-table row can address is cut to it (no read past the row)
    const int n_kv = PAGED ? min(pg.seq_lens[t.b], pg.max_pages * 64) : pp.N_kv;
    t.nkv = n_kv;
    t.nq = n_q;
    const int last_key = pp.causal ? min(n_kv - 1, last_row + (n_kv - n_q)) : n_kv - 1;   // bottom-right aligned
    t.T = (last_key < 0 || (PAGED && t.row0 >= n_q)) ? 0 : last_key / TILE + 1;
    return true;
  }
};

// EW: ablation variant of Section 7.4 (compensation placement): Delta_S is not seeded by the BF16 MMA but
// loaded by the softmax warps and added to the scores element by element in FP32, before masking and the maximum.
// PVB: precision-assignment variant of Section 3.1 (NVFP4 Q K^T, BF16 P V): P = 2^(lam S - lam m) is rounded to BF16
// and handed to the second MMA through shared memory (K-major A operand), V is the BF16 input in the tile layout
// written by mpfa_pack_v_bf16, the second MMA is kind::f16 (eight K = 16 steps per block).
// PV4: the NVFP4 + NVFP4 assignment: q = 448 P is quantized per row and 16 keys (E4M3 block scale of max q, E2M1 codes
// of q * (6 / scale)) and written with its scales to shared memory; V is the channel-major FP4 operand of
// mpfa_quantize_v_fp4; the second MMA is kind::mxf4nvf4 block-scaled (two K = 64 steps per block).
template <bool PAGED, bool EW, int PVK = 0>
__global__ void __launch_bounds__(NTHREADS, 1)
prefill_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const PrefillParams p, const PagedSrc pg) {
  constexpr bool PVB = PVK == 1, PV4 = PVK == 2;
  static_assert(!(PVK != 0 && (PAGED || EW)), "the precision variants exist for contiguous operands with the seed MMA only");
  using L = Lay<PVK>;
  constexpr int KST = L::KST, VST = L::VST;
  constexpr uint32_t OFF_Q = L::OFF_Q, OFF_K = L::OFF_K, OFF_V = L::OFF_V, OFF_DELTA = L::OFF_DELTA, OFF_ONES = L::OFF_ONES,
                     OFF_SFQ = L::OFF_SFQ, OFF_SFK = L::OFF_SFK, OFF_M = L::OFF_M, OFF_L = L::OFF_L, OFF_BAR = L::OFF_BAR,
                     OFF_MISC = L::OFF_MISC, OFF_RAW = L::OFF_RAW, RAW_STAGE = L::RAW_STAGE, OFF_PS = L::OFF_PS,
                     V_BYTES = L::V_BYTES, PS_BYTES = L::PS_BYTES, OFF_SFP = L::OFF_SFP, OFF_SFV = L::OFF_SFV;
  (void)OFF_PS; (void)OFF_RAW; (void)RAW_STAGE; (void)PS_BYTES; (void)OFF_SFP; (void)OFF_SFV;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

#ifdef MPFA_TRACE
  if ((int)blockIdx.x == g_trace_cta && tid == 12 * 32 && g_trace) g_trace[((0) * 256 + 255) * 8 + 1] = clock64();   // kernel entry
#endif
  Ctx cx;
  cx.bars = sbase + OFF_BAR;
  cx.abort_flag = reinterpret_cast<volatile int *>(smem + OFF_MISC + 4);
  cx.status = p.status;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + OFF_MISC);

  // ---- one-time setup
  if (tid == 0) {
    *cx.abort_flag = 0;
    for (int i = 0; i < 2; ++i) { mbar_init(cx.bar(BAR_Q_FULL + i), 1); mbar_init(cx.bar(BAR_Q_EMPTY + i), 1); }
    for (int i = 0; i < KSTAGES; ++i) { mbar_init(cx.bar(BAR_K_FULL + i), 1); mbar_init(cx.bar(BAR_K_EMPTY + i), 1); }
    for (int i = 0; i < VSTAGES; ++i) { mbar_init(cx.bar(BAR_V_FULL + i), 1); mbar_init(cx.bar(BAR_V_EMPTY + i), 1); }
    mbar_init(cx.bar(BAR_S_FULL), 1);
    mbar_init(cx.bar(BAR_S_FULL + 1), 1);
    mbar_init(cx.bar(BAR_S_EMPTY), 4);   // one arrival per warp (lane 0 after __syncwarp)
    for (int i = 0; i < 2; ++i) {
      mbar_init(cx.bar(BAR_P_FULL + i), 4);
      mbar_init(cx.bar(BAR_P_EMPTY + i), 1);
      mbar_init(cx.bar(BAR_M_FULL + i), 4);
      mbar_init(cx.bar(BAR_O_FULL + i), 1);
      mbar_init(cx.bar(BAR_O_READY + i), 4);
    }
    for (int i = 0; i < 4; ++i) mbar_init(cx.bar(BAR_L_FULL + i), 8);
    mbar_init(cx.bar(BAR_O_FREE), 4);
    for (int i = 0; i < KSTAGES; ++i) mbar_init(cx.bar(BAR_SF_READY + i), 1);
    mbar_init_fence();
    prefetch_tmap(&tm_q);
    if (!PAGED) {
      prefetch_tmap(&tm_k);
      prefetch_tmap(&tm_v);
    }
  }
  // rank-one operands: MN-major, 128B swizzle, K = 16.  Row k = 0 of each 64-element half
  // holds the data (ones / Delta_S), every other row stays zero for the CTA's lifetime.
  for (int i = tid; i < (KST * 4096 + 4096) / 16; i += NTHREADS)
    reinterpret_cast<uint4 *>(smem + OFF_DELTA)[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  if (tid < 128) reinterpret_cast<uint16_t *>(smem + OFF_ONES)[(tid >> 6) * 1024 + (tid & 63)] = 0x3F80;  // 1.0
  fence_proxy_async_smem();
  if (warp == 2) {
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = *tmem_slot;

  const bool has_delta = !EW && p.delta != nullptr;   // operand of the seed MMA
  TR_INIT();
  if (warp == 12) TR(0, 255, 2);   // roles start (after setup)

  // Every role walks the same list of work items (q tile x q head) and keeps the same running count of
  // KV blocks; ring slots and barrier phases are functions of those two counters, so the pipeline runs
  // straight through item boundaries: the next item's Q/K/V arrive and its first scores are computed while
  // the correction warps write the previous item's output.
  TileWalk walk;
  walk.init();
  Tile tl;
  uint32_t gb = 0;   // KV blocks of the items already walked
  uint32_t ti = 0;   // index of the current item in this CTA's list

  if (warp < 4) setmaxnreg_dec<REGS_UTIL<PAGED>>();
  if (warp == 0) {
    // =========================== TMA producer ===========================
    // The whole warp runs the loop (uniform control flow keeps addresses and barrier handles in
    // uniform registers); a single elected lane issues each copy.
    bool ok = true;
    uint32_t nk_armed = 0, nv_armed = 0, nq_armed = 0;
    for (; ok && walk.template next<PAGED>(p, pg, tl); gb += tl.T, ++ti) {
      const uint32_t qb = ti & 1;
      if (ti >= 2) ok = cx.wait(BAR_Q_EMPTY + qb, ((ti >> 1) - 1) & 1u);
      if (!ok) break;
      const size_t q_row = ((size_t)tl.b * p.H_q + tl.hq) * (size_t)(p.nq_tiles * TILE) + tl.row0;
      const size_t k_row = ((size_t)tl.b * p.H_kv + tl.hk) * (size_t)(p.nk_tiles * TILE);
      if (elect_one()) {
        mbar_expect_tx(cx.bar(BAR_Q_FULL + qb), 8192 + 1024);
        tma_load_2d(sbase + OFF_Q + qb * 8192, &tm_q, 0, (int)q_row, cx.bar(BAR_Q_FULL + qb));
        bulk_load(sbase + OFF_SFQ + qb * 1024, p.q_sf + (((size_t)tl.b * p.H_q + tl.hq) * p.nq_tiles + tl.qt) * 1024, 1024,
                  cx.bar(BAR_Q_FULL + qb));
      }
      nq_armed = ti + 1;
      PageLookup look;
      for (int t = 0; t < tl.T && ok; ++t) {
        const uint32_t c = gb + t;
        const int jb = tl.T - 1 - t;
        const uint32_t ks = c % KST, vs = c % VST;
        int page_lo = 0, page_hi = 0;
        if (PAGED) look.get(pg, p.status, tl.b, tl.nkv, t, jb, lane, page_lo, page_hi);
        if (c >= (uint32_t)KST) ok = cx.wait(BAR_K_EMPTY + ks, (c / KST - 1) & 1u);
        if (!ok) break;
        TR(0, c, 0);
        if (PAGED) {
          if (elect_one()) {
            const uint32_t bar = cx.bar(BAR_K_FULL + ks);
            mbar_expect_tx(bar, 8192 + 1024 + (has_delta ? 256 : 0));
            const size_t s_lo = (size_t)page_lo * p.H_kv + tl.hk, s_hi = (size_t)page_hi * p.H_kv + tl.hk;
            bulk_load(sbase + OFF_K + ks * 8192, pg.k_codes + s_lo * 4096, 4096, bar);
            bulk_load(sbase + OFF_K + ks * 8192 + 4096, pg.k_codes + s_hi * 4096, 4096, bar);
            bulk_load(sbase + OFF_RAW + ks * RAW_STAGE, pg.k_sf + s_lo * 512, 512, bar);
            bulk_load(sbase + OFF_RAW + ks * RAW_STAGE + 512, pg.k_sf + s_hi * 512, 512, bar);
            if (has_delta) {
              bulk_load(sbase + OFF_RAW + ks * RAW_STAGE + 1024, pg.delta + ((size_t)page_lo * p.H_q + tl.hq) * 64, 128, bar);
              bulk_load(sbase + OFF_RAW + ks * RAW_STAGE + 1152, pg.delta + ((size_t)page_hi * p.H_q + tl.hq) * 64, 128, bar);
            }
          }
        } else if (elect_one()) {
          mbar_expect_tx(cx.bar(BAR_K_FULL + ks), 8192 + 1024 + (has_delta ? 256 : 0));
          tma_load_2d(sbase + OFF_K + ks * 8192, &tm_k, 0, (int)(k_row + (size_t)jb * TILE), cx.bar(BAR_K_FULL + ks));
          bulk_load(sbase + OFF_SFK + ks * 1024, p.k_sf + (((size_t)tl.b * p.H_kv + tl.hk) * p.nk_tiles + jb) * 1024, 1024,
                    cx.bar(BAR_K_FULL + ks));
          if (has_delta) {
            const __nv_bfloat16 *d = p.delta + ((size_t)tl.b * p.H_q + tl.hq) * (size_t)(p.nk_tiles * TILE) + (size_t)jb * TILE;
            bulk_load(sbase + OFF_DELTA + ks * 4096, d, 128, cx.bar(BAR_K_FULL + ks));
            bulk_load(sbase + OFF_DELTA + ks * 4096 + 2048, d + 64, 128, cx.bar(BAR_K_FULL + ks));
          }
        }
        nk_armed = c + 1;
        if (c >= (uint32_t)VST) ok = cx.wait(BAR_V_EMPTY + vs, (c / VST - 1) & 1u);
        if (!ok) break;
        TR(0, c, 1);
        if (MPFA_DROP_V(c)) {
          // test build: this copy is left out on purpose
        } else if (PAGED) {
          if (elect_one()) {
            const uint32_t bar = cx.bar(BAR_V_FULL + vs);
            mbar_expect_tx(bar, 16384);
            bulk_load(sbase + OFF_V + vs * 16384, pg.v_fp8 + ((size_t)page_lo * p.H_kv + tl.hk) * 8192, 8192, bar);
            bulk_load(sbase + OFF_V + vs * 16384 + 8192, pg.v_fp8 + ((size_t)page_hi * p.H_kv + tl.hk) * 8192, 8192, bar);
          }
        } else if (elect_one()) {
          mbar_expect_tx(cx.bar(BAR_V_FULL + vs), V_BYTES + (PV4 ? 1024u : 0u));
          tma_load_2d(sbase + OFF_V + vs * V_BYTES, &tm_v, 0, (int)(k_row + (size_t)jb * TILE), cx.bar(BAR_V_FULL + vs));
          if (PV4)   // channel-major FP4 tile (same row arithmetic as K: 128 channel rows per key tile) + its block scales
            bulk_load(sbase + OFF_SFV + vs * 1024, p.v_sf + (((size_t)tl.b * p.H_kv + tl.hk) * p.nk_tiles + jb) * 1024, 1024,
                      cx.bar(BAR_V_FULL + vs));
          if (PVB)   // BF16 rows are 256 bytes: the second 64-channel half is a box of its own
            tma_load_2d(sbase + OFF_V + vs * V_BYTES + 16384, &tm_v, 128, (int)(k_row + (size_t)jb * TILE), cx.bar(BAR_V_FULL + vs));
        }
        if (!MPFA_DROP_V(c)) nv_armed = c + 1;
      }
    }
    if (*cx.abort_flag) {
      // Drain: copies still in flight must land before the CTA's shared memory is released.
      for (uint32_t c = nk_armed - min(nk_armed, (uint32_t)KST); c < nk_armed; ++c)
        mbar_wait_ns(cx.bar(BAR_K_FULL + c % KST), (c / KST) & 1u, WAIT_LIMIT_NS);
      for (uint32_t c = nv_armed - min(nv_armed, (uint32_t)VST); c < nv_armed; ++c)
        if (!MPFA_DROP_V(c)) mbar_wait_ns(cx.bar(BAR_V_FULL + c % VST), (c / VST) & 1u, WAIT_LIMIT_NS);
      for (uint32_t i = nq_armed - min(nq_armed, 2u); i < nq_armed; ++i)
        mbar_wait_ns(cx.bar(BAR_Q_FULL + (i & 1)), (i >> 1) & 1u, WAIT_LIMIT_NS);
    }
  } else if (warp == 1) {
    // =========================== Q K^T issuer ===========================
    // Whole warp in uniform control flow; lane 0 (always the elected lane of a full warp) issues
    // every tcgen05 instruction, so the commits track the MMAs of the same thread.  This warp
    // only waits for operands (K block in shared memory, score buffer handed back by its
    // softmax group), so it runs ahead of the P V issuer (warp 3), also into the next work item.
    const uint32_t id_fp4 = idesc_nvfp4(128, 128);
    const uint32_t id_bf16 = idesc_bf16(128, 128, 1, 1);
    // All shared-memory descriptors are built once; a ring stage or K step only adds a
    // constant to the 14-bit start-address field (shared addresses stay below 256 KB).
    const uint64_t d_ones = smem_desc(sbase + OFF_ONES, 2048, 1024, SWZ_128B);
    const uint64_t d_delta0 = smem_desc(sbase + OFF_DELTA, 2048, 1024, SWZ_128B);
    const uint64_t d_q00 = smem_desc(sbase + OFF_Q, 16, 512, SWZ_64B);
    const uint64_t d_k0 = smem_desc(sbase + OFF_K, 16, 512, SWZ_64B);
    const uint64_t d_sfq00 = smem_desc(sbase + OFF_SFQ, 0, 128, SWZ_NONE);
    const uint64_t d_sfk0 = smem_desc(sbase + OFF_SFK, 0, 128, SWZ_NONE);
    bool ok = true;
    for (; ok && walk.template next<PAGED>(p, pg, tl); gb += tl.T, ++ti) {
      const uint32_t qb = ti & 1;
      ok = cx.wait(BAR_Q_FULL + qb, (ti >> 1) & 1u);
      if (!ok) break;
      const uint64_t d_q0 = d_q00 + (uint64_t)((qb * 8192) >> 4);
      const uint32_t tSFQ = tm + TM_SFQ + qb * 8;
      tc_fence_after();
      if (elect_one()) {
        const uint64_t d_sfq0 = d_sfq00 + (uint64_t)((qb * 1024) >> 4);
        tmem_cp_32x128b_warpx4(tSFQ, d_sfq0);
        tmem_cp_32x128b_warpx4(tSFQ + 4, d_sfq0 + (512 >> 4));
      }
      for (int t = 0; t < tl.T && ok; ++t) {
        const uint32_t c = gb + t;
        const uint32_t ks = c % KST, sb = c & 1;
        TR(5, c, 0);
        ok = cx.wait(BAR_K_FULL + ks, (c / KST) & 1u);
        if (PAGED) ok = ok && cx.wait(BAR_SF_READY + ks, (c / KST) & 1u);
        if (!ok) break;
        const uint32_t tSFK = tm + (sb ? TM_SFK1 : TM_SFK0);
        const uint64_t d_sfk = d_sfk0 + (uint64_t)((ks * 1024) >> 4);
        const uint64_t d_k = d_k0 + (uint64_t)((ks * 8192) >> 4);
        const uint64_t d_delta = d_delta0 + (uint64_t)((ks * 4096) >> 4);
        tc_fence_after();
        if (elect_one()) {   // scale factors first: their TMEM columns were last used by block c-2
          tmem_cp_32x128b_warpx4(tSFK, d_sfk);
          tmem_cp_32x128b_warpx4(tSFK + 4, d_sfk + (512 >> 4));
        }
        // the softmax group of block c-1 has read its scores out of the buffer
        if (c >= 1) ok = cx.wait(BAR_S_EMPTY, (c - 1) & 1u);
        if (!ok) break;
        TR(5, c, 1);
        tc_fence_after();
        if (elect_one()) {
#ifdef MPFA_ABLATE_NO_QK
          if (t > 100000)
#endif
          {
          if (has_delta) mma_bf16_ss(tm + TM_S, d_ones, d_delta, id_bf16, 0);
          mma_nvfp4_ss(tm + TM_S, d_q0, d_k, id_fp4, tSFQ, tSFK, has_delta ? 1u : 0u);
          mma_nvfp4_ss(tm + TM_S, d_q0 + (32 >> 4), d_k + (32 >> 4), id_fp4, tSFQ + 4, tSFK + 4, 1u);
          }
          mma_commit(cx.bar(BAR_S_FULL + sb));
          mma_commit(cx.bar(BAR_K_EMPTY + ks));
        }
        TR(5, c, 5);
      }
      if (ok && elect_one()) mma_commit(cx.bar(BAR_Q_EMPTY + qb));   // after every MMA that reads this query tile
      __syncwarp();
    }
  } else if (PAGED && warp == 2) {
    // ==== paged source: re-tile the K scales and un-swizzle Delta_S of every stage ====
    const int G = p.H_q / p.H_kv;
    bool ok = true;
    for (; ok && walk.template next<PAGED>(p, pg, tl); gb += tl.T, ++ti) {
      const int rsw = tl.hq % G;
      for (int t = 0; t < tl.T && ok; ++t) {
        const uint32_t c = gb + t;
        const uint32_t ks = c % KST;
        ok = cx.wait(BAR_K_FULL + ks, (c / KST) & 1u);
        if (!ok) break;
        const uint8_t *raw = smem + OFF_RAW + ks * RAW_STAGE;
        // scales: row-major [key][8] -> the 32x128b tile layout tcgen05.cp expects (lane = key mod 32)
        uint2 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = *reinterpret_cast<const uint2 *>(raw + (q >> 1) * 512 + ((q & 1) * 32 + lane) * 8);
        uint8_t *dst = smem + OFF_SFK + ks * 1024 + lane * 16;
        *reinterpret_cast<uint4 *>(dst) = make_uint4(v[0].x, v[1].x, v[2].x, v[3].x);
        *reinterpret_cast<uint4 *>(dst + 512) = make_uint4(v[0].y, v[1].y, v[2].y, v[3].y);
        // Delta_S: 16-byte group c of a page is stored at c ^ (q head mod G); row 0 of the operand wants them in order
        if (has_delta && lane < 16) {
          const int half = lane >> 3, cg = lane & 7;
          const uint4 d = *reinterpret_cast<const uint4 *>(raw + 1024 + half * 128 + ((cg ^ rsw) << 4));
          *reinterpret_cast<uint4 *>(smem + OFF_DELTA + ks * 4096 + half * 2048 + (cg << 4)) = d;
        }
        fence_proxy_async_smem();
        warp_arrive(cx.bar(BAR_SF_READY + ks), lane);
      }
    }
  } else if (warp == 3) {
    // =========================== P V issuer ===========================
    const uint32_t id_fp8 = idesc_e4m3(128, 128, 0, 1);
    const uint32_t id_bf16_pv = idesc_bf16(128, 128, 0, 1);
    const uint32_t id_fp4_pv = idesc_nvfp4(128, 128);
    const uint64_t d_v0 = PV4 ? smem_desc(sbase + OFF_V, 16, 512, SWZ_64B) : smem_desc(sbase + OFF_V, PVB ? 16384 : 16, 1024, SWZ_128B);
    const uint64_t d_p0 = PV4 ? smem_desc(sbase + OFF_PS, 16, 512, SWZ_64B) : smem_desc(sbase + OFF_PS, 16, 1024, SWZ_128B);
    const uint64_t d_sfp0 = smem_desc(sbase + OFF_SFP, 0, 128, SWZ_NONE);
    const uint64_t d_sfv0 = smem_desc(sbase + OFF_SFV, 0, 128, SWZ_NONE);
    (void)id_fp8; (void)id_bf16_pv; (void)d_p0; (void)id_fp4_pv; (void)d_sfp0; (void)d_sfv0;
    bool ok = true;
    uint32_t n_used = 0;   // items so far that used the accumulators (T > 0)
    for (; ok && walk.template next<PAGED>(p, pg, tl); gb += tl.T, ++ti) {
      if (tl.T == 0) continue;
      // the previous such item's epilogue has read both accumulators
      if (n_used >= 1) ok = cx.wait(BAR_O_FREE, (n_used - 1) & 1u);
      ++n_used;
      for (int t = 0; t < tl.T && ok; ++t) {
        const uint32_t c = gb + t;
        TR(1, c, 0);
        const uint32_t sb = c & 1, vs = c % VST;
        ok = cx.wait(BAR_V_FULL + vs, (c / VST) & 1u);
        TR(1, c, 1);
        ok = ok && cx.wait(BAR_O_READY + sb, (c >> 1) & 1u);
        TR(1, c, 2);
        ok = ok && cx.wait(BAR_P_FULL + sb, (c >> 1) & 1u);
        TR(1, c, 3);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tP = tm + (sb ? TM_P1 : TM_P0);
        const uint32_t tOacc = tm + (sb ? TM_O1 : TM_O0);
        const uint64_t d_v = d_v0 + (uint64_t)((vs * V_BYTES) >> 4);
        if (elect_one()) {
          if constexpr (PVB) {
            // BF16: A = P of this group from shared memory (K-major, two 64-key halves of 16 KB), B = V (MN-major,
            // two 64-channel halves of 16 KB, 16 keys = 2 KB per K step)
            const uint64_t d_p = d_p0 + (uint64_t)((sb * 32768) >> 4);
#pragma unroll
            for (int k16 = 0; k16 < 8; ++k16)
              mma_bf16_ss(tOacc, d_p + (uint64_t)(((k16 >> 2) * 16384 + (k16 & 3) * 32) >> 4), d_v + (uint64_t)((2048 * k16) >> 4),
                          id_bf16_pv, (t >= 2 || k16 > 0) ? 1u : 0u);
          } else if constexpr (PV4) {
            // block-scaled FP4: A = P-hat codes of this group (K-major, 64-byte rows), B = V codes (channel-major);
            // both operands' block scales go to tensor memory first (their columns were last read by block c-2)
            const uint64_t d_p = d_p0 + (uint64_t)((sb * PS_BYTES) >> 4);
            const uint64_t d_sfp = d_sfp0 + (uint64_t)((sb * 1024) >> 4), d_sfv = d_sfv0 + (uint64_t)((vs * 1024) >> 4);
            const uint32_t tSFP = tm + (sb ? TM_SFP1 : TM_SFP0), tSFV = tm + (sb ? TM_SFV1 : TM_SFV0);
            tmem_cp_32x128b_warpx4(tSFP, d_sfp);
            tmem_cp_32x128b_warpx4(tSFP + 4, d_sfp + (512 >> 4));
            tmem_cp_32x128b_warpx4(tSFV, d_sfv);
            tmem_cp_32x128b_warpx4(tSFV + 4, d_sfv + (512 >> 4));
            mma_nvfp4_ss(tOacc, d_p, d_v, id_fp4_pv, tSFP, tSFV, t >= 2 ? 1u : 0u);
            mma_nvfp4_ss(tOacc, d_p + (32 >> 4), d_v + (32 >> 4), id_fp4_pv, tSFP + 4, tSFV + 4, 1u);
          } else {
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
#ifdef MPFA_ABLATE_NO_PV
            if (k4 > 100)
#endif
            mma_e4m3_ts(tOacc, tP + 8 * k4, d_v + (uint64_t)((4096 * k4) >> 4), id_fp8, (t >= 2 || k4 > 0) ? 1u : 0u);
          }
          mma_commit(cx.bar(BAR_O_FULL + sb));
          mma_commit(cx.bar(BAR_P_EMPTY + sb));
          mma_commit(cx.bar(BAR_V_EMPTY + vs));
        }
        TR(1, c, 5);
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // =========================== softmax groups ===========================
    setmaxnreg_inc<REGS_SOFTMAX>();
    const int grp = (warp - 4) >> 2;                 // takes the KV blocks whose running count has this parity
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const float *gq = p.q_gscale, *gk = p.k_gscale;
    float *s_m = reinterpret_cast<float *>(smem + OFF_M);
    const uint32_t tS = tm + TM_S + lane_off;
    const uint32_t tP = tm + (grp ? TM_P1 : TM_P0) + lane_off;
    uint8_t *const ps_row = smem + OFF_PS + grp * 32768 + row * 128;   // PVB: this thread's row of the group's P operand
    // PV4: this thread's 64-byte row of the group's FP4 operand (64B swizzle: 16-byte chunk ^ ((row >> 1) & 3)) and its
    // word in each of the group's two scale-factor atoms
    uint8_t *const p4_row = smem + OFF_PS + grp * 8192 + row * 64;
    uint8_t *const sfp_row = smem + OFF_SFP + grp * 1024 + (row & 31) * 16 + (row >> 5) * 4;
    (void)tP; (void)ps_row; (void)p4_row; (void)sfp_row;
    bool ok = true;
    uint32_t n_used = 0;   // items so far with T > 0: only those go through the row-sum ring
    for (; ok && walk.template next<PAGED>(p, pg, tl); gb += tl.T, ++ti) {
      const int T = tl.T;
      if (T == 0) continue;   // nothing to attend to: the epilogue writes zeros without waiting for this role
      const int r_abs = tl.row0 + row;
      const int n_kv = PAGED ? tl.nkv : p.N_kv;
      const int n_q = PAGED ? tl.nq : p.N_q;
      const int limit = (PAGED && r_abs >= n_q) ? -1   // a row past the request's own query count sees nothing
                        : p.causal ? min(n_kv - 1, r_abs + (n_kv - n_q)) : n_kv - 1;   // last visible key
      const float lam = __fmul_rn(__fmul_rn(__fmul_rn(p.softmax_scale, 1.4426950408889634f), gq[tl.b]), gk[tl.b]);
      bool p_pending = false;    // P-hat of the previous block written but not yet handed over
      float m_own = -INFINITY;   // running maximum after this group's previous block
      float l_own = 0.0f;        // sum of 448 P over this group's blocks, relative to m_own
      for (int t = (grp ^ (int)gb) & 1; t < T; t += 2) {
        const uint32_t c = gb + t;
        const int key0 = (T - 1 - t) * TILE;
        TR(2 + grp, c, 0);
        if (!__all_sync(0xffffffffu, cx.wait(BAR_S_FULL + grp, (c >> 1) & 1u))) { ok = false; break; }
        TR(2 + grp, c, 1);
        tc_fence_after();
        uint32_t s[128];
        {
          uint32_t(&s0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
          uint32_t(&s1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
          tmem_ld32(tS, s0);
          tmem_ld32(tS + 32, s1);
        }
        if (p_pending) {
          // P-hat of this group's previous block is handed to the P V issuer only now: its tensor-memory stores
          // have had the loop tail and the barrier wait above to complete, so this wait costs nothing, where the
          // same wait right after the stores held the warp for their whole latency (measured: +2.7 % at 16K,
          // +1.7 % at 64K).  P V of a block has a block and a half of slack before anything waits for it.
          tmem_st_wait();
          tc_fence_before();
          warp_arrive(cx.bar(BAR_P_FULL + grp), lane);
          p_pending = false;
        }
        // While the scores are on their way, test (without blocking) the two other conditions this
        // block needs; the answers are consumed later, so their latency overlaps the TMEM load:
        //  - P V of block c-2 has consumed this group's P_hat columns (this also means the
        //    correction warps have read the maximum this group published two blocks ago);
        //  - the other group's running maximum of block c-1 (same item) is published.
        const uint32_t par_pe = ((c >> 1) - 1) & 1u, par_m = ((c - 1) >> 1) & 1u;
        const bool pe_early = (c < 2) || cx.probe(BAR_P_EMPTY + grp, par_pe);
        bool have_prev = (t == 0) || cx.probe(BAR_M_FULL + (grp ^ 1), par_m);
        float m_prev = -INFINITY;
#ifdef MPFA_ABLATE_NO_MHAND
        have_prev = true;
#endif
        const bool ragged = key0 + TILE - 1 > limit;   // diagonal / ragged block only
        tmem_ld_wait();
        {
          // second half of the row in flight while the maximum of the first half is taken
          uint32_t(&s2)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[64]);
          uint32_t(&s3)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[96]);
          tmem_ld32(tS + 64, s2);
          tmem_ld32(tS + 96, s3);
        }
        if constexpr (EW) {
          const uint4 *dp = reinterpret_cast<const uint4 *>(
              p.delta + ((size_t)tl.b * p.H_q + tl.hq) * (size_t)(p.nk_tiles * TILE) + key0);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint4 d = __ldg(dp + i);
            const uint32_t w[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {   // packed pair: both halves round like the scalar add
              float x0 = __uint_as_float(s[8 * i + 2 * j]), x1 = __uint_as_float(s[8 * i + 2 * j + 1]);
              acc2(x0, x1, __uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xFFFF0000u));
              s[8 * i + 2 * j] = __float_as_uint(x0), s[8 * i + 2 * j + 1] = __float_as_uint(x1);
            }
          }
        }
        if (ragged) {
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (key0 + i > limit) s[i] = 0xFF800000u;   // -inf
        }
        // row maximum (Eq. 3)
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int i = 0; i < 64; i += 8) {
          mx0 = max3(mx0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
          mx1 = max3(mx1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
          mx2 = max3(mx2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
          mx3 = max3(mx3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
        }
        tmem_ld_wait();
        tc_fence_before();
        warp_arrive(cx.bar(BAR_S_EMPTY), lane);   // the row is in registers: Q K^T of block c+1 may overwrite it
        TR(2 + grp, c, 2);
        if constexpr (EW) {
          const uint4 *dp = reinterpret_cast<const uint4 *>(
              p.delta + ((size_t)tl.b * p.H_q + tl.hq) * (size_t)(p.nk_tiles * TILE) + key0 + 64);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint4 d = __ldg(dp + i);
            const uint32_t w[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              float x0 = __uint_as_float(s[64 + 8 * i + 2 * j]), x1 = __uint_as_float(s[64 + 8 * i + 2 * j + 1]);
              acc2(x0, x1, __uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xFFFF0000u));
              s[64 + 8 * i + 2 * j] = __float_as_uint(x0), s[64 + 8 * i + 2 * j + 1] = __float_as_uint(x1);
            }
          }
        }
        if (ragged) {
#pragma unroll
          for (int i = 64; i < 128; ++i)
            if (key0 + i > limit) s[i] = 0xFF800000u;   // -inf
        }
#pragma unroll
        for (int i = 64; i < 128; i += 8) {
          mx0 = max3(mx0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
          mx1 = max3(mx1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
          mx2 = max3(mx2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
          mx3 = max3(mx3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
        }
#ifdef MPFA_ABLATE_NO_MAX
        const float mx = fmaxf(__uint_as_float(s[0]), __uint_as_float(s[127])) + 30.0f;
#else
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
#endif
        // running maximum: the other group owns block c-1
        if (!__all_sync(0xffffffffu, have_prev)) {
          if (!__all_sync(0xffffffffu, cx.wait(BAR_M_FULL + (grp ^ 1), par_m))) { ok = false; break; }
        }
        if (t > 0) m_prev = s_m[(grp ^ 1) * 128 + row];
#ifdef MPFA_ABLATE_NO_MHAND
        m_prev = m_own;
#endif
        if (!__all_sync(0xffffffffu, pe_early)) {
          if (!__all_sync(0xffffffffu, cx.wait(BAR_P_EMPTY + grp, par_pe))) { ok = false; break; }
        }
        TR(2 + grp, c, 3);
        const float m_t = fmaxf(m_prev, mx);
        s_m[grp * 128 + row] = m_t;
        warp_arrive(cx.bar(BAR_M_FULL + grp), lane);
        TR(2 + grp, c, 4);
        const float a_own = (m_t == m_own) ? 1.0f : ex2_approx(__fmul_rn(m_own - m_t, lam));
        // P = 2^(lam S - lam m) (Eq. 4)
        // the factor 448 of the E4M3 operand is folded into the exponent: q = 448 P = 2^(lam S - lam m + log2 448)
        const float cc = (m_t == -INFINITY) ? 0.0f : __fsub_rn(PVB ? 0.0f : 8.8073549220576042f, __fmul_rn(m_t, lam));
        float sum0 = 0.0f, sum1 = 0.0f, sum2 = 0.0f, sum3 = 0.0f;
#ifdef MPFA_ABLATE_NO_SOFTMAX
        sum0 = __uint_as_float(s[5]);
        if (false)
#endif
        {
#ifdef MPFA_ABLATE_NO_EXP
#define EX2_(x) (x)
#else
#define EX2_(x) ex2_approx(x)
#endif
          // q = 448 P is the E4M3 operand (Section 4.1); the row sum is taken over q and the factor
          // 448 is divided out once in the epilogue.
          uint32_t sfw = 0u;   // PV4: the E4M3 block scales of 64 keys
          (void)sfw;
#pragma unroll
          for (int c0 = 0; c0 < 128; c0 += 32) {
            uint32_t packed[8];
            uint32_t pbf[4];
            float qv[32];
            (void)packed; (void)pbf; (void)qv;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              float x0, x1, x2, x3;
              fma2(x0, x1, __uint_as_float(s[c0 + 4 * i]), __uint_as_float(s[c0 + 4 * i + 1]), lam, cc);
              fma2(x2, x3, __uint_as_float(s[c0 + 4 * i + 2]), __uint_as_float(s[c0 + 4 * i + 3]), lam, cc);
              const float q0 = EX2_(x0), q1 = EX2_(x1), q2 = EX2_(x2), q3 = EX2_(x3);
              acc2(sum0, sum1, q0, q1);
              acc2(sum2, sum3, q2, q3);
              if constexpr (PV4) {
                qv[4 * i] = q0, qv[4 * i + 1] = q1, qv[4 * i + 2] = q2, qv[4 * i + 3] = q3;
              } else if constexpr (PVB) {
                // BF16 pairs (first operand of the conversion goes to the upper half)
                asm("cvt.rn.bf16x2.f32 %0, %2, %1;" : "=r"(pbf[2 * (i & 1)]) : "f"(q0), "f"(q1));
                asm("cvt.rn.bf16x2.f32 %0, %2, %1;" : "=r"(pbf[2 * (i & 1) + 1]) : "f"(q2), "f"(q3));
                if (i & 1) {
                  // eight keys = one 16-byte chunk of the row in the K-major, 128B-swizzled A operand
                  const int ch = (c0 >> 3) + (i >> 1);
                  *reinterpret_cast<uint4 *>(ps_row + (ch >> 3) * 16384 + (((ch & 7) ^ (row & 7)) << 4)) =
                      make_uint4(pbf[0], pbf[1], pbf[2], pbf[3]);
                }
              } else {
              // two conversions written into the halves of one register (no separate merge instruction)
              asm("{.reg .b16 lo, hi;\n\t"
                  "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
                  "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
                  "mov.b32 %0, {lo, hi};}"
                  : "=r"(packed[i])
                  : "f"(q0), "f"(q1), "f"(q2), "f"(q3));
              }
            }
            if constexpr (PV4) {
              // two blocks of 16 keys: scale = E4M3(max q), codes = E2M1(q * (6 / scale)) (Eq. 1 with the tensor scale
              // of P fixed at 1 / (6 * 448))
              uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
              for (int hb = 0; hb < 2; ++hb) {
                const float *qb = qv + 16 * hb;
                float a0 = max3(qb[0], qb[1], qb[2]), a1 = max3(qb[3], qb[4], qb[5]), a2 = max3(qb[6], qb[7], qb[8]),
                      a3 = max3(qb[9], qb[10], qb[11]);
                a0 = max3(a0, qb[12], qb[13]);
                a1 = max3(a1, qb[14], qb[15]);
                const float amax = fmaxf(fmaxf(a0, a1), fmaxf(a2, a3));
                const uint32_t sc = (uint32_t)__nv_cvt_float_to_fp8(amax, __NV_SATFINITE, __NV_E4M3);
                const float sdec = __half2float(__half(__nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)sc, __NV_E4M3)));
                const float inv = sdec > 0.0f ? __fdiv_rn(6.0f, sdec) : 0.0f;
                sfw |= sc << (8 * (((c0 >> 4) + hb) & 3));
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  const uint32_t byte = (uint32_t)__nv_cvt_float2_to_fp4x2(
                      make_float2(__fmul_rn(qb[2 * j], inv), __fmul_rn(qb[2 * j + 1], inv)), __NV_E2M1, cudaRoundNearest);
                  w[2 * hb + (j >> 2)] |= (byte & 0xFFu) << (8 * (j & 3));
                }
              }
              *reinterpret_cast<uint4 *>(p4_row + ((((c0 >> 5)) ^ ((row >> 1) & 3)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
              if (c0 & 32) {   // 64 keys done: one word of the row in this half's scale-factor atom
                *reinterpret_cast<uint32_t *>(sfp_row + (c0 >> 6) * 512) = sfw;
                sfw = 0u;
              }
            } else if constexpr (!PVB) {
#ifndef MPFA_ABLATE_NO_PST
            tmem_st8(tP + (c0 >> 2), packed);
#else
            if (packed[0] == 0x12345u && packed[7] == 77u) tmem_st8(tP + (c0 >> 2), packed);
#endif
            }
          }
        }
        l_own = __fadd_rn(__fmul_rn(a_own, l_own), (sum0 + sum1) + (sum2 + sum3));
        m_own = m_t;
        TR(2 + grp, c, 5);
        if constexpr (PVB || PV4) {
          fence_proxy_async_smem();   // the P rows were written through the generic proxy, the MMA reads them through the async one
          tc_fence_before();
          warp_arrive(cx.bar(BAR_P_FULL + grp), lane);
        } else if constexpr (EW) {   // measured: this variant is faster with the hand-over where the stores are
          tmem_st_wait();
          tc_fence_before();
          warp_arrive(cx.bar(BAR_P_FULL + grp), lane);
        } else {
          p_pending = true;   // handed over at the top of the next iteration, or below after the item's last block
        }
        TR(2 + grp, c, 6);
      }
      if (p_pending) {
        tmem_st_wait();
        tc_fence_before();
        warp_arrive(cx.bar(BAR_P_FULL + grp), lane);
        p_pending = false;
      }
      if (!ok) break;
      // which group took the item's last block decides how the epilogue combines the two accumulators
      float *s_fin = reinterpret_cast<float *>(smem + OFF_L) + (n_used & 3) * 512;
      s_fin[(grp * 2 + 0) * 128 + row] = l_own;
      s_fin[(grp * 2 + 1) * 128 + row] = m_own;
      warp_arrive(cx.bar(BAR_L_FULL + (n_used & 3)), lane);
      ++n_used;
    }
  } else if (warp >= 12) {
    // =========================== correction + epilogue ===========================
    setmaxnreg_dec<REGS_CORR<PAGED>>();
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const float *s_m = reinterpret_cast<const float *>(smem + OFF_M);
    const uint32_t tO0 = tm + TM_O0 + lane_off, tO1 = tm + TM_O1 + lane_off;
    bool ok = true;
    uint32_t n_used = 0;   // items so far with T > 0 (slot and phase of the row-sum ring)
    for (; walk.template next<PAGED>(p, pg, tl); gb += tl.T, ++ti) {
      const int T = tl.T;
      const int r_abs = tl.row0 + row;
      const float lam_c = __fmul_rn(__fmul_rn(__fmul_rn(p.softmax_scale, 1.4426950408889634f), p.q_gscale[tl.b]), p.k_gscale[tl.b]);
      float alpha_prev = 1.0f, alpha = 1.0f, m_before = -INFINITY;
      for (int t = 0; ok && t < T; ++t) {
        const uint32_t c = gb + t;
        const uint32_t sb = c & 1;
        TR(4, c, 0);
        ok = __all_sync(0xffffffffu, cx.wait(BAR_M_FULL + sb, (c >> 1) & 1u));
        if (!ok) break;
        TR(4, c, 1);
        // alpha_t = 2^(lam (m_{t-1} - m_t)) (Eq. 5/6), from the running maxima the softmax groups publish
        const float m_now = s_m[sb * 128 + row];
        alpha = (m_now == m_before) ? 1.0f : ex2_approx(__fmul_rn(m_before - m_now, lam_c));
        m_before = m_now;
        if (t >= 2) {
          // O[sb] holds blocks t-2, t-4, ... relative to the maximum after block t-2
          const float scale = __fmul_rn(alpha, alpha_prev);
          ok = __all_sync(0xffffffffu, cx.wait(BAR_O_FULL + sb, ((c >> 1) - 1) & 1u));
          if (!ok) break;
          TR(4, c, 2);
          tc_fence_after();
#ifdef MPFA_ABLATE_NO_CORR
          if (false) {
#else
          if (__any_sync(0xffffffffu, scale != 1.0f)) {   // identical result when every factor is exactly 1
#endif
            const uint32_t tO = sb ? tO1 : tO0;
#pragma unroll
            for (int c0 = 0; c0 < HEAD_DIM; c0 += 32) {
              uint32_t r[32];
              tmem_ld32(tO + c0, r);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; i += 2) {   // packed pairs: half the issue slots, same roundings
                float y0, y1;
                mul2(y0, y1, __uint_as_float(r[i]), __uint_as_float(r[i + 1]), scale);
                r[i] = __float_as_uint(y0), r[i + 1] = __float_as_uint(y1);
              }
              tmem_st32(tO + c0, r);
            }
            tmem_st_wait();
          }
          tc_fence_before();
        }
        alpha_prev = alpha;
        TR(4, c, 3);
        warp_arrive(cx.bar(BAR_O_READY + sb), lane);
      }
      // final normalisation (Algorithm 1 line 17): O / (448 l) * v_scale -> BF16.  The two softmax
      // groups hold partial sums relative to their own last maximum; bring both to the final one.
      // The accumulator of the last block is current; the other one is one alpha behind.
      const int last = (int)((gb + T - 1) & 1);
      float l = 0.0f, a_other = 0.0f;
      if (ok) {
        if (T > 0) ok = cx.wait(BAR_O_FULL + last, ((gb + T - 1) >> 1) & 1u);
        if (ok && T > 1) ok = cx.wait(BAR_O_FULL + (last ^ 1), ((gb + T - 2) >> 1) & 1u);
        if (T > 0) ok = ok && cx.wait(BAR_L_FULL + (n_used & 3), (n_used >> 2) & 1u);
        tc_fence_after();
        if (ok && T > 0) {
          const float lam = lam_c;
          const float *s_fin = reinterpret_cast<const float *>(smem + OFF_L) + (n_used & 3) * 512;
          const float l0 = s_fin[0 * 128 + row], m0 = s_fin[1 * 128 + row];
          const float l1 = s_fin[2 * 128 + row], m1 = s_fin[3 * 128 + row];
          const float mf = fmaxf(m0, m1);
          if (mf != -INFINITY) {
            const float w0 = (m0 == mf) ? 1.0f : ex2_approx(__fmul_rn(m0 - mf, lam));
            const float w1 = (m1 == mf) ? 1.0f : ex2_approx(__fmul_rn(m1 - mf, lam));
            l = __fadd_rn(__fmul_rn(w0, l0), __fmul_rn(w1, l1));
          }
          if (T > 1) a_other = alpha;   // alpha of the last block
        }
      }
      // tcgen05.ld is warp-collective: every lane loads, only the stores are predicated.
      const bool warp_ok = __all_sync(0xffffffffu, ok);
      const bool store = r_abs < p.N_q && (warp_ok || T == 0);
      const size_t o_off = (((size_t)tl.b * p.N_q + (store ? r_abs : 0)) * p.H_q + tl.hq) * HEAD_DIM;
      // one IEEE reciprocal per row; 128 divisions per thread would cost more than ten KV blocks
      const float inv_denom = (l > 0.0f) ? __frcp_rn(l) : 0.0f;   // l already carries the factor 448
      const uint32_t tOl = last ? tO1 : tO0, tOo = last ? tO0 : tO1;
#pragma unroll 1
      for (int c0 = 0; c0 < HEAD_DIM; c0 += 16) {
        uint32_t r[16], ro[16];
        if (T > 0 && warp_ok) {
          tmem_ld16(tOl + c0, r);
          if (T > 1) tmem_ld16(tOo + c0, ro);
          tmem_ld_wait();
        }
        if (c0 == HEAD_DIM - 16 && T > 0) {   // both accumulators are in registers: the next item's P V may overwrite them
          tc_fence_before();
          warp_arrive(cx.bar(BAR_O_FREE), lane);
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float acc = __uint_as_float(r[i]);
          if (T > 1) acc = __fadd_rn(acc, __fmul_rn(a_other, __uint_as_float(ro[i])));
          r[i] = (l > 0.0f) ? __float_as_uint(__fmul_rn(__fmul_rn(acc, inv_denom), p.v_scale)) : 0u;
        }
        if (store) {
          if (p.out_f32) {
#pragma unroll
            for (int i = 0; i < 16; i += 4)
              *reinterpret_cast<uint4 *>(p.out_f32 + o_off + c0 + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
          }
#pragma unroll
          for (int i = 0; i < 16; i += 8) {
            uint32_t h[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[i + 2 * j]), __uint_as_float(r[i + 2 * j + 1]));
              h[j] = *reinterpret_cast<uint32_t *>(&v);
            }
            *reinterpret_cast<uint4 *>(p.out + o_off + c0 + i) = make_uint4(h[0], h[1], h[2], h[3]);
          }
        }
      }
      if (T > 0) ++n_used;
      if (!ok) break;
    }
  }
  if (warp == 12) TR(0, 255, 3);   // epilogue stores issued
  tc_fence_before();
  __syncthreads();
  if (warp == 12) TR(0, 255, 4);
  if (warp == 2) tmem_dealloc(tm, TMEM_COLS);
}

}  // namespace
}  // namespace mpfa

using namespace mpfa;

#ifdef MPFA_TRACE
extern "C" int mpfa_debug_set_trace(long long *buf, int cta) {
  if (cudaMemcpyToSymbol(g_trace, &buf, sizeof(buf)) != cudaSuccess) return -1;
  if (cudaMemcpyToSymbol(g_trace_cta, &cta, sizeof(cta)) != cudaSuccess) return -1;
  return 0;
}
#endif

// 0: one query tile per CTA, two softmax groups alternating over KV blocks (the faster one on B200, see
// prefill_pair.cu's header for the measured comparison); 1: two query tiles per CTA (prefill_pair.cu)
static int g_arrangement = 0;
extern "C" int mpfa_set_prefill_arrangement(int a) {
  if (a != 0 && a != 1) return MPFA_ERR_INVALID_ARG;
  g_arrangement = a;
  return MPFA_OK;
}

extern "C" mpfa_status mpfa_prefill(const mpfa_fp4_tensor *q, const mpfa_fp4_tensor *k, const uint8_t *v_fp8,
                                    const void *delta_s_bf16, const mpfa_stats *st, float v_scale, int causal,
                                    float softmax_scale, void *out_bf16, float *out_f32, int32_t *device_status,
                                    void *stream) {
  return mpfa_prefill_variant(q, k, v_fp8, delta_s_bf16, st, v_scale, causal, softmax_scale, 0, out_bf16, out_f32,
                              device_status, stream);
}

extern "C" mpfa_status mpfa_prefill_variant(const mpfa_fp4_tensor *q, const mpfa_fp4_tensor *k, const uint8_t *v_fp8,
                                            const void *delta_s_bf16, const mpfa_stats *st, float v_scale, int causal,
                                            float softmax_scale, int variant, void *out_bf16, float *out_f32,
                                            int32_t *device_status, void *stream) {
  if (variant != 0 && variant != MPFA_VARIANT_COMP_ELEMENTWISE && variant != MPFA_VARIANT_PV_BF16 && variant != MPFA_VARIANT_PV_FP4)
    return MPFA_ERR_INVALID_ARG;
  const bool ew = variant == MPFA_VARIANT_COMP_ELEMENTWISE && delta_s_bf16 != nullptr;
  const bool pvb = variant == MPFA_VARIANT_PV_BF16;   // v_fp8 then points at the BF16 tile tensor of mpfa_pack_v_bf16
  const bool pv4 = variant == MPFA_VARIANT_PV_FP4;    // ... at the FP4 operand of mpfa_quantize_v_fp4, v_scale = its v_gscale
  if (!q || !k || !v_fp8 || !st || !out_bf16 || !device_status) return MPFA_ERR_INVALID_ARG;
  if (!q->codes || !q->sf || !k->codes || !k->sf || !st->q_gscale || !st->k_gscale) return MPFA_ERR_INVALID_ARG;
  if (q->B <= 0 || q->B != k->B || q->H <= 0 || k->H <= 0 || q->N <= 0 || k->N <= 0) return MPFA_ERR_INVALID_ARG;
  if (!(softmax_scale > 0.0f) || !(v_scale > 0.0f)) return MPFA_ERR_INVALID_ARG;
  if (q->H % k->H != 0 || q->H / k->H > 8) return MPFA_ERR_UNSUPPORTED;
  if (!aligned(q->codes, 1024) || !aligned(k->codes, 1024) || !aligned(q->sf, 1024) || !aligned(k->sf, 1024) ||
      !aligned(v_fp8, 1024) || !aligned(delta_s_bf16, 256) || !aligned(out_bf16, 16) || !aligned(out_f32, 16))
    return MPFA_ERR_ALIGNMENT;
  const int nq_tiles = pad128(q->N) / TILE, nk_tiles = pad128(k->N) / TILE;
  const uint64_t q_rows = (uint64_t)q->B * q->H * nq_tiles * TILE, k_rows = (uint64_t)k->B * k->H * nk_tiles * TILE;
  if (q_rows >= (1ull << 31) || k_rows >= (1ull << 31)) return MPFA_ERR_UNSUPPORTED;
  const uint64_t n_cta = (uint64_t)q->B * q->H * nq_tiles;
  if (n_cta >= (1ull << 31)) return MPFA_ERR_UNSUPPORTED;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  PrefillParams p;
  p.q_sf = q->sf;
  p.k_sf = k->sf;
  p.delta = static_cast<const __nv_bfloat16 *>(delta_s_bf16);
  p.q_gscale = st->q_gscale;
  p.k_gscale = st->k_gscale;
  p.out = static_cast<__nv_bfloat16 *>(out_bf16);
  p.out_f32 = out_f32;
  p.status = device_status;
  p.B = q->B;
  p.N_q = q->N;
  p.N_kv = k->N;
  p.H_q = q->H;
  p.H_kv = k->H;
  p.nq_tiles = nq_tiles;
  p.nk_tiles = nk_tiles;
  p.causal = causal ? 1 : 0;
  p.softmax_scale = softmax_scale;
  p.v_scale = v_scale;
  p.n_items = (int)n_cta;
  if (pv4) {
    // codes of all tiles first, then the block scales; the MMA result is in units of 6 * 448 P x V / v_gscale and the
    // row sum carries the 448
    p.v_sf = v_fp8 + (size_t)k->B * k->H * nk_tiles * 8192;
    p.v_scale = v_scale * (1.0f / 6.0f);
  }
  if (g_arrangement == 1 && !pvb && !pv4) return launch_prefill_pair(q, k, v_fp8, p, ew, static_cast<cudaStream_t>(stream));
  EncodeTiledFn enc;
  rc = get_encoder(&enc);
  if (rc != MPFA_OK) return rc;
  CUtensorMap tq, tk, tv;
  if ((rc = make_map(enc, &tq, q->codes, q_rows, 64)) != MPFA_OK) return rc;
  if ((rc = make_map(enc, &tk, k->codes, k_rows, 64)) != MPFA_OK) return rc;
  if ((rc = pvb ? make_map(enc, &tv, v_fp8, k_rows, 256, 128) : make_map(enc, &tv, v_fp8, k_rows, pv4 ? 64 : 128)) != MPFA_OK) return rc;
  int dev = 0, n_sm = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  MPFA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  const unsigned grid = (unsigned)(n_cta < (uint64_t)n_sm ? n_cta : (uint64_t)n_sm);   // one persistent CTA per SM
  if (pvb) {
    MPFA_CUDA_OK(cudaFuncSetAttribute(prefill_kernel<false, false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<1>::SMEM_BYTES));
    prefill_kernel<false, false, 1><<<grid, NTHREADS, Lay<1>::SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(tq, tk, tv, p, PagedSrc{});
  } else if (pv4) {
    MPFA_CUDA_OK(cudaFuncSetAttribute(prefill_kernel<false, false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<2>::SMEM_BYTES));
    prefill_kernel<false, false, 2><<<grid, NTHREADS, Lay<2>::SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(tq, tk, tv, p, PagedSrc{});
  } else if (ew) {
    MPFA_CUDA_OK(cudaFuncSetAttribute(prefill_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<0>::SMEM_BYTES));
    prefill_kernel<false, true><<<grid, NTHREADS, Lay<0>::SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(tq, tk, tv, p, PagedSrc{});
  } else {
    MPFA_CUDA_OK(cudaFuncSetAttribute(prefill_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<0>::SMEM_BYTES));
    prefill_kernel<false, false><<<grid, NTHREADS, Lay<0>::SMEM_BYTES, static_cast<cudaStream_t>(stream)>>>(tq, tk, tv, p, PagedSrc{});
  }
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

extern "C" mpfa_status mpfa_prefill_paged(const mpfa_fp4_tensor *q, const mpfa_paged_kv *kv, const int32_t *page_table,
                                          int max_pages_per_req, const int32_t *seq_lens, const int32_t *q_lens,
                                          const mpfa_stats *st,
                                          float v_scale, float softmax_scale, void *out_bf16, float *out_f32,
                                          int32_t *device_status, void *stream) {
  if (!q || !kv || !page_table || !seq_lens || !st || !out_bf16 || !device_status) return MPFA_ERR_INVALID_ARG;
  if (!q->codes || !q->sf || !kv->k_codes || !kv->k_sf || !kv->v_fp8 || !st->q_gscale || !st->k_gscale)
    return MPFA_ERR_INVALID_ARG;
  if (q->B <= 0 || q->H <= 0 || q->N <= 0 || kv->num_pages <= 0 || max_pages_per_req <= 0) return MPFA_ERR_INVALID_ARG;
  if (q->H != kv->H_q || kv->H_kv <= 0) return MPFA_ERR_INVALID_ARG;
  if (!(softmax_scale > 0.0f) || !(v_scale > 0.0f)) return MPFA_ERR_INVALID_ARG;
  if (kv->page_size != 64 || q->H % kv->H_kv != 0 || q->H / kv->H_kv > 8) return MPFA_ERR_UNSUPPORTED;
  if (!aligned(q->codes, 1024) || !aligned(q->sf, 1024) || !aligned(kv->k_codes, 256) || !aligned(kv->k_sf, 256) ||
      !aligned(kv->v_fp8, 256) || !aligned(kv->delta_s_bf16, 256) || !aligned(out_bf16, 16) || !aligned(out_f32, 16))
    return MPFA_ERR_ALIGNMENT;
  const int nq_tiles = pad128(q->N) / TILE;
  const uint64_t q_rows = (uint64_t)q->B * q->H * nq_tiles * TILE;
  if (q_rows >= (1ull << 31)) return MPFA_ERR_UNSUPPORTED;
  const uint64_t n_cta = (uint64_t)q->B * q->H * nq_tiles;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  PrefillParams p;
  p.q_sf = q->sf;
  p.k_sf = nullptr;
  p.delta = static_cast<const __nv_bfloat16 *>(kv->delta_s_bf16);   // the kernel only tests it against null
  p.q_gscale = st->q_gscale;
  p.k_gscale = st->k_gscale;
  p.out = static_cast<__nv_bfloat16 *>(out_bf16);
  p.out_f32 = out_f32;
  p.status = device_status;
  p.B = q->B;
  p.N_q = q->N;
  p.N_kv = 0;
  p.H_q = q->H;
  p.H_kv = kv->H_kv;
  p.nq_tiles = nq_tiles;
  p.nk_tiles = 0;
  p.causal = 1;
  p.softmax_scale = softmax_scale;
  p.v_scale = v_scale;
  p.n_items = (int)n_cta;
  PagedSrc pg;
  pg.k_codes = kv->k_codes;
  pg.k_sf = kv->k_sf;
  pg.v_fp8 = kv->v_fp8;
  pg.delta = static_cast<const __nv_bfloat16 *>(kv->delta_s_bf16);
  pg.page_table = page_table;
  pg.seq_lens = seq_lens;
  pg.q_lens = q_lens;
  pg.max_pages = max_pages_per_req;
  pg.num_pages = kv->num_pages;
  if (g_arrangement == 1) return launch_prefill_pair_paged(q, p, pg, static_cast<cudaStream_t>(stream));
  EncodeTiledFn enc;
  rc = get_encoder(&enc);
  if (rc != MPFA_OK) return rc;
  CUtensorMap tq;
  if ((rc = make_map(enc, &tq, q->codes, q_rows, 64)) != MPFA_OK) return rc;
  int dev = 0, n_sm = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  MPFA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  const unsigned grid = (unsigned)(n_cta < (uint64_t)n_sm ? n_cta : (uint64_t)n_sm);
  MPFA_CUDA_OK(cudaFuncSetAttribute(prefill_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Lay<0>::SMEM_BYTES_PAGED));
  prefill_kernel<true, false><<<grid, NTHREADS, Lay<0>::SMEM_BYTES_PAGED, static_cast<cudaStream_t>(stream)>>>(tq, tq, tq, p, pg);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}
