// QK4PV8 prefill (Algorithm 1 lines 6-20) for sm_100a, two query tiles per CTA (the arrangement of Section 5.1:
// two query stages r = 0, 1, each with its own softmax warpgroup and its own output accumulator).
//
// A work item is a PAIR of adjacent 128-row query tiles of one q head; stage 1 is the later tile.  Every KV block
// (128 keys, visited from the last visible block down to block 0, Section 4.1) is loaded once and used by both
// stages.  One persistent CTA per SM walks a static, length-sorted list of items and keeps its pipeline running
// across item boundaries.  Roles (512 threads):
//   warp 0       producer: Q tiles + their scale factors, K codes (tensor map, 64B swizzle), K scale factors and
//                Delta_S (bulk copies), V (tensor map, 128B swizzle); rings of 4 (K) and 3 (V) stages.  Paged
//                source (template parameter PAGED): every tile half is a bulk copy of a 64-token page slab;
//   warp 2       paged source only: re-tiles the pages' row-major K scales for tcgen05.cp and un-swizzles their
//                Delta_S rows (idle otherwise; it also owns the tensor-memory allocation);
//   warp 1       Q K^T issuer: per (block, stage) a rank-one BF16 MMA seeds S with 1 x Delta_S (Eq. 11) and two
//                block-scaled FP4 MMAs (K = 64 each) accumulate Q_r K^T into the one score buffer, which the two
//                stages use alternately;
//   warp 3       P V issuer: four FP8 MMAs per (block, stage), A = P_hat_r from tensor memory, B = V from shared
//                memory (MN-major), into O_r;
//   warps 4-7    softmax of stage 0, warps 8-11 softmax of stage 1.  One thread per query row; the row's running
//                maximum and sum never leave the thread (no exchange between the groups).  Per block: the 128
//                scores into registers (the buffer goes back to the MMA warp at once), mask, row maximum,
//                alpha = 2^(lam (m_old - m_new)) published for the correction warps, P = 2^(lam S - lam m) with
//                the factor 448 of the E4M3 operand folded into the exponent, row sum of the unquantized values,
//                P -> E4M3 into the stage's own 32 tensor-memory columns (Algorithm 1 lines 11-14);
//   warps 12-15  correction + epilogue: O_r *= alpha before the block's P V whenever some row's maximum moved
//                (Eq. 6), and at the end of an item O_r / (448 l) * v_scale -> BF16 (Algorithm 1 line 17).
// Tensor memory (496 of 512 columns): S [0,128), O_0 [128,256), O_1 [256,384), P_hat_0 [384,416), P_hat_1 [416,448),
// scale factors of 2 x 2 query tiles [448,480) and of two K blocks [480,496).
// Measured on B200 against the one-query-tile kernel of prefill.cu (same arithmetic row by row): 1264 against 1338
// TFLOPS at 16K, 1354 against 1445 at 64K (0.94x), although this kernel executes 12 % fewer instructions per
// block.  Before P-hat was handed to the P V issuer late (at the top of the stage's next block instead of after its
// tensor-memory stores) it stood at 1105 / 1188: with one accumulator per tile the rescale of O sits between two
// dependent P V MMAs of that tile (the other kernel alternates two accumulators), and at these lengths some row of a
// warp moves its maximum in most blocks; with the rescaling compiled out both kernels take the same time.  This
// arrangement is therefore not the default (mpfa_set_prefill_arrangement).
// Template parameter EW: the compensation-placement ablation (no seed MMA, Delta_S added element by element by the
// softmax threads).  Every mbarrier wait is bounded; on expiry the CTA raises MPFA_DEV_TIMEOUT in *device_status,
// all roles leave their loops, outstanding TMA copies are drained and tensor memory is released.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "prefill_common.cuh"

namespace mpfa {
namespace {

namespace pair {

// Optional timeline capture for tuning (compiled in only with -DMPFA_TRACE): one CTA records clock64() at fixed
// points of every role, [role][index of the stage's block][event].
#ifdef MPFA_TRACE
__device__ long long *g_ptrace = nullptr;
__device__ int g_ptrace_cta = 0;
#define TR_INIT() long long *tr_buf = ((int)blockIdx.x == g_ptrace_cta && lane == 0) ? g_ptrace : nullptr
#define TR(role, t, ev)                                                              \
  do {                                                                               \
    if (tr_buf && (t) < 512) tr_buf[((role) * 512 + (t)) * 8 + (ev)] = clock64();    \
  } while (0)
#else
#define TR_INIT() do {} while (0)
#define TR(role, t, ev) do {} while (0)
#endif

constexpr int KSTAGES = 4;
constexpr int VSTAGES = 3;
constexpr int NTHREADS = 512;
constexpr int REGS_SOFTMAX = 168;
#ifndef MPFA_PAIR_LATE
#define MPFA_PAIR_LATE 1
#endif
#ifndef MPFA_PAIR_REGS_UTIL
#define MPFA_PAIR_REGS_UTIL 56   // measured for this kernel: 56/120 1264 / 1354, 72/104 1245 / 1318, 80/96 1228 / 1288
#define MPFA_PAIR_REGS_CORR 120
#endif
template <bool PAGED> constexpr int REGS_UTIL = PAGED ? 64 : MPFA_PAIR_REGS_UTIL;
template <bool PAGED> constexpr int REGS_CORR = PAGED ? 112 : MPFA_PAIR_REGS_CORR;
// setmaxnreg only moves registers inside the pool the CTA got at launch (512 threads x 128 registers); a request
// beyond the pool would block forever, and a "dec" to more than 128 or an "inc" to less is an illegal instruction.
static_assert(4 * REGS_UTIL<false> + 8 * REGS_SOFTMAX + 4 * REGS_CORR<false> <= 16 * 128, "register pool");
static_assert(4 * REGS_UTIL<true> + 8 * REGS_SOFTMAX + 4 * REGS_CORR<true> <= 16 * 128, "register pool");
static_assert(REGS_UTIL<false> <= 128 && REGS_UTIL<true> <= 128 && REGS_CORR<false> <= 128 && REGS_CORR<true> <= 128 &&
              REGS_SOFTMAX >= 128 && REGS_SOFTMAX <= 255 && REGS_SOFTMAX % 8 == 0, "setmaxnreg direction");

constexpr uint32_t OFF_Q = 0;                                 // [item & 1][stage] x 8192
constexpr uint32_t OFF_K = OFF_Q + 4 * 8192;
constexpr uint32_t OFF_V = OFF_K + KSTAGES * 8192;
constexpr uint32_t OFF_DELTA = OFF_V + VSTAGES * 16384;
constexpr uint32_t OFF_ONES = OFF_DELTA + KSTAGES * 4096;
constexpr uint32_t OFF_SFQ = OFF_ONES + 4096;                 // [item & 1][stage] x 1024
constexpr uint32_t OFF_SFK = OFF_SFQ + 4 * 1024;
constexpr uint32_t OFF_ALPHA = OFF_SFK + KSTAGES * 1024;      // alpha[stage][block & 1][128]
constexpr uint32_t OFF_L = OFF_ALPHA + 2 * 2 * 128 * 4;       // row sums l[stage][use & 3][128]
constexpr uint32_t OFF_BAR = OFF_L + 2 * 4 * 128 * 4;
enum {
  BAR_Q_FULL = 0,                       // [2] query tiles of the item in buffer (item & 1)
  BAR_Q_EMPTY = 2,                      // [2] every Q K^T MMA of that item has completed
  BAR_K_FULL = 4,
  BAR_K_EMPTY = BAR_K_FULL + KSTAGES,
  BAR_V_FULL = BAR_K_EMPTY + KSTAGES,
  BAR_V_EMPTY = BAR_V_FULL + VSTAGES,
  BAR_S_FULL = BAR_V_EMPTY + VSTAGES,   // [2] scores of the stage's next block are in the score buffer
  BAR_S_EMPTY = BAR_S_FULL + 2,         // the scores have been read into registers (uses of the buffer alternate)
  BAR_A_FULL = BAR_S_EMPTY + 1,         // [2][2] alpha of the stage's n-th block published, barrier n & 1.  Two
                                        //     barriers per stage, as for O_READY: the producer can finish block n+1
                                        //     before the consumer has looked at block n (it only needs P V of block
                                        //     n-1), and a barrier that is two phases ahead of its waiter is lost
  BAR_P_FULL = BAR_A_FULL + 4,          // [2] P_hat of the stage's block written
  BAR_P_EMPTY = BAR_P_FULL + 2,         // [2] P V has consumed it
  BAR_O_FULL = BAR_P_EMPTY + 2,         // [2] P V of the stage's block accumulated into O_r
  BAR_O_READY = BAR_O_FULL + 2,         // [2][2] O_r rescaled for the stage's n-th block, barrier n & 1
  BAR_L_FULL = BAR_O_READY + 4,         // [2][4] row sums of the stage's u-th item, slot u & 3
  BAR_O_FREE = BAR_L_FULL + 8,          // [2] the epilogue has read O_r
  BAR_SF_READY = BAR_O_FREE + 2,        // [KSTAGES] paged source only: scales and Delta_S of the stage re-tiled
  NUM_BARS = BAR_SF_READY + KSTAGES
};
constexpr uint32_t OFF_MISC = OFF_BAR + NUM_BARS * 8;   // tmem base, abort flag
constexpr uint32_t RAW_STAGE = 1280;                    // paged source: 2 x 512 scale bytes + 2 x 128 Delta_S bytes
constexpr uint32_t OFF_RAW = (OFF_MISC + 16 + 127) & ~127u;
constexpr uint32_t SMEM_BYTES = OFF_MISC + 16 + 1024;   // + slack for the 1024-byte alignment
constexpr uint32_t SMEM_BYTES_PAGED = OFF_RAW + KSTAGES * RAW_STAGE + 1024;

constexpr uint32_t TM_S = 0, TM_O = 128 /* + 128 r */, TM_P = 384 /* + 32 r */, TM_SFQ = 448 /* + 8 (2 qb + r) */,
                   TM_SFK = 480 /* + 8 (block & 1) */;
constexpr uint32_t TMEM_COLS = 512;

// One work item: two adjacent query tiles of one q head.  T[r] = KV blocks stage r visits (0: the tile is absent
// or sees no key); both stages walk the blocks Tmax-1 .. 0, stage r joins at block T[r]-1.
struct Item {
  int b, hq, hk;
  int tile[2], T[2];
  bool present[2];
  int Tmax, nkv, nq;
};

// The list of work items of this CTA: ordered by length (latest tile pair first; all heads of a pair adjacent, so
// the G heads of a kv head stream the same K/V through L2 together) and dealt to the CTAs boustrophedon.
struct Walk {
  int round;
  __device__ __forceinline__ void init() { round = 0; }
  template <bool PAGED>
  __device__ __forceinline__ bool next(const PrefillParams &pp, const PagedSrc &pg, Item &t) {
    const int c = (round & 1) ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x;
    const int i = round * (int)gridDim.x + c;
    ++round;
    if (i >= pp.n_items) return false;
    const int n_heads = pp.B * pp.H_q;
    const int hi = pp.nq_tiles - 1 - 2 * (i / n_heads);
    const int h = i % n_heads;
    t.b = h / pp.H_q;
    t.hq = h % pp.H_q;
    t.hk = t.hq / (pp.H_q / pp.H_kv);
    const int n_q = (PAGED && pg.q_lens) ? min(pg.q_lens[t.b], pp.N_q) : pp.N_q;
    // a length beyond what the page-table row can address is cut to it (no read past the row)
    const int n_kv = PAGED ? min(pg.seq_lens[t.b], pg.max_pages * 64) : pp.N_kv;
    t.nkv = n_kv;
    t.nq = n_q;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int tile = hi - 1 + r;
      t.tile[r] = tile;
      t.present[r] = tile >= 0;
      const int row0 = tile * TILE;
      const int last_row = min(n_q - 1, row0 + TILE - 1);
      const int last_key = pp.causal ? min(n_kv - 1, last_row + (n_kv - n_q)) : n_kv - 1;   // bottom-right aligned
      t.T[r] = (tile < 0 || last_key < 0 || row0 >= n_q) ? 0 : last_key / TILE + 1;
    }
    t.Tmax = max(t.T[0], t.T[1]);
    return true;
  }
};

}  // namespace pair

using namespace pair;

template <bool PAGED, bool EW>
__global__ void __launch_bounds__(NTHREADS, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const PrefillParams p, const PagedSrc pg) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

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
    mbar_init(cx.bar(BAR_S_EMPTY), 4);   // one arrival per warp (lane 0 after __syncwarp)
    for (int i = 0; i < 2; ++i) {
      mbar_init(cx.bar(BAR_S_FULL + i), 1);
      mbar_init(cx.bar(BAR_A_FULL + 2 * i), 4);
      mbar_init(cx.bar(BAR_A_FULL + 2 * i + 1), 4);
      mbar_init(cx.bar(BAR_P_FULL + i), 4);
      mbar_init(cx.bar(BAR_P_EMPTY + i), 1);
      mbar_init(cx.bar(BAR_O_FULL + i), 1);
      mbar_init(cx.bar(BAR_O_READY + 2 * i), 4);
      mbar_init(cx.bar(BAR_O_READY + 2 * i + 1), 4);
      mbar_init(cx.bar(BAR_O_FREE + i), 4);
    }
    for (int i = 0; i < 8; ++i) mbar_init(cx.bar(BAR_L_FULL + i), 4);
    for (int i = 0; i < KSTAGES; ++i) mbar_init(cx.bar(BAR_SF_READY + i), 1);
    mbar_init_fence();
    prefetch_tmap(&tm_q);
    if (!PAGED) {
      prefetch_tmap(&tm_k);
      prefetch_tmap(&tm_v);
    }
  }
  // rank-one operands: MN-major, 128B swizzle, K = 16.  Row k = 0 of each 64-element half holds the data
  // (ones / Delta_S), every other row stays zero for the CTA's lifetime.
  for (int i = tid; i < (KSTAGES * 4096 + 4096) / 16; i += NTHREADS)
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

  // Every role walks the same list of items and keeps the same running counts: gb = KV blocks of the items walked
  // (slot and phase of the K and V rings), tq = items that had any block (Q buffers), n_r = blocks stage r has
  // taken (phases of the per-stage barriers), u_r = items in which stage r had blocks (row-sum ring, O_FREE).
  Walk walk;
  walk.init();
  Item it;
  uint32_t gb = 0;

  if (warp < 4) setmaxnreg_dec<REGS_UTIL<PAGED>>();
  if (warp == 0) {
    // =========================== TMA producer ===========================
    bool ok = true;
    uint32_t nk_armed = 0, nv_armed = 0, nq_armed = 0, tq = 0;
    while (ok && walk.template next<PAGED>(p, pg, it)) {
      if (it.Tmax == 0) continue;
      const uint32_t qb = tq & 1;
      if (tq >= 2) ok = cx.wait(BAR_Q_EMPTY + qb, ((tq >> 1) - 1) & 1u);
      if (!ok) break;
      const size_t q_head = ((size_t)it.b * p.H_q + it.hq);
      const size_t k_row = ((size_t)it.b * p.H_kv + it.hk) * (size_t)(p.nk_tiles * TILE);
      if (elect_one()) {
        const uint32_t bar = cx.bar(BAR_Q_FULL + qb);
        mbar_expect_tx(bar, (uint32_t)((it.T[0] > 0) + (it.T[1] > 0)) * (8192 + 1024));
#pragma unroll
        for (int r = 0; r < 2; ++r)
          if (it.T[r] > 0) {
            tma_load_2d(sbase + OFF_Q + (qb * 2 + r) * 8192, &tm_q, 0, (int)(q_head * (size_t)(p.nq_tiles * TILE) + it.tile[r] * TILE), bar);
            bulk_load(sbase + OFF_SFQ + (qb * 2 + r) * 1024, p.q_sf + (q_head * p.nq_tiles + it.tile[r]) * 1024, 1024, bar);
          }
      }
      nq_armed = tq + 1;
      PageLookup look;
      for (int t = 0; t < it.Tmax && ok; ++t) {
        const uint32_t c = gb + t;
        const int jb = it.Tmax - 1 - t;
        const uint32_t ks = c % KSTAGES, vs = c % VSTAGES;
        int page_lo = 0, page_hi = 0;
        if (PAGED) look.get(pg, p.status, it.b, it.nkv, t, jb, lane, page_lo, page_hi);
        if (c >= (uint32_t)KSTAGES) ok = cx.wait(BAR_K_EMPTY + ks, (c / KSTAGES - 1) & 1u);
        if (!ok) break;
        if (PAGED) {
          if (elect_one()) {
            const uint32_t bar = cx.bar(BAR_K_FULL + ks);
            mbar_expect_tx(bar, 8192 + 1024 + (has_delta ? 256 : 0));
            const size_t s_lo = (size_t)page_lo * p.H_kv + it.hk, s_hi = (size_t)page_hi * p.H_kv + it.hk;
            bulk_load(sbase + OFF_K + ks * 8192, pg.k_codes + s_lo * 4096, 4096, bar);
            bulk_load(sbase + OFF_K + ks * 8192 + 4096, pg.k_codes + s_hi * 4096, 4096, bar);
            bulk_load(sbase + OFF_RAW + ks * RAW_STAGE, pg.k_sf + s_lo * 512, 512, bar);
            bulk_load(sbase + OFF_RAW + ks * RAW_STAGE + 512, pg.k_sf + s_hi * 512, 512, bar);
            if (has_delta) {
              bulk_load(sbase + OFF_RAW + ks * RAW_STAGE + 1024, pg.delta + ((size_t)page_lo * p.H_q + it.hq) * 64, 128, bar);
              bulk_load(sbase + OFF_RAW + ks * RAW_STAGE + 1152, pg.delta + ((size_t)page_hi * p.H_q + it.hq) * 64, 128, bar);
            }
          }
        } else if (elect_one()) {
          const uint32_t bar = cx.bar(BAR_K_FULL + ks);
          mbar_expect_tx(bar, 8192 + 1024 + (has_delta ? 256 : 0));
          tma_load_2d(sbase + OFF_K + ks * 8192, &tm_k, 0, (int)(k_row + (size_t)jb * TILE), bar);
          bulk_load(sbase + OFF_SFK + ks * 1024, p.k_sf + (((size_t)it.b * p.H_kv + it.hk) * p.nk_tiles + jb) * 1024, 1024, bar);
          if (has_delta) {
            const __nv_bfloat16 *d = p.delta + q_head * (size_t)(p.nk_tiles * TILE) + (size_t)jb * TILE;
            bulk_load(sbase + OFF_DELTA + ks * 4096, d, 128, bar);
            bulk_load(sbase + OFF_DELTA + ks * 4096 + 2048, d + 64, 128, bar);
          }
        }
        nk_armed = c + 1;
        if (c >= (uint32_t)VSTAGES) ok = cx.wait(BAR_V_EMPTY + vs, (c / VSTAGES - 1) & 1u);
        if (!ok) break;
        if (MPFA_DROP_V(c)) {
          // test build: this copy is left out on purpose
        } else if (PAGED) {
          if (elect_one()) {
            const uint32_t bar = cx.bar(BAR_V_FULL + vs);
            mbar_expect_tx(bar, 16384);
            bulk_load(sbase + OFF_V + vs * 16384, pg.v_fp8 + ((size_t)page_lo * p.H_kv + it.hk) * 8192, 8192, bar);
            bulk_load(sbase + OFF_V + vs * 16384 + 8192, pg.v_fp8 + ((size_t)page_hi * p.H_kv + it.hk) * 8192, 8192, bar);
          }
        } else if (elect_one()) {
          mbar_expect_tx(cx.bar(BAR_V_FULL + vs), 16384);
          tma_load_2d(sbase + OFF_V + vs * 16384, &tm_v, 0, (int)(k_row + (size_t)jb * TILE), cx.bar(BAR_V_FULL + vs));
        }
        if (!MPFA_DROP_V(c)) nv_armed = c + 1;
      }
      gb += it.Tmax;
      ++tq;
    }
    if (*cx.abort_flag) {
      // Drain: copies still in flight must land before the CTA's shared memory is released.
      for (uint32_t c = nk_armed - min(nk_armed, (uint32_t)KSTAGES); c < nk_armed; ++c)
        mbar_wait_ns(cx.bar(BAR_K_FULL + c % KSTAGES), (c / KSTAGES) & 1u, WAIT_LIMIT_NS);
      for (uint32_t c = nv_armed - min(nv_armed, (uint32_t)VSTAGES); c < nv_armed; ++c)
        if (!MPFA_DROP_V(c)) mbar_wait_ns(cx.bar(BAR_V_FULL + c % VSTAGES), (c / VSTAGES) & 1u, WAIT_LIMIT_NS);
      for (uint32_t i = nq_armed - min(nq_armed, 2u); i < nq_armed; ++i)
        mbar_wait_ns(cx.bar(BAR_Q_FULL + (i & 1)), (i >> 1) & 1u, WAIT_LIMIT_NS);
    }
  } else if (warp == 1) {
    // =========================== Q K^T issuer ===========================
    // Whole warp in uniform control flow; the elected lane issues every tcgen05 instruction, so the commits track
    // the MMAs of the same thread.
    const uint32_t id_fp4 = idesc_nvfp4(128, 128);
    const uint32_t id_bf16 = idesc_bf16(128, 128, 1, 1);
    const uint64_t d_ones = smem_desc(sbase + OFF_ONES, 2048, 1024, SWZ_128B);
    const uint64_t d_delta0 = smem_desc(sbase + OFF_DELTA, 2048, 1024, SWZ_128B);
    const uint64_t d_q00 = smem_desc(sbase + OFF_Q, 16, 512, SWZ_64B);
    const uint64_t d_k0 = smem_desc(sbase + OFF_K, 16, 512, SWZ_64B);
    const uint64_t d_sfq00 = smem_desc(sbase + OFF_SFQ, 0, 128, SWZ_NONE);
    const uint64_t d_sfk0 = smem_desc(sbase + OFF_SFK, 0, 128, SWZ_NONE);
    bool ok = true;
    uint32_t tq = 0, ns = 0;   // ns: uses of the score buffer so far
    while (ok && walk.template next<PAGED>(p, pg, it)) {
      if (it.Tmax == 0) continue;
      const uint32_t qb = tq & 1;
      ok = cx.wait(BAR_Q_FULL + qb, (tq >> 1) & 1u);
      if (!ok) break;
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int r = 0; r < 2; ++r)
          if (it.T[r] > 0) {
            const uint64_t d_sfq = d_sfq00 + (uint64_t)(((qb * 2 + r) * 1024) >> 4);
            tmem_cp_32x128b_warpx4(tm + TM_SFQ + 8 * (qb * 2 + r), d_sfq);
            tmem_cp_32x128b_warpx4(tm + TM_SFQ + 8 * (qb * 2 + r) + 4, d_sfq + (512 >> 4));
          }
      }
      for (int t = 0; t < it.Tmax && ok; ++t) {
        const uint32_t c = gb + t;
        const int jb = it.Tmax - 1 - t;
        const uint32_t ks = c % KSTAGES;
        ok = cx.wait(BAR_K_FULL + ks, (c / KSTAGES) & 1u);
        if (PAGED) ok = ok && cx.wait(BAR_SF_READY + ks, (c / KSTAGES) & 1u);
        if (!ok) break;
        const uint32_t tSFK = tm + TM_SFK + 8 * (c & 1);
        const uint64_t d_sfk = d_sfk0 + (uint64_t)((ks * 1024) >> 4);
        const uint64_t d_k = d_k0 + (uint64_t)((ks * 8192) >> 4);
        const uint64_t d_delta = d_delta0 + (uint64_t)((ks * 4096) >> 4);
        tc_fence_after();
        if (elect_one()) {   // the K block's scale factors: these columns were last read by the MMAs of block c-2
          tmem_cp_32x128b_warpx4(tSFK, d_sfk);
          tmem_cp_32x128b_warpx4(tSFK + 4, d_sfk + (512 >> 4));
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          if (jb >= it.T[r]) continue;
          // the previous user of the score buffer has read its scores into registers
          TR(2, ns, 0);
          if (ns >= 1) ok = cx.wait(BAR_S_EMPTY, (ns - 1) & 1u);
          if (!ok) break;
          TR(2, ns, 1);
          tc_fence_after();
          if (elect_one()) {
            const uint64_t d_q = d_q00 + (uint64_t)(((qb * 2 + r) * 8192) >> 4);
            const uint32_t tSFQ = tm + TM_SFQ + 8 * (qb * 2 + r);
#ifdef MPFA_ABLATE_NO_QK
            if (t > 100000)
#endif
            {
              if (has_delta) mma_bf16_ss(tm + TM_S, d_ones, d_delta, id_bf16, 0);
              mma_nvfp4_ss(tm + TM_S, d_q, d_k, id_fp4, tSFQ, tSFK, has_delta ? 1u : 0u);
              mma_nvfp4_ss(tm + TM_S, d_q + (32 >> 4), d_k + (32 >> 4), id_fp4, tSFQ + 4, tSFK + 4, 1u);
            }
            mma_commit(cx.bar(BAR_S_FULL + r));
          }
          TR(2, ns, 2);
          ++ns;
        }
        if (!ok) break;
        if (elect_one()) mma_commit(cx.bar(BAR_K_EMPTY + ks));
      }
      if (ok && elect_one()) mma_commit(cx.bar(BAR_Q_EMPTY + qb));   // after every MMA that reads these query tiles
      __syncwarp();
      gb += it.Tmax;
      ++tq;
    }
  } else if (PAGED && warp == 2) {
    // ==== paged source: re-tile the K scales and un-swizzle Delta_S of every stage ====
    const int G = p.H_q / p.H_kv;
    bool ok = true;
    while (ok && walk.template next<PAGED>(p, pg, it)) {
      const int rsw = it.hq % G;
      for (int t = 0; t < it.Tmax && ok; ++t) {
        const uint32_t c = gb + t;
        const uint32_t ks = c % KSTAGES;
        ok = cx.wait(BAR_K_FULL + ks, (c / KSTAGES) & 1u);
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
      gb += it.Tmax;
    }
  } else if (warp == 3) {
    // =========================== P V issuer ===========================
    const uint32_t id_fp8 = idesc_e4m3(128, 128, 0, 1);
    const uint64_t d_v0 = smem_desc(sbase + OFF_V, 16, 1024, SWZ_128B);
    bool ok = true;
    uint32_t n0 = 0, n1 = 0, u0 = 0, u1 = 0;
    while (ok && walk.template next<PAGED>(p, pg, it)) {
      if (it.Tmax == 0) continue;
      for (int t = 0; t < it.Tmax && ok; ++t) {
        const uint32_t c = gb + t;
        const int jb = it.Tmax - 1 - t;
        const uint32_t vs = c % VSTAGES;
        ok = cx.wait(BAR_V_FULL + vs, (c / VSTAGES) & 1u);
        if (!ok) break;
        const uint64_t d_v = d_v0 + (uint64_t)((vs * 16384) >> 4);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          if (jb >= it.T[r]) continue;
          const uint32_t n = r ? n1 : n0, u = r ? u1 : u0;
          const bool first = jb == it.T[r] - 1;
          // the epilogue of the stage's previous item has read the accumulator that this block overwrites
          TR(3 + r, n, 0);
          if (first && u >= 1) ok = cx.wait(BAR_O_FREE + r, (u - 1) & 1u);
          ok = ok && cx.wait(BAR_O_READY + 2 * r + (n & 1), (n >> 1) & 1u);
          TR(3 + r, n, 1);
          ok = ok && cx.wait(BAR_P_FULL + r, n & 1u);
          TR(3 + r, n, 2);
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4)
#ifdef MPFA_ABLATE_NO_PV
              if (k4 > 100)
#endif
              mma_e4m3_ts(tm + TM_O + 128 * r, tm + TM_P + 32 * r + 8 * k4, d_v + (uint64_t)((4096 * k4) >> 4), id_fp8,
                          (!first || k4 > 0) ? 1u : 0u);
            mma_commit(cx.bar(BAR_O_FULL + r));
            mma_commit(cx.bar(BAR_P_EMPTY + r));
          }
          TR(3 + r, n, 3);
          if (r) ++n1; else ++n0;
        }
        if (!ok) break;
        if (elect_one()) mma_commit(cx.bar(BAR_V_EMPTY + vs));
        __syncwarp();
      }
      if (it.T[0] > 0) ++u0;
      if (it.T[1] > 0) ++u1;
      gb += it.Tmax;
    }
  } else if (warp >= 4 && warp < 12) {
    // =========================== softmax groups ===========================
    setmaxnreg_inc<REGS_SOFTMAX>();
    const int r = (warp - 4) >> 2;                   // stage = query tile of the pair
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    float *s_alpha = reinterpret_cast<float *>(smem + OFF_ALPHA) + r * 256;
    float *s_l = reinterpret_cast<float *>(smem + OFF_L) + r * 512;
    const uint32_t tS = tm + TM_S + lane_off;
    const uint32_t tP = tm + TM_P + 32 * r + lane_off;
    bool ok = true;
    uint32_t n = 0, u = 0;   // blocks / items this stage has taken
    while (ok && walk.template next<PAGED>(p, pg, it)) {
      const int T = it.T[r];
      if (T == 0) continue;
      const int r_abs = it.tile[r] * TILE + row;
      const int limit = (r_abs >= it.nq) ? -1   // a row past the request's own query count sees nothing
                        : p.causal ? min(it.nkv - 1, r_abs + (it.nkv - it.nq)) : it.nkv - 1;   // last visible key
      const float lam = __fmul_rn(__fmul_rn(__fmul_rn(p.softmax_scale, 1.4426950408889634f), p.q_gscale[it.b]), p.k_gscale[it.b]);
#if MPFA_PAIR_LATE
      bool p_pending = false;
#endif
      float m_run = -INFINITY;   // running maximum (Eq. 3)
      float l_run = 0.0f;        // running sum of 448 P (Eq. 5)
      for (int jb = T - 1; jb >= 0; --jb, ++n) {
        const int key0 = jb * TILE;
        TR(r, n, 0);
#if MPFA_PAIR_LATE == 2
        if (p_pending) {
          tmem_st_wait();
          tc_fence_before();
          warp_arrive(cx.bar(BAR_P_FULL + r), lane);
          p_pending = false;
        }
#endif
        if (!__all_sync(0xffffffffu, cx.wait(BAR_S_FULL + r, n & 1u))) { ok = false; break; }
        TR(r, n, 1);
        tc_fence_after();
        uint32_t s[128];
        {
          uint32_t(&s0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
          uint32_t(&s1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
          tmem_ld32(tS, s0);
          tmem_ld32(tS + 32, s1);
        }
#if MPFA_PAIR_LATE == 1
        if (p_pending) {
          tmem_st_wait();
          tc_fence_before();
          warp_arrive(cx.bar(BAR_P_FULL + r), lane);
          p_pending = false;
        }
#endif
        // P V of the stage's previous block has consumed the P_hat columns (tested early, used before the stores)
        const bool pe_early = (n < 1) || cx.probe(BAR_P_EMPTY + r, (n - 1) & 1u);
        const bool ragged = key0 + TILE - 1 > limit;   // diagonal / ragged block only
        tmem_ld_wait();
        {
          // second half of the row in flight while the maximum of the first half is taken
          uint32_t(&s2)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[64]);
          uint32_t(&s3)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[96]);
          tmem_ld32(tS + 64, s2);
          tmem_ld32(tS + 96, s3);
        }
#if MPFA_PAIR_LATE == 3
        if (p_pending) {
          tmem_st_wait();
          tc_fence_before();
          warp_arrive(cx.bar(BAR_P_FULL + r), lane);
          p_pending = false;
        }
#endif
        if constexpr (EW) {
          const uint4 *dp = reinterpret_cast<const uint4 *>(
              p.delta + ((size_t)it.b * p.H_q + it.hq) * (size_t)(p.nk_tiles * TILE) + key0);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint4 d = __ldg(dp + i);
            const uint32_t w[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              s[8 * i + 2 * j] = __float_as_uint(__fadd_rn(__uint_as_float(s[8 * i + 2 * j]), __uint_as_float(w[j] << 16)));
              s[8 * i + 2 * j + 1] =
                  __float_as_uint(__fadd_rn(__uint_as_float(s[8 * i + 2 * j + 1]), __uint_as_float(w[j] & 0xFFFF0000u)));
            }
          }
        }
        if (ragged) {
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (key0 + i > limit) s[i] = 0xFF800000u;   // -inf
        }
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
        warp_arrive(cx.bar(BAR_S_EMPTY), lane);   // the row is in registers: the other stage's Q K^T may overwrite it
        TR(r, n, 2);
        if constexpr (EW) {
          const uint4 *dp = reinterpret_cast<const uint4 *>(
              p.delta + ((size_t)it.b * p.H_q + it.hq) * (size_t)(p.nk_tiles * TILE) + key0 + 64);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const uint4 d = __ldg(dp + i);
            const uint32_t w[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              s[64 + 8 * i + 2 * j] =
                  __float_as_uint(__fadd_rn(__uint_as_float(s[64 + 8 * i + 2 * j]), __uint_as_float(w[j] << 16)));
              s[64 + 8 * i + 2 * j + 1] =
                  __float_as_uint(__fadd_rn(__uint_as_float(s[64 + 8 * i + 2 * j + 1]), __uint_as_float(w[j] & 0xFFFF0000u)));
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
        const float m_new = fmaxf(m_run, mx);
        // alpha = 2^(lam (m_old - m_new)) (Eq. 5/6): 1 when the maximum did not move, 0 for the row's first block
        const float alpha = (m_new == m_run) ? 1.0f : ex2_approx(__fmul_rn(m_run - m_new, lam));
        s_alpha[(n & 1) * 128 + row] = alpha;
        warp_arrive(cx.bar(BAR_A_FULL + 2 * r + (n & 1)), lane);
        TR(r, n, 3);
        m_run = m_new;
        // q = 448 P = 2^(lam S - lam m + log2 448) is the E4M3 operand (Section 4.1); the row sum is taken over q
        // and the factor 448 is divided out once in the epilogue.
        const float cc = (m_new == -INFINITY) ? 0.0f : __fsub_rn(8.8073549220576042f, __fmul_rn(m_new, lam));
        if (!__all_sync(0xffffffffu, pe_early)) {
          if (!__all_sync(0xffffffffu, cx.wait(BAR_P_EMPTY + r, (n - 1) & 1u))) { ok = false; break; }
        }
        TR(r, n, 4);
        float sum0 = 0.0f, sum1 = 0.0f, sum2 = 0.0f, sum3 = 0.0f;
#ifdef MPFA_ABLATE_NO_EXP
#define EX2_(x) (x)
#else
#define EX2_(x) ex2_approx(x)
#endif
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 32) {
          uint32_t packed[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float x0, x1, x2, x3;
            fma2(x0, x1, __uint_as_float(s[c0 + 4 * i]), __uint_as_float(s[c0 + 4 * i + 1]), lam, cc);
            fma2(x2, x3, __uint_as_float(s[c0 + 4 * i + 2]), __uint_as_float(s[c0 + 4 * i + 3]), lam, cc);
            const float q0 = EX2_(x0), q1 = EX2_(x1), q2 = EX2_(x2), q3 = EX2_(x3);
            acc2(sum0, sum1, q0, q1);
            acc2(sum2, sum3, q2, q3);
            // two conversions written into the halves of one register (no separate merge instruction)
            asm("{.reg .b16 lo, hi;\n\t"
                "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
                "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
                "mov.b32 %0, {lo, hi};}"
                : "=r"(packed[i])
                : "f"(q0), "f"(q1), "f"(q2), "f"(q3));
          }
          tmem_st8(tP + (c0 >> 2), packed);
        }
        l_run = __fadd_rn(__fmul_rn(alpha, l_run), (sum0 + sum1) + (sum2 + sum3));
#if MPFA_PAIR_LATE
        p_pending = true;
#else
        tmem_st_wait();
        TR(r, n, 5);
        tc_fence_before();
        warp_arrive(cx.bar(BAR_P_FULL + r), lane);
#endif
        TR(r, n, 6);
      }
#if MPFA_PAIR_LATE
      if (p_pending) {
        tmem_st_wait();
        tc_fence_before();
        warp_arrive(cx.bar(BAR_P_FULL + r), lane);
        p_pending = false;
      }
#endif
      if (!ok) break;
      s_l[(u & 3) * 128 + row] = l_run;
      warp_arrive(cx.bar(BAR_L_FULL + r * 4 + (u & 3)), lane);
      ++u;
    }
  } else if (warp >= 12) {
    // =========================== correction + epilogue ===========================
    setmaxnreg_dec<REGS_CORR<PAGED>>();
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const float *s_alpha = reinterpret_cast<const float *>(smem + OFF_ALPHA);
    const float *s_l = reinterpret_cast<const float *>(smem + OFF_L);
    bool ok = true;
    uint32_t n0 = 0, n1 = 0, u0 = 0, u1 = 0;
    while (walk.template next<PAGED>(p, pg, it)) {
      for (int t = 0; ok && t < it.Tmax; ++t) {
        const int jb = it.Tmax - 1 - t;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          if (jb >= it.T[r] || !ok) continue;
          const uint32_t n = r ? n1 : n0;
          TR(5 + r, n, 0);
          ok = __all_sync(0xffffffffu, cx.wait(BAR_A_FULL + 2 * r + (n & 1), (n >> 1) & 1u));
          if (!ok) break;
          TR(5 + r, n, 1);
          const float alpha = s_alpha[r * 256 + (n & 1) * 128 + row];
          if (jb != it.T[r] - 1) {
            // O_r holds the stage's earlier blocks relative to the previous maximum (Eq. 6)
#ifdef MPFA_ABLATE_NO_CORR
            if (false) {
#else
            if (__any_sync(0xffffffffu, alpha != 1.0f)) {   // identical result when every factor is exactly 1
#endif
              ok = __all_sync(0xffffffffu, cx.wait(BAR_O_FULL + r, (n - 1) & 1u));
              if (!ok) break;
              TR(5 + r, n, 2);
              tc_fence_after();
              const uint32_t tO = tm + TM_O + 128 * r + lane_off;
#pragma unroll
              for (int c0 = 0; c0 < HEAD_DIM; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tO + c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; i += 2) {   // packed pairs: half the issue slots, same roundings
                  float y0, y1;
                  mul2(y0, y1, __uint_as_float(v[i]), __uint_as_float(v[i + 1]), alpha);
                  v[i] = __float_as_uint(y0), v[i + 1] = __float_as_uint(y1);
                }
                tmem_st32(tO + c0, v);
              }
              tmem_st_wait();
              tc_fence_before();
            }
          }
          warp_arrive(cx.bar(BAR_O_READY + 2 * r + (n & 1)), lane);
          TR(5 + r, n, 3);
          if (r) ++n1; else ++n0;
        }
      }
      // final normalisation (Algorithm 1 line 17): O / (448 l) * v_scale -> BF16, one tile after the other
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        if (!it.present[r]) continue;
        const int T = it.T[r];
        const uint32_t n = r ? n1 : n0, u = r ? u1 : u0;
        const int r_abs = it.tile[r] * TILE + row;
        float l = 0.0f;
        if (ok && T > 0) {
          ok = cx.wait(BAR_O_FULL + r, (n - 1) & 1u);
          ok = ok && cx.wait(BAR_L_FULL + r * 4 + (u & 3), (u >> 2) & 1u);
          tc_fence_after();
          if (ok) l = s_l[r * 512 + (u & 3) * 128 + row];
        }
        // tcgen05.ld is warp-collective: every lane loads, only the stores are predicated.
        const bool warp_ok = __all_sync(0xffffffffu, ok);
        const bool store = r_abs < p.N_q && (warp_ok || T == 0);
        const size_t o_off = (((size_t)it.b * p.N_q + (store ? r_abs : 0)) * p.H_q + it.hq) * HEAD_DIM;
        // one IEEE reciprocal per row; l already carries the factor 448
        const float inv_denom = (l > 0.0f) ? __frcp_rn(l) : 0.0f;
        const uint32_t tO = tm + TM_O + 128 * r + lane_off;
#pragma unroll 1
        for (int c0 = 0; c0 < HEAD_DIM; c0 += 32) {
          uint32_t v[32];
          if (T > 0 && warp_ok) {
            tmem_ld32(tO + c0, v);
            tmem_ld_wait();
          }
          if (c0 == HEAD_DIM - 32 && T > 0) {   // the accumulator is in registers: the next item's P V may overwrite it
            tc_fence_before();
            warp_arrive(cx.bar(BAR_O_FREE + r), lane);
          }
#pragma unroll
          for (int i = 0; i < 32; ++i)
            v[i] = (l > 0.0f) ? __float_as_uint(__fmul_rn(__fmul_rn(__uint_as_float(v[i]), inv_denom), p.v_scale)) : 0u;
          if (store) {
            if (p.out_f32) {
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                *reinterpret_cast<uint4 *>(p.out_f32 + o_off + c0 + i) = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            }
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint32_t h[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                __nv_bfloat162 w = __floats2bfloat162_rn(__uint_as_float(v[i + 2 * j]), __uint_as_float(v[i + 2 * j + 1]));
                h[j] = *reinterpret_cast<uint32_t *>(&w);
              }
              *reinterpret_cast<uint4 *>(p.out + o_off + c0 + i) = make_uint4(h[0], h[1], h[2], h[3]);
            }
          }
        }
        if (T > 0) { if (r) ++u1; else ++u0; }
      }
      if (!ok) break;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) tmem_dealloc(tm, TMEM_COLS);
}

}  // namespace
}  // namespace mpfa

using namespace mpfa;

#ifdef MPFA_TRACE
extern "C" int mpfa_debug_set_pair_trace(long long *buf, int cta) {
  if (cudaMemcpyToSymbol(pair::g_ptrace, &buf, sizeof(buf)) != cudaSuccess) return -1;
  if (cudaMemcpyToSymbol(pair::g_ptrace_cta, &cta, sizeof(cta)) != cudaSuccess) return -1;
  return 0;
}
#endif

// Launchers used by the entry points in prefill.cu.
namespace mpfa {

mpfa_status launch_prefill_pair(const mpfa_fp4_tensor *q, const mpfa_fp4_tensor *k, const uint8_t *v_fp8,
                                const PrefillParams &p0, bool ew, cudaStream_t stream) {
  EncodeTiledFn enc;
  mpfa_status rc = get_encoder(&enc);
  if (rc != MPFA_OK) return rc;
  PrefillParams p = p0;
  const uint64_t q_rows = (uint64_t)q->B * q->H * p.nq_tiles * TILE, k_rows = (uint64_t)k->B * k->H * p.nk_tiles * TILE;
  CUtensorMap tq, tk, tv;
  if ((rc = make_map(enc, &tq, q->codes, q_rows, 64)) != MPFA_OK) return rc;
  if ((rc = make_map(enc, &tk, k->codes, k_rows, 64)) != MPFA_OK) return rc;
  if ((rc = make_map(enc, &tv, v_fp8, k_rows, 128)) != MPFA_OK) return rc;
  const uint64_t n_items = (uint64_t)q->B * q->H * ((p.nq_tiles + 1) / 2);
  p.n_items = (int)n_items;
  int dev = 0, n_sm = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  MPFA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  const unsigned grid = (unsigned)(n_items < (uint64_t)n_sm ? n_items : (uint64_t)n_sm);   // one persistent CTA per SM
  if (ew) {
    MPFA_CUDA_OK(cudaFuncSetAttribute(prefill_pair_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    prefill_pair_kernel<false, true><<<grid, NTHREADS, SMEM_BYTES, stream>>>(tq, tk, tv, p, PagedSrc{});
  } else {
    MPFA_CUDA_OK(cudaFuncSetAttribute(prefill_pair_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    prefill_pair_kernel<false, false><<<grid, NTHREADS, SMEM_BYTES, stream>>>(tq, tk, tv, p, PagedSrc{});
  }
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

mpfa_status launch_prefill_pair_paged(const mpfa_fp4_tensor *q, const PrefillParams &p0, const PagedSrc &pg,
                                      cudaStream_t stream) {
  EncodeTiledFn enc;
  mpfa_status rc = get_encoder(&enc);
  if (rc != MPFA_OK) return rc;
  PrefillParams p = p0;
  const uint64_t q_rows = (uint64_t)q->B * q->H * p.nq_tiles * TILE;
  CUtensorMap tq;
  if ((rc = make_map(enc, &tq, q->codes, q_rows, 64)) != MPFA_OK) return rc;
  const uint64_t n_items = (uint64_t)q->B * q->H * ((p.nq_tiles + 1) / 2);
  p.n_items = (int)n_items;
  int dev = 0, n_sm = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  MPFA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  const unsigned grid = (unsigned)(n_items < (uint64_t)n_sm ? n_items : (uint64_t)n_sm);
  MPFA_CUDA_OK(cudaFuncSetAttribute(prefill_pair_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES_PAGED));
  prefill_pair_kernel<true, false><<<grid, NTHREADS, SMEM_BYTES_PAGED, stream>>>(tq, tq, tq, p, pg);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

}  // namespace mpfa
