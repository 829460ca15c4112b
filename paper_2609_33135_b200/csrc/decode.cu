// QK4PV8 decode over a paged low-bit KV cache (Section 5.3) for sm_100a.
//
// The path is bound by streaming the cache from HBM (208 bytes per token and kv head plus
// Delta_S), so the kernel is a persistent streaming pipeline: one CTA per SM walks a list of
// (request, kv head, 1024-token partition) work items, and a producer warp keeps a ring of
// 128-key blocks (two 64-token pages: K codes, K scales, V, Delta_S) in flight with bulk
// asynchronous copies, across item boundaries.  The cache's physical byte order
// (include/mpfa.h) is the swizzled shared-memory image the tensor-core descriptors read, so a
// page needs one copy per tensor and no thread touches the bytes.
//
// The problem is transposed so that the long axis is the MMA's M dimension and the GQA group
// (Section 5.3 packs it into one MMA tile) is the N dimension, padded to 16:
//   S^T[key, head] = K Q^T       tcgen05.mma kind::mxf4nvf4 (E2M1 codes, UE4M3 block scales),
//                                M = 128 keys, N = 16, K = 2 x 64 channels, FP32 in TMEM;
//   softmax        one thread per key: + Delta_S (Eq. 10), running maximum of the reverse
//                  traversal (blocks 7..0 of the partition), P = 2^(lam S - lam m),
//                  P_hat = E4M3(448 P) written to shared memory as the next MMA's B operand;
//   O^T[ch, head] += V^T P_hat^T  tcgen05.mma kind::f8f6f4, M = 128 channels, N = 16,
//                                K = 4 x 32 keys, V read MN-major straight from the ring.
// When the running maximum grows, O^T is rescaled in TMEM (one row of 16 floats per thread).
// The partition state (m, l, O) goes to the workspace; a second kernel merges partitions by
// log-sum-exp (warp-shuffle maximum, partitions ascending) and writes BF16.
//
// Warps: 0 producer, 1 MMA issue (+ TMEM allocation), 2-5 softmax / rescale / partition
// write-out (TMEM lane quadrant = warp % 4), 6 rewrites the K scales of each block from
// [token][8] into the 32 x 16-byte tile tcgen05.cp expects.  Every wait is bounded.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mpfa {
namespace {

constexpr int PART_FLOATS = 130;  // m, l, O[128] per (request, q head, partition)
constexpr int MAXG = 8;
constexpr int NCOL = 16;          // MMA N: the GQA group padded to 16 columns

constexpr int D_NST = 7;          // KV ring stages, one 128-key block each
constexpr int D_NSF = 4;          // formatted K-scale tiles in flight
constexpr int D_THREADS = 224;

// one ring stage
constexpr uint32_t ST_K = 0;          // 2 pages x 4096 B of codes: 64-byte rows, 64-byte swizzle
constexpr uint32_t ST_V = 8192;       // 2 pages x 8192 B: 128-byte rows, 128-byte swizzle
constexpr uint32_t ST_SF = 24576;     // 2 pages x 512 B of K scales, [token][8]
constexpr uint32_t ST_DELTA = 25600;  // 2 pages x MAXG x 128 B of Delta_S (BF16)
constexpr uint32_t ST_BYTES = 27648;
// the rest of shared memory
constexpr uint32_t D_OFF_P = D_NST * ST_BYTES;      // 2 x 2048: P_hat^T, 16 rows of 128 keys, 128-byte swizzle
constexpr uint32_t D_OFF_Q = D_OFF_P + 4096;        // 2 x 1024: Q codes, 16 rows of 64 B, 64-byte swizzle
constexpr uint32_t D_OFF_SFQ = D_OFF_Q + 2048;      // 2 x (2 x 512): Q scales, one tile per 64 channels
constexpr uint32_t D_OFF_SFK = D_OFF_SFQ + 2048;    // D_NSF x (2 x 512): K scales
constexpr uint32_t D_OFF_BAR = D_OFF_SFK + D_NSF * 1024;
constexpr uint32_t D_OFF_X = D_OFF_BAR + 512;       // block maxima, l partial sums, TMEM address, abort flag
constexpr uint32_t D_SMEM_USED = D_OFF_X + 1024;
constexpr uint32_t D_SMEM = D_SMEM_USED + 1024;     // slack for the 1024-byte alignment of the base

// barriers (8 bytes each)
constexpr int B_FULL = 0;                    // [D_NST] stage landed (bytes)
constexpr int B_EMPTY = B_FULL + D_NST;      // [D_NST] stage consumed (MMA commit)
constexpr int B_SF_READY = B_EMPTY + D_NST;  // [D_NSF] K scales formatted
constexpr int B_SFK_FREE = B_SF_READY + D_NSF;  // [D_NSF] scale tile consumed (MMA commit)
constexpr int B_S_FULL = B_SFK_FREE + D_NSF;    // [2]
constexpr int B_S_EMPTY = B_S_FULL + 2;         // [2] 4 warps
constexpr int B_P_READY = B_S_EMPTY + 2;        // [2] 4 warps
constexpr int B_PV_DONE = B_P_READY + 2;        // [2] MMA commit
constexpr int B_Q_READY = B_PV_DONE + 2;        // [2] 4 warps
constexpr int B_O_FREE = B_Q_READY + 2;         // [1] 4 warps
constexpr int B_XCHG = B_O_FREE + 1;            // [1] 4 warps: block maxima written
constexpr int B_LX = B_XCHG + 1;                // [1] 4 warps: l partial sums written
constexpr int B_COUNT = B_LX + 1;
static_assert(B_COUNT * 8 <= 512, "barrier block");
static_assert(D_SMEM <= 232448, "shared memory");

// tensor-memory columns
constexpr uint32_t TM_S = 0;      // 2 x 16
constexpr uint32_t TM_O = 32;     // 16
constexpr uint32_t TM_SFQ = 48;   // 2 x 8
constexpr uint32_t TM_SFK = 64;   // D_NSF x 8
constexpr uint32_t TM_COLS = 128;

constexpr long long D_WAIT_CYCLES = 4000000000ll;   // about two seconds

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

#ifdef MPFA_TRACE
// clock64 stamps of CTA g_dtrace_cta: [block counter < 256][16 events]
__device__ long long *g_dtrace = nullptr;
__device__ int g_dtrace_cta = 0;
#define DTR(ev, blk)                                                                              \
  do {                                                                                            \
    if (g_dtrace && (threadIdx.x & 31) == 0 && (int)blockIdx.x == g_dtrace_cta && (blk) < 256u)   \
      g_dtrace[(blk) * 16 + (ev)] = clock64();                                                    \
  } while (0)
#else
#define DTR(ev, blk) do {} while (0)
#endif

struct DecodeParams {
  const uint8_t *q_codes;  // tile layout, N = 1: row 0 of each (b, hq) tile
  const uint8_t *q_sf;
  const uint8_t *k_codes, *k_sf, *v_fp8;
  const __nv_bfloat16 *delta;  // may be null
  const int32_t *page_table;
  const int32_t *seq_lens;
  const float *q_gscale, *k_gscale;
  float *parts;  // [B, H_q, n_split, 130]
  int32_t *status;
  int B, H_q, H_kv, max_pages, num_pages, n_split;
  float softmax_scale;
};

// The work list, walked identically by every role: items blockIdx.x, blockIdx.x + gridDim.x, ...
// in (partition fastest, kv head, request) order; partitions beyond the sequence are skipped.
struct WorkIter {
  int idx, stride, total, n_split, H_kv;
  int b, hk, sp, L, nblk;
  __device__ void init(const DecodeParams &p) {
    stride = gridDim.x;
    idx = (int)blockIdx.x - stride;
    n_split = p.n_split;
    H_kv = p.H_kv;
    total = p.B * p.H_kv * p.n_split;
  }
  __device__ bool next(const int32_t *__restrict__ seq_lens) {
    for (;;) {
      idx += stride;
      if (idx >= total) return false;
      sp = idx % n_split;
      const int r = idx / n_split;
      hk = r % H_kv;
      b = r / H_kv;
      L = seq_lens[b];
      const int rem = L - sp * DECODE_SPLIT;
      if (rem > 0) {
        nblk = (min(rem, DECODE_SPLIT) + TILE - 1) / TILE;
        return true;
      }
    }
  }
};

struct DCtx {
  uint32_t bar0;
  volatile int *abort_flag;
  int32_t *status;
  __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * (uint32_t)i; }
  // Bounded wait; a timeout (or another role's abort) ends in a status bit and `false`.
  __device__ bool wait(int i, uint32_t parity) const {
    const uint32_t a = bar(i);
    if (mbar_try_wait(a, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t n = 1;; ++n) {
      if (mbar_try_wait(a, parity)) return true;
      if ((n & 1023u) == 0u) {
        if (*abort_flag) return false;
        if (clock64() - t0 > D_WAIT_CYCLES) {
          *abort_flag = 1;
          atomicOr(status, MPFA_DEV_TIMEOUT);
          return false;
        }
      }
    }
  }
  // the same for a whole warp: every lane waits, the result is uniform
  __device__ __forceinline__ bool wait_warp(int i, uint32_t parity) const {
    return __all_sync(0xffffffffu, wait(i, parity));
  }
  __device__ __forceinline__ void warp_arrive(int i) const {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar(i));
  }
};

__global__ void __launch_bounds__(D_THREADS, 1) decode_split_kernel(const DecodeParams p) {
  extern __shared__ uint8_t dsm_raw[];
  uint8_t *dsm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dsm_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(dsm);
  float *xmax = reinterpret_cast<float *>(dsm + D_OFF_X);            // [2][4][MAXG]
  float *xl = reinterpret_cast<float *>(dsm + D_OFF_X + 256);        // [2][4][MAXG]
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(dsm + D_OFF_X + 512);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(dsm + D_OFF_X + 516);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = p.H_q / p.H_kv;
  DCtx cx{sbase + D_OFF_BAR, abort_flag, p.status};

  // ---- set-up: barriers, zeroed operand tiles (rows G..15 stay zero for good), TMEM
  if (threadIdx.x == 0) {
    for (int i = 0; i < D_NST; ++i) {
      mbar_init(cx.bar(B_FULL + i), 1);
      mbar_init(cx.bar(B_EMPTY + i), 1);
    }
    for (int i = 0; i < D_NSF; ++i) {
      mbar_init(cx.bar(B_SF_READY + i), 1);
      mbar_init(cx.bar(B_SFK_FREE + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(cx.bar(B_S_FULL + i), 1);
      mbar_init(cx.bar(B_S_EMPTY + i), 4);
      mbar_init(cx.bar(B_P_READY + i), 4);
      mbar_init(cx.bar(B_PV_DONE + i), 1);
      mbar_init(cx.bar(B_Q_READY + i), 4);
    }
    mbar_init(cx.bar(B_O_FREE), 4);
    mbar_init(cx.bar(B_XCHG), 4);
    mbar_init(cx.bar(B_LX), 4);
    mbar_init_fence();
    *abort_flag = 0;
  }
  for (uint32_t o = threadIdx.x * 16; o < 8192; o += D_THREADS * 16)   // P, Q and Q-scale tiles
    *reinterpret_cast<uint4 *>(dsm + D_OFF_P + o) = make_uint4(0u, 0u, 0u, 0u);
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), TM_COLS);
    tmem_relinquish();
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = *tmem_slot;

  if (warp == 0) {
    // ================= producer: page lookups and bulk copies
    WorkIter w;
    w.init(p);
    uint32_t it = 0;
    bool ok = true;
    const uint32_t d_bytes = p.delta ? (uint32_t)G * PAGE * 2 : 0u;
    const uint32_t page_bytes = 4096u + 8192u + 512u + d_bytes;
    while (ok && w.next(p.seq_lens)) {
      const int k_part = w.sp * DECODE_SPLIT;
      // lane l holds the two page ids of block l of this partition
      int pid0 = -1, pid1 = -1;
      bool bad = false;
      if (lane < w.nblk) {
        const int first = k_part + lane * TILE;
        const int pg = first / PAGE;
        const int32_t *row = p.page_table + (size_t)w.b * p.max_pages;
        if (pg < p.max_pages) pid0 = row[pg];
        if (pid0 < 0 || pid0 >= p.num_pages) pid0 = -1, bad = true;
        if (first + PAGE < w.L) {
          if (pg + 1 < p.max_pages) pid1 = row[pg + 1];
          if (pid1 < 0 || pid1 >= p.num_pages) pid1 = -1, bad = true;
        }
      }
      if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(p.status, MPFA_DEV_BAD_PAGE);
      for (int u = w.nblk - 1; u >= 0; --u, ++it) {
        const uint32_t st = it % D_NST;
        if (it >= (uint32_t)D_NST && !cx.wait_warp(B_EMPTY + st, ((it / D_NST) - 1) & 1)) {
          ok = false;
          break;
        }
        DTR(0, it);
        const int id0 = __shfl_sync(0xffffffffu, pid0, u), id1 = __shfl_sync(0xffffffffu, pid1, u);
        uint8_t *stage = dsm + st * ST_BYTES;
        // a page that is not there contributes P_hat = 0 times V: V must be finite, so zero it
        if (id0 < 0 || id1 < 0) {
#pragma unroll 1
          for (int half = 0; half < 2; ++half) {
            if ((half == 0 ? id0 : id1) >= 0) continue;
            for (int i = 0; i < 16; ++i)
              *reinterpret_cast<uint4 *>(stage + ST_V + half * 8192 + i * 512 + lane * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async_smem();
          __syncwarp();
        }
        if (elect_one()) {
          const uint32_t full = cx.bar(B_FULL + st);
          const uint32_t sdst = sbase + st * ST_BYTES;
          mbar_expect_tx(full, (id0 >= 0 ? page_bytes : 0u) + (id1 >= 0 ? page_bytes : 0u));
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int id = half == 0 ? id0 : id1;
            if (id < 0) continue;
            const size_t slab = (size_t)id * p.H_kv + w.hk;
            bulk_load(sdst + ST_K + half * 4096, p.k_codes + slab * 4096, 4096, full);
            bulk_load(sdst + ST_V + half * 8192, p.v_fp8 + slab * 8192, 8192, full);
            bulk_load(sdst + ST_SF + half * 512, p.k_sf + slab * 512, 512, full);
            if (d_bytes)
              bulk_load(sdst + ST_DELTA + half * 1024, p.delta + ((size_t)id * p.H_q + (size_t)w.hk * G) * PAGE, d_bytes,
                        full);
          }
        }
        __syncwarp();
      }
    }
    if (!ok) {
      // another role gave up: let the copies already issued land before shared memory goes away
      const uint32_t n = it < (uint32_t)D_NST ? it : (uint32_t)D_NST;
      for (uint32_t i = it - n; i < it; ++i) {
        const long long t0 = clock64();
        while (!mbar_try_wait(cx.bar(B_FULL + i % D_NST), (i / D_NST) & 1) && clock64() - t0 < D_WAIT_CYCLES) {
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issue: S^T = K Q^T one block ahead of O^T += V^T P_hat^T
    const uint32_t id_qk = idesc_nvfp4(128, NCOL);
    const uint32_t id_pv = idesc_e4m3(128, NCOL, 1, 0);
    WorkIter wa, wc;   // block being scored, block being accumulated
    wa.init(p);
    wc.init(p);
    bool va = wa.next(p.seq_lens), vc = wc.next(p.seq_lens);
    int ua = va ? wa.nblk - 1 : 0, uc = vc ? wc.nblk - 1 : 0;
    uint32_t ia = 0, ic = 0, ja = 0, jc = 0;   // block and item counters of the two walks
    bool ok = true;
    auto issue_qk = [&]() {
      const uint32_t st = ia % D_NST, sf = ia % D_NSF, sb = ia & 1, qs = ja & 1;
      const bool first = ua == wa.nblk - 1;
      ok = cx.wait_warp(B_FULL + st, (ia / D_NST) & 1);
      DTR(1, ia);
      ok = ok && cx.wait_warp(B_SF_READY + sf, (ia / D_NSF) & 1);
      if (ok && first) ok = cx.wait_warp(B_Q_READY + qs, (ja >> 1) & 1);
      if (ok && ia >= 2) ok = cx.wait_warp(B_S_EMPTY + sb, ((ia >> 1) - 1) & 1);
      if (!ok) return;
      DTR(2, ia);
      tc_fence_after();
      if (elect_one()) {
        const uint32_t tSFQ = tm + TM_SFQ + qs * 8, tSFK = tm + TM_SFK + sf * 8;
        if (first) {
          const uint64_t d_sfq = smem_desc(sbase + D_OFF_SFQ + qs * 1024, 0, 128, SWZ_NONE);
          tmem_cp_32x128b_warpx4(tSFQ, d_sfq);
          tmem_cp_32x128b_warpx4(tSFQ + 4, d_sfq + (512 >> 4));
        }
        const uint64_t d_sfk = smem_desc(sbase + D_OFF_SFK + sf * 1024, 0, 128, SWZ_NONE);
        tmem_cp_32x128b_warpx4(tSFK, d_sfk);
        tmem_cp_32x128b_warpx4(tSFK + 4, d_sfk + (512 >> 4));
        const uint64_t d_k = smem_desc(sbase + st * ST_BYTES + ST_K, 16, 512, SWZ_64B);
        const uint64_t d_q = smem_desc(sbase + D_OFF_Q + qs * 1024, 16, 512, SWZ_64B);
        mma_nvfp4_ss(tm + TM_S + sb * 16, d_k, d_q, id_qk, tSFK, tSFQ, 0u);
        mma_nvfp4_ss(tm + TM_S + sb * 16, d_k + (32 >> 4), d_q + (32 >> 4), id_qk, tSFK + 4, tSFQ + 4, 1u);
        mma_commit(cx.bar(B_S_FULL + sb));
        mma_commit(cx.bar(B_SFK_FREE + sf));
      }
      __syncwarp();
      DTR(3, ia);
      ++ia;
      if (--ua < 0) {
        ++ja;
        va = wa.next(p.seq_lens);
        ua = va ? wa.nblk - 1 : 0;
      }
    };
    if (va) issue_qk();
    while (ok && vc) {
      if (va) issue_qk();
      if (!ok) break;
      const uint32_t st = ic % D_NST, sb = ic & 1;
      const bool first = uc == wc.nblk - 1;
      ok = cx.wait_warp(B_P_READY + sb, (ic >> 1) & 1);
      if (ok && first && jc >= 1) ok = cx.wait_warp(B_O_FREE, (jc - 1) & 1);   // the previous item's O has been read
      if (!ok) break;
      DTR(4, ic);
      tc_fence_after();
      if (elect_one()) {
        const uint64_t d_v = smem_desc(sbase + st * ST_BYTES + ST_V, 16, 1024, SWZ_128B);
        const uint64_t d_p = smem_desc(sbase + D_OFF_P + sb * 2048, 16, 1024, SWZ_128B);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)   // 32 keys per MMA
          mma_e4m3_ss(tm + TM_O, d_v + (uint64_t)((4096 * k4) >> 4), d_p + (uint64_t)((32 * k4) >> 4), id_pv,
                      (!first || k4 > 0) ? 1u : 0u);
        mma_commit(cx.bar(B_PV_DONE + sb));
        mma_commit(cx.bar(B_EMPTY + st));
      }
      __syncwarp();
      DTR(5, ic);
      ++ic;
      if (--uc < 0) {
        ++jc;
        vc = wc.next(p.seq_lens);
        uc = vc ? wc.nblk - 1 : 0;
      }
    }
  } else if (warp == 6) {
    // ================= K scales of a block: [token][8 blocks] -> two 32 x 16-byte tiles
    // (tile h = blocks 4h..4h+3; row i holds tokens i, 32+i, 64+i, 96+i), the form tcgen05.cp spreads
    WorkIter w;
    w.init(p);
    uint32_t it = 0;
    bool ok = true;
    while (ok && w.next(p.seq_lens)) {
      for (int u = w.nblk - 1; u >= 0; --u, ++it) {
        const uint32_t st = it % D_NST, sf = it % D_NSF;
        ok = cx.wait_warp(B_FULL + st, (it / D_NST) & 1);
        if (ok && it >= (uint32_t)D_NSF) ok = cx.wait_warp(B_SFK_FREE + sf, ((it / D_NSF) - 1) & 1);
        if (!ok) break;
        const uint8_t *raw = dsm + st * ST_BYTES + ST_SF;
        uint2 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = *reinterpret_cast<const uint2 *>(raw + (q >> 1) * 512 + ((q & 1) * 32 + lane) * 8);
        uint8_t *dst = dsm + D_OFF_SFK + sf * 1024 + lane * 16;
        *reinterpret_cast<uint4 *>(dst) = make_uint4(v[0].x, v[1].x, v[2].x, v[3].x);
        *reinterpret_cast<uint4 *>(dst + 512) = make_uint4(v[0].y, v[1].y, v[2].y, v[3].y);
        fence_proxy_async_smem();
        cx.warp_arrive(B_SF_READY + sf);
        DTR(6, it);
      }
    }
  } else {
    // ================= softmax, one thread per key of the block (per channel for O^T)
    const int quad = warp & 3;                  // TMEM lane quadrant this warp may touch
    const int r = quad * 32 + lane;             // key within the block / channel of O^T
    const int t128 = (warp - 2) * 32 + lane;    // 0..127 among these warps
    const uint32_t tlane = (uint32_t)(quad * 32) << 16;
    WorkIter w, wn;   // current item, next item (its query tile is staged one item ahead)
    w.init(p);
    wn.init(p);
    bool vn = wn.next(p.seq_lens);
    auto stage_q = [&](const WorkIter &x, uint32_t slot) {
      if (t128 < G * 4) {
        const int n = t128 >> 2, c = t128 & 3;
        const uint4 v = *reinterpret_cast<const uint4 *>(p.q_codes + ((size_t)x.b * p.H_q + x.hk * G + n) * (TILE * 64) + c * 16);
        *reinterpret_cast<uint4 *>(dsm + D_OFF_Q + slot * 1024 + n * 64 + ((c ^ ((n & 7) >> 1)) << 4)) = v;
      }
      if (t128 < G) {
        const uint8_t *src = p.q_sf + ((size_t)x.b * p.H_q + x.hk * G + t128) * 1024;
        uint8_t *dst = dsm + D_OFF_SFQ + slot * 1024 + t128 * 16;
        *reinterpret_cast<uint32_t *>(dst) = *reinterpret_cast<const uint32_t *>(src);
        *reinterpret_cast<uint32_t *>(dst + 512) = *reinterpret_cast<const uint32_t *>(src + 512);
      }
      fence_proxy_async_smem();
      cx.warp_arrive(B_Q_READY + slot);
    };
    if (vn) stage_q(wn, 0);
    uint32_t it = 0, j = 0;
    bool ok = true;
    while (ok && w.next(p.seq_lens)) {
      vn = wn.next(p.seq_lens);
      if (vn) stage_q(wn, (j + 1) & 1);
      const float lam = __fmul_rn(__fmul_rn(__fmul_rn(p.softmax_scale, 1.4426950408889634f), p.q_gscale[w.b]), p.k_gscale[w.b]);
      const int k_part = w.sp * DECODE_SPLIT;
      float m_run[MAXG], l_r[MAXG];
#pragma unroll
      for (int g = 0; g < MAXG; ++g) m_run[g] = -INFINITY, l_r[g] = 0.0f;
      for (int u = w.nblk - 1; u >= 0; --u, ++it) {
        const uint32_t st = it % D_NST, sb = it & 1;
        ok = cx.wait_warp(B_S_FULL + sb, (it >> 1) & 1) && cx.wait_warp(B_FULL + st, (it / D_NST) & 1);
        if (!ok) break;
        if (warp == 2) DTR(7, it);
        tc_fence_after();
        uint32_t sraw[16];
        tmem_ld16(tm + TM_S + sb * 16 + tlane, sraw);
        tmem_ld_wait();
        tc_fence_before();
        cx.warp_arrive(B_S_EMPTY + sb);
        // ---- scores of this key for the G heads, block maximum
        const bool valid = k_part + u * TILE + r < w.L;
        const uint8_t *dptr = dsm + st * ST_BYTES + ST_DELTA + (r >> 6) * 1024 + (r & 63) * 2;
        float sv[MAXG];
#pragma unroll
        for (int g = 0; g < MAXG; ++g) {
          sv[g] = -INFINITY;
          if (g < G && valid) {
            const float dl = p.delta ? __uint_as_float((uint32_t)*reinterpret_cast<const uint16_t *>(dptr + g * 128) << 16) : 0.0f;
            sv[g] = __fadd_rn(__uint_as_float(sraw[g]), dl);
          }
          if (g < G) {
            float wm = sv[g];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
            if (lane == 0) xmax[(sb * 4 + (warp - 2)) * MAXG + g] = wm;
          }
        }
        if (warp == 2) DTR(8, it);
        cx.warp_arrive(B_XCHG);
        ok = cx.wait_warp(B_XCHG, it & 1);
        if (!ok) break;
        if (warp == 2) DTR(9, it);
        float alpha[MAXG];
        bool rescale = false;
        uint32_t pbytes[MAXG / 2];
#pragma unroll
        for (int g = 0; g < MAXG; g += 2) {
          float pq[2];
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int gg = g + e;
            float bm = -INFINITY;
            if (gg < G) {
#pragma unroll
              for (int q = 0; q < 4; ++q) bm = fmaxf(bm, xmax[(sb * 4 + q) * MAXG + gg]);
            }
            const float m_new = fmaxf(m_run[gg], bm);
            alpha[gg] = (m_run[gg] == -INFINITY) ? 1.0f : ex2_approx(__fmul_rn(m_run[gg] - m_new, lam));
            rescale |= (gg < G) && (alpha[gg] != 1.0f);
            const float pv = (gg < G && valid) ? ex2_approx(__fmaf_rn(sv[gg], lam, -__fmul_rn(m_new, lam))) : 0.0f;
            l_r[gg] = __fmaf_rn(l_r[gg], alpha[gg], pv);
            pq[e] = __fmul_rn(pv, 448.0f);
            m_run[gg] = m_new;
          }
          pbytes[g >> 1] = (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(pq[0], pq[1]), __NV_SATFINITE, __NV_E4M3);
        }
        // ---- P_hat^T into the B tile of this block's PV MMAs (free once PV of block it-2 is done)
        if (warp == 2) DTR(10, it);
        if (it >= 2) ok = cx.wait_warp(B_PV_DONE + sb, ((it >> 1) - 1) & 1);
        if (!ok) break;
        if (warp == 2) DTR(11, it);
        {
          uint8_t *pt = dsm + D_OFF_P + sb * 2048 + (r & 15);
#pragma unroll
          for (int g = 0; g < MAXG; ++g)
            if (g < G) pt[(g & 7) * 128 + (((r >> 4) ^ (g & 7)) << 4)] = (uint8_t)(pbytes[g >> 1] >> (8 * (g & 1)));
        }
        // ---- the running maximum grew: rescale O^T (needs the previous block's PV to be complete)
        if (u != w.nblk - 1 && rescale) {
          ok = cx.wait_warp(B_PV_DONE + ((it - 1) & 1), ((it - 1) >> 1) & 1);
          if (!ok) break;
          tc_fence_after();
          uint32_t o[16];
          tmem_ld16(tm + TM_O + tlane, o);
          tmem_ld_wait();
#pragma unroll
          for (int g = 0; g < MAXG; ++g) o[g] = __float_as_uint(__fmul_rn(__uint_as_float(o[g]), alpha[g]));
          tmem_st16(tm + TM_O + tlane, o);
          tmem_st_wait();
          tc_fence_before();
        }
        if (warp == 2) DTR(12, it);
        fence_proxy_async_smem();
        cx.warp_arrive(B_P_READY + sb);
        if (warp == 2) DTR(13, it);
      }
      if (!ok) break;
      // ---- partition state: O^T row of this thread's channel, l summed over the keys
      {
        const uint32_t last = it - 1;
        ok = cx.wait_warp(B_PV_DONE + (last & 1), (last >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
        uint32_t o[16];
        tmem_ld16(tm + TM_O + tlane, o);
        tmem_ld_wait();
        tc_fence_before();
        cx.warp_arrive(B_O_FREE);
        float *dst = p.parts + (((size_t)w.b * p.H_q + (size_t)w.hk * G) * p.n_split + w.sp) * PART_FLOATS;
        const size_t head_stride = (size_t)p.n_split * PART_FLOATS;
#pragma unroll
        for (int g = 0; g < MAXG; ++g) {
          if (g < G) {
            dst[g * head_stride + 2 + r] = __uint_as_float(o[g]);
            float ls = l_r[g];
#pragma unroll
            for (int o2 = 16; o2 > 0; o2 >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o2);
            if (lane == 0) xl[((j & 1) * 4 + (warp - 2)) * MAXG + g] = ls;
          }
        }
        cx.warp_arrive(B_LX);
        ok = cx.wait_warp(B_LX, j & 1);
        if (!ok) break;
#pragma unroll
        for (int g = 0; g < MAXG; ++g) {
          if (t128 == g && g < G) {
            float l = 0.0f;
#pragma unroll
            for (int q = 0; q < 4; ++q) l += xl[((j & 1) * 4 + q) * MAXG + g];
            dst[g * head_stride] = m_run[g];
            dst[g * head_stride + 1] = l;
          }
        }
      }
      ++j;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tm, TM_COLS);
}

// Merge of the partition states (Section 5.3): M = max m_s, w_s = 2^(lam (m_s - M)),
// l = sum w_s l_s, O = sum w_s O_s, out = O / (448 l) * v_scale.  grid (H_q, B), 128 threads.
__global__ void __launch_bounds__(128) decode_merge_kernel(const float *__restrict__ parts,
                                                           const int32_t *__restrict__ seq_lens,
                                                           const float *__restrict__ q_gscale,
                                                           const float *__restrict__ k_gscale, int H_q, int n_split,
                                                           float softmax_scale, float v_scale,
                                                           __nv_bfloat16 *__restrict__ out, float *__restrict__ out_f32) {
  const int hq = blockIdx.x, b = blockIdx.y, c = threadIdx.x, lane = threadIdx.x & 31;
  const int L = seq_lens[b];
  const int ns = min(n_split, (L + DECODE_SPLIT - 1) / DECODE_SPLIT);
  const float *base = parts + ((size_t)b * H_q + hq) * n_split * PART_FLOATS;
  const float lam = __fmul_rn(__fmul_rn(__fmul_rn(softmax_scale, 1.4426950408889634f), q_gscale[b]), k_gscale[b]);
  float M = -INFINITY;
  for (int s = lane; s < ns; s += 32) M = fmaxf(M, base[(size_t)s * PART_FLOATS]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float l = 0.0f, o = 0.0f;
  for (int s = 0; s < ns; ++s) {
    const float ms = base[(size_t)s * PART_FLOATS];
    if (ms == -INFINITY) continue;
    const float w = ex2_approx(__fmul_rn(ms - M, lam));
    l = __fadd_rn(l, __fmul_rn(w, base[(size_t)s * PART_FLOATS + 1]));
    o = __fadd_rn(o, __fmul_rn(w, base[(size_t)s * PART_FLOATS + 2 + c]));
  }
  const float r = (l > 0.0f) ? __fmul_rn(__fdiv_rn(o, __fmul_rn(448.0f, l)), v_scale) : 0.0f;
  const size_t idx = ((size_t)b * H_q + hq) * HEAD_DIM + c;
  out[idx] = __float2bfloat16_rn(r);
  if (out_f32) out_f32[idx] = r;
}

}  // namespace
}  // namespace mpfa

using namespace mpfa;

#ifdef MPFA_TRACE
extern "C" int mpfa_debug_set_decode_trace(long long *buf, int cta) {
  if (cudaMemcpyToSymbol(g_dtrace, &buf, sizeof(buf)) != cudaSuccess) return -1;
  if (cudaMemcpyToSymbol(g_dtrace_cta, &cta, sizeof(cta)) != cudaSuccess) return -1;
  return 0;
}
#endif

extern "C" size_t mpfa_decode_workspace_bytes(int B, int H_q, int H_kv, int max_pages_per_req) {
  if (B <= 0 || H_q <= 0 || H_kv <= 0 || max_pages_per_req <= 0) return 0;
  const size_t n_split = ((size_t)max_pages_per_req * PAGE + DECODE_SPLIT - 1) / DECODE_SPLIT;
  return (size_t)B * H_q * n_split * PART_FLOATS * sizeof(float);
}

extern "C" mpfa_status mpfa_decode(const mpfa_fp4_tensor *q, const mpfa_paged_kv *kv, const int32_t *page_table,
                                   int max_pages_per_req, const int32_t *seq_lens, const mpfa_stats *st, float v_scale,
                                   float softmax_scale, void *out_bf16, float *out_f32, void *workspace,
                                   size_t workspace_bytes, int32_t *device_status, void *stream) {
  if (!q || !kv || !page_table || !seq_lens || !st || !out_bf16 || !workspace || !device_status)
    return MPFA_ERR_INVALID_ARG;
  if (!q->codes || !q->sf || q->B <= 0 || q->H <= 0 || q->N != 1 || max_pages_per_req <= 0)
    return MPFA_ERR_INVALID_ARG;
  if (!kv->k_codes || !kv->k_sf || !kv->v_fp8 || kv->num_pages <= 0 || !st->q_gscale || !st->k_gscale)
    return MPFA_ERR_INVALID_ARG;
  if (!(softmax_scale > 0.0f) || !(v_scale > 0.0f)) return MPFA_ERR_INVALID_ARG;
  if (kv->page_size != PAGE) return MPFA_ERR_UNSUPPORTED;
  const int B = q->B, H_q = q->H, H_kv = kv->H_kv;
  if (H_kv <= 0 || kv->H_q != H_q) return MPFA_ERR_INVALID_ARG;
  if (H_q % H_kv != 0 || H_q / H_kv > MAXG) return MPFA_ERR_UNSUPPORTED;
  const size_t n_split = ((size_t)max_pages_per_req * PAGE + DECODE_SPLIT - 1) / DECODE_SPLIT;
  const size_t need = (size_t)B * H_q * n_split * PART_FLOATS * sizeof(float);
  if (workspace_bytes < need) return MPFA_ERR_WORKSPACE;
  if ((size_t)B * H_kv * n_split > 0x7FFFFFFFull || B > 65535) return MPFA_ERR_UNSUPPORTED;
  if (!aligned(q->codes, 16) || !aligned(q->sf, 16) || !aligned(kv->k_codes, 256) || !aligned(kv->k_sf, 256) ||
      !aligned(kv->v_fp8, 256) || !aligned(kv->delta_s_bf16, 256) || !aligned(workspace, 16))
    return MPFA_ERR_ALIGNMENT;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  int dev = 0, n_sm = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  MPFA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  DecodeParams p;
  p.q_codes = q->codes;
  p.q_sf = q->sf;
  p.k_codes = kv->k_codes;
  p.k_sf = kv->k_sf;
  p.v_fp8 = kv->v_fp8;
  p.delta = static_cast<const __nv_bfloat16 *>(kv->delta_s_bf16);
  p.page_table = page_table;
  p.seq_lens = seq_lens;
  p.q_gscale = st->q_gscale;
  p.k_gscale = st->k_gscale;
  p.parts = static_cast<float *>(workspace);
  p.status = device_status;
  p.B = B;
  p.H_q = H_q;
  p.H_kv = H_kv;
  p.max_pages = max_pages_per_req;
  p.num_pages = kv->num_pages;
  p.n_split = (int)n_split;
  p.softmax_scale = softmax_scale;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t items = (size_t)B * H_kv * n_split;
  const unsigned grid = (unsigned)(items < (size_t)n_sm ? items : (size_t)n_sm);   // one persistent CTA per SM
  MPFA_CUDA_OK(cudaFuncSetAttribute(decode_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)D_SMEM));
  decode_split_kernel<<<grid, D_THREADS, D_SMEM, s>>>(p);
  MPFA_LAUNCH_OK();
  decode_merge_kernel<<<dim3(H_q, B), 128, 0, s>>>(p.parts, seq_lens, st->q_gscale, st->k_gscale, H_q, (int)n_split,
                                                   softmax_scale, v_scale, static_cast<__nv_bfloat16 *>(out_bf16),
                                                   out_f32);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}
