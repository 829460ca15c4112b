// QK4PV8 decode over a paged low-bit KV cache (Section 5.3) for sm_100a.
//
// The path is bound by streaming the cache from HBM (208 bytes per token and kv head plus
// Delta_S), so the kernel is a persistent streaming pipeline: one CTA per SM walks a list of
// (request, kv head, 1024-token partition) work items, and a producer warp keeps two rings of
// 128-key blocks in flight with bulk asynchronous copies: a K ring (codes, block scales,
// Delta_S) that runs one item AHEAD of a V ring.  The cache's physical byte order
// (include/mpfa.h) is the swizzled shared-memory image the tensor-core descriptors read, so a
// page needs one copy per tensor and no thread touches the bytes.
//
// The problem is transposed so that the long axis is the MMA's M dimension and the GQA group
// (Section 5.3 packs it into one MMA tile) is the N dimension, padded to 16:
//   S^T[key, head] = K Q^T       tcgen05.mma kind::mxf4nvf4 (E2M1 codes, UE4M3 block scales),
//                                M = 128 keys, N = 16, K = 2 x 64 channels, FP32 in TMEM,
//                                one 16-column slot per block of the item;
//   softmax        one thread per key.  As each S^T lands: + Delta_S (Eq. 11), warp maximum.
//                  After the item's last block one exchange gives every block u the running
//                  maximum m_u of the reverse traversal (max over the blocks visited so far),
//                  then P = 2^(lam S - lam m_u), P_hat = E4M3(448 P) for all blocks at once,
//                  written to shared memory as the B operands of the PV MMAs;
//   O_u^T[ch, head] = V_u^T P_hat_u^T   tcgen05.mma kind::f8f6f4, M = 128 channels, N = 16,
//                                K = 4 x 32 keys, V read MN-major straight from the ring, one
//                                accumulator slot per block.
// Because the scores of an item are finished while the previous item's V is still streaming,
// a V block is consumed the moment it lands, and the softmax never sits on the critical path.
// The sequential rescaling O <- 2^(lam (m_old - m_new)) O + P_hat V becomes
// O = sum_u 2^(lam (m_u - m)) O_u at the end of the item (one thread per channel), the same
// sum with the factors multiplied out.  The partition state (m, l, O) goes to the workspace; a
// second kernel merges partitions by log-sum-exp and writes BF16.
//
// Warps: 10 draws work items, 0, 9 K producers, 8 V producer, 1 QK issue (+ TMEM allocation), 2 PV issue, 3 rewrites the K scales of
// each block from [token][8] into the 32 x 16-byte tiles tcgen05.cp expects, 4-7 softmax and
// partition write-out (TMEM lane quadrant = warp % 4).  Every wait is bounded.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mpfa {
namespace {

constexpr int PART_FLOATS = 130;  // m, l, O[128] per (request, q head, partition)
constexpr int MAXG = 8;
constexpr int NCOL = 16;          // MMA N: the GQA group padded to 16 columns
constexpr int MAXBLK = DECODE_SPLIT / TILE;   // 8 blocks per item

constexpr int D_NK = 4;           // K ring stages
constexpr int D_NV = 8;           // V ring stages
constexpr int D_THREADS = 352;
constexpr int D_NITEM = 8;        // work items published ahead of their use

// one K stage
constexpr uint32_t KST_K = 0;          // 2 pages x 4096 B of codes: 64-byte rows, 64-byte swizzle
constexpr uint32_t KST_SF = 8192;      // 2 pages x 512 B of K scales, [token][8]
constexpr uint32_t KST_DELTA = 9216;   // 2 pages x 8 rows x 128 B of Delta_S (BF16, 128-byte swizzle; rows G..7 stay zero)
constexpr uint32_t KST_BYTES = 11264;
constexpr uint32_t VST_BYTES = 16384;  // 2 pages x 8192 B: 128-byte rows, 128-byte swizzle
constexpr uint32_t D_OFF_K = 0;
constexpr uint32_t D_OFF_V = D_OFF_K + D_NK * KST_BYTES;
constexpr uint32_t D_OFF_P = D_OFF_V + D_NV * VST_BYTES;   // [2 items][8 blocks] x 1024: P_hat^T, 8 rows of 128 keys (rows 8..15: zero block)
constexpr uint32_t D_OFF_Q = D_OFF_P + 2 * MAXBLK * 1024;  // 2 x 1024: Q codes, 16 rows of 64 B, 64-byte swizzle
constexpr uint32_t D_OFF_SFQ = D_OFF_Q + 2048;             // 2 x (2 x 512): Q scales, one tile per 64 channels
constexpr uint32_t D_OFF_SFK = D_OFF_SFQ + 2048;           // D_NK x (2 x 512): K scales
constexpr uint32_t D_OFF_ZERO = D_OFF_SFK + D_NK * 1024;    // 2048 B of zeros: second K group of the Delta_S operand, rows 8..15 of P_hat^T
constexpr uint32_t D_OFF_IDENT = D_OFF_ZERO + 2048;        // 16 x 16 BF16 identity, MN-major, 128-byte swizzle
constexpr uint32_t D_OFF_BAR = D_OFF_IDENT + 2048;
constexpr uint32_t D_OFF_XMAX = D_OFF_BAR + 1024;           // [2][8 blocks][MAXG][4 warps] floats
constexpr uint32_t D_OFF_WTAB = D_OFF_XMAX + 2 * MAXBLK * MAXG * 16;   // [2][8 blocks][MAXG] floats
constexpr uint32_t D_OFF_MFIN = D_OFF_WTAB + 2 * MAXBLK * MAXG * 4;    // [2][MAXG]
constexpr uint32_t D_OFF_XL = D_OFF_MFIN + 2 * MAXG * 4;               // [2][4 warps][MAXG]
constexpr uint32_t D_OFF_MISC = D_OFF_XL + 2 * 4 * MAXG * 4;           // TMEM address, abort flag
constexpr int D_MAXREQ = 768;                                          // requests whose length / lambda are cached
constexpr uint32_t D_OFF_LEN = D_OFF_MISC + 64;                        // [D_MAXREQ] int32 lengths
constexpr uint32_t D_OFF_LAM = D_OFF_LEN + D_MAXREQ * 4;               // [D_MAXREQ] float
constexpr uint32_t D_OFF_RING = D_OFF_LAM + D_MAXREQ * 4;              // [D_NITEM] int4 work items {b, hk, sp, L}
constexpr uint32_t D_OFF_PRE = D_OFF_RING + D_NITEM * 16;              // [D_MAXREQ + 1] items of the requests before b
constexpr uint32_t D_SMEM_USED = D_OFF_PRE + (D_MAXREQ + 4) * 4;
constexpr uint32_t D_SMEM = D_SMEM_USED + 1024;     // slack for the 1024-byte alignment of the base

// barriers (8 bytes each)
constexpr int B_K_FULL = 0;                      // [D_NK] K stage landed (bytes)
constexpr int B_K_EMPTY = B_K_FULL + D_NK;       // [D_NK] QK commit
constexpr int B_V_FULL = B_K_EMPTY + D_NK;       // [D_NV]
constexpr int B_V_EMPTY = B_V_FULL + D_NV;       // [D_NV] PV commit
constexpr int B_SF_READY = B_V_EMPTY + D_NV;     // [D_NK] K scales formatted
constexpr int B_S_FULL = B_SF_READY + D_NK;      // [2][8] QK commit
constexpr int B_S_FREE = B_S_FULL + 2 * MAXBLK;  // [2] 4 warps: the item's scores have been read
constexpr int B_P_READY = B_S_FREE + 2;          // [2] 4 warps
constexpr int B_Q_READY = B_P_READY + 2;         // [2] scale warp
constexpr int B_O_FULL = B_Q_READY + 2;          // [1] PV commit after the item's last block
constexpr int B_O_FREE = B_O_FULL + 1;           // [1] 4 warps
constexpr int B_XCHG = B_O_FREE + 1;             // [1] 4 warps
constexpr int B_ITEM_FULL = B_XCHG + 1;          // [D_NITEM] work item published
constexpr int B_ITEM_EMPTY = B_ITEM_FULL + D_NITEM;   // [D_NITEM] read by all ten consumer warps
constexpr int B_COUNT = B_ITEM_EMPTY + D_NITEM;
static_assert(B_COUNT * 8 <= 1024, "barrier block");
static_assert(D_SMEM <= 232448, "shared memory");
static_assert(KST_BYTES % 1024 == 0 && D_OFF_V % 1024 == 0 && D_OFF_P % 1024 == 0, "swizzle atoms");

// tensor-memory columns
constexpr uint32_t TM_S = 0;       // [2 items][8 blocks] x 16
constexpr uint32_t TM_O = 256;     // [8 blocks] x 16
constexpr uint32_t TM_SFQ = 384;   // 2 x 8
constexpr uint32_t TM_SFK = 400;   // D_NK x 8
static_assert(TM_SFK + D_NK * 8 <= 512, "tensor memory");
constexpr uint32_t TM_COLS = 512;

#ifndef MPFA_WAIT_LIMIT_CYCLES
#define MPFA_WAIT_LIMIT_CYCLES 4000000000ll   // about two seconds of SM clock
#endif
constexpr long long D_WAIT_CYCLES = MPFA_WAIT_LIMIT_CYCLES;
// Test builds only (-DMPFA_TEST_DROP_V_COPY with a short limit): every CTA's V producer leaves out its first copy,
// so the give-up path runs (status bit, roles leave, copies in flight awaited, tensor memory released).

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The first G (1..8) TMEM columns at `taddr` of this thread's lane; the load width is the next power of two.
template <int G>
__device__ __forceinline__ void tmem_ld_g(uint32_t taddr, uint32_t (&r)[G]) {
  static_assert(G >= 1 && G <= 8, "group size");
  if constexpr (G == 1) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r[0]) : "r"(taddr) : "memory");
  } else if constexpr (G == 2) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(taddr) : "memory");
  } else if constexpr (G <= 4) {
    uint32_t x[4];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3])
                 : "r"(taddr)
                 : "memory");
#pragma unroll
    for (int g = 0; g < G; ++g) r[g] = x[g];
  } else {
    uint32_t x[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3]), "=r"(x[4]), "=r"(x[5]), "=r"(x[6]), "=r"(x[7])
                 : "r"(taddr)
                 : "memory");
#pragma unroll
    for (int g = 0; g < G; ++g) r[g] = x[g];
  }
}

#ifdef MPFA_TRACE
// clock64 stamps of CTA g_dtrace_cta: [counter < 256][16 events]
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
  unsigned int *ticket;   // global work counter, zeroed before the launch
  int B, H_q, H_kv, max_pages, num_pages, n_split;
  float softmax_scale;
};

// Work items (request, kv head, 1024-token partition) are handed out dynamically: one warp per CTA draws
// tickets from a global counter and publishes the decoded items in a small shared-memory ring; every other
// warp walks that ring.  SMs do not stream at the same rate (those far from the memory they read are up to
// 8 % slower), so a static split leaves the fast ones idle at the end.
struct WorkIter;

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
      if (mbar_try_wait_hint(a, parity, 2000u)) return true;   // the hardware may park the thread meanwhile
      if ((n & 255u) == 0u) {
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

struct WorkIter {
  uint32_t n;          // items taken so far
  bool release;        // the warp's main walk hands the ring slot back; look-ahead walks only read
  int b, hk, sp, L, nblk;
  __device__ void init(bool main_walk) {
    n = 0;
    release = main_walk;
  }
  // Whole warp.  false: no more items (or the CTA is giving up).
  __device__ bool next(const DCtx &cx, const int4 *ring) {
    const uint32_t slot = n % D_NITEM;
    if (!cx.wait_warp(B_ITEM_FULL + slot, (n / D_NITEM) & 1)) return false;
    const int4 it = ring[slot];
    if (it.x < 0) return false;   // end marker: stays in its slot, nobody moves past it
    if (release) cx.warp_arrive(B_ITEM_EMPTY + slot);
    ++n;
    b = it.x, hk = it.y, sp = it.z, L = it.w;
    nblk = (min(L - sp * DECODE_SPLIT, DECODE_SPLIT) + TILE - 1) / TILE;
    return true;
  }
};

// Page ids of the blocks of one item, lane l holding block l's two table entries (loads only: the values
// are range-checked where they are used, so that nothing waits for them here).
__device__ __forceinline__ void lookup_pages(const DecodeParams &p, const WorkIter &w, int lane, int &pid0, int &pid1) {
  pid0 = -1, pid1 = -1;
  if (lane < w.nblk) {
    const int pg = (w.sp * DECODE_SPLIT + lane * TILE) / PAGE;
    const int32_t *row = p.page_table + (size_t)w.b * p.max_pages;
    if (pg < p.max_pages) pid0 = row[pg];
    if (pg + 1 < p.max_pages) pid1 = row[pg + 1];
  }
}

template <int G>
__global__ void __launch_bounds__(D_THREADS, 1) decode_split_kernel(const DecodeParams p) {
  extern __shared__ uint8_t dsm_raw[];
  uint8_t *dsm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(dsm_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(dsm);
  float *xmax = reinterpret_cast<float *>(dsm + D_OFF_XMAX);
  float *wtab = reinterpret_cast<float *>(dsm + D_OFF_WTAB);
  float *mfin = reinterpret_cast<float *>(dsm + D_OFF_MFIN);
  float *xl = reinterpret_cast<float *>(dsm + D_OFF_XL);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(dsm + D_OFF_MISC);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(dsm + D_OFF_MISC + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  DCtx cx{sbase + D_OFF_BAR, abort_flag, p.status};
#ifdef MPFA_TRACE
  if (g_dtrace && threadIdx.x == 0) g_dtrace[4096 + 2 * blockIdx.x] = (long long)globaltimer_ns();
#endif

  // ---- set-up: barriers, zeroed operand tiles (rows G..15 stay zero for good), TMEM
  if (threadIdx.x == 0) {
    for (int i = 0; i < D_NK; ++i) {
      mbar_init(cx.bar(B_K_FULL + i), 2);
      mbar_init(cx.bar(B_K_EMPTY + i), 1);
      mbar_init(cx.bar(B_SF_READY + i), 1);
    }
    for (int i = 0; i < D_NV; ++i) {
      mbar_init(cx.bar(B_V_FULL + i), 1);
      mbar_init(cx.bar(B_V_EMPTY + i), 1);
    }
    for (int i = 0; i < 2 * MAXBLK; ++i) mbar_init(cx.bar(B_S_FULL + i), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(cx.bar(B_S_FREE + i), 4);
      mbar_init(cx.bar(B_P_READY + i), 4);
      mbar_init(cx.bar(B_Q_READY + i), 1);
    }
    mbar_init(cx.bar(B_O_FULL), 1);
    mbar_init(cx.bar(B_O_FREE), 4);
    mbar_init(cx.bar(B_XCHG), 4);
    for (int i = 0; i < D_NITEM; ++i) {
      mbar_init(cx.bar(B_ITEM_FULL + i), 1);
      mbar_init(cx.bar(B_ITEM_EMPTY + i), 10);
    }
    mbar_init_fence();
    *abort_flag = 0;
  }
  // zeroed once: the K ring (Delta_S rows G..7 are never written), P, Q and scale tiles, zero and identity blocks
  for (uint32_t o = threadIdx.x * 16; o < D_NK * KST_BYTES; o += D_THREADS * 16)
    *reinterpret_cast<uint4 *>(dsm + D_OFF_K + o) = make_uint4(0u, 0u, 0u, 0u);
  for (uint32_t o = threadIdx.x * 16; o < D_OFF_BAR - D_OFF_P; o += D_THREADS * 16)
    *reinterpret_cast<uint4 *>(dsm + D_OFF_P + o) = make_uint4(0u, 0u, 0u, 0u);
  int32_t *len_tab = reinterpret_cast<int32_t *>(dsm + D_OFF_LEN);
  float *lam_tab = reinterpret_cast<float *>(dsm + D_OFF_LAM);
  for (int i = threadIdx.x; i < min(p.B, D_MAXREQ); i += D_THREADS) {
    len_tab[i] = p.seq_lens[i];
    lam_tab[i] = __fmul_rn(__fmul_rn(__fmul_rn(p.softmax_scale, 1.4426950408889634f), p.q_gscale[i]), p.k_gscale[i]);
  }
  __syncthreads();
  if (threadIdx.x < 16) {   // identity[n][k]: element (n, k) at (k/8)*1024 + (k%8)*128 + ((n/8) ^ (k%8))*16 + (n%8)*2
    const int k = threadIdx.x;
    *reinterpret_cast<uint16_t *>(dsm + D_OFF_IDENT + (k >> 3) * 1024 + (k & 7) * 128 + (((k >> 3) ^ (k & 7)) << 4) + (k & 7) * 2) = 0x3F80;
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), TM_COLS);
    tmem_relinquish();
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = *tmem_slot;
  const int4 *ring = reinterpret_cast<const int4 *>(dsm + D_OFF_RING);

  if (warp == 10) {
    // ================= work distribution: tickets from the global counter, decoded, published D_NITEM ahead.
    // With at most D_MAXREQ requests the tickets number only the partitions that exist (prefix sums of
    // ceil(L / 1024) * H_kv per request, request found by bisection); otherwise they number every
    // (request, kv head, partition slot) and the empty ones are drawn again.
    int4 *ring_w = reinterpret_cast<int4 *>(dsm + D_OFF_RING);
    int32_t *pre = reinterpret_cast<int32_t *>(dsm + D_OFF_PRE);
    const bool compact = p.B <= D_MAXREQ;
    uint32_t total;
    if (compact) {
      // pre[b] = items of requests 0..b-1: every lane sums a contiguous run of requests, the warp scans the runs
      const int per = (p.B + 31) / 32, lo = min(p.B, lane * per), hi = min(p.B, lo + per);
      int run = 0;
      for (int i = lo; i < hi; ++i) run += min((max(len_tab[i], 0) + DECODE_SPLIT - 1) / DECODE_SPLIT, p.n_split) * p.H_kv;
      int incl = run;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      int acc = incl - run;
      for (int i = lo; i < hi; ++i) {
        pre[i] = acc;
        acc += min((max(len_tab[i], 0) + DECODE_SPLIT - 1) / DECODE_SPLIT, p.n_split) * p.H_kv;
      }
      total = (uint32_t)__shfl_sync(0xffffffffu, incl, 31);
      if (lane == 31) pre[p.B] = (int)total;
      __syncwarp();
    } else {
      total = (uint32_t)p.B * p.H_kv * p.n_split;
    }
    bool ok = true;
    for (uint32_t k = 0; ok; ++k) {
      const uint32_t slot = k % D_NITEM;
      if (k >= (uint32_t)D_NITEM) ok = cx.wait_warp(B_ITEM_EMPTY + slot, ((k / D_NITEM) - 1) & 1);
      if (!ok) break;
      int4 item = make_int4(-1, 0, 0, 0);
      if (lane == 0) {
        for (;;) {
          const uint32_t tkt = atomicAdd(p.ticket, 1u);
          if (tkt >= total) break;
          if (compact) {
            int lo = 0, hi = p.B;   // largest b with pre[b] <= tkt
            while (hi - lo > 1) {
              const int mid = (lo + hi) >> 1;
              if ((uint32_t)pre[mid] <= tkt) lo = mid; else hi = mid;
            }
            const int L = len_tab[lo], nsp = min((L + DECODE_SPLIT - 1) / DECODE_SPLIT, p.n_split);
            const int r = (int)tkt - pre[lo];
            item = make_int4(lo, r / nsp, r % nsp, L);
            break;
          }
          const int sp = (int)(tkt % (uint32_t)p.n_split), r = (int)(tkt / (uint32_t)p.n_split);
          const int b = r / p.H_kv, L = p.seq_lens[b];
          if (L - sp * DECODE_SPLIT > 0) {
            item = make_int4(b, r % p.H_kv, sp, L);
            break;
          }
        }
        ring_w[slot] = item;
        mbar_arrive(cx.bar(B_ITEM_FULL + slot));
      }
      item.x = __shfl_sync(0xffffffffu, item.x, 0);
      if (item.x < 0) break;   // the end marker is in the ring; this CTA draws no more
    }
  } else if (warp == 0 || warp >= 8) {
    // ================= producers: warps 0 and 9 stream the K ring (0: codes; 9: block scales and Delta_S,
    // both arriving on the stage's barrier), warp 8 the V ring.  Issuing a bulk copy costs a warp well over a
    // hundred cycles, so the ten copies of a block are spread over three warps.
    // Nothing orders the two streams but the data flow: a K stage is released by its QK MMAs, a V stage
    // only after the item's softmax, so K runs about one item ahead.  Page ids are loaded one item before
    // they are used and validated at use, so the loop never waits for the table.
    const bool is_k = warp != 8, is_codes = warp == 0;
    WorkIter w, wl;
    w.init(true);
    wl.init(false);
    uint32_t c = 0;   // block counter of this ring
    bool ok = true;
    const uint32_t d_bytes = p.delta ? (uint32_t)G * PAGE * 2 : 0u;
    const uint32_t kpage_bytes = is_codes ? 4096u : 512u + d_bytes;
    const int n_ring = is_k ? D_NK : D_NV;
    const int b_full = is_k ? B_K_FULL : B_V_FULL, b_empty = is_k ? B_K_EMPTY : B_V_EMPTY;
    int pc0 = -1, pc1 = -1, pn0 = -1, pn1 = -1;
    bool vw = w.next(cx, ring);
    bool vl = wl.next(cx, ring);
    if (vw) lookup_pages(p, w, lane, pc0, pc1);
    uint32_t jtr = 0;
    while (ok && vw) {
      if (is_codes) DTR(12, jtr);
      vl = wl.next(cx, ring);
      if (is_codes) DTR(13, jtr);
      if (vl) lookup_pages(p, wl, lane, pn0, pn1);   // consumed one item later
      if (is_codes) DTR(14, jtr);
      ++jtr;
      for (int t = 0; ok && t < w.nblk; ++t, ++c) {
        const uint32_t st = c % n_ring;
        if (c >= (uint32_t)n_ring && !cx.wait_warp(b_empty + st, ((c / n_ring) - 1) & 1)) {
          ok = false;
          break;
        }
        if (warp != 9) DTR(is_k ? 0 : 1, c);
        const int u = w.nblk - 1 - t;
        int id0 = __shfl_sync(0xffffffffu, pc0, u), id1 = __shfl_sync(0xffffffffu, pc1, u);
        const bool want1 = w.sp * DECODE_SPLIT + u * TILE + PAGE < w.L;
        const bool bad = id0 < 0 || id0 >= p.num_pages || (want1 && (id1 < 0 || id1 >= p.num_pages));
        if (bad && lane == 0 && !is_codes) atomicOr(p.status, MPFA_DEV_BAD_PAGE);
        if (id0 < 0 || id0 >= p.num_pages) id0 = -1;
        if (!want1 || id1 < 0 || id1 >= p.num_pages) id1 = -1;
        const uint32_t full = cx.bar(b_full + st);
        if (is_k) {
          if (elect_one()) {
            const uint32_t sdst = sbase + D_OFF_K + st * KST_BYTES;
            mbar_expect_tx(full, (id0 >= 0 ? kpage_bytes : 0u) + (id1 >= 0 ? kpage_bytes : 0u));
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const int id = half == 0 ? id0 : id1;
              if (id < 0) continue;
              const size_t slab = (size_t)id * p.H_kv + w.hk;
              if (is_codes) {
                bulk_load(sdst + KST_K + half * 4096, p.k_codes + slab * 4096, 4096, full);
              } else {
                bulk_load(sdst + KST_SF + half * 512, p.k_sf + slab * 512, 512, full);
                if (d_bytes)
                  bulk_load(sdst + KST_DELTA + half * 1024, p.delta + ((size_t)id * p.H_q + (size_t)w.hk * G) * PAGE, d_bytes, full);
              }
            }
          }
        } else {
          // a page that is not there contributes P_hat = 0 times V: V must be finite, so zero it
          if (id0 < 0 || id1 < 0) {
            uint8_t *stage = dsm + D_OFF_V + st * VST_BYTES;
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
              if ((half == 0 ? id0 : id1) >= 0) continue;
              for (int i = 0; i < 16; ++i)
                *reinterpret_cast<uint4 *>(stage + half * 8192 + i * 512 + lane * 16) = make_uint4(0u, 0u, 0u, 0u);
            }
            fence_proxy_async_smem();
            __syncwarp();
          }
#ifdef MPFA_TEST_DROP_V_COPY
          if (c == 0) {
            // left out on purpose (work items are drawn dynamically: any CTA may be the one that gets work)
          } else
#endif
          if (elect_one()) {
            const uint32_t sdst = sbase + D_OFF_V + st * VST_BYTES;
            mbar_expect_tx(full, (id0 >= 0 ? 8192u : 0u) + (id1 >= 0 ? 8192u : 0u));
            if (id0 >= 0) bulk_load(sdst, p.v_fp8 + ((size_t)id0 * p.H_kv + w.hk) * 8192, 8192, full);
            if (id1 >= 0) bulk_load(sdst + 8192, p.v_fp8 + ((size_t)id1 * p.H_kv + w.hk) * 8192, 8192, full);
          }
        }
        __syncwarp();
      }
      if (is_codes) DTR(15, jtr - 1);
      vw = w.next(cx, ring);
      pc0 = pn0, pc1 = pn1;
    }
    if (!ok) {
      // another role gave up: let the copies already issued land before shared memory goes away
      for (uint32_t i = c - min(c, (uint32_t)n_ring); i < c; ++i) {
        const long long t0 = clock64();
        while (!mbar_try_wait(cx.bar(b_full + i % n_ring), (i / n_ring) & 1) && clock64() - t0 < D_WAIT_CYCLES) {
        }
      }
    }
  } else if (warp == 1) {
    // ================= QK issue: S^T[item parity][block] = K Q^T as K stages land
    const uint32_t id_qk = idesc_nvfp4(128, NCOL);
    const uint32_t id_ds = idesc_bf16(128, NCOL, 1, 1);
    const uint64_t d_ident = smem_desc(sbase + D_OFF_IDENT, 2048, 1024, SWZ_128B);
    const bool has_delta = p.delta != nullptr;
    WorkIter w;
    w.init(true);
    uint32_t kc = 0, j = 0;
    bool ok = true;
    while (ok && w.next(cx, ring)) {
      const uint32_t par = j & 1;
      ok = cx.wait_warp(B_Q_READY + par, (j >> 1) & 1);
      if (ok && j >= 2) ok = cx.wait_warp(B_S_FREE + par, ((j >> 1) - 1) & 1);   // scores of item j-2 have been read
      for (int t = 0; ok && t < w.nblk; ++t, ++kc) {
        const uint32_t st = kc % D_NK;
        ok = cx.wait_warp(B_K_FULL + st, (kc / D_NK) & 1) && cx.wait_warp(B_SF_READY + st, (kc / D_NK) & 1);
        if (!ok) break;
        DTR(2, kc);
        tc_fence_after();
        if (elect_one()) {
          const uint32_t tSFQ = tm + TM_SFQ + par * 8, tSFK = tm + TM_SFK + st * 8;
          if (t == 0) {
            const uint64_t d_sfq = smem_desc(sbase + D_OFF_SFQ + par * 1024, 0, 128, SWZ_NONE);
            tmem_cp_32x128b_warpx4(tSFQ, d_sfq);
            tmem_cp_32x128b_warpx4(tSFQ + 4, d_sfq + (512 >> 4));
          }
          const uint64_t d_sfk = smem_desc(sbase + D_OFF_SFK + st * 1024, 0, 128, SWZ_NONE);
          tmem_cp_32x128b_warpx4(tSFK, d_sfk);
          tmem_cp_32x128b_warpx4(tSFK + 4, d_sfk + (512 >> 4));
          const uint64_t d_k = smem_desc(sbase + D_OFF_K + st * KST_BYTES + KST_K, 16, 512, SWZ_64B);
          const uint64_t d_q = smem_desc(sbase + D_OFF_Q + par * 1024, 16, 512, SWZ_64B);
          const uint32_t tS = tm + TM_S + (par * MAXBLK + t) * 16;
          if (has_delta) {
            // S^T = Delta_S^T I (Eq. 11 seed): A = the stage's Delta_S rows, MN-major (keys contiguous), its
            // second group of eight K rows read from the zero block; B = identity
            const uint32_t a_ds = sbase + D_OFF_K + st * KST_BYTES + KST_DELTA;
            mma_bf16_ss(tS, smem_desc(a_ds, 1024, sbase + D_OFF_ZERO - a_ds, SWZ_128B), d_ident, id_ds, 0u);
          }
          mma_nvfp4_ss(tS, d_k, d_q, id_qk, tSFK, tSFQ, has_delta ? 1u : 0u);
          mma_nvfp4_ss(tS, d_k + (32 >> 4), d_q + (32 >> 4), id_qk, tSFK + 4, tSFQ + 4, 1u);
          mma_commit(cx.bar(B_S_FULL + par * MAXBLK + t));
          mma_commit(cx.bar(B_K_EMPTY + st));
        }
        __syncwarp();
        DTR(3, kc);
      }
      // the slots this item does not use complete a phase as well: a barrier's phase is then a function of the item
      if (ok && w.nblk < MAXBLK && elect_one())
        for (int t = w.nblk; t < MAXBLK; ++t) mma_commit(cx.bar(B_S_FULL + par * MAXBLK + t));   // after the MMAs above
      __syncwarp();
      ++j;
    }
  } else if (warp == 2) {
    // ================= PV issue: O_u^T = V_u^T P_hat_u^T as V stages land
    const uint32_t id_pv = idesc_e4m3(128, NCOL, 1, 0);
    WorkIter w;
    w.init(true);
    uint32_t vc = 0, j = 0;
    bool ok = true;
    while (ok && w.next(cx, ring)) {
      const uint32_t par = j & 1;
      ok = cx.wait_warp(B_P_READY + par, (j >> 1) & 1);
      if (ok && j >= 1) ok = cx.wait_warp(B_O_FREE, (j - 1) & 1);   // the previous item's O has been read
      for (int t = 0; ok && t < w.nblk; ++t, ++vc) {
        const uint32_t st = vc % D_NV;
        ok = cx.wait_warp(B_V_FULL + st, (vc / D_NV) & 1);
        if (!ok) break;
        DTR(4, vc);
        tc_fence_after();
        if (elect_one()) {
          const uint64_t d_v = smem_desc(sbase + D_OFF_V + st * VST_BYTES, 16, 1024, SWZ_128B);
          // rows 0..7 of P_hat^T in the block's tile, rows 8..15 (the next 8-row group) from the zero block
          const uint32_t a_p = sbase + D_OFF_P + (par * MAXBLK + t) * 1024;
          const uint64_t d_p = smem_desc(a_p, 16, sbase + D_OFF_ZERO - a_p, SWZ_128B);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)   // 32 keys per MMA
            mma_e4m3_ss(tm + TM_O + t * 16, d_v + (uint64_t)((4096 * k4) >> 4), d_p + (uint64_t)((32 * k4) >> 4), id_pv,
                        k4 > 0 ? 1u : 0u);
          mma_commit(cx.bar(B_V_EMPTY + st));
          if (t == w.nblk - 1) mma_commit(cx.bar(B_O_FULL));
        }
        __syncwarp();
        DTR(5, vc);
      }
      ++j;
    }
  } else if (warp == 3) {
    // ================= K scales of a block: [token][8 blocks] -> two 32 x 16-byte tiles
    // (tile h = blocks 4h..4h+3; row i holds tokens i, 32+i, 64+i, 96+i), the form tcgen05.cp spreads.
    // The tile of stage st is free: the copy into the stage waited for the MMAs that read it.
    // The same warp stages the query tile (codes and scales of the group's G heads) of item j+1 while
    // item j is scored: that slot was last read by the MMAs of item j-1.
    WorkIter w, wq;
    w.init(true);
    wq.init(false);
    uint32_t kc = 0, j = 0, n_staged = 0;
    bool ok = true;
    uint4 qv = make_uint4(0u, 0u, 0u, 0u);
    uint32_t qs0 = 0, qs1 = 0;
    bool have_q = false;
    auto load_q = [&]() {   // global loads of the next item's tile, consumed one item later
      have_q = wq.next(cx, ring);
      if (!have_q) return;
      if (lane < G * 4)
        qv = *reinterpret_cast<const uint4 *>(p.q_codes + ((size_t)wq.b * p.H_q + wq.hk * G + (lane >> 2)) * (TILE * 64) + (lane & 3) * 16);
      if (lane < G) {
        const uint8_t *src = p.q_sf + ((size_t)wq.b * p.H_q + wq.hk * G + lane) * 1024;
        qs0 = *reinterpret_cast<const uint32_t *>(src);
        qs1 = *reinterpret_cast<const uint32_t *>(src + 512);
      }
    };
    auto store_q = [&]() {
      if (!have_q) return;
      const uint32_t slot = n_staged & 1;
      if (lane < G * 4) {
        const int n = lane >> 2, c = lane & 3;
        *reinterpret_cast<uint4 *>(dsm + D_OFF_Q + slot * 1024 + n * 64 + ((c ^ ((n & 7) >> 1)) << 4)) = qv;
      }
      if (lane < G) {
        uint8_t *dst = dsm + D_OFF_SFQ + slot * 1024 + lane * 16;
        *reinterpret_cast<uint32_t *>(dst) = qs0;
        *reinterpret_cast<uint32_t *>(dst + 512) = qs1;
      }
      fence_proxy_async_smem();
      cx.warp_arrive(B_Q_READY + slot);
      ++n_staged;
    };
    load_q();
    store_q();
    load_q();
    store_q();
    load_q();
    while (ok && w.next(cx, ring)) {
      if (j >= 1) {
        // all QK MMAs of item j-1 are complete once its last block's scores are
        const uint32_t pj = j - 1;
        ok = cx.wait_warp(B_S_FULL + (pj & 1) * MAXBLK + MAXBLK - 1, (pj >> 1) & 1);
        if (!ok) break;
        store_q();
        load_q();
      }
      ++j;
      for (int t = 0; t < w.nblk; ++t, ++kc) {
        const uint32_t st = kc % D_NK;
        ok = cx.wait_warp(B_K_FULL + st, (kc / D_NK) & 1);
        if (!ok) break;
        const uint8_t *raw = dsm + D_OFF_K + st * KST_BYTES + KST_SF;
        uint2 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = *reinterpret_cast<const uint2 *>(raw + (q >> 1) * 512 + ((q & 1) * 32 + lane) * 8);
        uint8_t *dst = dsm + D_OFF_SFK + st * 1024 + lane * 16;
        *reinterpret_cast<uint4 *>(dst) = make_uint4(v[0].x, v[1].x, v[2].x, v[3].x);
        *reinterpret_cast<uint4 *>(dst + 512) = make_uint4(v[0].y, v[1].y, v[2].y, v[3].y);
        fence_proxy_async_smem();
        cx.warp_arrive(B_SF_READY + st);
        DTR(6, kc);
      }
    }
  } else {
    // ================= softmax, one thread per key of a block (per channel for O^T)
    const int quad = warp & 3;                  // TMEM lane quadrant this warp may touch
    const int r = quad * 32 + lane;             // key within the block / channel of O^T
    const int t128 = (warp - 4) * 32 + lane;    // 0..127 among these warps
    const uint32_t tlane = (uint32_t)(quad * 32) << 16;
    bool ok = true;

    // partition write-out of the item before the current one (its PV MMAs finish meanwhile)
    struct Prev { int b, hk, sp, nblk; };
    auto write_out = [&](const Prev &pr, uint32_t jp) {
      const uint32_t par = jp & 1;
      ok = cx.wait_warp(B_O_FULL, jp & 1);
      if (!ok) return;
      tc_fence_after();
      uint32_t o[MAXBLK][G];
#pragma unroll
      for (int t = 0; t < MAXBLK; ++t)
        if (t < pr.nblk) tmem_ld_g<G>(tm + TM_O + t * 16 + tlane, o[t]);
      tmem_ld_wait();
      tc_fence_before();
      cx.warp_arrive(B_O_FREE);
      float acc[G];
#pragma unroll
      for (int g = 0; g < G; ++g) acc[g] = 0.0f;
#pragma unroll
      for (int t = 0; t < MAXBLK; ++t)
        if (t < pr.nblk) {
#pragma unroll
          for (int g = 0; g < G; ++g) acc[g] = __fmaf_rn(wtab[(par * MAXBLK + t) * MAXG + g], __uint_as_float(o[t][g]), acc[g]);
        }
      float *dst = p.parts + (((size_t)pr.b * p.H_q + (size_t)pr.hk * G) * p.n_split + pr.sp) * PART_FLOATS;
      const size_t head_stride = (size_t)p.n_split * PART_FLOATS;
#pragma unroll
      for (int g = 0; g < G; ++g) dst[g * head_stride + 2 + r] = acc[g];
      if (t128 < G) {
        float l = 0.0f;
#pragma unroll
        for (int q = 0; q < 4; ++q) l += xl[(par * 4 + q) * MAXG + t128];
        dst[t128 * head_stride] = mfin[par * MAXG + t128];
        dst[t128 * head_stride + 1] = l;
      }
    };

    WorkIter w;
    w.init(true);
    uint32_t j = 0;
    Prev prev{0, 0, 0, 0};
    while (ok && w.next(cx, ring)) {
      const uint32_t par = j & 1;
      const float lam = w.b < D_MAXREQ ? lam_tab[w.b]
                                       : __fmul_rn(__fmul_rn(__fmul_rn(p.softmax_scale, 1.4426950408889634f), p.q_gscale[w.b]), p.k_gscale[w.b]);
      const int k_part = w.sp * DECODE_SPLIT;
      // ---- all scores of the item at once: the last slot's barrier follows every QK MMA of the item
      ok = cx.wait_warp(B_S_FULL + par * MAXBLK + MAXBLK - 1, (j >> 1) & 1);
      if (!ok) break;
      if (warp == 4) DTR(7, j);
      tc_fence_after();
      float sv[MAXBLK][G];
      {
        uint32_t sraw[MAXBLK][G];
#pragma unroll
        for (int t = 0; t < MAXBLK; ++t)
          if (t < w.nblk) tmem_ld_g<G>(tm + TM_S + (par * MAXBLK + t) * 16 + tlane, sraw[t]);
        tmem_ld_wait();
        tc_fence_before();
        cx.warp_arrive(B_S_FREE + par);
#pragma unroll
        for (int t = 0; t < MAXBLK; ++t) {
          if (t < w.nblk) {
            const bool valid = k_part + (w.nblk - 1 - t) * TILE + r < w.L;
#pragma unroll
            for (int g = 0; g < G; ++g) {
              sv[t][g] = valid ? __uint_as_float(sraw[t][g]) : -INFINITY;
              // warp maximum through an order-preserving integer key and one redux
              const int bits = __float_as_int(sv[t][g]);
              const int key = bits ^ ((bits >> 31) & 0x7FFFFFFF);
              const int km = __reduce_max_sync(0xffffffffu, key);
              if (lane == 0) xmax[((par * MAXBLK + t) * MAXG + g) * 4 + (warp - 4)] = __int_as_float(km ^ ((km >> 31) & 0x7FFFFFFF));
            }
          }
        }
      }
      if (warp == 4) DTR(8, j);
      cx.warp_arrive(B_XCHG);
      ok = cx.wait_warp(B_XCHG, j & 1);
      if (!ok) break;
      if (warp == 4) DTR(9, j);
      // ---- running maxima of the reverse traversal, then all P_hat of the item
      {
        float m[MAXBLK][G], run[G], lsum[G];
#pragma unroll
        for (int g = 0; g < G; ++g) run[g] = -INFINITY, lsum[g] = 0.0f;
#pragma unroll
        for (int t = 0; t < MAXBLK; ++t) {
          if (t < w.nblk) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
              const float4 x = *reinterpret_cast<const float4 *>(&xmax[((par * MAXBLK + t) * MAXG + g) * 4]);
              run[g] = fmaxf(run[g], fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w)));
              m[t][g] = run[g];
            }
          }
        }
        uint8_t *pt = dsm + D_OFF_P + par * MAXBLK * 1024 + (r & 15);
#pragma unroll
        for (int t = 0; t < MAXBLK; ++t) {
          if (t < w.nblk) {
            float pq[G + 1];
#pragma unroll
            for (int g = 0; g < G; ++g) {
              const float pv = ex2_approx(__fmaf_rn(sv[t][g], lam, -__fmul_rn(m[t][g], lam)));   // -inf -> 0
              float wt = 1.0f;
              if (m[t][g] != run[g]) wt = ex2_approx(__fmul_rn(m[t][g] - run[g], lam));   // uniform, rare
              lsum[g] = __fmaf_rn(wt, pv, lsum[g]);
              pq[g] = __fmul_rn(pv, 448.0f);
              if (t128 == t * G + g) wtab[(par * MAXBLK + t) * MAXG + g] = wt;
            }
            pq[G] = 0.0f;
#pragma unroll
            for (int g = 0; g < G; g += 2) {
              const uint32_t two = (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(pq[g], pq[g + 1]), __NV_SATFINITE, __NV_E4M3);
              pt[t * 1024 + g * 128 + (((r >> 4) ^ g) << 4)] = (uint8_t)two;
              if (g + 1 < G) pt[t * 1024 + (g + 1) * 128 + (((r >> 4) ^ (g + 1)) << 4)] = (uint8_t)(two >> 8);
            }
          }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float ls = lsum[g];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
          if (lane == 0) xl[(par * 4 + (warp - 4)) * MAXG + g] = ls;
          if (t128 == g) mfin[par * MAXG + g] = run[g];
        }
      }
      fence_proxy_async_smem();
      cx.warp_arrive(B_P_READY + par);
      if (warp == 4) DTR(10, j);
      if (j >= 1) {
        write_out(prev, j - 1);
        if (!ok) break;
      }
      if (warp == 4) DTR(11, j);
      prev = Prev{w.b, w.hk, w.sp, w.nblk};
      ++j;
    }
    if (ok && j >= 1) {
      // the tables of the last item were written by other warps: one more exchange round
      cx.warp_arrive(B_XCHG);
      ok = cx.wait_warp(B_XCHG, j & 1);
      if (ok) write_out(prev, j - 1);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tm, TM_COLS);
#ifdef MPFA_TRACE
  if (g_dtrace && threadIdx.x == 0) g_dtrace[4096 + 2 * blockIdx.x + 1] = (long long)globaltimer_ns();
#endif
}

// Merge of the partition states (Section 5.3): M = max m_s, w_s = 2^(lam (m_s - M)),
// l = sum w_s l_s, O = sum w_s O_s, out = O / (448 l) * v_scale.  grid (H_q, B), 256 threads.
__global__ void __launch_bounds__(256) decode_merge_kernel(const float *__restrict__ parts,
                                                           const int32_t *__restrict__ seq_lens,
                                                           const float *__restrict__ q_gscale,
                                                           const float *__restrict__ k_gscale, int H_q, int n_split,
                                                           float softmax_scale, float v_scale,
                                                           __nv_bfloat16 *__restrict__ out, float *__restrict__ out_f32) {
  // 8 warps: warp w takes the partitions s = w, w + 8, ... in ascending order (the loads of four of them in
  // flight together), lane l the channels l, l + 32, l + 64, l + 96; the eight partial sums are then added in
  // warp order.  A fixed order, so the result is reproducible; with one thread walking all partitions a
  // single long request (128 partitions, 32 blocks in the grid) spent 25 us here.
  __shared__ float s_red[8], s_l[8], s_o[8][HEAD_DIM];
  const int hq = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int L = seq_lens[b];
  const int ns = min(n_split, (L + DECODE_SPLIT - 1) / DECODE_SPLIT);
  const float *base = parts + ((size_t)b * H_q + hq) * n_split * PART_FLOATS;
  const float lam = __fmul_rn(__fmul_rn(__fmul_rn(softmax_scale, 1.4426950408889634f), q_gscale[b]), k_gscale[b]);
  float M = -INFINITY;
  for (int s = tid; s < ns; s += 256) M = fmaxf(M, base[(size_t)s * PART_FLOATS]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  if (lane == 0) s_red[warp] = M;
  __syncthreads();
  M = s_red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) M = fmaxf(M, s_red[w]);
  float l = 0.0f, o[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  for (int s0 = warp; s0 < ns; s0 += 32) {
    float ms[4], ls[4], os[4][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int sp = s0 + 8 * j;
      const bool in = sp < ns;
      const float *ps = base + (size_t)(in ? sp : s0) * PART_FLOATS;
      ms[j] = in ? ps[0] : -INFINITY;
      ls[j] = ps[1];
#pragma unroll
      for (int q = 0; q < 4; ++q) os[j][q] = ps[2 + lane + 32 * q];
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (ms[j] == -INFINITY) continue;
      const float w = ex2_approx(__fmul_rn(ms[j] - M, lam));
      l = __fadd_rn(l, __fmul_rn(w, ls[j]));
#pragma unroll
      for (int q = 0; q < 4; ++q) o[q] = __fadd_rn(o[q], __fmul_rn(w, os[j][q]));
    }
  }
  if (lane == 0) s_l[warp] = l;
#pragma unroll
  for (int q = 0; q < 4; ++q) s_o[warp][lane + 32 * q] = o[q];
  __syncthreads();
  if (tid < HEAD_DIM) {
    float lt = s_l[0], ot = s_o[0][tid];
#pragma unroll
    for (int w = 1; w < 8; ++w) {
      lt = __fadd_rn(lt, s_l[w]);
      ot = __fadd_rn(ot, s_o[w][tid]);
    }
    const float r = (lt > 0.0f) ? __fmul_rn(__fdiv_rn(ot, __fmul_rn(448.0f, lt)), v_scale) : 0.0f;
    const size_t idx = ((size_t)b * H_q + hq) * HEAD_DIM + tid;
    out[idx] = __float2bfloat16_rn(r);
    if (out_f32) out_f32[idx] = r;
  }
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

// partition states, then (256-byte aligned) the work counter of the split kernel
static size_t decode_parts_bytes(int B, int H_q, size_t n_split) {
  return ((size_t)B * H_q * n_split * PART_FLOATS * sizeof(float) + 255) / 256 * 256;
}

extern "C" size_t mpfa_decode_workspace_bytes(int B, int H_q, int H_kv, int max_pages_per_req) {
  if (B <= 0 || H_q <= 0 || H_kv <= 0 || max_pages_per_req <= 0) return 0;
  const size_t n_split = ((size_t)max_pages_per_req * PAGE + DECODE_SPLIT - 1) / DECODE_SPLIT;
  return decode_parts_bytes(B, H_q, n_split) + 256;
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
  const size_t need = decode_parts_bytes(B, H_q, n_split) + 256;
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
  p.ticket = reinterpret_cast<unsigned int *>(static_cast<uint8_t *>(workspace) + decode_parts_bytes(B, H_q, n_split));
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
  void (*kern)(const DecodeParams) = nullptr;
  switch (H_q / H_kv) {
    case 1: kern = decode_split_kernel<1>; break;
    case 2: kern = decode_split_kernel<2>; break;
    case 3: kern = decode_split_kernel<3>; break;
    case 4: kern = decode_split_kernel<4>; break;
    case 5: kern = decode_split_kernel<5>; break;
    case 6: kern = decode_split_kernel<6>; break;
    case 7: kern = decode_split_kernel<7>; break;
    case 8: kern = decode_split_kernel<8>; break;
    default: return MPFA_ERR_UNSUPPORTED;
  }
  MPFA_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)D_SMEM));
  MPFA_CUDA_OK(cudaMemsetAsync(p.ticket, 0, sizeof(unsigned int), s));   // a memory-set node, no allocation
  kern<<<grid, D_THREADS, D_SMEM, s>>>(p);
  MPFA_LAUNCH_OK();
  decode_merge_kernel<<<dim3(H_q, B), 256, 0, s>>>(p.parts, seq_lens, st->q_gscale, st->k_gscale, H_q, (int)n_split,
                                                   softmax_scale, v_scale, static_cast<__nv_bfloat16 *>(out_bf16),
                                                   out_f32);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}
