// Stage 1 of the QK4PV8 path (Algorithm 1 lines 1-5): sequence means (Eq. 7), centering,
// per-tensor scales, NVFP4 quantization (Eq. 1) of Q and K into the tile layout consumed
// by the prefill kernel (or the fragment-ordered paged layout consumed by decode), the
// compensation vector Delta_S (Eq. 9) and the FP8 quantization of V.
//
// Everything here is bandwidth work: 16-byte global loads, 8/16-byte stores, tiles staged in
// shared memory where the destination order differs from the source order.  Every
// floating-point step uses an explicitly rounded intrinsic so the results are defined to
// the bit (no FMA contraction, IEEE division).
#include <cuda_bf16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>

#include <algorithm>
#include <mutex>

#include "common.cuh"

namespace mpfa {

thread_local int g_last_cuda_error = 0;

mpfa_status check_arch() {
  int dev = 0, major = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  MPFA_CUDA_OK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  return major == 10 ? MPFA_OK : MPFA_ERR_ARCH;
}

namespace {


__device__ __forceinline__ void unpack8(const uint4 &u, float (&f)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

// One pass over a tensor [B, N, cols] gives, per column, everything the statistics need:
//   the sum in FP64 (Eq. 7);
//   max x and max (-x) - rounding is monotonic and symmetric, so
//   max_t |fl(x_t - mu)| = max(fl(max x - mu), fl(mu - min x)) and no second pass over the tensor is
//   needed for the per-tensor scale.
// The token axis is cut into S contiguous slices.  A CTA covers 256 columns x one slice: thread = (token lane
// 0..7, 8 columns), a warp reads 512 contiguous bytes of one token row, four independent 16-byte loads in
// flight per thread; each thread adds its tokens in ascending order, the eight token lanes are folded in lane
// order in shared memory, and the slice's partial result goes to the workspace.  The finalize kernel adds the S
// partial sums in slice order.  Every addition order is fixed by (N, S), so the result is reproducible bit for
// bit for any input; it equals the oracle's single ascending FP64 sum whenever all these sums are exact (always
// true for BF16 inputs whose exponents span fewer than about 40 binades per column).
constexpr int COLSTAT_COLS = 256;
constexpr int STAT_MAX_SLICES = 32;

// One launch covers up to two tensors (Q and K): blockIdx.y runs over the 256-column groups of the first, then
// of the second; blocks past a tensor's last slice leave at once.  The block that finishes a column group last
// (a counter per group, zeroed by a memory-set node before the launch) adds the slices' partial sums in slice order
// - which block does it cannot change the result - and writes mean = fl(sum / N) (0 without smoothing) and the
// group's max |x - mean| from the column extremes (an exact, order-free maximum); the block that finishes the
// whole launch last turns the per-batch-element maxima into the tensor scales.
struct ColTensor {
  const __nv_bfloat16 *x;   // null: tensor absent (ygroups = 0)
  int N, cols, ygroups, slices, slice_len;
  double *psum;             // [B][slices][cols]
  float *pmax, *pneg;       // [B][slices][cols]
  unsigned int *amax;       // [B], zero at launch
  float *mean, *gscale;
};

__device__ __forceinline__ void colstat_body(const ColTensor &a, const int yg, unsigned int *group_counter,
                                             unsigned int *launch_counter, const unsigned int n_groups, const int smooth,
                                             const ColTensor &t0, const ColTensor &t1) {
  __shared__ double s_sum[8][COLSTAT_COLS];
  __shared__ float s_max[8][COLSTAT_COLS], s_neg[8][COLSTAT_COLS];
  __shared__ bool s_last;
  const int sl = blockIdx.x;
  if (sl >= a.slices) return;
  const int b = blockIdx.z;
  const int N = a.N, cols = a.cols;
  const __nv_bfloat16 *__restrict__ x = a.x;
  const int tl = threadIdx.x >> 5, cg = threadIdx.x & 31;
  const int col = yg * COLSTAT_COLS + cg * 8;
  const int t0i = sl * a.slice_len;
  const int t1i = min(N, t0i + a.slice_len);
  double acc[8];
  float mx[8], ng[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.0, mx[i] = -INFINITY, ng[i] = -INFINITY;
  if (col < cols) {
    const __nv_bfloat16 *p = x + ((size_t)b * N + t0i + tl) * cols + col;
    const size_t step = (size_t)8 * cols;
    int t = t0i + tl;
    // four loads of the next round are in flight while the current four are added (tokens still ascending)
    uint4 u[4], un[4];
    bool have = t + 24 < t1i;
    if (have) {
#pragma unroll
      for (int j = 0; j < 4; ++j) u[j] = __ldcs(reinterpret_cast<const uint4 *>(p + j * step));
    }
    while (have) {
      const bool more = t + 32 + 24 < t1i;
      if (more) {
#pragma unroll
        for (int j = 0; j < 4; ++j) un[j] = __ldcs(reinterpret_cast<const uint4 *>(p + (4 + j) * step));
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float f[8];
        unpack8(u[j], f);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] += (double)f[i], mx[i] = fmaxf(mx[i], f[i]), ng[i] = fmaxf(ng[i], -f[i]);
      }
      t += 32;
      p += 4 * step;
#pragma unroll
      for (int j = 0; j < 4; ++j) u[j] = un[j];
      have = more;
    }
    for (; t < t1i; t += 8, p += step) {
      float f[8];
      unpack8(__ldcs(reinterpret_cast<const uint4 *>(p)), f);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] += (double)f[i], mx[i] = fmaxf(mx[i], f[i]), ng[i] = fmaxf(ng[i], -f[i]);
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) s_sum[tl][cg * 8 + i] = acc[i], s_max[tl][cg * 8 + i] = mx[i], s_neg[tl][cg * 8 + i] = ng[i];
  __syncthreads();
  const int c = yg * COLSTAT_COLS + threadIdx.x;
  if (c < cols) {
    double sum = 0.0;
    float m = -INFINITY, g = -INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j) sum += s_sum[j][threadIdx.x], m = fmaxf(m, s_max[j][threadIdx.x]), g = fmaxf(g, s_neg[j][threadIdx.x]);
    const size_t o = ((size_t)b * a.slices + sl) * cols + c;
    a.psum[o] = sum;
    a.pmax[o] = m;
    a.pneg[o] = g;
  }
  // ---- the last block of this column group folds the slices
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(group_counter, 1u) == (unsigned int)a.slices - 1u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  float m = 0.0f;
  if (c < cols) {
    double sum = 0.0;
    float hi = -INFINITY, ng2 = -INFINITY;
    const size_t o0 = (size_t)b * a.slices * cols + c;
    for (int s0 = 0; s0 < a.slices; s0 += 4) {   // four slices' loads in flight; the additions stay in slice order
      double ps[4];
      float pm[4], pn[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool in = s0 + j < a.slices;
        const size_t o = o0 + (size_t)(s0 + j) * cols;
        ps[j] = in ? __ldcg(a.psum + o) : 0.0;
        pm[j] = in ? __ldcg(a.pmax + o) : -INFINITY;
        pn[j] = in ? __ldcg(a.pneg + o) : -INFINITY;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (s0 + j < a.slices) sum += ps[j];
        hi = fmaxf(hi, pm[j]);
        ng2 = fmaxf(ng2, pn[j]);
      }
    }
    const float mu = smooth ? __double2float_rn(__ddiv_rn(sum, (double)N)) : 0.0f;
    a.mean[(size_t)b * cols + c] = mu;
    m = fmaxf(__fsub_rn(hi, mu), __fsub_rn(mu, -ng2));   // non-negative: lo <= mu <= hi (or mu = 0 and the larger side wins)
    m = fmaxf(m, 0.0f);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float *wmax = &s_max[0][0];
  __syncthreads();
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 1; i < 8; ++i) m = fmaxf(m, wmax[i]);
    atomicMax(&a.amax[b], __float_as_uint(m));   // non-negative floats order like their bit patterns
    __threadfence();
    s_last = atomicAdd(launch_counter, 1u) == n_groups - 1u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int i = threadIdx.x; i < (int)gridDim.z; i += 256) {
    if (t0.x) {
      const float v = __uint_as_float(__ldcg(t0.amax + i));
      t0.gscale[i] = v > 0.0f ? __fdiv_rn(v, 2688.0f) : 1.0f;
    }
    if (t1.x) {
      const float v = __uint_as_float(__ldcg(t1.amax + i));
      t1.gscale[i] = v > 0.0f ? __fdiv_rn(v, 2688.0f) : 1.0f;
    }
  }
}

// counters: [B][ygroups of both tensors] group counters, then one launch counter; all zero at launch
__global__ void __launch_bounds__(256, 3) colstat_kernel(const ColTensor a0, const ColTensor a1, unsigned int *counters, int smooth) {
  const unsigned int groups = (unsigned int)(a0.ygroups + a1.ygroups);
  unsigned int *gc = counters + blockIdx.z * groups + blockIdx.y;
  unsigned int *lc = counters + gridDim.z * groups;
  if ((int)blockIdx.y < a0.ygroups)
    colstat_body(a0, (int)blockIdx.y, gc, lc, groups * gridDim.z, smooth, a0, a1);
  else
    colstat_body(a1, (int)blockIdx.y - a0.ygroups, gc, lc, groups * gridDim.z, smooth, a0, a1);
}

// One NVFP4 block (Eq. 1): 16 centered values -> E4M3 scale code + 8 bytes of E2M1 codes.
__device__ __forceinline__ void quantize_block16(const float (&xc)[16], float d, uint8_t &scale_code, uint2 &codes) {
  float a = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) a = fmaxf(a, fabsf(xc[i]));
  const float e = __fmul_rn(6.0f, d);
  const float r = __fdiv_rn(a, e);
  scale_code = (uint8_t)__nv_cvt_float_to_fp8(r, __NV_SATFINITE, __NV_E4M3);
  const float sdec = __half2float(__half(__nv_cvt_fp8_to_halfraw(scale_code, __NV_E4M3)));
  const float s = __fmul_rn(sdec, d);
  float inv = __fdiv_rn(1.0f, s);
  if (!(s > 0.0f) || isinf(inv)) inv = 0.0f;
  uint32_t w[2] = {0u, 0u};
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float2 v = make_float2(__fmul_rn(xc[2 * i], inv), __fmul_rn(xc[2 * i + 1], inv));
    uint32_t byte = (uint32_t)__nv_cvt_float2_to_fp4x2(v, __NV_E2M1, cudaRoundNearest);
    w[i >> 2] |= (byte & 0xFFu) << (8 * (i & 3));
  }
  codes = make_uint2(w[0], w[1]);
}

__device__ __forceinline__ void load_center16(const __nv_bfloat16 *row, const float *mu, float (&xc)[16]) {
  float f[8];
  unpack8(reinterpret_cast<const uint4 *>(row)[0], f);
#pragma unroll
  for (int i = 0; i < 8; ++i) xc[i] = __fsub_rn(f[i], mu[i]);
  unpack8(reinterpret_cast<const uint4 *>(row)[1], f);
#pragma unroll
  for (int i = 0; i < 8; ++i) xc[8 + i] = __fsub_rn(f[i], mu[8 + i]);
}

struct QuantTensor {
  const __nv_bfloat16 *x;   // null: tensor absent (H = 0)
  const float *mean, *gscale;
  int N, H, tiles;
  uint8_t *codes, *sf;
};

__device__ __forceinline__ void quantize_tile_body(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ mean,
                                                   const float *__restrict__ gscale, const int N, const int H,
                                                   const int tiles, uint8_t *__restrict__ codes,
                                                   uint8_t *__restrict__ sf, const int h, const int tile) {
  __shared__ float mu[HEAD_DIM];
  __shared__ __align__(16) uint8_t sf_tile[1024];
  const int b = blockIdx.z;
  if (tile >= tiles) return;
  const int n_pad = tiles * TILE;
  if (threadIdx.x < HEAD_DIM) mu[threadIdx.x] = mean[((size_t)b * H + h) * HEAD_DIM + threadIdx.x];
  __syncthreads();
  const float d = gscale[b];
  // the thread's block index g = threadIdx.x & 7 is the same in all four iterations: its 16 means live in registers
  // (read from shared memory per block they cost 4-way bank conflicts: the data pipe was the kernel's limiter)
  float mreg[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) mreg[i] = mu[(threadIdx.x & 7) * 16 + i];
  // all eight 16-byte loads of the thread's four blocks are issued before the first block is quantized
  uint4 raw[4][2];
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int r = id >> 3, g = id & 7;
    const int t = tile * TILE + r;
    raw[it][0] = raw[it][1] = make_uint4(0u, 0u, 0u, 0u);
    if (t < N) {
      const uint4 *src = reinterpret_cast<const uint4 *>(x + (((size_t)b * N + t) * H + h) * HEAD_DIM + g * 16);
      raw[it][0] = __ldcs(src);
      raw[it][1] = __ldcs(src + 1);
    }
  }
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int r = id >> 3, g = id & 7;
    const int t = tile * TILE + r;
    uint2 c = make_uint2(0u, 0u);
    uint8_t sc = 0;
    if (t < N) {
      float xc[16], f[8];
      unpack8(raw[it][0], f);
#pragma unroll
      for (int i = 0; i < 8; ++i) xc[i] = __fsub_rn(f[i], mreg[i]);
      unpack8(raw[it][1], f);
#pragma unroll
      for (int i = 0; i < 8; ++i) xc[8 + i] = __fsub_rn(f[i], mreg[8 + i]);
      quantize_block16(xc, d, sc, c);
    }
    __stcs(reinterpret_cast<uint2 *>(codes + (((size_t)b * H + h) * n_pad + t) * 64 + g * 8), c);
    sf_tile[(g >> 2) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (g & 3)] = sc;
  }
  __syncthreads();
  uint32_t *dst = reinterpret_cast<uint32_t *>(sf + (((size_t)b * H + h) * tiles + tile) * 1024);
  dst[threadIdx.x] = reinterpret_cast<const uint32_t *>(sf_tile)[threadIdx.x];
}

// K tile with the compensation vector (Eq. 9) in the same pass: the tile's rows are staged once in shared memory
// (coalesced 16-byte loads; a row is 256 contiguous bytes, rows of one head are H_kv * 256 bytes apart; row pitch
// 272 bytes so that the 16-byte reads of 8 consecutive threads fall into 8 different bank groups), quantized from
// there exactly like a Q tile, and then every key's Delta_S[hq][t] = qmean[hq] . (k[t] - kmean) is accumulated in
// FP64 with channels ascending by thread (key, part), part taking the heads g = part, part + 2, ... of the group as
// independent sequential chains; the result is expressed in units of gscale_q * gscale_k and rounded once to BF16.
struct DeltaArgs {
  const float *q_mean;     // null: no Delta_S (direct variant or statistics-only call)
  const float *q_gscale;
  __nv_bfloat16 *delta;    // [B, H_q, N_pad]
  int H_q;
};

constexpr int KROW_PITCH = 272;
constexpr int KTILE_SMEM = TILE * KROW_PITCH + 8 * HEAD_DIM * 8;   // staged rows + FP64 query means of the group

__device__ __forceinline__ void quantize_k_tile_delta_body(const QuantTensor &a, const DeltaArgs &da, const int h,
                                                           const int tile, uint8_t *dyn) {
  constexpr int MAXG = 8;
  __shared__ float mu[HEAD_DIM];
  __shared__ __align__(16) uint8_t sf_tile[1024];
  uint8_t *rows = dyn;
  double(*qmu)[HEAD_DIM] = reinterpret_cast<double(*)[HEAD_DIM]>(dyn + TILE * KROW_PITCH);
  const int b = blockIdx.z;
  if (tile >= a.tiles) return;
  const int N = a.N, H = a.H, n_pad = a.tiles * TILE;
  const int G = da.H_q / H;
  if (threadIdx.x < HEAD_DIM) mu[threadIdx.x] = a.mean[((size_t)b * H + h) * HEAD_DIM + threadIdx.x];
  for (int j = threadIdx.x; j < G * HEAD_DIM; j += 256)
    qmu[j >> 7][j & 127] = (double)da.q_mean[((size_t)b * da.H_q + h * G + (j >> 7)) * HEAD_DIM + (j & 127)];
  for (int i = threadIdx.x; i < TILE * 16; i += 256) {
    const int r = i >> 4, ch = i & 15;
    const int tt = tile * TILE + r;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (tt < N) v = __ldcs(reinterpret_cast<const uint4 *>(a.x + (((size_t)b * N + tt) * H + h) * HEAD_DIM + ch * 8));
    *reinterpret_cast<uint4 *>(rows + r * KROW_PITCH + ch * 16) = v;
  }
  __syncthreads();
  const float d = a.gscale[b];
  float mreg[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) mreg[i] = mu[(threadIdx.x & 7) * 16 + i];
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int r = id >> 3, g = id & 7;
    const int t = tile * TILE + r;
    uint2 c = make_uint2(0u, 0u);
    uint8_t sc = 0;
    if (t < N) {
      float xc[16];
      load_center16(reinterpret_cast<const __nv_bfloat16 *>(rows + r * KROW_PITCH + g * 32), mreg, xc);
      quantize_block16(xc, d, sc, c);
    }
    *reinterpret_cast<uint2 *>(a.codes + (((size_t)b * H + h) * n_pad + t) * 64 + g * 8) = c;
    sf_tile[(g >> 2) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (g & 3)] = sc;
  }
  // Delta_S.  The FP64 pipe is the scarce unit here (measured: an eighth of the FP32 rate on this GPU); two threads
  // per key, each with the chains of every other head of the group, keep enough independent chains in flight to
  // cover its latency.
  {
    const int key = threadIdx.x & 127, part = threadIdx.x >> 7;
    const int t = tile * TILE + key;
    double acc[MAXG / 2];
#pragma unroll
    for (int u = 0; u < MAXG / 2; ++u) acc[u] = 0.0;
    if (t < N) {
      const uint8_t *row = rows + key * KROW_PITCH;
      for (int c0 = 0; c0 < HEAD_DIM; c0 += 8) {
        float f[8];
        unpack8(*reinterpret_cast<const uint4 *>(row + c0 * 2), f);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const double kc = (double)__fsub_rn(f[i], mu[c0 + i]);
#pragma unroll
          for (int u = 0; u < MAXG / 2; ++u)
            if (2 * u + part < G) acc[u] = fma(qmu[2 * u + part][c0 + i], kc, acc[u]);
        }
      }
    }
    const double denom = (double)da.q_gscale[b] * (double)d;
#pragma unroll
    for (int u = 0; u < MAXG / 2; ++u) {
      const int g = 2 * u + part;
      if (g < G) {
        const float v = (t < N) ? __double2float_rn(__ddiv_rn(acc[u], denom)) : 0.0f;
        da.delta[((size_t)b * da.H_q + h * G + g) * n_pad + t] = __float2bfloat16_rn(v);
      }
    }
  }
  __syncthreads();
  uint32_t *dst = reinterpret_cast<uint32_t *>(a.sf + (((size_t)b * H + h) * a.tiles + tile) * 1024);
  dst[threadIdx.x] = reinterpret_cast<const uint32_t *>(sf_tile)[threadIdx.x];
}

// grid (max tiles * (H of the first + H of the second tensor), 1, B); one 128-token tile of one head per block,
// blockIdx.x = tile * heads + head: the head index runs fastest, so the blocks resident at any time read whole token
// rows of the [B, N, H, 128] input (contiguous DRAM) instead of 256-byte pieces 256 * H bytes apart.
__global__ void __launch_bounds__(256) quantize_fp4_tile_kernel(const QuantTensor a0, const QuantTensor a1) {
  const int heads = a0.H + a1.H;
  const int tile = (int)blockIdx.x / heads, y = (int)blockIdx.x % heads;
  if (y < a0.H)
    quantize_tile_body(a0.x, a0.mean, a0.gscale, a0.N, a0.H, a0.tiles, a0.codes, a0.sf, y, tile);
  else
    quantize_tile_body(a1.x, a1.mean, a1.gscale, a1.N, a1.H, a1.tiles, a1.codes, a1.sf, y - a0.H, tile);
}

// grid (tiles * H_kv, 1, B), KTILE_SMEM bytes of dynamic shared memory: K tiles with Delta_S, blockIdx.x = tile * H_kv +
// head.  A launch of its own: these blocks are bound by the FP64 pipe, the Q tiles by memory, and in one launch
// (kinds interleaved) they only competed for block slots (98 us against 42 + 38 at 16K).
__global__ void __launch_bounds__(256) quantize_k_delta_kernel(const QuantTensor a, const DeltaArgs da) {
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  quantize_k_tile_delta_body(a, da, (int)blockIdx.x % a.H, (int)blockIdx.x / a.H, dyn_smem);
}

// Eq. 9: Delta_S[hq][t] = qmean[hq] . (k[t] - kmean), FP64 accumulation with channels ascending,
// expressed in units of gscale_q * gscale_k and rounded once to BF16.  Two threads per key token
// (256 threads per 128-token tile): thread (key, part) takes the heads g = part, part + 2, ... of the
// group, each as its own sequential chain.  grid (N_pad/128, H_kv, B).  Used for the paged side cache (PAGED: the
// entries go to their page through the page-table row); the dense vector of mpfa_quantize_qk comes out of
// quantize_k_delta_kernel, which runs the same chains on rows it has already staged.
template <bool PAGED>
__global__ void __launch_bounds__(256) delta_s_kernel(const __nv_bfloat16 *__restrict__ k,
                                                      const float *__restrict__ q_mean,
                                                      const float *__restrict__ k_mean,
                                                      const float *__restrict__ q_gscale,
                                                      const float *__restrict__ k_gscale, int N, int H_q, int H_kv,
                                                      __nv_bfloat16 *__restrict__ delta,
                                                      const int32_t *__restrict__ page_row, int num_pages) {
  constexpr int MAXG = 8;
  __shared__ float kmu[HEAD_DIM];
  __shared__ double qmu[MAXG][HEAD_DIM];   // converted once: the conversion is as costly as the FMA
  const int tile = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int G = H_q / H_kv;
  const int n_pad = gridDim.x * TILE;
  if (threadIdx.x < HEAD_DIM) kmu[threadIdx.x] = k_mean[((size_t)b * H_kv + hk) * HEAD_DIM + threadIdx.x];
  for (int j = threadIdx.x; j < G * HEAD_DIM; j += 256)
    qmu[j >> 7][j & 127] = (double)q_mean[((size_t)b * H_q + hk * G + (j >> 7)) * HEAD_DIM + (j & 127)];
  __syncthreads();
  // The tile's K rows are staged in shared memory with coalesced 16-byte loads (a row is 256 contiguous
  // bytes, rows of one head are H_kv * 256 bytes apart); each thread then walks its own row.  Row pitch
  // 272 bytes: the 16-byte reads of 8 consecutive threads fall into 8 different bank groups.
  constexpr int PITCH = 272;
  __shared__ __align__(16) uint8_t rows[TILE * PITCH];
  for (int i = threadIdx.x; i < TILE * 16; i += 256) {
    const int r = i >> 4, ch = i & 15;
    const int tt = tile * TILE + r;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (tt < N) v = *reinterpret_cast<const uint4 *>(k + (((size_t)b * N + tt) * H_kv + hk) * HEAD_DIM + ch * 8);
    *reinterpret_cast<uint4 *>(rows + r * PITCH + ch * 16) = v;
  }
  __syncthreads();
  const int key = threadIdx.x & 127, part = threadIdx.x >> 7;
  const int t = tile * TILE + key;
  double acc[MAXG / 2];
#pragma unroll
  for (int u = 0; u < MAXG / 2; ++u) acc[u] = 0.0;
  if (t < N) {
    const uint8_t *row = rows + key * PITCH;
    for (int c0 = 0; c0 < HEAD_DIM; c0 += 8) {
      float f[8];
      unpack8(*reinterpret_cast<const uint4 *>(row + c0 * 2), f);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const double kc = (double)__fsub_rn(f[i], kmu[c0 + i]);
#pragma unroll
        for (int u = 0; u < MAXG / 2; ++u)
          if (2 * u + part < G) acc[u] = fma(qmu[2 * u + part][c0 + i], kc, acc[u]);
      }
    }
  }
  const double denom = (double)q_gscale[b] * (double)k_gscale[b];
#pragma unroll
  for (int u = 0; u < MAXG / 2; ++u) {
    const int g = 2 * u + part;
    if (g < G) {
      const float v = (t < N) ? __double2float_rn(__ddiv_rn(acc[u], denom)) : 0.0f;
      if (PAGED) {
        if ((t >> 6) < (N + PAGE - 1) / PAGE) {   // slots past N inside the last page are zero-filled
          const int page = page_row[t >> 6];
          if (page >= 0 && page < num_pages)
            // 16-byte chunks XOR-swizzled by the head's index in its group: the row is read as a
            // swizzled MN-major tensor-core operand by the decode kernel
            delta[((size_t)page * H_q + hk * G + g) * PAGE + (((((t & 63) >> 3) ^ g) << 3) | (t & 7))] = __float2bfloat16_rn(v);
        }
      } else {
        delta[((size_t)b * H_q + hk * G + g) * n_pad + t] = __float2bfloat16_rn(v);
      }
    }
  }
}

__device__ __forceinline__ uint4 quantize_v16(const __nv_bfloat16 *row, float inv) {
  float f[16];
  {
    float t8[8];
    unpack8(reinterpret_cast<const uint4 *>(row)[0], t8);
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = t8[i];
    unpack8(reinterpret_cast<const uint4 *>(row)[1], t8);
#pragma unroll
    for (int i = 0; i < 8; ++i) f[8 + i] = t8[i];
  }
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint32_t lo = (uint32_t)__nv_cvt_float2_to_fp8x2(
        make_float2(__fmul_rn(f[4 * i], inv), __fmul_rn(f[4 * i + 1], inv)), __NV_SATFINITE, __NV_E4M3);
    uint32_t hi = (uint32_t)__nv_cvt_float2_to_fp8x2(
        make_float2(__fmul_rn(f[4 * i + 2], inv), __fmul_rn(f[4 * i + 3], inv)), __NV_SATFINITE, __NV_E4M3);
    w[i] = (lo & 0xFFFFu) | (hi << 16);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// grid (N_pad/128, H, B): V tile -> [B, H, N_pad, 128] E4M3.
__global__ void __launch_bounds__(256) quantize_v_tile_kernel(const __nv_bfloat16 *__restrict__ v, int N, int H,
                                                              float inv_scale, uint8_t *__restrict__ out) {
  const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int n_pad = gridDim.x * TILE;
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int r = id >> 3, seg = id & 7;
    const int t = tile * TILE + r;
    uint4 c = make_uint4(0u, 0u, 0u, 0u);
    if (t < N) c = quantize_v16(v + (((size_t)b * N + t) * H + h) * HEAD_DIM + seg * 16, inv_scale);
    *reinterpret_cast<uint4 *>(out + (((size_t)b * H + h) * n_pad + t) * HEAD_DIM + seg * 16) = c;
  }
}

// grid (N_pad/128, H, B): V tile -> [B, H, N_pad, 128] BF16, unchanged values (the NVFP4 + BF16 precision assignment
// of Section 3.1 reads V in BF16); pad rows zero.
__global__ void __launch_bounds__(256) pack_v_bf16_kernel(const __nv_bfloat16 *__restrict__ v, int N, int H,
                                                          __nv_bfloat16 *__restrict__ out) {
  const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int n_pad = gridDim.x * TILE;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int r = id >> 4, seg = id & 15;
    const int t = tile * TILE + r;
    uint4 c = make_uint4(0u, 0u, 0u, 0u);
    if (t < N) c = *reinterpret_cast<const uint4 *>(v + (((size_t)b * N + t) * H + h) * HEAD_DIM + seg * 8);
    *reinterpret_cast<uint4 *>(out + (((size_t)b * H + h) * n_pad + t) * HEAD_DIM + seg * 8) = c;
  }
}

// grid (N_pad/128, H, B): V tile for the NVFP4 + NVFP4 precision assignment of Section 3.1.  The second MMA contracts
// over the keys, so the 16-element blocks of Eq. 1 lie along the token axis and the operand is stored channel-major
// (K-major B operand): codes [B, H, N_pad/128, 128 channels, 64 bytes] (two keys per byte, the even key in the low
// nibble), block scales as two 512-byte tcgen05.cp atoms per tile (atom = 64 keys: byte (c mod 32) 16 + (c / 32) 4 +
// block mod 4).  Recipe of the Q/K quantizer with the caller's tensor scale d and no centering; keys past N are zero.
__global__ void __launch_bounds__(256) quantize_v_fp4_tile_kernel(const __nv_bfloat16 *__restrict__ v, int N, int H, float d,
                                                                  uint8_t *__restrict__ codes, uint8_t *__restrict__ sf) {
  __shared__ __align__(16) __nv_bfloat16 tile[TILE][HEAD_DIM + 8];   // padded rows: the column reads below stay conflict-free
  __shared__ __align__(16) uint8_t ctile[HEAD_DIM][64];
  __shared__ __align__(16) uint8_t stile[1024];
  const int t0 = blockIdx.x * TILE, h = blockIdx.y, b = blockIdx.z;
  const int n_tiles = gridDim.x;
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int r = id >> 4, seg = id & 15;
    uint4 u = make_uint4(0u, 0u, 0u, 0u);
    if (t0 + r < N) u = __ldcs(reinterpret_cast<const uint4 *>(v + (((size_t)b * N + t0 + r) * H + h) * HEAD_DIM + seg * 8));
    *reinterpret_cast<uint4 *>(&tile[r][seg * 8]) = u;
  }
  __syncthreads();
#pragma unroll 1
  for (int it = 0; it < 4; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int c = id & 127, kb = id >> 7;   // channel, 16-key block of the tile
    float x[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = __bfloat162float(tile[kb * 16 + i][c]);
    uint8_t sc;
    uint2 cw;
    quantize_block16(x, d, sc, cw);
    *reinterpret_cast<uint2 *>(&ctile[c][kb * 8]) = cw;
    stile[(kb >> 2) * 512 + (c & 31) * 16 + (c >> 5) * 4 + (kb & 3)] = sc;
  }
  __syncthreads();
  const size_t tile_id = ((size_t)b * H + h) * n_tiles + blockIdx.x;
  uint4 *cdst = reinterpret_cast<uint4 *>(codes + tile_id * 8192);
#pragma unroll
  for (int it = 0; it < 2; ++it) cdst[it * 256 + threadIdx.x] = reinterpret_cast<const uint4 *>(&ctile[0][0])[it * 256 + threadIdx.x];
  if (threadIdx.x < 64) reinterpret_cast<uint4 *>(sf + tile_id * 1024)[threadIdx.x] = reinterpret_cast<const uint4 *>(stile)[threadIdx.x];
}

// Paged cache write for one request: grid (pages, H_kv).  K and V of one (page, head) are
// quantized into shared memory in the byte order of the decode kernel's shared-memory operand
// tiles (so that decode fills a tile with one bulk copy) and copied out with 16-byte stores.
__global__ void __launch_bounds__(256) quantize_kv_page_kernel(const __nv_bfloat16 *__restrict__ k,
                                                               const __nv_bfloat16 *__restrict__ v,
                                                               const float *__restrict__ k_mean,
                                                               const float *__restrict__ k_gscale, int N, int H_kv,
                                                               float inv_vscale, const int32_t *__restrict__ page_row,
                                                               int first_page, int num_pages,
                                                               uint8_t *__restrict__ k_codes, uint8_t *__restrict__ k_sf,
                                                               uint8_t *__restrict__ v_fp8) {
  __shared__ float mu[HEAD_DIM];
  __shared__ __align__(16) uint8_t sk[4096];
  __shared__ __align__(16) uint8_t ssf[512];
  __shared__ __align__(16) uint8_t sv[8192];
  const int lp = blockIdx.x, h = blockIdx.y;
  const int page = page_row[first_page + lp];
  if (page < 0 || page >= num_pages) return;  // the host validates the shape; a bad id is skipped
  if (threadIdx.x < HEAD_DIM) mu[threadIdx.x] = k_mean[(size_t)h * HEAD_DIM + threadIdx.x];
  __syncthreads();
  const float d = k_gscale[0];
#pragma unroll
  for (int it = 0; it < 2; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int t = id >> 3, g = id & 7;   // token in page, 16-channel block / segment
    const int tok = lp * PAGE + t;
    uint2 c = make_uint2(0u, 0u);
    uint8_t sc = 0;
    uint4 vc = make_uint4(0u, 0u, 0u, 0u);
    if (tok < N) {
      float xc[16];
      load_center16(k + ((size_t)tok * H_kv + h) * HEAD_DIM + g * 16, mu + g * 16, xc);
      quantize_block16(xc, d, sc, c);
      vc = quantize_v16(v + ((size_t)tok * H_kv + h) * HEAD_DIM + g * 16, inv_vscale);
    }
    // K: the 8 code bytes of block g of token t, in the 64-byte-swizzled row order the decode
    // kernel's tensor-core descriptor reads: (t/8)*512 + (t%8)*64 + ((g/2) ^ ((t%8)/2))*16 + (g%2)*8
    *reinterpret_cast<uint2 *>(sk + (t >> 3) * 512 + (t & 7) * 64 + (((g >> 1) ^ ((t & 7) >> 1)) << 4) + (g & 1) * 8) = c;
    ssf[t * 8 + g] = sc;
    // V: channels 16g..16g+15 of token t, 128-byte-swizzled: (t/8)*1024 + (t%8)*128 + (g ^ (t%8))*16
    *reinterpret_cast<uint4 *>(sv + (t >> 3) * 1024 + (t & 7) * 128 + ((g ^ (t & 7)) << 4)) = vc;
  }
  __syncthreads();
  const size_t slab = (size_t)page * H_kv + h;
  reinterpret_cast<uint4 *>(k_codes + slab * 4096)[threadIdx.x] = reinterpret_cast<const uint4 *>(sk)[threadIdx.x];
  if (threadIdx.x < 32) reinterpret_cast<uint4 *>(k_sf + slab * 512)[threadIdx.x] = reinterpret_cast<const uint4 *>(ssf)[threadIdx.x];
  reinterpret_cast<uint4 *>(v_fp8 + slab * 8192)[threadIdx.x] = reinterpret_cast<const uint4 *>(sv)[threadIdx.x];
  reinterpret_cast<uint4 *>(v_fp8 + slab * 8192)[threadIdx.x + 256] = reinterpret_cast<const uint4 *>(sv)[threadIdx.x + 256];
}

// Decode-time append (Section 6: new tokens are centered with the frozen means and quantized with the
// frozen tensor scale): tokens first_token .. first_token + N - 1 of one request go to their slots of the
// paged cache, wherever in a page they fall.  Thread = (token slot, 16-channel block); a block covers 32
// slots of one kv head.  The grid runs to the end of the last page touched: slots past the last new token
// are zero-filled if this call started their page (a recycled page may hold anything, and decode needs
// finite bytes there); slots of a page that was started earlier are left alone.
__global__ void __launch_bounds__(256) append_kv_kernel(const __nv_bfloat16 *__restrict__ k,
                                                        const __nv_bfloat16 *__restrict__ v,
                                                        const float *__restrict__ q_mean,
                                                        const float *__restrict__ k_mean,
                                                        const float *__restrict__ q_gscale,
                                                        const float *__restrict__ k_gscale, int N, int first_token,
                                                        int H_q, int H_kv, float inv_vscale, int smooth,
                                                        const int32_t *__restrict__ page_row, int num_pages,
                                                        uint8_t *__restrict__ k_codes, uint8_t *__restrict__ k_sf,
                                                        uint8_t *__restrict__ v_fp8, __nv_bfloat16 *__restrict__ delta,
                                                        const int32_t *__restrict__ positions, int max_pages) {
  constexpr int MAXG = 8;
  __shared__ float kmu[HEAD_DIM];
  __shared__ double qmu[MAXG][HEAD_DIM];
  __shared__ float kc[32][HEAD_DIM + 4];   // centered K rows of the block's tokens (for Delta_S)
  if (positions) {
    // batch form: request blockIdx.z appends the one token k[b] / v[b] at index positions[b] with its own
    // statistics and page-table row; a negative position skips the request
    const int b = blockIdx.z;
    first_token = positions[b];
    if (first_token < 0) return;
    N = 1;
    k += (size_t)b * H_kv * HEAD_DIM;
    v += (size_t)b * H_kv * HEAD_DIM;
    q_mean += (size_t)b * H_q * HEAD_DIM;
    k_mean += (size_t)b * H_kv * HEAD_DIM;
    q_gscale += b;
    k_gscale += b;
    page_row += (size_t)b * max_pages;
    if ((first_token >> 6) >= max_pages) return;   // no page-table entry for that position
  }
  const int h = blockIdx.y, G = H_q / H_kv;
  const int slot = threadIdx.x >> 3, g = threadIdx.x & 7;
  const int i = blockIdx.x * 32 + slot;          // index among the slots this call covers
  const int tok = first_token + i;               // absolute token position
  const bool is_new = i < N;
  const bool in_range = tok < ((first_token + N + PAGE - 1) / PAGE) * PAGE;   // the grid is rounded up to 32 slots
  if (threadIdx.x < HEAD_DIM) kmu[threadIdx.x] = k_mean[(size_t)h * HEAD_DIM + threadIdx.x];
  if (smooth)
    for (int j = threadIdx.x; j < G * HEAD_DIM; j += 256)
      qmu[j >> 7][j & 127] = (double)q_mean[((size_t)h * G + (j >> 7)) * HEAD_DIM + (j & 127)];
  __syncthreads();
  const int page = in_range ? page_row[tok >> 6] : -1;
  const bool page_ok = page >= 0 && page < num_pages;
  const bool fresh_pad = !is_new && (tok & ~63) >= first_token;   // padding slot of a page this call started
  const int t = tok & 63;
  uint2 c = make_uint2(0u, 0u);
  uint8_t sc = 0;
  uint4 vc = make_uint4(0u, 0u, 0u, 0u);
  if (is_new) {
    float xc[16];
    load_center16(k + ((size_t)i * H_kv + h) * HEAD_DIM + g * 16, kmu + g * 16, xc);
    quantize_block16(xc, k_gscale[0], sc, c);
    vc = quantize_v16(v + ((size_t)i * H_kv + h) * HEAD_DIM + g * 16, inv_vscale);
#pragma unroll
    for (int j = 0; j < 16; ++j) kc[slot][g * 16 + j] = xc[j];
  }
  if (page_ok && (is_new || fresh_pad)) {
    const size_t slab = (size_t)page * H_kv + h;
    *reinterpret_cast<uint2 *>(k_codes + slab * 4096 + (t >> 3) * 512 + (t & 7) * 64 + (((g >> 1) ^ ((t & 7) >> 1)) << 4) + (g & 1) * 8) = c;
    k_sf[slab * 512 + t * 8 + g] = sc;
    *reinterpret_cast<uint4 *>(v_fp8 + slab * 8192 + (t >> 3) * 1024 + (t & 7) * 128 + ((g ^ (t & 7)) << 4)) = vc;
  }
  __syncthreads();
  // Delta_S (Eq. 9) of the new tokens: thread (slot, g) takes head g of the group, FP64, channels ascending
  if (smooth && g < G && page_ok && (is_new || fresh_pad)) {
    float val = 0.0f;
    if (is_new) {
      double acc = 0.0;
      for (int ch = 0; ch < HEAD_DIM; ++ch) acc = fma(qmu[g][ch], (double)kc[slot][ch], acc);
      val = __double2float_rn(__ddiv_rn(acc, (double)q_gscale[0] * (double)k_gscale[0]));
    }
    delta[((size_t)page * H_q + h * G + g) * PAGE + ((((t >> 3) ^ g) << 3) | (t & 7))] = __float2bfloat16_rn(val);
  }
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// Workspace of the statistics pass: for each tensor S slices of per-column partial results (FP64 sum, maximum,
// maximum of the negated values), then the per-batch-element maxima and one counter word.  S is the largest
// slice count <= STAT_MAX_SLICES that fits the bytes the caller gave (at least 1).
struct StatsWorkspace {
  double *psum_q, *psum_k;
  float *pmax_q, *pneg_q, *pmax_k, *pneg_k;
  unsigned int *amax_q, *amax_k, *counter;
  uint8_t *fixed;
  size_t fixed_bytes;
  int slices;
  size_t bytes;
};

// amax words of both tensors, a counter per (batch element, 256-column group) and the launch counter
size_t stats_fixed_bytes(int B, int H_q, int H_kv) {
  return align256(((size_t)2 * B + (size_t)B * ((H_q + 1) / 2 + (H_kv + 1) / 2) + 1) * sizeof(unsigned int));
}
size_t stats_slice_bytes(int B, int H_q, int H_kv) {   // one slice of both tensors
  return align256((size_t)B * H_q * HEAD_DIM * 8) + 2 * align256((size_t)B * H_q * HEAD_DIM * 4) +
         align256((size_t)B * H_kv * HEAD_DIM * 8) + 2 * align256((size_t)B * H_kv * HEAD_DIM * 4);
}

StatsWorkspace carve(void *ws, size_t ws_bytes, int B, int H_q, int H_kv) {
  StatsWorkspace w{};
  const size_t fixed = stats_fixed_bytes(B, H_q, H_kv), per = stats_slice_bytes(B, H_q, H_kv);
  size_t S = ws_bytes > fixed ? (ws_bytes - fixed) / per : 0;
  if (S > (size_t)STAT_MAX_SLICES) S = STAT_MAX_SLICES;
  w.slices = (int)S;
  size_t o = 0;
  uint8_t *base = static_cast<uint8_t *>(ws);
  const size_t nq = (size_t)B * H_q * HEAD_DIM, nk = (size_t)B * H_kv * HEAD_DIM;
  w.psum_q = reinterpret_cast<double *>(base + o);  o += S * align256(nq * 8);
  w.psum_k = reinterpret_cast<double *>(base + o);  o += S * align256(nk * 8);
  w.pmax_q = reinterpret_cast<float *>(base + o);   o += S * align256(nq * 4);
  w.pneg_q = reinterpret_cast<float *>(base + o);   o += S * align256(nq * 4);
  w.pmax_k = reinterpret_cast<float *>(base + o);   o += S * align256(nk * 4);
  w.pneg_k = reinterpret_cast<float *>(base + o);   o += S * align256(nk * 4);
  w.fixed = base + o;                                      // zeroed before every statistics launch
  w.fixed_bytes = fixed;
  w.amax_q = reinterpret_cast<unsigned int *>(base + o);
  w.amax_k = w.amax_q + B;
  w.counter = w.amax_k + B;
  o += fixed;
  w.bytes = o;
  return w;
}

// One tensor [B, N, H, 128] of a statistics pass (x == nullptr: absent).
struct StatsJob {
  const __nv_bfloat16 *x;
  int N, H;
  double *psum;
  float *pmax, *pneg;
  unsigned int *amax;
  float *mean, *gscale;
};

// Means and per-tensor scales of up to two tensors: one pass over the data, one memory-set node (the amax words
// and counters) and one launch.
mpfa_status tensor_stats(const StatsJob &j0, const StatsJob &j1, int B, const StatsWorkspace &w, bool smooth, cudaStream_t st) {
  ColTensor c[2];
  int slices_x = 0;
  const StatsJob *jobs[2] = {&j0, &j1};
  // as many slices as keep the whole launch resident at once (three 256-thread blocks per SM), within what the
  // workspace holds
  int dev = 0, n_sm = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  MPFA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
  int groups = 0;
  for (int i = 0; i < 2; ++i)
    if (jobs[i]->x) groups += (jobs[i]->H * HEAD_DIM + COLSTAT_COLS - 1) / COLSTAT_COLS;
  if (groups == 0) return MPFA_OK;
  const int max_slices = std::min(w.slices, std::max(1, 3 * n_sm / (groups * B)));
  for (int i = 0; i < 2; ++i) {
    const StatsJob &j = *jobs[i];
    const int cols = j.H * HEAD_DIM;
    // slices of at least 256 tokens, a multiple of 8 tokens long (the eight token lanes of a CTA)
    int S = j.x ? std::min(max_slices, std::max(1, (j.N + 255) / 256)) : 0;
    const int len = j.x ? ((j.N + S - 1) / S + 7) / 8 * 8 : 0;
    if (j.x) S = (j.N + len - 1) / len;
    c[i] = ColTensor{j.x, j.x ? j.N : 0, cols, j.x ? (cols + COLSTAT_COLS - 1) / COLSTAT_COLS : 0, S, len, j.psum, j.pmax,
                     j.pneg, j.amax, j.mean, j.gscale};
    if (j.x) slices_x = std::max(slices_x, S);
  }
  MPFA_CUDA_OK(cudaMemsetAsync(w.fixed, 0, w.fixed_bytes, st));
  colstat_kernel<<<dim3(slices_x, c[0].ygroups + c[1].ygroups, B), 256, 0, st>>>(c[0], c[1], w.counter, smooth ? 1 : 0);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

}  // namespace
}  // namespace mpfa

using namespace mpfa;

extern "C" size_t mpfa_quantize_workspace_bytes(int B, int H_q, int H_kv) {
  if (B <= 0 || H_q <= 0 || H_kv <= 0) return 0;
  return stats_fixed_bytes(B, H_q, H_kv) + (size_t)STAT_MAX_SLICES * stats_slice_bytes(B, H_q, H_kv);
}

extern "C" size_t mpfa_quantize_workspace_min_bytes(int B, int H_q, int H_kv) {
  if (B <= 0 || H_q <= 0 || H_kv <= 0) return 0;
  return stats_fixed_bytes(B, H_q, H_kv) + stats_slice_bytes(B, H_q, H_kv);
}

extern "C" mpfa_status mpfa_quantize_qk(const void *q_bf16, const void *k_bf16, int B, int N_q, int N_kv, int H_q,
                                        int H_kv, int flags, mpfa_stats *st, mpfa_fp4_tensor *q_out,
                                        mpfa_fp4_tensor *k_out, void *delta_s_bf16, void *workspace,
                                        size_t workspace_bytes, void *stream) {
  const bool smooth = flags & MPFA_SMOOTH, frozen = flags & MPFA_STATS_FROZEN;
  if (!st || (!q_bf16 && !k_bf16) || B <= 0 || H_q <= 0 || H_kv <= 0) return MPFA_ERR_INVALID_ARG;
  if ((q_bf16 && (N_q <= 0 || !q_out)) || (k_bf16 && (N_kv <= 0 || !k_out))) return MPFA_ERR_INVALID_ARG;
  if (!st->q_mean || !st->k_mean || !st->q_gscale || !st->k_gscale) return MPFA_ERR_INVALID_ARG;
  if (H_q % H_kv != 0 || H_q / H_kv > 8) return MPFA_ERR_UNSUPPORTED;
  if (N_q > (1 << 24) || N_kv > (1 << 24)) return MPFA_ERR_UNSUPPORTED;
  if (smooth && k_bf16 && !delta_s_bf16) return MPFA_ERR_INVALID_ARG;
  if (smooth && !q_bf16 && !frozen) return MPFA_ERR_INVALID_ARG;  // Delta_S needs the query mean
  if (q_bf16 && (q_out->B != B || q_out->H != H_q || q_out->N != N_q || !q_out->codes || !q_out->sf))
    return MPFA_ERR_INVALID_ARG;
  if (k_bf16 && (k_out->B != B || k_out->H != H_kv || k_out->N != N_kv || !k_out->codes || !k_out->sf))
    return MPFA_ERR_INVALID_ARG;
  if (!aligned(q_bf16, 16) || !aligned(k_bf16, 16) || !aligned(delta_s_bf16, 256)) return MPFA_ERR_ALIGNMENT;
  if (q_bf16 && (!aligned(q_out->codes, 1024) || !aligned(q_out->sf, 1024))) return MPFA_ERR_ALIGNMENT;
  if (k_bf16 && (!aligned(k_out->codes, 1024) || !aligned(k_out->sf, 1024))) return MPFA_ERR_ALIGNMENT;
  StatsWorkspace w{};
  if (!frozen) {
    if (!workspace) return MPFA_ERR_INVALID_ARG;
    if (!aligned(workspace, 256)) return MPFA_ERR_ALIGNMENT;
    w = carve(workspace, workspace_bytes, B, H_q, H_kv);
    if (w.slices < 1) return MPFA_ERR_WORKSPACE;
  }
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(q_bf16);
  const __nv_bfloat16 *k = static_cast<const __nv_bfloat16 *>(k_bf16);
  if (!frozen) {
    rc = tensor_stats(StatsJob{q, N_q, H_q, w.psum_q, w.pmax_q, w.pneg_q, w.amax_q, st->q_mean, st->q_gscale},
                      StatsJob{k, N_kv, H_kv, w.psum_k, w.pmax_k, w.pneg_k, w.amax_k, st->k_mean, st->k_gscale}, B, w, smooth, s);
    if (rc != MPFA_OK) return rc;
  }
  {
    // Q and K tiles in one launch
    QuantTensor tq{q, st->q_mean, st->q_gscale, N_q, q ? H_q : 0, q ? pad128(N_q) / TILE : 0, q ? q_out->codes : nullptr,
                   q ? q_out->sf : nullptr};
    QuantTensor tk{k, st->k_mean, st->k_gscale, N_kv, k ? H_kv : 0, k ? pad128(N_kv) / TILE : 0,
                   k ? k_out->codes : nullptr, k ? k_out->sf : nullptr};
    // with smoothing the K tiles also produce Delta_S (Eq. 9) from the rows they have staged (no third pass over
    // K), in a launch of their own
    const bool with_delta = k && smooth;
    if (with_delta) {
      DeltaArgs da{st->q_mean, st->q_gscale, static_cast<__nv_bfloat16 *>(delta_s_bf16), H_q};
      MPFA_CUDA_OK(cudaFuncSetAttribute(quantize_k_delta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)KTILE_SMEM));
      quantize_k_delta_kernel<<<dim3(tk.tiles * tk.H, 1, B), 256, KTILE_SMEM, s>>>(tk, da);
      MPFA_LAUNCH_OK();
      tk.H = 0;
      tk.tiles = 0;
    }
    if (tq.H + tk.H > 0) {
      quantize_fp4_tile_kernel<<<dim3(std::max(tq.tiles, tk.tiles) * (tq.H + tk.H), 1, B), 256, 0, s>>>(tq, tk);
      MPFA_LAUNCH_OK();
    }
  }
  return MPFA_OK;
}

extern "C" mpfa_status mpfa_quantize_v(const void *v_bf16, int B, int N_kv, int H_kv, float v_scale, uint8_t *v_fp8,
                                       void *stream) {
  if (!v_bf16 || !v_fp8 || B <= 0 || N_kv <= 0 || H_kv <= 0 || !(v_scale > 0.0f)) return MPFA_ERR_INVALID_ARG;
  if (!aligned(v_bf16, 16) || !aligned(v_fp8, 1024)) return MPFA_ERR_ALIGNMENT;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  dim3 grid(pad128(N_kv) / TILE, H_kv, B);
  quantize_v_tile_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16 *>(v_bf16), N_kv, H_kv, 1.0f / v_scale, v_fp8);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

extern "C" mpfa_status mpfa_pack_v_bf16(const void *v_bf16, int B, int N_kv, int H_kv, void *v_tiles_bf16, void *stream) {
  if (!v_bf16 || !v_tiles_bf16 || B <= 0 || N_kv <= 0 || H_kv <= 0) return MPFA_ERR_INVALID_ARG;
  if (!aligned(v_bf16, 16) || !aligned(v_tiles_bf16, 1024)) return MPFA_ERR_ALIGNMENT;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  pack_v_bf16_kernel<<<dim3(pad128(N_kv) / TILE, H_kv, B), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16 *>(v_bf16), N_kv, H_kv, static_cast<__nv_bfloat16 *>(v_tiles_bf16));
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

extern "C" size_t mpfa_v_fp4_bytes(int B, int H_kv, int N_kv) {
  if (B <= 0 || H_kv <= 0 || N_kv <= 0) return 0;
  return (size_t)B * H_kv * (pad128(N_kv) / TILE) * (8192 + 1024);
}

extern "C" mpfa_status mpfa_quantize_v_fp4(const void *v_bf16, int B, int N_kv, int H_kv, float v_gscale, uint8_t *v_fp4,
                                           void *stream) {
  if (!v_bf16 || !v_fp4 || B <= 0 || N_kv <= 0 || H_kv <= 0 || !(v_gscale > 0.0f)) return MPFA_ERR_INVALID_ARG;
  if (!aligned(v_bf16, 16) || !aligned(v_fp4, 1024)) return MPFA_ERR_ALIGNMENT;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  const size_t n_tiles = (size_t)B * H_kv * (pad128(N_kv) / TILE);
  quantize_v_fp4_tile_kernel<<<dim3(pad128(N_kv) / TILE, H_kv, B), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16 *>(v_bf16), N_kv, H_kv, v_gscale, v_fp4, v_fp4 + n_tiles * 8192);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

extern "C" mpfa_status mpfa_quantize_kv_paged(const void *k_bf16, const void *v_bf16, int N_tokens, int first_token,
                                              int H_q, int H_kv, int flags, mpfa_stats *st, float v_scale,
                                              const mpfa_paged_kv *kv, const int32_t *page_table_row,
                                              void *workspace, size_t workspace_bytes, void *stream) {
  const bool smooth = flags & MPFA_SMOOTH, frozen = flags & MPFA_STATS_FROZEN;
  if (!k_bf16 || !v_bf16 || !st || !kv || !page_table_row || N_tokens <= 0 || first_token < 0 || H_q <= 0 ||
      H_kv <= 0 || !(v_scale > 0.0f))
    return MPFA_ERR_INVALID_ARG;
  if (!st->q_mean || !st->k_mean || !st->q_gscale || !st->k_gscale) return MPFA_ERR_INVALID_ARG;
  if (!kv->k_codes || !kv->k_sf || !kv->v_fp8 || kv->num_pages <= 0) return MPFA_ERR_INVALID_ARG;
  if (smooth && !kv->delta_s_bf16) return MPFA_ERR_INVALID_ARG;
  if (kv->page_size != PAGE || H_q % H_kv != 0 || H_q / H_kv > 8) return MPFA_ERR_UNSUPPORTED;
  if (kv->H_q != H_q || kv->H_kv != H_kv) return MPFA_ERR_INVALID_ARG;
  if (!frozen && first_token != 0) return MPFA_ERR_INVALID_ARG;
  if (!aligned(k_bf16, 16) || !aligned(v_bf16, 16) || !aligned(kv->k_codes, 256) || !aligned(kv->k_sf, 256) ||
      !aligned(kv->v_fp8, 256) || !aligned(kv->delta_s_bf16, 256))
    return MPFA_ERR_ALIGNMENT;
  StatsWorkspace w{};
  if (!frozen) {
    if (!workspace) return MPFA_ERR_INVALID_ARG;
    if (!aligned(workspace, 256)) return MPFA_ERR_ALIGNMENT;
    w = carve(workspace, workspace_bytes, 1, H_q, H_kv);
    if (w.slices < 1) return MPFA_ERR_WORKSPACE;
  }
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16 *k = static_cast<const __nv_bfloat16 *>(k_bf16);
  const __nv_bfloat16 *v = static_cast<const __nv_bfloat16 *>(v_bf16);
  if (!frozen) {
    rc = tensor_stats(StatsJob{k, N_tokens, H_kv, w.psum_k, w.pmax_k, w.pneg_k, w.amax_k, st->k_mean, st->k_gscale},
                      StatsJob{nullptr, 0, 0, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr}, 1, w, smooth, s);
    if (rc != MPFA_OK) return rc;
  }
  if (first_token % PAGE != 0) {
    // append into a partly filled page (frozen statistics; checked above): slot-granular kernel
    const int last_page_end = (first_token + N_tokens + PAGE - 1) / PAGE * PAGE;
    const int n_slots = last_page_end - first_token;
    append_kv_kernel<<<dim3((n_slots + 31) / 32, H_kv), 256, 0, s>>>(
        k, v, st->q_mean, st->k_mean, st->q_gscale, st->k_gscale, N_tokens, first_token, H_q, H_kv, 1.0f / v_scale,
        smooth ? 1 : 0, page_table_row, kv->num_pages, kv->k_codes, kv->k_sf, kv->v_fp8,
        static_cast<__nv_bfloat16 *>(kv->delta_s_bf16), nullptr, 0);
    MPFA_LAUNCH_OK();
    return MPFA_OK;
  }
  const int n_pages = (N_tokens + PAGE - 1) / PAGE;
  quantize_kv_page_kernel<<<dim3(n_pages, H_kv), 256, 0, s>>>(k, v, st->k_mean, st->k_gscale, N_tokens, H_kv,
                                                              1.0f / v_scale, page_table_row, first_token / PAGE,
                                                              kv->num_pages, kv->k_codes, kv->k_sf, kv->v_fp8);
  MPFA_LAUNCH_OK();
  if (smooth) {
    delta_s_kernel<true><<<dim3(pad128(N_tokens) / TILE, H_kv, 1), 256, 0, s>>>(
        k, st->q_mean, st->k_mean, st->q_gscale, st->k_gscale, N_tokens, H_q, H_kv,
        static_cast<__nv_bfloat16 *>(kv->delta_s_bf16), page_table_row + first_token / PAGE, kv->num_pages);
    MPFA_LAUNCH_OK();
  }
  return MPFA_OK;
}

// ---------------------------------------------------------------------------------------
extern "C" mpfa_status mpfa_append_kv_paged(const void *k_bf16, const void *v_bf16, int B, int H_q, int H_kv, int flags,
                                            const mpfa_stats *st, float v_scale, const mpfa_paged_kv *kv,
                                            const int32_t *page_table, int max_pages_per_req,
                                            const int32_t *positions, void *stream) {
  const bool smooth = flags & MPFA_SMOOTH;
  if (!k_bf16 || !v_bf16 || !st || !kv || !page_table || !positions || B <= 0 || H_q <= 0 || H_kv <= 0 ||
      max_pages_per_req <= 0 || !(v_scale > 0.0f))
    return MPFA_ERR_INVALID_ARG;
  if (!st->k_mean || !st->k_gscale || (smooth && (!st->q_mean || !st->q_gscale))) return MPFA_ERR_INVALID_ARG;
  if (!kv->k_codes || !kv->k_sf || !kv->v_fp8 || kv->num_pages <= 0) return MPFA_ERR_INVALID_ARG;
  if (smooth && !kv->delta_s_bf16) return MPFA_ERR_INVALID_ARG;
  if (kv->page_size != PAGE || H_q % H_kv != 0 || H_q / H_kv > 8 || B > 65535) return MPFA_ERR_UNSUPPORTED;
  if (kv->H_q != H_q || kv->H_kv != H_kv) return MPFA_ERR_INVALID_ARG;
  if (!aligned(k_bf16, 16) || !aligned(v_bf16, 16) || !aligned(kv->k_codes, 256) || !aligned(kv->k_sf, 256) ||
      !aligned(kv->v_fp8, 256) || !aligned(kv->delta_s_bf16, 256))
    return MPFA_ERR_ALIGNMENT;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  // 64 slots per request: the token's own and, when it starts a page, the 63 to be zeroed after it
  append_kv_kernel<<<dim3(2, H_kv, B), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16 *>(k_bf16), static_cast<const __nv_bfloat16 *>(v_bf16), st->q_mean, st->k_mean,
      st->q_gscale, st->k_gscale, 1, 0, H_q, H_kv, 1.0f / v_scale, smooth ? 1 : 0, page_table, kv->num_pages,
      kv->k_codes, kv->k_sf, kv->v_fp8, static_cast<__nv_bfloat16 *>(kv->delta_s_bf16), positions, max_pages_per_req);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

// mpfa_quantize_qk_static: the same stage-1 call for callers that cannot provide scratch.
// ---------------------------------------------------------------------------------------
namespace mpfa {
namespace {

// Scratch for the column sums and maxima, resident in every device that loads the library.
constexpr size_t STATIC_SCRATCH_BYTES = MPFA_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
void *g_static_scratch_addr[MAX_DEVICES] = {};
std::mutex g_static_scratch_mutex;

// In host code the array's name is only a handle; the device address has to be asked for,
// once per device, with that device current.
mpfa_status static_scratch_address(void **out) {
  int dev = 0;
  MPFA_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return MPFA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (!g_static_scratch_addr[dev]) {
    void *ptr = nullptr;
    MPFA_CUDA_OK(cudaGetSymbolAddress(&ptr, g_static_scratch));
    g_static_scratch_addr[dev] = ptr;
  }
  *out = g_static_scratch_addr[dev];
  return MPFA_OK;
}

}  // namespace
}  // namespace mpfa

extern "C" size_t mpfa_static_scratch_bytes(void) { return STATIC_SCRATCH_BYTES; }

extern "C" mpfa_status mpfa_quantize_qk_static(const void *q_bf16, const void *k_bf16, int B, int N_q, int N_kv,
                                               int H_q, int H_kv, int flags, mpfa_stats *st, mpfa_fp4_tensor *q_out,
                                               mpfa_fp4_tensor *k_out, void *delta_s_bf16, void *stream) {
  if (B <= 0 || H_q <= 0 || H_kv <= 0) return MPFA_ERR_INVALID_ARG;
  // with frozen statistics nothing is accumulated: no scratch is touched, so no size limit applies
  if (flags & MPFA_STATS_FROZEN)
    return mpfa_quantize_qk(q_bf16, k_bf16, B, N_q, N_kv, H_q, H_kv, flags, st, q_out, k_out, delta_s_bf16, nullptr, 0,
                            stream);
  if (stats_fixed_bytes(B, H_q, H_kv) + stats_slice_bytes(B, H_q, H_kv) > STATIC_SCRATCH_BYTES) return MPFA_ERR_WORKSPACE;
  void *scratch = nullptr;
  mpfa_status rc = static_scratch_address(&scratch);
  if (rc != MPFA_OK) return rc;
  return mpfa_quantize_qk(q_bf16, k_bf16, B, N_q, N_kv, H_q, H_kv, flags, st, q_out, k_out, delta_s_bf16, scratch,
                          STATIC_SCRATCH_BYTES, stream);
}
