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
//   the sum in FP64 (Eq. 7) - for BF16 inputs whose nonzero magnitudes are >= 2^-14 every partial sum
//   of up to 2^17 tokens is exactly representable, so the accumulation order cannot change the result;
//   max x and max (-x) - rounding is monotonic and symmetric, so
//   max_t |fl(x_t - mu)| = max(fl(max x - mu), fl(mu - min x)) and no second pass over the tensor is
//   needed for the per-tensor scale.
// A CTA covers 256 columns x COLSTAT_TOKENS tokens: thread = (token lane 0..7, 8 columns), a warp
// reads 512 contiguous bytes of one token row, four independent 16-byte loads in flight per thread;
// the eight token lanes are folded in shared memory, then one atomic per column and statistic.
// Maxima are stored as order-preserving unsigned keys so that a zeroed workspace is the identity.
constexpr int COLSTAT_COLS = 256;
constexpr int COLSTAT_TOKENS = 256;

__device__ __forceinline__ unsigned int ordered_key(float f) {   // monotonic float -> unsigned, key(-inf) > 0
  const unsigned int b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_key(unsigned int k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// One launch covers up to two tensors (Q and K): blockIdx.y runs over the 256-column groups of the first, then
// of the second; blocks past a tensor's last token tile leave at once.
struct ColTensor {
  const __nv_bfloat16 *x;   // null: tensor absent (ygroups = 0)
  int N, cols, ygroups;
  double *sums;
  unsigned int *kmax, *knegmax;
};

__device__ __forceinline__ void colstat_body(const __nv_bfloat16 *__restrict__ x, const int N, const int cols,
                                             double *__restrict__ sums, unsigned int *__restrict__ kmax,
                                             unsigned int *__restrict__ knegmax, const int yg) {
  __shared__ double s_sum[8][COLSTAT_COLS];
  __shared__ float s_max[8][COLSTAT_COLS], s_neg[8][COLSTAT_COLS];
  if ((int)blockIdx.x * COLSTAT_TOKENS >= N) return;
  const int b = blockIdx.z;
  const int tl = threadIdx.x >> 5, cg = threadIdx.x & 31;
  const int col = yg * COLSTAT_COLS + cg * 8;
  const int t0 = blockIdx.x * COLSTAT_TOKENS;
  const int t1 = min(N, t0 + COLSTAT_TOKENS);
  double acc[8];
  float mx[8], ng[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.0, mx[i] = -INFINITY, ng[i] = -INFINITY;
  if (col < cols) {
    const __nv_bfloat16 *p = x + ((size_t)b * N + t0 + tl) * cols + col;
    const size_t step = (size_t)8 * cols;
    int t = t0 + tl;
    for (; t + 24 < t1; t += 32, p += 4 * step) {
      uint4 u[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) u[j] = *reinterpret_cast<const uint4 *>(p + j * step);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float f[8];
        unpack8(u[j], f);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] += (double)f[i], mx[i] = fmaxf(mx[i], f[i]), ng[i] = fmaxf(ng[i], -f[i]);
      }
    }
    for (; t < t1; t += 8, p += step) {
      float f[8];
      unpack8(*reinterpret_cast<const uint4 *>(p), f);
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] += (double)f[i], mx[i] = fmaxf(mx[i], f[i]), ng[i] = fmaxf(ng[i], -f[i]);
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) s_sum[tl][cg * 8 + i] = acc[i], s_max[tl][cg * 8 + i] = mx[i], s_neg[tl][cg * 8 + i] = ng[i];
  __syncthreads();
  const int c = yg * COLSTAT_COLS + threadIdx.x;
  if (c < cols) {
    double a = 0.0;
    float m = -INFINITY, g = -INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j) a += s_sum[j][threadIdx.x], m = fmaxf(m, s_max[j][threadIdx.x]), g = fmaxf(g, s_neg[j][threadIdx.x]);
    const size_t o = (size_t)b * cols + c;
    atomicAdd(&sums[o], a);
    atomicMax(&kmax[o], ordered_key(m));
    atomicMax(&knegmax[o], ordered_key(g));
  }
}

__global__ void __launch_bounds__(256) colstat_kernel(const ColTensor a0, const ColTensor a1) {
  if ((int)blockIdx.y < a0.ygroups)
    colstat_body(a0.x, a0.N, a0.cols, a0.sums, a0.kmax, a0.knegmax, (int)blockIdx.y);
  else
    colstat_body(a1.x, a1.N, a1.cols, a1.sums, a1.kmax, a1.knegmax, (int)blockIdx.y - a0.ygroups);
}

// Per column: mean = fl(sum / N) (0 without smoothing); per batch element: max |x - mean| from the
// column extremes.  grid (ceil(cols / 256), B).
struct FinTensor {
  const double *sums;   // null: tensor absent
  const unsigned int *kmax, *knegmax;
  int cols, N;
  float *mean;
  unsigned int *amax;
  float *gscale;
};

// grid (ceil(max cols / 256), B, 2): blockIdx.z selects the tensor.
__global__ void __launch_bounds__(256) finalize_stats_kernel(const FinTensor a0, const FinTensor a1, int smooth) {
  const bool second = blockIdx.z != 0;
  const double *__restrict__ sums = second ? a1.sums : a0.sums;
  if (!sums) return;
  const unsigned int *__restrict__ kmax = second ? a1.kmax : a0.kmax;
  const unsigned int *__restrict__ knegmax = second ? a1.knegmax : a0.knegmax;
  const int cols = second ? a1.cols : a0.cols, N = second ? a1.N : a0.N;
  float *__restrict__ mean = second ? a1.mean : a0.mean;
  unsigned int *__restrict__ amax = second ? a1.amax : a0.amax;
  if ((int)blockIdx.x * 256 >= cols) return;
  const int b = blockIdx.y, c = blockIdx.x * 256 + threadIdx.x;
  float m = 0.0f;
  if (c < cols) {
    const size_t o = (size_t)b * cols + c;
    const float mu = smooth ? __double2float_rn(__ddiv_rn(sums[o], (double)N)) : 0.0f;
    mean[o] = mu;
    const float hi = from_ordered_key(kmax[o]), lo = -from_ordered_key(knegmax[o]);
    m = fmaxf(__fsub_rn(hi, mu), __fsub_rn(mu, lo));   // non-negative: lo <= mu <= hi (or mu = 0 and the larger side wins)
    m = fmaxf(m, 0.0f);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ float wmax[8];
  if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 1; i < 8; ++i) m = fmaxf(m, wmax[i]);
    atomicMax(&amax[b], __float_as_uint(m));   // non-negative floats order like their bit patterns
  }
}

__global__ void finalize_scale_kernel(const FinTensor a0, const FinTensor a1, int B) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < B) {
    if (a0.sums) {
      float a = __uint_as_float(a0.amax[i]);
      a0.gscale[i] = a > 0.0f ? __fdiv_rn(a, 2688.0f) : 1.0f;
    }
    if (a1.sums) {
      float a = __uint_as_float(a1.amax[i]);
      a1.gscale[i] = a > 0.0f ? __fdiv_rn(a, 2688.0f) : 1.0f;
    }
  }
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
                                                   uint8_t *__restrict__ sf, const int h) {
  __shared__ float mu[HEAD_DIM];
  __shared__ __align__(16) uint8_t sf_tile[1024];
  const int tile = blockIdx.x, b = blockIdx.z;
  if (tile >= tiles) return;
  const int n_pad = tiles * TILE;
  if (threadIdx.x < HEAD_DIM) mu[threadIdx.x] = mean[((size_t)b * H + h) * HEAD_DIM + threadIdx.x];
  __syncthreads();
  const float d = gscale[b];
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int id = it * 256 + threadIdx.x;
    const int r = id >> 3, g = id & 7;
    const int t = tile * TILE + r;
    uint2 c = make_uint2(0u, 0u);
    uint8_t sc = 0;
    if (t < N) {
      float xc[16];
      load_center16(x + (((size_t)b * N + t) * H + h) * HEAD_DIM + g * 16, mu + g * 16, xc);
      quantize_block16(xc, d, sc, c);
    }
    *reinterpret_cast<uint2 *>(codes + (((size_t)b * H + h) * n_pad + t) * 64 + g * 8) = c;
    sf_tile[(g >> 2) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (g & 3)] = sc;
  }
  __syncthreads();
  uint32_t *dst = reinterpret_cast<uint32_t *>(sf + (((size_t)b * H + h) * tiles + tile) * 1024);
  dst[threadIdx.x] = reinterpret_cast<const uint32_t *>(sf_tile)[threadIdx.x];
}

// grid (max tiles, H of the first + H of the second tensor, B); one 128-token tile of one head per block.
__global__ void __launch_bounds__(256) quantize_fp4_tile_kernel(const QuantTensor a0, const QuantTensor a1) {
  if ((int)blockIdx.y < a0.H)
    quantize_tile_body(a0.x, a0.mean, a0.gscale, a0.N, a0.H, a0.tiles, a0.codes, a0.sf, (int)blockIdx.y);
  else
    quantize_tile_body(a1.x, a1.mean, a1.gscale, a1.N, a1.H, a1.tiles, a1.codes, a1.sf, (int)blockIdx.y - a0.H);
}

// Eq. 9: Delta_S[hq][t] = qmean[hq] . (k[t] - kmean), FP64 accumulation with channels ascending,
// expressed in units of gscale_q * gscale_k and rounded once to BF16.  Two threads per key token
// (256 threads per 128-token tile): thread (key, part) takes the heads g = part, part + 2, ... of the
// group, each as its own sequential chain.  grid (N_pad/128, H_kv, B).  dst_stride / dst_base let the same
// kernel write the dense [B, H_q, N_pad] vector or one page of the paged side cache.
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

struct StatsWorkspace {
  double *sums_q, *sums_k;
  unsigned int *max_q, *neg_q, *max_k, *neg_k;   // per-column extremes as ordered keys
  unsigned int *amax_q, *amax_k;
  size_t bytes;
};

StatsWorkspace carve(void *ws, int B, int H_q, int H_kv) {
  StatsWorkspace w;
  size_t o = 0;
  uint8_t *base = static_cast<uint8_t *>(ws);
  w.sums_q = reinterpret_cast<double *>(base + o);
  o += align256((size_t)B * H_q * HEAD_DIM * sizeof(double));
  w.sums_k = reinterpret_cast<double *>(base + o);
  o += align256((size_t)B * H_kv * HEAD_DIM * sizeof(double));
  w.max_q = reinterpret_cast<unsigned int *>(base + o);
  o += align256((size_t)B * H_q * HEAD_DIM * sizeof(unsigned int));
  w.neg_q = reinterpret_cast<unsigned int *>(base + o);
  o += align256((size_t)B * H_q * HEAD_DIM * sizeof(unsigned int));
  w.max_k = reinterpret_cast<unsigned int *>(base + o);
  o += align256((size_t)B * H_kv * HEAD_DIM * sizeof(unsigned int));
  w.neg_k = reinterpret_cast<unsigned int *>(base + o);
  o += align256((size_t)B * H_kv * HEAD_DIM * sizeof(unsigned int));
  w.amax_q = reinterpret_cast<unsigned int *>(base + o);
  o += align256((size_t)B * sizeof(unsigned int));
  w.amax_k = reinterpret_cast<unsigned int *>(base + o);
  o += align256((size_t)B * sizeof(unsigned int));
  w.bytes = o;
  return w;
}

// One tensor [B, N, H, 128] of a statistics pass (x == nullptr: absent).
struct StatsJob {
  const __nv_bfloat16 *x;
  int N, H;
  double *sums;
  unsigned int *kmax, *knegmax, *amax;
  float *mean, *gscale;
};

// Means and per-tensor scales of up to two tensors: one pass over the data, three launches in all.
mpfa_status tensor_stats(const StatsJob &j0, const StatsJob &j1, int B, bool smooth, cudaStream_t st) {
  ColTensor c[2];
  FinTensor f[2];
  int tiles = 0, colgroups = 0;
  const StatsJob *jobs[2] = {&j0, &j1};
  for (int i = 0; i < 2; ++i) {
    const StatsJob &j = *jobs[i];
    const int cols = j.H * HEAD_DIM;
    c[i] = ColTensor{j.x, j.x ? j.N : 0, cols, j.x ? (cols + COLSTAT_COLS - 1) / COLSTAT_COLS : 0, j.sums, j.kmax, j.knegmax};
    f[i] = FinTensor{j.x ? j.sums : nullptr, j.kmax, j.knegmax, cols, j.N, j.mean, j.amax, j.gscale};
    if (j.x) {
      tiles = std::max(tiles, (j.N + COLSTAT_TOKENS - 1) / COLSTAT_TOKENS);
      colgroups = std::max(colgroups, (cols + 255) / 256);
    }
  }
  if (c[0].ygroups + c[1].ygroups == 0) return MPFA_OK;
  colstat_kernel<<<dim3(tiles, c[0].ygroups + c[1].ygroups, B), 256, 0, st>>>(c[0], c[1]);
  MPFA_LAUNCH_OK();
  finalize_stats_kernel<<<dim3(colgroups, B, 2), 256, 0, st>>>(f[0], f[1], smooth ? 1 : 0);
  MPFA_LAUNCH_OK();
  finalize_scale_kernel<<<(B + 127) / 128, 128, 0, st>>>(f[0], f[1], B);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}

}  // namespace
}  // namespace mpfa

using namespace mpfa;

extern "C" size_t mpfa_quantize_workspace_bytes(int B, int H_q, int H_kv) {
  if (B <= 0 || H_q <= 0 || H_kv <= 0) return 0;
  return carve(nullptr, B, H_q, H_kv).bytes;
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
    w = carve(workspace, B, H_q, H_kv);
    if (workspace_bytes < w.bytes) return MPFA_ERR_WORKSPACE;
  }
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(q_bf16);
  const __nv_bfloat16 *k = static_cast<const __nv_bfloat16 *>(k_bf16);
  if (!frozen) {
    MPFA_CUDA_OK(cudaMemsetAsync(workspace, 0, w.bytes, s));
    rc = tensor_stats(StatsJob{q, N_q, H_q, w.sums_q, w.max_q, w.neg_q, w.amax_q, st->q_mean, st->q_gscale},
                      StatsJob{k, N_kv, H_kv, w.sums_k, w.max_k, w.neg_k, w.amax_k, st->k_mean, st->k_gscale}, B, smooth, s);
    if (rc != MPFA_OK) return rc;
  }
  {
    // Q and K tiles in one launch
    QuantTensor tq{q, st->q_mean, st->q_gscale, N_q, q ? H_q : 0, q ? pad128(N_q) / TILE : 0, q ? q_out->codes : nullptr,
                   q ? q_out->sf : nullptr};
    QuantTensor tk{k, st->k_mean, st->k_gscale, N_kv, k ? H_kv : 0, k ? pad128(N_kv) / TILE : 0,
                   k ? k_out->codes : nullptr, k ? k_out->sf : nullptr};
    quantize_fp4_tile_kernel<<<dim3(std::max(tq.tiles, tk.tiles), tq.H + tk.H, B), 256, 0, s>>>(tq, tk);
    MPFA_LAUNCH_OK();
  }
  if (k) {
    dim3 grid(pad128(N_kv) / TILE, H_kv, B);
    if (smooth) {
      delta_s_kernel<false><<<grid, 256, 0, s>>>(k, st->q_mean, st->k_mean, st->q_gscale, st->k_gscale, N_kv, H_q,
                                                 H_kv, static_cast<__nv_bfloat16 *>(delta_s_bf16), nullptr, 0);
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
    w = carve(workspace, 1, H_q, H_kv);
    if (workspace_bytes < w.bytes) return MPFA_ERR_WORKSPACE;
  }
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16 *k = static_cast<const __nv_bfloat16 *>(k_bf16);
  const __nv_bfloat16 *v = static_cast<const __nv_bfloat16 *>(v_bf16);
  if (!frozen) {
    MPFA_CUDA_OK(cudaMemsetAsync(workspace, 0, w.bytes, s));
    rc = tensor_stats(StatsJob{k, N_tokens, H_kv, w.sums_k, w.max_k, w.neg_k, w.amax_k, st->k_mean, st->k_gscale},
                      StatsJob{nullptr, 0, 0, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr}, 1, smooth, s);
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
  if (carve(nullptr, B, H_q, H_kv).bytes > STATIC_SCRATCH_BYTES) return MPFA_ERR_WORKSPACE;
  void *scratch = nullptr;
  mpfa_status rc = static_scratch_address(&scratch);
  if (rc != MPFA_OK) return rc;
  return mpfa_quantize_qk(q_bf16, k_bf16, B, N_q, N_kv, H_q, H_kv, flags, st, q_out, k_out, delta_s_bf16, scratch,
                          STATIC_SCRATCH_BYTES, stream);
}
