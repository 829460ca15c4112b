// QK4PV8 decode over a paged low-bit KV cache (Section 5.3) for sm_100a.
//
// The path is bound by streaming the cache from HBM (208 bytes per token and kv head), so the
// kernel is organised around 16-byte coalesced loads that land directly in tensor-core
// register fragments; the cache's physical byte order (include/mpfa.h) is that fragment order.
//
// Grid: (1024-token partition, kv head, request).  Warp w of a CTA owns KV block w (128 keys,
// two 64-token pages) of the partition:
//   S[head, key]  = Delta_S + sum over 16-channel blocks of (Q codes x scale) . (K codes x scale)
//                   with mma.sync m16n8k16 (FP16 operands hold code x E4M3 scale exactly, FP32
//                   accumulate); the GQA group's heads are the M rows (Section 5.3: the group is
//                   packed into the MMA's M dimension);
//   block maxima are exchanged through shared memory, giving every block the running maximum
//   m_w it would see in the reverse traversal (max over blocks >= w), so P = 2^(lam S - lam m_w)
//   and P_hat = E4M3(448 P) are the same values the sequential loop produces;
//   O_w = P_hat V with mma.sync m16n8k32 (E4M3 x E4M3, FP32 accumulate), the accumulator
//   fragment of S being reused as the A fragment without leaving registers.
// The partition state (m, l, O) = (max m_w, sum 2^(lam (m_w - m)) l_w, sum 2^(...) O_w) goes to
// the workspace; a second kernel merges partitions by log-sum-exp (warp-shuffle maximum,
// partitions ascending) and writes BF16.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp4.h>
#include <cuda_fp8.h>

#include "common.cuh"

namespace mpfa {
namespace {

constexpr int PART_FLOATS = 130;  // m, l, O[128] per (request, q head, partition)
constexpr int MAXG = 8;

__device__ __forceinline__ uint4 ldg_stream16(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 ldg_stream8(const void *p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ldg_stream4(const void *p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// two E2M1 codes (one byte) -> two FP16 values
__device__ __forceinline__ __half2 fp4x2_to_half2(uint32_t byte) {
  __half2_raw r = __nv_cvt_fp4x2_to_halfraw2((__nv_fp4x2_storage_t)(byte & 0xFFu), __NV_E2M1);
  return __half2(r);
}
// one unsigned E4M3 scale byte -> the same FP16 value in both halves
__device__ __forceinline__ __half2 e4m3_to_half2_bcast(uint32_t byte) {
  const uint32_t b = byte & 0xFFu;
  __half2_raw r = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(b | (b << 8)), __NV_E4M3);
  return __half2(r);
}
__device__ __forceinline__ uint32_t h2_bits(__half2 h) { return *reinterpret_cast<uint32_t *>(&h); }

__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_e4m3_16832(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

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

__global__ void __launch_bounds__(256, 2) decode_split_kernel(const DecodeParams p) {
  __shared__ float s_bmax[8][MAXG];
  __shared__ float s_l[8][MAXG];
  __shared__ __align__(16) float s_o[8][MAXG][HEAD_DIM];  // 32 KB

  const int sp = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int L = p.seq_lens[b];
  const int k_part = sp * DECODE_SPLIT;
  if (k_part >= L) return;   // whole CTA; the merge kernel only reads partitions below ceil(L / 1024)
  const int G = p.H_q / p.H_kv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, tq = lane & 3;
  const int hq = hk * G + (g < G ? g : 0);
  const bool head_ok = g < G;
  const int n_blocks = (min(DECODE_SPLIT, L - k_part) + TILE - 1) / TILE;
  const int key0 = k_part + warp * TILE;   // first key of this warp's block
  const bool active = warp < n_blocks;
  const float lam = __fmul_rn(__fmul_rn(__fmul_rn(p.softmax_scale, 1.4426950408889634f), p.q_gscale[b]), p.k_gscale[b]);

  float S[16][2];
  float bmax = -INFINITY;
  int phys[2] = {-1, -1};
  if (active) {
    // ---- query fragments: head g of the group, codes x scale in FP16 (exact)
    uint32_t qa[8][2];
    {
      const uint8_t *qc = p.q_codes + ((size_t)b * p.H_q + hq) * (TILE * 64);
      const uint8_t *qs = p.q_sf + ((size_t)b * p.H_q + hq) * 1024;
#pragma unroll
      for (int kb = 0; kb < 8; ++kb) {
        const uint32_t two = *reinterpret_cast<const uint16_t *>(qc + kb * 8 + 2 * tq);
        const __half2 sc = e4m3_to_half2_bcast(qs[(kb >> 2) * 512 + (kb & 3)]);
        qa[kb][0] = head_ok ? h2_bits(__hmul2(fp4x2_to_half2(two), sc)) : 0u;
        qa[kb][1] = head_ok ? h2_bits(__hmul2(fp4x2_to_half2(two >> 8), sc)) : 0u;
      }
    }
    // ---- pages of this block
#pragma unroll
    for (int pg = 0; pg < 2; ++pg) {
      const int first = key0 + pg * PAGE;
      if (first < L) {
        const int id = p.page_table[(size_t)b * p.max_pages + first / PAGE];
        if (id >= 0 && id < p.num_pages) {
          phys[pg] = id;
        } else if (lane == 0) {
          atomicOr(p.status, MPFA_DEV_BAD_PAGE);
        }
      }
    }
    // ---- S = Delta_S + Q K^T  (Eq. 10), 8 keys per n-tile
#pragma unroll
    for (int pg = 0; pg < 2; ++pg) {
      if (phys[pg] >= 0) {
        const size_t slab = (size_t)phys[pg] * p.H_kv + hk;
        const uint8_t *kc = p.k_codes + slab * 4096 + lane * 16;
        const uint8_t *ks = p.k_sf + slab * 512 + g * 8;
        uint4 kw[8];
        uint2 sw[8];
        uint32_t dw[8];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          kw[nt] = ldg_stream16(kc + nt * 512);
          sw[nt] = ldg_stream8(ks + nt * 64);
          dw[nt] = (p.delta && head_ok)
                       ? ldg_stream4(p.delta + ((size_t)phys[pg] * p.H_q + hq) * PAGE + nt * 8 + 2 * tq)
                       : 0u;
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          float c[4] = {__uint_as_float(dw[nt] << 16), __uint_as_float(dw[nt] & 0xFFFF0000u), 0.0f, 0.0f};
          const uint32_t cw[4] = {kw[nt].x, kw[nt].y, kw[nt].z, kw[nt].w};
          const uint32_t scw[2] = {sw[nt].x, sw[nt].y};
#pragma unroll
          for (int kb = 0; kb < 8; ++kb) {
            const uint32_t two = cw[kb >> 1] >> (16 * (kb & 1));
            const __half2 sc = e4m3_to_half2_bcast(scw[kb >> 2] >> (8 * (kb & 3)));
            const uint32_t b0 = h2_bits(__hmul2(fp4x2_to_half2(two), sc));
            const uint32_t b1 = h2_bits(__hmul2(fp4x2_to_half2(two >> 8), sc));
            mma_f16_16816(c, qa[kb][0], 0u, qa[kb][1], 0u, b0, b1);
          }
          const int kabs = key0 + pg * PAGE + nt * 8 + 2 * tq;
          S[pg * 8 + nt][0] = (kabs < L) ? c[0] : -INFINITY;
          S[pg * 8 + nt][1] = (kabs + 1 < L) ? c[1] : -INFINITY;
        }
      } else {
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) S[pg * 8 + nt][0] = S[pg * 8 + nt][1] = -INFINITY;
      }
    }
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) bmax = fmaxf(bmax, fmaxf(S[nt][0], S[nt][1]));
    bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 1));
    bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 2));
  }
  if (tq == 0) s_bmax[warp][g] = active ? bmax : -INFINITY;
  __syncthreads();
  // running maximum of the reverse traversal: blocks >= w have been visited when block w is
  float m_w = -INFINITY, m_all = -INFINITY;
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const float v = s_bmax[u][g];
    m_all = fmaxf(m_all, v);
    if (u >= warp) m_w = fmaxf(m_w, v);
  }

  float O[16][2];
#pragma unroll
  for (int nt = 0; nt < 16; ++nt) O[nt][0] = O[nt][1] = 0.0f;
  float lsum = 0.0f;
  if (active) {
    // ---- P = 2^(lam S - lam m_w), l from the unquantized P, P_hat = E4M3(448 P)
    const float neg_mlam = (m_w == -INFINITY) ? 0.0f : -__fmul_rn(m_w, lam);
    uint32_t pa[4][2];   // A fragments of the four 32-key steps
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int nt = k4 * 4 + h * 2;
        const float p0 = ex2_approx(__fmaf_rn(S[nt][0], lam, neg_mlam));
        const float p1 = ex2_approx(__fmaf_rn(S[nt][1], lam, neg_mlam));
        const float p2 = ex2_approx(__fmaf_rn(S[nt + 1][0], lam, neg_mlam));
        const float p3 = ex2_approx(__fmaf_rn(S[nt + 1][1], lam, neg_mlam));
        lsum += (p0 + p1) + (p2 + p3);
        const uint32_t lo = (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(p0, 448.0f), __fmul_rn(p1, 448.0f)),
                                                               __NV_SATFINITE, __NV_E4M3);
        const uint32_t hi = (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(p2, 448.0f), __fmul_rn(p3, 448.0f)),
                                                               __NV_SATFINITE, __NV_E4M3);
        pa[k4][h] = head_ok ? ((lo & 0xFFFFu) | (hi << 16)) : 0u;
      }
    }
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
    // ---- O_w = P_hat V, 32 keys per step, two 8-channel n-tiles per 16-byte load
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {
      const int pg = k4 >> 1;
      if (phys[pg] >= 0) {
        const uint8_t *vp = p.v_fp8 + ((size_t)phys[pg] * p.H_kv + hk) * 8192 + (k4 & 1) * 4096 + lane * 16;
        uint4 vw[8];
#pragma unroll
        for (int np = 0; np < 8; ++np) vw[np] = ldg_stream16(vp + np * 512);
#pragma unroll
        for (int np = 0; np < 8; ++np) {
          float c0[4] = {O[2 * np][0], O[2 * np][1], 0.0f, 0.0f};
          mma_e4m3_16832(c0, pa[k4][0], 0u, pa[k4][1], 0u, vw[np].x, vw[np].y);
          O[2 * np][0] = c0[0];
          O[2 * np][1] = c0[1];
          float c1[4] = {O[2 * np + 1][0], O[2 * np + 1][1], 0.0f, 0.0f};
          mma_e4m3_16832(c1, pa[k4][0], 0u, pa[k4][1], 0u, vw[np].z, vw[np].w);
          O[2 * np + 1][0] = c1[0];
          O[2 * np + 1][1] = c1[1];
        }
      }
    }
  }
  // ---- fold the blocks of this partition: weights 2^(lam (m_w - m_all))
  const float wgt = (active && m_w != -INFINITY) ? ex2_approx(__fmul_rn(m_w - m_all, lam)) : 0.0f;
  if (head_ok) {
    if (tq == 0) s_l[warp][g] = wgt * lsum;
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
      *reinterpret_cast<float2 *>(&s_o[warp][g][nt * 8 + 2 * tq]) = make_float2(wgt * O[nt][0], wgt * O[nt][1]);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < G * HEAD_DIM; i += 256) {
    const int hh = i >> 7, c = i & 127;
    float acc = 0.0f;
    for (int u = n_blocks - 1; u >= 0; --u) acc += s_o[u][hh][c];   // same order as the traversal
    p.parts[(((size_t)b * p.H_q + hk * G + hh) * p.n_split + sp) * PART_FLOATS + 2 + c] = acc;
  }
  if (threadIdx.x < G) {
    const int hh = threadIdx.x;
    float acc = 0.0f, mm = -INFINITY;
    for (int u = n_blocks - 1; u >= 0; --u) {
      acc += s_l[u][hh];
      mm = fmaxf(mm, s_bmax[u][hh]);
    }
    float *dst = p.parts + (((size_t)b * p.H_q + hk * G + hh) * p.n_split + sp) * PART_FLOATS;
    dst[0] = mm;
    dst[1] = acc;
  }
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
  if (n_split > 65535 || B > 65535) return MPFA_ERR_UNSUPPORTED;
  if (!aligned(q->codes, 16) || !aligned(q->sf, 16) || !aligned(kv->k_codes, 256) || !aligned(kv->k_sf, 256) ||
      !aligned(kv->v_fp8, 256) || !aligned(kv->delta_s_bf16, 256) || !aligned(workspace, 16))
    return MPFA_ERR_ALIGNMENT;
  mpfa_status rc = check_arch();
  if (rc != MPFA_OK) return rc;
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
  decode_split_kernel<<<dim3((unsigned)n_split, H_kv, B), 256, 0, s>>>(p);
  MPFA_LAUNCH_OK();
  decode_merge_kernel<<<dim3(H_q, B), 128, 0, s>>>(p.parts, seq_lens, st->q_gscale, st->k_gscale, H_q, (int)n_split,
                                                   softmax_scale, v_scale, static_cast<__nv_bfloat16 *>(out_bf16),
                                                   out_f32);
  MPFA_LAUNCH_OK();
  return MPFA_OK;
}
