// Pieces shared by the prefill kernels: launch parameters, the bounded barrier wait, packed FP32 helpers, the
// page look-up of the paged source and the tensor-map encoder.  Included by prefill.cu and prefill_pair.cu only.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace mpfa {

struct PrefillParams {
  const uint8_t *q_sf;
  const uint8_t *k_sf;
  const uint8_t *v_sf = nullptr;   // NVFP4 + NVFP4 variant only: block scales of the FP4 V operand
  const __nv_bfloat16 *delta;  // may be null
  const float *q_gscale;
  const float *k_gscale;
  __nv_bfloat16 *out;
  float *out_f32;  // may be null
  int32_t *status;
  int B, N_q, N_kv, H_q, H_kv, nq_tiles, nk_tiles, n_items;
  int causal;
  float softmax_scale, v_scale;
};

// K, V and Delta_S read from the paged cache instead of contiguous tensors: 64-token pages whose
// (page, kv head) slabs are stored as halves of this kernel's operand tiles (same swizzles), K scales
// row-major [token][8] and Delta_S [page][q head][64] with its 16-byte groups XOR-ed by (q head mod G).
struct PagedSrc {
  const uint8_t *k_codes, *k_sf, *v_fp8;
  const __nv_bfloat16 *delta;   // may be null
  const int32_t *page_table;    // [B, max_pages]
  const int32_t *seq_lens;      // [B] keys of each request (the last q_lens[b] of them are the queries' own)
  const int32_t *q_lens;        // [B] queries of each request, <= N_q; null: N_q for all
  int max_pages, num_pages;
};

// two query tiles per CTA (prefill_pair.cu)
mpfa_status launch_prefill_pair(const mpfa_fp4_tensor *q, const mpfa_fp4_tensor *k, const uint8_t *v_fp8,
                                const PrefillParams &p, bool elementwise, cudaStream_t stream);
mpfa_status launch_prefill_pair_paged(const mpfa_fp4_tensor *q, const PrefillParams &p, const PagedSrc &pg,
                                      cudaStream_t stream);

namespace {

#ifndef MPFA_WAIT_LIMIT_CYCLES
#define MPFA_WAIT_LIMIT_CYCLES 4000000000ll   // about 2 s of SM clock: far beyond any legitimate wait
#endif
constexpr long long WAIT_LIMIT_CYCLES = MPFA_WAIT_LIMIT_CYCLES;
#ifndef MPFA_DRAIN_LIMIT_NS
#define MPFA_DRAIN_LIMIT_NS 2000000000ull
#endif
constexpr uint64_t WAIT_LIMIT_NS = MPFA_DRAIN_LIMIT_NS;   // drain path only
// Test builds only (-DMPFA_TEST_DROP_V_COPY, together with short limits): the producer of CTA 0 leaves out the
// first V copy of the launch, so the P V issuer's wait for it runs out and the whole give-up path executes -
// status bit, every role leaving its loops, copies in flight drained, tensor memory released.  Never defined in
// the product library.
#ifdef MPFA_TEST_DROP_V_COPY
#define MPFA_DROP_V(c) ((c) == 0u && blockIdx.x == 0)
#else
#define MPFA_DROP_V(c) false
#endif

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Packed FP32 pairs (one issue slot for two IEEE operations; each half rounds like the scalar form).
__device__ __forceinline__ void fma2(float &d0, float &d1, float a0, float a1, float b, float c) {
  asm("{.reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %5};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;}"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ void mul2(float &d0, float &d1, float a0, float a1, float b) {
  asm("{.reg .b64 ra, rb, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\t"
      "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;}"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b));
}
__device__ __forceinline__ void acc2(float &d0, float &d1, float a0, float a1) {
  asm("{.reg .b64 ra, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rd, {%0, %1};\n\t"
      "add.rn.f32x2 rd, rd, ra;\n\tmov.b64 {%0, %1}, rd;}"
      : "+f"(d0), "+f"(d1)
      : "f"(a0), "f"(a1));
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}

// One arrival per warp: every lane's earlier shared-memory writes and tensor-memory accesses are
// ordered before it by the warp-level barrier.
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}

struct Ctx {
  uint32_t bars;      // shared address of barrier 0
  volatile int *abort_flag;
  int32_t *status;
  __device__ __forceinline__ uint32_t bar(int i) const { return bars + 8u * (uint32_t)i; }
  __device__ __forceinline__ bool probe(int i, uint32_t parity) const { return mbar_try_wait(bar(i), parity); }
  // Bounded wait.  try_wait may itself suspend the thread for a system-dependent interval, so
  // the bound is on elapsed SM clock cycles (about 2 s), checked once per 32 polls to keep the
  // hand-off latency at the cost of a poll.  Also gives up as soon as another role has failed.
  __device__ __forceinline__ bool wait(int i, uint32_t parity) const {
    const uint32_t a = bar(i);
    if (mbar_try_wait(a, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
      for (int k = 0; k < 32; ++k) {
        if (mbar_try_wait_hint(a, parity, 1000u)) return true;   // the hardware may park the thread meanwhile
      }
      if (*abort_flag) return false;
      if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
    }
    *abort_flag = 1;
    atomicOr(status, MPFA_DEV_TIMEOUT);
    return false;
  }
};

// Paged source: the two physical pages of KV block jb (t-th block of the traversal) of an item.  Every 16 blocks
// the warp reads 32 page ids with one coalesced load (lane l: page index 2 jb + 1 - l); in between the ids come
// from the lanes' registers.  A page past the end of the context (all its keys are masked) or with an id outside
// the pool (reported in *status) is replaced by the block's other page, so operand tiles always hold finite bytes.
struct PageLookup {
  int ids;
  __device__ __forceinline__ void get(const PagedSrc &pg, int32_t *status, int b, int nkv, int t, int jb, int lane,
                                      int &page_lo, int &page_hi) {
    if ((t & 15) == 0) {
      const int n_pg = (nkv + 63) >> 6;
      const int pi = 2 * jb + 1 - lane;
      int id = -1;
      if (pi >= 0 && pi < n_pg) {
        id = pg.page_table[(size_t)b * pg.max_pages + pi];
        if (id < 0 || id >= pg.num_pages) {
          atomicOr(status, MPFA_DEV_BAD_PAGE);
          id = -1;
        }
      }
      ids = id;
    }
    page_hi = __shfl_sync(0xffffffffu, ids, (t & 15) * 2);
    page_lo = __shfl_sync(0xffffffffu, ids, (t & 15) * 2 + 1);
    if (page_hi < 0) page_hi = page_lo;
    if (page_lo < 0) page_lo = page_hi < 0 ? 0 : page_hi;
    if (page_hi < 0) page_hi = 0;
  }
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up through the runtime so the library does not link libcuda.
mpfa_status get_encoder(EncodeTiledFn *fn) {
  static EncodeTiledFn cached = nullptr;
  if (!cached) {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    MPFA_CUDA_OK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q));
    if (q != cudaDriverEntryPointSuccess || !ptr) return cuda_fail(cudaErrorNotSupported);
    cached = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  *fn = cached;
  return MPFA_OK;
}

// 2D byte tensor [rows][row_bytes], box = 128 rows x box_bytes (default: the whole row), hardware swizzle = box_bytes.
inline mpfa_status make_map(EncodeTiledFn enc, CUtensorMap *m, const void *base, uint64_t rows, uint32_t row_bytes,
                            uint32_t box_bytes = 0) {
  if (box_bytes == 0) box_bytes = row_bytes;
  cuuint64_t dims[2] = {row_bytes, rows};
  cuuint64_t strides[1] = {row_bytes};
  cuuint32_t box[2] = {box_bytes, 128};
  cuuint32_t es[2] = {1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, es,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, box_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda_error = (int)r;
    return MPFA_ERR_CUDA;
  }
  return MPFA_OK;
}

}  // namespace
}  // namespace mpfa
