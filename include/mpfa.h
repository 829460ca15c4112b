/*
 * mpfa.h - C ABI of the QK4PV8 mixed-precision attention library for NVIDIA B200 (sm_100a).
 *
 * The library implements the two stages of the paper's Algorithm 1:
 *   stage 1 (lines 1-5, Sections 4.2-4.3): sequence centering of Q and K, NVFP4
 *     quantization of the centered tensors (E2M1 values, one E4M3 scale per 16
 *     head-dimension elements, Eq. 1), FP8 E4M3 quantization of V, and the
 *     compensation vector Delta_S (Eq. 9);
 *   stage 2 (lines 6-20, Sections 4.1, 5.1-5.3): the attention main loop that consumes
 *     only those quantized tensors - a rank-one BF16 MMA seeding the score accumulator
 *     with Delta_S (Eq. 11), the block-scaled FP4 MMA, online softmax (Eq. 3-6) with P
 *     quantized to E4M3 at the fixed scale 448, the FP8 PV MMA - for causal GQA
 *     prefill and for split-KV decode over a paged KV cache.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name starts with h_.  The caller owns
 *     all buffers.  No call allocates, frees or synchronises: work is only enqueued on
 *     `stream`.
 *   - head_dim is 128.  H_q must be a multiple of H_kv (GQA); q head hq uses kv head
 *     hq / (H_q / H_kv).
 *   - Inputs Q, K, V are BF16, token-major: [B, N, H, 128].  Outputs are BF16
 *     [B, N_q, H_q, 128] (prefill) or [B, H_q, 128] (decode).
 *   - Every function returns an mpfa_status (0 = success, negative = error).  Argument,
 *     shape and alignment errors are detected on the host before anything is launched.
 *     Errors found on the device (a bounded wait that gave up, a page index out of range)
 *     are OR-ed into *device_status, which the caller reads after synchronising.
 *   - Results are deterministic: the same call (shapes, workspace size) on the same inputs gives bit-identical
 *     outputs; no floating-point atomics are used anywhere.
 *
 * Physical layouts (all offsets in bytes, N_pad = N rounded up to a multiple of 128)
 *   NVFP4 tensor ("tile layout", mpfa_fp4_tensor):
 *     codes  [B, H, N_pad, 64]   two E2M1 codes per byte, even channel in bits 3:0;
 *                                rows N..N_pad-1 are zero.
 *     sf     [B, H, N_pad/128, 2, 512]   unsigned E4M3 block scales.  Token t, 16-channel
 *                                block g (0..7) lives in tile t/128, half g/4, at byte
 *                                (r%32)*16 + (r/32)*4 + (g%4) with r = t%128 - the
 *                                32-lane x 16-byte image the tensor core's scale-factor
 *                                copy expects.  mpfa_sf_offset() is this map.
 *   Delta_S  BF16 [B, H_q, N_kv_pad], in units of (true logit) / (q_gscale * k_gscale).
 *   V        E4M3 [B, H_kv, N_kv_pad, 128], pad rows zero.
 *   Paged KV cache (mpfa_paged_kv): 64-token pages; within a page and kv head the bytes are
 *     ordered as the decode kernel's shared-memory operand tiles, see mpfa_paged_kv below.
 */
#ifndef MPFA_H_
#define MPFA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int mpfa_status;
enum {
  MPFA_OK = 0,
  MPFA_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, inconsistent struct fields */
  MPFA_ERR_UNSUPPORTED = -2, /* H_q % H_kv != 0, page_size != 64, GQA group > 8 (decode), ... */
  MPFA_ERR_ALIGNMENT = -3,   /* a buffer is not aligned as documented */
  MPFA_ERR_WORKSPACE = -4,   /* workspace_bytes smaller than the matching *_workspace_bytes() */
  MPFA_ERR_ARCH = -5,        /* the current device is not compute capability 10.x */
  MPFA_ERR_CUDA = -6,        /* a CUDA call failed; see mpfa_last_cuda_error() */
  MPFA_ERR_TIMEOUT = -7      /* reserved for device_status: a bounded device wait gave up */
};

/* bits OR-ed into *device_status by the kernels */
enum {
  MPFA_DEV_TIMEOUT = 1,  /* a bounded mbarrier wait expired; the output is invalid */
  MPFA_DEV_BAD_PAGE = 2  /* a page-table entry was outside [0, num_pages); that page was skipped */
};

/* flags of mpfa_quantize_qk / mpfa_quantize_kv_paged */
enum {
  MPFA_SMOOTH = 1,       /* center with the sequence means and emit Delta_S (Section 4.2-4.3).
                            Without it: the paper's "direct" variant, means = 0, no Delta_S. */
  MPFA_STATS_FROZEN = 2  /* read means and tensor scales from `stats` instead of computing them
                            (decode-time tokens are centered against the frozen prefill
                            statistics, Section 6). */
};

/* Per-request statistics, caller-owned.  Written by the quantizers unless
 * MPFA_STATS_FROZEN, read by them when it is set, and read by the attention calls
 * (tensor scales only). */
typedef struct {
  float *q_mean;   /* [B, H_q, 128]  Eq. 7 */
  float *k_mean;   /* [B, H_kv, 128] Eq. 7 */
  float *q_gscale; /* [B] per-tensor scale d_Q = max|Q - mean| / 2688 (1.0 if the tensor is all zero) */
  float *k_gscale; /* [B] d_K */
} mpfa_stats;

/* One NVFP4 tensor in the tile layout described at the top. codes and sf must be
 * 1024-byte aligned.  Sizes: mpfa_fp4_codes_bytes / mpfa_fp4_sf_bytes. */
typedef struct {
  uint8_t *codes;
  uint8_t *sf;
  int32_t B, H, N;
} mpfa_fp4_tensor;

/* Paged KV cache for decode: num_pages physical pages of 64 tokens, shared by all
 * requests through a page table.  Inside a (page, kv head) slab the bytes are ordered as the
 * decode kernel's shared-memory operand tiles (rows of 8 tokens, 16-byte chunks XOR-swizzled
 * by the row), so that one bulk copy per slab fills a tile.  With token t (0..63) of the page:
 *   k_codes [P, H_kv, 4096]  byte j (0..7) of 16-channel block g (0..7) of token t at
 *             (t/8)*512 + (t%8)*64 + ((g/2) ^ ((t%8)/2))*16 + (g%2)*8 + j
 *   k_sf    [P, H_kv, 512]   block g of token t at t*8 + g
 *   v_fp8   [P, H_kv, 8192]  channel c (0..127) of token t at
 *             (t/8)*1024 + (t%8)*128 + ((c/16) ^ (t%8))*16 + c%16
 *   delta_s [P, H_q, 64]     BF16, token t of q head h at index ((t/8) ^ (h % (H_q/H_kv)))*8 + t%8
 *                            (NULL when compensation is off)
 * Tokens of a page beyond the sequence length hold zeros (mpfa_quantize_kv_paged writes them).
 * mpfa_paged_k_offset / mpfa_paged_v_offset are these maps.  All pools 256-byte aligned. */
typedef struct {
  uint8_t *k_codes;
  uint8_t *k_sf;
  uint8_t *v_fp8;
  void *delta_s_bf16;
  int32_t num_pages;
  int32_t page_size; /* must be 64 */
  int32_t H_q, H_kv; /* head counts the pools were sized for */
} mpfa_paged_kv;

/* ---- stage 1: Algorithm 1 lines 1-5 -------------------------------------------------- */

/* Means (Eq. 7), centering, per-tensor scales, NVFP4 quantization (Eq. 1) of Q and K,
 * and Delta_S (Eq. 9; needs both tensors' statistics, written when k_bf16 != NULL).
 *   q_bf16 [B, N_q, H_q, 128] or NULL (quantize K only; needs MPFA_STATS_FROZEN for the Q side
 *          if MPFA_SMOOTH, because Delta_S uses the query mean);
 *   k_bf16 [B, N_kv, H_kv, 128] or NULL (quantize Q only);
 *   q_out / k_out: tile-layout tensors with B, H, N filled in by the caller;
 *   delta_s_bf16 [B, H_q, N_kv_pad]: required iff MPFA_SMOOTH and k_bf16 != NULL;
 *   workspace: 256-byte aligned scratch, overwritten by every call (not needed with MPFA_STATS_FROZEN).  The call
 *          enqueues one memory-set node over its first few hundred bytes (maxima and block counters) and four
 *          kernels; two calls that overlap on the GPU need separate workspaces.
 *          mpfa_quantize_workspace_bytes() is the size that lets the statistics pass cut the token axis into
 *          its full 32 slices; any size down to mpfa_quantize_workspace_min_bytes() (one slice) is accepted and
 *          only lowers the parallelism of that pass; less: MPFA_ERR_WORKSPACE.
 * All arithmetic is specified step by step (FP64 column sums, one rounding to FP32, IEEE divisions).  The column
 * sums are added in a fixed order (tokens ascending within a thread, then token lanes, then slices; the order is a
 * function of the shapes, the workspace size and the device's SM count), so the outputs are reproducible bit for
 * bit for any input.  They
 * equal the single ascending FP64 sum of Eq. 7 - and every code and scale derived from it - bit for bit whenever
 * each partial sum is exactly representable in FP64, which holds for BF16 inputs whose nonzero magnitudes in a
 * column span fewer than about 40 binades over up to 2^17 tokens; outside that range the mean may differ from the
 * sequential sum in its last FP32 bit. */
mpfa_status mpfa_quantize_qk(const void *q_bf16, const void *k_bf16, int B, int N_q, int N_kv, int H_q,
                             int H_kv, int flags, mpfa_stats *h_stats, mpfa_fp4_tensor *h_q_out,
                             mpfa_fp4_tensor *h_k_out, void *delta_s_bf16, void *workspace,
                             size_t workspace_bytes, void *stream);

/* (No counterpart in the paper: a convenience for embedders.)
 * mpfa_quantize_qk for callers that cannot hand the library any scratch memory - code
 * that runs where device allocation is forbidden or unavailable: inside a serving loop
 * whose memory pool is fully pre-assigned, in a plugin that is given only its input and
 * output tensors, or after the process has dropped the right to call the allocator.
 * Arguments and results are exactly those of mpfa_quantize_qk without the workspace pair.
 * The column sums and maxima live in a fixed MPFA_STATIC_SCRATCH_BYTES buffer that is
 * part of the library image: every GPU that loads the library carries it until the
 * process exits (the statistics pass uses as many token slices as fit in it).  Shapes whose
 * statistics need more (mpfa_quantize_workspace_min_bytes(B, H_q, H_kv) >
 * MPFA_STATIC_SCRATCH_BYTES, i.e. roughly B * (H_q + H_kv) > 250) are rejected
 * with MPFA_ERR_WORKSPACE and nothing is launched; with MPFA_STATS_FROZEN no statistics are
 * accumulated, the buffer is not used and no limit applies.  The call allocates nothing and frees
 * nothing.  The first call on each device looks up the buffer's device address (with that
 * device current); make that first call before starting any stream capture.  All calls on
 * a device share the one buffer, which keeps whatever the previous call left in it: each
 * call clears what it needs on `stream` before use, and two calls whose GPU work overlaps
 * (different streams, or different host threads on different streams) race on it - keep
 * them on one stream or order them yourself. */
#define MPFA_STATIC_SCRATCH_BYTES (512 * 1024)
mpfa_status mpfa_quantize_qk_static(const void *q_bf16, const void *k_bf16, int B, int N_q, int N_kv, int H_q,
                                    int H_kv, int flags, mpfa_stats *h_stats, mpfa_fp4_tensor *h_q_out,
                                    mpfa_fp4_tensor *h_k_out, void *delta_s_bf16, void *stream);
size_t mpfa_static_scratch_bytes(void);

/* Algorithm 1 line 4: V is not centered; code = E4M3(v / v_scale), round to nearest even,
 * saturating at +-448.  v_bf16 [B, N_kv, H_kv, 128] -> v_fp8 [B, H_kv, N_kv_pad, 128]
 * (1024-byte aligned).  v_scale = 1.0f is the plain cast. */
mpfa_status mpfa_quantize_v(const void *v_bf16, int B, int N_kv, int H_kv, float v_scale, uint8_t *v_fp8,
                            void *stream);

/* For MPFA_VARIANT_PV_BF16 only (Section 3.1's NVFP4 + BF16 assignment): V unchanged, re-tiled from
 * [B, N_kv, H_kv, 128] to [B, H_kv, N_kv_pad, 128] BF16 (pad rows zero; 1024-byte aligned, 2 * mpfa_v_fp8_bytes()). */
mpfa_status mpfa_pack_v_bf16(const void *v_bf16, int B, int N_kv, int H_kv, void *v_tiles_bf16, void *stream);

/* For MPFA_VARIANT_PV_FP4 only (Section 3.1's NVFP4 + NVFP4 assignment): V as the block-scaled FP4 operand of the
 * second MMA.  That MMA contracts over the keys, so the 16-element blocks of Eq. 1 lie along the TOKEN axis (tokens
 * 16 g .. 16 g + 15 of one channel; tokens past N_kv count as zero).  Recipe of the Q/K quantizer with the caller's
 * tensor scale in place of a statistic and no centering: block scale = E4M3(amax / (6 v_gscale)), code =
 * E2M1(v * (1 / (decode(scale) * v_gscale))); v_gscale = max|V| / (6 * 448) uses the whole range.
 * v_fp4 (1024-byte aligned, mpfa_v_fp4_bytes()): codes [B, H_kv, N_kv_pad/128, 128 channels, 64 bytes] (two keys per
 * byte, the even key in the low nibble) followed by the block scales, two 512-byte atoms per (b, h, tile) in the
 * tcgen05.cp order (atom = 64 keys; byte (channel mod 32) * 16 + (channel / 32) * 4 + block mod 4). */
size_t mpfa_v_fp4_bytes(int B, int H_kv, int N_kv);
mpfa_status mpfa_quantize_v_fp4(const void *v_bf16, int B, int N_kv, int H_kv, float v_gscale, uint8_t *v_fp4,
                                void *stream);

/* The same arithmetic for ONE request, written through its page-table row into the paged
 * cache (Section 6: low-bit K/V cache writes fused with quantization and compensation
 * generation).  k_bf16, v_bf16 [N_tokens, H_kv, 128] are the tokens at positions
 * [first_token, first_token + N_tokens) of the request; page_table_row[i] is the physical
 * page of tokens [64 i, 64 i + 64).  h_stats points at this request's statistics
 * (B = 1 slices).  Without MPFA_STATS_FROZEN (allowed only when first_token == 0) k_mean and
 * k_gscale are computed from these tokens; q_mean and q_gscale are always read.
 * With MPFA_STATS_FROZEN first_token may be any position (decode-time append, Section 6: a
 * new token is centered with the frozen means and quantized with the frozen tensor scale):
 * the tokens land in their slots of partly filled pages without touching their neighbours.
 * Slots beyond the written tokens are zero-filled in every page that this call starts
 * (position 0 of the page is among the written tokens); decode relies on that. */
mpfa_status mpfa_quantize_kv_paged(const void *k_bf16, const void *v_bf16, int N_tokens, int first_token,
                                   int H_q, int H_kv, int flags, mpfa_stats *h_stats, float v_scale,
                                   const mpfa_paged_kv *h_kv, const int32_t *page_table_row,
                                   void *workspace, size_t workspace_bytes, void *stream);

/* Decode-time append for a whole batch in one launch (Section 6): request b gets ONE new token,
 * k_bf16 / v_bf16 [B, 1, H_kv, 128], written at token index positions[b] (device int32 [B]; normally the
 * request's length before the call; negative: the request is skipped) of the pages page_table[b, :]
 * ([B, max_pages_per_req], device).  The token is centered with the request's frozen k_mean, quantized with
 * its frozen k_gscale (stats holds [B, ...] arrays and is only read), V with v_scale, and with MPFA_SMOOTH its
 * Delta_S entries are written for the H_q / H_kv heads of each group.  A token that starts a page zeroes the
 * other 63 slots of that page.  Same bytes as B calls of mpfa_quantize_kv_paged with N_tokens = 1 and
 * MPFA_STATS_FROZEN.  A position without a page-table entry or a page id outside the pool is skipped. */
mpfa_status mpfa_append_kv_paged(const void *k_bf16, const void *v_bf16, int B, int H_q, int H_kv, int flags,
                                 const mpfa_stats *h_stats, float v_scale, const mpfa_paged_kv *h_kv,
                                 const int32_t *page_table, int max_pages_per_req, const int32_t *positions,
                                 void *stream);

/* ---- stage 2: Algorithm 1 lines 6-20 -------------------------------------------------- */

/* QK4PV8 prefill.  q: [B, H_q, N_q] tile-layout tensor, k: [B, H_kv, N_kv], v_fp8 and
 * delta_s_bf16 as written by stage 1 (delta_s_bf16 == NULL: no compensation MMA).
 * KV blocks of 128 keys are visited from the last visible block down to block 0
 * (Section 4.1); causal != 0 masks key j for query i when j > i + N_kv - N_q.
 * softmax_scale is folded into the exponent together with the tensor scales
 * (Section 5.1): lambda = softmax_scale * log2(e) * q_gscale[b] * k_gscale[b].
 * out_bf16 [B, N_q, H_q, 128]; out_f32 (optional, may be NULL) receives the same values
 * before the final BF16 rounding.  device_status: one int32, caller-zeroed. */
mpfa_status mpfa_prefill(const mpfa_fp4_tensor *h_q, const mpfa_fp4_tensor *h_k, const uint8_t *v_fp8,
                         const void *delta_s_bf16, const mpfa_stats *h_stats, float v_scale, int causal,
                         float softmax_scale, void *out_bf16, float *out_f32, int32_t *device_status,
                         void *stream);

/* Ablation variants of mpfa_prefill (Section 7.4; same arguments, same outputs):
 *   variant 0                             the product path, identical to mpfa_prefill;
 *   MPFA_VARIANT_COMP_ELEMENTWISE         compensation placed on the softmax path (Section 3.2): the BF16 seed
 *                                         MMA is not issued; the softmax threads load the same BF16 Delta_S values
 *                                         and add them to the FP32 scores one by one, before masking and the
 *                                         running maximum.  Same term, one FP32 rounding placed differently; it
 *                                         exists to measure what the rank-one MMA saves.  With delta_s_bf16 == NULL
 *                                         it is the same as variant 0.
 *   MPFA_VARIANT_PV_BF16                  the NVFP4 + BF16 precision assignment of Section 3.1 / Section 7.2: Q K^T as in
 *                                         the product path (block-scaled FP4 MMA + rank-one seed), but P = 2^(lam S -
 *                                         lam m) is rounded to BF16 (no scale 448) and the second MMA is BF16 x BF16 on
 *                                         the UNQUANTIZED V.  For this variant the v_fp8 argument points at the BF16
 *                                         tile tensor [B, H_kv, N_kv_pad, 128] written by mpfa_pack_v_bf16 (1024-byte
 *                                         aligned) and v_scale must be 1.  It exists to measure what FP8 for P V buys
 *                                         (always in the one-query-tile arrangement).
 *   MPFA_VARIANT_PV_FP4                   the NVFP4 + NVFP4 precision assignment of Section 3.1 / Section 7.2: Q K^T as in
 *                                         the product path; q = 448 P is quantized per row and 16 keys (block scale
 *                                         E4M3(max q), codes E2M1(q * (6 / scale)): the tensor scale of P is fixed at
 *                                         1 / (6 * 448)), written to shared memory as a K-major operand with its scale
 *                                         factors, and the second MMA is block-scaled FP4 x FP4 on the V operand written
 *                                         by mpfa_quantize_v_fp4 (passed as the v_fp8 argument; v_scale = the v_gscale
 *                                         given there).  It exists to reproduce the paper's observation that this
 *                                         assignment is slower than FP8 for P V (always in the one-query-tile arrangement).
 * Any other value: MPFA_ERR_INVALID_ARG. */
enum { MPFA_VARIANT_COMP_ELEMENTWISE = 1, MPFA_VARIANT_PV_BF16 = 2, MPFA_VARIANT_PV_FP4 = 3 };
mpfa_status mpfa_prefill_variant(const mpfa_fp4_tensor *h_q, const mpfa_fp4_tensor *h_k, const uint8_t *v_fp8,
                                 const void *delta_s_bf16, const mpfa_stats *h_stats, float v_scale, int causal,
                                 float softmax_scale, int variant, void *out_bf16, float *out_f32,
                                 int32_t *device_status, void *stream);

/* The prefill calls have two work arrangements with identical per-row arithmetic (every row visits the same
 * 128-key blocks in the same order, so outputs agree to FP32 rounding of the accumulator rescaling):
 *   0 (default) one query tile per CTA, two softmax groups alternating over the KV blocks, two output
 *     accumulators so that the rescaling of one is off the critical path of the MMAs into the other;
 *   1 two adjacent query tiles per CTA, each with its own softmax warpgroup and output accumulator (the two query
 *     stages of Section 5.1), every K/V block loaded once for both.  Measured slower on B200 (the single
 *     accumulator per tile puts the rescaling between dependent MMAs); kept for that comparison.
 * Process-wide switch (mpfa_prefill, mpfa_prefill_variant, mpfa_prefill_paged); MPFA_ERR_INVALID_ARG for other values. */
int mpfa_set_prefill_arrangement(int arrangement);

/* QK4PV8 prefill of a chunk of queries against the paged cache (Section 6: the serving path keeps
 * K/V only in low-bit pages; a later chunk of the prompt, or a prompt with a cached prefix,
 * attends to them there).  q: [B, H_q, N_q] tile-layout tensor holding, for every request, the
 * LAST N_q tokens of its context, quantized with the request's frozen statistics; seq_lens[b]
 * (device) is the request's context length including those tokens, whose K/V must already be in
 * the cache (mpfa_quantize_kv_paged).  Causal, bottom-right aligned: query i of the chunk sees
 * keys 0 .. seq_lens[b] - N_q + i.  Same arithmetic and block order as mpfa_prefill (128-key
 * blocks counted from key 0, visited last to first); lambda uses q_gscale[b] * k_gscale[b].
 * Delta_S is applied when the cache has a delta_s pool.  A page-table entry outside
 * [0, num_pages) raises MPFA_DEV_BAD_PAGE in *device_status (output of that request undefined,
 * no out-of-pool access); a seq_lens[b] above 64 * max_pages_per_req is treated as that bound.
 * q_lens (device, may be NULL): per-request number of queries, 0 <= q_lens[b] <= N_q
 * (a batch of chunks of different lengths): request b's queries are rows 0 .. q_lens[b]-1 of its slab of q and
 * are the last q_lens[b] tokens of its context; the outputs of the remaining rows are zero.
 * out_bf16 [B, N_q, H_q, 128]; out_f32 optional. */
mpfa_status mpfa_prefill_paged(const mpfa_fp4_tensor *h_q, const mpfa_paged_kv *h_kv, const int32_t *page_table,
                               int max_pages_per_req, const int32_t *seq_lens, const int32_t *q_lens,
                               const mpfa_stats *h_stats,
                               float v_scale, float softmax_scale, void *out_bf16, float *out_f32,
                               int32_t *device_status, void *stream);

/* QK4PV8 decode (Section 5.3): one query token per request (q: tile-layout tensor with
 * N = 1, centered with the frozen means), its first seq_lens[b] keys found through
 * page_table [B, max_pages_per_req].  Each (request, kv head, 1024-token partition) keeps a
 * local (m, l, O) state for its GQA group in `workspace`; a second kernel merges the
 * partitions by log-sum-exp.  The number of partitions is fixed by max_seq_len, so the call
 * sequence (one 4-byte memory set of the work counter at the end of `workspace`, two kernels)
 * does not depend on seq_lens.  Work items are drawn from that counter by the running CTAs, so
 * two calls that overlap on the GPU need separate workspaces.  out_bf16 [B, H_q, 128]; out_f32 optional. */
mpfa_status mpfa_decode(const mpfa_fp4_tensor *h_q, const mpfa_paged_kv *h_kv, const int32_t *page_table,
                        int max_pages_per_req, const int32_t *seq_lens, const mpfa_stats *h_stats,
                        float v_scale, float softmax_scale, void *out_bf16, float *out_f32, void *workspace,
                        size_t workspace_bytes, int32_t *device_status, void *stream);

/* ---- measurement aid ------------------------------------------------------------------- */

/* (Not a step of the paper's method: the roofline denominator for Sections 5.1-5.2's three MMA kinds.)
 * Launches one CTA per SM that issues 4 * iters back-to-back tcgen05.mma instructions of one kind,
 * M = 128, N = n_cols (128 or 256), on operands resident in shared / tensor memory, and waits for the last:
 *   kind 0  kind::f16, BF16 x BF16, K = 16 (the rank-one seed of Eq. 11)
 *   kind 1  kind::f8f6f4, E4M3 x E4M3, K = 32, both operands in shared memory
 *   kind 2  kind::f8f6f4, E4M3 x E4M3, K = 32, A in tensor memory (the P V form)
 *   kind 3  kind::mxf4nvf4.block_scale.scale_vec::4X, E2M1 x E2M1, K = 64 (the Q K^T form)
 * The caller times the call with CUDA events; mpfa_bench_mma_flops gives the FLOPs ONE CTA issued
 * (multiply by the SM count).  Results are not meaningful data.  device_status as for the attention calls. */
mpfa_status mpfa_bench_mma_peak(int kind, int n_cols, int iters, int32_t *device_status, void *stream);
double mpfa_bench_mma_flops(int kind, int n_cols, int iters);

/* ---- sizes, layout maps, diagnostics (host only, no CUDA calls) ----------------------- */
size_t mpfa_quantize_workspace_bytes(int B, int H_q, int H_kv);
size_t mpfa_quantize_workspace_min_bytes(int B, int H_q, int H_kv);
size_t mpfa_decode_workspace_bytes(int B, int H_q, int H_kv, int max_pages_per_req);
size_t mpfa_fp4_codes_bytes(int B, int H, int N);
size_t mpfa_fp4_sf_bytes(int B, int H, int N);
size_t mpfa_delta_s_bytes(int B, int H_q, int N_kv);
size_t mpfa_v_fp8_bytes(int B, int H_kv, int N_kv);
/* byte offset of the scale of (b, h, token, block) inside mpfa_fp4_tensor.sf */
size_t mpfa_sf_offset(int H, int N, int b, int h, int token, int block);
/* byte offsets inside one (page, kv head) slab of the paged cache */
size_t mpfa_paged_k_offset(int token, int block, int byte_in_block);
size_t mpfa_paged_v_offset(int token, int channel);
const char *mpfa_status_string(mpfa_status s);
int mpfa_last_cuda_error(void);
int mpfa_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MPFA_H_ */
