/*
 * hyq_decode.h - C ABI of the decode side of the B200 (sm_100a) HyQuant library:
 *
 *   hyq_freeze                    Algorithm 4 (prefill -> decode hybrid KV-cache organisation)
 *   hyq_hybrid_attention_decode   Algorithm 3 / Section 3.3 (one new token against the hybrid cache,
 *                                 low-bit rows dequantized inside the attention kernel)
 *
 * The common rules of hyq.h hold (device pointers, contiguous row-major arrays, caller-owned buffers,
 * calls enqueue on `stream` and return, arguments checked on the host before anything is launched,
 * D = 128, Hq % Hkv == 0 with g = Hq / Hkv <= 64 query heads per KV head; more than 8 are served 8 at a time by
 * separate CTAs that read the same cache rows).
 *
 * The hybrid cache of one layer (Algorithm 4's four buffers), per (batch b, KV head h):
 *
 *   window       k_win, v_win  [B,Hkv,W',D] bf16   the last W' = min(window, N) prefill rows
 *   vertical     k_vl, v_vl    [B,Hkv,k,D]  bf16   rows vl_idx[b,h,:] of the prefill cache, in that order
 *   staging      k_s, v_s      [B,Hkv,staging_capacity,D] bf16, of which the first n_staging rows are
 *                              valid; hyq_kv_cache_append writes a new token's rows to row n_staging and
 *                              the caller counts them in n_staging.  Folding staged rows into the other
 *                              buffers is not described by the paper and not part of this library.
 *   quantized    the other nQ = N - W' - k prefix rows, COMPACTED in ascending position order and cut
 *                into groups of `group` (G = 32, 64 or 128) consecutive compacted rows x all D channels; each group is
 *                quantized exactly as hyq_quantize_blocks quantizes a tile (INT4, c_B = 7; INT8, c_B = 127; FP8 e4m3, c_B = 448;
 *                fp32 scale per group; the last group may be ragged).  Per head the row count is padded to
 *                nQp = G * ceil(nQ / G); padding rows hold unspecified codes and are never used.
 *       kq_codes  [B,Hkv,nQp,D/2] bytes: row-major, channel 2m in the low nibble and 2m+1 in the high
 *                 nibble of byte m, two's complement (hyq_quantize_blocks' INT4 layout).
 *       vq_codes  [B,Hkv,nQp/16,1024] bytes, FRAGMENT-MAJOR: the codes of 16 consecutive compacted rows
 *                 form one 1024-byte tile of 32 lanes x 8 little-endian 32-bit words, word x of lane l at
 *                 byte 512*(x >> 2) + 16*l + 4*(x & 3); nibble n (bits 4n..4n+3) of word x of lane
 *                 l = 4r + j holds
 *                     channel 64*(x >> 2) + 8*r + 2*(x & 3) + (n & 1)
 *                     of row  2*j + (n >> 2) + 8*((n >> 1) & 1)          of the tile,
 *                 i.e. each lane of a warp reads two 16-byte pieces (the warp: two contiguous 512-byte
 *                 runs) and owns, without any shuffle, the operand registers of the warp-level matrix
 *                 instruction that accumulates P.V.
 *       INT8 and FP8 caches: kq_codes [B,Hkv,nQp,D] bytes row-major (two's complement / e4m3); vq_codes [B,Hkv,nQp/16,2048]
 *                 bytes, fragment-major again: the tile is four 512-byte runs, lane l = 4r + j owns bytes
 *                 [16l, 16l + 16) of each, i.e. 16 words; word w = 2x + (row >> 3) sits at byte
 *                 512*(w >> 2) + 16*l + 4*(w & 3), and its four bytes hold, in order, the codes of
 *                 (channel c, row 2j + 8*(row >> 3)), (c, that row + 1), (c + 1, row), (c + 1, row + 1) with
 *                 c = 64*(x >> 2) + 8*r + 2*(x & 3).
 *       kq_scales, vq_scales  [B,Hkv,nQp/G] fp32.
 *
 * With capacities set (cap_* fields) the row counts after [B,Hkv, in the shapes above are the capacities.
 *
 * (Quant(.; G) over compacted rows, and one vertical set per KV head given by the caller, are this
 * library's readings: Algorithm 4 does not say how groups are cut after rows are removed, and Algorithm 1
 * yields one set per query head.)
 */
#ifndef HYQ_DECODE_H_
#define HYQ_DECODE_H_

#include "hyq.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  uint32_t struct_size;
  int32_t B, Hq, Hkv, D;
  int32_t N;                    /* prefill rows frozen */
  int32_t window;               /* W; the window buffers hold min(W, N) rows */
  int32_t k;                    /* vertical rows per KV head, 0 <= k <= N - min(W, N) */
  int32_t group;                /* G: 32, 64 or 128 rows per scale group */
  int32_t format;               /* K and V code format: HYQ_FMT_INT4 (K4V4), HYQ_FMT_INT8 or HYQ_FMT_FP8_E4M3 (K8V8) */
  int32_t staging_capacity;     /* W_s: rows allocated per head in k_s / v_s (may be 0) */
  int32_t n_staging;            /* valid staging rows, 0 <= n_staging <= staging_capacity */
  void* kq_codes;
  void* vq_codes;
  float* kq_scales;
  float* vq_scales;
  void* k_vl;
  void* v_vl;
  void* k_win;
  void* v_win;
  void* k_s;
  void* v_s;
  /* Row capacities per (b, KV head) of the quantized, vertical and window buffers, i.e. the strides between
   * heads: 0 = tight (nQp, k, W' as derived from N, window, k).  Larger capacities let sequences of different
   * lengths share one batch allocation (see hyq_hybrid_attention_decode_ragged); cap_quantized_rows must be a
   * multiple of G and each capacity at least the tight value. */
  int32_t cap_quantized_rows, cap_vertical, cap_window;
} hyq_kv_cache;

typedef struct {
  int64_t quantized_rows;        /* nQ */
  int64_t padded_rows;           /* nQp */
  size_t kq_codes_bytes, vq_codes_bytes;     /* whole batch, each */
  size_t scales_bytes;                       /* each of kq_scales, vq_scales */
  size_t vertical_bytes, window_bytes, staging_bytes;   /* each of the K and V buffers */
} hyq_kv_cache_sizes;

/* Host-only: buffer sizes for a cache description (pointers ignored).  Errors as hyq_freeze. */
int hyq_kv_cache_query_sizes(const hyq_kv_cache* cache, hyq_kv_cache_sizes* sizes /* host, out */);

/* ---------------------------------------------------------------------------------------------
 * hyq_freeze - Algorithm 4.  Reads the prefill cache k_, v [B,Hkv,N,D] bf16 and vl_idx [B,Hkv,k]
 * int32 (each row strictly ascending, values in [0, N - min(W,N)); NULL iff k == 0), writes the window,
 * vertical and quantized buffers of `cache` (layouts above).  The staging buffers are not touched
 * (an empty staging buffer is n_staging = 0).  The prefill cache may be freed once the enqueued
 * work has completed.  Errors: INVALID_ARG (null pointer, sizes out of range, struct_size),
 * UNSUPPORTED (D != 128, group not 32 / 64 / 128, format not INT4 / INT8 / FP8_E4M3, g > 64), ALIGNMENT (a code or bf16 buffer not 16-byte aligned, a scale array not 4-byte aligned).
 * ------------------------------------------------------------------------------------------- */
int hyq_freeze(const void* k_, const void* v, const int32_t* vl_idx, const hyq_kv_cache* cache, void* stream);

/* ---------------------------------------------------------------------------------------------
 * hyq_kv_cache_append - places one new token's key and value rows in the staging buffer (Algorithm 4's
 * "newly generated tokens are first placed in a small staging buffer"): k_new, v_new [B,Hkv,D] bf16 (device)
 * are copied to row cache->n_staging of k_s / v_s.  The description is not modified: the caller counts the row
 * (n_staging + 1) in the description it passes to the next attention call.  n_staging == staging_capacity ->
 * HYQ_ERR_INVALID_ARG (buffer full).  Other errors as hyq_freeze.
 * ------------------------------------------------------------------------------------------- */
int hyq_kv_cache_append(const void* k_new, const void* v_new, const hyq_kv_cache* cache, void* stream);

/* ---------------------------------------------------------------------------------------------
 * hyq_hybrid_attention_decode - Algorithm 3 / Section 3.3 for one token per sequence:
 *     s_j   = softmax_scale * <q[b,h], key_j>      over every cached row j of KV head h / g, where
 *             key_j / value_j = scale(group) * code for quantized rows, the bf16 row otherwise
 *     out[b,h] = sum_j softmax(s)_j value_j
 *   The four segments are read once; the rows are cut into `splits` slices that independent CTAs reduce
 *   with an online softmax, and a second kernel merges the slices (the split/ReduceSoftmax of Algorithm 3,
 *   applied to all four segments instead of the quantized one only: one softmax either way).
 *
 *   q [B,Hq,D] bf16 (device).  out [B,Hq,D]: bf16 (out_dtype 0) or fp32 (1).  lse: optional [B,Hq] fp32,
 *   natural-log-sum-exp of the scaled scores (NULL to skip).  softmax_scale 0 => 1/sqrt(D).
 *   splits: 1 <= S <= 1024, or 0 for a choice that fills the GPU.  workspace: hyq_hybrid_attention_decode_workspace
 *   bytes (the slices' partial results).  The cache must hold at least one row in total.
 *   Errors: as hyq_freeze, plus WORKSPACE.
 * ------------------------------------------------------------------------------------------- */
int hyq_hybrid_attention_decode_workspace(const hyq_kv_cache* cache, int splits, size_t* bytes /* host, out */);
int hyq_hybrid_attention_decode(const void* q, const hyq_kv_cache* cache, float softmax_scale, int splits,
                                int out_dtype, void* out, float* lse, void* workspace, size_t workspace_bytes,
                                void* stream);

/* ---------------------------------------------------------------------------------------------
 * hyq_hybrid_attention_decode_ragged - the same attention for a batch of sequences of DIFFERENT lengths
 * (the serving case: every sequence has its own prefix length, vertical count and staging fill).
 *   `cache` describes the allocation: B sequences, strides given by the capacities (tight values if 0), and
 *   N / window / k / n_staging are upper bounds only.  lengths [B][4] int32 (device): for sequence b the valid
 *   rows {quantized, vertical, window, staging}, each at most the corresponding capacity, at least one row in
 *   total.  Sequence b's buffers are what hyq_freeze writes when called with B = 1, that sequence's own
 *   N / window / k, the batch's capacities, and the buffer pointers advanced to sequence b.
 *   Everything else as hyq_hybrid_attention_decode (same kernels; the slices of a head are cut from its own rows).
 * ------------------------------------------------------------------------------------------- */
int hyq_hybrid_attention_decode_ragged(const void* q, const hyq_kv_cache* cache, const int32_t* lengths,
                                       float softmax_scale, int splits, int out_dtype, void* out, float* lse,
                                       void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HYQ_DECODE_H_ */
