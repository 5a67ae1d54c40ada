/*
 * hyq.h - C ABI of the B200 (sm_100a) HyQuant prefill path.
 *
 * Three operations, in the order the paper's prefill operator runs them
 * (Algorithm 2: Stage 1 -> Stage 2 -> Stage 3):
 *
 *   hyq_select_vertical            Algorithm 1 (vertical token identification)
 *   hyq_select_vertical_mass       Eq. 4-5 (the same selection from accumulated softmax column mass)
 *   hyq_quantize_blocks            Algorithm 2, Stage 2 (per-tile quantization)
 *   hyq_hybrid_attention_prefill   Eq. 6-7 / Algorithm 2, Stage 3 (fused hybrid softmax attention)
 *   hyq_*_varlen                   the same three stages over a ragged batch of prompts
 *
 * Common rules
 *   - Every tensor pointer is a DEVICE pointer to a contiguous row-major array.
 *     Q is [B, Hq, L, D]; K and V are [B, Hkv, L, D]; bf16 unless stated.
 *     Hq % Hkv == 0; query head h reads kv head h / (Hq / Hkv) (Algorithm 1's
 *     reshape Hq -> Hkv x g).  D must be 128.  L >= 1 is arbitrary (ragged tails
 *     are handled).  The attention call also takes a query block of Lq < L rows
 *     (see there); everywhere else the queries number L.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *     enqueue work and return; they never synchronise.
 *   - The caller owns every buffer, including `workspace`; the library allocates
 *     no device memory and keeps no pointer once the enqueued work has completed.
 *     Workspace sizes come from the *_workspace queries (host-only, no launches).
 *     Workspace and tensor pointers must be 16-byte aligned.
 *   - Return value: HYQ_OK or an error code.  Arguments are checked on the host
 *     before anything is launched; on error nothing has been enqueued.  Device-side
 *     anomalies (a bounded wait that ran out) are written to `status_word` and
 *     the kernel exits normally - no trap, no hang.
 *   - NaN / Inf inputs are undefined behaviour.
 */
#ifndef HYQ_H_
#define HYQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  HYQ_OK = 0,
  HYQ_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, k > P, Hq % Hkv != 0 ... */
  HYQ_ERR_UNSUPPORTED = 2,   /* D != 128, block_tokens not 32 / 64 / 128, format combination not built */
  HYQ_ERR_WORKSPACE = 3,     /* workspace_bytes smaller than the matching *_workspace query */
  HYQ_ERR_ALIGNMENT = 4,     /* a pointer is not 16-byte aligned */
  HYQ_ERR_CUDA = 5,          /* a CUDA runtime / driver call failed (launch, tensor map) */
  HYQ_ERR_TIMEOUT = 6        /* value written to status_word by a kernel whose bounded wait expired */
};

/* low-bit formats of Algorithm 2 Stage 2 (c_B = 127 / 448; 7 for INT4) */
enum { HYQ_FMT_INT8 = 0, HYQ_FMT_FP8_E4M3 = 1, HYQ_FMT_INT4 = 2 };

/* attention kernel choice */
enum {
  HYQ_IMPL_AUTO = 0,      /* the tensor-core kernel */
  HYQ_IMPL_TCGEN05 = 1,   /* TMA + tcgen05.mma + TMEM kernel */
  HYQ_IMPL_SIMT = 2       /* plain fp32 CUDA-core kernel: slow, used to cross-check at sizes the CPU cannot */
};

/* Static string for a status code. */
const char* hyq_status_string(int status);

/* Library ABI version (bumped when a signature or struct changes). */
int hyq_version(void);

/* Algorithm 1's count: k = min(P, max(1, ceil(P * ratio))) with P = max(0, Lk - window); 0 when P == 0. */
int hyq_paper_k(int Lk, int window, double ratio);

/* ---------------------------------------------------------------------------------------------
 * hyq_select_vertical - Algorithm 1 (vertical token identification).
 *
 *   P    = max(0, Lk - window)                      candidate keys: the non-window prefix [0, P)
 *   t    = n_tail, or min(window, Lq) if n_tail == 0
 *   qbar = mean of the last t query rows of head (b, h)           (fp64)
 *   S[p] = qbar . K[b, h / g, p, :]                               (fp64 fma chain over channels 0..D-1)
 *   idx_out[b, h, :] = positions of the k largest S, equal scores resolved towards the
 *                      lower position, written in ASCENDING position order.
 *
 *   q [B,Hq,Lq,D] bf16, k_ [B,Hkv,Lk,D] bf16 (device, read-only).
 *   idx_out [B,Hq,k] int32 (device, written).  k == 0 or P == 0: nothing is written, HYQ_OK.
 *   Errors: k > P or k < 0, n_tail > Lq, window == 0 with n_tail == 0 and k > 0 -> INVALID_ARG.
 *   workspace: hyq_select_vertical_workspace bytes (tail means + one fp64 score per (b,h,p)).
 * ------------------------------------------------------------------------------------------- */
int hyq_select_vertical_workspace(int B, int Hq, int Hkv, int Lq, int Lk, int D, int window, int k,
                                  size_t* bytes /* host, out */);
int hyq_select_vertical(const void* q, const void* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D,
                        int window, int n_tail, int k, int32_t* idx_out, void* workspace,
                        size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * hyq_select_vertical_static - hyq_select_vertical for callers that have no device memory to lend.
 * (No counterpart in the paper: it computes exactly what hyq_select_vertical computes and exists
 * only because of how its scratch memory is provided.)
 *
 *   Some callers cannot hand over a workspace: a plug-in running inside a serving process whose
 *   memory pool already owns the whole GPU has nothing left to allocate from, and a latency-critical
 *   loop cannot afford cudaMalloc, which synchronises the device.  For them the tail means and the fp64
 *   scores are kept in a fixed array of HYQ_SELECT_STATIC_SCRATCH_BYTES that is part of the library
 *   image: every GPU that loads the library carries those bytes until the process exits, used or not.
 *   The call allocates nothing and frees nothing, neither itself nor through a library routine.
 *
 *   Arguments, results and errors are those of hyq_select_vertical without workspace / workspace_bytes,
 *   plus: a problem whose scratch need (hyq_select_vertical_workspace) exceeds
 *   HYQ_SELECT_STATIC_SCRATCH_BYTES returns HYQ_ERR_WORKSPACE and launches nothing.
 *   (8 MiB covers B*Hq*(P + 128) <= 1 Mi scores, e.g. 32 query heads at L = 32768, window 1024.)
 *
 *   The first call on each device looks up the array's device address (one runtime query, made with
 *   that device current, result cached); make that first call outside any stream capture.  The cached
 *   address belongs to the device's primary context: a process that destroys that context
 *   (cudaDeviceReset) and creates a new one must not go on using this entry point.
 *   All calls on a device share the one array and each call overwrites what the previous one left
 *   (nothing in it has to start at zero): two calls whose kernels overlap on the GPU - different
 *   streams, or different host threads - race on it.  Run them one after the other.
 * ------------------------------------------------------------------------------------------- */
#define HYQ_SELECT_STATIC_SCRATCH_BYTES (8u << 20)
int hyq_select_vertical_static(const void* q, const void* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D,
                               int window, int n_tail, int k, int32_t* idx_out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * hyq_select_vertical_mass - Eq. 4-5: the vertical-line score as accumulated column mass.
 *
 *   T    = the last n_queries query rows (n_queries == 0: min(window, Lq), Algorithm 1's tail); the query
 *          block is end-aligned with the keys: row i sits at position Lk - Lq + i.  n_queries <= window, so
 *          that every candidate key is visible to every query of T.
 *   a_tj = softmax over the keys j <= pos(t) of softmax_scale * <Q[t], K[j]>            (bf16 originals)
 *   S[p] = sum over t in T of a_tp,    p in the non-window prefix [0, P),  P = max(0, Lk - window)
 *   idx_out[b, h, :] = positions of the k largest S, ties towards the lower position, ASCENDING.
 *
 *   All arithmetic is fp64 with a fixed order of operations (fma chain over channels, a polynomial exp,
 *   row sums as 64-key chunk trees combined in ascending order, queries added in ascending order), so the
 *   selected set is reproducible bit for bit.  Cost: two passes of n_queries * Lk * D fp64 fma per head -
 *   meant for a handful of tail queries (tens), not for the whole window.
 *
 *   Arguments, outputs and errors as hyq_select_vertical, plus: n_queries > min(window, Lq) or Lq > Lk ->
 *   INVALID_ARG.  softmax_scale 0 => 1/sqrt(D).  workspace: hyq_select_vertical_mass_workspace bytes.
 * ------------------------------------------------------------------------------------------- */
int hyq_select_vertical_mass_workspace(int B, int Hq, int Hkv, int Lq, int Lk, int D, int window, int n_queries,
                                       int k, size_t* bytes /* host, out */);
int hyq_select_vertical_mass(const void* q, const void* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D,
                             int window, int n_queries, int k, float softmax_scale, int32_t* idx_out,
                             void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * hyq_quantize_blocks - Algorithm 2, Stage 2 (per-tile symmetric quantization).
 *
 *   One tile = block_tokens (32, 64 or 128; the workloads use 64) consecutive tokens x all D channels of one (b, head), cut by
 *   original position; the last tile of a head may be ragged.
 *     absmax = max |x| over the tile
 *     scale  = absmax / c          c = 127 (INT8), 448 (FP8 e4m3), 7 (INT4)
 *     code   = round_half_even(x * (c / absmax))     INT8 / INT4: integer, clamped to [-c, c]
 *                                                    FP8: e4m3 (RNE, saturating at +-448)
 *   All in fp32 with one rounding per operation.  absmax < 2^-100 (all-zero tile): scale 0, codes 0.
 *
 *   x [B,H,L,D] bf16 (device, read-only).
 *   codes_out (device, written): INT8 / FP8: [B,H,L,D] bytes; INT4: [B,H,L,D/2] bytes, channel 2m
 *       in the low nibble and 2m+1 in the high nibble of byte m, two's complement.
 *   scales_out [B,H,ceil(L/block_tokens)] fp32 (device, written).
 * ------------------------------------------------------------------------------------------- */
int hyq_quantize_blocks(const void* x, int B, int H, int L, int D, int block_tokens, int format,
                        void* codes_out, float* scales_out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * hyq_hybrid_attention_prefill - Eq. 6-7 / Algorithm 2 Stage 3: causal attention forward in which,
 * for query row i of head (b,h) and every key j <= i,
 *     the pair is FULL PRECISION when j is in vl_idx[b,h,:] or i - j < window,
 *         score = softmax_scale * <Q[i], K[j]>  (bf16 originals),   value row = V[j]
 *     and LOW-BIT otherwise,
 *         score = softmax_scale * q_scale * k_scale * <q_code[i], k_code[j]>,
 *         value row = v_scale * v_code[j]
 * and one softmax runs over all keys of the row:  out[i] = sum_j p_ij value_j / sum_j p_ij.
 *
 *   Query block (Algorithm 2 takes a query block against the full K, V): with 0 < Lq < L the call computes
 *   the LAST Lq query rows of a context of L keys - query row r sits at position L - Lq + r and sees the keys
 *   j <= L - Lq + r, with the same two predicates on positions.  q, q_codes, out then hold Lq rows per head,
 *   q_scales ceil(Lq/64) entries per head (quantization blocks counted from the first row of the block, as
 *   hyq_quantize_blocks writes them for a [B,Hq,Lq,D] tensor) and lse Lq entries; K, V and vl_idx are those
 *   of the whole context.  Lq = 0 or Lq = L is the whole prefill.  Lq > L -> HYQ_ERR_INVALID_ARG.
 *   (For short blocks the tensor-core path splits the keys over several CTAs per query tile and merges the
 *   partial results; the workspace query accounts for their buffers.  Results do not depend on the split up to
 *   fp32 rounding.)
 *
 *   Window form: HYQ_WINDOW_SLIDING - key j is a window key of the row at position i iff i - j < window (every
 *   row has its own last `window` positions; the form the whole prefill needs).  HYQ_WINDOW_FIXED_TAIL -
 *   Algorithm 2's K_Win taken literally: the window keys are the last `window` keys [L - window, L) for every
 *   row of the block (rows before L - window then have no window keys).  Both forms agree on the last row.
 *
 *   struct_size must be sizeof(hyq_attn_args).  Supported format triples (q,k,v):
 *   (INT8,INT8,INT8), (FP8_E4M3,FP8_E4M3,FP8_E4M3) - the paper's two bit widths, c_B = 127 and 448 - and
 *   (INT4,INT4,FP8_E4M3); anything else -> HYQ_ERR_UNSUPPORTED.
 *   Value range: the value rows enter the P.V products as fp16, so |V| must stay below 65504 (attention values of
 *   real layers do); larger magnitudes are clamped to +-65504 instead of becoming infinities.  Inputs must be
 *   finite.
 *   vl_idx [B,Hq,k] int32, each row strictly ascending, values in [0, L); NULL iff k == 0.
 *   out [B,Hq,L,D]: fp32 (out_dtype 1) or bf16 (out_dtype 0, RNE of the fp32 result).
 *   lse: optional [B,Hq,L] fp32 natural-log-sum-exp of the scaled scores (NULL to skip).
 *   status_word: optional device int32; the kernel stores HYQ_ERR_TIMEOUT there if one of its
 *   bounded waits expires (the output is then undefined); untouched otherwise.
 *   ev_kernel_start / ev_kernel_stop: optional caller-created CUDA events for profiling (NULL to skip).
 * ------------------------------------------------------------------------------------------- */
enum { HYQ_WINDOW_SLIDING = 0, HYQ_WINDOW_FIXED_TAIL = 1 };

typedef struct {
  uint32_t struct_size;
  int32_t B, Hq, Hkv, L, D;
  int32_t window, k, block_tokens;   /* block_tokens: 32, 64 or 128, as given to hyq_quantize_blocks for Q, K and V */
  int32_t q_format, k_format, v_format;
  int32_t out_dtype;                 /* 0 = bf16, 1 = fp32 */
  int32_t impl;                      /* HYQ_IMPL_* */
  float softmax_scale;               /* 0 => 1/sqrt(D) */
  const void* q;                     /* bf16 originals */
  const void* k_;
  const void* v;
  const void* q_codes;               /* as written by hyq_quantize_blocks */
  const void* k_codes;
  const void* v_codes;
  const float* q_scales;
  const float* k_scales;
  const float* v_scales;
  const int32_t* vl_idx;
  void* out;
  float* lse;
  int32_t* status_word;
  void* workspace;
  size_t workspace_bytes;
  void* ev_kernel_start;             /* optional cudaEvent_t, recorded on the stream right before ... */
  void* ev_kernel_stop;              /* ... and right after the attention kernel proper (pre-pass excluded) */
  int32_t Lq;                        /* query rows; 0 => L (whole prefill).  See "query block" above. */
  int32_t window_mode;               /* HYQ_WINDOW_SLIDING (0, default) or HYQ_WINDOW_FIXED_TAIL (1) */
} hyq_attn_args;

int hyq_hybrid_attention_prefill_workspace(const hyq_attn_args* args, size_t* bytes /* host, out */);
int hyq_hybrid_attention_prefill(const hyq_attn_args* args, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Ragged batches (several prompts of different lengths in one call; the serving shape of the paper's batching
 * study, Section 4.3).  The three stages run per sequence exactly as the calls above define them - every sequence is
 * its own problem with its own L, its own candidate prefix, its own quantization blocks (which restart at the
 * sequence's first token) and its own causal / window / vertical-key predicates - so each *_varlen call returns,
 * sequence by sequence, bit for bit what the plain call returns for that sequence alone.
 *
 *   Packing.  cu_seqlens is a HOST array of n_seq + 1 ascending token offsets (cu_seqlens[0] = 0; sequence s has
 *   L_s = cu_seqlens[s+1] - cu_seqlens[s] >= 1 tokens).  A packed tensor with H heads holds the sequences one after
 *   the other, each as a contiguous [H, L_s, D] block: sequence s starts at element H * D * cu_seqlens[s].
 *   Packed codes follow the same rule in bytes per row (D, or D/2 for INT4).  Packed scales hold [H, nb_s] per
 *   sequence with nb_s = ceil(L_s / block_tokens): sequence s starts at H * (sum of nb_r over r < s).  k_per_seq is
 *   a HOST array of n_seq vertical counts (0 <= k_s <= max(0, L_s - window)); the packed index buffer holds
 *   [Hq, k_s] per sequence, sequence s starting at Hq * (sum of k_r over r < s).
 *
 *   The sequences are processed one after the other on `stream` (longest first); one workspace of the size the
 *   plain query returns for the LONGEST sequence (B = 1) serves them all.  Host arrays are read during the call
 *   and may be freed afterwards.  Errors: as the plain calls, checked for every sequence before anything is
 *   launched; n_seq <= 0 or a non-ascending cu_seqlens -> INVALID_ARG.
 *
 *   hyq_hybrid_attention_prefill_varlen takes a hyq_attn_args whose tensor pointers are the PACKED buffers and
 *   whose B, L, Lq and k fields are ignored (whole prefills only: every sequence's queries are its L_s rows);
 *   out [packed, Hq heads] and lse (optional, Hq * L_s floats per sequence, sequence s at Hq * cu_seqlens[s]).
 * ------------------------------------------------------------------------------------------- */
int hyq_select_vertical_varlen(const void* q, const void* k_, int n_seq, const int32_t* cu_seqlens /* host */,
                               int Hq, int Hkv, int D, int window, int n_tail, const int32_t* k_per_seq /* host */,
                               int32_t* idx_out, void* workspace, size_t workspace_bytes, void* stream);
int hyq_quantize_blocks_varlen(const void* x, int n_seq, const int32_t* cu_seqlens /* host */, int H, int D,
                               int block_tokens, int format, void* codes_out, float* scales_out, void* stream);
int hyq_hybrid_attention_prefill_varlen(const hyq_attn_args* args, int n_seq, const int32_t* cu_seqlens /* host */,
                                        const int32_t* k_per_seq /* host */, void* stream);

/* ---------------------------------------------------------------------------------------------
 * hyq_test_set_attention_hooks - test hook (the paper has no counterpart): exercises the tensor-core
 * kernel's bounded-wait unwind without faulting anything.  Process-wide, not thread-safe, meant for tests only.
 *   wait_limit_clocks    SM clocks a single device-side barrier wait may take before the kernel gives up
 *                        (0: the default of about two seconds)
 *   drop_load_position   walk position (0-based key tile of a CTA) whose K/V copy the producer announces on its
 *                        barrier but never issues, so that every wait that depends on it runs out (-1: none)
 * With a dropped load the kernel returns normally, stores HYQ_ERR_TIMEOUT in status_word and leaves the output
 * undefined.  Returns HYQ_ERR_INVALID_ARG for negative limits or positions below -1.
 * ------------------------------------------------------------------------------------------- */
int hyq_test_set_attention_hooks(long long wait_limit_clocks, int drop_load_position);

/* ---------------------------------------------------------------------------------------------
 * hyq_test_read_attention_restarts - test hook (the paper has no counterpart).  The tensor-core kernel takes the
 * exponentials of most low-bit tiles against a row's reference as it stands and checks each tile's row sum
 * afterwards; a CTA in which some row's sum shows an fp16 overflow (a score more than 2^16 above all the row had
 * seen) discards its work and goes through its keys a second time with the maximum looked at in every tile.  This
 * call synchronises the device and returns in *count_out (host) how many CTAs have done so since the library was
 * loaded or the counter was last reset (reset != 0 clears it).  Errors: INVALID_ARG (null pointer), CUDA.
 * ------------------------------------------------------------------------------------------- */
int hyq_test_read_attention_restarts(unsigned long long* count_out /* host */, int reset);

#ifdef __cplusplus
}
#endif
#endif /* HYQ_H_ */
