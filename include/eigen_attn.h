/*
 * eigen_attn.h -- C ABI of libeigenattn: Eigen Attention (attention in a per-head rank-r space)
 * for one decoder layer on one NVIDIA B200 (sm_100a).
 *
 * What is computed (paper: "Eigen Attention", Sections 2 and 4.2):
 *   - every new key/value row is projected onto the head's orthonormal bases,
 *       k' = k U^K_i ,  v' = v U^V_i                      (the r-wide factor of Eq. 6; Eq. 8 merged form)
 *     and appended to a rank-r KV cache, K'_i <- Concat(K'_i, k'), V'_i <- Concat(V'_i, v')
 *                                                          (Section 2, "LLM Inference")
 *   - a decode step attends one query per sequence over the n cached rows,
 *       h_i = Softmax( (q U^K_i) K'_i^T / sqrt(d_h) ) V'_i (U^V_i)^T          (Eq. 3 in the space of Eq. 7)
 *     the scale is 1/sqrt(d_head) although the vectors are r wide (Eq. 7);
 *   - a prefill call does the same for T prompt tokens at once with a causal mask
 *     (query t sees rows 0..len0+t) and leaves their rank-r rows in the cache (Section 2, prefill phase).
 *
 * Conventions
 *   - "d_" pointers are DEVICE pointers, "h_" pointers are HOST pointers.  Token tensors are
 *     [batch][T][n_heads][d_head] in the layer's IO dtype; the head and d_head axes are contiguous,
 *     the batch and token strides are passed in ELEMENTS.  The packed rank-space tensors selected by
 *     the *_PREPROJECTED / EA_OUT_LOWRANK flags are always contiguous; strides do not apply to them.
 *   - The caller owns every buffer, including the cache and the workspace (sizes from
 *     eigen_attn_cache_bytes).  The library allocates no device memory; a handle owns host memory only.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All calls
 *     are asynchronous with respect to that stream unless stated otherwise.
 *   - Every function returns an ea_status.  Argument, shape and capacity errors are found on the
 *     host before anything is launched and leave the handle unchanged.  Kernels never trap: a wait that
 *     exceeds its bound records EA_ERR_TIMEOUT in a device status word read by eigen_attn_poll_status.
 *   - A handle is not thread-safe.  The sequences of a handle share one length (`len`) unless
 *     eigen_attn_set_lens is in effect; `len` is then the length of the longest sequence.
 */
#ifndef EIGEN_ATTN_H_
#define EIGEN_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct eigen_attn* eigen_attn_t;   /* opaque; one per decoder layer */

typedef enum {
  EA_OK = 0,
  EA_ERR_INVALID_ARG = -1,      /* NULL pointer, bad enum, bad flag combination            */
  EA_ERR_SHAPE = -2,            /* a dimension out of the supported range, len == 0 decode */
  EA_ERR_CAPACITY = -3,         /* cache / workspace too small, len + T > n_max            */
  EA_ERR_UNSUPPORTED = -4,      /* a valid request this version does not implement         */
  EA_ERR_CUDA = -5,             /* a CUDA runtime call failed; see eigen_attn_last_error   */
  EA_ERR_TIMEOUT = -6,          /* a bounded device-side wait gave up                      */
  EA_ERR_NOT_ORTHONORMAL = -7   /* EA_CHECK_ORTHONORMAL: max|U^T U - I| > 1e-4             */
} ea_status;

typedef enum { EA_BF16 = 0, EA_FP32 = 1 } ea_dtype;   /* cache + IO dtype; accumulation is always fp32 */

/* ea_desc.flags */
#define EA_CHECK_ORTHONORMAL 0x1u   /* verify U^T U = I on the host at create (Section 4.2 assumes it) */
#define EA_ROPE_PROMPT_SCRATCH 0x2u /* the workspace also holds the prompt's rotated full-rank queries and lifted,
                                       rotated keys (2 * batch * max_prefill_tokens * n_heads * d_head 16-bit values):
                                       eigen_attn_prefill of a layer with rotary embedding then runs on the tensor
                                       cores while the rows cached after the call fit max_prefill_tokens */

/* per-call flags */
#define EA_Q_PREPROJECTED  0x1u  /* d_q already holds q U^K (merged W^Q', Eq. 8): [B][T][sum_h rp_k[h]]      */
#define EA_OUT_LOWRANK     0x2u  /* write o' without the (U^V)^T lift (merged W^O', Eq. 8): [B][T][sum rp_v] */
#define EA_KV_PREPROJECTED 0x4u  /* d_k/d_v already hold k U^K, v U^V (merged W^K', W^V'): packed like q above */

typedef struct {
  int32_t batch;               /* B >= 1                                                             */
  int32_t n_heads;             /* H, 1..256 (multi-head attention: one K/V head per query head)      */
  int32_t d_head;              /* d_h, multiple of 8, 8..128                                          */
  int32_t n_max;               /* cache capacity in rows per sequence                                 */
  int32_t dtype;               /* ea_dtype                                                            */
  int32_t max_prefill_tokens;  /* largest T of one eigen_attn_prefill call (sizes its scratch); 0 = none */
  const int32_t* r_k;          /* HOST [H]: rank of U^K per head, 1..d_head                           */
  const int32_t* r_v;          /* HOST [H] or NULL (= r_k): rank of U^V per head                      */
  const float* U_k;            /* HOST fp32, heads back to back; head h is row-major d_head x r_k[h], */
  const float* U_v;            /*   columns = basis vectors u_1..u_r (Section 4.1)                    */
  uint32_t flags;
} ea_desc;

/* Cache rows are padded to rp = 8*ceil(r/8) elements; padding columns hold zeros. */

/* Sizes of the two device buffers the caller must provide for this layer.  Pure host arithmetic. */
ea_status eigen_attn_cache_bytes(const ea_desc* desc, size_t* cache_bytes, size_t* workspace_bytes);

/* Builds a handle: validates desc, pads and uploads the bases into the workspace, fills the cache
 * with zeros (rows that no call has written must hold finite values) and sets len = 0.  Synchronises
 * `cuda_stream` before returning; desc's host arrays are not retained.
 * d_cache and d_workspace must be 256-byte aligned and stay valid for the life of the handle. */
ea_status eigen_attn_create(const ea_desc* desc, void* d_cache, size_t cache_bytes,
                            void* d_workspace, size_t workspace_bytes,
                            void* cuda_stream, eigen_attn_t* out);

/* Frees host memory only.  NULL is allowed. */
void eigen_attn_destroy(eigen_attn_t h);

/* Section 2 (generation phase) + Eq. 6: project T new rows per sequence and write them at rows
 * len..len+T-1 of the rank-r cache; then len += T.  d_k, d_v: [B][T][H][d_head].
 * flags: EA_KV_PREPROJECTED. */
ea_status eigen_attn_append_kv(eigen_attn_t h, const void* d_k, const void* d_v, int32_t T,
                               int64_t stride_b, int64_t stride_t, uint32_t flags, void* cuda_stream);

/* Eq. 3 in the rank-r space of Eq. 7: one query per sequence against rows [0, len).  Call it after
 * the append of the same token (the new token attends to itself).  d_q, d_out: [B][1][H][d_head]
 * with batch strides `stride_b_q`, `stride_b_out`.  flags: EA_Q_PREPROJECTED, EA_OUT_LOWRANK.
 * len == 0 -> EA_ERR_SHAPE. */
ea_status eigen_attn_decode(eigen_attn_t h, const void* d_q, int64_t stride_b_q, void* d_out,
                            int64_t stride_b_out, uint32_t flags, void* cuda_stream);

/* (No counterpart in the paper: an engineering variant of eigen_attn_decode.)
 * Same result as eigen_attn_decode, but the split-KV partial results (per-piece max, sum and
 * un-normalised o') are kept in an array built into the library image instead of the workspace.
 * It is meant for callers that must not obtain device memory while they run -- e.g. a plugin inside
 * an inference engine whose memory plan is frozen, a real-time loop where cudaMalloc's device-wide
 * synchronisation is unacceptable, or a process whose memory pool is already handed out in full --
 * and that therefore cannot size a partials area for a plan they do not know in advance.
 *   - Only the partials move.  The call still reads the head table and the bases in the workspace given
 *     at create and, with EA_OPT_DECODE_FUSED = 1 (the default), counts arrivals in that workspace's
 *     per-unit counters and reports through its status word, exactly as eigen_attn_decode does.
 *   - Limit: (batch * n_heads + decode CTAs) * (4 + widest rp_v) <= 270336 floats (2048 slots of 132
 *     floats, 1.03 MiB, resident on every GPU that loads the library until the process exits).
 *     Larger layers get EA_ERR_CAPACITY and a message; use eigen_attn_decode for them.
 *   - Every call asks the CUDA runtime for the array's device address on the current device (a lookup,
 *     no allocation; correct again after a cudaDeviceReset).  The first call on a device also makes the
 *     runtime load the library image there: make that first call outside any stream capture.  The call
 *     itself never calls cudaMalloc/cudaFree or any allocating routine.
 *   - All handles and all calls on a device share the one array, and it keeps whatever the previous
 *     call left.  Nothing in it has to start at zero: every slot the combine step reads is written
 *     earlier in the same call.  Two calls that may overlap on the GPU (different streams, or several
 *     host threads) race on the array and give undefined results; serialise them.  A decode and a
 *     decode_static of the SAME handle that overlap also race on the handle's arrival counters. */
ea_status eigen_attn_decode_static(eigen_attn_t h, const void* d_q, int64_t stride_b_q, void* d_out,
                                   int64_t stride_b_out, uint32_t flags, void* cuda_stream);

/* eigen_attn_append_kv with T = 1 followed by eigen_attn_decode (one generated token), fused into a
 * single launch when the cache already holds at least one row.
 * d_k and d_v share the batch stride `stride_b_kv`.  flags: EA_Q_PREPROJECTED, EA_KV_PREPROJECTED (d_k, d_v are the
 * packed rank-space rows [B][1][sum rp_k] and [B][1][sum rp_v]; their stride argument is ignored), EA_OUT_LOWRANK.
 * With all three the call is the attention core of a layer whose weights carry the bases (Eq. 8): no
 * multiplication by U remains in it. */
ea_status eigen_attn_decode_step(eigen_attn_t h, const void* d_q, int64_t stride_b_q,
                                 const void* d_k, const void* d_v, int64_t stride_b_kv,
                                 void* d_out, int64_t stride_b_out, uint32_t flags, void* cuda_stream);

/* The same step for HOST tensors (contiguous [B][1][H][d_head], ideally pinned): copies q, k, v to a
 * staging area of the workspace, runs the step, copies the result back and synchronises the stream.
 * When h_k == h_q + bytes and h_v == h_k + bytes (bytes = size of one of the tensors) the three travel as one copy. */
ea_status eigen_attn_decode_step_host(eigen_attn_t h, const void* h_q, const void* h_k, const void* h_v,
                                      void* h_out, uint32_t flags, void* cuda_stream);

/* Section 2 (prefill phase) with Eq. 7 and a causal mask: append T rows (as eigen_attn_append_kv) and
 * compute the attention output of the T queries, query t over rows [0, len0 + t] where len0 is the
 * length before the call.  T <= max_prefill_tokens.  d_q, d_k, d_v: [B][T][H][d_head] sharing
 * (stride_b, stride_t); d_out: [B][T][H][d_head] with its own strides.  flags: EA_OUT_LOWRANK; EA_Q_PREPROJECTED
 * (d_q is the packed [B][T][sum rp_k]); EA_KV_PREPROJECTED (d_k, d_v are the packed [B][T][sum rp_k], [B][T][sum rp_v]).
 * With either input flag the rows are copied, not multiplied (Eq. 8: the weights carry the bases); a tensor left
 * d_head-wide in such a call is projected on the CUDA cores. */
ea_status eigen_attn_prefill(eigen_attn_t h, const void* d_q, const void* d_k, const void* d_v,
                             int32_t T, int64_t stride_b, int64_t stride_t, void* d_out,
                             int64_t out_stride_b, int64_t out_stride_t,
                             uint32_t flags, void* cuda_stream);

/* Section 5.1 (MPT models use ALiBi; the paper prints no formula, this is the published bias): from the
 * next call on, the score of the query at position pos against cached row j of head i gets
 * -slopes[i] * (pos - j) before the softmax, pos = len - 1 in a decode call (after the new row is
 * appended) and len0 + t for prompt token t.  slopes: HOST [H], each finite and >= 0; NULL or all
 * zeros switches the bias off (the default).  Copies into the workspace and synchronises `cuda_stream`;
 * calls still in flight on other streams must have finished.  Every decode and prefill kernel carries the bias. */
ea_status eigen_attn_set_alibi(eigen_attn_t h, const float* slopes, void* cuda_stream);

/* Grouped-query attention (the Llama-2-70b / Llama-3 models of Section 5.1): the layer's n_heads are the K/V
 * heads; each has `group` query heads, query head hq = kv_head * group + i, which all attend over that K/V
 * head's rank-r rows with its U^K and are lifted with its U^V (Eq. 7 per query head).  d_q and d_out:
 * [B][1][n_heads * group][d_head], batch strides in elements.  One pass over the cache serves the whole
 * group.  1 <= group <= 16; bf16 layers with d_head % 16 == 0 and no ALiBi bias set (EA_ERR_UNSUPPORTED
 * otherwise).  With a rotary embedding set (the Llama models: Section 4.3 per query head) the keys of a tile are
 * lifted and turned once for the whole group and scored on the tensor cores (fp16 operand tiles: turned keys and
 * scaled queries must stay below 65504); where the tiles do not fit shared memory (r_k above 96 at d_head 128) or a
 * page table is set, every query head is served as its own unit of the multi-head rotary kernel.  Without a rotary
 * embedding a page table is followed where every padded key rank is a multiple of 16 and d_head <= 128 (the
 * warp-level kernel, see EA_OPT_GQA_IMPL; EA_ERR_UNSUPPORTED otherwise).  The partials of batch x n_heads x group x
 * splits must fit the workspace (EA_ERR_CAPACITY).  Attends over the rows the cache holds: append the new token's
 * rows first. */
ea_status eigen_attn_decode_gqa(eigen_attn_t h, const void* d_q, int64_t stride_b_q, int32_t group, void* d_out,
                                int64_t stride_b_out, void* cuda_stream);

/* Section 4.3 + Fig. 6(b) (models with rotary position embedding): from the next call on, decode keeps the
 * query full rank, takes every cached low-dimensional key back to d_head dimensions through (U^K)^T, rotates
 * it by its position (row j of the cache = position j) and the query by position len - 1, and scores them
 * with 1/sqrt(d_head); the value side is unchanged.  Pair i is turned by pos * base^(-2i/d_head); pairs are
 * (i, i + d_head/2), or (2i, 2i+1) with interleaved != 0.  d_q must then be the un-rotated [B][1][H][d_head]
 * query (EA_Q_PREPROJECTED is rejected) and the cache must hold projections of un-rotated keys, as
 * eigen_attn_append_kv writes them.  The paper shares one U^K among the heads of a layer; here that is the
 * special case of equal U_k[h].  base == 0 switches back.  bf16 layers with d_head % 16 == 0 only
 * (EA_ERR_UNSUPPORTED otherwise).  eigen_attn_prefill follows the same reading for a prompt (query t at position
 * len0 + t, the cache filled with projections of the un-rotated keys).  A layer created with EA_ROPE_PROMPT_SCRATCH
 * runs it on the tensor cores while the rows cached after the call fit max_prefill_tokens (the rotated queries and
 * the lifted, rotated keys of those rows are written to the workspace once per call, then the prompt's causal
 * product runs over d_head-wide rows); otherwise, and for later chunks of a longer prompt, a CUDA-core kernel does
 * the same arithmetic tile by tile (two orders of magnitude slower).  eigen_attn_decode_static returns
 * EA_ERR_UNSUPPORTED while a rotary embedding is set.  Synchronises `cuda_stream`. */
ea_status eigen_attn_set_rope(eigen_attn_t h, double base, int32_t interleaved, void* cuda_stream);

/* Section 5.3 ("Eigen Attention with Quantization") and Table 8: a quantised copy of the rank-r cache.
 * Integer codes of `bits` bits with one half-precision scale per group of `group` numbers (the storage cost
 * behind every size printed in Table 8: bits + 16/group bits per element).  Keys are grouped per channel
 * (a group = `group` consecutive tokens of one channel of one head), values per token (a group = `group`
 * consecutive channels of one token's row; the last group of a row may be shorter).  Codes are symmetric:
 *     s = half(min(max|x| / (2^(bits-1) - 1), 65504)),  c = clip(rint(x / s)),  x^ = c * s ,
 * x being the stored 16-bit row, the two divisions IEEE single precision, rint to nearest even.  Rows that do
 * not fill a block of `group` tokens yet stay in the 16-bit cache and are attended from there.
 * Built: bits in {3, 4} (every Eigen Attention row of Table 8), group in {16, 32, 64, 128}, bf16 layers
 * (EA_ERR_UNSUPPORTED otherwise).
 *
 * quant_bytes:  size of the caller's quantised buffer for this layer (host arithmetic).
 * quant_attach: hands the library that DEVICE buffer (256-byte aligned, >= quant_bytes; owned by the caller, as
 *               the cache is) and writes the per-head table at its start; no row is quantised yet.  NULL
 *               detaches.  Synchronises `cuda_stream`.
 * quant_sync:   quantises every complete block of `group` rows of the 16-bit cache that is not quantised yet
 *               (rows [quant_len, floor(len / group) * group)); asynchronous.  The 16-bit rows stay where they
 *               are; a caller that wants the memory back keeps only a window of the 16-bit cache.
 * decode_quant: eigen_attn_decode (same arguments, flags and ALiBi bias) over the codes of rows [0, quant_len)
 *               and the 16-bit rows [quant_len, len).  Not available with a rotary embedding.
 * quant_len:    rows currently held as codes (of the sequence that holds most, while lengths differ).
 *               eigen_attn_set_len below quant_len rounds it down to a whole block.
 * quant_lens:   the same per sequence: HOST array [batch].  While lengths differ (eigen_attn_set_lens) every sequence
 *               keeps its own count: set_lens keeps a sequence's codes of the complete blocks below its new length,
 *               quant_sync quantises each sequence's own complete blocks, decode_quant attends each sequence's own
 *               codes and 16-bit tail.
 * quant_layout: where head `head` lives in the buffer: byte offset of its slab [B][n_max / group][block_bytes],
 *               and inside a block the offsets of the key scales [rp_k] halves, the value codes and the value
 *               scales [ceil(rp_v / group)][group] halves; key codes sit at offset 0.
 *               3-bit: a code area is [rp / 8][group] units, unit j of row i holding channels 8j..8j+7 in 24 bits,
 *               channel 8j+k in bits 3k..3k+2 as c + 4, kept as two planes: the low 16 bits of all units
 *               ([rp / 8][group] halfwords), then their high 8 bits ([rp / 8][group] bytes).
 *               4-bit: units are 32-bit words of eight nibbles, each c + 8, ordered for the operand fragments of the
 *               integer tensor-core products of decode_quant.  Keys: word j of row i holds channels 8j..8j+7
 *               (channel 8j+k in bits 4k..4k+3) and sits at word j * group + ((i + 8 * (j mod 4)) mod group).
 *               Values: chunks of min(group, 32) rows; a chunk is [rp_v][rows / 8] words, word (c, o) holding rows
 *               8o..8o+7 of channel c (row 8o+k in bits 4k..4k+3).
 *               Keys therefore cost exactly bits + 16/group bits per (padded) element, the accounting behind
 *               Table 8; a value row pays one scale per started group of its rp_v channels. */
ea_status eigen_attn_quant_bytes(eigen_attn_t h, int32_t bits, int32_t group, size_t* bytes);
ea_status eigen_attn_quant_attach(eigen_attn_t h, int32_t bits, int32_t group, void* d_qcache, size_t bytes,
                                  void* cuda_stream);
ea_status eigen_attn_quant_sync(eigen_attn_t h, void* cuda_stream);
ea_status eigen_attn_decode_quant(eigen_attn_t h, const void* d_q, int64_t stride_b_q, void* d_out,
                                  int64_t stride_b_out, uint32_t flags, void* cuda_stream);
ea_status eigen_attn_quant_len(eigen_attn_t h, int32_t* qlen);
ea_status eigen_attn_quant_lens(eigen_attn_t h, int32_t* qlens);
ea_status eigen_attn_quant_layout(eigen_attn_t h, int32_t head, size_t* slab_offset, size_t* block_bytes,
                                  size_t* k_scale_offset, size_t* v_code_offset, size_t* v_scale_offset);

/* Current number of cached rows; set_len truncates or rewinds (0 <= len <= n_max), e.g. to re-run
 * a step at a fixed context length.  Rows beyond the previous length hold whatever was last written. */
ea_status eigen_attn_get_len(eigen_attn_t h, int32_t* len);
ea_status eigen_attn_set_len(eigen_attn_t h, int32_t len);

/* A batch of unequal lengths (the serving case: the prompts of a batch differ in length; the paper's generation
 * phase, Section 2 "LLM Inference", is stated per sequence, so each sequence attends its own n cached rows).
 * lens: HOST array [batch], 0 <= lens[b] <= n_max; sequence b then holds rows [0, lens[b]) of its slabs, whatever
 * was written there before (a prompt batch padded to a common T and prefilled keeps its first lens[b] rows).
 * eigen_attn_get_len reports the longest sequence.  Afterwards eigen_attn_append_kv and eigen_attn_decode_step
 * add rows behind each sequence's own end, eigen_attn_decode / _decode_step / _decode_static / _decode_gqa attend each
 * sequence's own rows (ALiBi positions count from the sequence's own end); decode needs lens[b] >= 1 for every
 * b (EA_ERR_SHAPE otherwise).  The split-KV work decomposition follows the true lengths, so a step costs what
 * the rows actually cached cost.  batch <= 1024.  eigen_attn_set_len returns to equal lengths.
 * With a rotary embedding each sequence's query sits at its own last position.  With a quantised cache attached
 * every sequence keeps its own count of rows held as codes (eigen_attn_quant_lens).  eigen_attn_prefill places
 * the T new tokens of sequence b behind that sequence's own rows (token t at position lens[b] + t, attending over
 * the sequence's rows only; the projections then run on the CUDA cores).  The lengths are uploaded on the stream
 * (asynchronous; the array may be reused when the call returns), so the calls that follow must run on that
 * stream or be ordered after it. */
ea_status eigen_attn_set_lens(eigen_attn_t h, const int32_t* lens, void* cuda_stream);
ea_status eigen_attn_get_lens(eigen_attn_t h, int32_t* lens);

/* A paged cache (the paper's introduction lists paging among the systems-level ways to fit long contexts, and its
 * outlook names the serving frameworks built on it; the generation phase of Section 2 is stated on a sequence's
 * rows K, V wherever they are kept, so paging changes addresses and nothing else).
 * Each head's K' (and V') slab is viewed as one array of batch * n_max rows cut into physical pages of `page_rows`
 * rows (a power of two, at least 128: a page holds whole tiles, so a tile is still one bulk copy); page p is rows
 * [p * page_rows, (p + 1) * page_rows).  h_table: HOST array [batch][pages_per_seq]; logical row r of sequence b
 * lives in physical page h_table[b][r / page_rows] at offset r % page_rows, in every head's slabs.  -1 = not mapped;
 * mapped entries of a sequence come first, no physical page may appear twice (EA_ERR_INVALID_ARG).  A sequence can
 * then hold as many rows as its mapped pages, which may exceed n_max when others map fewer: calls that add rows
 * return EA_ERR_CAPACITY when a sequence's next row has no page.  Rows are not moved: after the call a sequence's
 * rows are whatever its pages hold (the identity table h_table[b][i] = b * (n_max / page_rows) + i keeps a
 * contiguous cache as it is, when page_rows divides n_max).  NULL returns to the contiguous layout.
 * Available for eigen_attn_append_kv, _decode, _decode_step(_host), _decode_static, _set_len(s), and
 * eigen_attn_prefill (which then runs on the CUDA cores), and with a rotary embedding for all of these and for
 * eigen_attn_decode_gqa when page_rows divides n_max (a page then lies inside one sequence's slab, which the tiled
 * copies of the rotary decode kernel need); not (EA_ERR_UNSUPPORTED) with a quantised cache, nor
 * eigen_attn_decode_gqa without a rotary embedding.  batch * pages_per_seq entries must fit the table area of the workspace
 * (batch * batch * n_max / 128 entries, at most 4 Mi).  Uploaded on the stream (asynchronous; the array may be reused
 * when the call returns): later calls must run on that stream or be ordered after it. */
ea_status eigen_attn_set_page_table(eigen_attn_t h, const int32_t* h_table, int32_t pages_per_seq, int32_t page_rows,
                                    void* cuda_stream);

/* Synchronises the stream and returns the device status word (EA_OK or EA_ERR_TIMEOUT), then clears it. */
ea_status eigen_attn_poll_status(eigen_attn_t h, void* cuda_stream);

/* Text of the last error of this handle (never NULL; valid until the next call on the handle). */
const char* eigen_attn_last_error(eigen_attn_t h);

/* Element offsets of each head inside the packed low-rank vectors used by the *_PREPROJECTED and
 * EA_OUT_LOWRANK flags: prefix sums of rp_k / rp_v.  offs arrays: HOST [H+1] (last = total width). */
ea_status eigen_attn_head_offsets(eigen_attn_t h, int32_t* offs_k, int32_t* offs_v);

/* Where head `head` lives in the cache buffer: byte offsets of its K' and V' slabs, each laid out
 * [B][n_max][rp] row-major in the cache dtype, and the padded widths. */
ea_status eigen_attn_cache_layout(eigen_attn_t h, int32_t head, size_t* k_offset, size_t* v_offset,
                                  int32_t* rp_k, int32_t* rp_v);

/* Tuning / instrumentation knobs (all optional). */
typedef enum {
  EA_OPT_DECODE_CTAS = 1,     /* CTAs of the split-KV decode kernel; 0 = one per SM                      */
  EA_OPT_DECODE_TILE_ROWS = 2,/* rows per shared-memory tile (multiple of 16, <= 128); 0 = automatic     */
  EA_OPT_DECODE_STAGES = 3,   /* depth of the shared-memory ring (2..12); 0 = as many as fit              */
  EA_OPT_PREFILL_IMPL = 4,    /* 0 = automatic, 1 = CUDA-core kernel, 2 = tcgen05 tensor-core kernels, 3 = the
                                 single-tile tcgen05 kernel (otherwise only used for ranks too wide for the
                                 warp-specialised one)                                                     */
  EA_OPT_DECODE_FUSED = 5,    /* 1 (default): a decode step is one launch (append row, attend, merge the
                                 splits, lift); 0: separate append / attention / merge launches           */
  EA_OPT_PREFILL_PROJECT = 6, /* tensor-core projections of prefill: 0 = automatic (the persistent kernel that
                                 streams token tiles by TMA when d_head % 64 == 0 and T >= 128), 1 = always
                                 one CTA per tile of 128 tokens, n >= 2 = the persistent kernel with at most
                                 n CTAs                                                                    */
  EA_OPT_DECODE_MIN_COPY_BYTES = 8, /* split-KV decode: heads whose K' or V' tile is smaller than this many bytes
                                 put up to four consecutive tiles into one ring slot, i.e. one bulk copy;
                                 -1 = the default (16 KiB), 0 = always one tile per slot                     */
  EA_OPT_GQA_IMPL = 9,        /* eigen_attn_decode_gqa without a rotary embedding: 0 = automatic (warp-level mma.sync
                                 products where every padded key rank is a multiple of 16 and d_head <= 128, else the
                                 tcgen05 kernel), 1 = always the tcgen05 kernel                              */
  EA_OPT_TEST_WAIT_GIVES_UP = 7 /* failure-path test hook.  1 arms it for the NEXT eigen_attn_decode /
                                 _decode_step / _decode_static launch only: one warp of one CTA treats its
                                 first wait for a tile as having exceeded the bound.  The launch then ends the
                                 way a real timeout ends it (the CTA stops computing, the producer waits for
                                 its copies in flight, the kernel returns), the call's output is undefined and
                                 eigen_attn_poll_status reports EA_ERR_TIMEOUT once.  Nothing hangs or faults. */
} ea_option;
ea_status eigen_attn_set_option(eigen_attn_t h, int32_t option, int64_t value);

/* Number of kernels this handle has launched since create. */
ea_status eigen_attn_launch_count(eigen_attn_t h, uint64_t* count);

/* If both are non-NULL cudaEvent_t handles, every later decode, decode_step or prefill call records
 * `start` immediately before and `stop` immediately after its attention kernel (the split-KV kernel, or
 * the causal prefill kernel) on the call's stream (NULL, NULL = off). */
ea_status eigen_attn_set_decode_events(eigen_attn_t h, void* start_event, void* stop_event);

/* Library version: major*10000 + minor*100 + patch. */
int32_t eigen_attn_version(void);

#ifdef __cplusplus
}
#endif
#endif  /* EIGEN_ATTN_H_ */
