// Internal declarations shared by the translation units of libeigenattn (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ea {

// One entry per head, resident in the workspace; every kernel reads it.
struct HeadInfo {
  int64_t k_off;      // byte offset of the head's K' slab [B][n_max][rp_k] in the cache
  int64_t v_off;      // byte offset of the head's V' slab [B][n_max][rp_v]
  int64_t w_prefix;   // sum over earlier heads of (rp_k + rp_v): decode work weight prefix
  int32_t r_k, r_v;   // ranks
  int32_t rp_k, rp_v; // ranks padded to a multiple of 8
  int32_t uk_off;     // float offset of U^K  (d_head x rp_k, row-major, zero padded) in the basis area
  int32_t uv_off;     // float offset of U^V  (d_head x rp_v)
  int32_t uvt_off;    // float offset of (U^V)^T (rp_v x d_head)
  int32_t lr_k_off;   // element offset of the head in packed rank-space K/Q vectors (prefix of rp_k)
  int32_t lr_v_off;   // same for V / O
  int32_t ukt16_off;  // float offset of the tensor-core image of (U^K)^T: bf16 high part then low part, each
  int32_t uvt16_off;  //   [rp16][d_head] in the canonical core-matrix order (rp16 = rank padded to 16); same for U^V
  int32_t uvl16_off;  // float offset of the lift image of U^V: bf16 high then low part, each [d_head][rv16] canonical
  float alibi_slope2;  // ALiBi slope of the head times log2(e); 0 = no position bias
  int32_t ukl16_off;   // float offset of the lift image of U^K (as uvl16_off, [d_head][rk16] canonical, high then low)
};

// Paged cache: where logical row `row` of sequence `b` lives in a head's slab, viewed as one array of
// batch * n_max rows cut into pages of `page_rows` rows (a power of two, at least 128).  table == NULL: the
// contiguous layout, sequence b at rows [b * n_max, (b + 1) * n_max).
struct PageMap {
  const int32_t* table;     // [B][width]: physical page of every logical page of a sequence (-1 = not mapped)
  int32_t width;            // logical pages per sequence
  int32_t shift;            // log2(page_rows)
};
#ifdef __CUDACC__
__device__ __forceinline__ int64_t physical_row(const PageMap& pm, int b, int n_max, int row) {
  if (pm.table == nullptr) return static_cast<int64_t>(b) * n_max + row;
  const int page = __ldg(pm.table + static_cast<int64_t>(b) * pm.width + (row >> pm.shift));
  return (static_cast<int64_t>(page) << pm.shift) + (row & ((1 << pm.shift) - 1));
}
#endif

constexpr int kDecodeConsumerWarps = 8;
// + one warpgroup whose first thread is the producer: register reallocation works on whole warpgroups, and the
// producer's group hands most of its registers to the consumers
constexpr int kDecodeThreads = (kDecodeConsumerWarps + 4) * 32;
constexpr int kMaxHeads = 256;
constexpr int kStatusTimeout = -6;
constexpr int kMaxRaggedBatch = 1024;   // largest batch that may hold sequences of unequal lengths

struct DecodeParams {
  const HeadInfo* heads;
  const float* basis;       // basis area of the workspace
  char* cache;
  const void* q;            // [B][1][H][d_head] or packed rank-space [B][sum rp_k]
  int64_t q_stride_b;       // elements
  const void* k_new;        // [B][1][H][d_head] new token to project, store at row n and attend; or NULL.
  const void* v_new;        //   With flag 0x4 the rows are already rank-space: packed [B][sum rp_k] and [B][sum rp_v]
  int64_t kv_stride_b;      // batch stride of k_new (and of v_new unless the rows are packed)
  int64_t v_stride_b;       // batch stride of v_new
  void* out;                // [B][1][H][d_head] or packed [B][sum rp_v]
  int64_t out_stride_b;
  float* partials;          // [(B*H + grid)][part_stride]: m, l, pad, pad, o'[rp_v]
  int* counters;            // [B*H] arrivals per unit (all zero between calls); NULL = separate combine launch
  int* status;
  const int32_t* deficit;   // [B]: sequence b holds n - deficit[b] rows (a batch of unequal lengths); NULL = all hold n
  int32_t part_stride;      // floats per partial slot (multiple of 4)
  int32_t B, H, d_head;
  int32_t n;                // cached rows of the longest sequence (the new token's row, if any, comes on top)
  int32_t n_max;
  int32_t tile_rows;        // rows per tile
  int32_t nt;               // tiles per unit = ceil(n / tile_rows)
  int32_t ring_bytes;       // shared memory of the tile ring; slots are sized per head inside the kernel
  int32_t inflight_bytes;   // target bytes of copies in flight per SM (sets the slot count per head)
  int32_t min_copy_bytes;   // a slot of a narrow head holds several tiles, so that one bulk copy moves about this much
  int32_t fixed_stages;     // > 0: use this many slots (if they fit) instead of the in-flight target
  int64_t nt_total;         // tiles of one head: B * nt, or the sum of the sequences' own tile counts
  int64_t w_total;          // nt_total * sum_h (rp_k + rp_v)
  float q_scale;            // log2(e) / sqrt(d_head)
  uint32_t flags;
  int32_t give_up_once;     // test hook: warp 0 of CTA 0 reports its first wait for a tile as run out
  PageMap pages;            // paged cache (tile_rows divides the page size, one tile per ring slot)
};

struct CombineParams {
  const HeadInfo* heads;
  const float* basis;
  const float* partials;
  void* out;                // [B][1][H][d_head] or packed [B][sum rp_v]
  int64_t out_stride_b;
  int32_t part_stride;
  int32_t B, H, d_head;
  int32_t nt;
  int32_t grid;             // CTAs of the split-KV kernel that produced the partials
  const int32_t* deficit;   // as in DecodeParams (NULL: equal lengths)
  int32_t n, tile_rows;
  int64_t nt_total;
  int64_t w_total;
  uint32_t flags;
};

struct ProjectParams {       // project rows with U and scatter them into the cache
  const HeadInfo* heads;
  const float* basis;
  const void* k;            // [B][T][H][d_head]   (or packed rank-space rows)
  const void* v;
  char* cache;
  int64_t stride_b, stride_t;
  int32_t B, T, H, d_head;
  int32_t n_max;
  int32_t row0;             // first cache row to write (= len before the call)
  const int32_t* deficit;   // [B]: sequence b starts at row0 - deficit[b] (unequal lengths); NULL = all at row0
  int32_t lr_k_width, lr_v_width;   // widths of the packed rank-space rows (sum of rp_k / rp_v)
  uint32_t flags;
  PageMap pages;
};

struct QProjectParams {      // prefill: Q' = Q U^K into a scratch buffer (IO dtype)
  const HeadInfo* heads;
  const float* basis;
  const void* q;
  char* qp;                 // scratch base: head h at lr_k_off[h] * B * T elements, then [B][T][rp_k]
  int64_t stride_b, stride_t;
  int32_t B, T, H, d_head;
};

struct ProjectTcParams {     // prefill: Q', K', V' projections on the tensor cores (bf16 layers)
  const HeadInfo* heads;
  const float* basis;
  const void* q;            // [B][T][H][d_head], shared strides
  const void* k;
  const void* v;
  char* cache;
  char* qp;                 // Q' scratch (layout as in QProjectParams)
  int64_t stride_b, stride_t;
  int32_t B, T, H, d_head;
  int32_t n_max;
  int32_t row0;
  int* status;
};

struct PrefillParams {
  const HeadInfo* heads;
  const float* basis;
  const char* cache;
  const char* qp;           // Q' scratch (layout as in QProjectParams)
  void* out;                // [B][T][H][d_head] or packed [B][T][sum rp_v]
  int64_t out_stride_b, out_stride_t;
  int32_t B, T, H, d_head;
  int32_t n_max;
  int32_t len0;             // rows cached before the call (of the longest sequence)
  const int32_t* deficit;   // [B]: sequence b held len0 - deficit[b] rows before the call; NULL = all held len0
  int32_t max_rp;           // widest padded rank over heads and over K/V
  float scale_log2;         // log2(e) / sqrt(d_head)
  uint32_t flags;
  int* status;
  const void* tmaps;        // CUtensorMap[2 * H]: K' and V' slab of every head (warp-specialised kernel only)
  // Key side taken from elsewhere than the cache (the rotary prompt path: full-rank rotated queries against lifted,
  // rotated keys): every head's query and key rows are k_width wide, the queries sit at qp + h * k_width * B * T
  // elements, the key tiles come through tmaps_k (CUtensorMap[H]).  0 / NULL: the rank-r rows of the cache.
  int32_t k_width;
  const void* tmaps_k;
  PageMap pages;            // paged cache (CUDA-core kernel only)
  // RoPE variant (prefill_rope.cu): the full-rank, un-rotated queries and the rotation's frequencies
  const void* q_raw;        // [B][T][H][d_head]
  int64_t q_stride_b, q_stride_t;
  const double* inv_freq;   // [d_head/2]: base^(-2i/d_head)
  int32_t rope_interleaved; // pairs (2i, 2i+1) instead of (i, i + d_head/2)
  const float4* el_table;   // [32][128]: cos, cos, sin, sin of l phi for pairs 2k, 2k + 1 and row offset l
  void* krot;               // lifted, rotated keys [H][B][krot_rows][d_head] (16-bit), written by the preparing kernels
  int32_t krot_rows;
};

struct RopeDecodeParams {    // decode for models with rotary position embedding (bf16 layers)
  const HeadInfo* heads;
  const float* basis;
  const char* cache;
  const void* q;            // [B][1][H][d_head], full rank, not rotated
  int64_t q_stride_b;
  void* out;                // [B][1][H][d_head] or packed [B][sum rp_v]
  int64_t out_stride_b;
  float* partials;          // [B*H][splits][part_stride]: m, l, pad, pad, o'[rp_v]
  int* status;
  const double* inv_freq;   // [d_head/2]: base^(-2i/d_head)
  const float2* tile_step;  // [64]: cos, sin of -128 phi_i (one tile back along the cache)
  const float4* el_table;   // [32][128]: cos, cos, sin, sin of l phi for pairs 2k, 2k + 1 and row offset l
  const int32_t* deficit;   // [B]: sequence b holds n - deficit[b] rows; NULL = all hold n
  const void* tmaps;        // CUtensorMap[2 * H]: K' and V' slab of every head
  int32_t part_stride;
  int32_t B, H, d_head;
  int32_t n, n_max;
  int32_t nt;               // tiles of 128 rows per unit
  int32_t splits;           // CTAs per unit
  int32_t interleaved;      // pairs (2i, 2i+1) instead of (i, i + d_head/2)
  int32_t group;            // query heads per K/V head (1: every head has its own rows); q and out have H * group heads
  float q_scale;            // log2(e) / sqrt(d_head)
  uint32_t flags;
  PageMap pages;            // paged cache: a tile of 128 rows lies inside one page; pages lie inside one sequence's slab
};

struct GqaDecodeParams {     // grouped-query decode (bf16 layers): `group` query heads per K/V head
  const HeadInfo* heads;
  const float* basis;
  const char* cache;
  const void* q;            // [B][1][H * group][d_head]
  int64_t q_stride_b;
  void* out;                // [B][1][H * group][d_head]
  int64_t out_stride_b;
  float* partials;          // [B*H][splits][group][part_stride]: m, l, pad, pad, o'[rp_v]
  int* status;
  const void* tmaps;        // CUtensorMap[2 * H]: K' and V' slab of every K/V head
  const int32_t* deficit;   // [B]: sequence b holds n - deficit[b] rows; NULL = all hold n
  int32_t part_stride;
  int32_t B, H, d_head;
  int32_t n, n_max;
  int32_t nt;               // tiles of 128 rows per unit (of the longest sequence)
  int32_t splits;           // CTAs per unit
  int32_t group;            // 1..16
  float q_scale;            // log2(e) / sqrt(d_head)
  uint32_t flags;
  // with a rotary embedding (decode_gqa_rope_kernel): the constants of eigen_attn_set_rope
  const double* inv_freq;   // [d_head/2]
  const float2* tile_step;  // [64]: cos, sin of -128 phi_i
  const float4* el_table;   // [32][128]: cos, cos, sin, sin of l phi for pairs 2k, 2k + 1 and row offset l
  int32_t interleaved;
  PageMap pages;            // paged cache (decode_gqa_mma_kernel): a tile of 128 rows lies inside one page
};

// Quantised copy of the cache (Section 5.3 of the paper): per head a slab [B][blocks_max][block_bytes]; a block
// holds G consecutive rows of one sequence as integer codes and half-precision scales:
//   K codes  [rp_k/8][G] units     K scales [rp_k] halves        (one scale per channel and block)
//   V codes  [rp_v/8][G] units     V scales [nvg][G] halves      (one scale per row and G channels)
// 3-bit codes: a unit holds the eight channels 8j..8j+7 of one row in 24 bits, channel 8j+k in bits 3k..3k+2 as
// code + 4, stored as two planes, the low 16 bits of every unit ([rp/8][G] halfwords) followed by the high 8 bits of
// every unit ([rp/8][G] bytes): exactly 3 bits per element, and a warp's loads of either plane are consecutive.
// 4-bit codes: a unit is a 32-bit word of eight nibbles, each code + 8, laid out for the operand fragments of the
// integer tensor-core products.  Keys: word j of row i holds channels 8j..8j+7 (channel 8j+k in bits 4k..4k+3) and
// sits at j G + ((i + 8 (j mod 4)) mod G).  Values: chunks of min(G, 32) rows, a chunk [rp_v][rows/8] words, word
// (c, o) holding rows 8o..8o+7 of channel c (row 8o+k in bits 4k..4k+3).
struct QuantHead {
  int64_t slab_off;        // byte offset of the head's slab in the quantised buffer
  int32_t block_bytes;
  int32_t ks_off, vc_off, vs_off;   // byte offsets of K scales, V codes, V scales inside a block
  int32_t nvg;             // scale groups per value row = ceil(rp_v / G)
  int32_t pad_;
};

struct QuantParams {
  const HeadInfo* heads;
  const QuantHead* qheads;
  const float* basis;
  const char* cache;        // the 16-bit cache: source of the quantiser, and rows [nq, n) of a decode
  char* qcache;
  const void* q;            // decode: [B][1][H][d_head] or packed rank-space [B][sum rp_k]
  int64_t q_stride_b;
  void* out;
  int64_t out_stride_b;
  float* partials;          // [B*H][splits][part_stride]: m, l, pad, pad, o'[rp_v]
  int* status;
  const int32_t* deficit;   // [B]: sequence b holds n - deficit[b] rows (unequal lengths); NULL = all hold n
  const int32_t* qlens;     // [B]: rows of sequence b held as codes (unequal lengths); NULL = all hold nq
  int32_t part_stride;
  int32_t B, H, d_head;
  int32_t n, n_max;
  int32_t nq;               // rows held as codes (a multiple of group); the longest sequence's with unequal lengths
  int32_t group;            // G: 16, 32, 64 or 128
  int32_t bits;             // 3 or 4
  int32_t blocks_max;       // blocks per sequence the buffer holds = n_max / G
  int32_t nst;              // stages of 128 rows per unit = ceil(nq / 128)
  int32_t splits;           // CTAs per unit
  int32_t b0, b1;           // quantiser: blocks [b0, b1) of every sequence
  float q_scale;            // log2(e) / sqrt(d_head)
  uint32_t flags;
  uint32_t magic[4];        // float exponent patterns the decode kernel ORs nibbles into (set by its launcher)
};

// Launchers (each returns the CUDA error of its launch); `launches` is incremented per kernel.
cudaError_t launch_project_append(const ProjectParams& p, int dtype, cudaStream_t s, uint64_t* launches);
cudaError_t launch_decode(const DecodeParams& p, int dtype, int grid, size_t smem_bytes,
                          cudaStream_t s, uint64_t* launches);
cudaError_t launch_combine(const CombineParams& p, int dtype, cudaStream_t s, uint64_t* launches);
cudaError_t launch_q_project(const QProjectParams& p, int dtype, cudaStream_t s, uint64_t* launches);
// Q' rows that are already rank-space (packed [B][T][sum rp_k]) into the per-head layout of the Q' scratch.
cudaError_t launch_q_scatter(const QProjectParams& p, int lr_k_width, int dtype, cudaStream_t s, uint64_t* launches);
cudaError_t launch_prefill_simt(const PrefillParams& p, int dtype, cudaStream_t s, uint64_t* launches);
// the rotary prompt path on the tensor cores: rotated queries into p.qp, lifted rotated keys into p.krot
cudaError_t launch_rope_prompt_prepare(const PrefillParams& p, int max_rp_k, int sm_count, cudaStream_t s, uint64_t* launches);
cudaError_t launch_rope_lift_tc(const PrefillParams& p, int max_rp_k, int sm_count, cudaStream_t s, uint64_t* launches);
size_t rope_lift_tc_smem_bytes(int max_rp_k, int d_head);
cudaError_t launch_prefill_rope(const PrefillParams& p, int max_rp_k, int max_rp_v, cudaStream_t s, uint64_t* launches);
size_t decode_gqa_smem_bytes(int max_rp_k, int max_rp_v);
// grouped queries with a rotary embedding on the tensor cores; 0 bytes = the tiles do not fit
size_t decode_gqa_rope_smem_bytes(int max_rp_k, int d_head);
cudaError_t launch_decode_gqa_rope(const GqaDecodeParams& p, int max_rp_k, cudaStream_t s, uint64_t* launches);
cudaError_t launch_decode_gqa(const GqaDecodeParams& p, int max_rp_k, int max_rp_v, cudaStream_t s, uint64_t* launches);
// grouped queries with warp-level products (ranks that are multiples of 16, d_head <= 128); 0 bytes = does not fit
size_t decode_gqa_mma_smem_bytes(int max_rp_k, int max_rp_v);
cudaError_t launch_decode_gqa_mma(const GqaDecodeParams& p, int max_rp, int min_rp, cudaStream_t s, uint64_t* launches);
cudaError_t launch_gqa_combine(const GqaDecodeParams& p, cudaStream_t s, uint64_t* launches);
size_t decode_rope_smem_bytes(int max_rp_k, int max_rp_v, int d_head);
// bytes of the rotary constants a layer keeps: inverse frequencies (64 doubles), per-tile steps (64 float2),
// the row-offset table (32 x 128 float4)
constexpr size_t kRopeStepOffset = 64 * sizeof(double);
constexpr size_t kRopeTableOffset = kRopeStepOffset + 64 * 2 * sizeof(float);
constexpr size_t kRopeConstBytes = kRopeTableOffset + 32 * 128 * 4 * sizeof(float);
cudaError_t launch_decode_rope(const RopeDecodeParams& p, size_t smem, cudaStream_t s, uint64_t* launches);
int prefill_tc_ws_stages(int max_rp_k, int max_rp_v, int d_head, size_t* smem_bytes);   // 0 = does not fit
cudaError_t launch_prefill_tc_ws(const PrefillParams& p, int stages, size_t smem, bool alibi, cudaStream_t s,
                                 uint64_t* launches);
cudaError_t launch_project_tc(const ProjectTcParams& p, int max_rp, cudaStream_t s, uint64_t* launches);
// Persistent variant: maps_qkv = CUtensorMap[3] (host) of the q, k, v tensors; needs d_head % 64 == 0.
size_t project_tc_stream_smem(int max_rp, int d_head, int* stages);
cudaError_t launch_project_tc_stream(const ProjectTcParams& p, const void* maps_qkv, int max_rp, int sm_count,
                                     cudaStream_t s, uint64_t* launches);
cudaError_t launch_prefill_tc(const PrefillParams& p, int max_rp_k, int max_rp_v, cudaStream_t s,
                              uint64_t* launches);

cudaError_t launch_quantize_blocks(const QuantParams& p, cudaStream_t s, uint64_t* launches);
size_t decode_quant_smem_bytes(int max_stage_bytes, int max_rp_v);
cudaError_t launch_decode_quant(const QuantParams& p, int max_rp, int min_rp, size_t smem, cudaStream_t s,
                                uint64_t* launches);   // min_rp: narrowest padded rank over heads and K/V
// 4-bit codes: the integer tensor-core kernel
size_t decode_quant_mma_smem_bytes(int max_stage_bytes, int max_rp, int group);
cudaError_t launch_decode_quant_mma(const QuantParams& p, int max_rp, int min_rp, size_t smem, cudaStream_t s,
                                    uint64_t* launches);   // min_rp: narrowest padded rank over heads and K/V
cudaError_t launch_quant_combine(const QuantParams& p, cudaStream_t s, uint64_t* launches);

// Built-in scratch for eigen_attn_decode_static: device address and capacity (in floats) of the
// library's own partials array on the current device (queried from the runtime on every call).
constexpr size_t kStaticPartialFloats = 2048 * 132;
cudaError_t static_partials(float** ptr);

// Opts `kernel` in to `smem` bytes of dynamic shared memory on the CURRENT device.  The attribute belongs to
// the (kernel, device) pair, so every launcher keeps its own table `done` of the largest size set so far,
// indexed by device ordinal; a process that drives several GPUs configures each of them once.
constexpr int kMaxDevices = 64;
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, size_t smem, size_t (&done)[kMaxDevices]) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < kMaxDevices;
  if (tracked && smem <= done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e == cudaSuccess && tracked) done[dev] = smem;
  return e;
}

size_t decode_fixed_smem_bytes();         // shared memory the decode kernel needs besides the ring
cudaError_t decode_configure(int dtype);  // opt in to large dynamic shared memory (once per device)

}  // namespace ea
