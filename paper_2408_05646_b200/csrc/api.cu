// Host side of libeigenattn: the C ABI declared in include/eigen_attn.h.  Validates arguments,
// lays out the cache and the workspace, plans each launch and calls the kernels.  No device memory is
// allocated here: the cache and the workspace belong to the caller.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include <cuda.h>   // CUtensorMap and its enums only; the encoder is resolved at run time, libcuda is not linked

#include "../../include/eigen_attn.h"
#include "internal.h"

using ea::HeadInfo;

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxDecodeCtas = 1024;
constexpr int kPartialSlack = 4;     // the partials area holds this many times (batch x heads + kMaxDecodeCtas) slots
constexpr int kSmemLimit = 227 * 1024;
constexpr int kInFlightBytes = 120 * 1024;   // target bytes of bulk copies in flight per SM (decode)
constexpr int kMinCopyBytes = 16 * 1024;     // a bulk copy should move at least about this much (decode; narrow heads)

size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }
uint16_t bf16_rne(float x) {          // round to nearest even; inputs are finite
  uint32_t u;
  memcpy(&u, &x, 4);
  return static_cast<uint16_t>((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}
float bf16_to_float(uint16_t b) {
  const uint32_t u = static_cast<uint32_t>(b) << 16;
  float x;
  memcpy(&x, &u, 4);
  return x;
}
int ceil8(int r) { return (r + 7) / 8 * 8; }

struct Layout {
  std::vector<HeadInfo> heads;
  size_t cache_bytes = 0;
  // workspace
  size_t off_status = 0, off_heads = 0, off_basis = 0, off_partials = 0, off_counters = 0, off_staging = 0, off_qp = 0, off_tmaps = 0, off_rope = 0, off_deficit = 0, off_qlens = 0, off_pages = 0, off_krot = 0, off_tmaps_krot = 0;
  bool rope_scratch = false;   // the workspace holds the rotated queries and lifted keys of a prompt (EA_ROPE_PROMPT_SCRATCH)
  size_t page_entries = 0;   // capacity of the page-table area, in entries
  size_t basis_floats = 0, staging_each = 0, workspace_bytes = 0;
  int sum_rp_k = 0, sum_rp_v = 0, max_rp_k = 0, max_rp_v = 0, max_w = 0;
  int part_stride = 0;
  int64_t sum_w = 0;
  int es = 2;
};

ea_status check_desc(const ea_desc* d) {
  if (!d || !d->r_k) return EA_ERR_INVALID_ARG;
  if (d->dtype != EA_BF16 && d->dtype != EA_FP32) return EA_ERR_INVALID_ARG;
  if (d->batch < 1 || d->n_heads < 1 || d->n_heads > ea::kMaxHeads || d->n_max < 1) return EA_ERR_SHAPE;
  if (d->d_head < 8 || d->d_head > 128 || d->d_head % 8) return EA_ERR_SHAPE;
  if (d->max_prefill_tokens < 0 || d->max_prefill_tokens > d->n_max) return EA_ERR_SHAPE;
  for (int h = 0; h < d->n_heads; ++h) {
    const int rk = d->r_k[h], rv = d->r_v ? d->r_v[h] : d->r_k[h];
    if (rk < 1 || rk > d->d_head || rv < 1 || rv > d->d_head) return EA_ERR_SHAPE;
  }
  if (static_cast<int64_t>(d->batch) * d->n_max > (1ll << 40)) return EA_ERR_SHAPE;
  return EA_OK;
}

void make_layout(const ea_desc* d, Layout* L) {
  const int H = d->n_heads, dh = d->d_head;
  L->es = d->dtype == EA_BF16 ? 2 : 4;
  L->heads.resize(H);
  size_t cache = 0, basis = 0;
  int64_t wsum = 0;
  int lk = 0, lv = 0;
  for (int h = 0; h < H; ++h) {
    HeadInfo& hi = L->heads[h];
    memset(&hi, 0, sizeof(hi));
    hi.r_k = d->r_k[h];
    hi.r_v = d->r_v ? d->r_v[h] : d->r_k[h];
    hi.rp_k = ceil8(hi.r_k);
    hi.rp_v = ceil8(hi.r_v);
    hi.k_off = static_cast<int64_t>(cache);
    cache = align_up(cache + static_cast<size_t>(d->batch) * d->n_max * hi.rp_k * L->es);
    hi.v_off = static_cast<int64_t>(cache);
    cache = align_up(cache + static_cast<size_t>(d->batch) * d->n_max * hi.rp_v * L->es);
    hi.uk_off = static_cast<int32_t>(basis);  basis += static_cast<size_t>(dh) * hi.rp_k;
    hi.uv_off = static_cast<int32_t>(basis);  basis += static_cast<size_t>(dh) * hi.rp_v;
    hi.uvt_off = static_cast<int32_t>(basis); basis += static_cast<size_t>(dh) * hi.rp_v;
    if (dh % 16 == 0) {   // bf16 high/low images of U^T for the tensor-core projections (2 bytes per element)
      basis = (basis + 3) & ~static_cast<size_t>(3);
      hi.ukt16_off = static_cast<int32_t>(basis); basis += static_cast<size_t>((hi.rp_k + 15) & ~15) * dh;
      hi.uvt16_off = static_cast<int32_t>(basis); basis += static_cast<size_t>((hi.rp_v + 15) & ~15) * dh;
      hi.uvl16_off = static_cast<int32_t>(basis); basis += static_cast<size_t>((hi.rp_v + 15) & ~15) * dh;
      hi.ukl16_off = static_cast<int32_t>(basis); basis += static_cast<size_t>((hi.rp_k + 15) & ~15) * dh;
    }
    hi.lr_k_off = lk; lk += hi.rp_k;
    hi.lr_v_off = lv; lv += hi.rp_v;
    hi.w_prefix = wsum; wsum += hi.rp_k + hi.rp_v;
    if (hi.rp_k > L->max_rp_k) L->max_rp_k = hi.rp_k;
    if (hi.rp_v > L->max_rp_v) L->max_rp_v = hi.rp_v;
    if (hi.rp_k + hi.rp_v > L->max_w) L->max_w = hi.rp_k + hi.rp_v;
  }
  L->cache_bytes = cache;
  L->basis_floats = basis;
  L->sum_rp_k = lk; L->sum_rp_v = lv; L->sum_w = wsum;
  L->part_stride = 4 + L->max_rp_v;
  size_t off = 0;
  L->off_status = off;   off = align_up(off + 64);
  L->off_heads = off;    off = align_up(off + sizeof(HeadInfo) * H);
  L->off_basis = off;    off = align_up(off + basis * sizeof(float));
  L->off_partials = off;
  off = align_up(off + (static_cast<size_t>(d->batch) * H + kMaxDecodeCtas) * kPartialSlack * L->part_stride * sizeof(float));
  L->off_counters = off; off = align_up(off + static_cast<size_t>(d->batch) * H * sizeof(int));
  L->staging_each = align_up(static_cast<size_t>(d->batch) * H * dh * L->es);
  L->off_staging = off;  off += 4 * L->staging_each;
  // Q' of a prompt call; with EA_ROPE_PROMPT_SCRATCH at least the rotated full-rank queries, and behind them the
  // lifted, rotated keys of up to max_prefill_tokens rows per sequence ([H][B][max_prefill_tokens][d_head], 16-bit)
  const bool rope_scratch = (d->flags & EA_ROPE_PROMPT_SCRATCH) != 0 && d->dtype == EA_BF16 && dh % 16 == 0;
  size_t qp_bytes = static_cast<size_t>(d->batch) * d->max_prefill_tokens * lk * L->es;
  const size_t rot_bytes = static_cast<size_t>(d->batch) * d->max_prefill_tokens * H * dh * 2;
  if (rope_scratch && rot_bytes > qp_bytes) qp_bytes = rot_bytes;
  L->off_qp = off;       off = align_up(off + qp_bytes);
  L->off_krot = off;     off = align_up(off + (rope_scratch ? rot_bytes : 0));
  L->off_tmaps_krot = off; off = align_up(off + (rope_scratch ? static_cast<size_t>(H) * sizeof(CUtensorMap) : 0));
  L->rope_scratch = rope_scratch && d->max_prefill_tokens >= 1;
  L->off_rope = off;     off = align_up(off + ea::kRopeConstBytes);   // constants of the rotary embedding
  L->off_tmaps = off;    off = align_up(off + 2 * static_cast<size_t>(H) * sizeof(CUtensorMap));   // K', V' per head
  L->off_deficit = off;  off = align_up(off + static_cast<size_t>(d->batch) * sizeof(int32_t));   // unequal lengths
  L->off_qlens = off;    off = align_up(off + static_cast<size_t>(d->batch) * sizeof(int32_t));   // ... of the quantised copy
  // page table [batch][pages per sequence]: room for every sequence to map the whole pool of 128-row pages,
  // at most 4 Mi entries
  const size_t pool_pages = static_cast<size_t>(d->batch) * d->n_max / 128;
  L->page_entries = static_cast<size_t>(d->batch) * pool_pages;
  if (L->page_entries > (1u << 22)) L->page_entries = 1u << 22;
  L->off_pages = off;    off = align_up(off + L->page_entries * sizeof(int32_t));
  L->workspace_bytes = off;
}

// Tensor maps of the K' and V' slabs of every head for the prefill kernel's TMA loads: a 3-D view
// {rank (inner), n_max rows, batch} of bf16, box = 64 elements x 64 rows with the 128-byte swizzle.  Elements
// past the rank and rows past n_max read as zero.  Returns false when the driver's encoder is unavailable or
// rejects a shape; the caller then keeps the prefill kernels that do not use TMA.
bool encode_tensor_maps(const ea_desc* d, const Layout& L, char* cache, std::vector<CUtensorMap>* maps) {
  using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return false;
  const EncodeFn encode = reinterpret_cast<EncodeFn>(fn);
  maps->resize(2 * static_cast<size_t>(d->n_heads));
  for (int h = 0; h < d->n_heads; ++h)
    for (int which = 0; which < 2; ++which) {
      const HeadInfo& hi = L.heads[h];
      const cuuint64_t rp = which ? hi.rp_v : hi.rp_k;
      const cuuint64_t dims[3] = {rp, static_cast<cuuint64_t>(d->n_max), static_cast<cuuint64_t>(d->batch)};
      const cuuint64_t strides[2] = {rp * 2, static_cast<cuuint64_t>(d->n_max) * rp * 2};
      const cuuint32_t box[3] = {64, 64, 1};
      const cuuint32_t estr[3] = {1, 1, 1};
      void* base = cache + (which ? hi.v_off : hi.k_off);
      if (encode(&(*maps)[2 * h + which], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    }
  return true;
}

// Tensor maps of the lifted, rotated keys a prompt call of a layer with rotary embedding keeps in the workspace:
// per head a 3-D view {d_head (inner), max_prefill_tokens rows, batch} of bf16, boxes as for the cache slabs.
bool encode_krot_maps(const ea_desc* d, char* base, std::vector<CUtensorMap>* maps) {
  using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess)
    return false;
  const EncodeFn encode = reinterpret_cast<EncodeFn>(fn);
  const cuuint64_t dh = d->d_head, R = d->max_prefill_tokens, B = d->batch;
  maps->resize(d->n_heads);
  for (int h = 0; h < d->n_heads; ++h) {
    const cuuint64_t dims[3] = {dh, R, B};
    const cuuint64_t strides[2] = {dh * 2, R * dh * 2};
    const cuuint32_t box[3] = {64, 64, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (encode(&(*maps)[h], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base + static_cast<size_t>(h) * B * R * dh * 2, dims, strides,
               box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  }
  return true;
}

// Tensor maps of the q, k, v tensors of one prefill call for the streaming projection kernel: a 3-D view
// {n_heads * d_head (inner), T tokens, batch} of bf16, box = 64 elements x 128 tokens with the 128-byte
// swizzle; tokens past T read as zero.  Encoded on the host per call (the pointers are the caller's).
bool encode_input_maps(const void* const ptrs[3], int H, int d_head, int T, int B, int64_t stride_b, int64_t stride_t,
                       CUtensorMap maps[3]) {
  using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return false;
    encode = reinterpret_cast<EncodeFn>(fn);
  }
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(H) * d_head, static_cast<cuuint64_t>(T), static_cast<cuuint64_t>(B)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(stride_t) * 2, static_cast<cuuint64_t>(stride_b) * 2};
  const cuuint32_t box[3] = {64, 128, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  for (int i = 0; i < 3; ++i)
    if (encode(&maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptrs[i]), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return false;
  return true;
}

}  // namespace

struct eigen_attn {
  ea_desc desc;           // the host array pointers are cleared after create
  Layout L;
  char* cache = nullptr;
  char* ws = nullptr;
  int32_t len = 0;        // cached rows of the longest sequence
  std::vector<int32_t> deficit;   // [B]: sequence b holds len - deficit[b] rows (eigen_attn_set_lens)
  int32_t max_deficit = 0;        // > 0: the batch has unequal lengths and the workspace holds `deficit`
  int sm_count = 148;
  bool tmaps_ok = false;  // the workspace holds tensor maps of the cache slabs
  bool krot_ok = false;   // ... and the scratch + tensor maps of a rotary layer's prompt on the tensor cores
  bool alibi = false;     // some head has a non-zero ALiBi slope
  bool rope = false;      // decode follows Section 4.3 (rotary position embedding)
  int rope_interleaved = 0;
  int64_t opt_ctas = 0, opt_tile_rows = 0, opt_stages = 0, opt_prefill = 0, opt_fused = 1, opt_project = 0;
  // paged cache (eigen_attn_set_page_table)
  bool paged = false;
  int page_shift = 0, page_width = 0;
  std::vector<int32_t> page_cap;      // [B]: rows sequence b can hold = leading mapped pages * page_rows
  int64_t opt_min_copy = -1;  // EA_OPT_DECODE_MIN_COPY_BYTES; < 0 = the built-in default
  int64_t opt_give_up = 0;   // EA_OPT_TEST_WAIT_GIVES_UP: armed for the next split-KV decode launch
  int64_t opt_gqa_impl = 0;  // EA_OPT_GQA_IMPL
  uint64_t launches = 0;
  cudaEvent_t ev_start = nullptr, ev_stop = nullptr;
  // quantised copy of the cache (Section 5.3), attached by the caller
  char* qcache = nullptr;
  int q_group = 0;
  int q_bits = 0;
  int32_t qlen = 0;       // rows held as codes (a multiple of q_group); with unequal lengths the largest of `qlens`
  std::vector<int32_t> qlens;   // [B]: rows of each sequence held as codes, kept (and uploaded) while lengths differ
  int q_max_stage_bytes = 0;
  std::vector<ea::QuantHead> qheads;
  char err[256];
};

namespace {

ea_status fail(eigen_attn_t h, ea_status st, const char* fmt, ...) {
  if (h) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(h->err, sizeof(h->err), fmt, ap);
    va_end(ap);
  }
  return st;
}
ea_status cuda_fail(eigen_attn_t h, cudaError_t e, const char* what) {
  return fail(h, EA_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

// Layout of the quantised buffer for group size G: the per-head table, then one slab per head.
size_t make_quant_layout(const eigen_attn* h, int bits, int G, std::vector<ea::QuantHead>* qheads, int* max_stage_bytes) {
  const int H = h->desc.n_heads;
  const int64_t blocks_max = h->desc.n_max / G;
  qheads->resize(H);
  size_t off = align_up(sizeof(ea::QuantHead) * H);
  int widest = 0;
  for (int i = 0; i < H; ++i) {
    const HeadInfo& hi = h->L.heads[i];
    ea::QuantHead& q = (*qheads)[i];
    memset(&q, 0, sizeof(q));
    q.nvg = (hi.rp_v + G - 1) / G;
    q.ks_off = G * hi.rp_k * bits / 8;           // a multiple of 16: G % 16 == 0, rp % 8 == 0
    q.vc_off = q.ks_off + 2 * hi.rp_k;
    q.vs_off = q.vc_off + G * hi.rp_v * bits / 8;
    q.block_bytes = q.vs_off + 2 * G * q.nvg;
    q.slab_off = static_cast<int64_t>(off);
    off = align_up(off + static_cast<size_t>(h->desc.batch) * blocks_max * q.block_bytes);
    const int stage = (128 / G) * q.block_bytes;
    if (stage > widest) widest = stage;
  }
  if (max_stage_bytes) *max_stage_bytes = widest;
  return off;
}

ea_status check_quant_args(eigen_attn_t h, const char* who, int32_t bits, int32_t group) {
  if (bits != 3 && bits != 4) return fail(h, EA_ERR_UNSUPPORTED, "%s: %d-bit codes (3 and 4 are built)", who, bits);
  if (group != 16 && group != 32 && group != 64 && group != 128)
    return fail(h, EA_ERR_UNSUPPORTED, "%s: group %d (16, 32, 64 or 128)", who, group);
  if (h->desc.dtype != EA_BF16) return fail(h, EA_ERR_UNSUPPORTED, "%s: needs a bf16 layer", who);
  if (h->desc.n_max < group) return fail(h, EA_ERR_SHAPE, "%s: n_max %d holds no group of %d rows", who, h->desc.n_max, group);
  return EA_OK;
}

const HeadInfo* dev_heads(eigen_attn_t h) { return reinterpret_cast<const HeadInfo*>(h->ws + h->L.off_heads); }
const float* dev_basis(eigen_attn_t h) { return reinterpret_cast<const float*>(h->ws + h->L.off_basis); }
int* dev_status(eigen_attn_t h) { return reinterpret_cast<int*>(h->ws + h->L.off_status); }
ea::PageMap dev_pages(eigen_attn_t h) {
  ea::PageMap pm{};
  if (h->paged) {
    pm.table = reinterpret_cast<const int32_t*>(h->ws + h->L.off_pages);
    pm.width = h->page_width;
    pm.shift = h->page_shift;
  }
  return pm;
}
// Rows sequence b can hold: n_max, or what its page table maps.
int64_t capacity_of(const eigen_attn* h, int b) { return h->paged ? h->page_cap[b] : h->desc.n_max; }
// True if every sequence has room for T more rows; *bad = a sequence that has not.
bool room_for(const eigen_attn* h, int64_t T, int* bad) {
  for (int b = 0; b < h->desc.batch; ++b) {
    const int64_t have = h->len - (h->max_deficit > 0 ? h->deficit[b] : 0);
    if (have + T > capacity_of(h, b)) { *bad = b; return false; }
  }
  return true;
}
const int32_t* dev_deficit(eigen_attn_t h) {
  return h->max_deficit > 0 ? reinterpret_cast<const int32_t*>(h->ws + h->L.off_deficit) : nullptr;
}
int* dev_counters(eigen_attn_t h) { return reinterpret_cast<int*>(h->ws + h->L.off_counters); }

ea_status do_append(eigen_attn_t h, const void* d_k, const void* d_v, int32_t T, int64_t stride_b,
                    int64_t stride_t, uint32_t flags, cudaStream_t s) {
  if (!d_k || !d_v) return fail(h, EA_ERR_INVALID_ARG, "append_kv: NULL k or v");
  if (flags & ~EA_KV_PREPROJECTED) return fail(h, EA_ERR_INVALID_ARG, "append_kv: unknown flag 0x%x", flags);
  if (T < 1) return fail(h, EA_ERR_SHAPE, "append_kv: T = %d", T);
  int bad = 0;
  if (!room_for(h, T, &bad))
    return fail(h, EA_ERR_CAPACITY, "append_kv: T %d more rows exceed the capacity of sequence %d (%lld rows)", T, bad,
                static_cast<long long>(capacity_of(h, bad)));
  ea::ProjectParams p{};
  p.heads = dev_heads(h); p.basis = dev_basis(h); p.k = d_k; p.v = d_v; p.cache = h->cache;
  p.stride_b = stride_b; p.stride_t = stride_t;
  p.B = h->desc.batch; p.T = T; p.H = h->desc.n_heads; p.d_head = h->desc.d_head;
  p.n_max = h->desc.n_max; p.row0 = h->len; p.deficit = dev_deficit(h); p.flags = flags;
  p.lr_k_width = h->L.sum_rp_k; p.lr_v_width = h->L.sum_rp_v;
  p.pages = dev_pages(h);
  const cudaError_t e = ea::launch_project_append(p, h->desc.dtype, s, &h->launches);
  if (e != cudaSuccess) return cuda_fail(h, e, "append_kv launch");
  h->len += T;
  return EA_OK;
}

struct DecodePlan {
  ea::DecodeParams p;
  ea::CombineParams c;
  int grid = 0;
  size_t smem = 0;
};

// Validates a decode request and plans its two launches; `partials` is where the split-KV pieces go.
// With k_new/v_new the cache holds len rows and the new token's row is projected, stored at row len and
// attended inside the same launch; otherwise the len cached rows are attended.
ea_status plan_decode(eigen_attn_t h, const char* who, const void* d_q, int64_t stride_b_q, void* d_out,
                      int64_t stride_b_out, uint32_t flags, float* partials, const void* k_new,
                      const void* v_new, int64_t kv_stride_b, DecodePlan* plan) {
  if (!d_q || !d_out) return fail(h, EA_ERR_INVALID_ARG, "%s: NULL q or out", who);
  if (flags & ~(EA_Q_PREPROJECTED | EA_OUT_LOWRANK | (k_new ? EA_KV_PREPROJECTED : 0u)))
    return fail(h, EA_ERR_INVALID_ARG, "%s: unknown flag 0x%x", who, flags);
  if (h->len < 1) return fail(h, EA_ERR_SHAPE, "%s: the cache is empty", who);
  if (!k_new && h->len - h->max_deficit < 1)
    return fail(h, EA_ERR_SHAPE, "%s: a sequence of the batch has no cached row", who);
  const Layout& L = h->L;
  const int B = h->desc.batch, H = h->desc.n_heads, n = h->len;
  const int fixed = static_cast<int>(ea::decode_fixed_smem_bytes());
  const int sms = h->opt_ctas > 0 ? static_cast<int>(h->opt_ctas) : h->sm_count;

  // paged cache: one tile per ring slot (consecutive tiles need not be neighbours in memory)
  const int min_copy = h->paged ? 0 : h->opt_min_copy >= 0 ? static_cast<int>(h->opt_min_copy) : kMinCopyBytes;
  if (h->paged && (h->opt_tile_rows & (h->opt_tile_rows - 1)) != 0)
    return fail(h, EA_ERR_UNSUPPORTED, "%s: with a page table DECODE_TILE_ROWS must be a power of two", who);
  // rows per tile: 128 unless the context is short (keep a few tiles per CTA) or a stage would be too big
  int tile_rows = 128;
  if (h->opt_tile_rows > 0) {
    tile_rows = static_cast<int>(h->opt_tile_rows);
  } else {
    while (tile_rows > 16 && static_cast<int64_t>(B) * H * ((n + tile_rows - 1) / tile_rows) < 4ll * sms)
      tile_rows >>= 1;
  }
  // The ring: slots are sized per head inside the kernel.  Measured on B200: about 120 KB of copies in
  // flight per SM saturates HBM and deeper rings lose bandwidth again (more concurrent DRAM streams), so
  // the ring holds max(3 slots, 120 KB) of the widest head, as far as shared memory allows.
  int ring_bytes = 0;
  for (;;) {
    const int widest = static_cast<int>(align_up(static_cast<size_t>(tile_rows) * L.max_w * L.es, 128));
    const int avail = kSmemLimit - fixed;
    if (3 * widest <= avail || tile_rows <= 16) {
      int want = 3 * widest > kInFlightBytes + widest ? 3 * widest : kInFlightBytes + widest;
      // narrow heads put several tiles into a slot (one copy of about min_copy bytes): room for three such slots
      for (const HeadInfo& hi : L.heads) {
        const int kb = tile_rows * hi.rp_k * L.es, vb = tile_rows * hi.rp_v * L.es;
        const int narrow = kb < vb ? kb : vb;
        int tps = (min_copy + narrow - 1) / narrow;
        if (tps > 4) tps = 4;
        const int slot = static_cast<int>(align_up(static_cast<size_t>(kb + vb) * tps, 128));
        if (3 * slot > want) want = 3 * slot;
      }
      if (h->opt_stages > 0) want = static_cast<int>(h->opt_stages) * widest;
      ring_bytes = want < avail ? want : avail;
      if (ring_bytes < widest)
        return fail(h, EA_ERR_UNSUPPORTED, "%s: a tile of %d rows does not fit in shared memory", who, tile_rows);
      break;
    }
    tile_rows >>= 1;
  }

  const int nt = (n + tile_rows - 1) / tile_rows;
  // Tiles of one head.  Unequal lengths: every sequence contributes its own tiles (at least one, so that some CTA
  // attends the new token of a sequence without rows), hence the CTA ranges follow the true lengths.
  int64_t nt_total = static_cast<int64_t>(nt) * B;
  if (h->max_deficit > 0) {
    nt_total = 0;
    for (int b = 0; b < B; ++b) {
      const int tiles = (n - h->deficit[b] + tile_rows - 1) / tile_rows;
      nt_total += tiles > 0 ? tiles : 1;
    }
  }
  const int64_t w_total = nt_total * L.sum_w;
  int grid = sms;
  const int64_t cap = w_total / L.max_w;          // every CTA must own at least one tile
  if (grid > cap) grid = static_cast<int>(cap);
  if (grid < 1) grid = 1;

  ea::DecodeParams& p = plan->p;
  p = ea::DecodeParams{};
  p.heads = dev_heads(h); p.basis = dev_basis(h); p.cache = h->cache;
  p.q = d_q; p.q_stride_b = (flags & EA_Q_PREPROJECTED) ? L.sum_rp_k : stride_b_q;
  p.k_new = k_new; p.v_new = v_new;
  p.kv_stride_b = (flags & EA_KV_PREPROJECTED) ? L.sum_rp_k : kv_stride_b;
  p.v_stride_b = (flags & EA_KV_PREPROJECTED) ? L.sum_rp_v : kv_stride_b;
  p.out = d_out; p.out_stride_b = (flags & EA_OUT_LOWRANK) ? L.sum_rp_v : stride_b_out;
  p.partials = partials;
  p.counters = h->opt_fused ? dev_counters(h) : nullptr;
  p.status = dev_status(h);
  p.deficit = dev_deficit(h);
  p.part_stride = L.part_stride;
  p.B = B; p.H = H; p.d_head = h->desc.d_head; p.n = n; p.n_max = h->desc.n_max;
  p.tile_rows = tile_rows; p.nt = nt; p.ring_bytes = ring_bytes; p.inflight_bytes = kInFlightBytes;
  p.fixed_stages = static_cast<int>(h->opt_stages);
  p.min_copy_bytes = min_copy > 0 ? min_copy : 1;
  p.nt_total = nt_total;
  p.w_total = w_total;
  p.q_scale = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(h->desc.d_head)));
  p.flags = flags;
  p.give_up_once = h->opt_give_up ? 1 : 0;
  p.pages = dev_pages(h);
  plan->grid = grid;
  plan->smem = static_cast<size_t>(fixed) + static_cast<size_t>(ring_bytes);

  ea::CombineParams& c = plan->c;
  c = ea::CombineParams{};
  c.heads = p.heads; c.basis = p.basis; c.partials = partials; c.out = d_out;
  c.out_stride_b = (flags & EA_OUT_LOWRANK) ? L.sum_rp_v : stride_b_out;
  c.part_stride = L.part_stride; c.B = B; c.H = H; c.d_head = h->desc.d_head; c.nt = nt; c.grid = grid;
  c.deficit = p.deficit; c.n = n; c.tile_rows = tile_rows; c.nt_total = nt_total;
  c.w_total = w_total; c.flags = flags;
  return EA_OK;
}

ea_status launch_plan(eigen_attn_t h, const char* who, const DecodePlan& plan, bool events, cudaStream_t s) {
  if (events && h->ev_start) cudaEventRecord(h->ev_start, s);
  cudaError_t e = ea::launch_decode(plan.p, h->desc.dtype, plan.grid, plan.smem, s, &h->launches);
  if (events && h->ev_stop) cudaEventRecord(h->ev_stop, s);
  h->opt_give_up = 0;                 // one launch only
  if (e != cudaSuccess) return cuda_fail(h, e, who);
  if (plan.p.counters == nullptr) {   // the merge + lift as its own launch
    e = ea::launch_combine(plan.c, h->desc.dtype, s, &h->launches);
    if (e != cudaSuccess) return cuda_fail(h, e, who);
  }
  return EA_OK;
}

// Section 4.3: decode for a layer with rotary position embedding.  Row j of the cache sits at position j, the
// query at position len - 1.
ea_status do_decode_rope(eigen_attn_t h, const void* d_q, int64_t stride_b, void* d_out, int64_t stride_b_out,
                         uint32_t flags, cudaStream_t s, int group = 1) {
  if (!d_q || !d_out) return fail(h, EA_ERR_INVALID_ARG, "decode: NULL q or out");
  if (h->paged && h->desc.n_max % (1 << h->page_shift) != 0)
    return fail(h, EA_ERR_UNSUPPORTED, "decode with rotary embedding and a page table: page_rows %d must divide n_max %d",
                1 << h->page_shift, h->desc.n_max);
  if (flags & ~EA_OUT_LOWRANK)
    return fail(h, EA_ERR_INVALID_ARG, "decode with rotary embedding: flag 0x%x (the query must be full rank)", flags);
  if (h->len < 1) return fail(h, EA_ERR_SHAPE, "decode: the cache is empty");
  if (h->len - h->max_deficit < 1) return fail(h, EA_ERR_SHAPE, "decode: a sequence of the batch has no cached row");
  const Layout& L = h->L;
  const int B = h->desc.batch, H = h->desc.n_heads, n = h->len;
  const size_t smem = ea::decode_rope_smem_bytes(L.max_rp_k, L.max_rp_v, h->desc.d_head);
  if (smem > static_cast<size_t>(kSmemLimit)) return fail(h, EA_ERR_UNSUPPORTED, "decode with rotary embedding: tiles do not fit");
  ea::RopeDecodeParams p{};
  p.heads = dev_heads(h); p.basis = dev_basis(h); p.cache = h->cache;
  p.q = d_q; p.q_stride_b = stride_b;
  p.out = d_out; p.out_stride_b = (flags & EA_OUT_LOWRANK) ? L.sum_rp_v : stride_b_out;
  p.partials = reinterpret_cast<float*>(h->ws + L.off_partials);
  p.status = dev_status(h);
  p.inv_freq = reinterpret_cast<const double*>(h->ws + L.off_rope);
  p.tile_step = reinterpret_cast<const float2*>(h->ws + L.off_rope + ea::kRopeStepOffset);
  p.el_table = reinterpret_cast<const float4*>(h->ws + L.off_rope + ea::kRopeTableOffset);
  p.tmaps = h->ws + L.off_tmaps;
  p.deficit = dev_deficit(h);
  p.part_stride = L.part_stride;
  p.B = B; p.H = H; p.d_head = h->desc.d_head; p.n = n; p.n_max = h->desc.n_max;
  p.nt = (n + 127) / 128;
  // CTAs per unit.  The CTAs run in waves of (SMs x CTAs per SM) and each one pays a start-up (the U^K image, the
  // rotation constants, the first tiles' way from memory) worth a few tiles: take the split count with the least
  // waves x (tiles + start-up), within the partials the workspace holds.
  const int ctas_per_sm = smem * 2 + 4096 <= static_cast<size_t>(228 * 1024) ? 2 : 1;
  const int64_t units = static_cast<int64_t>(B) * H * group;    // (sequence, query head) pairs
  int64_t cap = (static_cast<int64_t>(B) * H + kMaxDecodeCtas) * kPartialSlack / units;
  if (cap < 1) return fail(h, EA_ERR_CAPACITY, "decode with rotary embedding: batch x heads x group = %lld partials exceed the workspace",
                           static_cast<long long>(units));
  if (cap > p.nt) cap = p.nt;
  if (cap > 65535) cap = 65535;
  int64_t splits = 1;
  if (h->opt_ctas > 0) {
    splits = (h->opt_ctas + units - 1) / units;
    if (splits > cap) splits = cap;
  } else {
    const int64_t wave = static_cast<int64_t>(h->sm_count) * ctas_per_sm;
    int64_t best = INT64_MAX;
    for (int64_t s2 = 1; s2 <= cap && s2 <= 256; ++s2) {
      const int64_t cost = ((units * s2 + wave - 1) / wave) * ((p.nt + s2 - 1) / s2 + 6);
      if (cost < best) { best = cost; splits = s2; }
    }
  }
  p.splits = static_cast<int32_t>(splits);
  p.interleaved = h->rope_interleaved;
  p.group = group;
  p.q_scale = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(h->desc.d_head)));
  p.flags = flags;
  p.pages = dev_pages(h);
  if (h->ev_start) cudaEventRecord(h->ev_start, s);
  const cudaError_t e = ea::launch_decode_rope(p, smem, s, &h->launches);
  if (h->ev_stop) cudaEventRecord(h->ev_stop, s);
  if (e != cudaSuccess) return cuda_fail(h, e, "decode launch (rotary embedding)");
  return EA_OK;
}

ea_status do_decode(eigen_attn_t h, const void* d_q, int64_t stride_b, void* d_out, int64_t stride_b_out,
                    uint32_t flags, cudaStream_t s) {
  if (h->rope) return do_decode_rope(h, d_q, stride_b, d_out, stride_b_out, flags, s);
  DecodePlan plan;
  const ea_status st = plan_decode(h, "decode", d_q, stride_b, d_out, stride_b_out, flags,
                                   reinterpret_cast<float*>(h->ws + h->L.off_partials), nullptr, nullptr, 0,
                                   &plan);
  if (st != EA_OK) return st;
  return launch_plan(h, "decode launch", plan, true, s);
}

// One generated token.  Fused form: a single launch projects and stores the new row, attends over the
// cached rows plus that row, merges the splits and lifts.  It needs at least one cached row (the work
// decomposition is over cached rows); otherwise, or with fusion switched off, append then decode.
ea_status do_step(eigen_attn_t h, const void* d_q, int64_t stride_b_q, const void* d_k, const void* d_v,
                  int64_t stride_b_kv, void* d_out, int64_t stride_b_out, uint32_t flags, cudaStream_t s) {
  if (h->opt_fused && h->len >= 1 && !h->rope) {
    if (!d_k || !d_v) return fail(h, EA_ERR_INVALID_ARG, "decode_step: NULL k or v");
    int bad = 0;
    if (!room_for(h, 1, &bad))
      return fail(h, EA_ERR_CAPACITY, "decode_step: one more row exceeds the capacity of sequence %d (%lld rows)", bad,
                  static_cast<long long>(capacity_of(h, bad)));
    DecodePlan plan;
    const ea_status st = plan_decode(h, "decode_step", d_q, stride_b_q, d_out, stride_b_out, flags,
                                     reinterpret_cast<float*>(h->ws + h->L.off_partials), d_k, d_v, stride_b_kv,
                                     &plan);
    if (st != EA_OK) return st;
    const ea_status sl = launch_plan(h, "decode_step launch", plan, true, s);
    if (sl == EA_OK) h->len += 1;
    return sl;
  }
  const ea_status st = do_append(h, d_k, d_v, 1, stride_b_kv, stride_b_kv, flags & EA_KV_PREPROJECTED, s);
  if (st != EA_OK) return st;
  return do_decode(h, d_q, stride_b_q, d_out, stride_b_out, flags & ~EA_KV_PREPROJECTED, s);
}

}  // namespace

extern "C" {

int32_t eigen_attn_version(void) { return 100; }

ea_status eigen_attn_cache_bytes(const ea_desc* desc, size_t* cache_bytes, size_t* workspace_bytes) {
  if (!cache_bytes || !workspace_bytes) return EA_ERR_INVALID_ARG;
  const ea_status st = check_desc(desc);
  if (st != EA_OK) return st;
  Layout L;
  make_layout(desc, &L);
  *cache_bytes = L.cache_bytes;
  *workspace_bytes = L.workspace_bytes;
  return EA_OK;
}

ea_status eigen_attn_create(const ea_desc* desc, void* d_cache, size_t cache_bytes, void* d_workspace,
                            size_t workspace_bytes, void* cuda_stream, eigen_attn_t* out) {
  if (!out) return EA_ERR_INVALID_ARG;
  *out = nullptr;
  ea_status st = check_desc(desc);
  if (st != EA_OK) return st;
  if (!desc->U_k || !desc->U_v || !d_cache || !d_workspace) return EA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_cache) % kAlign) || (reinterpret_cast<uintptr_t>(d_workspace) % kAlign))
    return EA_ERR_INVALID_ARG;
  eigen_attn* h = new (std::nothrow) eigen_attn();
  if (!h) return EA_ERR_INVALID_ARG;
  h->err[0] = 0;
  h->desc = *desc;
  make_layout(desc, &h->L);
  const Layout& L = h->L;
  if (cache_bytes < L.cache_bytes || workspace_bytes < L.workspace_bytes) {
    delete h;
    return EA_ERR_CAPACITY;
  }
  const int H = desc->n_heads, dh = desc->d_head;

  // pad the bases (zero columns), build (U^V)^T, optionally check orthonormality
  std::vector<float> basis(L.basis_floats, 0.f);
  const float* uk = desc->U_k;
  const float* uv = desc->U_v;
  for (int hh = 0; hh < H; ++hh) {
    const HeadInfo& hi = L.heads[hh];
    for (int d = 0; d < dh; ++d) {
      for (int c = 0; c < hi.r_k; ++c)
        basis[hi.uk_off + static_cast<size_t>(d) * hi.rp_k + c] = uk[static_cast<size_t>(d) * hi.r_k + c];
      for (int c = 0; c < hi.r_v; ++c) {
        const float x = uv[static_cast<size_t>(d) * hi.r_v + c];
        basis[hi.uv_off + static_cast<size_t>(d) * hi.rp_v + c] = x;
        basis[hi.uvt_off + static_cast<size_t>(c) * dh + d] = x;
      }
    }
    if (dh % 16 == 0) {
      for (int pass = 0; pass < 2; ++pass) {
        const float* U = pass ? uv : uk;
        const int r = pass ? hi.r_v : hi.r_k;
        const int rp16 = ((pass ? hi.rp_v : hi.rp_k) + 15) & ~15;
        uint16_t* img_hi = reinterpret_cast<uint16_t*>(basis.data() + (pass ? hi.uvt16_off : hi.ukt16_off));
        uint16_t* img_lo = img_hi + static_cast<size_t>(rp16) * dh;
        const int grp = (dh / 8) * 128;                       // bytes per group of 8 rank columns
        for (int c = 0; c < rp16; ++c)
          for (int d = 0; d < dh; ++d) {
            const float x = c < r ? U[static_cast<size_t>(d) * r + c] : 0.f;
            const uint16_t xh = bf16_rne(x);
            const uint16_t xl = bf16_rne(x - bf16_to_float(xh));
            const size_t off = (static_cast<size_t>(c >> 3) * grp + (d >> 3) * 128 + (c & 7) * 16 + (d & 7) * 2) / 2;
            img_hi[off] = xh;
            img_lo[off] = xl;
          }
      }
    }
    for (int pass = 0; pass < 2 && dh % 16 == 0; ++pass) {
      // lift images of U^V (pass 0) and U^K (pass 1): rows = d (the N index of the lift product), contraction over the rank
      const float* U = pass ? uk : uv;
      const int r = pass ? hi.r_k : hi.r_v;
      const int rv16 = ((pass ? hi.rp_k : hi.rp_v) + 15) & ~15;
      uint16_t* img_hi = reinterpret_cast<uint16_t*>(basis.data() + (pass ? hi.ukl16_off : hi.uvl16_off));
      uint16_t* img_lo = img_hi + static_cast<size_t>(rv16) * dh;
      const int grp = (rv16 / 8) * 128;                       // bytes per group of 8 rows (d values)
      for (int d = 0; d < dh; ++d)
        for (int c = 0; c < rv16; ++c) {
          const float x = c < r ? U[static_cast<size_t>(d) * r + c] : 0.f;
          const uint16_t xh = bf16_rne(x);
          const uint16_t xl = bf16_rne(x - bf16_to_float(xh));
          const size_t off = (static_cast<size_t>(d >> 3) * grp + (c >> 3) * 128 + (d & 7) * 16 + (c & 7) * 2) / 2;
          img_hi[off] = xh;
          img_lo[off] = xl;
        }
    }
    if (desc->flags & EA_CHECK_ORTHONORMAL) {
      for (int pass = 0; pass < 2; ++pass) {
        const float* U = pass ? uv : uk;
        const int r = pass ? hi.r_v : hi.r_k;
        for (int a = 0; a < r; ++a)
          for (int b = a; b < r; ++b) {
            double dot = 0;
            for (int d = 0; d < dh; ++d)
              dot += static_cast<double>(U[static_cast<size_t>(d) * r + a]) * U[static_cast<size_t>(d) * r + b];
            if (fabs(dot - (a == b ? 1.0 : 0.0)) > 1e-4) {
              delete h;
              return EA_ERR_NOT_ORTHONORMAL;
            }
          }
      }
    }
    uk += static_cast<size_t>(dh) * hi.r_k;
    uv += static_cast<size_t>(dh) * hi.r_v;
  }
  h->cache = static_cast<char*>(d_cache);
  h->ws = static_cast<char*>(d_workspace);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemsetAsync(h->ws + L.off_status, 0, 64, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->ws + L.off_counters, 0, static_cast<size_t>(desc->batch) * H * sizeof(int), s);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(h->ws + L.off_heads, L.heads.data(), sizeof(HeadInfo) * H, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(h->ws + L.off_basis, basis.data(), basis.size() * sizeof(float), cudaMemcpyHostToDevice, s);
  // Rows of the cache that no call has written yet must hold finite values: the tensor-core prefill loads
  // whole 64-row tiles and multiplies the rows past the current length by zero weights.
  if (e == cudaSuccess) e = cudaMemsetAsync(h->cache, 0, L.cache_bytes, s);
  std::vector<CUtensorMap> tmaps;
  if (e == cudaSuccess && desc->dtype == EA_BF16 && dh % 16 == 0 &&
      static_cast<int64_t>(desc->n_max) * L.max_rp_k * 2 < (1ll << 40) &&
      encode_tensor_maps(desc, L, h->cache, &tmaps)) {
    e = cudaMemcpyAsync(h->ws + L.off_tmaps, tmaps.data(), tmaps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, s);
    h->tmaps_ok = true;
    std::vector<CUtensorMap> kmaps;
    if (e == cudaSuccess && L.rope_scratch && encode_krot_maps(desc, h->ws + L.off_krot, &kmaps)) {
      e = cudaMemcpyAsync(h->ws + L.off_tmaps_krot, kmaps.data(), kmaps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, s);
      // rows the first prompt does not write are read by whole key tiles and must be finite
      if (e == cudaSuccess) e = cudaMemsetAsync(h->ws + L.off_krot, 0, L.off_tmaps_krot - L.off_krot, s);
      h->krot_ok = true;
    }
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  int dev = 0;
  if (e == cudaSuccess) e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = ea::decode_configure(desc->dtype);
  if (e != cudaSuccess) {
    delete h;
    return EA_ERR_CUDA;
  }
  h->desc.r_k = nullptr; h->desc.r_v = nullptr; h->desc.U_k = nullptr; h->desc.U_v = nullptr;
  h->len = 0;
  *out = h;
  return EA_OK;
}

void eigen_attn_destroy(eigen_attn_t h) { delete h; }

ea_status eigen_attn_append_kv(eigen_attn_t h, const void* d_k, const void* d_v, int32_t T, int64_t stride_b,
                               int64_t stride_t, uint32_t flags, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  return do_append(h, d_k, d_v, T, stride_b, stride_t, flags, static_cast<cudaStream_t>(cuda_stream));
}

ea_status eigen_attn_decode(eigen_attn_t h, const void* d_q, int64_t stride_b_q, void* d_out,
                            int64_t stride_b_out, uint32_t flags, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  return do_decode(h, d_q, stride_b_q, d_out, stride_b_out, flags, static_cast<cudaStream_t>(cuda_stream));
}

ea_status eigen_attn_decode_step(eigen_attn_t h, const void* d_q, int64_t stride_b_q, const void* d_k,
                                 const void* d_v, int64_t stride_b_kv, void* d_out, int64_t stride_b_out,
                                 uint32_t flags, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (!d_q || !d_out) return fail(h, EA_ERR_INVALID_ARG, "decode_step: NULL q or out");
  if (flags & ~(EA_Q_PREPROJECTED | EA_OUT_LOWRANK | EA_KV_PREPROJECTED))
    return fail(h, EA_ERR_INVALID_ARG, "decode_step: unknown flag 0x%x", flags);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  return do_step(h, d_q, stride_b_q, d_k, d_v, stride_b_kv, d_out, stride_b_out, flags, s);
}

ea_status eigen_attn_decode_step_host(eigen_attn_t h, const void* h_q, const void* h_k, const void* h_v,
                                      void* h_out, uint32_t flags, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (!h_q || !h_k || !h_v || !h_out) return fail(h, EA_ERR_INVALID_ARG, "decode_step_host: NULL buffer");
  if (flags) return fail(h, EA_ERR_INVALID_ARG, "decode_step_host: flags must be 0");
  int bad = 0;
  if (!room_for(h, 1, &bad)) return fail(h, EA_ERR_CAPACITY, "decode_step_host: cache full (sequence %d)", bad);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const Layout& L = h->L;
  const size_t bytes = static_cast<size_t>(h->desc.batch) * h->desc.n_heads * h->desc.d_head * L.es;
  char* sq = h->ws + L.off_staging;
  char* sk = sq + L.staging_each;
  char* sv = sk + L.staging_each;
  char* so = sv + L.staging_each;
  cudaError_t e;
  const char* hq = static_cast<const char*>(h_q);
  if (static_cast<const char*>(h_k) == hq + bytes && static_cast<const char*>(h_v) == hq + 2 * bytes &&
      L.staging_each == bytes) {
    // q, k, v adjacent on the host (and in the staging area): one copy instead of three.  Adjacent addresses
    // can still belong to separate pinned allocations, which one copy may not span: then three copies after all.
    e = cudaMemcpyAsync(sq, h_q, 3 * bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaErrorInvalidValue) {
      (void)cudaGetLastError();
      e = cudaMemcpyAsync(sq, h_q, bytes, cudaMemcpyHostToDevice, s);
      if (e == cudaSuccess) e = cudaMemcpyAsync(sk, h_k, bytes, cudaMemcpyHostToDevice, s);
      if (e == cudaSuccess) e = cudaMemcpyAsync(sv, h_v, bytes, cudaMemcpyHostToDevice, s);
    }
  } else {
    e = cudaMemcpyAsync(sq, h_q, bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sk, h_k, bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sv, h_v, bytes, cudaMemcpyHostToDevice, s);
  }
  if (e != cudaSuccess) return cuda_fail(h, e, "decode_step_host H2D");
  const int64_t sb = static_cast<int64_t>(h->desc.n_heads) * h->desc.d_head;
  const ea_status st = do_step(h, sq, sb, sk, sv, sb, so, sb, 0, s);
  if (st != EA_OK) return st;
  e = cudaMemcpyAsync(h_out, so, bytes, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(h, e, "decode_step_host D2H");
  return EA_OK;
}

// Same computation and launch plan as eigen_attn_decode, with the split-KV partials in the library's
// built-in device array instead of the caller's workspace.
ea_status eigen_attn_decode_static(eigen_attn_t h, const void* d_q, int64_t stride_b_q, void* d_out,
                                   int64_t stride_b_out, uint32_t flags, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (h->rope) return fail(h, EA_ERR_UNSUPPORTED, "decode_static: not available with a rotary embedding");
  DecodePlan plan;
  ea_status st = plan_decode(h, "decode_static", d_q, stride_b_q, d_out, stride_b_out, flags, nullptr, nullptr,
                             nullptr, 0, &plan);
  if (st != EA_OK) return st;
  const size_t need = (static_cast<size_t>(plan.p.B) * plan.p.H + plan.grid) * plan.p.part_stride;
  if (need > ea::kStaticPartialFloats)
    return fail(h, EA_ERR_CAPACITY,
                "decode_static: (batch*heads + CTAs) * (4 + widest rp_v) = %zu floats exceeds the built-in "
                "scratch of %zu floats; use eigen_attn_decode with a workspace",
                need, static_cast<size_t>(ea::kStaticPartialFloats));
  float* scratch = nullptr;
  const cudaError_t e = ea::static_partials(&scratch);
  if (e != cudaSuccess) return cuda_fail(h, e, "decode_static: address of the built-in scratch");
  plan.p.partials = scratch;
  plan.c.partials = scratch;
  return launch_plan(h, "decode_static launch", plan, false, static_cast<cudaStream_t>(cuda_stream));
}

ea_status eigen_attn_prefill(eigen_attn_t h, const void* d_q, const void* d_k, const void* d_v, int32_t T,
                             int64_t stride_b, int64_t stride_t, void* d_out, int64_t out_stride_b,
                             int64_t out_stride_t, uint32_t flags, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (!d_q || !d_out) return fail(h, EA_ERR_INVALID_ARG, "prefill: NULL q or out");
  if (h->rope && (flags & EA_Q_PREPROJECTED))
    return fail(h, EA_ERR_INVALID_ARG, "prefill with rotary embedding: EA_Q_PREPROJECTED (the query must be full rank)");
  if (flags & ~(EA_OUT_LOWRANK | EA_Q_PREPROJECTED | EA_KV_PREPROJECTED))
    return fail(h, EA_ERR_INVALID_ARG, "prefill: unknown flag 0x%x", flags);
  const bool merged_in = (flags & (EA_Q_PREPROJECTED | EA_KV_PREPROJECTED)) != 0;
  if (T < 1) return fail(h, EA_ERR_SHAPE, "prefill: T = %d", T);
  if (T > h->desc.max_prefill_tokens)
    return fail(h, EA_ERR_CAPACITY, "prefill: T %d exceeds max_prefill_tokens %d", T, h->desc.max_prefill_tokens);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const int len0 = h->len;
  const Layout& L = h->L;
  const bool tc_shape = h->desc.dtype == EA_BF16 && h->desc.d_head % 16 == 0;
  // tensor-core kernels need 16-byte aligned rows on both sides
  const bool in_aligned = reinterpret_cast<uintptr_t>(d_q) % 16 == 0 && reinterpret_cast<uintptr_t>(d_k) % 16 == 0 &&
                          reinterpret_cast<uintptr_t>(d_v) % 16 == 0 && stride_b % 8 == 0 && stride_t % 8 == 0;
  const bool out_aligned = (flags & EA_OUT_LOWRANK) || (reinterpret_cast<uintptr_t>(d_out) % 16 == 0 &&
                                                        out_stride_b % 8 == 0 && out_stride_t % 8 == 0);
  const bool tc_attn = tc_shape && out_aligned && !h->paged;    // the tensor-core kernels address contiguous slabs
  if (h->opt_prefill == 2 && !tc_attn)
    return fail(h, EA_ERR_UNSUPPORTED, "prefill: the tcgen05 kernel needs bf16, d_head %% 16 == 0 and 16-byte aligned output rows");
  // Q', K', V' of the call's tokens in one tensor-core launch (K', V' into the cache, Q' into the workspace).  Its
  // rows equal eigen_attn_append_kv's except where the two fp32 summation orders round to different bf16 values
  // (one unit in the last place).
  const bool tc_project = tc_shape && in_aligned && h->opt_prefill != 1 && !h->paged && h->max_deficit == 0 && d_k && d_v;
  auto project_on_tensor_cores = [&]() -> ea_status {
    if (static_cast<int64_t>(len0) + T > h->desc.n_max)
      return fail(h, EA_ERR_CAPACITY, "prefill: len %d + T %d exceeds n_max %d", len0, T, h->desc.n_max);
    ea::ProjectTcParams pp{};
    pp.heads = dev_heads(h); pp.basis = dev_basis(h); pp.q = d_q; pp.k = d_k; pp.v = d_v;
    pp.cache = h->cache; pp.qp = h->ws + L.off_qp; pp.stride_b = stride_b; pp.stride_t = stride_t;
    pp.B = h->desc.batch; pp.T = T; pp.H = h->desc.n_heads; pp.d_head = h->desc.d_head;
    pp.n_max = h->desc.n_max; pp.row0 = len0; pp.status = dev_status(h);
    const int max_rp = L.max_rp_k > L.max_rp_v ? L.max_rp_k : L.max_rp_v;
    // Whole tiles of 64-element atoms and at least one full tile of tokens: the persistent kernel that streams
    // the token tiles by TMA and keeps the basis images in shared memory; otherwise one CTA per tile.
    CUtensorMap in_maps[3];
    const void* const in_ptrs[3] = {d_q, d_k, d_v};
    int ps_stages = 0;
    bool stream = h->opt_project != 1 && h->desc.d_head % 64 == 0 && T >= 128 && stride_t > 0 && stride_b > 0 &&
                  stride_t >= static_cast<int64_t>(h->desc.n_heads) * h->desc.d_head;
    if (stream) {
      ea::project_tc_stream_smem(max_rp, h->desc.d_head, &ps_stages);
      stream = ps_stages >= 2 && encode_input_maps(in_ptrs, h->desc.n_heads, h->desc.d_head, T, h->desc.batch,
                                                   stride_b, stride_t, in_maps);
    }
    const cudaError_t ep =
        stream ? ea::launch_project_tc_stream(pp, in_maps, max_rp, h->opt_project >= 2 ? static_cast<int>(h->opt_project) : h->sm_count,
                                              s, &h->launches)
               : ea::launch_project_tc(pp, max_rp, s, &h->launches);
    if (ep != cudaSuccess) return cuda_fail(h, ep, "prefill projection launch");
    h->len += T;
    return EA_OK;
  };
  cudaError_t e;
  if (h->rope) {
    // Section 4.3 for the prompt: the cache takes the projections of the un-rotated keys, as in the generation
    // phase; the attention kernel lifts and rotates them and rotates the full-rank queries itself.
    // On the tensor cores when the layer was created with the scratch for it and the rows cached after the call fit
    // it: the rotated queries and the lifted, rotated keys are written out once, then the warp-specialised kernel
    // runs an ordinary causal product over d_head-wide rows with the rank-r values of the cache.
    size_t ws_smem = 0;
    const int dh = h->desc.d_head;
    const int ws_stages = h->krot_ok && tc_attn && h->opt_prefill != 1 && h->opt_prefill != 3 &&
                                  static_cast<int64_t>(len0) + T <= h->desc.max_prefill_tokens &&
                                  ea::rope_lift_tc_smem_bytes(L.max_rp_k, dh) <= static_cast<size_t>(kSmemLimit)
                              ? ea::prefill_tc_ws_stages(dh, L.max_rp_v, dh, &ws_smem) : 0;
    if (h->opt_prefill == 2 && ws_stages < 3)
      return fail(h, EA_ERR_UNSUPPORTED, "prefill with rotary embedding: the tcgen05 kernel needs EA_ROPE_PROMPT_SCRATCH at create, "
                                         "16-byte aligned output rows, no page table and len + T <= max_prefill_tokens");
    // the tokens' rows: on the tensor cores when the attention runs there too (the Q' that launch also writes is
    // not used: the rotated full-rank queries take its place in the workspace)
    const ea_status st = ws_stages >= 3 && tc_project && !(flags & EA_KV_PREPROJECTED)
                             ? project_on_tensor_cores()
                             : do_append(h, d_k, d_v, T, stride_b, stride_t, flags & EA_KV_PREPROJECTED, s);
    if (st != EA_OK) return st;
    ea::PrefillParams p{};
    p.heads = dev_heads(h); p.basis = dev_basis(h); p.cache = h->cache; p.out = d_out;
    if (flags & EA_OUT_LOWRANK) {
      p.out_stride_t = L.sum_rp_v;
      p.out_stride_b = static_cast<int64_t>(T) * L.sum_rp_v;
    } else {
      p.out_stride_b = out_stride_b; p.out_stride_t = out_stride_t;
    }
    p.B = h->desc.batch; p.T = T; p.H = h->desc.n_heads; p.d_head = h->desc.d_head; p.n_max = h->desc.n_max;
    p.len0 = len0; p.deficit = dev_deficit(h);
    p.scale_log2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(h->desc.d_head)));
    p.flags = flags & EA_OUT_LOWRANK; p.status = dev_status(h);
    p.pages = dev_pages(h);
    p.q_raw = d_q; p.q_stride_b = stride_b; p.q_stride_t = stride_t;
    p.inv_freq = reinterpret_cast<const double*>(h->ws + L.off_rope);
    p.rope_interleaved = h->rope_interleaved;
    if (ws_stages >= 3) {
      p.qp = h->ws + L.off_qp;
      p.krot = h->ws + L.off_krot; p.krot_rows = h->desc.max_prefill_tokens;
      p.el_table = reinterpret_cast<const float4*>(h->ws + L.off_rope + ea::kRopeTableOffset);
      p.tmaps = h->ws + L.off_tmaps; p.tmaps_k = h->ws + L.off_tmaps_krot; p.k_width = dh;
      p.max_rp = dh;
      e = ea::launch_rope_prompt_prepare(p, L.max_rp_k, h->sm_count, s, &h->launches);
      if (e != cudaSuccess) return cuda_fail(h, e, "prefill preparation launch (rotary embedding)");
      if (h->ev_start) cudaEventRecord(h->ev_start, s);
      e = ea::launch_prefill_tc_ws(p, ws_stages, ws_smem, false, s, &h->launches);
      if (h->ev_stop) cudaEventRecord(h->ev_stop, s);
      if (e != cudaSuccess) return cuda_fail(h, e, "prefill attention launch (rotary embedding, tensor cores)");
      return EA_OK;
    }
    if (h->ev_start) cudaEventRecord(h->ev_start, s);
    e = ea::launch_prefill_rope(p, L.max_rp_k, L.max_rp_v, s, &h->launches);
    if (h->ev_stop) cudaEventRecord(h->ev_stop, s);
    if (e != cudaSuccess) return cuda_fail(h, e, "prefill attention launch (rotary embedding)");
    return EA_OK;
  }
  if (merged_in) {
    // Rank-space rows from merged weights (Eq. 8): nothing to multiply.  K', V' rows are copied into the cache, Q'
    // rows into the per-head layout the attention kernels read; a tensor the caller left d_head-wide is projected
    // on the CUDA cores.
    const ea_status st = do_append(h, d_k, d_v, T, stride_b, stride_t, flags & EA_KV_PREPROJECTED, s);
    if (st != EA_OK) return st;
    ea::QProjectParams qp{};
    qp.heads = dev_heads(h); qp.basis = dev_basis(h); qp.q = d_q; qp.qp = h->ws + L.off_qp;
    qp.stride_b = stride_b; qp.stride_t = stride_t;
    qp.B = h->desc.batch; qp.T = T; qp.H = h->desc.n_heads; qp.d_head = h->desc.d_head;
    e = (flags & EA_Q_PREPROJECTED) ? ea::launch_q_scatter(qp, L.sum_rp_k, h->desc.dtype, s, &h->launches)
                                    : ea::launch_q_project(qp, h->desc.dtype, s, &h->launches);
    if (e != cudaSuccess) return cuda_fail(h, e, "prefill q launch");
  } else if (tc_shape && in_aligned && h->opt_prefill != 1 && !h->paged && h->max_deficit == 0) {
    if (!d_k || !d_v) return fail(h, EA_ERR_INVALID_ARG, "prefill: NULL k or v");
    const ea_status st = project_on_tensor_cores();
    if (st != EA_OK) return st;
  } else {
    const ea_status st = do_append(h, d_k, d_v, T, stride_b, stride_t, 0, s);
    if (st != EA_OK) return st;
    ea::QProjectParams qp{};
    qp.heads = dev_heads(h); qp.basis = dev_basis(h); qp.q = d_q; qp.qp = h->ws + L.off_qp;
    qp.stride_b = stride_b; qp.stride_t = stride_t;
    qp.B = h->desc.batch; qp.T = T; qp.H = h->desc.n_heads; qp.d_head = h->desc.d_head;
    e = ea::launch_q_project(qp, h->desc.dtype, s, &h->launches);
    if (e != cudaSuccess) return cuda_fail(h, e, "prefill q projection launch");
  }
  ea::PrefillParams p{};
  p.heads = dev_heads(h); p.basis = dev_basis(h); p.cache = h->cache; p.qp = h->ws + L.off_qp; p.out = d_out;
  if (flags & EA_OUT_LOWRANK) {
    p.out_stride_t = L.sum_rp_v;
    p.out_stride_b = static_cast<int64_t>(T) * L.sum_rp_v;
  } else {
    p.out_stride_b = out_stride_b; p.out_stride_t = out_stride_t;
  }
  p.B = h->desc.batch; p.T = T; p.H = h->desc.n_heads; p.d_head = h->desc.d_head; p.n_max = h->desc.n_max;
  p.len0 = len0; p.deficit = dev_deficit(h);   // unequal lengths: every sequence's T tokens follow its own rows
  p.max_rp = L.max_rp_k > L.max_rp_v ? L.max_rp_k : L.max_rp_v;
  p.scale_log2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(h->desc.d_head)));
  p.flags = flags & EA_OUT_LOWRANK; p.status = dev_status(h);
  p.tmaps = h->ws + L.off_tmaps;
  p.pages = dev_pages(h);
  if (h->ev_start) cudaEventRecord(h->ev_start, s);
  size_t ws_smem = 0;
  const int ws_stages = tc_attn && h->tmaps_ok ? ea::prefill_tc_ws_stages(L.max_rp_k, L.max_rp_v, h->desc.d_head, &ws_smem) : 0;
  if (tc_attn && h->opt_prefill != 1 && h->opt_prefill != 3 && ws_stages >= 3)
    e = ea::launch_prefill_tc_ws(p, ws_stages, ws_smem, h->alibi, s, &h->launches);   // warp-specialised, 256 query rows per CTA
  else if (tc_attn && h->opt_prefill != 1)
    e = ea::launch_prefill_tc(p, L.max_rp_k, L.max_rp_v, s, &h->launches);  // single query tile per CTA (wide ranks)
  else
    e = ea::launch_prefill_simt(p, h->desc.dtype, s, &h->launches);
  if (h->ev_stop) cudaEventRecord(h->ev_stop, s);
  if (e != cudaSuccess) return cuda_fail(h, e, "prefill attention launch");
  return EA_OK;
}

ea_status eigen_attn_get_len(eigen_attn_t h, int32_t* len) {
  if (!h || !len) return EA_ERR_INVALID_ARG;
  *len = h->len;
  return EA_OK;
}

ea_status eigen_attn_set_len(eigen_attn_t h, int32_t len) {
  if (!h) return EA_ERR_INVALID_ARG;
  int64_t cap = h->desc.n_max;
  if (h->paged) {
    cap = INT32_MAX;
    for (int b = 0; b < h->desc.batch; ++b) cap = capacity_of(h, b) < cap ? capacity_of(h, b) : cap;
  }
  if (len < 0 || len > cap)
    return fail(h, EA_ERR_CAPACITY, "set_len: %d outside [0, %lld]", len, static_cast<long long>(cap));
  if (h->q_group && h->max_deficit > 0)      // leaving unequal lengths: rows every sequence holds as codes
    for (int b = 0; b < h->desc.batch; ++b)
      if (h->qlens[b] < h->qlen) h->qlen = h->qlens[b];
  h->len = len;
  h->max_deficit = 0;     // every sequence holds len rows again
  if (h->q_group && h->qlen > len) h->qlen = len / h->q_group * h->q_group;   // rows past len are forgotten
  return EA_OK;
}

ea_status eigen_attn_set_lens(eigen_attn_t h, const int32_t* lens, void* cuda_stream) {
  if (!h || !lens) return EA_ERR_INVALID_ARG;
  const int B = h->desc.batch;
  if (B > ea::kMaxRaggedBatch)
    return fail(h, EA_ERR_UNSUPPORTED, "set_lens: batch %d exceeds %d", B, ea::kMaxRaggedBatch);
  int32_t longest = 0;
  for (int b = 0; b < B; ++b) {
    if (lens[b] < 0 || lens[b] > capacity_of(h, b))
      return fail(h, EA_ERR_CAPACITY, "set_lens: lens[%d] = %d outside [0, %lld]", b, lens[b],
                  static_cast<long long>(capacity_of(h, b)));
    if (lens[b] > longest) longest = lens[b];
  }
  std::vector<int32_t> deficit(B);
  int32_t widest = 0;
  for (int b = 0; b < B; ++b) {
    deficit[b] = longest - lens[b];
    if (deficit[b] > widest) widest = deficit[b];
  }
  if (widest > 0) {
    // a pageable source is staged by the runtime before the call returns, so the vector may change afterwards
    const cudaError_t e = cudaMemcpyAsync(h->ws + h->L.off_deficit, deficit.data(), sizeof(int32_t) * B,
                                          cudaMemcpyHostToDevice, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(h, e, "set_lens: upload");
  }
  if (h->q_group) {
    // a sequence keeps the codes of its complete blocks below its new length
    std::vector<int32_t> q(B);
    int32_t qmax = 0, qmin = INT32_MAX;
    for (int b = 0; b < B; ++b) {
      const int32_t had = h->max_deficit > 0 ? h->qlens[b] : h->qlen;
      const int32_t cap = lens[b] / h->q_group * h->q_group;
      q[b] = had < cap ? had : cap;
      if (q[b] > qmax) qmax = q[b];
      if (q[b] < qmin) qmin = q[b];
    }
    if (widest > 0) {
      const cudaError_t e = cudaMemcpyAsync(h->ws + h->L.off_qlens, q.data(), sizeof(int32_t) * B, cudaMemcpyHostToDevice,
                                            static_cast<cudaStream_t>(cuda_stream));
      if (e != cudaSuccess) return cuda_fail(h, e, "set_lens: upload");
      h->qlens.swap(q);
      h->qlen = qmax;
    } else {
      h->qlen = qmin;
    }
  }
  h->deficit.swap(deficit);
  h->len = longest;
  h->max_deficit = widest;
  return EA_OK;
}

ea_status eigen_attn_set_page_table(eigen_attn_t h, const int32_t* h_table, int32_t pages_per_seq, int32_t page_rows,
                                    void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  const int B = h->desc.batch;
  if (!h_table) {                       // back to the contiguous layout
    int64_t longest = h->len;
    if (longest > h->desc.n_max) return fail(h, EA_ERR_CAPACITY, "set_page_table: len %d exceeds n_max %d", h->len, h->desc.n_max);
    h->paged = false;
    return EA_OK;
  }
  if (h->q_group) return fail(h, EA_ERR_UNSUPPORTED, "set_page_table: not available with a quantised cache");
  if (page_rows < 128 || (page_rows & (page_rows - 1)) != 0)
    return fail(h, EA_ERR_SHAPE, "set_page_table: page_rows %d (a power of two, at least 128)", page_rows);
  const int64_t pool = static_cast<int64_t>(B) * h->desc.n_max / page_rows;      // physical pages of a head's slab
  if (pool < 1) return fail(h, EA_ERR_SHAPE, "set_page_table: the cache holds no page of %d rows", page_rows);
  if (pages_per_seq < 1 || static_cast<int64_t>(pages_per_seq) * page_rows > INT32_MAX)
    return fail(h, EA_ERR_SHAPE, "set_page_table: pages_per_seq %d", pages_per_seq);
  if (static_cast<size_t>(B) * pages_per_seq > h->L.page_entries)
    return fail(h, EA_ERR_CAPACITY, "set_page_table: %d x %d entries exceed the table area (%zu)", B, pages_per_seq, h->L.page_entries);
  std::vector<bool> used(static_cast<size_t>(pool), false);
  std::vector<int32_t> cap(B, 0);
  for (int b = 0; b < B; ++b) {
    bool gap = false;
    for (int i = 0; i < pages_per_seq; ++i) {
      const int32_t pg = h_table[static_cast<size_t>(b) * pages_per_seq + i];
      if (pg == -1) { gap = true; continue; }
      if (pg < 0 || pg >= pool) return fail(h, EA_ERR_INVALID_ARG, "set_page_table: table[%d][%d] = %d outside [0, %lld)", b, i, pg, static_cast<long long>(pool));
      if (gap) return fail(h, EA_ERR_INVALID_ARG, "set_page_table: sequence %d maps page %d behind an unmapped one", b, i);
      if (used[pg]) return fail(h, EA_ERR_INVALID_ARG, "set_page_table: physical page %d is mapped twice", pg);
      used[pg] = true;
      cap[b] = (i + 1) * page_rows;
    }
    const int64_t have = h->len - (h->max_deficit > 0 ? h->deficit[b] : 0);
    if (have > cap[b]) return fail(h, EA_ERR_CAPACITY, "set_page_table: sequence %d holds %lld rows, the table maps %d", b, static_cast<long long>(have), cap[b]);
  }
  const cudaError_t e = cudaMemcpyAsync(h->ws + h->L.off_pages, h_table, sizeof(int32_t) * B * pages_per_seq,
                                        cudaMemcpyHostToDevice, static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) return cuda_fail(h, e, "set_page_table: upload");
  h->paged = true;
  h->page_width = pages_per_seq;
  h->page_shift = 0;
  while ((1 << h->page_shift) < page_rows) ++h->page_shift;
  h->page_cap.swap(cap);
  return EA_OK;
}

ea_status eigen_attn_get_lens(eigen_attn_t h, int32_t* lens) {
  if (!h || !lens) return EA_ERR_INVALID_ARG;
  for (int b = 0; b < h->desc.batch; ++b)
    lens[b] = h->len - (h->max_deficit > 0 ? h->deficit[b] : 0);
  return EA_OK;
}

ea_status eigen_attn_poll_status(eigen_attn_t h, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, dev_status(h), sizeof(int), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(dev_status(h), 0, sizeof(int), s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(h, e, "poll_status");
  if (word == ea::kStatusTimeout) {
    // an aborted launch may have left arrival counters half way: clear them for the next call
    cudaMemsetAsync(dev_counters(h), 0, static_cast<size_t>(h->desc.batch) * h->desc.n_heads * sizeof(int), s);
    cudaStreamSynchronize(s);
    return fail(h, EA_ERR_TIMEOUT, "a device-side wait exceeded its bound");
  }
  return EA_OK;
}

const char* eigen_attn_last_error(eigen_attn_t h) { return h ? h->err : "null handle"; }

ea_status eigen_attn_head_offsets(eigen_attn_t h, int32_t* offs_k, int32_t* offs_v) {
  if (!h || !offs_k || !offs_v) return EA_ERR_INVALID_ARG;
  const int H = h->desc.n_heads;
  for (int i = 0; i < H; ++i) {
    offs_k[i] = h->L.heads[i].lr_k_off;
    offs_v[i] = h->L.heads[i].lr_v_off;
  }
  offs_k[H] = h->L.sum_rp_k;
  offs_v[H] = h->L.sum_rp_v;
  return EA_OK;
}

ea_status eigen_attn_cache_layout(eigen_attn_t h, int32_t head, size_t* k_offset, size_t* v_offset,
                                  int32_t* rp_k, int32_t* rp_v) {
  if (!h || !k_offset || !v_offset || !rp_k || !rp_v) return EA_ERR_INVALID_ARG;
  if (head < 0 || head >= h->desc.n_heads) return fail(h, EA_ERR_SHAPE, "cache_layout: head %d", head);
  const HeadInfo& hi = h->L.heads[head];
  *k_offset = static_cast<size_t>(hi.k_off);
  *v_offset = static_cast<size_t>(hi.v_off);
  *rp_k = hi.rp_k;
  *rp_v = hi.rp_v;
  return EA_OK;
}

ea_status eigen_attn_set_alibi(eigen_attn_t h, const float* slopes, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (h->rope && slopes) return fail(h, EA_ERR_INVALID_ARG, "set_alibi: the layer has a rotary embedding");
  const int H = h->desc.n_heads;
  bool any = false;
  for (int i = 0; i < H; ++i) {
    const float sl = slopes ? slopes[i] : 0.f;
    if (!(sl >= 0.f) || !isfinite(sl)) return fail(h, EA_ERR_INVALID_ARG, "set_alibi: slope[%d] = %g", i, sl);
    h->L.heads[i].alibi_slope2 = static_cast<float>(static_cast<double>(sl) * 1.4426950408889634);
    any = any || sl != 0.f;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(h->ws + h->L.off_heads, h->L.heads.data(), sizeof(HeadInfo) * H, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(h, e, "set_alibi");
  h->alibi = any;
  return EA_OK;
}

ea_status eigen_attn_decode_gqa(eigen_attn_t h, const void* d_q, int64_t stride_b_q, int32_t group, void* d_out,
                                int64_t stride_b_out, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (!d_q || !d_out) return fail(h, EA_ERR_INVALID_ARG, "decode_gqa: NULL q or out");
  if (group < 1 || group > 16) return fail(h, EA_ERR_SHAPE, "decode_gqa: group %d (1..16)", group);
  if (h->desc.dtype != EA_BF16 || h->desc.d_head % 16 || !h->tmaps_ok)
    return fail(h, EA_ERR_UNSUPPORTED, "decode_gqa: needs a bf16 layer with d_head %% 16 == 0");
  if (h->alibi) return fail(h, EA_ERR_UNSUPPORTED, "decode_gqa: not available with an ALiBi bias set");
  if (h->len - h->max_deficit < 1) return fail(h, EA_ERR_SHAPE, "decode_gqa: the cache is empty (for some sequence)");
  // Section 4.3 for a group.  On the tensor cores where the tiles fit (decode_gqa_rope_kernel: the keys of a tile are
  // lifted and turned once for the whole group); otherwise (wide ranks, a page table) every query head of the group
  // is a unit of the multi-head rotary kernel over its K/V head's rows.
  const bool rope_tc = h->rope && !h->paged && group > 1 && ea::decode_gqa_rope_smem_bytes(h->L.max_rp_k, h->desc.d_head) != 0;
  if (h->rope && !rope_tc)
    return do_decode_rope(h, d_q, stride_b_q, d_out, stride_b_out, 0u, static_cast<cudaStream_t>(cuda_stream), group);
  const Layout& L = h->L;
  const int B = h->desc.batch, H = h->desc.n_heads, n = h->len;
  // without a rotary embedding: warp-level products where every rank is a multiple of 16 (EA_OPT_GQA_IMPL = 1 keeps
  // the tcgen05 kernel)
  const int max_rp = L.max_rp_k > L.max_rp_v ? L.max_rp_k : L.max_rp_v;
  int min_rp = max_rp;
  bool ranks16 = true;
  for (const HeadInfo& hi : L.heads) {
    if (hi.rp_k < min_rp) min_rp = hi.rp_k;
    if (hi.rp_v < min_rp) min_rp = hi.rp_v;
    if (hi.rp_k % 16) ranks16 = false;
  }
  const bool warp_mma = !rope_tc && h->opt_gqa_impl != 1 && ranks16 && h->desc.d_head <= 128 &&
                        ea::decode_gqa_mma_smem_bytes(max_rp, max_rp) != 0;
  if (h->paged && !warp_mma)
    return fail(h, EA_ERR_UNSUPPORTED, "decode_gqa: with a page table the ranks must be multiples of 16 and d_head <= 128 "
                                       "(EA_OPT_GQA_IMPL = 0)");
  const size_t smem = rope_tc ? ea::decode_gqa_rope_smem_bytes(L.max_rp_k, h->desc.d_head)
                      : warp_mma ? ea::decode_gqa_mma_smem_bytes(max_rp, max_rp) : ea::decode_gqa_smem_bytes(L.max_rp_k, L.max_rp_v);
  if (smem > static_cast<size_t>(kSmemLimit)) return fail(h, EA_ERR_UNSUPPORTED, "decode_gqa: tiles do not fit");
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  ea::GqaDecodeParams p{};
  p.heads = dev_heads(h); p.basis = dev_basis(h); p.cache = h->cache;
  p.q = d_q; p.q_stride_b = stride_b_q; p.out = d_out; p.out_stride_b = stride_b_out;
  p.partials = reinterpret_cast<float*>(h->ws + L.off_partials);
  p.status = dev_status(h);
  p.tmaps = h->ws + L.off_tmaps;
  p.deficit = dev_deficit(h);
  p.pages = dev_pages(h);
  p.part_stride = L.part_stride;
  p.B = B; p.H = H; p.d_head = h->desc.d_head; p.n = n; p.n_max = h->desc.n_max;
  p.nt = (n + 127) / 128;
  p.group = group;
  // CTAs per unit: waves of (SMs x CTAs per SM), a start-up worth a few tiles per CTA, and room for
  // units x splits x group partials in the workspace
  const int ctas_per_sm = smem * 2 + 4096 <= static_cast<size_t>(228 * 1024) ? 2 : 1;
  const int64_t units = static_cast<int64_t>(B) * H;
  int64_t cap = (units + kMaxDecodeCtas) * kPartialSlack / (units * group);
  if (cap < 1) return fail(h, EA_ERR_CAPACITY, "decode_gqa: batch x heads x group = %lld partials exceed the workspace",
                           static_cast<long long>(units * group));
  if (cap > p.nt) cap = p.nt;
  int64_t splits = 1;
  if (h->opt_ctas > 0) {
    splits = (h->opt_ctas + units - 1) / units;
    if (splits > cap) splits = cap;
  } else {
    const int64_t wave = static_cast<int64_t>(h->sm_count) * ctas_per_sm;
    int64_t best = INT64_MAX;
    for (int64_t s2 = 1; s2 <= cap && s2 <= 256; ++s2) {
      const int64_t cost = ((units * s2 + wave - 1) / wave) * ((p.nt + s2 - 1) / s2 + 6);
      if (cost < best) { best = cost; splits = s2; }
    }
  }
  p.splits = static_cast<int32_t>(splits);
  p.q_scale = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(h->desc.d_head)));
  if (h->ev_start) cudaEventRecord(h->ev_start, s);
  if (rope_tc) {
    p.inv_freq = reinterpret_cast<const double*>(h->ws + L.off_rope);
    p.tile_step = reinterpret_cast<const float2*>(h->ws + L.off_rope + ea::kRopeStepOffset);
    p.el_table = reinterpret_cast<const float4*>(h->ws + L.off_rope + ea::kRopeTableOffset);
    p.interleaved = h->rope_interleaved;
  }
  const cudaError_t e = rope_tc ? ea::launch_decode_gqa_rope(p, L.max_rp_k, s, &h->launches)
                        : warp_mma ? ea::launch_decode_gqa_mma(p, max_rp, min_rp, s, &h->launches)
                                   : ea::launch_decode_gqa(p, L.max_rp_k, L.max_rp_v, s, &h->launches);
  if (h->ev_stop) cudaEventRecord(h->ev_stop, s);
  if (e != cudaSuccess) return cuda_fail(h, e, "decode_gqa launch");
  return EA_OK;
}

ea_status eigen_attn_set_rope(eigen_attn_t h, double base, int32_t interleaved, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (base == 0.0) {
    h->rope = false;
    return EA_OK;
  }
  if (!(base > 1.0) || !isfinite(base)) return fail(h, EA_ERR_INVALID_ARG, "set_rope: base %g", base);
  if (h->desc.dtype != EA_BF16 || h->desc.d_head % 16 || !h->tmaps_ok)
    return fail(h, EA_ERR_UNSUPPORTED, "set_rope: needs a bf16 layer with d_head %% 16 == 0 (and the driver's tensor-map encoder)");
  if (h->alibi) return fail(h, EA_ERR_INVALID_ARG, "set_rope: the layer has an ALiBi bias");
  const int dh = h->desc.d_head;
  // the constants the kernels read: the inverse frequencies phi_i, e^{-i 128 phi_i} (one tile of cached rows back)
  // and e^{i l phi_i} for the 128 row offsets of a tile, worked out here in double precision
  std::vector<unsigned char> host(ea::kRopeConstBytes, 0);
  double* freq = reinterpret_cast<double*>(host.data());
  float* step = reinterpret_cast<float*>(host.data() + ea::kRopeStepOffset);
  float* table = reinterpret_cast<float*>(host.data() + ea::kRopeTableOffset);
  for (int i = 0; i < dh / 2; ++i) freq[i] = pow(base, -2.0 * i / dh);
  for (int i = 0; i < 64; ++i) {
    step[2 * i] = static_cast<float>(cos(-128.0 * freq[i]));
    step[2 * i + 1] = static_cast<float>(sin(-128.0 * freq[i]));
  }
  for (int k = 0; k < 32; ++k)
    for (int l = 0; l < 128; ++l) {
      float* e = table + (static_cast<size_t>(k) * 128 + l) * 4;
      e[0] = static_cast<float>(cos(l * freq[2 * k]));
      e[1] = static_cast<float>(cos(l * freq[2 * k + 1]));
      e[2] = static_cast<float>(sin(l * freq[2 * k]));
      e[3] = static_cast<float>(sin(l * freq[2 * k + 1]));
    }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(h->ws + h->L.off_rope, host.data(), host.size(), cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(h, e, "set_rope");
  h->rope = true;
  h->rope_interleaved = interleaved ? 1 : 0;
  return EA_OK;
}

// ---- Section 5.3: quantised copy of the rank-r cache

ea_status eigen_attn_quant_bytes(eigen_attn_t h, int32_t bits, int32_t group, size_t* bytes) {
  if (!h || !bytes) return EA_ERR_INVALID_ARG;
  const ea_status st = check_quant_args(h, "quant_bytes", bits, group);
  if (st != EA_OK) return st;
  std::vector<ea::QuantHead> qh;
  *bytes = make_quant_layout(h, bits, group, &qh, nullptr);
  return EA_OK;
}

ea_status eigen_attn_quant_attach(eigen_attn_t h, int32_t bits, int32_t group, void* d_qcache, size_t bytes,
                                  void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (!d_qcache) {             // detach
    h->qcache = nullptr; h->q_group = 0; h->q_bits = 0; h->qlen = 0;
    return EA_OK;
  }
  const ea_status st = check_quant_args(h, "quant_attach", bits, group);
  if (st != EA_OK) return st;
  if (h->paged) return fail(h, EA_ERR_UNSUPPORTED, "quant_attach: not available with a page table");
  if (reinterpret_cast<uintptr_t>(d_qcache) % kAlign) return fail(h, EA_ERR_INVALID_ARG, "quant_attach: buffer not 256-byte aligned");
  std::vector<ea::QuantHead> qh;
  int widest = 0;
  const size_t need = make_quant_layout(h, bits, group, &qh, &widest);
  if (bytes < need) return fail(h, EA_ERR_CAPACITY, "quant_attach: %zu bytes given, %zu needed", bytes, need);
  const int widest_rp = h->L.max_rp_k > h->L.max_rp_v ? h->L.max_rp_k : h->L.max_rp_v;
  if ((bits == 4 ? ea::decode_quant_mma_smem_bytes(widest, widest_rp, group)
                 : ea::decode_quant_smem_bytes(widest, h->L.max_rp_v)) > static_cast<size_t>(kSmemLimit))
    return fail(h, EA_ERR_UNSUPPORTED, "quant_attach: a stage of 128 rows does not fit in shared memory");
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(d_qcache, qh.data(), sizeof(ea::QuantHead) * qh.size(), cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(h, e, "quant_attach");
  h->qcache = static_cast<char*>(d_qcache);
  h->q_group = group;
  h->q_bits = bits;
  h->qlen = 0;
  if (h->max_deficit > 0) {    // attached to a batch of unequal lengths: no sequence has codes yet
    h->qlens.assign(h->desc.batch, 0);
    e = cudaMemsetAsync(h->ws + h->L.off_qlens, 0, sizeof(int32_t) * h->desc.batch, s);
    if (e != cudaSuccess) return cuda_fail(h, e, "quant_attach");
  }
  h->q_max_stage_bytes = widest;
  h->qheads.swap(qh);
  return EA_OK;
}

namespace {
void fill_quant_params(eigen_attn_t h, ea::QuantParams* p) {
  *p = ea::QuantParams{};
  p->heads = dev_heads(h);
  p->qheads = reinterpret_cast<const ea::QuantHead*>(h->qcache);
  p->basis = dev_basis(h);
  p->cache = h->cache; p->qcache = h->qcache;
  p->status = dev_status(h);
  p->part_stride = h->L.part_stride;
  p->B = h->desc.batch; p->H = h->desc.n_heads; p->d_head = h->desc.d_head;
  p->n = h->len; p->n_max = h->desc.n_max;
  p->nq = h->qlen; p->group = h->q_group; p->bits = h->q_bits; p->blocks_max = h->desc.n_max / h->q_group;
  p->deficit = dev_deficit(h);
  p->qlens = h->max_deficit > 0 ? reinterpret_cast<const int32_t*>(h->ws + h->L.off_qlens) : nullptr;
}
}  // namespace

ea_status eigen_attn_quant_sync(eigen_attn_t h, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (!h->qcache) return fail(h, EA_ERR_INVALID_ARG, "quant_sync: no quantised buffer attached");
  const int G = h->q_group;
  int b0 = h->qlen / G, b1 = h->len / G;
  const bool ragged = h->max_deficit > 0;
  std::vector<int32_t> q_new;
  if (ragged) {
    // every sequence's own complete blocks: the launch spans the union of the ranges, the kernel skips by sequence
    q_new.resize(h->desc.batch);
    b0 = INT32_MAX; b1 = 0;
    for (int b = 0; b < h->desc.batch; ++b) {
      const int lo = h->qlens[b] / G, hi = (h->len - h->deficit[b]) / G;
      q_new[b] = (hi > lo ? hi : lo) * G;
      if (hi > lo) {
        if (lo < b0) b0 = lo;
        if (hi > b1) b1 = hi;
      }
    }
  }
  if (b1 <= b0) return EA_OK;
  ea::QuantParams p;
  fill_quant_params(h, &p);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // the second grid dimension holds at most 65535 blocks
  for (int lo = b0; lo < b1; lo += 65535) {
    p.b0 = lo; p.b1 = lo + 65535 < b1 ? lo + 65535 : b1;
    const cudaError_t e = ea::launch_quantize_blocks(p, s, &h->launches);
    if (e != cudaSuccess) return cuda_fail(h, e, "quant_sync launch");
  }
  if (ragged) {
    // the kernel read the old per-sequence counts; the new ones follow it on the stream
    const cudaError_t e = cudaMemcpyAsync(h->ws + h->L.off_qlens, q_new.data(), sizeof(int32_t) * q_new.size(),
                                          cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(h, e, "quant_sync: upload");
    h->qlens.swap(q_new);
    h->qlen = 0;
    for (int32_t q : h->qlens) if (q > h->qlen) h->qlen = q;
  } else {
    h->qlen = b1 * G;
  }
  return EA_OK;
}

ea_status eigen_attn_quant_lens(eigen_attn_t h, int32_t* qlens) {
  if (!h || !qlens) return EA_ERR_INVALID_ARG;
  if (!h->qcache) return fail(h, EA_ERR_INVALID_ARG, "quant_lens: no quantised buffer attached");
  for (int b = 0; b < h->desc.batch; ++b) qlens[b] = h->max_deficit > 0 ? h->qlens[b] : h->qlen;
  return EA_OK;
}

ea_status eigen_attn_quant_len(eigen_attn_t h, int32_t* qlen) {
  if (!h || !qlen) return EA_ERR_INVALID_ARG;
  *qlen = h->qlen;
  return EA_OK;
}

ea_status eigen_attn_quant_layout(eigen_attn_t h, int32_t head, size_t* slab_offset, size_t* block_bytes,
                                  size_t* k_scale_offset, size_t* v_code_offset, size_t* v_scale_offset) {
  if (!h || !slab_offset || !block_bytes || !k_scale_offset || !v_code_offset || !v_scale_offset) return EA_ERR_INVALID_ARG;
  if (!h->qcache) return fail(h, EA_ERR_INVALID_ARG, "quant_layout: no quantised buffer attached");
  if (head < 0 || head >= h->desc.n_heads) return fail(h, EA_ERR_SHAPE, "quant_layout: head %d", head);
  const ea::QuantHead& q = h->qheads[head];
  *slab_offset = static_cast<size_t>(q.slab_off);
  *block_bytes = static_cast<size_t>(q.block_bytes);
  *k_scale_offset = static_cast<size_t>(q.ks_off);
  *v_code_offset = static_cast<size_t>(q.vc_off);
  *v_scale_offset = static_cast<size_t>(q.vs_off);
  return EA_OK;
}

ea_status eigen_attn_decode_quant(eigen_attn_t h, const void* d_q, int64_t stride_b_q, void* d_out,
                                  int64_t stride_b_out, uint32_t flags, void* cuda_stream) {
  if (!h) return EA_ERR_INVALID_ARG;
  if (!h->qcache) return fail(h, EA_ERR_INVALID_ARG, "decode_quant: no quantised buffer attached");
  if (!d_q || !d_out) return fail(h, EA_ERR_INVALID_ARG, "decode_quant: NULL q or out");
  if (flags & ~(EA_Q_PREPROJECTED | EA_OUT_LOWRANK)) return fail(h, EA_ERR_INVALID_ARG, "decode_quant: unknown flag 0x%x", flags);
  if (h->rope) return fail(h, EA_ERR_UNSUPPORTED, "decode_quant: not available with a rotary embedding");
  if (h->len - h->max_deficit < 1) return fail(h, EA_ERR_SHAPE, "decode_quant: the cache is empty (for some sequence)");
  const Layout& L = h->L;
  ea::QuantParams p;
  fill_quant_params(h, &p);
  p.q = d_q; p.q_stride_b = (flags & EA_Q_PREPROJECTED) ? L.sum_rp_k : stride_b_q;
  p.out = d_out; p.out_stride_b = (flags & EA_OUT_LOWRANK) ? L.sum_rp_v : stride_b_out;
  p.partials = reinterpret_cast<float*>(h->ws + L.off_partials);
  p.nst = (p.nq + 127) / 128;
  p.q_scale = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(h->desc.d_head)));
  p.flags = flags;
  const int max_rp = L.max_rp_k > L.max_rp_v ? L.max_rp_k : L.max_rp_v;
  const bool mma = p.bits == 4;          // 4-bit codes run on the integer tensor-core kernel
  const size_t smem = mma ? ea::decode_quant_mma_smem_bytes(h->q_max_stage_bytes, max_rp, p.group)
                          : ea::decode_quant_smem_bytes(h->q_max_stage_bytes, L.max_rp_v);
  // CTAs per unit: waves of (SMs x resident CTAs), a start-up worth a few stages per CTA, and room for
  // units x splits partials in the workspace
  int ctas_per_sm = static_cast<int>(static_cast<size_t>(228 * 1024) / (smem + 1024));
  const int reg_limit = mma ? 5 : max_rp <= 80 ? 3 : 2;
  if (ctas_per_sm > reg_limit) ctas_per_sm = reg_limit;
  if (ctas_per_sm < 1) ctas_per_sm = 1;
  const int64_t units = static_cast<int64_t>(p.B) * p.H;
  int64_t cap = (units + kMaxDecodeCtas) * kPartialSlack / units;
  if (cap > p.nst) cap = p.nst;
  if (cap > 65535) cap = 65535;
  if (cap < 1) cap = 1;
  int64_t splits = 1;
  if (h->opt_ctas > 0) {
    splits = (h->opt_ctas + units - 1) / units;
    if (splits > cap) splits = cap;
  } else {
    const int64_t wave = static_cast<int64_t>(h->sm_count) * ctas_per_sm;
    int64_t best = INT64_MAX;
    for (int64_t s2 = 1; s2 <= cap && s2 <= 256; ++s2) {
      const int64_t cost = ((units * s2 + wave - 1) / wave) * ((p.nst + s2 - 1) / s2 + 4);
      if (cost < best) { best = cost; splits = s2; }
    }
  }
  p.splits = static_cast<int32_t>(splits);
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (h->ev_start) cudaEventRecord(h->ev_start, s);
  int min_rp = max_rp;
  for (const HeadInfo& hi : L.heads) {
    if (hi.rp_k < min_rp) min_rp = hi.rp_k;
    if (hi.rp_v < min_rp) min_rp = hi.rp_v;
  }
  const cudaError_t e = mma ? ea::launch_decode_quant_mma(p, max_rp, min_rp, smem, s, &h->launches)
                            : ea::launch_decode_quant(p, max_rp, min_rp, smem, s, &h->launches);
  if (h->ev_stop) cudaEventRecord(h->ev_stop, s);
  if (e != cudaSuccess) return cuda_fail(h, e, "decode_quant launch");
  return EA_OK;
}

ea_status eigen_attn_set_option(eigen_attn_t h, int32_t option, int64_t value) {
  if (!h) return EA_ERR_INVALID_ARG;
  switch (option) {
    case EA_OPT_DECODE_CTAS:
      if (value < 0 || value > kMaxDecodeCtas)
        return fail(h, EA_ERR_INVALID_ARG, "DECODE_CTAS %lld", static_cast<long long>(value));
      h->opt_ctas = value;
      return EA_OK;
    case EA_OPT_DECODE_TILE_ROWS:
      if (value < 0 || value > 128 || value % 16)
        return fail(h, EA_ERR_INVALID_ARG, "DECODE_TILE_ROWS %lld", static_cast<long long>(value));
      h->opt_tile_rows = value;
      return EA_OK;
    case EA_OPT_DECODE_STAGES:
      if (value != 0 && (value < 2 || value > 12))
        return fail(h, EA_ERR_INVALID_ARG, "DECODE_STAGES %lld", static_cast<long long>(value));
      h->opt_stages = value;
      return EA_OK;
    case EA_OPT_PREFILL_IMPL:
      if (value < 0 || value > 3)
        return fail(h, EA_ERR_INVALID_ARG, "PREFILL_IMPL %lld", static_cast<long long>(value));
      h->opt_prefill = value;
      return EA_OK;
    case EA_OPT_DECODE_FUSED:
      if (value < 0 || value > 1) return fail(h, EA_ERR_INVALID_ARG, "DECODE_FUSED %lld", static_cast<long long>(value));
      h->opt_fused = value;
      return EA_OK;
    case EA_OPT_PREFILL_PROJECT:
      if (value < 0 || value > 65535) return fail(h, EA_ERR_INVALID_ARG, "PREFILL_PROJECT %lld", static_cast<long long>(value));
      h->opt_project = value;
      return EA_OK;
    case EA_OPT_DECODE_MIN_COPY_BYTES:
      if (value < -1 || value > (1 << 20)) return fail(h, EA_ERR_INVALID_ARG, "DECODE_MIN_COPY_BYTES %lld", static_cast<long long>(value));
      h->opt_min_copy = value;
      return EA_OK;
    case EA_OPT_GQA_IMPL:
      if (value < 0 || value > 1) return fail(h, EA_ERR_INVALID_ARG, "GQA_IMPL %lld", static_cast<long long>(value));
      h->opt_gqa_impl = value;
      return EA_OK;
    case EA_OPT_TEST_WAIT_GIVES_UP:
      if (value < 0 || value > 1) return fail(h, EA_ERR_INVALID_ARG, "TEST_WAIT_GIVES_UP %lld", static_cast<long long>(value));
      h->opt_give_up = value;
      return EA_OK;
    default:
      return fail(h, EA_ERR_INVALID_ARG, "unknown option %d", option);
  }
}

ea_status eigen_attn_launch_count(eigen_attn_t h, uint64_t* count) {
  if (!h || !count) return EA_ERR_INVALID_ARG;
  *count = h->launches;
  return EA_OK;
}

ea_status eigen_attn_set_decode_events(eigen_attn_t h, void* start_event, void* stop_event) {
  if (!h) return EA_ERR_INVALID_ARG;
  if ((start_event == nullptr) != (stop_event == nullptr))
    return fail(h, EA_ERR_INVALID_ARG, "set_decode_events: pass both or neither");
  h->ev_start = static_cast<cudaEvent_t>(start_event);
  h->ev_stop = static_cast<cudaEvent_t>(stop_event);
  return EA_OK;
}

}  // extern "C"
