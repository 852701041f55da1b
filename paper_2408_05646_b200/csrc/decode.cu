// Split-KV decode attention in the rank-r space (Eq. 3 of the paper evaluated in the space of Eq. 7)
// and the cross-split combine + lift through (U^V)^T.
//
// Kernel 1 (decode_splitkv_kernel): persistent CTAs, one per SM.  The (head, sequence) units are laid
// end to end as a list of row tiles weighted by their bytes (rp_k + rp_v per row); every CTA takes an
// equal share of that weight, i.e. a contiguous run of tiles that may start and end inside a unit.
// One producer thread streams the K' and V' tiles of the run from HBM into a shared-memory ring with
// bulk asynchronous copies (mbarrier completion); eight consumer warps take the scores, an online
// softmax and the weighted sum of value rows from shared memory.  A lane pair owns one row of a tile.
// A piece that covers its whole unit is normalised and lifted through (U^V)^T on the spot.  Otherwise
// the CTA writes an un-normalised partial (max, sum, o'[rp_v]) and bumps a per-unit counter; the CTA
// that arrives last merges the unit's partials (exact re-association of the softmax), normalises and
// lifts.  The new token's row can be handed to the kernel directly (k_new/v_new): the CTA that owns
// the end of a unit projects it, stores it in the cache and attends to it from shared memory, so a
// whole decode step (append + attend + combine + lift) is one launch.
//
// Kernel 2 (combine_lift_kernel): the same merge + lift as a separate launch, used when the fused
// merge is switched off.
#include <cuda_bf16.h>

#include "internal.h"

namespace ea {
namespace {

constexpr int kMaxStages = 12;
constexpr uint64_t kWaitBoundNs = 2000000000ull;   // every device-side wait gives up after 2 s
// Registers per thread after the reallocation.  The CTA is launched with 384 threads x 168 registers (three
// warps per scheduler share its 16 384); the warpgroup of the producer and the helper warps keeps 96 each, the
// two consumer warpgroups take 200: 128 x 96 + 256 x 200 <= 384 x 168.
constexpr int kRegsProducerGroup = 96, kRegsConsumers = 200;
constexpr int kHelperThreads = 96;                 // warps 9..11: the projections of the next piece
static_assert(128 * kRegsProducerGroup + 256 * kRegsConsumers <= kDecodeThreads * 168, "register split exceeds the launch");

struct __align__(128) DecodeSmemFixed {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  long long range[2];
  int abort_flag;
  int is_last;
  float piece_m, piece_l;
  unsigned long long proj_full[2];         // the helper warps have written q' (and the new row) of a piece
  unsigned long long proj_empty[2];        // the consumers are done with them
  float raw[2][3][128];                    // a unit's q, new k, new v as fp32: [0] for the consumers, [1] for the helpers
  float proj_part[256];                    // partial sums of the projections
  float qp[2][128];                        // q' * log2(e)/sqrt(d_head), for this piece and the next
  __align__(16) unsigned char new_k[2][512];  // the new token's k', v' in cache format (one row each)
  __align__(16) unsigned char new_v[2][512];
  float wmax[kDecodeConsumerWarps];
  float wsum[kDecodeConsumerWarps];
  float o_acc[128];                        // the piece's (later the unit's) o'
  float stage_o[kDecodeConsumerWarps][4][128];
  int pre[kMaxRaggedBatch + 1];            // unequal lengths: tiles of the sequences before b (exclusive prefix)
};

// ---------------------------------------------------------------- PTX helpers

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(void* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(void* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false (and the status word set) if the phase did not complete within the bound.  With
// `abort_flag` the wait also ends (false) once another role of the CTA has given up: after that nobody
// may be left to complete the phase.
__device__ __forceinline__ bool mbar_wait(void* bar, uint32_t parity, int* status,
                                          const volatile int* abort_flag = nullptr) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (abort_flag != nullptr && *abort_flag != 0) return false;
    if (global_ns() - t0 > kWaitBoundNs) {
      atomicExch(status, kStatusTimeout);
      return false;
    }
  }
}
__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kDecodeConsumerWarps * 32) : "memory");
}
__device__ __forceinline__ void helper_sync() { asm volatile("bar.sync 2, %0;" ::"n"(kHelperThreads) : "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The shared-memory ring as one role sees it.  Slots are sized for the head being streamed (a narrow
// head gets more, smaller slots, so the bytes in flight stay the same), hence the slot count can change
// from one piece to the next; every slot's mbarriers keep their own phase, tracked as one parity bit per
// slot.  Producer and consumers derive the same geometry from the head and walk the slots in the same order.
struct Ring {
  int stage = 0;            // next slot
  int stages = 0;           // slots of the current geometry
  int stage_bytes = 0;      // bytes per slot: K tiles, then V tiles at v_off
  int v_off = 0;
  int tps = 1;              // tiles per slot (consecutive tiles of a unit are one contiguous range of rows)
  uint32_t full_bits = 0;   // bit s: parity of slot s's next "full" phase
  uint32_t empty_bits = 0;  // bit s: parity of slot s's next "empty" phase (producer only)
  uint32_t filled = 0;      // bit s: the slot holds a tile not yet known to be released (producer only)
  __device__ __forceinline__ void advance() { if (++stage == stages) stage = 0; }
};

// Slot geometry for a head: about p.inflight_bytes of copies in flight, at least three slots if they fit.
// A slot of a narrow head holds `tps` consecutive tiles (one bulk copy for their K' rows, one for their V'
// rows), so that a copy moves about p.min_copy_bytes: small copies do not reach the memory system's rate.
template <typename T>
__device__ __forceinline__ void ring_geometry(const DecodeParams& p, const HeadInfo& hd, int* stage_bytes,
                                              int* v_off, int* stages, int* tiles_per_slot) {
  int kb = p.tile_rows * hd.rp_k * static_cast<int>(sizeof(T));
  int vb = p.tile_rows * hd.rp_v * static_cast<int>(sizeof(T));
  const int narrow = kb < vb ? kb : vb;
  int tps = (p.min_copy_bytes + narrow - 1) / narrow;
  if (tps > 4) tps = 4;
  while (tps > 1 && 3 * (((kb + vb) * tps + 127) & ~127) > p.ring_bytes) --tps;   // keep three slots
  if (tps < 1) tps = 1;
  kb *= tps;
  vb *= tps;
  const int sb = (kb + vb + 127) & ~127;
  int fit = p.ring_bytes / sb;
  if (fit > kMaxStages) fit = kMaxStages;
  int want = p.fixed_stages > 0 ? p.fixed_stages : (p.inflight_bytes + sb - 1) / sb;
  if (want < 3 && p.fixed_stages == 0) want = 3;
  *stage_bytes = sb;
  *v_off = kb;
  *stages = want < fit ? want : fit;
  *tiles_per_slot = tps;
}

// L2 policy for data that is read once: evict it first.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s_hint(void* dst, const void* src, uint32_t bytes, void* bar,
                                              uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

// ---------------------------------------------------------------- element access

template <typename T>
struct Elem;
template <>
struct Elem<__nv_bfloat16> {
  static constexpr int kPerChunk = 8;   // elements in 16 bytes
  static __device__ __forceinline__ void load_chunk(const unsigned char* p, float (&f)[8]) {
    const uint4 x = *reinterpret_cast<const uint4*>(p);
    f[0] = __uint_as_float(x.x << 16); f[1] = __uint_as_float(x.x & 0xffff0000u);
    f[2] = __uint_as_float(x.y << 16); f[3] = __uint_as_float(x.y & 0xffff0000u);
    f[4] = __uint_as_float(x.z << 16); f[5] = __uint_as_float(x.z & 0xffff0000u);
    f[6] = __uint_as_float(x.w << 16); f[7] = __uint_as_float(x.w & 0xffff0000u);
  }
  static __device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
  static __device__ __forceinline__ __nv_bfloat16 from_float(float v) { return __float2bfloat16_rn(v); }
};
template <>
struct Elem<float> {
  static constexpr int kPerChunk = 4;
  static __device__ __forceinline__ void load_chunk(const unsigned char* p, float (&f)[4]) {
    const float4 x = *reinterpret_cast<const float4*>(p);
    f[0] = x.x; f[1] = x.y; f[2] = x.z; f[3] = x.w;
  }
  static __device__ __forceinline__ float to_float(float v) { return v; }
  static __device__ __forceinline__ float from_float(float v) { return v; }
};

// ---------------------------------------------------------------- work decomposition

// First tile (in the flat order head-major, then sequence, then tile) whose start weight x
// satisfies x * grid >= c * w_total.  Tiles of head h weigh (rp_k + rp_v).
__device__ long long first_tile_of_cta(const DecodeParams& p, int grid, int c) {
  const long long per_head_tiles = p.nt_total;
  if (c >= grid) return per_head_tiles * p.H;
  const long long num = static_cast<long long>(c) * p.w_total;
  const long long target = (num + grid - 1) / grid;
  int h = 0;
  for (int j = 1; j < p.H; ++j)
    if (per_head_tiles * p.heads[j].w_prefix <= target) h = j;
  const long long base = per_head_tiles * p.heads[h].w_prefix;
  const long long w = p.heads[h].rp_k + p.heads[h].rp_v;
  long long idx = (target - base + w - 1) / w;
  if (idx > per_head_tiles) idx = per_head_tiles;
  return per_head_tiles * h + idx;
}

// Cached rows of sequence b: p.n for a batch of equal lengths, else p.n minus the sequence's deficit.
__device__ __forceinline__ int seq_rows(const DecodeParams& p, int b) {
  return p.deficit != nullptr ? p.n - __ldg(p.deficit + b) : p.n;
}
// Tiles of a sequence of n_b rows; a sequence without rows still owns one (empty) tile, so that some CTA
// attends its new token.
__device__ __forceinline__ int seq_tiles(const DecodeParams& p, int n_b) {
  const int t = (n_b + p.tile_rows - 1) / p.tile_rows;
  return t > 0 ? t : 1;
}

// Where the flat tile index F falls: the unit (head h, sequence b), the tile i0 inside it, the unit's tile count
// and the tiles of the head that precede the unit.  Equal lengths: plain division.  Unequal lengths: the flat
// order holds each sequence's own tiles only, and `pre` (shared memory) is their exclusive prefix over b.
struct Piece {
  int unit, h, b, i0, nt_u;
  long long t0;
};
__device__ __forceinline__ Piece locate(const DecodeParams& p, const int* pre, long long F) {
  Piece u;
  if (p.deficit == nullptr) {
    u.unit = static_cast<int>(F / p.nt);
    u.i0 = static_cast<int>(F - static_cast<long long>(u.unit) * p.nt);
    u.h = u.unit / p.B;
    u.b = u.unit - u.h * p.B;
    u.nt_u = p.nt;
    u.t0 = static_cast<long long>(u.b) * p.nt;
  } else {
    u.h = static_cast<int>(F / p.nt_total);
    const int rem = static_cast<int>(F - static_cast<long long>(u.h) * p.nt_total);
    int lo = 0, hi = p.B;                            // largest b with pre[b] <= rem
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (pre[mid] <= rem) lo = mid; else hi = mid;
    }
    u.b = lo;
    u.i0 = rem - pre[lo];
    u.nt_u = pre[lo + 1] - pre[lo];
    u.t0 = pre[lo];
    u.unit = u.h * p.B + lo;
  }
  return u;
}

// ---------------------------------------------------------------- one (CTA, unit) piece

template <typename T, int NCH>
__device__ __forceinline__ void run_segment(const DecodeParams& p, DecodeSmemFixed* fx,
                                            unsigned char* ring, const HeadInfo& hd, int i0, int i1,
                                            Ring& ring_state, int warp, int lane, bool with_new_row, int n_b, int buf) {
  constexpr int EPC = Elem<T>::kPerChunk;
  const int pair = lane >> 1, half = lane & 1;
  const int rowb_k = hd.rp_k * static_cast<int>(sizeof(T));
  const int rowb_v = hd.rp_v * static_cast<int>(sizeof(T));
  const int nch_k = rowb_k >> 4, nch_v = rowb_v >> 4;

  // Chunk rotation that spreads the four lane pairs of a quarter warp over all banks when the
  // row pitch is a multiple of 64 bytes.
  auto rotation = [&](int rowb) {
    const int s = (rowb >> 2) & 31;
    return s == 0 ? (pair & 3) : (s == 16 ? ((pair >> 1) & 1) : 0);
  };
  const int rot_k = rotation(rowb_k), rot_v = rotation(rowb_v);

  int off_k[NCH], off_v[NCH];
  float q[NCH][EPC];
  float o[NCH][EPC];
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    const int ck = ((j ^ rot_k) << 1) + half;
    const int cv = ((j ^ rot_v) << 1) + half;
    const bool vk = ck < nch_k;
    off_k[j] = vk ? (ck << 4) : 0;
    off_v[j] = cv < nch_v ? (cv << 4) : 0;
#pragma unroll
    for (int e = 0; e < EPC; ++e) {
      q[j][e] = vk ? fx->qp[buf][ck * EPC + e] : 0.f;
      o[j][e] = 0.f;
    }
  }

  volatile int* abort_flag = &fx->abort_flag;
  float m = -INFINITY, l = 0.f;

  // score of one cached row against q', online-softmax update, weighted accumulation of its value row
  // ALiBi: the query sits at position n_total - 1; row j gets slope * (j - (n_total - 1)) <= 0 (log2 domain)
  const float slope2 = hd.alibi_slope2;
  const int pos_q = n_b - 1 + (p.k_new != nullptr ? 1 : 0);
  auto process_row = [&](const unsigned char* kr, const unsigned char* vr, bool valid, int j_abs) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      float x[EPC];
      Elem<T>::load_chunk(kr + off_k[j], x);
#pragma unroll
      for (int e = 0; e < EPC; e += 4) {
        a0 = fmaf(x[e + 0], q[j][e + 0], a0); a1 = fmaf(x[e + 1], q[j][e + 1], a1);
        a2 = fmaf(x[e + 2], q[j][e + 2], a2); a3 = fmaf(x[e + 3], q[j][e + 3], a3);
      }
    }
    float s = (a0 + a1) + (a2 + a3);
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s = fmaf(slope2, static_cast<float>(j_abs - pos_q), s);
    if (valid) {
      if (s > m) {                      // rare after the first rows: rescale the running state
        const float c = fast_exp2(m - s);
        l *= c;
#pragma unroll
        for (int j = 0; j < NCH; ++j)
#pragma unroll
          for (int e = 0; e < EPC; ++e) o[j][e] *= c;
        m = s;
      }
      const float pr = fast_exp2(s - m);
      l += pr;
#pragma unroll
      for (int j = 0; j < NCH; ++j) {
        float x[EPC];
        Elem<T>::load_chunk(vr + off_v[j], x);
#pragma unroll
        for (int e = 0; e < EPC; ++e) o[j][e] = fmaf(pr, x[e], o[j][e]);
      }
    }
  };

  for (int i = i0; i < i1; i += ring_state.tps) {           // one slot: up to tps tiles, contiguous rows
    const int stage = ring_state.stage;
    const uint32_t parity = (ring_state.full_bits >> stage) & 1u;
    ring_state.full_bits ^= 1u << stage;
    ring_state.advance();
    // warp-uniform decisions: the row code below shuffles across the whole warp
    if (__any_sync(0xffffffffu, *abort_flag != 0)) continue;
    bool landed = mbar_wait(&fx->full[stage], parity, p.status);
    if (p.give_up_once != 0 && blockIdx.x == 0 && warp == 0) {
      // test hook: behave exactly as if this wait had exceeded its bound (the copy itself still lands
      // and the producer waits for it before the CTA exits)
      if (lane == 0) atomicExch(p.status, kStatusTimeout);
      landed = false;
    }
    if (__any_sync(0xffffffffu, !landed)) {
      *abort_flag = 1;
      continue;
    }
    const unsigned char* kt = ring + static_cast<size_t>(stage) * ring_state.stage_bytes;
    const unsigned char* vt = kt + ring_state.v_off;
    const int rows = min(min(ring_state.tps, i1 - i) * p.tile_rows, n_b - i * p.tile_rows);
    // The loop bound is the same for all lanes of a warp (the shuffle inside needs every lane);
    // lane pairs past the last row recompute the group's first row and drop the result.
    for (int rbase = warp * 16; rbase < rows; rbase += kDecodeConsumerWarps * 16) {
      const bool valid = rbase + pair < rows;
      const int row = valid ? rbase + pair : rbase;
      process_row(kt + row * rowb_k, vt + row * rowb_v, valid, i * p.tile_rows + row);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&fx->empty[stage]);
  }

  // the new token's row (already projected, in shared memory) is attended by one lane pair
  if (with_new_row && warp == 0 && !__any_sync(0xffffffffu, *abort_flag != 0))
    process_row(fx->new_k[buf], fx->new_v[buf], pair == 0, pos_q);

  // ---- merge the 128 lane pairs of the CTA into one partial
  float wm = m;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, d));
  if (lane == 0) fx->wmax[warp] = wm;
  consumer_sync();
  float M = fx->wmax[0];
#pragma unroll
  for (int w = 1; w < kDecodeConsumerWarps; ++w) M = fmaxf(M, fx->wmax[w]);
  const float f = (m == -INFINITY) ? 0.f : fast_exp2(m - M);
  float ls = half == 0 ? l * f : 0.f;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, d);
  if (lane == 0) fx->wsum[warp] = ls;
#pragma unroll
  for (int j = 0; j < NCH; ++j)
#pragma unroll
    for (int e = 0; e < EPC; ++e) {
      float v = o[j][e] * f;
      v += __shfl_xor_sync(0xffffffffu, v, 8);    // pairs p, p+4, p+8, p+12 hold the same columns
      v += __shfl_xor_sync(0xffffffffu, v, 16);
      o[j][e] = v;
    }
  if (lane < 8) {
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      const int cv = ((j ^ rot_v) << 1) + half;
      if (cv < nch_v) {
#pragma unroll
        for (int e = 0; e < EPC; ++e) fx->stage_o[warp][pair][cv * EPC + e] = o[j][e];
      }
    }
  }
  consumer_sync();
  const int t = warp * 32 + lane;
  if (t < hd.rp_v) {
    float acc = 0.f;
#pragma unroll
    for (int w = 0; w < kDecodeConsumerWarps; ++w)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc += fx->stage_o[w][c][t];
    fx->o_acc[t] = acc;
  }
  if (t == 0) {
    float L = 0.f;
#pragma unroll
    for (int w = 0; w < kDecodeConsumerWarps; ++w) L += fx->wsum[w];
    fx->piece_m = M;
    fx->piece_l = L;
  }
  consumer_sync();
}

// Projections of a piece: q' = q U^K * log2(e)/sqrt(d_head) into fx->qp[buf], and, when the piece ends its unit and
// a new token is supplied, k' = k U^K and v' = v U^V, rounded to the cache dtype, into fx->new_k / fx->new_v [buf]
// and into row n_b (the sequence's length) of the cache.  A CTA's first piece is projected by its 256 consumer
// threads (NT = 256), every later one by the 96 threads of the helper warps (NT = 96) while the consumers stream
// the piece before it.  t = 0 .. NT - 1.
template <typename T, int NT>
__device__ __forceinline__ void project_inputs(const DecodeParams& p, DecodeSmemFixed* fx, int buf,
                                               const HeadInfo& hd, int h, int b, int t, bool with_new_row,
                                               int n_b) {
  constexpr bool kHelpers = NT == kHelperThreads;
  float* qraw = fx->raw[kHelpers ? 1 : 0][0];
  float* kraw = fx->raw[kHelpers ? 1 : 0][1];
  float* vraw = fx->raw[kHelpers ? 1 : 0][2];
  auto group_sync = [] { if (kHelpers) helper_sync(); else consumer_sync(); };
  const T* q = static_cast<const T*>(p.q);
  const int d_head = p.d_head;
  const bool q_lowrank = (p.flags & 0x1u) != 0;   // rank-space query supplied by the caller (merged W^Q')
  float* qp = fx->qp[buf];
  T* knew = reinterpret_cast<T*>(fx->new_k[buf]);
  T* vnew = reinterpret_cast<T*>(fx->new_v[buf]);
  if (q_lowrank) {
    for (int c = t; c < hd.rp_k; c += NT) qp[c] = Elem<T>::to_float(q[b * p.q_stride_b + hd.lr_k_off + c]) * p.q_scale;
  } else {
    for (int d = t; d < d_head; d += NT) qraw[d] = Elem<T>::to_float(q[b * p.q_stride_b + static_cast<int64_t>(h) * d_head + d]);
  }
  const bool kv_lowrank = (p.flags & 0x4u) != 0;  // rank-space k', v' supplied by the caller (merged W^K', W^V')
  const int64_t crow = physical_row(p.pages, b, p.n_max, n_b);
  if (with_new_row && kv_lowrank) {
    // nothing to project: the packed rows go into the cache (padding columns zero) and into shared memory
    for (int c = t; c < hd.rp_k; c += NT) {
      const T val = c < hd.r_k ? static_cast<const T*>(p.k_new)[b * p.kv_stride_b + hd.lr_k_off + c] : Elem<T>::from_float(0.f);
      knew[c] = val;
      reinterpret_cast<T*>(p.cache + hd.k_off)[crow * hd.rp_k + c] = val;
    }
    for (int c = t; c < hd.rp_v; c += NT) {
      const T val = c < hd.r_v ? static_cast<const T*>(p.v_new)[b * p.v_stride_b + hd.lr_v_off + c] : Elem<T>::from_float(0.f);
      vnew[c] = val;
      reinterpret_cast<T*>(p.cache + hd.v_off)[crow * hd.rp_v + c] = val;
    }
    with_new_row = false;                         // for the projection below
  }
  if (with_new_row)
    for (int d = t; d < d_head; d += NT) {
      kraw[d] = Elem<T>::to_float(static_cast<const T*>(p.k_new)[b * p.kv_stride_b + static_cast<int64_t>(h) * d_head + d]);
      vraw[d] = Elem<T>::to_float(static_cast<const T*>(p.v_new)[b * p.v_stride_b + static_cast<int64_t>(h) * d_head + d]);
    }
  group_sync();
  // outputs: [0, nq) = q' columns, [nq, nq + rp_k) = k' columns, then rp_v v' columns
  const int nq = q_lowrank ? 0 : hd.rp_k;
  const int total = nq + (with_new_row ? hd.rp_k + hd.rp_v : 0);
  // k' and v' are summed over d_head in one fixed order (the append kernel's), so that a row stored by
  // this kernel is bit-identical to the same row stored by eigen_attn_append_kv
  auto finish = [&](int o, float acc) {
    if (o < nq) {
      qp[o] = acc * p.q_scale;
    } else if (o < nq + hd.rp_k) {
      const int c = o - nq;
      const T val = Elem<T>::from_float(acc);
      knew[c] = val;
      reinterpret_cast<T*>(p.cache + hd.k_off)[crow * hd.rp_k + c] = val;
    } else {
      const int c = o - nq - hd.rp_k;
      const T val = Elem<T>::from_float(acc);
      vnew[c] = val;
      reinterpret_cast<T*>(p.cache + hd.v_off)[crow * hd.rp_v + c] = val;
    }
  };
  for (int o = t; o < total; o += NT) {
    const float* x;
    const float* U;
    int rp;
    if (o < nq) { x = qraw; U = p.basis + hd.uk_off + o; rp = hd.rp_k; }
    else if (o < nq + hd.rp_k) { x = kraw; U = p.basis + hd.uk_off + (o - nq); rp = hd.rp_k; }
    else { x = vraw; U = p.basis + hd.uv_off + (o - nq - hd.rp_k); rp = hd.rp_v; }
    float acc = 0.f;
#pragma unroll 32
    for (int d = 0; d < d_head; ++d) acc = fmaf(x[d], __ldg(U + d * rp), acc);
    finish(o, acc);
  }
  group_sync();                                   // the raw vectors are reused by the next piece
}

// CTA that owns the tile with start weight x: floor(x * grid / w_total).
__device__ __forceinline__ int owner_cta(long long x, int grid, long long w_total) {
  return static_cast<int>((x * grid) / w_total);
}

// After run_segment: turn the piece in shared memory (o_acc, piece_m, piece_l) into the unit's output,
// directly if the piece is the whole unit, else through the partial slots and the arrival counter.
template <typename T>
__device__ __forceinline__ void finish_piece(const DecodeParams& p, DecodeSmemFixed* fx, const HeadInfo& hd,
                                             const Piece& pc, int cta, int grid, bool whole, int t) {
  const int unit = pc.unit, h = pc.h, b = pc.b;
  bool finalize = whole && p.counters != nullptr;
  float inv_l = 1.f / fx->piece_l;
  if (!finalize) {
    float* part = p.partials + static_cast<size_t>(unit + cta) * p.part_stride;
    if (t < hd.rp_v) part[4 + t] = fx->o_acc[t];
    if (t == 0) { part[0] = fx->piece_m; part[1] = fx->piece_l; }
    if (p.counters == nullptr) {      // a separate combine launch follows
      consumer_sync();
      return;
    }
    const long long w = hd.rp_k + hd.rp_v;
    const long long x0 = p.nt_total * hd.w_prefix + pc.t0 * w;
    const int c0 = owner_cta(x0, grid, p.w_total);
    const int c1 = owner_cta(x0 + static_cast<long long>(pc.nt_u - 1) * w, grid, p.w_total);
    __threadfence();                  // this thread's partial is visible before the arrival is counted
    consumer_sync();
    if (t == 0) {
      const int arrived = atomicAdd(&p.counters[unit], 1);
      const int last = arrived == c1 - c0;
      if (last) p.counters[unit] = 0; // ready for the next call
      fx->is_last = last;
    }
    consumer_sync();
    if (fx->is_last) {
      __threadfence();
      float M = -INFINITY;
      for (int c = c0; c <= c1; ++c)
        M = fmaxf(M, __ldcg(p.partials + static_cast<size_t>(unit + c) * p.part_stride));
      float L = 0.f, acc = 0.f;
      for (int c = c0; c <= c1; ++c) {
        const float* pc = p.partials + static_cast<size_t>(unit + c) * p.part_stride;
        const float f = fast_exp2(__ldcg(pc) - M);
        L = fmaf(__ldcg(pc + 1), f, L);
        if (t < hd.rp_v) acc = fmaf(__ldcg(pc + 4 + t), f, acc);
      }
      if (t < hd.rp_v) fx->o_acc[t] = acc;
      inv_l = 1.f / L;
      finalize = true;
    }
    consumer_sync();
  }
  if (finalize) {
    T* out = static_cast<T*>(p.out);
    if (p.flags & 0x2u) {             // rank-space output for a merged W^O'
      if (t < hd.rp_v) out[b * p.out_stride_b + hd.lr_v_off + t] = Elem<T>::from_float(fx->o_acc[t] * inv_l);
    } else if (t < p.d_head) {
      const float* Ut = p.basis + hd.uvt_off + t;   // (U^V)^T: rp_v x d_head
      float y = 0.f;
#pragma unroll 16
      for (int c = 0; c < hd.rp_v; ++c) y = fmaf(fx->o_acc[c], __ldg(Ut + c * p.d_head), y);
      out[b * p.out_stride_b + static_cast<int64_t>(h) * p.d_head + t] = Elem<T>::from_float(y * inv_l);
    }
  }
  consumer_sync();                    // o_acc, q' and the staging area are reused by the next piece
}

template <typename T>
__global__ void __launch_bounds__(kDecodeThreads, 1) decode_splitkv_kernel(const DecodeParams p) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  DecodeSmemFixed* fx = reinterpret_cast<DecodeSmemFixed*>(smem_raw);
  unsigned char* ring = smem_raw + sizeof(DecodeSmemFixed);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grid = gridDim.x, cta = blockIdx.x;

  if (p.deficit != nullptr) {         // unequal lengths: tiles per sequence, then their exclusive prefix
    for (int b = tid; b < p.B; b += kDecodeThreads) fx->pre[b + 1] = seq_tiles(p, seq_rows(p, b));
    __syncthreads();
    if (warp == 0) {                  // inclusive scan, 32 sequences per step
      int carry = 0;
      for (int base = 0; base < p.B; base += 32) {
        const int b = base + lane;
        int v = b < p.B ? fx->pre[b + 1] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int up = __shfl_up_sync(0xffffffffu, v, d);
          if (lane >= d) v += up;
        }
        if (b < p.B) fx->pre[b + 1] = v + carry;
        carry += __shfl_sync(0xffffffffu, v, 31);
      }
      if (lane == 0) fx->pre[0] = 0;
      __syncwarp();                   // thread 0 reads the prefix right below
    }
  }
  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(&fx->full[s], 1);
      mbar_init(&fx->empty[s], kDecodeConsumerWarps);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&fx->proj_full[i], kHelperThreads);
      mbar_init(&fx->proj_empty[i], kDecodeConsumerWarps * 32);
    }
    fx->abort_flag = 0;
    fx->range[0] = first_tile_of_cta(p, grid, cta);
    fx->range[1] = first_tile_of_cta(p, grid, cta + 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const long long f_lo = fx->range[0], f_hi = fx->range[1];
  volatile int* abort_flag = &fx->abort_flag;

  if (warp >= kDecodeConsumerWarps) {
    // ------------------------------------------------------------ producer (first thread of its warpgroup)
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsProducerGroup));
    if (warp == kDecodeConsumerWarps && lane == 0) {
      const uint64_t policy = policy_evict_first();
      Ring rg;
      bool ok = true;
      long long F = f_lo;
      while (F < f_hi && ok) {
        // one (CTA, unit) piece: tiles [i0, i1) of `unit`; everything per tile below is incremental
        const Piece pc = locate(p, fx->pre, F);
        const int i0 = pc.i0, b = pc.b;
        const int i1 = static_cast<int>(min(static_cast<long long>(pc.nt_u), i0 + (f_hi - F)));
        const HeadInfo hd = p.heads[pc.h];
        const int n_b = seq_rows(p, b);
        int sb, voff, nst, tps;
        ring_geometry<T>(p, hd, &sb, &voff, &nst, &tps);
        if (sb != rg.stage_bytes || nst != rg.stages) {
          // New slot layout: the new slots overlap the old ones differently, so every tile still in the
          // ring must have been released before the first copy into the new layout.
          for (int s2 = 0; s2 < kMaxStages && ok; ++s2)
            if (rg.filled & (1u << s2)) {
              ok = mbar_wait(&fx->empty[s2], (rg.empty_bits >> s2) & 1u, p.status, abort_flag);
              rg.empty_bits ^= 1u << s2;
              rg.filled &= ~(1u << s2);
            }
          if (!ok) { *abort_flag = 1; break; }
          rg.stage = 0; rg.stages = nst; rg.stage_bytes = sb;
        }
        rg.v_off = voff;                  // two heads can share the slot size and still split it differently
        rg.tps = tps;
        const uint32_t rowb_k = hd.rp_k * sizeof(T), rowb_v = hd.rp_v * sizeof(T);
        const int64_t row0 = static_cast<int64_t>(b) * p.n_max + static_cast<int64_t>(i0) * p.tile_rows;
        const char* src_k = p.cache + hd.k_off + row0 * rowb_k;
        const char* src_v = p.cache + hd.v_off + row0 * rowb_v;
        const uint32_t tile_k = p.tile_rows * rowb_k, tile_v = p.tile_rows * rowb_v;
        // paged cache: a tile lies inside one page (tps == 1); its page is looked up one tile ahead, so that the
        // table read has a whole tile's time to come back
        const bool paged = p.pages.table != nullptr;
        int64_t next_phys = paged && i0 < i1 ? physical_row(p.pages, b, p.n_max, i0 * p.tile_rows) : 0;
        for (int i = i0; i < i1; i += tps) {
          if (*abort_flag) { ok = false; break; }
          if (paged) {
            src_k = p.cache + hd.k_off + next_phys * rowb_k;
            src_v = p.cache + hd.v_off + next_phys * rowb_v;
            if (i + 1 < i1) next_phys = physical_row(p.pages, b, p.n_max, (i + 1) * p.tile_rows);
          }
          const int st = rg.stage;
          const uint32_t bit = 1u << st;
          if (rg.filled & bit) {          // the slot's previous tile must have been released
            if (!mbar_wait(&fx->empty[st], (rg.empty_bits >> st) & 1u, p.status, abort_flag)) {
              *abort_flag = 1;
              ok = false;
              break;
            }
            rg.empty_bits ^= bit;
          }
          const int span = min(tps, i1 - i);
          uint32_t bytes_k = span * tile_k, bytes_v = span * tile_v;
          if (i + span == pc.nt_u) {      // the slot ends with the unit's (ragged) last tile
            const uint32_t rows = n_b - i * p.tile_rows;
            bytes_k = rows * rowb_k;
            bytes_v = rows * rowb_v;
          }
          unsigned char* dst = ring + static_cast<size_t>(st) * rg.stage_bytes;
          void* bar = &fx->full[st];
          mbar_arrive_expect_tx(bar, bytes_k + bytes_v);
          if (bytes_k != 0) {             // a sequence without cached rows owns one empty tile
            bulk_g2s_hint(dst, src_k, bytes_k, bar, policy);
            bulk_g2s_hint(dst + rg.v_off, src_v, bytes_v, bar, policy);
          }
          rg.filled |= bit;
          rg.full_bits ^= bit;            // bit now holds the parity of the slot's next fill
          src_k += span * tile_k;
          src_v += span * tile_v;
          rg.advance();
        }
        F += i1 - i0;
      }
      // Make sure every copy this thread issued has landed before the CTA can exit: the latest fill of
      // every slot in use (its phase parity is the opposite of the slot's next one).
      for (int s2 = 0; s2 < kMaxStages; ++s2)
        if (rg.filled & (1u << s2)) mbar_wait(&fx->full[s2], ((rg.full_bits >> s2) & 1u) ^ 1u, p.status);
    } else if (warp > kDecodeConsumerWarps) {
      // -------------------------------------------------------- helper warps: the projections of every piece
      // but a CTA's first, one piece ahead of the consumers (two buffers).  They never leave their loop early: a wait that gave up
      // sets the abort flag and the piece's buffers hold garbage, which the consumers then ignore.
      const int ht = tid - (kDecodeConsumerWarps + 1) * 32;
      long long F = f_lo;
      for (int k = 0; F < f_hi; ++k) {
        const Piece pc = locate(p, fx->pre, F);
        const int i1 = static_cast<int>(min(static_cast<long long>(pc.nt_u), pc.i0 + (f_hi - F)));
        if (k >= 1) {                     // the first piece is the consumers' own
          const HeadInfo hd = p.heads[pc.h];
          const int bufk = k & 1;
          if (k >= 2 && !mbar_wait(&fx->proj_empty[bufk], ((k >> 1) - 1) & 1u, p.status, abort_flag)) *abort_flag = 1;
          project_inputs<T, kHelperThreads>(p, fx, bufk, hd, pc.h, pc.b, ht, p.k_new != nullptr && i1 == pc.nt_u,
                                            seq_rows(p, pc.b));
          mbar_arrive(&fx->proj_full[bufk]);
        }
        F += i1 - pc.i0;
      }
    }
  } else {
    // ------------------------------------------------------------ consumers
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsConsumers));
    Ring rg;
    long long F = f_lo;
    int piece_no = 0;
    while (F < f_hi) {
      const Piece pc = locate(p, fx->pre, F);
      const int i0 = pc.i0, h = pc.h, b = pc.b;
      const long long left = f_hi - F;
      const int i1 = static_cast<int>(min(static_cast<long long>(pc.nt_u), i0 + left));
      const HeadInfo hd = p.heads[h];
      {
        int sb, voff, nst, tps;
        ring_geometry<T>(p, hd, &sb, &voff, &nst, &tps);
        if (sb != rg.stage_bytes || nst != rg.stages) {      // same decision as the producer's
          rg.stage = 0; rg.stages = nst; rg.stage_bytes = sb;
        }
        rg.v_off = voff;
        rg.tps = tps;
      }
      const bool whole = i0 == 0 && i1 == pc.nt_u;
      const bool with_new_row = p.k_new != nullptr && i1 == pc.nt_u;
      const int n_b = seq_rows(p, b);
      const int bufk = piece_no & 1;
      if (piece_no == 0)
        project_inputs<T, kDecodeConsumerWarps * 32>(p, fx, 0, hd, h, b, tid, with_new_row, n_b);
      else if (!mbar_wait(&fx->proj_full[bufk], ((piece_no - 1) >> 1) & 1u, p.status, abort_flag))
        *abort_flag = 1;
      const int mx = max(hd.rp_k, hd.rp_v);
      const int cls = (mx + 15) >> 4;               // a lane pair covers 16 columns per step
      constexpr int MUL = 8 / Elem<T>::kPerChunk;   // 16-byte chunks per 8 columns: 1 (bf16) or 2 (fp32)
      switch (cls) {
        case 1: run_segment<T, 1 * MUL>(p, fx, ring, hd, i0, i1, rg, warp, lane, with_new_row, n_b, bufk); break;
        case 2: run_segment<T, 2 * MUL>(p, fx, ring, hd, i0, i1, rg, warp, lane, with_new_row, n_b, bufk); break;
        case 3: run_segment<T, 3 * MUL>(p, fx, ring, hd, i0, i1, rg, warp, lane, with_new_row, n_b, bufk); break;
        case 4: run_segment<T, 4 * MUL>(p, fx, ring, hd, i0, i1, rg, warp, lane, with_new_row, n_b, bufk); break;
        case 5: run_segment<T, 5 * MUL>(p, fx, ring, hd, i0, i1, rg, warp, lane, with_new_row, n_b, bufk); break;
        case 6: run_segment<T, 6 * MUL>(p, fx, ring, hd, i0, i1, rg, warp, lane, with_new_row, n_b, bufk); break;
        case 7: run_segment<T, 7 * MUL>(p, fx, ring, hd, i0, i1, rg, warp, lane, with_new_row, n_b, bufk); break;
        default: run_segment<T, 8 * MUL>(p, fx, ring, hd, i0, i1, rg, warp, lane, with_new_row, n_b, bufk); break;
      }
      mbar_arrive(&fx->proj_empty[bufk]);           // q' is in registers, the new row has been attended
      finish_piece<T>(p, fx, hd, pc, cta, grid, whole, tid);
      F += i1 - i0;
      ++piece_no;
    }
  }
  __syncthreads();
}

// ---------------------------------------------------------------- combine + lift

template <typename T>
__global__ void __launch_bounds__(128) combine_lift_kernel(const CombineParams p) {
  __shared__ float o_sm[128];
  const int unit = blockIdx.x;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const long long w = hd.rp_k + hd.rp_v;
  long long t0 = static_cast<long long>(b) * p.nt;        // tiles of the head before this unit
  int nt_u = p.nt;
  if (p.deficit != nullptr) {                             // unequal lengths: each sequence has its own tile count
    auto tiles_of = [&](int bb) {
      const int t = (p.n - __ldg(p.deficit + bb) + p.tile_rows - 1) / p.tile_rows;
      return t > 0 ? t : 1;
    };
    t0 = 0;
    for (int bb = 0; bb < b; ++bb) t0 += tiles_of(bb);
    nt_u = tiles_of(b);
  }
  const long long x0 = p.nt_total * hd.w_prefix + t0 * w;
  const long long x1 = x0 + static_cast<long long>(nt_u - 1) * w;
  const int c0 = owner_cta(x0, p.grid, p.w_total);
  const int c1 = owner_cta(x1, p.grid, p.w_total);
  const int t = threadIdx.x;

  // global max and denominator (every thread computes them; the piece count is small)
  float M = -INFINITY;
  for (int c = c0; c <= c1; ++c)
    M = fmaxf(M, p.partials[static_cast<size_t>(unit + c) * p.part_stride]);
  float L = 0.f, acc = 0.f;
  for (int c = c0; c <= c1; ++c) {
    const float* part = p.partials + static_cast<size_t>(unit + c) * p.part_stride;
    const float f = fast_exp2(part[0] - M);
    L = fmaf(part[1], f, L);
    if (t < hd.rp_v) acc = fmaf(part[4 + t], f, acc);
  }
  const float o = acc / L;
  T* out = static_cast<T*>(p.out);
  if (p.flags & 0x2u) {   // rank-space output for a merged W^O'
    if (t < hd.rp_v) out[b * p.out_stride_b + hd.lr_v_off + t] = Elem<T>::from_float(o);
    return;
  }
  if (t < hd.rp_v) o_sm[t] = o;
  __syncthreads();
  if (t < p.d_head) {
    const float* Ut = p.basis + hd.uvt_off;   // (U^V)^T: rp_v x d_head
    float y = 0.f;
#pragma unroll 8
    for (int c = 0; c < hd.rp_v; ++c) y = fmaf(o_sm[c], __ldg(Ut + c * p.d_head + t), y);
    out[b * p.out_stride_b + static_cast<int64_t>(h) * p.d_head + t] = Elem<T>::from_float(y);
  }
}

// Scratch of eigen_attn_decode_static: split-KV partials kept inside the library image, so that the
// call needs no caller-provided scratch.  2048 slots x (4 + 128) floats = 1.03 MiB on every GPU that
// loads the library.  Host code must not pass this name to a kernel: on the host it is only a stand-in
// for the device object; static_partials() asks the runtime for the real device address.
static __device__ __align__(256) float g_static_partials[kStaticPartialFloats];

}  // namespace

// The address is asked for on every call and never kept: the query is a host-side table lookup once the
// library image is loaded on the device (the first call per device loads it, which is why that call belongs
// outside stream capture), it allocates nothing, it needs no lock between host threads, and it stays right
// after a cudaDeviceReset, which would leave a remembered address dangling.
cudaError_t static_partials(float** ptr) {
  float* p = nullptr;
  const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_partials);   // current device
  if (e != cudaSuccess) return e;
  *ptr = p;
  return cudaSuccess;
}

size_t decode_fixed_smem_bytes() { return sizeof(DecodeSmemFixed); }

cudaError_t decode_configure(int dtype) {
  const int max_smem = 227 * 1024;
  if (dtype == 0)
    return cudaFuncSetAttribute(decode_splitkv_kernel<__nv_bfloat16>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
  return cudaFuncSetAttribute(decode_splitkv_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              max_smem);
}

cudaError_t launch_decode(const DecodeParams& p, int dtype, int grid, size_t smem_bytes, cudaStream_t s,
                          uint64_t* launches) {
  if (dtype == 0)
    decode_splitkv_kernel<__nv_bfloat16><<<grid, kDecodeThreads, smem_bytes, s>>>(p);
  else
    decode_splitkv_kernel<float><<<grid, kDecodeThreads, smem_bytes, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_combine(const CombineParams& p, int dtype, cudaStream_t s, uint64_t* launches) {
  const int units = p.B * p.H;
  if (dtype == 0)
    combine_lift_kernel<__nv_bfloat16><<<units, 128, 0, s>>>(p);
  else
    combine_lift_kernel<float><<<units, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
