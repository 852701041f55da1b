// Grouped-query decode on the rank-r cache (the Llama-2-70b / Llama-3 models of Section 5.1 share each K/V head
// among a group of g query heads): one pass over the K'/V' rows of a K/V head serves all g queries of its group,
// so the bytes per query head drop by g and the arithmetic per byte rises by g, which is what makes the
// tensor cores worthwhile for a decode step.
//
// Per tile of 128 cached rows (tcgen05, accumulators in TMEM):
//   S    [128 rows x 16]  = K'_tile [128 x r_k] . Q'^T    Q' = q U^K of the g queries (rows past g are zero), scaled by
//                                                         log2(e)/sqrt(d_h) and rounded to bf16
//   softmax in base 2, one thread per cached row, g running maxima kept identical in every thread (lazy
//   reference: a maximum moves only when it grew by more than 8), P rounded to bf16 into P^T [16 x 128 rows]
//   O'^T [r_v x 16]       += V'_tile^T [r_v x 128 rows] . P^T^T   the rank runs over the TMEM lanes, the queries over
//                                                         16 columns: both operands exist in full (the V' tile is
//                                                         128 elements wide with zeros past the rank, P^T has its 16 rows)
// One CTA per SM with three roles that meet on mbarriers only:
//   * one thread streams the K'/V' tiles by TMA (tensor maps of the cache slabs, 64 x 64 boxes, 128-byte swizzle:
//     the layout the MMA descriptors name, so no thread ever moves a tile) into a ring of three or more stages,
//     about 120 KB in flight;
//   * one thread issues the MMAs: S(t + 1) goes out before the weighted sum of tile t, so it runs under tile t's
//     softmax (S is double-buffered in TMEM, P^T in shared memory);
//   * 128 workers (one per cached row of a tile = one TMEM lane of S; one per rank element = one lane of O'^T).
// A unit split over several CTAs leaves partials (m, l, o') per query that gqa_combine_kernel merges and lifts
// through (U^V)^T.  Every wait is bounded.
#include <cstddef>
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kMaxGroup = 16;                 // query heads per K/V head (N of both products)
constexpr int kGqaThreads = kThreads + 64;    // 128 workers + the MMA-issuing warp + the TMA warp
constexpr int kGqaAtom = kTile * 128;         // one swizzled atom column of a tile: 128 rows x 64 elements
constexpr int kGqaMaxStages = 6;
constexpr int kGqaHeader = 1024;

__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory"); }
// The same barrier, returning the OR of a predicate over the 128 workers: the barrier has no time limit, so the
// decision to leave the tile loop is taken through it and every worker leaves after the same tile.
__device__ __forceinline__ bool worker_sync_or(bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out)
      : "r"(pred ? 1u : 0u), "n"(kThreads)
      : "memory");
  return out != 0;
}

// Warp maximum of a float in one instruction: floats ordered as integers (sign-magnitude -> two's complement).
__device__ __forceinline__ float warp_max(float v) {
  int i = __float_as_int(v);
  i ^= (i >> 31) & 0x7fffffff;
  i = __reduce_max_sync(0xffffffffu, i);
  i ^= (i >> 31) & 0x7fffffff;
  return __int_as_float(i);
}

struct __align__(16) GqaSmemHeader {
  unsigned long long kv_full[kGqaMaxStages], kv_empty[kGqaMaxStages];
  unsigned long long s_done[2], p_ready[2], o_done[2];   // per S / P^T buffer
  unsigned long long q_ready;
  uint32_t tmem_base;
  int abort_flag;
  float red[2][kMaxGroup][4];                 // per query: the four warps' maxima / sums, alternating between tiles
};
static_assert(sizeof(GqaSmemHeader) <= kGqaHeader, "header outgrew its area");
static_assert(offsetof(GqaSmemHeader, red) % 16 == 0, "the maxima are read as float4");

// Instruction descriptor with the A operand MN-major (bit 15) and B K-major: O'^T = V'^T P.
__host__ __device__ constexpr uint32_t instr_desc_a_mn(int n) { return instr_desc(n, false) | (1u << 15); }

// GP: query slots the kernel carries (the group size rounded up to 4, 8 or 16); slots past the group score zero
// queries and are never written out.
template <int GP>
__global__ void __launch_bounds__(kGqaThreads, 1) decode_gqa_kernel(const GqaDecodeParams p, int stages) {
  extern __shared__ __align__(1024) unsigned char smem[];
  GqaSmemHeader* hdr = reinterpret_cast<GqaSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x, split = blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const int G = p.group;
  const HeadInfo hd = p.heads[h];
  const int rpk16 = (hd.rp_k + 15) & ~15, rpv16 = (hd.rp_v + 15) & ~15;
  const int grp_k = (rpk16 >> 3) << 7, grp_p = (kTile >> 3) << 7;
  const int ak = (rpk16 + 63) >> 6, av = (rpv16 + 63) >> 6;  // atom columns (64 elements) the copies fill
  const int k_bytes = ak * kGqaAtom;
  const int stage_bytes = k_bytes + 2 * kGqaAtom;            // the V' part always spans two atom columns (M = 128 of O'^T)
  const int p_bytes = kMaxGroup * kTile * 2;                 // one P^T buffer

  unsigned char* Qs = smem + kGqaHeader;                     // Q' image [16][rk16], canonical (4 KB reserved)
  unsigned char* Ps = Qs + 4096;                             // P^T [2][16 queries][128 rows], canonical
  unsigned char* ring = Ps + 2 * p_bytes;                    // stages x (K' atoms, V' atoms), 128-byte swizzle

  // rows and tiles of this sequence (a batch of unequal lengths gives every sequence its own count; the splits
  // of a unit divide the sequence's own tiles)
  const int n_b = p.deficit != nullptr ? p.n - __ldg(p.deficit + b) : p.n;
  const int nt_b = (n_b + kTile - 1) / kTile;
  const int per = (nt_b + p.splits - 1) / p.splits;
  const int t_lo = split * per, t_hi = min(nt_b, t_lo + per);
  float* part = p.partials + (static_cast<size_t>(unit) * p.splits + split) * G * p.part_stride;
  if (t_lo >= t_hi) {                                        // an empty piece: neutral partials
    for (int qi = 0; qi < G; ++qi) {
      if (tid == 0) { part[qi * p.part_stride] = -INFINITY; part[qi * p.part_stride + 1] = 0.f; }
      if (tid < hd.rp_v) part[qi * p.part_stride + 4 + tid] = 0.f;
    }
    return;
  }
  const int nt = t_hi - t_lo;

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 128);
  if (tid == 0) {
    for (int s = 0; s < kGqaMaxStages; ++s) {
      mbar_init(&hdr->kv_full[s], 1);
      mbar_init(&hdr->kv_empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&hdr->s_done[i], 1);
      mbar_init(&hdr->p_ready[i], kThreads);
      mbar_init(&hdr->o_done[i], 1);
    }
    mbar_init(&hdr->q_ready, kThreads);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Q' and P^T start as zeros (padding rows and columns); a V' atom column that no copy fills must hold zeros too
  for (int idx = tid; idx < (4096 + 2 * p_bytes) / 16; idx += kGqaThreads) reinterpret_cast<uint4*>(Qs)[idx] = make_uint4(0u, 0u, 0u, 0u);
  if (av < 2)
    for (int st = 0; st < stages; ++st)
      for (int idx = tid; idx < kGqaAtom / 16; idx += kGqaThreads)
        reinterpret_cast<uint4*>(ring + st * stage_bytes + k_bytes + kGqaAtom)[idx] = make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  const uint32_t tO = tmem + 64;                             // O'^T: lanes = rank of V, columns = queries
  volatile int* abort_flag = &hdr->abort_flag;
  const int ks_steps = rpk16 >> 4;

  if (warp == 5) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const unsigned char* maps = static_cast<const unsigned char*>(p.tmaps) + static_cast<size_t>(h) * 256;
      const void* map_k = maps;
      const void* map_v = maps + 128;
      tensormap_acquire(map_k);
      tensormap_acquire(map_v);
      const uint32_t tx_bytes = static_cast<uint32_t>((ak + av) * kGqaAtom);   // what the copies of a stage deliver
      bool ok = true;
      int stage = 0, issued = 0;
      uint32_t empty_parity = 1;
      for (int i = 0; i < nt; ++i) {
        if (i >= stages) {
          ok = mbar_wait(&hdr->kv_empty[stage], empty_parity, p.status) && !*abort_flag;
          if (!ok) { *abort_flag = 1; break; }
        }
        unsigned char* st = ring + stage * stage_bytes;
        const int row0 = (t_lo + i) * kTile;
        mbar_arrive_expect_tx(&hdr->kv_full[stage], tx_bytes);
        for (int a = 0; a < ak; ++a)
          for (int hh = 0; hh < 2; ++hh)                     // two boxes of 64 rows fill one atom column of 128 rows
            tma_load_3d(st + a * kGqaAtom + hh * (kGqaAtom / 2), map_k, a * 64, row0 + hh * 64, b, &hdr->kv_full[stage]);
        for (int a = 0; a < av; ++a)
          for (int hh = 0; hh < 2; ++hh)
            tma_load_3d(st + k_bytes + a * kGqaAtom + hh * (kGqaAtom / 2), map_v, a * 64, row0 + hh * 64, b, &hdr->kv_full[stage]);
        ++issued;
        if (++stage == stages) { stage = 0; empty_parity ^= 1u; }
      }
      // if the CTA gives up, its copies in flight must land before it leaves
      if (!ok || *abort_flag) {
        for (int s2 = 0; s2 < stages; ++s2) {
          int last = -1;
          for (int jj = s2; jj < issued; jj += stages) last = jj;
          if (last >= 0) mbar_wait(&hdr->kv_full[s2], (last / stages) & 1u, p.status);
        }
      }
    }
  } else if (warp == 4) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = instr_desc(kMaxGroup, false);
      const uint32_t idesc_o = instr_desc_a_mn(kMaxGroup);
      const uint32_t ra = smem_u32(ring);
      const uint64_t dk0 = smem_desc_sw128(ra, 16, 1024);                      // K' tile of stage 0: A, K-major
      const uint64_t dv0 = smem_desc_sw128(ra + k_bytes, kGqaAtom, 1024);      // V' tile of stage 0: A, MN-major
      const uint64_t dq = smem_desc(smem_u32(Qs), 128, grp_k);                 // Q': B, K-major, 16 rows
      const uint64_t dp0 = smem_desc(smem_u32(Ps), 128, grp_p);                // P^T: B, K-major, 16 rows
      const uint64_t stage_step = static_cast<uint64_t>(stage_bytes >> 4);
      bool ok = mbar_wait(&hdr->q_ready, 0, p.status);
      int s_stage = 0;
      uint32_t s_parity = 0;
      auto issue_s = [&](int buf) {                          // S(next tile in the ring) into score buffer `buf`
        ok = mbar_wait(&hdr->kv_full[s_stage], s_parity, p.status);
        if (!ok) return;
        tc_fence_after();
        const uint64_t dk = dk0 + s_stage * stage_step;
        for (int s = 0; s < ks_steps; ++s)
          mma_ss(tmem + 32 * buf, dk + (s >> 2) * (kGqaAtom >> 4) + (s & 3) * 2, dq + s * 16, idesc_s, s > 0);
        mma_commit(&hdr->s_done[buf]);
        if (++s_stage == stages) { s_stage = 0; s_parity ^= 1u; }
      };
      if (ok) issue_s(0);
      int stage = 0;
      for (int i = 0; i < nt && ok; ++i) {
        const int buf = i & 1;
        const uint32_t par = (i >> 1) & 1u;
        if (i + 1 < nt) {                                    // S(i + 1) runs under the softmax of tile i
          issue_s(buf ^ 1);
          if (!ok) break;
        }
        ok = mbar_wait(&hdr->p_ready[buf], par, p.status) && !*abort_flag;     // P^T(i) written, O'^T rescaled if needed
        if (!ok) break;
        tc_fence_after();
        const uint64_t dv = dv0 + stage * stage_step, dp = dp0 + static_cast<uint64_t>(buf) * (p_bytes >> 4);
#pragma unroll
        for (int s = 0; s < kTile / 16; ++s)                 // O'^T += V'(i)^T P(i), 16 cached rows a step
          mma_ss(tO, dv + s * (2048 >> 4), dp + s * 16, idesc_o, i > 0 || s > 0);
        mma_commit(&hdr->o_done[buf]);
        mma_commit(&hdr->kv_empty[stage]);                   // the weighted sum is the stage's last reader
        if (++stage == stages) stage = 0;
      }
      // the last commits' arrivals must have landed before the CTA may leave
      if (ok) ok = mbar_wait(&hdr->kv_empty[(nt - 1) % stages], ((nt - 1) / stages) & 1u, p.status);
      if (!ok) *abort_flag = 1;
    }
  }
  if (warp >= 4) {
    __syncthreads();                                         // the workers' epilogue
    __syncthreads();
    return;
  }

  // -------------------------------------------------------------------- the 128 workers
  // Q' = q U^K for the g queries of the group, times log2(e)/sqrt(d_h), rounded to bf16
  {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + b * p.q_stride_b +
                              static_cast<int64_t>(h) * G * p.d_head;
    const float* U = p.basis + hd.uk_off;                    // d_head x rp_k, zero padded columns
    // The queries go through shared memory as fp32 (the P^T buffers are idle until the first tile), a thread owns
    // column c of U^K for all queries of the group, 32 loads of U in flight: the projection costs a few
    // microseconds per CTA, and every CTA pays it before its first product.
    float* qs = reinterpret_cast<float*>(Ps);                // [G][d_head]
    for (int idx = tid; idx < G * p.d_head; idx += kThreads) qs[idx] = __bfloat162float(qg[idx]);
    worker_sync();
    for (int c = tid; c < hd.rp_k; c += kThreads) {
      float acc[GP];
#pragma unroll
      for (int qi = 0; qi < GP; ++qi) acc[qi] = 0.f;
#pragma unroll 32
      for (int d = 0; d < p.d_head; ++d) {
        const float u = __ldg(U + d * hd.rp_k + c);
#pragma unroll
        for (int qi = 0; qi < GP; ++qi)
          if (qi < G) acc[qi] = fmaf(qs[qi * p.d_head + d], u, acc[qi]);
      }
#pragma unroll
      for (int qi = 0; qi < GP; ++qi)
        if (qi < G)
          *reinterpret_cast<__nv_bfloat16*>(Qs + chunk_off(qi, c >> 3, grp_k) + (c & 7) * 2) = __float2bfloat16_rn(acc[qi] * p.q_scale);
    }
    worker_sync();                                           // every thread is done reading the staged queries
    for (int idx = tid; idx < (2 * p_bytes) / 16; idx += kThreads) reinterpret_cast<uint4*>(Ps)[idx] = make_uint4(0u, 0u, 0u, 0u);
    fence_async_smem();
    mbar_arrive(&hdr->q_ready);
  }
  const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
  float m_run[GP], l_thr[GP];
#pragma unroll
  for (int qi = 0; qi < GP; ++qi) { m_run[qi] = -INFINITY; l_thr[qi] = 0.f; }
  bool ok = true;

  for (int i = 0; i < nt; ++i) {
    const int t = t_lo + i, buf = i & 1;
    const uint32_t par = (i >> 1) & 1u;
    if (!mbar_wait(&hdr->s_done[buf], par, p.status)) *abort_flag = 1;
    tc_fence_after();
    uint32_t sr[16];
    tmem_ld16(tmem + lane_base + 32 * buf, sr);
    tmem_wait_ld();
    const bool live = t * kTile + tid < n_b;
    // ---- per-query maximum over the tile: one reduction instruction per query and warp, lane q keeps query q's
#pragma unroll
    for (int qi = 0; qi < GP; ++qi) {
      const float v = warp_max(live ? __uint_as_float(sr[qi]) : -INFINITY);
      if (lane == qi) hdr->red[buf][qi][warp] = v;
    }
    // the P^T buffer of this tile was read by the weighted sum of tile i - 2
    if (i >= 2 && !mbar_wait(&hdr->o_done[buf], par ^ 1u, p.status)) *abort_flag = 1;
    if (worker_sync_or(*abort_flag != 0)) { ok = false; break; }   // some role gave up: all workers leave here
    // lazy reference: m_run follows the maximum only when that grew by more than 8 (every thread decides alike)
    unsigned char* Pb = Ps + buf * p_bytes;
    float alpha[GP];
    bool rescale = false;
#pragma unroll
    for (int qi = 0; qi < GP; ++qi) {
      const float4 r4 = *reinterpret_cast<const float4*>(&hdr->red[buf][qi][0]);
      const float tm = fmaxf(fmaxf(r4.x, r4.y), fmaxf(r4.z, r4.w));
      alpha[qi] = 1.f;
      if (tm > m_run[qi] + 8.f) {
        alpha[qi] = ex2(m_run[qi] - tm);
        m_run[qi] = tm;
        rescale = rescale || i > 0;
      }
      const float pj = live ? ex2(__uint_as_float(sr[qi]) - m_run[qi]) : 0.f;
      l_thr[qi] = fmaf(l_thr[qi], alpha[qi], pj);
      *reinterpret_cast<__nv_bfloat16*>(Pb + chunk_off(qi, tid >> 3, grp_p) + (tid & 7) * 2) = __float2bfloat16_rn(pj);
    }
    if (rescale) {                                           // uniform over the workers; this thread's lane of O'^T
      if (!mbar_wait(&hdr->o_done[buf ^ 1], ((i - 1) >> 1) & 1u, p.status)) *abort_flag = 1;   // the sum of tile i - 1 is in
      tc_fence_after();
      uint32_t o[16];
      tmem_ld16(tO + lane_base, o);
      tmem_wait_ld();
#pragma unroll
      for (int qi = 0; qi < GP; ++qi) o[qi] = __float_as_uint(__uint_as_float(o[qi]) * alpha[qi]);
      tmem_st16(tO + lane_base, o);
      tmem_wait_st();
    }
    fence_async_smem();
    tc_fence_before();
    mbar_arrive(&hdr->p_ready[buf]);                         // the issuer sends the weighted sum of this tile off
  }
  if (ok) {
    if (!mbar_wait(&hdr->o_done[(nt - 1) & 1], ((nt - 1) >> 1) & 1u, p.status)) ok = false;
  }
  if (!ok) *abort_flag = 1;
  tc_fence_after();
  worker_sync();                                             // every worker is done with the last tile's maxima

  // ---- partials per query: m, l (summed over the threads' rows), o' (column `query` of O'^T)
#pragma unroll
  for (int qi = 0; qi < GP; ++qi) {
    float v = l_thr[qi];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) hdr->red[0][qi][warp] = v;
  }
  __syncthreads();
  if (tid < G) {
    float mine_m = -INFINITY;
#pragma unroll
    for (int qi = 0; qi < GP; ++qi) mine_m = tid == qi ? m_run[qi] : mine_m;
    part[tid * p.part_stride] = mine_m;
    part[tid * p.part_stride + 1] = (hdr->red[0][tid][0] + hdr->red[0][tid][1]) + (hdr->red[0][tid][2] + hdr->red[0][tid][3]);
  }
  {
    uint32_t o[16];
    tmem_ld16(tO + lane_base, o);
    tmem_wait_ld();
    if (tid < hd.rp_v)
      for (int qi = 0; qi < G; ++qi) part[qi * p.part_stride + 4 + tid] = __uint_as_float(o[qi]);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 128);
}

// Merges the partials of one query head and lifts o'/l through (U^V)^T of its K/V head.
__global__ void __launch_bounds__(128) gqa_combine_kernel(const GqaDecodeParams p) {
  __shared__ float o_sm[128];
  const int unit = blockIdx.x / p.group, qi = blockIdx.x - unit * p.group, t = threadIdx.x;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const float* base = p.partials + (static_cast<size_t>(unit) * p.splits * p.group + qi) * p.part_stride;
  const size_t step = static_cast<size_t>(p.group) * p.part_stride;
  float M = -INFINITY;
  for (int c = 0; c < p.splits; ++c) M = fmaxf(M, base[c * step]);
  float L = 0.f, acc = 0.f;
  for (int c = 0; c < p.splits; ++c) {
    const float* part = base + c * step;
    const float f = ex2(part[0] - M);                        // 0 for an empty piece
    L = fmaf(part[1], f, L);
    if (t < hd.rp_v) acc = fmaf(part[4 + t], f, acc);
  }
  if (t < hd.rp_v) o_sm[t] = acc / L;
  __syncthreads();
  if (t < p.d_head) {
    const float* Ut = p.basis + hd.uvt_off;                  // (U^V)^T : rp_v x d_head
    float y = 0.f;
    for (int c = 0; c < hd.rp_v; ++c) y = fmaf(o_sm[c], __ldg(Ut + c * p.d_head + t), y);
    static_cast<__nv_bfloat16*>(p.out)[b * p.out_stride_b + (static_cast<int64_t>(h) * p.group + qi) * p.d_head + t] =
        __float2bfloat16_rn(y);
  }
}

// ---------------------------------------------------------------------------------------------------------------
// Grouped queries with a rotary position embedding (Section 4.3 for the models of Section 5.1 that share K/V heads
// and rotate their keys), on the tensor cores.
//
// Per tile of 128 cached rows of a K/V head:
//   X     [128 x d_h]  = K'_tile (U^K)^T                      the lift (tcgen05, bf16 image of U^K in shared memory)
//   Y_l   = E_l X_l     (pairwise complex product, E_l = e^{i l phi})   each key row turned by its offset inside the tile,
//                                                             rounded to fp16 into a K-major operand tile in shared memory
//                                                             (fp16, not bf16: both operands of the score product are
//                                                             written here, and the three extra mantissa bits keep peaked
//                                                             softmax weights inside the tolerance; the turned keys and the
//                                                             scaled queries must stay inside fp16's range, 65504)
//   S     [128 x 16]   = Y . Qt^T                             Qt = q e^{i (p - 128 t) phi} log2(e)/sqrt(d_h) of the g queries:
//                                                             the tile's share of the angle sits on the queries, which a
//                                                             recurrence turns by e^{-i 128 phi} per tile (fp32 state,
//                                                             renormalised), so a key costs 2 packed operations per pair
//   softmax and O'^T += V'^T P exactly as in decode_gqa_kernel.
// Re(Qt conj(Y)) = Re(q e^{i (p - j) phi} conj(X)) for row j = 128 t + l: the rotated dot product of Section 4.3.
//
// Roles: sixteen worker warps (four threads per cached row turn the keys: warps w, w + 4, w + 8, w + 12 share a TMEM lane
// quadrant and take every fourth chunk of eight pairs; warps 0-3 then run the softmax of the tile before, one thread per
// row: with one CTA per SM it takes this many warps to cover the latencies of the TMEM reads and of the arithmetic), one
// thread issuing the score and weighted-sum products (scores of tile i, weighted sum of tile i - 1 per round), one
// thread issuing the lifts (a tile ahead), one thread
// streaming K' tiles (two buffers, free again as soon as their lift is complete) and V' tiles (two buffers) by TMA.
// Everything meets on mbarriers; the softmax warps' loop exit goes through their reducing barrier.

constexpr int kGrWorkers = 512;
constexpr int kGrThreads = kGrWorkers + 96;   // + the warp issuing scores and weighted sums, the TMA warp, the warp issuing lifts
constexpr int kGrHeader = 3072;
constexpr double kGrTwoPi = 6.283185307179586476925286766559;

struct __align__(16) GrSmemHeader {
  unsigned long long k_full[2], x_full[2], kr_ready[2], s_done[2], p_ready[2], o_done[2], v_full[2], v_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  alignas(16) float red[2][kMaxGroup][4];     // per query: the four softmax warps' maxima / sums, alternating between tiles
                                              // (read 16 bytes at a time)
};
static_assert(sizeof(GrSmemHeader) <= kGrHeader, "header outgrew its area");
static_assert(offsetof(GrSmemHeader, red) % 16 == 0, "the maxima are read as float4");

__host__ __device__ constexpr int gr_kb(int bytes) { return (bytes + 1023) & ~1023; }

template <int GP, bool INTERLEAVED>
__global__ void __launch_bounds__(kGrThreads, 1) decode_gqa_rope_kernel(const GqaDecodeParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  GrSmemHeader* hdr = reinterpret_cast<GrSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x, split = blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const int G = p.group;
  const HeadInfo hd = p.heads[h];
  const int dh = p.d_head, half = dh >> 1;
  const int rpk16 = (hd.rp_k + 15) & ~15, rpv16 = (hd.rp_v + 15) & ~15;
  const int grp_k = (rpk16 >> 3) << 7, grp_d = (dh >> 3) << 7, grp_p = (kTile >> 3) << 7;
  const int ak = (rpk16 + 63) >> 6, av = (rpv16 + 63) >> 6;  // atom columns (64 elements) the copies fill
  const int k_bytes = ak * kGqaAtom, v_bytes = 2 * kGqaAtom; // the V' tile always spans two atom columns (M = 128 of O'^T)
  const int u_bytes = dh * rpk16 * 2;
  const int q_bytes = kMaxGroup * dh * 2;                    // one Qt image (16 rows, canonical)
  const int p_bytes = kMaxGroup * kTile * 2;                 // one P^T buffer
  const int y_bytes = kTile * dh * 2;                        // one Y tile (128 rows, canonical)

  unsigned char* Qs = smem + kGrHeader;                      // Qt [16][d_h], canonical (one buffer: see rotate_tile)
  unsigned char* Ps = Qs + gr_kb(q_bytes);                   // P^T [2][16 queries][128 rows], canonical
  unsigned char* Us = Ps + 2 * p_bytes;                      // U^K image, canonical
  unsigned char* Ys = Us + gr_kb(u_bytes);                   // Y [2]
  unsigned char* Kr = Ys + 2 * y_bytes;                      // K' tiles [2], 128-byte swizzle
  unsigned char* Vr = Kr + 2 * k_bytes;                      // V' tiles [2], 128-byte swizzle

  const int n_b = p.deficit != nullptr ? p.n - __ldg(p.deficit + b) : p.n;
  const int nt_b = (n_b + kTile - 1) / kTile;
  const int per = (nt_b + p.splits - 1) / p.splits;
  const int t_lo = split * per, t_hi = min(nt_b, t_lo + per);
  float* part = p.partials + (static_cast<size_t>(unit) * p.splits + split) * G * p.part_stride;
  if (t_lo >= t_hi) {                                        // an empty piece: neutral partials
    for (int qi = 0; qi < G; ++qi) {
      if (tid == 0) { part[qi * p.part_stride] = -INFINITY; part[qi * p.part_stride + 1] = 0.f; }
      if (tid < hd.rp_v) part[qi * p.part_stride + 4 + tid] = 0.f;
    }
    return;
  }
  const int nt = t_hi - t_lo;

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 512);           // X[2] (128 columns each), S[2] (32), O'^T (16)
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&hdr->k_full[i], 1);
      mbar_init(&hdr->x_full[i], 1);
      mbar_init(&hdr->kr_ready[i], kGrWorkers / 32);         // one arrival per worker warp
      mbar_init(&hdr->s_done[i], 1);
      mbar_init(&hdr->p_ready[i], kThreads);
      mbar_init(&hdr->o_done[i], 1);
      mbar_init(&hdr->v_full[i], 1);
      mbar_init(&hdr->v_empty[i], 1);
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  {
    const uint4* Ug = reinterpret_cast<const uint4*>(p.basis + hd.ukl16_off);
    for (int idx = tid; idx < u_bytes / 16; idx += kGrThreads) cp_async16(Us + idx * 16, Ug + idx, 16u);
    cp_async_commit();
  }
  // Qt and P^T start as zeros (rows of queries past the group, padding); a V' atom column that no copy fills too
  for (int idx = tid; idx < (gr_kb(q_bytes) + 2 * p_bytes) / 16; idx += kGrThreads) reinterpret_cast<uint4*>(Qs)[idx] = make_uint4(0u, 0u, 0u, 0u);
  if (av < 2)
    for (int st = 0; st < 2; ++st)
      for (int idx = tid; idx < kGqaAtom / 16; idx += kGrThreads)
        reinterpret_cast<uint4*>(Vr + st * v_bytes + kGqaAtom)[idx] = make_uint4(0u, 0u, 0u, 0u);
  cp_async_wait<0>();
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  const uint32_t tS = tmem + 256, tO = tmem + 320;           // S buffers at +0 / +32; O'^T: lanes = rank of V, columns = queries
  volatile int* abort_flag = &hdr->abort_flag;
  if (warp == kGrWorkers / 32 + 1) {
    // ------------------------------------------------------------------ TMA producer: K' runs a tile ahead of V'
    if (lane == 0) {
      const unsigned char* maps = static_cast<const unsigned char*>(p.tmaps) + static_cast<size_t>(h) * 256;
      const void* map_k = maps;
      const void* map_v = maps + 128;
      tensormap_acquire(map_k);
      tensormap_acquire(map_v);
      bool ok = true;
      auto fetch_k = [&](int i) {                            // buffer i & 1 is free once the lift of tile i - 2 is complete
        if (i >= 2) ok = mbar_wait(&hdr->x_full[i & 1], ((i - 2) >> 1) & 1u, p.status) && !*abort_flag;
        if (!ok) return;
        unsigned char* dst = Kr + (i & 1) * k_bytes;
        const int row0 = (t_lo + i) * kTile;
        mbar_arrive_expect_tx(&hdr->k_full[i & 1], static_cast<uint32_t>(k_bytes));
        for (int a = 0; a < ak; ++a)
          for (int hh = 0; hh < 2; ++hh)                     // two boxes of 64 rows fill one atom column of 128 rows
            tma_load_3d(dst + a * kGqaAtom + hh * (kGqaAtom / 2), map_k, a * 64, row0 + hh * 64, b, &hdr->k_full[i & 1]);
      };
      auto fetch_v = [&](int i) {                            // ... once the weighted sum of tile i - 2 is complete
        if (i >= 2) ok = mbar_wait(&hdr->v_empty[i & 1], ((i - 2) >> 1) & 1u, p.status) && !*abort_flag;
        if (!ok) return;
        unsigned char* dst = Vr + (i & 1) * v_bytes;
        const int row0 = (t_lo + i) * kTile;
        mbar_arrive_expect_tx(&hdr->v_full[i & 1], static_cast<uint32_t>(av * kGqaAtom));
        for (int a = 0; a < av; ++a)
          for (int hh = 0; hh < 2; ++hh)
            tma_load_3d(dst + a * kGqaAtom + hh * (kGqaAtom / 2), map_v, a * 64, row0 + hh * 64, b, &hdr->v_full[i & 1]);
      };
      int k_issued = 0, v_issued = 0;
      fetch_k(0);
      k_issued = 1;
      for (int i = 0; i < nt && ok; ++i) {
        if (i + 1 < nt) { fetch_k(i + 1); if (ok) ++k_issued; }
        if (ok) { fetch_v(i); if (ok) ++v_issued; }
      }
      if (!ok || *abort_flag) {                              // the CTA gives up: its copies in flight must land first
        *abort_flag = 1;
        for (int j = max(0, k_issued - 2); j < k_issued; ++j) mbar_wait(&hdr->k_full[j & 1], (j >> 1) & 1u, p.status);
        for (int j = max(0, v_issued - 2); j < v_issued; ++j) mbar_wait(&hdr->v_full[j & 1], (j >> 1) & 1u, p.status);
      }
    }
  } else if (warp == kGrWorkers / 32) {
    // ------------------------------------------------------------------ MMA issuer
    // round r: the scores of tile r, the weighted sum of tile r - 1 (the lifts come from a thread of their own, so that
    // neither waits for the other's hand-overs)
    if (lane == 0) {
      const uint32_t idesc_s = instr_desc_f16(kMaxGroup);                      // Y and Qt are fp16 (see the head of this part)
      const uint32_t idesc_o = instr_desc_a_mn(kMaxGroup);
      bool ok = true;
      auto scores = [&](int i) {                             // S(i) = Y(i) Qt(i)^T: both written by the workers
        ok = mbar_wait(&hdr->kr_ready[i & 1], (i >> 1) & 1u, p.status);
        if (!ok) return;
        tc_fence_after();
        const uint64_t dy = smem_desc(smem_u32(Ys + (i & 1) * y_bytes), 128, grp_d);
        const uint64_t dq = smem_desc(smem_u32(Qs), 128, grp_d);
        for (int s = 0; s < (dh >> 4); ++s)
          mma_ss(tS + 32 * (i & 1), dy + s * 16, dq + s * 16, idesc_s, s > 0);
        mma_commit(&hdr->s_done[i & 1]);
      };
      auto weighted_sum = [&](int i) {                       // O'^T += V'(i)^T P(i), 16 cached rows a step
        ok = mbar_wait(&hdr->p_ready[i & 1], (i >> 1) & 1u, p.status) && !*abort_flag;
        if (ok) ok = mbar_wait(&hdr->v_full[i & 1], (i >> 1) & 1u, p.status);
        if (!ok) return;
        tc_fence_after();
        const uint64_t dv = smem_desc_sw128(smem_u32(Vr + (i & 1) * v_bytes), kGqaAtom, 1024);
        const uint64_t dp = smem_desc(smem_u32(Ps + (i & 1) * p_bytes), 128, grp_p);
#pragma unroll
        for (int s = 0; s < kTile / 16; ++s)
          mma_ss(tO, dv + s * (2048 >> 4), dp + s * 16, idesc_o, i > 0 || s > 0);
        mma_commit(&hdr->o_done[i & 1]);
        mma_commit(&hdr->v_empty[i & 1]);
      };
      for (int r = 0; r <= nt && ok; ++r) {
        if (r < nt) scores(r);
        if (ok && r >= 1) weighted_sum(r - 1);
      }
      // the last commits' arrivals must have landed before the CTA may leave
      if (ok) ok = mbar_wait(&hdr->v_empty[(nt - 1) & 1], ((nt - 1) >> 1) & 1u, p.status);
      if (!ok) *abort_flag = 1;
    }
  }
  else if (warp == kGrWorkers / 32 + 2) {
    // ------------------------------------------------------------------ lift issuer: X(i) = K'(i) (U^K)^T
    if (lane == 0) {
      const uint32_t idesc_l = instr_desc(dh, false);
      const uint64_t du = smem_desc(smem_u32(Us), 128, grp_k);                 // U^K image: B of the lift
      bool ok = true;
      for (int i = 0; i < nt && ok; ++i) {
        ok = mbar_wait(&hdr->k_full[i & 1], (i >> 1) & 1u, p.status) && !*abort_flag;
        if (ok && i >= 2) ok = mbar_wait(&hdr->kr_ready[i & 1], ((i - 2) >> 1) & 1u, p.status);   // X(i - 2) has been read
        if (!ok) break;
        tc_fence_after();
        const uint64_t dk = smem_desc_sw128(smem_u32(Kr + (i & 1) * k_bytes), 16, 1024);
        for (int s = 0; s < (rpk16 >> 4); ++s)
          mma_ss(tmem + (i & 1) * kTile, dk + (s >> 2) * (kGqaAtom >> 4) + (s & 3) * 2, du + s * 16, idesc_l, s > 0);
        mma_commit(&hdr->x_full[i & 1]);
      }
      if (!ok) *abort_flag = 1;
    }
  }
  if (warp >= kGrWorkers / 32) {
    __syncthreads();                                         // the workers' epilogue
    __syncthreads();
    return;
  }
  // -------------------------------------------------------------------- the 512 workers
  // Thread (row, qd): row = 32 (warp & 3) + lane is its TMEM lane, qd = warp >> 2 picks the chunks of eight pairs
  // 4m + qd (m = 0, 1); E_l = e^{i row phi} for those pairs from the layer's table: cos, sin and -sin
  const int row = (warp & 3) * 32 + lane, qd = warp >> 2;
  unsigned long long el_c[8], el_s[8], el_n[8];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float4 c = __ldg(p.el_table + ((4 * m + qd) * 4 + e) * kTile + row);
      el_c[4 * m + e] = pack2(c.x, c.y);
      el_s[4 * m + e] = pack2(c.z, c.w);
      el_n[4 * m + e] = pack2(-c.z, -c.w);
    }
  // The queries: thread tid owns query tid >> 5 and the two pairs 2 (tid & 31), + 1, scaled by log2(e)/sqrt(d_h) and
  // turned to the first tile's offset (the angle reduced in fp64), then by e^{-i 128 phi} per tile
  const int qi_own = tid >> 5, i0 = (tid & 31) * 2;
  const bool q_on = qi_own < G && i0 < half;
  float q_re[2], q_im[2], st_c[2], st_s[2], q_n2[2];
#pragma unroll
  for (int k = 0; k < 2; ++k) { q_re[k] = q_im[k] = 0.f; st_c[k] = 1.f; st_s[k] = 0.f; q_n2[k] = 1.f; }
  if (q_on) {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + b * p.q_stride_b +
                              (static_cast<int64_t>(h) * G + qi_own) * dh;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int i = i0 + k;
      const int ia = INTERLEAVED ? 2 * i : i, ib = INTERLEAVED ? 2 * i + 1 : i + half;
      const float a_re = __bfloat162float(qg[ia]) * p.q_scale, a_im = __bfloat162float(qg[ib]) * p.q_scale;
      double ang = static_cast<double>(n_b - 1 - t_lo * kTile) * p.inv_freq[i];
      ang -= kGrTwoPi * rint(ang / kGrTwoPi);
      float s_, c_;
      sincosf(static_cast<float>(ang), &s_, &c_);
      q_re[k] = a_re * c_ - a_im * s_;
      q_im[k] = a_re * s_ + a_im * c_;
      q_n2[k] = fmaxf(a_re * a_re + a_im * a_im, 1e-30f);
      const float2 st = __ldg(p.tile_step + i);
      st_c[k] = st.x;
      st_s[k] = st.y;
    }
  }
  const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
  const int im_chunk0 = half >> 3;                           // first 16-byte chunk of the imaginary halves (pairs (i, i + d_h/2))

  // One tile's keys turned and written as the A operand of the score product, and the tile's queries beside them
  auto rotate_tile = [&](int it) -> bool {
    const uint32_t par = it & 1u;
    bool have = mbar_wait(&hdr->x_full[par], (it >> 1) & 1u, p.status);
    if (have && it >= 2) have = mbar_wait(&hdr->s_done[par], ((it - 2) >> 1) & 1u, p.status);   // Y, Qt of tile it - 2 were read
    if (!have) { *abort_flag = 1; return false; }
    tc_fence_after();
    const uint32_t tX = tmem + lane_base + par * kTile;
    unsigned char* Yb = Ys + par * y_bytes;
#pragma unroll
    for (int m = 0; m < 2; ++m) {
      const int c = 4 * m + qd;
      if (8 * c < half) {
        uint32_t xc[16];                                     // re[8], im[8] (pairs (i, i + d_h/2)) or re, im alternating
        if (INTERLEAVED) {
          tmem_ld16(tX + 16 * c, xc);
        } else {
          tmem_ld8(tX + 8 * c, *reinterpret_cast<uint32_t(*)[8]>(&xc[0]));
          tmem_ld8(tX + half + 8 * c, *reinterpret_cast<uint32_t(*)[8]>(&xc[8]));
        }
        tmem_wait_ld();
        uint32_t w[8];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
          unsigned long long x_re, x_im;
          if (INTERLEAVED) {
            x_re = pack2(__uint_as_float(xc[2 * e]), __uint_as_float(xc[2 * e + 2]));
            x_im = pack2(__uint_as_float(xc[2 * e + 1]), __uint_as_float(xc[2 * e + 3]));
          } else {
            x_re = pack2(__uint_as_float(xc[e]), __uint_as_float(xc[e + 1]));
            x_im = pack2(__uint_as_float(xc[8 + e]), __uint_as_float(xc[8 + e + 1]));
          }
          const unsigned long long er = el_c[4 * m + (e >> 1)], ei = el_s[4 * m + (e >> 1)], en = el_n[4 * m + (e >> 1)];
          const unsigned long long yr = fma2p(er, x_re, mul2p(en, x_im));      // Y = E_l X
          const unsigned long long yi = fma2p(er, x_im, mul2p(ei, x_re));
          float r0, r1, i0_, i1_;
          unpack2(yr, r0, r1);
          unpack2(yi, i0_, i1_);
          if (INTERLEAVED) {
            w[e] = pack_f16(r0, i0_);
            w[e + 1] = pack_f16(r1, i1_);
          } else {
            w[e >> 1] = pack_f16(r0, r1);
            w[4 + (e >> 1)] = pack_f16(i0_, i1_);
          }
        }
        const int ca = INTERLEAVED ? 2 * c : c, cb = INTERLEAVED ? 2 * c + 1 : im_chunk0 + c;
        *reinterpret_cast<uint4*>(Yb + chunk_off(row, ca, grp_d)) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(Yb + chunk_off(row, cb, grp_d)) = make_uint4(w[4], w[5], w[6], w[7]);
      }
    }
    // Qt of this tile (one buffer: the scores of the tile before, issued a whole key turning ago, must have read
    // theirs), then one more turn by -128 phi
    if (it >= 1 && !mbar_wait(&hdr->s_done[par ^ 1u], ((it - 1) >> 1) & 1u, p.status)) { *abort_flag = 1; return false; }
    if (q_on) {
      unsigned char* Qb = Qs;
      if (INTERLEAVED) {                                     // dims 2 i0 .. 2 i0 + 3: re, im, re, im
        *reinterpret_cast<uint2*>(Qb + chunk_off(qi_own, i0 >> 2, grp_d) + (i0 & 3) * 4) =
            make_uint2(pack_f16(q_re[0], q_im[0]), pack_f16(q_re[1], q_im[1]));
      } else {                                               // dims i0, i0 + 1 and d_h/2 + i0, + 1
        *reinterpret_cast<uint32_t*>(Qb + chunk_off(qi_own, i0 >> 3, grp_d) + (i0 & 7) * 2) = pack_f16(q_re[0], q_re[1]);
        *reinterpret_cast<uint32_t*>(Qb + chunk_off(qi_own, im_chunk0 + (i0 >> 3), grp_d) + (i0 & 7) * 2) = pack_f16(q_im[0], q_im[1]);
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const float n_re = q_re[k] * st_c[k] - q_im[k] * st_s[k], n_im = q_re[k] * st_s[k] + q_im[k] * st_c[k];
        const float fix = 1.5f - 0.5f * (n_re * n_re + n_im * n_im) / q_n2[k];   // ~ |q| / |n|: no drift over many tiles
        q_re[k] = n_re * fix;
        q_im[k] = n_im * fix;
      }
    }
    fence_async_smem();
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&hdr->kr_ready[par]);
    return true;
  };
  if (warp >= 4) {
    // warps 4-15 only turn keys (their barriers are mbarriers with a time limit: each may leave on its own)
    for (int it = 0; it < nt; ++it)
      if (!rotate_tile(it)) break;
    __syncthreads();                                         // the softmax warps' epilogue
    __syncthreads();
    return;
  }

  // warps 0-3: the keys of tile `it`, then the softmax of tile it - 1 (its scores ran under the turning of tile it)
  float m_run[GP], l_thr[GP];
#pragma unroll
  for (int qi = 0; qi < GP; ++qi) { m_run[qi] = -INFINITY; l_thr[qi] = 0.f; }
  bool ok = true;
  for (int it = 0; it <= nt; ++it) {
    if (it < nt) rotate_tile(it);                            // a wait that gave up shows at the barrier below
    if (it == 0) continue;
    const int i = it - 1, t = t_lo + i, buf = i & 1;
    const uint32_t par = (i >> 1) & 1u;
    if (!mbar_wait(&hdr->s_done[buf], par, p.status)) *abort_flag = 1;
    tc_fence_after();
    uint32_t sr[16];
    tmem_ld16(tS + lane_base + 32 * buf, sr);
    tmem_wait_ld();
    const bool live = t * kTile + tid < n_b;
    // ---- per-query maximum over the tile: one reduction instruction per query and warp, lane q keeps query q's
#pragma unroll
    for (int qi = 0; qi < GP; ++qi) {
      const float v = warp_max(live ? __uint_as_float(sr[qi]) : -INFINITY);
      if (lane == qi) hdr->red[buf][qi][warp] = v;
    }
    // the P^T buffer of this tile was read by the weighted sum of tile i - 2
    if (i >= 2 && !mbar_wait(&hdr->o_done[buf], par ^ 1u, p.status)) *abort_flag = 1;
    if (worker_sync_or(*abort_flag != 0)) { ok = false; break; }   // some role gave up: all four warps leave here
    // lazy reference: m_run follows the maximum only when that grew by more than 8 (every thread decides alike)
    unsigned char* Pb = Ps + buf * p_bytes;
    float alpha[GP];
    bool rescale = false;
#pragma unroll
    for (int qi = 0; qi < GP; ++qi) {
      const float4 r4 = *reinterpret_cast<const float4*>(&hdr->red[buf][qi][0]);
      const float tm = fmaxf(fmaxf(r4.x, r4.y), fmaxf(r4.z, r4.w));
      alpha[qi] = 1.f;
      if (tm > m_run[qi] + 8.f) {
        alpha[qi] = ex2(m_run[qi] - tm);
        m_run[qi] = tm;
        rescale = rescale || i > 0;
      }
      const float pj = live ? ex2(__uint_as_float(sr[qi]) - m_run[qi]) : 0.f;
      l_thr[qi] = fmaf(l_thr[qi], alpha[qi], pj);
      *reinterpret_cast<__nv_bfloat16*>(Pb + chunk_off(qi, tid >> 3, grp_p) + (tid & 7) * 2) = __float2bfloat16_rn(pj);
    }
    if (rescale) {                                           // uniform over the four warps; this thread's lane of O'^T
      if (!mbar_wait(&hdr->o_done[buf ^ 1], ((i - 1) >> 1) & 1u, p.status)) *abort_flag = 1;   // the sum of tile i - 1 is in
      tc_fence_after();
      uint32_t o[16];
      tmem_ld16(tO + lane_base, o);
      tmem_wait_ld();
#pragma unroll
      for (int qi = 0; qi < GP; ++qi) o[qi] = __float_as_uint(__uint_as_float(o[qi]) * alpha[qi]);
      tmem_st16(tO + lane_base, o);
      tmem_wait_st();
    }
    fence_async_smem();
    tc_fence_before();
    mbar_arrive(&hdr->p_ready[buf]);                         // the issuer sends the weighted sum of this tile off
  }
  if (ok) {
    if (!mbar_wait(&hdr->o_done[(nt - 1) & 1], ((nt - 1) >> 1) & 1u, p.status)) ok = false;
  }
  if (!ok) *abort_flag = 1;
  tc_fence_after();
  worker_sync();                                             // every softmax warp is done with the last tile's maxima

  // ---- partials per query: m, l (summed over the threads' rows), o' (column `query` of O'^T)
#pragma unroll
  for (int qi = 0; qi < GP; ++qi) {
    float v = l_thr[qi];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) hdr->red[0][qi][warp] = v;
  }
  __syncthreads();
  if (tid < G) {
    float mine_m = -INFINITY;
#pragma unroll
    for (int qi = 0; qi < GP; ++qi) mine_m = tid == qi ? m_run[qi] : mine_m;
    part[tid * p.part_stride] = mine_m;
    part[tid * p.part_stride + 1] = (hdr->red[0][tid][0] + hdr->red[0][tid][1]) + (hdr->red[0][tid][2] + hdr->red[0][tid][3]);
  }
  {
    uint32_t o[16];
    tmem_ld16(tO + lane_base, o);
    tmem_wait_ld();
    if (tid < hd.rp_v)
      for (int qi = 0; qi < G; ++qi) part[qi * p.part_stride + 4 + tid] = __uint_as_float(o[qi]);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

}  // namespace

// Stages of the K'/V' ring: about 120 KB of copies in flight, at least two, as far as shared memory reaches.
static int gqa_stages(int max_rp_k, int max_rp_v, size_t* stage_bytes) {
  const size_t k16 = (max_rp_k + 15) & ~15;
  (void)max_rp_v;
  const size_t stage = (((k16 + 63) >> 6) + 2) * static_cast<size_t>(kGqaAtom);
  const size_t avail = 227 * 1024 - (kGqaHeader + 4096 + 2 * kMaxGroup * kTile * 2);
  size_t st = (150 * 1024 + stage - 1) / stage;              // the tiles are padded to 64-element atoms: 120 KB of rows
  if (st < 3) st = 3;
  if (st > static_cast<size_t>(kGqaMaxStages)) st = kGqaMaxStages;
  while (st > 1 && st * stage > avail) --st;
  *stage_bytes = stage;
  return static_cast<int>(st);
}

size_t decode_gqa_smem_bytes(int max_rp_k, int max_rp_v) {
  size_t stage = 0;
  const int st = gqa_stages(max_rp_k, max_rp_v, &stage);
  if (st < 2) return 1 << 30;                                // does not fit: the caller refuses
  return kGqaHeader + 4096 + 2 * kMaxGroup * kTile * 2 + st * stage;
}

template <int GP>
cudaError_t launch_gqa_variant(const GqaDecodeParams& p, size_t smem, int stages, cudaStream_t s) {
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(decode_gqa_kernel<GP>, smem, configured);
  if (ec != cudaSuccess) return ec;
  dim3 grid(p.B * p.H, p.splits);
  decode_gqa_kernel<GP><<<grid, kGqaThreads, smem, s>>>(p, stages);
  return cudaGetLastError();
}

cudaError_t launch_decode_gqa(const GqaDecodeParams& p, int max_rp_k, int max_rp_v, cudaStream_t s, uint64_t* launches) {
  size_t stage_bytes = 0;
  const int stages = gqa_stages(max_rp_k, max_rp_v, &stage_bytes);
  if (stages < 2) return cudaErrorInvalidConfiguration;
  const size_t smem = decode_gqa_smem_bytes(max_rp_k, max_rp_v);
  cudaError_t e = p.group <= 4 ? launch_gqa_variant<4>(p, smem, stages, s)
                  : p.group <= 8 ? launch_gqa_variant<8>(p, smem, stages, s) : launch_gqa_variant<16>(p, smem, stages, s);
  ++*launches;
  if (e != cudaSuccess) return e;
  gqa_combine_kernel<<<p.B * p.H * p.group, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

// Shared memory of decode_gqa_rope_kernel; 0 where it does not fit (wide ranks: the caller then serves every query
// head as a unit of the multi-head rotary kernel).
cudaError_t launch_gqa_combine(const GqaDecodeParams& p, cudaStream_t s, uint64_t* launches) {
  gqa_combine_kernel<<<p.B * p.H * p.group, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

size_t decode_gqa_rope_smem_bytes(int max_rp_k, int d_head) {
  const int k16 = (max_rp_k + 15) & ~15;
  const size_t bytes = kGrHeader + static_cast<size_t>(gr_kb(kMaxGroup * d_head * 2)) + 2 * kMaxGroup * kTile * 2 +
                       gr_kb(d_head * k16 * 2) + 2 * static_cast<size_t>(kTile) * d_head * 2 +
                       2 * static_cast<size_t>((k16 + 63) >> 6) * kGqaAtom + 2 * 2 * static_cast<size_t>(kGqaAtom);
  return bytes <= static_cast<size_t>(227 * 1024) ? bytes : 0;
}

template <int GP, bool INTERLEAVED>
cudaError_t launch_gqa_rope_variant(const GqaDecodeParams& p, size_t smem, cudaStream_t s) {
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(decode_gqa_rope_kernel<GP, INTERLEAVED>, smem, configured);
  if (ec != cudaSuccess) return ec;
  decode_gqa_rope_kernel<GP, INTERLEAVED><<<dim3(p.B * p.H, p.splits), kGrThreads, smem, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_decode_gqa_rope(const GqaDecodeParams& p, int max_rp_k, cudaStream_t s, uint64_t* launches) {
  const size_t smem = decode_gqa_rope_smem_bytes(max_rp_k, p.d_head);
  if (smem == 0) return cudaErrorInvalidConfiguration;
  cudaError_t e;
  if (p.interleaved)
    e = p.group <= 4 ? launch_gqa_rope_variant<4, true>(p, smem, s)
        : p.group <= 8 ? launch_gqa_rope_variant<8, true>(p, smem, s) : launch_gqa_rope_variant<16, true>(p, smem, s);
  else
    e = p.group <= 4 ? launch_gqa_rope_variant<4, false>(p, smem, s)
        : p.group <= 8 ? launch_gqa_rope_variant<8, false>(p, smem, s) : launch_gqa_rope_variant<16, false>(p, smem, s);
  ++*launches;
  if (e != cudaSuccess) return e;
  gqa_combine_kernel<<<p.B * p.H * p.group, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
