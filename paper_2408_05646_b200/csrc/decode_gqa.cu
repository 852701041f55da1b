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

}  // namespace ea
