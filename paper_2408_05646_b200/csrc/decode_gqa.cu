// Grouped-query decode on the rank-r cache (the Llama-2-70b / Llama-3 models of Section 5.1 share each K/V head
// among a group of g query heads): one pass over the K'/V' rows of a K/V head serves all g queries of its group,
// so the bytes per query head drop by g and the arithmetic per byte rises by g, which is what makes the
// tensor cores worthwhile for a decode step.
//
// Per tile of 128 cached rows (tcgen05, accumulators in TMEM):
//   S  [128 rows x 16]   = K'_tile [128 x r_k] . Q'^T   Q' = q U^K of the g queries (rows past g are zero), scaled
//                                                       by log2(e)/sqrt(d_h), as bf16 high + low parts (two products)
//   softmax in base 2, one thread per cached row, g running maxima kept identical in every thread (lazy
//   reference: a maximum moves only when it grew by more than 8), P rounded to bf16
//   O' [16(128) x r_v] += P^T [16(128) x 128 rows] . V'_tile   P^T has the queries as rows.  The product has M = 128,
//                                                       but only 16 rows of P^T exist in shared memory: the other
//                                                       112 rows of the operand fall on whatever follows (Q', the
//                                                       tiles: finite numbers) and fill rows of O' nobody reads
// A tile of K' or V' rows is contiguous in the cache and arrives as one bulk copy (cp.async.bulk) into a row-major
// staging buffer; the threads move it into the core-matrix layout the tensor core reads and the staging buffer takes
// the next tile at once, a whole tile ahead of its use.  The score
// product of tile t+1 goes out at the top of tile t, so it runs under tile t's softmax.  A fifth warp issues the
// MMAs and the copies: tcgen05.mma issue blocks while the tensor pipe is busy, and a worker thread that issued them
// held all 128 workers at the next barrier.  Workers and the issuer meet on mbarriers only.  Two CTAs per SM.  A unit split over several CTAs leaves partials (m, l, o') per query that
// gqa_combine_kernel merges and lifts through (U^V)^T.  Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kMaxGroup = 16;                 // query heads per K/V head (N of the score product)
constexpr int kGqaThreads = kThreads + 32;    // 128 workers (one per cached row of a tile) + the issuing warp

__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory"); }

// Warp maximum of a float in one instruction: floats ordered as integers (sign-magnitude -> two's complement).
__device__ __forceinline__ float warp_max(float v) {
  int i = __float_as_int(v);
  i ^= (i >> 31) & 0x7fffffff;
  i = __reduce_max_sync(0xffffffffu, i);
  i ^= (i >> 31) & 0x7fffffff;
  return __int_as_float(i);
}
// S = K'_tile Q'^T, KS steps of 16 rank elements, Q' high part then low part; unrolled so that the issuing thread
// spends its time in the MMAs and not in address arithmetic
template <int KS>
__device__ __forceinline__ void issue_scores(uint32_t d_tmem, uint64_t dk, uint64_t dq, uint32_t q_lo, uint32_t idesc) {
#pragma unroll
  for (int s = 0; s < KS; ++s) mma_ss(d_tmem, dk + s * 16, dq + s * 16, idesc, s > 0);
#pragma unroll
  for (int s = 0; s < KS; ++s) mma_ss(d_tmem, dk + s * 16, dq + q_lo + s * 16, idesc, true);
}

struct __align__(16) GqaSmemHeader {
  unsigned long long s_done, o_done, k_full, v_full;
  unsigned long long tiles_ready, p_ready;    // 128 arrivals each: tiles moved into place / P^T written
  uint32_t tmem_base;
  int abort_flag;
  float pad_[2];
  float red[2][kMaxGroup][4];                 // per query: the four warps' maxima / sums, alternating between tiles
};

// GP: query slots the kernel carries (the group size rounded up to 4, 8 or 16); slots past the group score zero
// queries and are never written out.
template <int GP>
__global__ void __launch_bounds__(kGqaThreads, 2) decode_gqa_kernel(const GqaDecodeParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  GqaSmemHeader* hdr = reinterpret_cast<GqaSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x, split = blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const int G = p.group;
  const HeadInfo hd = p.heads[h];
  const int rpk16 = (hd.rp_k + 15) & ~15, rpv16 = (hd.rp_v + 15) & ~15;
  const int grp_k = (rpk16 >> 3) << 7, grp_v = (rpv16 >> 3) << 7, grp_p = (kTile >> 3) << 7;
  const int rowb_k = hd.rp_k * 2, rowb_v = hd.rp_v * 2;      // bytes per cached row
  const int kst_bytes = kTile * rowb_k, vst_bytes = kTile * rowb_v;          // staging, row-major
  const int km_bytes = kTile * rpk16 * 2, vm_bytes = kTile * rpv16 * 2;      // core-matrix layout
  const int q_bytes = kMaxGroup * rpk16 * 2;                 // one image (high or low part) of Q'
  const int p_bytes = kMaxGroup * kTile * 2;                 // the 16 rows of P^T that exist

  unsigned char* tiles = smem + 1024;
  unsigned char* Ps = tiles;                                 // P^T [16 queries][128 rows], canonical (two 8-row groups)
  unsigned char* Qs = Ps + p_bytes;                          // Q' images [16][rk16], canonical: high, then low
  unsigned char* Kst = Qs + 2 * q_bytes;                     // K' tile as it lands
  unsigned char* Vst = Kst + kst_bytes;                      // V' tile as it lands
  unsigned char* Km = Vst + vst_bytes;                       // K' tile, canonical core-matrix layout
  unsigned char* Vm = Km + km_bytes;                         // V' tile, canonical core-matrix layout

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

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 256);
  if (tid == 0) {
    mbar_init(&hdr->s_done, 1);
    mbar_init(&hdr->o_done, 1);
    mbar_init(&hdr->k_full, 1);
    mbar_init(&hdr->v_full, 1);
    mbar_init(&hdr->tiles_ready, kThreads);
    mbar_init(&hdr->p_ready, kThreads);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // P^T, the Q' images and the tiles start as zeros (rows that no copy fills meet zero weights and must be finite;
  // padding chunks of the core-matrix tiles stay zero)
  for (int idx = tid; idx < (p_bytes + 2 * q_bytes + kst_bytes + vst_bytes + km_bytes + vm_bytes) / 16; idx += kGqaThreads)
    reinterpret_cast<uint4*>(Ps)[idx] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  // Q' = q U^K for the g queries of the group, times log2(e)/sqrt(d_h), split into bf16 high + low parts
  {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + b * p.q_stride_b +
                              static_cast<int64_t>(h) * G * p.d_head;
    const float* U = p.basis + hd.uk_off;                    // d_head x rp_k, zero padded columns
    for (int idx = tid; idx < G * hd.rp_k; idx += kGqaThreads) {
      const int qi = idx / hd.rp_k, c = idx - qi * hd.rp_k;
      float acc = 0.f;
      for (int d = 0; d < p.d_head; ++d) acc = fmaf(__bfloat162float(qg[qi * p.d_head + d]), __ldg(U + d * hd.rp_k + c), acc);
      acc *= p.q_scale;
      const __nv_bfloat16 hi = __float2bfloat16_rn(acc);
      const __nv_bfloat16 lo = __float2bfloat16_rn(acc - __bfloat162float(hi));
      const uint32_t off = chunk_off(qi, c >> 3, grp_k) + (c & 7) * 2;
      *reinterpret_cast<__nv_bfloat16*>(Qs + off) = hi;
      *reinterpret_cast<__nv_bfloat16*>(Qs + q_bytes + off) = lo;
    }
  }
  const uint64_t policy = policy_evict_first();
  const char* k_src = p.cache + hd.k_off + static_cast<int64_t>(b) * p.n_max * rowb_k;
  const char* v_src = p.cache + hd.v_off + static_cast<int64_t>(b) * p.n_max * rowb_v;
  auto fetch_k = [&](int t) {
    const uint32_t bytes = static_cast<uint32_t>(min(kTile, n_b - t * kTile)) * rowb_k;
    mbar_arrive_expect_tx(&hdr->k_full, bytes);
    bulk_load(Kst, k_src + static_cast<int64_t>(t) * kTile * rowb_k, bytes, &hdr->k_full, policy);
  };
  auto fetch_v = [&](int t) {
    const uint32_t bytes = static_cast<uint32_t>(min(kTile, n_b - t * kTile)) * rowb_v;
    mbar_arrive_expect_tx(&hdr->v_full, bytes);
    bulk_load(Vst, v_src + static_cast<int64_t>(t) * kTile * rowb_v, bytes, &hdr->v_full, policy);
  };
  // staging -> core-matrix layout: chunk (row, c) of 16 bytes goes to (row / 8) * group + c * 128 + (row % 8) * 16
  auto relayout = [&](unsigned char* dst, const unsigned char* src, int rowb, int grp) {
    relayout_tile(dst, src, rowb, grp, warp, lane);
  };
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
  const uint32_t tO = tmem + 64;                             // O': lanes = queries, columns = rank of V
  volatile int* abort_flag = &hdr->abort_flag;
  const uint32_t idesc_s = instr_desc(kMaxGroup, false);
  const uint32_t idesc_o = instr_desc(rpv16, true);
  const int ks_steps = rpk16 >> 4;
  const uint64_t desc_k = smem_desc(smem_u32(Km), 128, grp_k);
  const uint64_t desc_q = smem_desc(smem_u32(Qs), 128, grp_k);
  const uint64_t desc_p = smem_desc(smem_u32(Ps), 128, grp_p);
  const uint64_t desc_v = smem_desc(smem_u32(Vm), grp_v, 128);   // MN-major operand: 8-row groups along K, chunks along N
  // S(t) = K'(t) Q'^T into score buffer `buf` (columns 32 buf .. 32 buf + 15)
  auto issue_s = [&](int buf) {
    tc_fence_after();
    const uint32_t d = tmem + 32 * buf, q_lo = static_cast<uint32_t>(q_bytes >> 4);
    switch (ks_steps) {
      case 1: issue_scores<1>(d, desc_k, desc_q, q_lo, idesc_s); break;
      case 2: issue_scores<2>(d, desc_k, desc_q, q_lo, idesc_s); break;
      case 3: issue_scores<3>(d, desc_k, desc_q, q_lo, idesc_s); break;
      case 4: issue_scores<4>(d, desc_k, desc_q, q_lo, idesc_s); break;
      case 5: issue_scores<5>(d, desc_k, desc_q, q_lo, idesc_s); break;
      case 6: issue_scores<6>(d, desc_k, desc_q, q_lo, idesc_s); break;
      case 7: issue_scores<7>(d, desc_k, desc_q, q_lo, idesc_s); break;
      default: issue_scores<8>(d, desc_k, desc_q, q_lo, idesc_s); break;
    }
    mma_commit(&hdr->s_done);
  };
  bool ok = true;
  const bool issuer = warp == kThreads / 32;                 // warp 4
  if (issuer && lane == 0) {
    fetch_k(t_lo);
    fetch_v(t_lo);
  }
  // the first K' tile: into the core-matrix layout, its score product, and the staging buffer takes the second
  if (!issuer) {
    if (!mbar_wait(&hdr->k_full, 0, p.status)) *abort_flag = 1;
    relayout(Km, Kst, rowb_k, grp_k);
    fence_async_smem();
  }
  __syncthreads();
  if (*abort_flag) ok = false;

  if (issuer) {
    // ------------------------------------------------------------------ the issuing warp
    if (lane == 0 && ok) {
      issue_s(0);
      if (t_lo + 1 < t_hi) fetch_k(t_lo + 1);
      for (int t = t_lo; t < t_hi && ok; ++t) {
        const uint32_t par = (t - t_lo) & 1u;
        ok = mbar_wait(&hdr->tiles_ready, par, p.status) && !*abort_flag;   // K'(t+1), V'(t) are in place
        if (!ok) break;
        if (t + 1 < t_hi) {
          issue_s(static_cast<int>(par ^ 1u));
          fetch_v(t + 1);
          if (t + 2 < t_hi) fetch_k(t + 2);
        }
        ok = mbar_wait(&hdr->p_ready, par, p.status) && !*abort_flag;       // P^T(t) written, O' rescaled if needed
        if (!ok) break;
        tc_fence_after();
        for (int s = 0; s < kTile / 16; ++s)                 // O' += P^T V'(t), 16 cached rows (two 8-row groups) a step
          mma_ss(tO, desc_p + s * 16, desc_v + s * ((2 * grp_v) >> 4), idesc_o, t > t_lo || s > 0);
        mma_commit(&hdr->o_done);
      }
      if (!ok) *abort_flag = 1;
    }
    __syncthreads();                                         // the workers' epilogue
    __syncthreads();
    return;
  }

  // -------------------------------------------------------------------- the 128 workers
  float m_run[GP], l_thr[GP];
#pragma unroll
  for (int qi = 0; qi < GP; ++qi) { m_run[qi] = -INFINITY; l_thr[qi] = 0.f; }

  for (int t = t_lo; t < t_hi && ok; ++t) {
    const uint32_t par = (t - t_lo) & 1u;
    // ---- S(t) is complete: the K' core-matrix tile is free; PV(t-1) is complete: P^T and the V' core-matrix tile
    //      are free.  K'(t+1) and V'(t) have landed: move them and tell the issuer.
    if (!mbar_wait(&hdr->s_done, par, p.status)) *abort_flag = 1;
    if (t > t_lo && !mbar_wait(&hdr->o_done, par ^ 1u, p.status)) *abort_flag = 1;
    if (t + 1 < t_hi) {
      if (!mbar_wait(&hdr->k_full, par ^ 1u, p.status)) *abort_flag = 1;
      relayout(Km, Kst, rowb_k, grp_k);
    }
    if (!mbar_wait(&hdr->v_full, par, p.status)) *abort_flag = 1;
    relayout(Vm, Vst, rowb_v, grp_v);
    fence_async_smem();
    tc_fence_before();
    mbar_arrive(&hdr->tiles_ready);
    tc_fence_after();
    uint32_t sr[16];
    tmem_ld16(tmem + lane_base + 32 * par, sr);
    tmem_wait_ld();
    const bool live = t * kTile + tid < n_b;
    // ---- per-query maximum over the tile: one reduction instruction per query and warp, lane q keeps query q's
#pragma unroll
    for (int qi = 0; qi < GP; ++qi) {
      const float v = warp_max(live ? __uint_as_float(sr[qi]) : -INFINITY);
      if (lane == qi) hdr->red[par][qi][warp] = v;
    }
    worker_sync();
    if (*abort_flag) { ok = false; break; }
    // lazy reference: m_run follows the maximum only when that grew by more than 8 (every thread decides alike)
    bool rescale = false;
    float alpha_mine = 1.f;                                  // for the O' row this thread owns (lane = query)
#pragma unroll
    for (int qi = 0; qi < GP; ++qi) {
      const float4 r4 = *reinterpret_cast<const float4*>(&hdr->red[par][qi][0]);
      const float tm = fmaxf(fmaxf(r4.x, r4.y), fmaxf(r4.z, r4.w));
      float alpha = 1.f;
      if (tm > m_run[qi] + 8.f) {
        alpha = ex2(m_run[qi] - tm);
        m_run[qi] = tm;
        rescale = rescale || t > t_lo;
      }
      const float pj = live ? ex2(__uint_as_float(sr[qi]) - m_run[qi]) : 0.f;
      l_thr[qi] = fmaf(l_thr[qi], alpha, pj);
      if (tid == qi) alpha_mine = alpha;
      *reinterpret_cast<__nv_bfloat16*>(Ps + chunk_off(qi, tid >> 3, grp_p) + (tid & 7) * 2) = __float2bfloat16_rn(pj);
    }
    if (rescale && warp == 0) {                              // O' rows (lanes 0..g-1 of warp 0) times their alpha
      tc_fence_after();
      for (int c0 = 0; c0 < rpv16; c0 += 16) {
        uint32_t o[16];
        tmem_ld16(tO + c0, o);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha_mine);
        tmem_st16(tO + c0, o);
      }
      tmem_wait_st();
    }
    fence_async_smem();
    tc_fence_before();
    mbar_arrive(&hdr->p_ready);                              // the issuer sends the weighted sum of this tile off
  }
  if (ok) {
    if (!mbar_wait(&hdr->o_done, (t_hi - 1 - t_lo) & 1u, p.status)) ok = false;
  }
  if (!ok) *abort_flag = 1;
  tc_fence_after();
  worker_sync();                                             // every worker is done with the last tile's maxima

  // ---- partials per query: m, l (summed over the threads' rows), o' (row `query` of O')
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
  if (warp == 0) {
    for (int c0 = 0; c0 < rpv16; c0 += 16) {
      uint32_t o[16];
      tmem_ld16(tO + c0, o);
      tmem_wait_ld();
      if (lane < G)
        for (int i = 0; i < 16; ++i)
          if (c0 + i < hd.rp_v) part[lane * p.part_stride + 4 + c0 + i] = __uint_as_float(o[i]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
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

size_t decode_gqa_smem_bytes(int max_rp_k, int max_rp_v) {
  const size_t k16 = (max_rp_k + 15) & ~15;
  // P^T (16 rows), Q' images, K' and V' tiles as they land and in the core-matrix layout; the P^T operand of the
  // weighted sum spans 32 KB from its start, which the tiles behind it cover
  const size_t v16 = (max_rp_v + 15) & ~15;
  size_t total = 1024 + kMaxGroup * kTile * 2 + 2 * kMaxGroup * k16 * 2 + kTile * static_cast<size_t>(max_rp_k + max_rp_v + k16 + v16) * 2;
  const size_t need = 1024 + static_cast<size_t>(kTile) * kTile * 2;
  return total < need ? need : total;
}

template <int GP>
cudaError_t launch_gqa_variant(const GqaDecodeParams& p, size_t smem, cudaStream_t s) {
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(decode_gqa_kernel<GP>, smem, configured);
  if (ec != cudaSuccess) return ec;
  dim3 grid(p.B * p.H, p.splits);
  decode_gqa_kernel<GP><<<grid, kGqaThreads, smem, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_decode_gqa(const GqaDecodeParams& p, size_t smem, cudaStream_t s, uint64_t* launches) {
  cudaError_t e = p.group <= 4 ? launch_gqa_variant<4>(p, smem, s)
                  : p.group <= 8 ? launch_gqa_variant<8>(p, smem, s) : launch_gqa_variant<16>(p, smem, s);
  ++*launches;
  if (e != cudaSuccess) return e;
  gqa_combine_kernel<<<p.B * p.H * p.group, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
