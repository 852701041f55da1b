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
// K' and V' tiles arrive by TMA (tensor maps of the cache slabs, 128-byte swizzle): K'(t+1) once the scores of tile
// t are done, V'(t+1) (two buffers) once the weighted sum of tile t-1 is done; two CTAs per SM.  A unit split over several CTAs leaves partials (m, l, o') per query that
// gqa_combine_kernel merges and lifts through (U^V)^T.  Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kAtom = kTile * 128;            // one swizzled atom column of a 128-row tile: 64 elements wide
constexpr int kMaxGroup = 16;                 // query heads per K/V head (N of the score product)

struct __align__(16) GqaSmemHeader {
  unsigned long long s_done, o_done, k_full, v_full[2];
  uint32_t tmem_base;
  int abort_flag;
  float pad_[2];
  float red[4][kMaxGroup];                    // per-warp maxima / sums per query
};

__global__ void __launch_bounds__(kThreads, 2) decode_gqa_kernel(const GqaDecodeParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  GqaSmemHeader* hdr = reinterpret_cast<GqaSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x, split = blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const int G = p.group;
  const HeadInfo hd = p.heads[h];
  const int rpk16 = (hd.rp_k + 15) & ~15, rpv16 = (hd.rp_v + 15) & ~15;
  const int grp_k = (rpk16 >> 3) << 7, grp_p = (kTile >> 3) << 7;
  const int atoms_k = (rpk16 + 63) >> 6, atoms_v = (hd.rp_v + 63) >> 6;
  const int k_bytes = atoms_k * kAtom, v_bytes = atoms_v * kAtom;
  const int q_bytes = kMaxGroup * rpk16 * 2;                 // one image (high or low part) of Q'
  const int p_bytes = kMaxGroup * kTile * 2;                 // the 16 rows of P^T that exist

  unsigned char* tiles = smem + 1024;
  unsigned char* Ps = tiles;                                 // P^T [16 queries][128 rows], canonical (two 8-row groups)
  unsigned char* Qs = Ps + p_bytes;                          // Q' images [16][rk16], canonical: high, then low
  unsigned char* Ks = Qs + 2 * q_bytes;                      // K' tile, swizzled atom columns of 128 rows (1024-aligned)
  unsigned char* Vs = Ks + k_bytes;                          // two V' tiles, same layout

  const int per = (p.nt + p.splits - 1) / p.splits;
  const int t_lo = split * per, t_hi = min(p.nt, t_lo + per);
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
    mbar_init(&hdr->v_full[0], 1);
    mbar_init(&hdr->v_full[1], 1);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // P^T and the Q' images start as zeros
  for (int idx = tid; idx < (p_bytes + 2 * q_bytes) / 16; idx += kThreads)
    reinterpret_cast<uint4*>(Ps)[idx] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  // Q' = q U^K for the g queries of the group, times log2(e)/sqrt(d_h), split into bf16 high + low parts
  {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + b * p.q_stride_b +
                              static_cast<int64_t>(h) * G * p.d_head;
    const float* U = p.basis + hd.uk_off;                    // d_head x rp_k, zero padded columns
    for (int idx = tid; idx < G * hd.rp_k; idx += kThreads) {
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
  const unsigned char* maps = static_cast<const unsigned char*>(p.tmaps) + static_cast<size_t>(h) * 256;
  auto fetch_k = [&](int t) {
    mbar_arrive_expect_tx(&hdr->k_full, static_cast<uint32_t>(k_bytes));
    for (int a = 0; a < atoms_k; ++a)
      for (int hf = 0; hf < 2; ++hf)
        tma_load_3d(Ks + a * kAtom + hf * (kAtom / 2), maps, a * 64, t * kTile + hf * 64, b, &hdr->k_full);
  };
  auto fetch_v = [&](int t) {                                // into buffer (t - t_lo) % 2
    const int vb = (t - t_lo) & 1;
    mbar_arrive_expect_tx(&hdr->v_full[vb], static_cast<uint32_t>(v_bytes));
    for (int a = 0; a < atoms_v; ++a)
      for (int hf = 0; hf < 2; ++hf)
        tma_load_3d(Vs + vb * v_bytes + a * kAtom + hf * (kAtom / 2), maps + 128, a * 64, t * kTile + hf * 64, b,
                    &hdr->v_full[vb]);
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
  const uint64_t desc_k = smem_desc_sw128(smem_u32(Ks), 16, 1024);
  const uint64_t desc_q = smem_desc(smem_u32(Qs), 128, grp_k);
  const uint64_t desc_p = smem_desc(smem_u32(Ps), 128, grp_p);
  const uint64_t desc_v = smem_desc_sw128(smem_u32(Vs), kAtom, 1024);
  // S(t) = K'(t) Q'^T into score buffer `buf` (columns 32 buf .. 32 buf + 15)
  auto issue_s = [&](int buf) {
    tc_fence_after();
    for (int part_i = 0; part_i < 2; ++part_i)               // Q' high part, then low part
      for (int s = 0; s < ks_steps; ++s)
        mma_ss(tmem + 32 * buf, desc_k + (s >> 2) * (kAtom >> 4) + (s & 3) * 2, desc_q + part_i * (q_bytes >> 4) + s * 16,
               idesc_s, part_i > 0 || s > 0);
    mma_commit(&hdr->s_done);
  };
  bool ok = true;
  if (tid == 0) {
    tensormap_acquire(maps);
    tensormap_acquire(maps + 128);
    fetch_k(t_lo);
    fetch_v(t_lo);
    if (t_lo + 1 < t_hi) fetch_v(t_lo + 1);
    ok = mbar_wait(&hdr->k_full, 0, p.status);
    if (ok) issue_s(0);
    else *abort_flag = 1;
  }

  float m_run[kMaxGroup], l_thr[kMaxGroup];
#pragma unroll
  for (int qi = 0; qi < kMaxGroup; ++qi) { m_run[qi] = -INFINITY; l_thr[qi] = 0.f; }

  for (int t = t_lo; t < t_hi && ok; ++t) {
    const uint32_t par = (t - t_lo) & 1u;
    // ---- S(t) is complete: K'(t+1) may replace K'(t); PV(t-1) is complete: P^T and the V' tile are free
    if (!mbar_wait(&hdr->s_done, par, p.status)) *abort_flag = 1;
    if (t > t_lo && !mbar_wait(&hdr->o_done, par ^ 1u, p.status)) *abort_flag = 1;
    if (tid == 0 && t + 1 < t_hi) fetch_k(t + 1);
    if (tid == 0 && t > t_lo && t + 1 < t_hi) fetch_v(t + 1);   // its buffer was PV(t-1)'s; the first two went out earlier
    tc_fence_after();
    uint32_t sr[16];
    tmem_ld16(tmem + lane_base + 32 * par, sr);
    tmem_wait_ld();
    const bool live = t * kTile + tid < p.n;
    // ---- per-query maximum over the tile
    float mx[kMaxGroup];
#pragma unroll
    for (int qi = 0; qi < kMaxGroup; ++qi) {
      mx[qi] = -INFINITY;
      if (qi < G) {
        float v = live ? __uint_as_float(sr[qi]) : -INFINITY;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
        mx[qi] = v;
      }
    }
    if (lane < kMaxGroup) {
      float mine = -INFINITY;
#pragma unroll
      for (int qi = 0; qi < kMaxGroup; ++qi) mine = lane == qi ? mx[qi] : mine;
      hdr->red[warp][lane] = mine;
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) { ok = false; break; }
    // lazy reference: m_run follows the maximum only when that grew by more than 8 (every thread decides alike)
    bool rescale = false;
    float alpha_mine = 1.f;                                  // for the O' row this thread owns (lane = query)
#pragma unroll
    for (int qi = 0; qi < kMaxGroup; ++qi) {
      if (qi < G) {
        const float tm = fmaxf(fmaxf(hdr->red[0][qi], hdr->red[1][qi]), fmaxf(hdr->red[2][qi], hdr->red[3][qi]));
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
    if (!mbar_wait(&hdr->v_full[par], ((t - t_lo) >> 1) & 1u, p.status)) *abort_flag = 1;
    __syncthreads();
    if (*abort_flag) { ok = false; break; }
    // ---- O' += P^T V'(t); then S(t+1) as soon as K'(t+1) is there
    if (tid == 0) {
      tc_fence_after();
      for (int s = 0; s < kTile / 16; ++s)                   // 16 cached rows a step
        mma_ss(tO, desc_p + s * 16, desc_v + par * (v_bytes >> 4) + s * (2048 >> 4), idesc_o, t > t_lo || s > 0);
      mma_commit(&hdr->o_done);
      if (t + 1 < t_hi) {
        if (mbar_wait(&hdr->k_full, par ^ 1u, p.status)) issue_s(static_cast<int>(par ^ 1u));
        else *abort_flag = 1;
      }
    }
  }
  if (ok) {
    if (!mbar_wait(&hdr->o_done, (t_hi - 1 - t_lo) & 1u, p.status)) ok = false;
  }
  if (!ok) *abort_flag = 1;
  tc_fence_after();

  // ---- partials per query: m, l (summed over the threads' rows), o' (row `query` of O')
#pragma unroll
  for (int qi = 0; qi < kMaxGroup; ++qi) {
    if (qi < G) {
      float v = l_thr[qi];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) hdr->red[warp][qi] = v;
    }
  }
  __syncthreads();
  if (tid < G) {
    float mine_m = -INFINITY;
#pragma unroll
    for (int qi = 0; qi < kMaxGroup; ++qi) mine_m = tid == qi ? m_run[qi] : mine_m;
    part[tid * p.part_stride] = mine_m;
    part[tid * p.part_stride + 1] = (hdr->red[0][tid] + hdr->red[1][tid]) + (hdr->red[2][tid] + hdr->red[3][tid]);
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
  // P^T (16 rows), Q' images, one K' tile, two V' tiles; the P^T operand of the weighted sum spans 32 KB from its
  // start, which the tiles behind it cover
  return 1024 + kMaxGroup * kTile * 2 + 2 * kMaxGroup * k16 * 2 +
         (((k16 + 63) >> 6) + 2 * ((max_rp_v + 63) >> 6)) * static_cast<size_t>(kAtom);
}

cudaError_t launch_decode_gqa(const GqaDecodeParams& p, size_t smem, cudaStream_t s, uint64_t* launches) {
  static size_t configured = 0;
  if (smem > configured) {
    const cudaError_t e = cudaFuncSetAttribute(decode_gqa_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  dim3 grid(p.B * p.H, p.splits);
  decode_gqa_kernel<<<grid, kThreads, smem, s>>>(p);
  ++*launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  gqa_combine_kernel<<<p.B * p.H * p.group, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
