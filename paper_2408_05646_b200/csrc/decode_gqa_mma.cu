// Grouped-query decode (the models of Section 5.1 that share K/V heads) with warp-level tensor-core products
// (mma.sync m16n8k16, bf16 operands, fp32 accumulators).
//
// With at most 16 queries per K/V head the two products of a tile are thin: S^T has 16 rows, of which `group`
// are real.  The kernel is bound by the bytes of K' and V', so what matters is that the tiles stream without a
// stall; a product per warp, issued by the warp that consumes it, has no hand-over between threads at all:
//   * K' and V' tiles of 128 rows arrive row-major, as they lie in the cache (or in the page that holds them),
//     through a ring of bulk copies;
//   * a warp owns 32 rows of every tile: S = Q' K'^T (A = Q' fragments, loaded once per CTA; B = K' rows, ldmatrix),
//     online softmax on the accumulator fragments, which are at the same time the A fragments of the second
//     product, O' += P V' (B = V' rows through ldmatrix.trans);
//   * the four warps walk the tiles on their own; the warp that is last to finish a slot refills it.
// The warps' states (m, l, O') are merged at the end; a unit split over several CTAs leaves partials per query
// that the combine kernel merges and lifts through (U^V)^T.  Every wait is bounded.
#include <cstddef>
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kGmThreads = 128;
constexpr int kGmTile = 128;
constexpr int kGmMaxStages = 4;
constexpr unsigned kFull = 0xffffffffu;
constexpr float kGmRaise = 8.f;            // a running maximum is raised when a score exceeds it by this much

struct __align__(16) GmHeader {
  unsigned long long full[kGmMaxStages];
  int done[kGmMaxStages];
  int abort_flag;
};
constexpr int kGmHeaderBytes = 128;
static_assert(sizeof(GmHeader) <= kGmHeaderBytes, "header outgrew its area");
constexpr int kGmQrawBytes = 16 * 128 * 4;                  // the group's queries as fp32 [16][d_head <= 128]
constexpr int kGmQsStride = 128 + 8;                        // Q' image [16][136] bf16: rows 272 bytes apart
constexpr int kGmQsBytes = 16 * kGmQsStride * 2;
constexpr int kGmRingOffset = (kGmHeaderBytes + kGmQrawBytes + kGmQsBytes + 127) & ~127;

__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm2(uint32_t (&r)[2], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ float quad_max(float v) {
  v = fmaxf(v, __shfl_xor_sync(kFull, v, 1));
  return fmaxf(v, __shfl_xor_sync(kFull, v, 2));
}

// NKS: 16-channel steps of the widest key row; NVT: 8-channel tiles of the widest value row; HI: more than 8
// queries (rows 8..15 of the fragments are in use); FULL: every head has exactly 16 NKS key and 8 NVT value channels.
template <int NKS, int NVT, bool HI, bool FULL>
__global__ void __launch_bounds__(kGmThreads, 2) decode_gqa_mma_kernel(const GqaDecodeParams p, int stages) {
  extern __shared__ __align__(1024) unsigned char smem[];
  GmHeader* hdr = reinterpret_cast<GmHeader*>(smem);
  float* qraw = reinterpret_cast<float*>(smem + kGmHeaderBytes);
  __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem + kGmHeaderBytes + kGmQrawBytes);
  unsigned char* ring = smem + kGmRingOffset;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int unit = blockIdx.x, split = blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const int G = p.group;
  const HeadInfo hd = p.heads[h];
  const int rp_k = FULL ? 16 * NKS : hd.rp_k, rp_v = FULL ? 8 * NVT : hd.rp_v;
  const int nks = FULL ? NKS : rp_k >> 4, nvt = FULL ? NVT : rp_v >> 3;
  const int kb = rp_k * 2, vb = rp_v * 2;                    // bytes of a key row, of a value row
  const int k_tile = kGmTile * kb, stage_bytes = (kGmTile * (kb + vb) + 127) & ~127;

  const int n_b = p.deficit != nullptr ? p.n - __ldg(p.deficit + b) : p.n;
  const int nt_b = (n_b + kGmTile - 1) / kGmTile;
  const int per = (nt_b + p.splits - 1) / p.splits;
  const int t_lo = min(nt_b, split * per), t_hi = min(nt_b, t_lo + per);
  const char* k_slab = p.cache + hd.k_off;
  const char* v_slab = p.cache + hd.v_off;

  if (tid == 0) {
    for (int s = 0; s < kGmMaxStages; ++s) {
      mbar_init(&hdr->full[s], 1);
      hdr->done[s] = 0;
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const uint64_t policy = policy_evict_first();
  auto issue = [&](int t, int slot) {                        // one thread: the K' and the V' rows of tile t
    const int rows = min(kGmTile, n_b - t * kGmTile);
    unsigned char* dst = ring + slot * stage_bytes;
    mbar_arrive_expect_tx(&hdr->full[slot], static_cast<uint32_t>(rows) * (kb + vb));
    const int64_t row0 = physical_row(p.pages, b, p.n_max, t * kGmTile);     // a tile lies inside one page
    bulk_load(dst, k_slab + row0 * kb, static_cast<uint32_t>(rows) * kb, &hdr->full[slot], policy);
    bulk_load(dst + k_tile, v_slab + row0 * vb, static_cast<uint32_t>(rows) * vb, &hdr->full[slot], policy);
  };
  if (tid == 0)
    for (int i = 0; i < stages && t_lo + i < t_hi; ++i) issue(t_lo + i, i);

  // Q' = Q U^K of the group's queries, scaled into the base-2 domain, as bf16 rows; rows past the group are zero
  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(p.q);
  for (int i = tid; i < G * p.d_head; i += kGmThreads) {
    const int g = i / p.d_head, d = i - g * p.d_head;
    qraw[g * 128 + d] = __bfloat162float(q[b * p.q_stride_b + (static_cast<int64_t>(h) * G + g) * p.d_head + d]);
  }
  for (int i = tid; i < 16 * kGmQsStride; i += kGmThreads) Qs[i] = __float2bfloat16_rn(0.f);
  __syncthreads();
  for (int o = tid; o < G * rp_k; o += kGmThreads) {
    const int g = o / rp_k, c = o - g * rp_k;
    const float* U = p.basis + hd.uk_off + c;
    const float* x = qraw + g * 128;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
    for (int d = 0; d < p.d_head; d += 4) {
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[i] = fmaf(x[d + i], __ldg(U + (d + i) * rp_k), acc[i]);
    }
    Qs[g * kGmQsStride + c] = __float2bfloat16_rn(((acc[0] + acc[1]) + (acc[2] + acc[3])) * p.q_scale);
  }
  __syncthreads();
  uint32_t qa[NKS][4];                                       // A fragments of Q': rows gid, gid + 8
#pragma unroll
  for (int ks = 0; ks < NKS; ++ks) {
    const uint32_t* r0 = reinterpret_cast<const uint32_t*>(Qs + gid * kGmQsStride + 16 * ks + 2 * tig);
    const uint32_t* r1 = reinterpret_cast<const uint32_t*>(Qs + (gid + 8) * kGmQsStride + 16 * ks + 2 * tig);
    qa[ks][0] = r0[0]; qa[ks][2] = r0[4];
    qa[ks][1] = HI ? r1[0] : 0u; qa[ks][3] = HI ? r1[4] : 0u;
  }

  float o[NVT][4];                                           // O' fragments: (query gid, channels 8c + 2tig, +1), (gid + 8, ...)
#pragma unroll
  for (int c = 0; c < NVT; ++c)
#pragma unroll
    for (int i = 0; i < 4; ++i) o[c][i] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // queries gid and gid + 8; l: this lane's share
  const int r0w = warp * 32;
  // per-lane byte offsets of the ldmatrix rows: K' matrices (row l & 7 of row group j, the k half (l >> 3) & 1 of
  // step ks + (l >> 4)); V' matrices (row l of the warp's 32)
  const uint32_t k_lane = static_cast<uint32_t>((r0w + (lane & 7)) * kb + ((lane >> 3) & 1) * 16 + (lane >> 4) * 32);
  const uint32_t v_lane = static_cast<uint32_t>((r0w + lane) * vb);

  for (int t = t_lo; t < t_hi; ++t) {
    const int it = t - t_lo, slot = it % stages;
    if (__any_sync(kFull, !mbar_wait(&hdr->full[slot], (it / stages) & 1, p.status))) {
      hdr->abort_flag = 1;
      break;
    }
    unsigned char* st = ring + slot * stage_bytes;
    const int rows = min(kGmTile, n_b - t * kGmTile);
    if (r0w < rows) {
      if (rows < kGmTile) {                                  // the sequence's last tile: rows past its end read as zero
        const int r = r0w + lane;
        if (r >= rows) {
          uint4* kr = reinterpret_cast<uint4*>(st + r * kb);
          uint4* vr = reinterpret_cast<uint4*>(st + k_tile + r * vb);
          for (int i = 0; i < (kb >> 4); ++i) kr[i] = make_uint4(0u, 0u, 0u, 0u);
          for (int i = 0; i < (vb >> 4); ++i) vr[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncwarp();
      }
      const uint32_t k_addr = smem_u32(st) + k_lane, v_addr = smem_u32(st + k_tile) + v_lane;
      // ---- S = Q' K'^T for the warp's 32 rows: four groups of 8 rows
      float s[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int i = 0; i < 4; ++i) s[j][i] = 0.f;
#pragma unroll
        for (int ks = 0; ks < NKS; ks += 2) {
          if (ks + 1 < NKS) {
            if (FULL || ks < nks) {
              uint32_t bfr[4];
              ldsm4(bfr, k_addr + j * 8 * kb + ks * 32);
              mma_bf16(s[j], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], bfr[0], bfr[1]);
              if (FULL || ks + 1 < nks) mma_bf16(s[j], qa[ks + 1][0], qa[ks + 1][1], qa[ks + 1][2], qa[ks + 1][3], bfr[2], bfr[3]);
            }
          } else if (FULL || ks < nks) {
            uint32_t bfr[2];
            ldsm2(bfr, k_addr + j * 8 * kb + ks * 32);
            mma_bf16(s[j], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], bfr[0], bfr[1]);
          }
        }
      }
      // ---- online softmax on the fragments: s[j][0..1] = (query gid, rows 8j + 2tig, +1), s[j][2..3] = query gid + 8
      if (rows - r0w < 32) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i)
            if (r0w + 8 * j + 2 * tig + (i & 1) >= rows) s[j][i] = -INFINITY;
      }
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mx0 = fmaxf(mx0, fmaxf(s[j][0], s[j][1]));
        if (HI) mx1 = fmaxf(mx1, fmaxf(s[j][2], s[j][3]));
      }
      if (__any_sync(kFull, mx0 > m0 + kGmRaise || (HI && mx1 > m1 + kGmRaise))) {
        const float n0 = fmaxf(m0, quad_max(mx0)), n1 = HI ? fmaxf(m1, quad_max(mx1)) : m1;
        const float f0 = ex2(m0 - n0), f1 = HI ? ex2(m1 - n1) : 1.f;      // ex2(-inf) = 0 on the first tile
        l0 *= f0; l1 *= f1;
#pragma unroll
        for (int c = 0; c < NVT; ++c) {
          o[c][0] *= f0; o[c][1] *= f0;
          if (HI) { o[c][2] *= f1; o[c][3] *= f1; }
        }
        m0 = n0; m1 = n1;
      }
      uint32_t pa[2][4];                                     // A fragments of P for the two 16-row steps
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float p0 = ex2(s[j][0] - m0), p1 = ex2(s[j][1] - m0);
        l0 += p0 + p1;
        pa[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
        if (HI) {
          const float p2 = ex2(s[j][2] - m1), p3 = ex2(s[j][3] - m1);
          l1 += p2 + p3;
          pa[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
        } else {
          pa[j >> 1][(j & 1) * 2 + 1] = 0u;
        }
      }
      // ---- O' += P V': tiles of 8 channels, two steps of 16 rows
#pragma unroll
      for (int c = 0; c < NVT; ++c)
        if (FULL || c < nvt) {
          uint32_t bfr[4];
          ldsm4_t(bfr, v_addr + c * 16);
          mma_bf16(o[c], pa[0][0], pa[0][1], pa[0][2], pa[0][3], bfr[0], bfr[1]);
          mma_bf16(o[c], pa[1][0], pa[1][1], pa[1][2], pa[1][3], bfr[2], bfr[3]);
        }
    }
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();       // the warp's reads of the slot come before the count that may trigger the refill
      if ((atomicAdd(&hdr->done[slot], 1) & 3) == 3 && t + stages < t_hi) issue(t + stages, slot);
    }
  }
  __syncthreads();
  const bool aborted = *reinterpret_cast<volatile int*>(&hdr->abort_flag) != 0;

  // ---- merge the four warps: per query the maximum, then sums and O' scaled to it (the ring is idle now)
  float* wm = reinterpret_cast<float*>(ring);                // [4][16] maxima
  float* wl = wm + 64;                                       // [4][16] sums
  float* wo = wl + 64;                                       // [4][16][rp_v + 1]
  const int ostride = rp_v + 1;
  l0 += __shfl_xor_sync(kFull, l0, 1); l0 += __shfl_xor_sync(kFull, l0, 2);
  l1 += __shfl_xor_sync(kFull, l1, 1); l1 += __shfl_xor_sync(kFull, l1, 2);
  if (tig == 0) {
    wm[warp * 16 + gid] = m0; wm[warp * 16 + gid + 8] = HI ? m1 : -INFINITY;
    wl[warp * 16 + gid] = l0; wl[warp * 16 + gid + 8] = HI ? l1 : 0.f;
  }
#pragma unroll
  for (int c = 0; c < NVT; ++c)
    if (FULL || c < nvt) {
      float* d0 = wo + (warp * 16 + gid) * ostride + 8 * c + 2 * tig;
      d0[0] = o[c][0]; d0[1] = o[c][1];
      if (HI) {
        float* d1 = wo + (warp * 16 + gid + 8) * ostride + 8 * c + 2 * tig;
        d1[0] = o[c][2]; d1[1] = o[c][3];
      }
    }
  __syncthreads();
  float* part = p.partials + (static_cast<size_t>(unit) * p.splits + split) * G * p.part_stride;
  for (int i = tid; i < G * (rp_v + 2); i += kGmThreads) {
    const int qi = i / (rp_v + 2), c = i - qi * (rp_v + 2);
    const float M = fmaxf(fmaxf(wm[qi], wm[16 + qi]), fmaxf(wm[32 + qi], wm[48 + qi]));
    float acc = 0.f;
    if (!aborted)
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float mw = wm[w * 16 + qi];
        const float f = mw == -INFINITY ? 0.f : ex2(mw - M);
        acc = fmaf(c < rp_v ? wo[(w * 16 + qi) * ostride + c] : wl[w * 16 + qi], f, acc);
      }
    if (c < rp_v) part[qi * p.part_stride + 4 + c] = acc;
    else if (c == rp_v) part[qi * p.part_stride + 1] = acc;
    else part[qi * p.part_stride] = M;
  }
}

int gm_stages(int max_rp_k, int max_rp_v, size_t* smem) {
  const size_t stage = (static_cast<size_t>(kGmTile) * (max_rp_k + max_rp_v) * 2 + 127) & ~static_cast<size_t>(127);
  const size_t budget = 113 * 1024;                          // two CTAs per SM
  int stages = static_cast<int>((budget - kGmRingOffset) / stage);
  if (stages > kGmMaxStages) stages = kGmMaxStages;
  if (stages < 2) {                                          // wide ranks: one CTA per SM
    stages = static_cast<int>((static_cast<size_t>(227 * 1024) - kGmRingOffset) / stage);
    if (stages > kGmMaxStages) stages = kGmMaxStages;
  }
  size_t bytes = kGmRingOffset + stages * stage;
  const size_t merge = kGmRingOffset + (128 + 64 * static_cast<size_t>(max_rp_v + 1)) * sizeof(float);
  if (bytes < merge) bytes = merge;
  if (smem) *smem = bytes;
  return stages;
}

template <int NKS, int NVT, bool HI, bool FULL>
cudaError_t launch_gm_variant(const GqaDecodeParams& p, size_t smem, int stages, cudaStream_t s) {
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(decode_gqa_mma_kernel<NKS, NVT, HI, FULL>, smem, configured);
  if (ec != cudaSuccess) return ec;
  decode_gqa_mma_kernel<NKS, NVT, HI, FULL><<<dim3(p.B * p.H, p.splits), kGmThreads, smem, s>>>(p, stages);
  return cudaGetLastError();
}
template <int NKS, int NVT>
cudaError_t launch_gm_shape(const GqaDecodeParams& p, bool full, size_t smem, int stages, cudaStream_t s) {
  if (p.group > 8)
    return full ? launch_gm_variant<NKS, NVT, true, true>(p, smem, stages, s) : launch_gm_variant<NKS, NVT, true, false>(p, smem, stages, s);
  return full ? launch_gm_variant<NKS, NVT, false, true>(p, smem, stages, s) : launch_gm_variant<NKS, NVT, false, false>(p, smem, stages, s);
}

}  // namespace

size_t decode_gqa_mma_smem_bytes(int max_rp_k, int max_rp_v) {
  size_t smem = 0;
  return gm_stages(max_rp_k, max_rp_v, &smem) >= 2 ? smem : 0;
}

cudaError_t launch_decode_gqa_mma(const GqaDecodeParams& p, int max_rp, int min_rp, cudaStream_t s, uint64_t* launches) {
  size_t smem = 0;
  const int stages = gm_stages(max_rp, max_rp, &smem);
  if (stages < 2) return cudaErrorInvalidConfiguration;
  cudaError_t e;
  if (max_rp <= 64) e = launch_gm_shape<4, 8>(p, min_rp == 64, smem, stages, s);
  else if (max_rp <= 80) e = launch_gm_shape<5, 10>(p, min_rp == 80, smem, stages, s);
  else e = launch_gm_shape<8, 16>(p, min_rp == 128, smem, stages, s);
  if (e != cudaSuccess) return e;
  ++*launches;
  return launch_gqa_combine(p, s, launches);
}

}  // namespace ea
