// Decode over the 4-bit codes of the quantised rank-r cache (Section 5.3 of the paper) on the integer tensor-core
// path: the codes never become floats.
//
//   score_i = sum_c (n_ic - 8) s_c q'_c          n = stored nibble, s_c = key scale of the block, q' scaled to base 2
//   o'_c    = sum_i (n_ic - 8) s_ig p_i          s_ig = value scale of row i and channel group g, p_i = 2^(score_i - m)
//
// Both sums are 8-bit integer products with 32-bit accumulators (mma.sync m16n8k32).  A nibble word becomes two
// operand registers with two masks and no shift: w & 0x0F0F0F0F holds nibbles 0, 2, 4, 6 as bytes, w & 0xF0F0F0F0
// holds 16 times nibbles 1, 3, 5, 7; the factor 16 is taken out of the other operand (the fixed-point value of an
// odd channel, or of an odd row in the second product, is formed with a 16 times smaller scale, so it has four bits
// fewer).  The real-valued factor goes into the other operand as fixed-point digits, one digit per operand column:
//   keys:   x_c = q'_c s_c of a block -> F_c = rint(x_c 2^19 / 2^E) with 2^E above the block's largest |x_c|;
//           the three signed bytes of F_c are columns 0..2, score = 2^(E-19) (sum_n 256^n D_n - 8 sum_c F_c).
//   values: w_ig = p_i s_ig -> F = rint(w_ig kappa), an unsigned 32-bit integer whose four bytes are columns 0..3;
//           kappa = (2^30 - 1024) / S with S a power of two above every value scale met so far, and p <= 4 because the
//           running maximum is raised as soon as a score exceeds it by 2.  The accumulators stay integers from
//           block to block; they are folded into fp32 (o' += sum_n 256^n D_n - 8 sum_i F_i, times 1/kappa) only when
//           the maximum or S is raised, every 1024 blocks, and at the end.
// A warp owns 32 rows of every 128-row stage and walks the stages on its own; the stages arrive through a ring of
// bulk copies.  Code layout of a block (written by quantize_blocks_kernel for 4-bit codes):
//   keys:   [rp_k/8][G] words, word j of row i (channels 8j..8j+7) at j G + ((i + 8 (j & 3)) mod G): the rotation by
//           8 rows per word makes the fragment loads of a warp (8 rows x 4 words) hit 32 different banks.
//   values: chunks of min(G, 32) rows; a chunk is [rp_v][rows/8] words, word (c, o) holding rows 8o..8o+7 of channel c:
//           the contraction of the second product runs over rows, so a word must hold rows.
// Rows not quantised yet are attended from the 16-bit cache by the warps of the last split, one row per warp at a
// time.  Every wait is bounded.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stddef.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kMThreads = 128;
constexpr int kMStages = 3;
constexpr int kMStageRows = 128;
constexpr uint32_t kNib = 0x0F0F0F0Fu, kNibHi = 0xF0F0F0F0u;
constexpr unsigned kFull = 0xffffffffu;
constexpr float kRaise = 2.f;            // the running maximum is raised when a score exceeds it by this much
constexpr int kFlushBlocks = 1024;       // 1024 blocks x (16 rows x 240 + 16 rows x 15) x 255 < 2^30

struct __align__(16) MmaSmemHeader {
  unsigned long long full[kMStages];
  int done[kMStages];
  int abort_flag;
  float wmax[4], wsum[4], wfac[4];
  __align__(16) float qraw[128];
  __align__(16) float qp[128];           // q' * log2(e)/sqrt(d_head)
};
constexpr int kMHeaderBytes = 1152;
static_assert(sizeof(MmaSmemHeader) <= kMHeaderBytes, "header overlaps the warps' areas");

// per warp: digits of q' s [NB][3][kDigitStride] bytes, digits of the weights [NVG][4][32] bytes, o' in fp32 [128]
constexpr int kDigitStride = 144;        // 128 channels + 16: the three digit rows of a block start 4 banks apart
constexpr int kQdBytes = 3 * kDigitStride;
__host__ __device__ constexpr int warp_area_bytes(int nb, int nvg) { return nb * kQdBytes + nvg * 128 + 512; }
__host__ __device__ constexpr int ring_offset(int nb, int nvg) { return (kMHeaderBytes + 4 * warp_area_bytes(nb, nvg) + 127) & ~127; }

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_u8u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, d));
  return v;
}

// NKS: 32-channel steps of the widest key row; NMT: 16-channel tiles of the widest value row; G: group size;
// FULL: every head's padded key and value ranks are 16 NMT (no per-word, per-tile or per-group guards).
template <int NKS, int NMT, int G, bool FULL>
__global__ void __launch_bounds__(kMThreads, 5) decode_quant_mma_kernel(const QuantParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  constexpr int gshift = G == 16 ? 4 : G == 32 ? 5 : G == 64 ? 6 : 7;
  constexpr int bps = kMStageRows >> gshift;                    // blocks per stage
  constexpr int NVG = (16 * NMT + G - 1) / G;                   // value scale groups a row can have
  constexpr int NB = G == 16 ? 2 : 1;                           // blocks the 32 rows of a warp span
  constexpr int kArea = warp_area_bytes(NB, NVG);
  MmaSmemHeader* hdr = reinterpret_cast<MmaSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tig = lane & 3;
  unsigned char* qd = smem + kMHeaderBytes + warp * kArea;      // [NB][3][128]
  unsigned char* pd = qd + NB * kQdBytes;                            // [NVG][4][32]
  float* ow = reinterpret_cast<float*>(pd + NVG * 128);         // [128]
  unsigned char* ring = smem + ring_offset(NB, NVG);
  const int unit_i = blockIdx.x, split = blockIdx.y;
  const int h = unit_i / p.B, b = unit_i - h * p.B;
  const HeadInfo hd = p.heads[h];
  const QuantHead qh = p.qheads[h];
  const int n_b = p.deficit != nullptr ? p.n - __ldg(p.deficit + b) : p.n;      // this sequence's rows
  const int nq_b = p.qlens != nullptr ? __ldg(p.qlens + b) : p.nq;              // ... of which held as codes
  const int nqb = nq_b >> gshift;
  const int rp_k = FULL ? 16 * NMT : hd.rp_k, rp_v = FULL ? 16 * NMT : hd.rp_v;
  const int nwk = rp_k >> 3, nks = FULL ? NKS : (rp_k + 31) >> 5, nmt = FULL ? NMT : (rp_v + 15) >> 4;
  const int nvg = FULL ? NVG : qh.nvg;
  const int stage_stride = (bps * qh.block_bytes + 127) & ~127;
  const int nst_b = (nq_b + kMStageRows - 1) / kMStageRows;
  const int per = (nst_b + p.splits - 1) / p.splits;
  const int s_lo = min(nst_b, split * per), s_hi = min(nst_b, s_lo + per);
  const char* slab = p.qcache + qh.slab_off + static_cast<int64_t>(b) * p.blocks_max * qh.block_bytes;

  if (tid == 0) {
    for (int s = 0; s < kMStages; ++s) {
      mbar_init(&hdr->full[s], 1);
      hdr->done[s] = 0;
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const uint64_t policy = policy_evict_first();
  auto issue = [&](int s, int slot) {                           // one thread
    const int nblk = min(bps, nqb - s * bps);
    const uint32_t bytes = static_cast<uint32_t>(nblk) * qh.block_bytes;
    mbar_arrive_expect_tx(&hdr->full[slot], bytes);
    bulk_load(ring + slot * stage_stride, slab + static_cast<int64_t>(s) * bps * qh.block_bytes, bytes,
              &hdr->full[slot], policy);
  };
  if (tid == 0)
    for (int i = 0; i < kMStages && s_lo + i < s_hi; ++i) issue(s_lo + i, i);

  // q' = q U^K, scaled into the base-2 domain
  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(p.q);
  if (p.flags & 0x1u) {
    if (tid < hd.rp_k) hdr->qp[tid] = __bfloat162float(q[b * p.q_stride_b + hd.lr_k_off + tid]) * p.q_scale;
  } else {
    if (tid < p.d_head) hdr->qraw[tid] = __bfloat162float(q[b * p.q_stride_b + static_cast<int64_t>(h) * p.d_head + tid]);
    __syncthreads();
    if (tid < hd.rp_k) {
      const float* U = p.basis + hd.uk_off + tid;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
      for (int d = 0; d < p.d_head; d += 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = fmaf(hdr->qraw[d + i], __ldg(U + (d + i) * hd.rp_k), acc[i]);
      }
      hdr->qp[tid] = ((acc[0] + acc[1]) + (acc[2] + acc[3])) * p.q_scale;
    }
  }
  for (int c = lane; c < 128; c += 32) ow[c] = 0.f;
  __syncthreads();

  int oacc[NMT][4];
#pragma unroll
  for (int i = 0; i < NMT; ++i)
#pragma unroll
    for (int k = 0; k < 4; ++k) oacc[i][k] = 0;
  float sig[NVG];                    // this lane's share of sum_i F_i per value group
#pragma unroll
  for (int g = 0; g < NVG; ++g) sig[g] = 0.f;
  float m = -INFINITY, l = 0.f;      // m is the same in every lane of the warp; l is this lane's share
  float S = 0.f, kappa = 0.f, unit = 0.f;
  int since_flush = 0;
  const float slope2 = hd.alibi_slope2;
  const int pos_q = n_b - 1;

  // integer accumulators -> ow[] (fp32, under the current maximum and scale)
  auto flush = [&]() {
    float sg[NVG];
#pragma unroll
    for (int g = 0; g < NVG; ++g) {
      sg[g] = warp_sum((gid & 1) ? 16.f * sig[g] : sig[g]);
      sig[g] = 0.f;
    }
#pragma unroll
    for (int mt = 0; mt < NMT; ++mt)
      if (mt < nmt) {
        const int g = (16 * mt) >> gshift;
        // even lanes of a pair hold digits 0 and 1, odd lanes digits 2 and 3
        const float lo = (tig & 1) ? 65536.f : 1.f, hi = (tig & 1) ? 16777216.f : 256.f;
        float va = fmaf(hi, static_cast<float>(oacc[mt][1]), lo * static_cast<float>(oacc[mt][0]));
        float vb = fmaf(hi, static_cast<float>(oacc[mt][3]), lo * static_cast<float>(oacc[mt][2]));
        va += __shfl_xor_sync(kFull, va, 1);
        vb += __shfl_xor_sync(kFull, vb, 1);
        if (tig == 0) {
          ow[16 * mt + gid] = fmaf(unit, va - 8.f * sg[g], ow[16 * mt + gid]);
          ow[16 * mt + gid + 8] = fmaf(unit, vb - 8.f * sg[g], ow[16 * mt + gid + 8]);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) oacc[mt][k] = 0;
      }
    __syncwarp();
    since_flush = 0;
  };
  auto rescale = [&](float mx) {     // mx: the new maximum, the same in every lane
    flush();
    const float f = ex2(m - mx);
    l *= f;
    for (int c = lane; c < 128; c += 32) ow[c] *= f;
    __syncwarp();
    m = mx;
  };

  // what a lane's loads depend on besides the stage: word offsets of its key rows, its row, its digit positions
  const int r0 = warp * 32, blk0 = r0 >> gshift;
  const int rho = 8 * tig + gid;                   // the row of the warp's 32 this lane owns after the score products
  int koff[2][2];                                  // [tile][row gid / gid + 8]: word offset in the block's key codes
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int ro = (r0 + 16 * t) & (G - 1);
    koff[t][0] = tig * G + ((ro + gid + 8 * tig) & (G - 1));
    koff[t][1] = tig * G + ((ro + gid + 8 + 8 * tig) & (G - 1));
  }
  const int kpos0 = ((lane & 1) << 4) | (((lane >> 3) & 3) << 2) | ((lane >> 1) & 3);   // channel lane + 32 k -> 32 k + kpos0
  const int ppos = ((rho & 1) << 4) | ((rho >> 3) << 2) | ((rho >> 1) & 3);
  const int dn = gid & 3;                          // operand columns 4..7 repeat 0..3
  const int odd4 = (lane & 1) << 2;                // channel lane + 32 k is odd: its fixed-point value is 16 times coarser

  for (int s = s_lo; s < s_hi; ++s) {
    const int it = s - s_lo, slot = it % kMStages;
    if (__any_sync(kFull, !mbar_wait(&hdr->full[slot], (it / kMStages) & 1, p.status))) {
      hdr->abort_flag = 1;
      break;
    }
    const unsigned char* st = ring + slot * stage_stride;
    const int nblk = min(bps, nqb - s * bps);
    if (blk0 < nblk) {
      // ---- digits of x_c = q'_c s_c for the warp's block(s)
      int corr[NB];
      float delta[NB];
#pragma unroll
      for (int i = 0; i < NB; ++i) {
        const bool have = i == 0 || blk0 + i < nblk;
        const __half* ks = reinterpret_cast<const __half*>(st + (blk0 + i) * qh.block_bytes + qh.ks_off);
        float x[NKS];
        uint32_t ab = 0;
#pragma unroll
        for (int k = 0; k < NKS; ++k) {
          const int c = lane + 32 * k;
          x[k] = (have && c < rp_k) ? hdr->qp[c] * __half2float(ks[c]) : 0.f;
          ab = max(ab, __float_as_uint(x[k]) & 0x7fffffffu);
        }
        ab = __reduce_max_sync(kFull, ab);
        const int e = max(static_cast<int>(ab >> 23), 40);               // every |x| < 2^(e - 126)
        // 2^(19 - (e - 126)); odd channels meet 16 n in the product and take 2^(15 - (e - 126))
        const float sc = __uint_as_float(static_cast<uint32_t>(272 - e - odd4) << 23);
        delta[i] = __uint_as_float(static_cast<uint32_t>(e - 18) << 23);           // 2^((e - 126) - 19)
        int fs = 0;
#pragma unroll
        for (int k = 0; k < NKS; ++k) {
          const int c = lane + 32 * k;
          const int F = __float2int_rn(x[k] * sc);
          fs += F << odd4;
          const uint32_t u = static_cast<uint32_t>(F + 0x808080) ^ 0x808080u;      // three signed bytes
          unsigned char* dst = qd + i * kQdBytes + 32 * k + kpos0;
          dst[0] = static_cast<unsigned char>(u);
          dst[kDigitStride] = static_cast<unsigned char>(u >> 8);
          dst[2 * kDigitStride] = static_cast<unsigned char>(u >> 16);
        }
        corr[i] = 8 * __reduce_add_sync(kFull, fs);
      }
      __syncwarp();
      uint32_t bq[NB][NKS][2];
#pragma unroll
      for (int i = 0; i < NB; ++i)
#pragma unroll
        for (int k = 0; k < NKS; ++k) {
          const uint32_t* src = reinterpret_cast<const uint32_t*>(qd + i * kQdBytes + (dn < 3 ? dn : 0) * kDigitStride + 32 * k + 4 * tig);
          bq[i][k][0] = dn < 3 ? src[0] : 0u;
          bq[i][k][1] = dn < 3 ? src[4] : 0u;
        }

      // ---- scores of the 32 rows: two tiles of 16 rows
      int tot[2][2];
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int bi = G == 16 ? t : 0;
        const uint32_t* kc = reinterpret_cast<const uint32_t*>(st + ((r0 + 16 * t) >> gshift) * qh.block_bytes);
        int acc[4] = {0, 0, 0, 0};
#pragma unroll
        for (int k = 0; k < NKS; ++k)
          if (k < nks) {
            const int j = 4 * k + tig;
            const bool ok = (FULL && 4 * k + 3 < 2 * NMT) || j < nwk;
            const uint32_t wa = ok ? kc[4 * k * G + koff[t][0]] : 0u;
            const uint32_t wb = ok ? kc[4 * k * G + koff[t][1]] : 0u;
            mma_u8s8(acc, wa & kNib, wb & kNib, wa & kNibHi, wb & kNibHi, bq[bi][k][0], bq[bi][k][1]);
          }
        // even lanes of a pair hold digits 0 and 1 of rows gid and gid + 8, odd lanes digit 2 (and a zero column)
        const int ka = (tig & 1) ? 65536 : 1, kb = (tig & 1) ? 0 : 256;
        int v0 = acc[0] * ka + acc[1] * kb, v1 = acc[2] * ka + acc[3] * kb;
        v0 += __shfl_xor_sync(kFull, v0, 1);
        v1 += __shfl_xor_sync(kFull, v1, 1);
        tot[t][0] = v0 - corr[bi];
        tot[t][1] = v1 - corr[bi];
      }
      // lane (gid, tig) owns row rho = 8 tig + gid of the warp's 32: tile tig >> 1, half tig & 1
      const int mine = (tig & 2) ? ((tig & 1) ? tot[1][1] : tot[1][0]) : ((tig & 1) ? tot[0][1] : tot[0][0]);
      const float dl = (G == 16 && (tig & 2)) ? delta[NB - 1] : delta[0];
      const int rblk = (r0 + rho) >> gshift, ri = (r0 + rho) & (G - 1);
      const bool valid = NB == 1 || rblk < nblk;
      const int j_abs = s * kMStageRows + r0 + rho;
      const float score = valid ? fmaf(slope2, static_cast<float>(j_abs - pos_q), static_cast<float>(mine) * dl) : -INFINITY;
      if (__any_sync(kFull, score > m + kRaise)) rescale(warp_max(score));
      const float pr = ex2(score - m);
      l += pr;

      // ---- digits of the weights p_i s_ig
      const __half* vs = reinterpret_cast<const __half*>(st + rblk * qh.block_bytes + qh.vs_off) + ri;
      float wv[NVG];
      float smax = 0.f;
#pragma unroll
      for (int g = 0; g < NVG; ++g) {
        const float sv = (valid && (FULL || g < nvg)) ? __half2float(vs[g * G]) : 0.f;
        smax = fmaxf(smax, sv);
        wv[g] = pr * sv;
      }
      if (__any_sync(kFull, smax >= S)) {          // a larger value scale: fold what was accumulated under the old one
        const uint32_t sb = __reduce_max_sync(kFull, __float_as_uint(smax));
        flush();
        const uint32_t e = max(sb >> 23, 64u);
        S = __uint_as_float((e + 1u) << 23);       // a power of two above every scale so far
        // 2^30 - 1024: p <= 4 keeps p s kappa below 2^32; odd rows meet 16 n in the product and take kappa / 16
        kappa = ((gid & 1) ? 67108800.f : 1073740800.f) / S;
        unit = S / 1073740800.f;
      }
#pragma unroll
      for (int g = 0; g < NVG; ++g)
        if (FULL || g < nvg) {
          const uint32_t F = __float2uint_rn(wv[g] * kappa);
          sig[g] += static_cast<float>(F);
          unsigned char* dst = pd + g * 128 + ppos;
          dst[0] = static_cast<unsigned char>(F);
          dst[32] = static_cast<unsigned char>(F >> 8);
          dst[64] = static_cast<unsigned char>(F >> 16);
          dst[96] = static_cast<unsigned char>(F >> 24);
        }
      __syncwarp();
      uint32_t pb[NVG][2];
#pragma unroll
      for (int g = 0; g < NVG; ++g) {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(pd + g * 128 + dn * 32 + 4 * tig);
        pb[g][0] = (FULL || g < nvg) ? src[0] : 0u;
        pb[g][1] = (FULL || g < nvg) ? src[4] : 0u;
      }

      // ---- weighted sums: tiles of 16 channels, contraction over the 32 rows
      const uint32_t* vw;
      int wstride, woff;                           // word (c, oct tig) at vw[c * wstride + woff]
      if (G == 16) {
        vw = reinterpret_cast<const uint32_t*>(st + (blk0 + (tig >> 1)) * qh.block_bytes + qh.vc_off);
        wstride = 2;
        woff = tig & 1;
      } else {
        vw = reinterpret_cast<const uint32_t*>(st + blk0 * qh.block_bytes + qh.vc_off) + ((r0 & (G - 1)) >> 5) * rp_v * 4;
        wstride = 4;
        woff = tig;
      }
#pragma unroll
      for (int mt = 0; mt < NMT; ++mt)
        if (mt < nmt) {
          const int g = (16 * mt) >> gshift;
          const int c = 16 * mt + gid;
          const uint32_t wa = (FULL || c < rp_v) ? vw[c * wstride + woff] : 0u;
          const uint32_t wb = (FULL || c + 8 < rp_v) ? vw[(c + 8) * wstride + woff] : 0u;
          mma_u8u8(oacc[mt], wa & kNib, wb & kNib, wa & kNibHi, wb & kNibHi, pb[g][0], pb[g][1]);
        }
      if (++since_flush >= kFlushBlocks) flush();
    }
    // this warp is done with the slot (and with its digit areas)
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();       // the warp's reads of the slot come before the count that may trigger the refill
      if ((atomicAdd(&hdr->done[slot], 1) & 3) == 3 && s + kMStages < s_hi) issue(s + kMStages, slot);
    }
  }
  __syncthreads();
  const bool aborted = *reinterpret_cast<volatile int*>(&hdr->abort_flag) != 0;

  // rows that are not quantised yet, straight from the 16-bit cache: the warps of the last split, a row at a time
  if (split == p.splits - 1 && !aborted) {
    for (int j = nq_b + warp; j < n_b; j += 4) {
      const int64_t row = static_cast<int64_t>(b) * p.n_max + j;
      const __nv_bfloat16* kr = reinterpret_cast<const __nv_bfloat16*>(p.cache + hd.k_off + row * hd.rp_k * 2);
      const __nv_bfloat16* vr = reinterpret_cast<const __nv_bfloat16*>(p.cache + hd.v_off + row * hd.rp_v * 2);
      float part = 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = lane + 32 * k;
        if (c < hd.rp_k) part = fmaf(hdr->qp[c], __bfloat162float(kr[c]), part);
      }
      const float sc = fmaf(slope2, static_cast<float>(j - pos_q), warp_sum(part));
      if (sc > m + kRaise) rescale(sc);
      const float pr = ex2(sc - m);
      if (lane == 0) l += pr;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int c = lane + 32 * k;
        if (c < hd.rp_v) ow[c] = fmaf(pr, __bfloat162float(vr[c]), ow[c]);
      }
    }
  }
  flush();

  // ---- merge the four warps into one partial (max, sum, o'[rp_v])
  if (lane == 0) hdr->wmax[warp] = m;
  __syncthreads();
  const float M = fmaxf(fmaxf(hdr->wmax[0], hdr->wmax[1]), fmaxf(hdr->wmax[2], hdr->wmax[3]));
  const float f = (m == -INFINITY) ? 0.f : ex2(m - M);
  const float ls = warp_sum(l * f);
  if (lane == 0) {
    hdr->wsum[warp] = ls;
    hdr->wfac[warp] = f;
  }
  __syncthreads();
  float* part = p.partials + (static_cast<size_t>(unit_i) * p.splits + split) * p.part_stride;
  if (tid < hd.rp_v) {
    float acc = 0.f;
    if (!aborted)
#pragma unroll
      for (int w = 0; w < 4; ++w)
        acc = fmaf(reinterpret_cast<const float*>(smem + kMHeaderBytes + w * kArea + NB * kQdBytes + NVG * 128)[tid], hdr->wfac[w], acc);
    part[4 + tid] = acc;
  }
  if (tid == 0) {
    part[0] = M;
    part[1] = (hdr->wsum[0] + hdr->wsum[1]) + (hdr->wsum[2] + hdr->wsum[3]);
  }
}

template <int NKS, int NMT, int G, bool FULL>
cudaError_t launch_mma_variant(const QuantParams& p, size_t smem, cudaStream_t s) {
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(decode_quant_mma_kernel<NKS, NMT, G, FULL>, smem, configured);
  if (ec != cudaSuccess) return ec;
  decode_quant_mma_kernel<NKS, NMT, G, FULL><<<dim3(p.B * p.H, p.splits), kMThreads, smem, s>>>(p);
  return cudaGetLastError();
}
template <int NKS, int NMT>
cudaError_t launch_mma_group(const QuantParams& p, bool full, size_t smem, cudaStream_t s) {
  switch (p.group) {
    case 16: return full ? launch_mma_variant<NKS, NMT, 16, true>(p, smem, s) : launch_mma_variant<NKS, NMT, 16, false>(p, smem, s);
    case 32: return full ? launch_mma_variant<NKS, NMT, 32, true>(p, smem, s) : launch_mma_variant<NKS, NMT, 32, false>(p, smem, s);
    case 64: return full ? launch_mma_variant<NKS, NMT, 64, true>(p, smem, s) : launch_mma_variant<NKS, NMT, 64, false>(p, smem, s);
    default: return full ? launch_mma_variant<NKS, NMT, 128, true>(p, smem, s) : launch_mma_variant<NKS, NMT, 128, false>(p, smem, s);
  }
}
// the template arguments a layer's widest padded rank selects
void mma_shape(int max_rp, int* nks, int* nmt) {
  if (max_rp <= 64) { *nks = 2; *nmt = 4; }
  else if (max_rp <= 80) { *nks = 3; *nmt = 5; }
  else { *nks = 4; *nmt = 8; }
}

}  // namespace

size_t decode_quant_mma_smem_bytes(int max_stage_bytes, int max_rp, int group) {
  int nks, nmt;
  mma_shape(max_rp, &nks, &nmt);
  const int nvg = (16 * nmt + group - 1) / group, nb = group == 16 ? 2 : 1;
  return ring_offset(nb, nvg) + static_cast<size_t>(kMStages) * ((max_stage_bytes + 127) & ~127);
}

cudaError_t launch_decode_quant_mma(const QuantParams& p, int max_rp, int min_rp, size_t smem, cudaStream_t s,
                                    uint64_t* launches) {
  cudaError_t e;
  if (max_rp <= 64) e = launch_mma_group<2, 4>(p, min_rp == 64, smem, s);
  else if (max_rp <= 80) e = launch_mma_group<3, 5>(p, min_rp == 80, smem, s);
  else e = launch_mma_group<4, 8>(p, min_rp == 128, smem, s);
  if (e != cudaSuccess) return e;
  ++*launches;
  return launch_quant_combine(p, s, launches);
}

}  // namespace ea
