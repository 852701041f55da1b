// Quantised rank-r cache (Section 5.3 of the paper, "Eigen Attention with Quantization"; sizes in Table 8):
// keys per channel, values per token, integer codes of 3 or 4 bits with one half-precision scale per group of G.
//
//   qmax = 2^(bits-1) - 1,  s = half( min(max|x| / qmax, 65504) ),  c = clip( rint(x / s), -qmax, qmax ),  x^ = c * s
//   (c + qmax + 1 is stored)
//
// A key group is G consecutive tokens of one channel, a value group is G consecutive channels of one token.
// Rows that do not fill a block of G tokens yet stay in the 16-bit cache and are attended from there.
//
// quantize_blocks_kernel: one CTA per (sequence, head, block); reads the block's G rows of K' and V' from the
//   16-bit cache, takes the group maxima, writes codes and scales.  Divisions are IEEE single precision and the
//   rounding is to nearest even, so the codes are a function of the stored rows alone.
// decode_quant_kernel: split-KV decode over the codes.  A CTA owns a run of 128-row stages of one unit; one
//   thread streams them into a shared-memory ring with bulk copies, every thread owns one row of a stage.  The
//   key scales are folded into the query once per block (q'_c * s_c), the value scale into the softmax weight
//   (p * s_g), so a cached element costs one mask, half a packed subtract and half a packed multiply-add.
//   A nibble is turned into a float without a conversion instruction: masked in place and OR-ed with the
//   exponent whose unit in the last place lines up with the nibble's lowest bit, (w & (15 << 4k)) | E_k is
//   2^(23-4k) + nibble exactly; subtracting 2^(23-4k) + 8 leaves the signed code.
// quant_combine_kernel: merges the splits of a unit, normalises and lifts through (U^V)^T.
// Every wait is bounded.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stddef.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kQThreads = 128;
constexpr int kQStages = 4;           // ring slots of the decode kernel
constexpr int kStageRows = 128;

// ---------------------------------------------------------------- quantiser

// clip(rint(x / s), -qmax, qmax) + qmax + 1: the stored (unsigned) code
__device__ __forceinline__ uint32_t stored_code(float x, float s, float qmax) {
  float c = s > 0.f ? rintf(x / s) : 0.f;
  c = fminf(fmaxf(c, -qmax), qmax);
  return static_cast<uint32_t>(static_cast<int>(c + qmax) + 1);
}

__global__ void __launch_bounds__(kQThreads) quantize_blocks_kernel(const QuantParams p) {
  __shared__ __align__(16) __nv_bfloat16 tile[128 * 128];   // G rows x rp (row-major), K' then V'
  __shared__ float scale_sm[256];                         // K: [rp_k]; V: [nvg][G]
  const int tid = threadIdx.x;
  const int unit = blockIdx.x, blk = p.b0 + blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const QuantHead qh = p.qheads[h];
  const int G = p.group;
  if (p.qlens != nullptr) {   // unequal lengths: this sequence's own range of complete blocks not quantised yet
    const int n_b = p.n - (p.deficit != nullptr ? __ldg(p.deficit + b) : 0);
    if (blk < __ldg(p.qlens + b) / G || blk >= n_b / G) return;
  }
  const float qmax = p.bits == 3 ? 3.f : 7.f;
  const int64_t row0 = static_cast<int64_t>(b) * p.n_max + static_cast<int64_t>(blk) * G;
  char* dst = p.qcache + qh.slab_off + (static_cast<int64_t>(b) * p.blocks_max + blk) * qh.block_bytes;

  for (int pass = 0; pass < 2; ++pass) {
    const int rp = pass ? hd.rp_v : hd.rp_k;
    const uint4* src = reinterpret_cast<const uint4*>(p.cache + (pass ? hd.v_off : hd.k_off) + row0 * rp * 2);
    const int chunks = G * rp / 8;
    for (int i = tid; i < chunks; i += kQThreads) reinterpret_cast<uint4*>(tile)[i] = src[i];
    __syncthreads();
    if (pass == 0) {          // keys: one scale per channel over the block's G tokens
      __half* ks = reinterpret_cast<__half*>(dst + qh.ks_off);
      for (int c = tid; c < rp; c += kQThreads) {
        float amax = 0.f;
        for (int r = 0; r < G; ++r) amax = fmaxf(amax, fabsf(__bfloat162float(tile[r * rp + c])));
        const __half s16 = __float2half_rn(fminf(amax / qmax, 65504.f));
        ks[c] = s16;
        scale_sm[c] = __half2float(s16);
      }
    } else {                  // values: one scale per token and G channels
      __half* vs = reinterpret_cast<__half*>(dst + qh.vs_off);
      for (int i = tid; i < qh.nvg * G; i += kQThreads) {
        const int g = i / G, r = i - g * G;
        const int c1 = min(rp, (g + 1) * G);
        float amax = 0.f;
        for (int c = g * G; c < c1; ++c) amax = fmaxf(amax, fabsf(__bfloat162float(tile[r * rp + c])));
        const __half s16 = __float2half_rn(fminf(amax / qmax, 65504.f));
        vs[i] = s16;
        scale_sm[i] = __half2float(s16);
      }
    }
    __syncthreads();
    char* code_base = dst + (pass ? qh.vc_off : 0);
    const int words = (rp / 8) * G;
    if (p.bits == 4 && pass == 1) {
      // 4-bit values: chunks of min(G, 32) rows, a chunk [rp][rows / 8] words, a word = eight rows of one channel
      const int opc = (G < 32 ? G : 32) / 8;
      for (int i = tid; i < words; i += kQThreads) {
        const int qc = i / (rp * opc), rem = i - qc * rp * opc;
        const int c = rem / opc, o = rem - c * opc;
        uint32_t w = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int r = qc * 32 + o * 8 + k;
          w |= stored_code(__bfloat162float(tile[r * rp + c]), scale_sm[(c / G) * G + r], qmax) << (4 * k);
        }
        reinterpret_cast<uint32_t*>(code_base)[i] = w;
      }
    } else {
      for (int i = tid; i < words; i += kQThreads) {
        const int j = i / G, r = i - j * G;
        uint32_t w = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int c = 8 * j + k;
          const float s = pass ? scale_sm[(c / G) * G + r] : scale_sm[c];
          w |= stored_code(__bfloat162float(tile[r * rp + c]), s, qmax) << (p.bits * k);
        }
        if (p.bits == 4) {      // keys: the word of row r sits 8 (j mod 4) rows further on (modulo G)
          reinterpret_cast<uint32_t*>(code_base)[j * G + ((r + 8 * (j & 3)) & (G - 1))] = w;
        } else {                // two planes: low 16 bits of every unit, then the high 8 bits
          reinterpret_cast<uint16_t*>(code_base)[i] = static_cast<uint16_t>(w);
          reinterpret_cast<uint8_t*>(code_base + 2 * words)[i] = static_cast<uint8_t>(w >> 16);
        }
      }
    }
    __syncthreads();          // the tile and the scales are reused by the second pass
  }
}

// ---------------------------------------------------------------- decode over the codes

struct __align__(16) QuantSmemHeader {
  unsigned long long full[kQStages];
  int done[kQStages];      // running count of warps that have finished with a stage in the slot (4 per stage)
  int abort_flag;
  float wmax[4], wsum[4];
  __align__(16) float qraw[128];   // the unit's query as fp32
  __align__(16) float qp[128];     // q' * log2(e)/sqrt(d_head); read 16 bytes at a time
};
static_assert(offsetof(QuantSmemHeader, qp) % 16 == 0, "q' is read with 16-byte loads");
constexpr int kQsOffset = 2048;                     // per warp: q'_c * s_c of (up to) two blocks, [2][128] floats
constexpr int kRingOffset = kQsOffset + 4 * 2 * 128 * 4;
static_assert(sizeof(QuantSmemHeader) <= kQsOffset, "header overlaps the scaled-query area");

// Two 32-bit patterns as one 64-bit register pair (low word first).  Written as integer arithmetic so that the
// compiler assigns the halves in place; a move instruction per half would double the cost of a cached element.
__device__ __forceinline__ unsigned long long pair_of(uint32_t lo, uint32_t hi) {
  return static_cast<unsigned long long>(lo) | (static_cast<unsigned long long>(hi) << 32);
}
__device__ __forceinline__ unsigned long long pair_of(float lo, float hi) {
  return pair_of(__float_as_uint(lo), __float_as_uint(hi));
}
__device__ __forceinline__ float low_plus_high(unsigned long long v) {
  return __uint_as_float(static_cast<uint32_t>(v)) + __uint_as_float(static_cast<uint32_t>(v >> 32));
}

// Eight codes of a word as four packed float pairs (exact small integers in -7..7; a nibble 0 gives -8).
// Nibbles 0..3 sit at bits 0, 4, 8, 12 and meet the exponents of 2^23, 2^19, 2^15, 2^11; nibbles 4..7 do the
// same after a shift by 16, so two packed constants serve the whole word.  3-bit codes: fields at bits 0, 3, 6, 9
// meet 2^23, 2^20, 2^17, 2^14, fields 4..7 after a shift by 12; the stored code is c + 4.
struct Consts {
  unsigned long long c01, c23;
  uint32_t e23, e19, e15, e11;         // exponent patterns of 2^23, 2^19, 2^15, 2^11 (3-bit: 2^23, 2^20, 2^17, 2^14)
};
// The exponent patterns come in as kernel arguments, not as literals: (w & mask) | pattern is one logic
// instruction when the pattern sits in a register; with two literals the compiler emits a second logic
// instruction and a move per element (counted on the device: 327 logic + 160 moves per row instead of 160).
template <int BITS>
__device__ __forceinline__ Consts make_consts(const QuantParams& p) {
  Consts c;
  c.e23 = p.magic[0]; c.e19 = p.magic[1]; c.e15 = p.magic[2]; c.e11 = p.magic[3];
  if (BITS == 4) {
    c.c01 = pair_of(-8388616.f, -524296.f);          // -(2^23 + 8), -(2^19 + 8)
    c.c23 = pair_of(-32776.f, -2056.f);              // -(2^15 + 8), -(2^11 + 8)
  } else {
    c.c01 = pair_of(-8388612.f, -1048580.f);         // -(2^23 + 4), -(2^20 + 4)
    c.c23 = pair_of(-131076.f, -16388.f);            // -(2^17 + 4), -(2^14 + 4)
  }
  return c;
}
template <int BITS>
__device__ __forceinline__ void codes_to_floats(uint32_t w, const Consts& k, unsigned long long (&f)[4]) {
  if (BITS == 4) {
    const uint32_t u = w >> 16;
    f[0] = add2p(pair_of((w & 0x000Fu) | k.e23, (w & 0x00F0u) | k.e19), k.c01);
    f[1] = add2p(pair_of((w & 0x0F00u) | k.e15, (w & 0xF000u) | k.e11), k.c23);
    f[2] = add2p(pair_of((u & 0x000Fu) | k.e23, (u & 0x00F0u) | k.e19), k.c01);
    f[3] = add2p(pair_of((u & 0x0F00u) | k.e15, (u & 0xF000u) | k.e11), k.c23);
  } else {
    const uint32_t u = w >> 12;
    f[0] = add2p(pair_of((w & 0x007u) | k.e23, (w & 0x038u) | k.e19), k.c01);
    f[1] = add2p(pair_of((w & 0x1C0u) | k.e15, (w & 0xE00u) | k.e11), k.c23);
    f[2] = add2p(pair_of((u & 0x007u) | k.e23, (u & 0x038u) | k.e19), k.c01);
    f[3] = add2p(pair_of((u & 0x1C0u) | k.e15, (u & 0xE00u) | k.e11), k.c23);
  }
}
// The unit (eight channels 8j..8j+7) of row `ri` of a block's code area: a word, or the two planes of 3-bit codes
// (`units` = units of the whole area = (rp / 8) * G).
template <int BITS, int G>
__device__ __forceinline__ uint32_t load_unit(const unsigned char* area, int units, int j, int ri) {
  if (BITS == 4) return reinterpret_cast<const uint32_t*>(area)[j * G + ri];
  const uint32_t lo = reinterpret_cast<const uint16_t*>(area)[j * G + ri];
  const uint32_t hi = area[2 * units + j * G + ri];
  return lo | (hi << 16);
}
__device__ __forceinline__ void bf16x8_to_floats(const uint4& x, unsigned long long (&f)[4]) {
  f[0] = pair_of(x.x << 16, x.x & 0xffff0000u);
  f[1] = pair_of(x.y << 16, x.y & 0xffff0000u);
  f[2] = pair_of(x.z << 16, x.z & 0xffff0000u);
  f[3] = pair_of(x.w << 16, x.w & 0xffff0000u);
}

// NW: 8-channel words a row can have (widest padded rank / 8); G: group size (row offsets inside a block become
// immediates); FULL: every head has exactly NW words of keys and of values (no per-word guards).
template <int NW, int MINB, int G, bool FULL, int BITS>
__global__ void __launch_bounds__(kQThreads, MINB) decode_quant_kernel(const QuantParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  QuantSmemHeader* hdr = reinterpret_cast<QuantSmemHeader*>(smem);
  float* qs_w = reinterpret_cast<float*>(smem + kQsOffset) + (threadIdx.x >> 5) * 256;
  unsigned char* ring = smem + kRingOffset;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x, split = blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const QuantHead qh = p.qheads[h];
  constexpr int gshift = G == 16 ? 4 : G == 32 ? 5 : G == 64 ? 6 : 7;
  constexpr int bps = kStageRows >> gshift;                      // blocks per stage
  const int n_b = p.deficit != nullptr ? p.n - __ldg(p.deficit + b) : p.n;      // this sequence's rows
  const int nq_b = p.qlens != nullptr ? __ldg(p.qlens + b) : p.nq;              // ... of which held as codes
  const int nqb = nq_b >> gshift;                             // blocks held as codes
  const int nwk = hd.rp_k >> 3, nwv = hd.rp_v >> 3;
  const int stage_stride = (bps * qh.block_bytes + 127) & ~127;

  const int nst_b = (nq_b + kStageRows - 1) / kStageRows;     // the splits divide the sequence's own stages
  const int per = (nst_b + p.splits - 1) / p.splits;
  const int s_lo = min(nst_b, split * per), s_hi = min(nst_b, s_lo + per);
  const char* slab = p.qcache + qh.slab_off + static_cast<int64_t>(b) * p.blocks_max * qh.block_bytes;

  if (tid == 0) {
    for (int s = 0; s < kQStages; ++s) {
      mbar_init(&hdr->full[s], 1);
      hdr->done[s] = 0;
    }
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const uint64_t policy = policy_evict_first();
  auto issue = [&](int s, int slot) {                         // one thread
    const int nblk = min(bps, nqb - s * bps);
    const uint32_t bytes = static_cast<uint32_t>(nblk) * qh.block_bytes;
    mbar_arrive_expect_tx(&hdr->full[slot], bytes);
    bulk_load(ring + slot * stage_stride, slab + static_cast<int64_t>(s) * bps * qh.block_bytes, bytes,
              &hdr->full[slot], policy);
  };
  if (tid == 0)
    for (int i = 0; i < kQStages && s_lo + i < s_hi; ++i) issue(s_lo + i, i);

  // q' = q U^K, scaled into the base-2 domain
  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(p.q);
  if (p.flags & 0x1u) {
    if (tid < hd.rp_k) hdr->qp[tid] = __bfloat162float(q[b * p.q_stride_b + hd.lr_k_off + tid]) * p.q_scale;
  } else {
    if (tid < p.d_head) hdr->qraw[tid] = __bfloat162float(q[b * p.q_stride_b + static_cast<int64_t>(h) * p.d_head + tid]);
    __syncthreads();
    if (tid < hd.rp_k) {
      const float* U = p.basis + hd.uk_off + tid;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};       // d_head is a multiple of 8; four chains keep 32 loads in flight
#pragma unroll 8
      for (int d = 0; d < p.d_head; d += 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = fmaf(hdr->qraw[d + i], __ldg(U + (d + i) * hd.rp_k), acc[i]);
      }
      hdr->qp[tid] = ((acc[0] + acc[1]) + (acc[2] + acc[3])) * p.q_scale;
    }
  }
  __syncthreads();

  const Consts kc = make_consts<BITS>(p);
  unsigned long long o[NW * 4];
#pragma unroll
  for (int i = 0; i < NW * 4; ++i) o[i] = 0ull;
  float m = -INFINITY, l = 0.f;
  const float slope2 = hd.alibi_slope2;
  const int pos_q = n_b - 1;
  // online softmax of one score: returns the weight of the row under the (possibly raised) running maximum
  // (the maximum is only raised when a score exceeds it by more than 8: weights stay below 2^8, and a warp
  // leaves the common path only when one of its lanes meets such a score)
  auto weight = [&](float s) {
    if (s > m + 8.f) {
      const float c = ex2(m - s);
      const unsigned long long cc = pair_of(c, c);
      l *= c;
#pragma unroll
      for (int i = 0; i < NW * 4; ++i) o[i] = mul2p(o[i], cc);
      m = s;
    }
    const float pr = ex2(s - m);
    l += pr;
    return pr;
  };

  // The four warps walk the stages independently (no CTA-wide barrier per stage): a warp waits for the slot's
  // copy, works on its 32 rows and counts itself off; the warp that counts off last refills the slot.
  for (int s = s_lo; s < s_hi; ++s) {
    const int it = s - s_lo, slot = it % kQStages;
    if (__any_sync(0xffffffffu, !mbar_wait(&hdr->full[slot], (it / kQStages) & 1, p.status))) {
      hdr->abort_flag = 1;         // a wait gave up: the status word is set, the other warps' waits end early
      break;
    }
    const unsigned char* st = ring + slot * stage_stride;
    const int nblk = min(bps, nqb - s * bps);
    {   // the warp's blocks: q'_c * s_c
      const int wb0 = (warp * 32) >> gshift, nwb = G >= 32 ? 1 : 2;
      for (int i = 0; i < nwb; ++i)
        if (wb0 + i < nblk) {
          const __half* ks = reinterpret_cast<const __half*>(st + (wb0 + i) * qh.block_bytes + qh.ks_off);
          for (int c = lane; c < hd.rp_k; c += 32) qs_w[i * 128 + c] = hdr->qp[c] * __half2float(ks[c]);
        }
      __syncwarp();
    }
    const int blk = tid >> gshift, ri = tid & (G - 1);
    if (blk < nblk) {
      const unsigned char* bb = st + blk * qh.block_bytes;
      const float* qsr = qs_w + (G >= 32 ? 0 : (lane >> 4) * 128);
      unsigned long long a0 = 0ull, a1 = 0ull, a2 = 0ull, a3 = 0ull;
#pragma unroll
      for (int j = 0; j < NW; ++j)
        if (FULL || j < nwk) {
          unsigned long long f[4];
          codes_to_floats<BITS>(load_unit<BITS, G>(bb, nwk * G, j, ri), kc, f);
          const ulonglong2 q0 = *reinterpret_cast<const ulonglong2*>(qsr + 8 * j);
          const ulonglong2 q1 = *reinterpret_cast<const ulonglong2*>(qsr + 8 * j + 4);
          a0 = fma2p(f[0], q0.x, a0); a1 = fma2p(f[1], q0.y, a1);
          a2 = fma2p(f[2], q1.x, a2); a3 = fma2p(f[3], q1.y, a3);
        }
      const int j_abs = s * kStageRows + tid;
      const float pr = weight(fmaf(slope2, static_cast<float>(j_abs - pos_q),
                                   low_plus_high(add2p(add2p(a0, a1), add2p(a2, a3)))));
      const unsigned char* varea = bb + qh.vc_off;
      const __half* vs = reinterpret_cast<const __half*>(bb + qh.vs_off) + ri;
#pragma unroll
      for (int j = 0; j < NW; ++j)
        if (FULL || j < nwv) {
          const float sv = pr * __half2float(vs[((8 * j) >> gshift) * G]);
          const unsigned long long svp = pair_of(sv, sv);
          unsigned long long f[4];
          codes_to_floats<BITS>(load_unit<BITS, G>(varea, nwv * G, j, ri), kc, f);
#pragma unroll
          for (int i = 0; i < 4; ++i) o[4 * j + i] = fma2p(f[i], svp, o[4 * j + i]);
        }
    }
    // this warp is done with the slot (and with its scaled query)
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();       // the warp's reads of the slot come before the count that may trigger the refill
      if ((atomicAdd(&hdr->done[slot], 1) & 3) == 3 && s + kQStages < s_hi) issue(s + kQStages, slot);
    }
  }
  __syncthreads();
  const bool aborted = *reinterpret_cast<volatile int*>(&hdr->abort_flag) != 0;

  // rows that are not quantised yet, straight from the 16-bit cache (the last split takes them)
  if (split == p.splits - 1 && !aborted) {
    for (int j = nq_b + tid; j < n_b; j += kQThreads) {
      const int64_t row = static_cast<int64_t>(b) * p.n_max + j;
      const uint4* kr = reinterpret_cast<const uint4*>(p.cache + hd.k_off + row * hd.rp_k * 2);
      const uint4* vr = reinterpret_cast<const uint4*>(p.cache + hd.v_off + row * hd.rp_v * 2);
      unsigned long long a0 = 0ull, a1 = 0ull, a2 = 0ull, a3 = 0ull;
#pragma unroll
      for (int c = 0; c < NW; ++c)
        if (FULL || c < nwk) {
          unsigned long long f[4];
          bf16x8_to_floats(__ldg(kr + c), f);
          const ulonglong2 q0 = *reinterpret_cast<const ulonglong2*>(hdr->qp + 8 * c);
          const ulonglong2 q1 = *reinterpret_cast<const ulonglong2*>(hdr->qp + 8 * c + 4);
          a0 = fma2p(f[0], q0.x, a0); a1 = fma2p(f[1], q0.y, a1);
          a2 = fma2p(f[2], q1.x, a2); a3 = fma2p(f[3], q1.y, a3);
        }
      const float pr = weight(fmaf(slope2, static_cast<float>(j - pos_q),
                                   low_plus_high(add2p(add2p(a0, a1), add2p(a2, a3)))));
      const unsigned long long prp = pair_of(pr, pr);
#pragma unroll
      for (int c = 0; c < NW; ++c)
        if (FULL || c < nwv) {
          unsigned long long f[4];
          bf16x8_to_floats(__ldg(vr + c), f);
#pragma unroll
          for (int i = 0; i < 4; ++i) o[4 * c + i] = fma2p(f[i], prp, o[4 * c + i]);
        }
    }
  }

  // ---- merge the 128 threads into one partial (max, sum, o'[rp_v]); the ring doubles as the staging area
  float wm = m;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, d));
  if (lane == 0) hdr->wmax[warp] = wm;
  __syncthreads();
  const float M = fmaxf(fmaxf(hdr->wmax[0], hdr->wmax[1]), fmaxf(hdr->wmax[2], hdr->wmax[3]));
  const float f = (m == -INFINITY) ? 0.f : ex2(m - M);
  float ls = l * f;
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, d);
  if (lane == 0) hdr->wsum[warp] = ls;
  float* red = reinterpret_cast<float*>(ring);               // [128][rp_v + 1]
  const int rstride = hd.rp_v + 1;
  if (!aborted) {
#pragma unroll
    for (int i = 0; i < NW * 4; ++i)
      if (2 * i < hd.rp_v) {
        red[tid * rstride + 2 * i] = __uint_as_float(static_cast<uint32_t>(o[i])) * f;
        red[tid * rstride + 2 * i + 1] = __uint_as_float(static_cast<uint32_t>(o[i] >> 32)) * f;
      }
  }
  __syncthreads();
  float* part = p.partials + (static_cast<size_t>(unit) * p.splits + split) * p.part_stride;
  if (tid < hd.rp_v) {
    float acc = 0.f;
    if (!aborted)
      for (int r = 0; r < kQThreads; ++r) acc += red[r * rstride + tid];
    part[4 + tid] = acc;
  }
  if (tid == 0) {
    part[0] = M;
    part[1] = (hdr->wsum[0] + hdr->wsum[1]) + (hdr->wsum[2] + hdr->wsum[3]);
  }
}

__global__ void __launch_bounds__(128) quant_combine_kernel(const QuantParams p) {
  __shared__ float o_sm[128];
  const int unit = blockIdx.x, t = threadIdx.x;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const float* base = p.partials + static_cast<size_t>(unit) * p.splits * p.part_stride;
  float M = -INFINITY;
  for (int c = 0; c < p.splits; ++c) M = fmaxf(M, base[static_cast<size_t>(c) * p.part_stride]);
  float L = 0.f, acc = 0.f;
  for (int c = 0; c < p.splits; ++c) {
    const float* part = base + static_cast<size_t>(c) * p.part_stride;
    const float f = ex2(part[0] - M);                        // 0 for a piece without rows
    L = fmaf(part[1], f, L);
    if (t < hd.rp_v) acc = fmaf(part[4 + t], f, acc);
  }
  const float o = acc / L;
  __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.out);
  if (p.flags & 0x2u) {
    if (t < hd.rp_v) out[b * p.out_stride_b + hd.lr_v_off + t] = __float2bfloat16_rn(o);
    return;
  }
  if (t < hd.rp_v) o_sm[t] = o;
  __syncthreads();
  if (t < p.d_head) {
    const float* Ut = p.basis + hd.uvt_off;                  // (U^V)^T : rp_v x d_head
    float y = 0.f;
    for (int c = 0; c < hd.rp_v; ++c) y = fmaf(o_sm[c], __ldg(Ut + c * p.d_head + t), y);
    out[b * p.out_stride_b + static_cast<int64_t>(h) * p.d_head + t] = __float2bfloat16_rn(y);
  }
}

template <int NW, int MINB, int G, bool FULL, int BITS>
cudaError_t launch_variant(const QuantParams& p, size_t smem, cudaStream_t s) {
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(decode_quant_kernel<NW, MINB, G, FULL, BITS>, smem, configured);
  if (ec != cudaSuccess) return ec;
  decode_quant_kernel<NW, MINB, G, FULL, BITS><<<dim3(p.B * p.H, p.splits), kQThreads, smem, s>>>(p);
  return cudaGetLastError();
}
template <int NW, int MINB, int G>
cudaError_t launch_full_or_not(const QuantParams& p, bool full, size_t smem, cudaStream_t s) {
  return full ? launch_variant<NW, MINB, G, true, 3>(p, smem, s) : launch_variant<NW, MINB, G, false, 3>(p, smem, s);
}
template <int NW, int MINB>
cudaError_t launch_group(const QuantParams& p, bool full, size_t smem, cudaStream_t s) {
  switch (p.group) {
    case 16: return launch_full_or_not<NW, MINB, 16>(p, full, smem, s);
    case 32: return launch_full_or_not<NW, MINB, 32>(p, full, smem, s);
    case 64: return launch_full_or_not<NW, MINB, 64>(p, full, smem, s);
    default: return launch_full_or_not<NW, MINB, 128>(p, full, smem, s);
  }
}

}  // namespace

cudaError_t launch_quantize_blocks(const QuantParams& p, cudaStream_t s, uint64_t* launches) {
  if (p.b1 <= p.b0) return cudaSuccess;
  quantize_blocks_kernel<<<dim3(p.B * p.H, p.b1 - p.b0), kQThreads, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

size_t decode_quant_smem_bytes(int max_stage_bytes, int max_rp_v) {
  const size_t ring = static_cast<size_t>(kQStages) * ((max_stage_bytes + 127) & ~127);
  const size_t red = static_cast<size_t>(kQThreads) * (max_rp_v + 1) * sizeof(float);
  return kRingOffset + (ring > red ? ring : red);
}

cudaError_t launch_decode_quant(const QuantParams& p0, int max_rp, int min_rp, size_t smem, cudaStream_t s,
                                uint64_t* launches) {
  QuantParams p = p0;
  if (p.bits == 3) {   // 2^23, 2^20, 2^17, 2^14
    p.magic[0] = 0x4B000000u; p.magic[1] = 0x49800000u; p.magic[2] = 0x48000000u; p.magic[3] = 0x46800000u;
  } else {             // 2^23, 2^19, 2^15, 2^11
    p.magic[0] = 0x4B000000u; p.magic[1] = 0x49000000u; p.magic[2] = 0x47000000u; p.magic[3] = 0x45000000u;
  }
  cudaError_t e;
  if (max_rp <= 64) e = launch_group<8, 3>(p, min_rp == 64, smem, s);
  else if (max_rp <= 80) e = launch_group<10, 3>(p, min_rp == 80, smem, s);
  else e = launch_group<16, 2>(p, min_rp == 128, smem, s);
  if (e != cudaSuccess) return e;
  ++*launches;
  return launch_quant_combine(p, s, launches);
}

cudaError_t launch_quant_combine(const QuantParams& p, cudaStream_t s, uint64_t* launches) {
  quant_combine_kernel<<<p.B * p.H, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
