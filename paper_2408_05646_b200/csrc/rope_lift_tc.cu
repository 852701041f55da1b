// Lifted, rotated keys of a prompt for layers with rotary position embedding (Section 4.3), on the tensor cores.
//
//   Kr[j] = RoPE_j( k'_j (U^K)^T )     for the rows j a sequence holds after the call, written 16-bit, d_head wide,
//
// which is what the prompt's attention product needs on its key side (the warp-specialised prompt kernel then runs an
// ordinary causal product of the rotated full-rank queries against these rows).  The lift is the product the rotary
// decode kernel issues: X = K'_tile (U^K)^T for 128 cached rows (tcgen05, M = 128 rows, N = d_head, K = r, the bf16
// image of U^K resident in shared memory, the K' tile brought by TMA straight in the operand's swizzled layout, two
// tile buffers and two TMEM accumulators).  Rotation by the absolute position j = 128 t + l: e^{i j phi} = T_t E_l with
// T_t = e^{i 128 t phi} (per tile, 64 angles reduced in double precision, in shared memory) and E_l = e^{i l phi} (a
// per-thread constant in registers, from the table the layer keeps).  Two threads per row (warps w and w + 4 share a
// TMEM lane quadrant and take every other chunk of eight pairs).  One thread requests tiles and issues lifts at the
// top of a tile; every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kLiftAtom = kTile * 128;        // one swizzled atom column of a K' tile: 128 rows x 64 elements
constexpr int kLiftThreads = 256;
constexpr int kLiftIssuer = 224;              // first lane of warp 7
constexpr int kLiftHeaderBytes = 3072;        // barriers, the tiles' rotation factors
constexpr double kTwoPi = 6.283185307179586476925286766559;

struct __align__(16) LiftSmemHeader {
  unsigned long long x_full[2], k_full[2];
  uint32_t tmem_base;
  int pad_;
};

__host__ __device__ constexpr int lift_kb(int bytes) { return (bytes + 1023) & ~1023; }

template <bool INTERLEAVED>
__global__ void __launch_bounds__(kLiftThreads, 2) rope_lift_tc_kernel(const PrefillParams p, int splits) {
  extern __shared__ __align__(1024) unsigned char smem[];
  LiftSmemHeader* hdr = reinterpret_cast<LiftSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x, split = blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const int rpk16 = (hd.rp_k + 15) & ~15;
  const int grp_k = (rpk16 >> 3) << 7;
  const int ak = (rpk16 + 63) >> 6;                          // atom columns (64 elements) of a K' tile
  const int kt_bytes = ak * kLiftAtom;
  const int u_bytes = p.d_head * rpk16 * 2;                  // bf16 image of U^K
  const int dh = p.d_head, half = dh >> 1;

  // tile factors T_t: [2 buffers][4 arrays: re, im, -re, -im][64 pairs]
  float* t_fac = reinterpret_cast<float*>(smem + 256);
  unsigned char* Us = smem + kLiftHeaderBytes;               // U^K image, canonical layout
  unsigned char* Kt = Us + lift_kb(u_bytes);                 // K' tiles [2], 128-byte swizzle

  // rows this sequence holds after the call, up to the end of the 64-row key tile of its last row (the attention
  // kernel reads whole key tiles; rows past the length meet masked scores and must only be finite)
  const int len_b = p.len0 - (p.deficit != nullptr ? __ldg(p.deficit + b) : 0) + p.T;
  const int rows_b = min(min(p.krot_rows, p.n_max), (len_b + 63) & ~63);
  const int nt_b = (rows_b + kTile - 1) / kTile;
  const int per = (nt_b + splits - 1) / splits;
  const int t_lo = split * per, t_hi = min(nt_b, t_lo + per);
  if (t_lo >= t_hi) return;
  const int nt_cta = t_hi - t_lo;

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 256);
  if (tid == 0) {
    mbar_init(&hdr->x_full[0], 1);
    mbar_init(&hdr->x_full[1], 1);
    mbar_init(&hdr->k_full[0], 1);
    mbar_init(&hdr->k_full[1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  {
    const uint4* Ug = reinterpret_cast<const uint4*>(p.basis + hd.ukl16_off);
    for (int idx = tid; idx < u_bytes / 16; idx += kLiftThreads) cp_async16(Us + idx * 16, Ug + idx, 16u);
    cp_async_commit();
  }
  // Thread (row, hf): row = 32 (warp & 3) + lane is its TMEM lane, hf = warp >> 2 picks the chunks of eight pairs
  // 2m + hf (m = 0..3); its constants E_l for those pairs: entry [k][row] = cos, cos, sin, sin of pairs 2k, 2k + 1
  const int row = (warp & 3) * 32 + lane, hf = warp >> 2;
  unsigned long long el_c[16], el_s[16];
#pragma unroll
  for (int m = 0; m < 4; ++m)
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float4 c = __ldg(p.el_table + ((2 * m + hf) * 4 + e) * kTile + row);
      el_c[4 * m + e] = pack2(c.x, c.y);
      el_s[4 * m + e] = pack2(c.z, c.w);
    }
  // T_t of tile t into buffer `buf`: thread i < 64 owns pair i
  auto tile_factor = [&](int t, int buf) {
    if (tid < 64) {
      float c_ = 1.f, s_ = 0.f;
      if (tid < half) {
        double ang = static_cast<double>(t) * kTile * p.inv_freq[tid];
        ang -= kTwoPi * rint(ang / kTwoPi);
        sincosf(static_cast<float>(ang), &s_, &c_);
      }
      float* f = t_fac + buf * 256;
      f[tid] = c_; f[64 + tid] = s_; f[128 + tid] = -c_; f[192 + tid] = -s_;
    }
  };
  tile_factor(t_lo, 0);

  cp_async_wait<0>();
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  const void* map_k = static_cast<const unsigned char*>(p.tmaps) + static_cast<size_t>(h) * 256;
  auto fetch_k = [&](int i) {
    const int buf = i & 1, t = t_lo + i;
    mbar_arrive_expect_tx(&hdr->k_full[buf], static_cast<uint32_t>(kt_bytes));
    for (int a = 0; a < ak; ++a)
      for (int hh = 0; hh < 2; ++hh)
        tma_load_3d(Kt + buf * kt_bytes + a * kLiftAtom + hh * (kLiftAtom / 2), map_k, a * 64, t * kTile + hh * 64, b,
                    &hdr->k_full[buf]);
  };
  auto issue_lift = [&](int i) -> bool {
    if (!mbar_wait(&hdr->k_full[i & 1], (i >> 1) & 1u, p.status)) return false;
    tc_fence_after();
    const uint32_t idesc = instr_desc(dh, false);
    const uint64_t dk = smem_desc_sw128(smem_u32(Kt + (i & 1) * kt_bytes), 16, 1024), du = smem_desc(smem_u32(Us), 128, grp_k);
    for (int s = 0; s < (rpk16 >> 4); ++s)
      mma_ss(tmem + (i & 1) * kTile, dk + (s >> 2) * (kLiftAtom >> 4) + (s & 3) * 2, du + s * 16, idesc, s > 0);
    mma_commit(&hdr->x_full[i & 1]);
    return true;
  };
  bool live = true;
  if (tid == kLiftIssuer) {
    tensormap_acquire(map_k);
    fetch_k(0);
    if (nt_cta > 1) fetch_k(1);
    live = issue_lift(0);
  }
  __syncwarp();
  const uint32_t tX0 = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
  __nv_bfloat16* out_unit = static_cast<__nv_bfloat16*>(p.krot) + (static_cast<int64_t>(h) * p.B + b) * p.krot_rows * dh;
  for (int i = 0; i < nt_cta; ++i) {
    const uint32_t par = i & 1u;
    const bool have_x = mbar_wait(&hdr->x_full[par], (i >> 1) & 1u, p.status);
    tc_fence_after();
    // X(i) is complete, so its K' buffer takes tile i + 2; X(i + 1) goes into the accumulator that was read during tile
    // i - 1 (every thread has passed that tile's closing barrier)
    if (tid == kLiftIssuer && live && have_x) {
      if (i + 2 < nt_cta) fetch_k(i + 2);
      if (i + 1 < nt_cta) live = issue_lift(i + 1);
    }
    __syncwarp();
    if (i + 1 < nt_cta) tile_factor(t_lo + i + 1, par ^ 1);  // read after this tile's closing barrier
    const float* tf = t_fac + par * 256;
    const int j = (t_lo + i) * kTile + row;                  // this thread's row of the sequence
    const bool store = have_x && j < rows_b;
    __nv_bfloat16* dst = out_unit + static_cast<int64_t>(j) * dh;
    const uint32_t tX = tX0 + par * kTile;
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const int c = 2 * m + hf;
      uint32_t xc[16];                                       // re[8], im[8] (pairs (i, i + d_h/2)) or re, im alternating
      if (have_x && 8 * c < half) {
        if (INTERLEAVED) {
          tmem_ld16(tX + 16 * c, xc);
        } else {
          tmem_ld8(tX + 8 * c, *reinterpret_cast<uint32_t(*)[8]>(&xc[0]));
          tmem_ld8(tX + half + 8 * c, *reinterpret_cast<uint32_t(*)[8]>(&xc[8]));
        }
      }
      tmem_wait_ld();
      if (8 * c < half) {
        uint32_t w[8];                                       // the chunk's 16 output values as bf16 pairs
        const float* tc_ = tf + 8 * c;
#pragma unroll
        for (int e = 0; e < 8; e += 4) {                     // four pairs a step
          const float4 tr4 = *reinterpret_cast<const float4*>(tc_ + e);
          const float4 ti4 = *reinterpret_cast<const float4*>(tc_ + 64 + e);
          const float4 tnr4 = *reinterpret_cast<const float4*>(tc_ + 128 + e);
          const float4 tni4 = *reinterpret_cast<const float4*>(tc_ + 192 + e);
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            const int ee = e + 2 * k;
            unsigned long long x_re, x_im;
            if (INTERLEAVED) {
              x_re = pack2(__uint_as_float(xc[2 * ee]), __uint_as_float(xc[2 * ee + 2]));
              x_im = pack2(__uint_as_float(xc[2 * ee + 1]), __uint_as_float(xc[2 * ee + 3]));
            } else {
              x_re = pack2(__uint_as_float(xc[ee]), __uint_as_float(xc[ee + 1]));
              x_im = pack2(__uint_as_float(xc[8 + ee]), __uint_as_float(xc[8 + ee + 1]));
            }
            const unsigned long long tr = k == 0 ? pack2(tr4.x, tr4.y) : pack2(tr4.z, tr4.w);
            const unsigned long long ti = k == 0 ? pack2(ti4.x, ti4.y) : pack2(ti4.z, ti4.w);
            const unsigned long long tnr = k == 0 ? pack2(tnr4.x, tnr4.y) : pack2(tnr4.z, tnr4.w);
            const unsigned long long tni = k == 0 ? pack2(tni4.x, tni4.y) : pack2(tni4.z, tni4.w);
            const unsigned long long er = el_c[4 * m + (ee >> 1)], ei = el_s[4 * m + (ee >> 1)];
            // W = T_t E_l, Y = W X
            const unsigned long long wr = fma2p(tr, er, mul2p(tni, ei));
            const unsigned long long wi = fma2p(tr, ei, mul2p(ti, er));
            const unsigned long long nwi = fma2p(tnr, ei, mul2p(tni, er));
            const unsigned long long yr = fma2p(wr, x_re, mul2p(nwi, x_im));
            const unsigned long long yi = fma2p(wr, x_im, mul2p(wi, x_re));
            float r0, r1, i0, i1;
            unpack2(yr, r0, r1);
            unpack2(yi, i0, i1);
            if (INTERLEAVED) {
              w[ee] = pack_bf16(r0, i0);
              w[ee + 1] = pack_bf16(r1, i1);
            } else {
              w[ee >> 1] = pack_bf16(r0, r1);
              w[4 + (ee >> 1)] = pack_bf16(i0, i1);
            }
          }
        }
        if (store) {
          if (INTERLEAVED) {
            *reinterpret_cast<uint4*>(dst + 16 * c) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(dst + 16 * c + 8) = make_uint4(w[4], w[5], w[6], w[7]);
          } else {
            *reinterpret_cast<uint4*>(dst + 8 * c) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(dst + half + 8 * c) = make_uint4(w[4], w[5], w[6], w[7]);
          }
        }
      }
    }
    tc_fence_before();
    // X(i) is read and the next tile's factor is written; a wait that gave up anywhere ends the loop for all
    if (__syncthreads_or((!have_x || !live) ? 1 : 0)) break;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
}

}  // namespace

size_t rope_lift_tc_smem_bytes(int max_rp_k, int d_head) {
  const int k16 = (max_rp_k + 15) & ~15;
  return kLiftHeaderBytes + lift_kb(d_head * k16 * 2) + 2 * static_cast<size_t>((k16 + 63) >> 6) * kLiftAtom;
}

// Lifted, rotated keys of every sequence's rows after the call into p.krot (see the head of this file).
cudaError_t launch_rope_lift_tc(const PrefillParams& p, int max_rp_k, int sm_count, cudaStream_t s, uint64_t* launches) {
  const size_t smem = rope_lift_tc_smem_bytes(max_rp_k, p.d_head);
  static size_t configured[2][kMaxDevices] = {};
  const cudaError_t ec = p.rope_interleaved ? ensure_dynamic_smem(rope_lift_tc_kernel<true>, smem, configured[1])
                                            : ensure_dynamic_smem(rope_lift_tc_kernel<false>, smem, configured[0]);
  if (ec != cudaSuccess) return ec;
  // pieces per unit: enough CTAs for a few waves of two per SM, each keeping at least a few tiles (its start-up is the
  // U^K image and the constants)
  const int rows = min(min(p.krot_rows, p.n_max), (p.len0 + p.T + 63) & ~63);
  const int nt = (rows + kTile - 1) / kTile;
  const int units = p.B * p.H;
  int splits = (4 * 2 * sm_count + units - 1) / units;
  if (splits > (nt + 3) / 4) splits = (nt + 3) / 4;
  if (splits < 1) splits = 1;
  if (p.rope_interleaved) rope_lift_tc_kernel<true><<<dim3(units, splits), kLiftThreads, smem, s>>>(p, splits);
  else rope_lift_tc_kernel<false><<<dim3(units, splits), kLiftThreads, smem, s>>>(p, splits);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
