// Generation-phase Eigen Attention for models with rotary position embedding (Section 4.3, Fig. 6b).
//
// The query stays full rank.  Each cached low-dimensional key row k'_j is taken back to d_h dimensions
// through (U^K)^T, rotated by its position j and dotted with the rotated query; the value side is the
// rank-r path unchanged.  Per cached row that is a d_h x r product instead of an r-long dot product, so the
// lift runs on the tensor cores: for a tile of 128 cached rows, X = K'_tile (U^K)^T is one tcgen05 product
// (M = 128 rows, N = d_h, K = r; U^K rounded to bf16, the precision the cached rows already have) with X in
// TMEM, one row per thread.
//
// Rotation without a table per position: with complex pairs Q = q_a + i q_b, X = x_a + i x_b and the
// pair's frequency phi, the rotated dot product of the pair is Re(Q e^{i p phi} conj(X e^{i j phi})) =
// Re(Q e^{i (p - j) phi} conj(X)).  For row l of tile t, p - j = D_t - l with D_t = p - 128 t, so
// e^{i (p-j) phi} = e^{i D_t phi} conj(e^{i l phi}): the first factor is applied to the query once per tile
// (64 threads; the first tile's angle is reduced in fp64, every further tile turns the query by the constant
// e^{-i 128 phi}, one complex multiplication, renormalised), the second is a per-thread constant in registers.
//
// One CTA (128 threads, two per SM) walks a contiguous range of the tiles of one (sequence, head) unit.  A tile
// of K' or V' rows is contiguous in the cache, so each arrives as one bulk copy (cp.async.bulk).  K' lands
// row-major in a staging buffer, the threads move it into the core-matrix layout the tensor core reads (16-byte
// chunks, 20 KB a tile), and the staging buffer takes the next tile at once, a whole tile ahead of its use: with
// a single tile in flight per CTA it is the distance between request and use that sets the pace, not the kind of
// copy (tiled TMA boxes stream at the same rate when four tiles are in flight).  V' is read row-major where it
// lands.  Scores -> online softmax in base 2 ->
// o' += p V' on the CUDA cores (thread (g, c) owns a column pair over a row group).  A unit split over several CTAs leaves partials (m, l, o') that
// rope_combine_kernel merges and lifts through (U^V)^T.  Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;


struct __align__(16) RopeSmemHeader {
  unsigned long long mma_done, k_full, v_full;
  uint32_t tmem_base;
  int abort_flag;
  float red[8];          // cross-warp reductions
  float tile_max;
  float pad_[3];
};

template <bool INTERLEAVED>
__global__ void __launch_bounds__(kThreads, 2) decode_rope_kernel(const RopeDecodeParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  RopeSmemHeader* hdr = reinterpret_cast<RopeSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x, split = blockIdx.y;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const int rpk16 = (hd.rp_k + 15) & ~15;
  const int nch_k = rpk16 >> 3, grp_k = nch_k << 7;
  const int rowb_k = hd.rp_k * 2, rowb_v = hd.rp_v * 2;      // bytes per cached row
  const int kst_bytes = kTile * rowb_k, km_bytes = kTile * rpk16 * 2, v_bytes = kTile * rowb_v;
  const int u_bytes = p.d_head * rpk16 * 2;                  // bf16 image of U^K (the high part of the stored pair)
  const int half = p.d_head >> 1;

  float* q_tile = reinterpret_cast<float*>(smem + 256);      // the query pairs for this tile: re[64], then im[64]
  float* p_row = q_tile + 128;                               // [128] softmax weights of the tile
  unsigned char* tiles = smem + 2048;
  unsigned char* Kst = tiles;                                // K' tile as it lands: row-major
  unsigned char* Km = Kst + kst_bytes;                       // K' tile in the canonical core-matrix layout
  unsigned char* Vs = Km + km_bytes;                         // V' tile, row-major
  unsigned char* Us = Vs + v_bytes;                          // U^K image, canonical layout

  // tiles [t_lo, t_hi) of the unit
  // rows and tiles of this sequence (a batch of unequal lengths gives every sequence its own count and its own
  // query position; the splits of a unit divide the sequence's own tiles)
  const int n_b = p.deficit != nullptr ? p.n - __ldg(p.deficit + b) : p.n;
  const int nt_b = (n_b + kTile - 1) / kTile;
  const int per = (nt_b + p.splits - 1) / p.splits;
  const int t_lo = split * per, t_hi = min(nt_b, t_lo + per);
  float* part = p.partials + (static_cast<size_t>(unit) * p.splits + split) * p.part_stride;
  if (t_lo >= t_hi) {                                        // an empty piece: the neutral partial
    if (tid == 0) { part[0] = -INFINITY; part[1] = 0.f; }
    if (tid < hd.rp_v) part[4 + tid] = 0.f;
    return;
  }

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 256);           // two accumulators: X(t) is read while X(t+1) is computed
  if (tid == 0) {
    mbar_init(&hdr->mma_done, 1);
    mbar_init(&hdr->k_full, 1);
    mbar_init(&hdr->v_full, 1);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }

  // U^K image (read through L2 by every CTA of the head)
  {
    const uint4* Ug = reinterpret_cast<const uint4*>(p.basis + hd.ukl16_off);
    for (int idx = tid; idx < u_bytes / 16; idx += kThreads) cp_async16(Us + idx * 16, Ug + idx, 16u);
    cp_async_commit();
  }
  // rows that no copy has filled must hold finite numbers: they meet zero weights (a ragged last tile)
  for (int idx = tid; idx < (kst_bytes + km_bytes + v_bytes) / 16; idx += kThreads)
    reinterpret_cast<uint4*>(Kst)[idx] = make_uint4(0u, 0u, 0u, 0u);
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
    bulk_load(Vs, v_src + static_cast<int64_t>(t) * kTile * rowb_v, bytes, &hdr->v_full, policy);
  };
  // staging -> core-matrix layout: chunk (row, c) of 16 bytes goes to (row / 8) * grp_k + c * 128 + (row % 8) * 16
  auto relayout_k = [&]() { relayout_tile(Km, Kst, rowb_k, grp_k, warp, lane); };

  // this thread's constants: e^{i l phi_i} for its row l = tid and every pair i
  unsigned long long el_c[32], el_s[32];                     // pairs (2k, 2k+1) packed: (cos, cos), (sin, sin)
#pragma unroll
  for (int k = 0; k < 32; ++k) {
    float s0_, c0_, s1_, c1_;
    sincosf(static_cast<float>(tid) * static_cast<float>(2 * k < half ? p.inv_freq[2 * k] : 0.0), &s0_, &c0_);
    sincosf(static_cast<float>(tid) * static_cast<float>(2 * k + 1 < half ? p.inv_freq[2 * k + 1] : 0.0), &s1_, &c1_);
    el_c[k] = pack2(c0_, c1_);
    el_s[k] = pack2(s0_, s1_);
  }
  // the query of this unit, scaled by log2(e)/sqrt(d_h): thread i < half owns pair i
  // turned to the first tile's offset here (fp64 once), then by (step_c, step_s) = e^{-i 128 phi} per tile
  float q_re = 0.f, q_im = 0.f, step_c = 1.f, step_s = 0.f, q_norm2 = 0.f;
  if (tid < half) {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + b * p.q_stride_b + static_cast<int64_t>(h) * p.d_head;
    const int ia = INTERLEAVED ? 2 * tid : tid, ib = INTERLEAVED ? 2 * tid + 1 : tid + half;
    const float a_re = __bfloat162float(qg[ia]) * p.q_scale, a_im = __bfloat162float(qg[ib]) * p.q_scale;
    const double freq = p.inv_freq[tid];
    double s_, c_;
    sincos(static_cast<double>(n_b - 1 - t_lo * kTile) * freq, &s_, &c_);
    q_re = static_cast<float>(a_re * c_ - a_im * s_);
    q_im = static_cast<float>(a_re * s_ + a_im * c_);
    q_norm2 = a_re * a_re + a_im * a_im;
    sincos(-static_cast<double>(kTile) * freq, &s_, &c_);
    step_c = static_cast<float>(c_);
    step_s = static_cast<float>(s_);
  }

  cp_async_wait<0>();
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    fetch_k(t_lo);
    fetch_v(t_lo);
  }
  const uint32_t tmem = hdr->tmem_base;
  const uint32_t tX0 = tmem + (static_cast<uint32_t>(warp * 32) << 16);
  volatile int* abort_flag = &hdr->abort_flag;
  const uint32_t idesc = instr_desc(p.d_head, false);
  const int ks_steps = rpk16 >> 4;
  const int pos_q = n_b - 1;

  // weighted sum o' += p V': thread (g, c) owns the column pair (2c, 2c+1) over the rows of row group g of every
  // tile; the groups are added up once, at the end
  const int col_pairs = hd.rp_v >> 1;
  const int row_groups = min(kThreads / col_pairs, 16);
  const int rows_per_group = (((kTile + row_groups - 1) / row_groups) + 7) & ~7;   // whole blocks of 8 rows
  const int pv_g = tid / col_pairs, pv_c = tid - pv_g * col_pairs;
  const int r_lo = min(kTile, pv_g * rows_per_group), r_hi = pv_g < row_groups ? min(kTile, r_lo + rows_per_group) : r_lo;
  const unsigned char* v_col = Vs + 4 * pv_c;
  float m_run = -INFINITY, l_thr = 0.f, o_acc0 = 0.f, o_acc1 = 0.f;
  bool ok = true;
  // lift of one tile (thread 0): X = K' (U^K)^T into accumulator `acc`
  const uint64_t desc_k = smem_desc(smem_u32(Km), 128, grp_k), desc_u = smem_desc(smem_u32(Us), 128, grp_k);
  auto issue_lift = [&](int acc) {
    tc_fence_after();
    for (int s = 0; s < ks_steps; ++s)                       // 16 rank elements (two chunks) a step
      mma_ss(tmem + acc * kTile, desc_k + s * 16, desc_u + s * 16, idesc, s > 0);
    mma_commit(&hdr->mma_done);
  };
  // the first tile: into the core-matrix layout, lift, and the staging buffer takes the second tile
  if (!mbar_wait(&hdr->k_full, 0, p.status)) *abort_flag = 1;
  relayout_k();
  fence_async_smem();
  __syncthreads();
  if (*abort_flag) ok = false;
  if (tid == 0 && ok) {
    issue_lift(0);
    if (t_lo + 1 < t_hi) fetch_k(t_lo + 1);
  }
  for (int t = t_lo; t < t_hi && ok; ++t) {
    const uint32_t par = (t - t_lo) & 1u;
    const uint32_t tX = tX0 + par * kTile;
    // ---- the query pairs turned by (pos_q - 128 t) phi
    if (tid < half) {
      q_tile[tid] = q_re;
      q_tile[64 + tid] = q_im;
      // the next tile's query: one more turn by -128 phi; the length is pulled back to |q| so that rounding
      // does not drift over a thousand tiles
      const float n_re = q_re * step_c - q_im * step_s, n_im = q_re * step_s + q_im * step_c;
      const float fix = 1.5f - 0.5f * (n_re * n_re + n_im * n_im) / fmaxf(q_norm2, 1e-30f);   // ~ |q| / |n|
      q_re = n_re * fix;
      q_im = n_im * fix;
    }
    // ---- X(t) is complete (its lift went out during the previous tile): the core-matrix buffer is free
    if (!mbar_wait(&hdr->mma_done, par, p.status)) *abort_flag = 1;
    __syncthreads();                                         // q_tile written
    if (*abort_flag) { ok = false; break; }
    tc_fence_after();
    // two pairs per packed instruction: W = Q_t conj(E_l), pair term = Re(W conj(X)) = W_re x_re + W_im x_im
    unsigned long long acc_re = 0ull, acc_im = 0ull;         // (0.f, 0.f)
#pragma unroll
    for (int c0 = 0; c0 < 64; c0 += 16) {
      if (c0 < half) {
        uint32_t xa[16], xb[16];
        if (INTERLEAVED) {                                   // pairs (2i, 2i+1): columns 2 c0 .. 2 c0 + 31
          tmem_ld16(tX + 2 * c0, xa);
          tmem_ld16(tX + 2 * c0 + 16, xb);
        } else {                                             // pairs (i, i + d_h/2)
          tmem_ld16(tX + c0, xa);
          tmem_ld16(tX + half + c0, xb);
        }
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          unsigned long long x_re, x_im;
          if (INTERLEAVED) {
            const uint32_t* src = i < 8 ? xa : xb;
            x_re = pack2(__uint_as_float(src[(2 * i) & 15]), __uint_as_float(src[(2 * i + 2) & 15]));
            x_im = pack2(__uint_as_float(src[(2 * i + 1) & 15]), __uint_as_float(src[(2 * i + 3) & 15]));
          } else {
            x_re = pack2(__uint_as_float(xa[i]), __uint_as_float(xa[i + 1]));
            x_im = pack2(__uint_as_float(xb[i]), __uint_as_float(xb[i + 1]));
          }
          const unsigned long long qr = *reinterpret_cast<const unsigned long long*>(q_tile + c0 + i);
          const unsigned long long qi = *reinterpret_cast<const unsigned long long*>(q_tile + 64 + c0 + i);
          const unsigned long long ec = el_c[(c0 + i) >> 1], es = el_s[(c0 + i) >> 1];
          const unsigned long long w_re = fma2p(qi, es, mul2p(qr, ec));                  // Qr c + Qi s
          const unsigned long long w_im = fma2p(qr ^ 0x8000000080000000ull, es, mul2p(qi, ec));   // Qi c - Qr s
          acc_re = fma2p(w_re, x_re, acc_re);
          acc_im = fma2p(w_im, x_im, acc_im);
        }
      }
    }
    float s0, s1, s2, s3;
    unpack2(acc_re, s0, s1);
    unpack2(acc_im, s2, s3);
    s0 += s2;
    s1 += s3;
    // ---- K'(t+1) landed a tile ago: into the core-matrix layout now, its lift goes out after the barrier below
    if (t + 1 < t_hi) {
      if (!mbar_wait(&hdr->k_full, par ^ 1u, p.status)) *abort_flag = 1;
      relayout_k();
      fence_async_smem();
    }
    const int j = t * kTile + tid;
    const bool live = j < n_b;
    const float s = live ? s0 + s1 : -INFINITY;
    // ---- online softmax over the tile: block maximum, weights, running sum per thread
    float mx = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) hdr->red[warp] = mx;
    tc_fence_before();
    __syncthreads();                                         // every thread has read its row of X and moved its chunks
    if (tid == 0 && t + 1 < t_hi && !*abort_flag) {          // lift of tile t+1 behind the softmax and the weighted sum;
      issue_lift(static_cast<int>(par ^ 1u));                // the staging buffer takes tile t+2
      if (t + 2 < t_hi) fetch_k(t + 2);
    }
    const float m_new = fmaxf(m_run, fmaxf(fmaxf(hdr->red[0], hdr->red[1]), fmaxf(hdr->red[2], hdr->red[3])));
    const float alpha = ex2(m_run - m_new);                  // 0 at the first tile
    m_run = m_new;
    const float pj = live ? ex2(s - m_new) : 0.f;
    l_thr = fmaf(l_thr, alpha, pj);
    p_row[tid] = pj;
    if (!mbar_wait(&hdr->v_full, par, p.status)) *abort_flag = 1;
    __syncthreads();
    if (*abort_flag) { ok = false; break; }
    // ---- o' = alpha o' + sum_j p_j V'[j][2c..2c+1] over this thread's rows (row-major tile)
    {
      float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f;
      for (int r = r_lo; r < r_hi; r += 8) {
        const float4 pa = *reinterpret_cast<const float4*>(p_row + r);
        const float4 pb = *reinterpret_cast<const float4*>(p_row + r + 4);
        const unsigned char* vr = v_col + r * rowb_v;
        uint32_t v[8];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) v[jj] = *reinterpret_cast<const uint32_t*>(vr + jj * rowb_v);
        a0 = fmaf(pa.x, __uint_as_float(v[0] << 16), a0); a1 = fmaf(pa.x, __uint_as_float(v[0] & 0xffff0000u), a1);
        b0 = fmaf(pa.y, __uint_as_float(v[1] << 16), b0); b1 = fmaf(pa.y, __uint_as_float(v[1] & 0xffff0000u), b1);
        a0 = fmaf(pa.z, __uint_as_float(v[2] << 16), a0); a1 = fmaf(pa.z, __uint_as_float(v[2] & 0xffff0000u), a1);
        b0 = fmaf(pa.w, __uint_as_float(v[3] << 16), b0); b1 = fmaf(pa.w, __uint_as_float(v[3] & 0xffff0000u), b1);
        a0 = fmaf(pb.x, __uint_as_float(v[4] << 16), a0); a1 = fmaf(pb.x, __uint_as_float(v[4] & 0xffff0000u), a1);
        b0 = fmaf(pb.y, __uint_as_float(v[5] << 16), b0); b1 = fmaf(pb.y, __uint_as_float(v[5] & 0xffff0000u), b1);
        a0 = fmaf(pb.z, __uint_as_float(v[6] << 16), a0); a1 = fmaf(pb.z, __uint_as_float(v[6] & 0xffff0000u), a1);
        b0 = fmaf(pb.w, __uint_as_float(v[7] << 16), b0); b1 = fmaf(pb.w, __uint_as_float(v[7] & 0xffff0000u), b1);
      }
      o_acc0 = fmaf(o_acc0, alpha, a0 + b0);
      o_acc1 = fmaf(o_acc1, alpha, a1 + b1);
    }
    __syncthreads();                                         // the V' tile is free again
    if (tid == 0 && t + 1 < t_hi) fetch_v(t + 1);
  }
  if (!ok) *abort_flag = 1;

  // ---- the piece's partial: m, l (sum over the threads' rows), o'
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l_thr += __shfl_xor_sync(0xffffffffu, l_thr, o);
  __syncthreads();
  if (lane == 0) hdr->red[4 + warp] = l_thr;
  __syncthreads();
  if (tid == 0) {
    part[0] = m_run;
    part[1] = (hdr->red[4] + hdr->red[5]) + (hdr->red[6] + hdr->red[7]);
  }
  // add up the row groups (the V' tile's shared memory is free now)
  float* o_red = reinterpret_cast<float*>(Vs);
  if (pv_g < row_groups) {
    o_red[pv_g * hd.rp_v + 2 * pv_c] = o_acc0;
    o_red[pv_g * hd.rp_v + 2 * pv_c + 1] = o_acc1;
  }
  __syncthreads();
  if (tid < hd.rp_v) {
    float o = 0.f;
    for (int g = 0; g < row_groups; ++g) o += o_red[g * hd.rp_v + tid];
    part[4 + tid] = o;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
}

// Merges the partials of a unit and lifts o'/l through (U^V)^T (or writes the rank-space row).
__global__ void __launch_bounds__(128) rope_combine_kernel(const RopeDecodeParams p) {
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
    const float f = ex2(part[0] - M);                        // 0 for an empty piece
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

}  // namespace

size_t decode_rope_smem_bytes(int max_rp_k, int max_rp_v, int d_head) {
  const size_t k16 = (max_rp_k + 15) & ~15;
  // header, U^K image, K' staging + core-matrix copy, V' tile
  return 2048 + static_cast<size_t>(d_head) * k16 * 2 + kTile * static_cast<size_t>(max_rp_k + k16 + max_rp_v) * 2;
}

cudaError_t launch_decode_rope(const RopeDecodeParams& p, size_t smem, cudaStream_t s, uint64_t* launches) {
  static size_t configured[2][kMaxDevices] = {};
  const cudaError_t ec = p.interleaved ? ensure_dynamic_smem(decode_rope_kernel<true>, smem, configured[1])
                                       : ensure_dynamic_smem(decode_rope_kernel<false>, smem, configured[0]);
  if (ec != cudaSuccess) return ec;
  dim3 grid(p.B * p.H, p.splits);
  if (p.interleaved) decode_rope_kernel<true><<<grid, kThreads, smem, s>>>(p);
  else decode_rope_kernel<false><<<grid, kThreads, smem, s>>>(p);
  ++*launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  rope_combine_kernel<<<p.B * p.H, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
