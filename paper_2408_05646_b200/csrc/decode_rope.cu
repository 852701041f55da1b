// Generation-phase Eigen Attention for models with rotary position embedding (Section 4.3, Fig. 6b).
//
// The query stays full rank.  Each cached low-dimensional key row k'_j is taken back to d_h dimensions
// through (U^K)^T, rotated by its position j and dotted with the rotated query; the value side is the
// rank-r path unchanged.  Per cached row that is a d_h x r product instead of an r-long dot product, so the
// lift runs on the tensor cores: for a tile of 128 cached rows, X = K'_tile (U^K)^T is one tcgen05 product
// (M = 128 rows, N = d_h, K = r; U^K rounded to bf16, the precision the cached rows already have) with X in
// TMEM, one row per lane.
//
// Rotation without a table per position: with complex pairs Q = q_a + i q_b, X = x_a + i x_b and the
// pair's frequency phi, the rotated dot product of the pair is Re(Q e^{i p phi} conj(X e^{i j phi})) =
// Re(Q e^{i (p - j) phi} conj(X)).  For row l of tile t, p - j = D_t - l with D_t = p - 128 t, so
// e^{i (p-j) phi} = e^{i D_t phi} conj(e^{i l phi}): the first factor is applied to the query once per tile
// (64 threads; the first tile's angle is reduced in fp64, every further tile turns the query by the constant
// e^{-i 128 phi}, one complex multiplication, renormalised), the second is a per-thread constant in registers.
//
// One CTA (nine warps, two CTAs per SM) walks a contiguous range of the tiles of one (sequence, head) unit.
//   * Warp 8 (its first lane) requests and issues: a K' tile arrives by TMA straight in the swizzled layout the
//     lift's A operand names (two buffers, no thread moves it), a V' tile as one bulk copy (contiguous in the
//     cache, read row-major where it lands), and the lift of tile i + 1 goes out while the other warps work on
//     X(i) (two accumulators in TMEM).  mbarriers carry every hand-over: rows landed, X complete (which also
//     frees the K' buffer), X read, V' landed, V' read.
//   * Warps 0-7 do the arithmetic.  A TMEM lane (= cached row) is shared by two threads, warp w and warp w + 4,
//     each taking every other chunk of eight pairs, so a thread keeps only half of its row's rotation constants
//     in registers.  The two partial scores meet in shared memory; every thread adds up its lane's four rows, so
//     the tile maximum is one warp reduction with no further barrier.  Online softmax in base 2, then
//     o' += p V' on the CUDA cores (thread (g, c) owns a column pair over a row group).
// The rotation constants (e^{i l phi} per row offset, e^{-i 128 phi} per tile) are built on the host in double
// precision when the embedding is set; a CTA only loads them.  A unit split over several CTAs leaves partials
// (m, l, o') that rope_combine_kernel merges and lifts through (U^V)^T.  Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;


constexpr int kRopeAtom = kTile * 128;        // one swizzled atom column of a K' tile: 128 rows x 64 elements
constexpr int kRopeThreads = 256;             // eight warps: two threads per cached row of the tile
constexpr int kRopeRequester = 192;           // first lane of warp 6: requests the K' and V' tiles
constexpr int kRopeLifter = 224;              // first lane of warp 7: issues the lifts
constexpr int kRopeSumThreads = 192;          // warps 0-5 do the weighted sum while those two lanes issue
constexpr int kRopeHeaderBytes = 4096;        // barriers, the tile's query, weights and partial scores
constexpr float kRopeLazy = 8.f;              // the softmax reference moves when a score passes it by this much (base 2)
constexpr double kTwoPi = 6.283185307179586476925286766559;

// Barrier of the CTA with a predicate ORed over its threads: every thread gets the same answer, so what follows it
// (leaving the tile loop when a wait gave up) is decided alike by all and the next barrier is met by all.
__device__ __forceinline__ bool cta_sync_or(bool pred) { return __syncthreads_or(pred ? 1 : 0) != 0; }

struct __align__(16) RopeSmemHeader {
  unsigned long long x_full[2], k_full[2], v_full, v_free;
  uint32_t tmem_base;
  int pad_;
  float red[4];          // the row sums of warps 0-3
};

// parts of the shared memory image are multiples of 1 KB (the swizzled tiles need that alignment)
__host__ __device__ constexpr int rope_kb(int bytes) { return (bytes + 1023) & ~1023; }

// HALF = d_head / 2 known at compile time (64: the usual head of 128 dimensions; no chunk of pairs is ever empty
// and the TMEM columns are constants), or 0: taken from the launch parameters.
// PAGED: the tiles' addresses come through a page table.
template <bool INTERLEAVED, int HALF, bool PAGED>
__global__ void __launch_bounds__(kRopeThreads, 2) decode_rope_kernel(const RopeDecodeParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  RopeSmemHeader* hdr = reinterpret_cast<RopeSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // a unit is a (sequence, query head) pair; with grouped queries `group` query heads read the rows of one K/V head
  // (its units are B apart, so they run at the same time and all but the first find the tiles in L2)
  const int unit = blockIdx.x, split = blockIdx.y;
  const int hq = unit / p.B, b = unit - hq * p.B;
  const int h = hq / p.group;
  const HeadInfo hd = p.heads[h];
  const int rpk16 = (hd.rp_k + 15) & ~15;
  const int nch_k = rpk16 >> 3, grp_k = nch_k << 7;
  const int rowb_v = hd.rp_v * 2;                            // bytes per cached value row
  const int ak = (rpk16 + 63) >> 6;                          // atom columns (64 elements) of a K' tile
  const int kt_bytes = ak * kRopeAtom, v_bytes = kTile * rowb_v;
  const int u_bytes = p.d_head * rpk16 * 2;                  // bf16 image of U^K (the high part of the stored pair)
  const int half = HALF ? HALF : p.d_head >> 1;

  float* q_tile = reinterpret_cast<float*>(smem + 256);      // [2][192] the query pairs of a tile: re[64], im[64], -re[64]
  float* p_row = q_tile + 384;                               // [128] softmax weights of the tile
  float* sc = p_row + 128;                                   // [2][128] the two partial scores of every row
  unsigned char* Us = smem + kRopeHeaderBytes;               // U^K image, canonical layout
  unsigned char* Kt = Us + rope_kb(u_bytes);                 // K' tiles [2], as TMA writes them: 128-byte swizzle
  unsigned char* Vs = Kt + 2 * kt_bytes;                     // V' tile, row-major

  // rows and tiles of this sequence (a batch of unequal lengths gives every sequence its own count and its own
  // query position; the splits of a unit divide the sequence's own tiles): this CTA takes tiles [t_lo, t_hi)
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
  const int nt_cta = t_hi - t_lo;

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 256);           // two accumulators: X(i) is read while X(i+1), X(i+2) are computed
  if (tid == 0) {
    mbar_init(&hdr->x_full[0], 1);
    mbar_init(&hdr->x_full[1], 1);
    mbar_init(&hdr->k_full[0], 1);
    mbar_init(&hdr->k_full[1], 1);
    mbar_init(&hdr->v_full, 1);
    mbar_init(&hdr->v_free, kRopeSumThreads / 32);           // one arrival per warp
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // U^K image (read through L2 by every CTA of the head)
  {
    const uint4* Ug = reinterpret_cast<const uint4*>(p.basis + hd.ukl16_off);
    for (int idx = tid; idx < u_bytes / 16; idx += kRopeThreads) cp_async16(Us + idx * 16, Ug + idx, 16u);
    cp_async_commit();
  }
  // rows that no copy has filled must hold finite numbers: they meet zero weights (a ragged last tile)
  for (int idx = tid; idx < v_bytes / 16; idx += kRopeThreads) reinterpret_cast<uint4*>(Vs)[idx] = make_uint4(0u, 0u, 0u, 0u);

  // Thread (row, hf): row = 32 (warp & 3) + lane is its TMEM lane, hf = warp >> 2 picks the chunks of eight pairs
  // 2m + hf (m = 0..3).  Its constants e^{i row phi} for those pairs come from the table the layer keeps:
  // entry [k][row] = cos, cos, sin, sin of pairs 2k, 2k + 1.
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
  // the query of this unit, scaled by log2(e)/sqrt(d_h): thread i < half owns pair i, turned to the first tile's
  // offset here (the angle reduced in fp64), then by e^{-i 128 phi} per tile
  float q_re = 0.f, q_im = 0.f, step_c = 1.f, step_s = 0.f, q_norm2 = 0.f;
  if (tid < half) {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q) + b * p.q_stride_b + static_cast<int64_t>(hq) * p.d_head;
    const int ia = INTERLEAVED ? 2 * tid : tid, ib = INTERLEAVED ? 2 * tid + 1 : tid + half;
    const float a_re = __bfloat162float(qg[ia]) * p.q_scale, a_im = __bfloat162float(qg[ib]) * p.q_scale;
    double ang = static_cast<double>(n_b - 1 - t_lo * kTile) * p.inv_freq[tid];
    ang -= kTwoPi * rint(ang / kTwoPi);
    float s_, c_;
    sincosf(static_cast<float>(ang), &s_, &c_);
    q_re = a_re * c_ - a_im * s_;
    q_im = a_re * s_ + a_im * c_;
    q_norm2 = a_re * a_re + a_im * a_im;
    const float2 st = __ldg(p.tile_step + tid);
    step_c = st.x;
    step_s = st.y;
    q_tile[tid] = q_re;                                      // the first tile's query
    q_tile[64 + tid] = q_im;
    q_tile[128 + tid] = -q_re;
  }

  cp_async_wait<0>();
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;

  // ---- what the two issuing threads do (tile i of this CTA is tile t_lo + i of the unit)
  const uint64_t policy = policy_evict_first();
  const void* map_k = static_cast<const unsigned char*>(p.tmaps) + static_cast<size_t>(h) * 256;
  // K' tile i into buffer i & 1: two boxes of 64 rows per atom column, in the layout the lift's A operand names (no
  // thread moves the tile); elements past the rank and rows past the capacity arrive as zeros, rows between the
  // sequence's length and the capacity are finite (the cache starts as zeros) and meet zero weights
  // With a page table the tile's rows are where the table says: a page holds whole tiles and lies inside one
  // sequence's slab, so the tile is still two boxes of the slab's tensor map and one contiguous run of V' rows.
  auto fetch_k = [&](int i) {
    const int buf = i & 1, t = t_lo + i;
    int row0 = t * kTile, slab = b;
    if (PAGED) {
      const int64_t prow = physical_row(p.pages, b, p.n_max, row0);
      slab = static_cast<int>(prow / p.n_max);
      row0 = static_cast<int>(prow - static_cast<int64_t>(slab) * p.n_max);
    }
    mbar_arrive_expect_tx(&hdr->k_full[buf], static_cast<uint32_t>(kt_bytes));
    for (int a = 0; a < ak; ++a)
      for (int hh = 0; hh < 2; ++hh)
        tma_load_3d(Kt + buf * kt_bytes + a * kRopeAtom + hh * (kRopeAtom / 2), map_k, a * 64, row0 + hh * 64, slab,
                    &hdr->k_full[buf]);
  };
  auto fetch_v = [&](int i) {
    const int t = t_lo + i;
    const uint32_t bytes = static_cast<uint32_t>(min(kTile, n_b - t * kTile)) * rowb_v;
    mbar_arrive_expect_tx(&hdr->v_full, bytes);
    const int64_t prow = PAGED ? physical_row(p.pages, b, p.n_max, t * kTile) : static_cast<int64_t>(b) * p.n_max + t * kTile;
    bulk_load(Vs, p.cache + hd.v_off + prow * rowb_v, bytes, &hdr->v_full, policy);
  };
  // X(i) = K'(i) (U^K)^T into accumulator i & 1, once the tile's rows have landed; false if that wait gave up
  auto issue_lift = [&](int i) -> bool {
    if (!mbar_wait(&hdr->k_full[i & 1], (i >> 1) & 1u, p.status)) return false;
    tc_fence_after();
    const uint32_t idesc = instr_desc(p.d_head, false);
    const uint64_t dk = smem_desc_sw128(smem_u32(Kt + (i & 1) * kt_bytes), 16, 1024), du = smem_desc(smem_u32(Us), 128, grp_k);
    for (int s = 0; s < (rpk16 >> 4); ++s)                   // 16 rank elements a step: 32 bytes along the swizzled rows
      mma_ss(tmem + (i & 1) * kTile, dk + (s >> 2) * (kRopeAtom >> 4) + (s & 3) * 2, du + s * 16, idesc, s > 0);
    mma_commit(&hdr->x_full[i & 1]);
    return true;
  };
  // ---- before the first tile: two K' tiles and the V' tile requested, X(0) and X(1) under way, then K'(2) behind X(0)
  bool live = true;                                          // an issuing thread: none of its waits has given up
  if (tid == kRopeRequester) {
    tensormap_acquire(map_k);
    fetch_k(0);
    if (nt_cta > 1) fetch_k(1);
    fetch_v(0);
    if (nt_cta > 2) {
      live = mbar_wait(&hdr->x_full[0], 0u, p.status);
      if (live) fetch_k(2);
    }
  } else if (tid == kRopeLifter) {
    live = issue_lift(0);
    if (live && nt_cta > 1) live = issue_lift(1);
  }
  __syncwarp();

  const uint32_t tX = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
  // weighted sum o' += p V' (warps 0-5): thread (vg, vc) owns the eight columns of 16-byte chunk vc over the rows of
  // row group vg of every tile; the row groups are added up once, at the end
  const int chunks = hd.rp_v >> 3;
  const int row_groups = min(kRopeSumThreads / chunks, 64);
  const int rows_per_group = (kTile + row_groups - 1) / row_groups;
  const int pv_g = tid / chunks, pv_c = tid - pv_g * chunks;
  const bool pv_on = tid < kRopeSumThreads && pv_g < row_groups;
  const int r_lo = min(kTile, pv_g * rows_per_group), r_hi = pv_on ? min(kTile, r_lo + rows_per_group) : r_lo;
  unsigned long long o_acc[4] = {0ull, 0ull, 0ull, 0ull};   // columns (0,1), (2,3), (4,5), (6,7) of the chunk
  // online softmax in base 2 against a reference m_ref that every thread of the CTA holds alike; it moves only when
  // a score of the tile passes it by more than kRopeLazy (the first tile always does)
  float m_ref = -INFINITY, l_thr = 0.f;
  bool ok = true;
  for (int i = 0; i < nt_cta; ++i) {
    const int t = t_lo + i;
    const uint32_t par = i & 1u;
    const float* qt = q_tile + par * 192;                    // this tile's query pairs (written a tile ago)
    // the V' tile is free once the weighted sum of tile i - 1 is over: request this tile's rows
    if (tid == kRopeRequester && i >= 1 && live) {
      live = mbar_wait(&hdr->v_free, (i - 1) & 1u, p.status);
      if (live) fetch_v(i);
    }
    __syncwarp();
    const bool have_x = mbar_wait(&hdr->x_full[par], (i >> 1) & 1u, p.status);
    tc_fence_after();
    // ---- this thread's half of the row's score.  Two pairs per packed instruction:
    // W = Q_t conj(E_l), pair term = Re(W conj(X)) = W_re x_re + W_im x_im.
    unsigned long long acc_re = 0ull, acc_im = 0ull;         // (0.f, 0.f)
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const int c = 2 * m + hf;
      uint32_t xc[16];                                       // re[8], im[8] (pairs (i, i + d_h/2)) or re, im alternating
      if (have_x && (HALF == 64 || 8 * c < half)) {
        if (INTERLEAVED) {
          tmem_ld16(tX + par * kTile + 16 * c, xc);
        } else {
          tmem_ld8(tX + par * kTile + 8 * c, *reinterpret_cast<uint32_t(*)[8]>(&xc[0]));
          tmem_ld8(tX + par * kTile + half + 8 * c, *reinterpret_cast<uint32_t(*)[8]>(&xc[8]));
        }
      }
      tmem_wait_ld();
      if (HALF == 64 || 8 * c < half) {
        const float* qc = qt + 8 * c;
#pragma unroll
        for (int e = 0; e < 8; e += 4) {                     // four pairs a step
          const float4 qr4 = *reinterpret_cast<const float4*>(qc + e);
          const float4 qi4 = *reinterpret_cast<const float4*>(qc + 64 + e);
          const float4 qn4 = *reinterpret_cast<const float4*>(qc + 128 + e);
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
            const unsigned long long qr = k == 0 ? pack2(qr4.x, qr4.y) : pack2(qr4.z, qr4.w);
            const unsigned long long qi = k == 0 ? pack2(qi4.x, qi4.y) : pack2(qi4.z, qi4.w);
            const unsigned long long qn = k == 0 ? pack2(qn4.x, qn4.y) : pack2(qn4.z, qn4.w);
            const unsigned long long ec = el_c[4 * m + (ee >> 1)], es = el_s[4 * m + (ee >> 1)];
            const unsigned long long w_re = fma2p(qi, es, mul2p(qr, ec));                  // Qr c + Qi s
            const unsigned long long w_im = fma2p(qn, es, mul2p(qi, ec));                  // Qi c - Qr s
            acc_re = fma2p(w_re, x_re, acc_re);
            acc_im = fma2p(w_im, x_im, acc_im);
          }
        }
      }
    }
    {
      float s0, s1, s2, s3;
      unpack2(acc_re, s0, s1);
      unpack2(acc_im, s2, s3);
      sc[hf * kTile + row] = (s0 + s2) + (s1 + s3);
    }
    tc_fence_before();
    // both halves of every row's score are in shared memory and X(i) is read; a wait that gave up anywhere ends the loop
    if (cta_sync_or(!have_x || !live)) { ok = false; break; }
    // ---- the next tile's query: one more turn by -128 phi into the other buffer (read after the next barrier);
    // the length is pulled back to |q| so that rounding does not drift over a thousand tiles
    if (tid < half) {
      const float n_re = q_re * step_c - q_im * step_s, n_im = q_re * step_s + q_im * step_c;
      const float fix = 1.5f - 0.5f * (n_re * n_re + n_im * n_im) / fmaxf(q_norm2, 1e-30f);   // ~ |q| / |n|
      q_re = n_re * fix;
      q_im = n_im * fix;
      float* qn = q_tile + (par ^ 1u) * 192;
      qn[tid] = q_re;
      qn[64 + tid] = q_im;
      qn[128 + tid] = -q_re;
    }
    // ---- the row's weight against the reference as it stands (warps 0-3: one thread per row)
    float s = -INFINITY, pj = 0.f;
    if (hf == 0) {
      if (t * kTile + row < n_b) s = sc[row] + sc[kTile + row];
      pj = ex2(s - m_ref);                                   // redone below if the reference moves
      p_row[row] = pj;
    }
    const bool have_v = tid >= kRopeSumThreads || mbar_wait(&hdr->v_full, par, p.status);
    // the weights are written, the V' tile has landed; the reference must move if a score passed it by kRopeLazy
    if (cta_sync_or(s > m_ref + kRopeLazy || !have_v)) {
      if (cta_sync_or(!have_v)) { ok = false; break; }       // (also: every thread has read the weights' flag state)
      // every thread adds up the four rows lane, lane + 32, ...: the tile maximum is one warp reduction
      float mx = -INFINITY;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int r = k * 32 + lane;
        if (t * kTile + r < n_b) mx = fmaxf(mx, sc[r] + sc[kTile + r]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_ref, mx);
      const float alpha = ex2(m_ref - m_new);                // 0 at the first tile
      const unsigned long long alpha2 = pack2(alpha, alpha);
#pragma unroll
      for (int k = 0; k < 4; ++k) o_acc[k] = mul2p(o_acc[k], alpha2);
      l_thr *= alpha;
      m_ref = m_new;
      if (hf == 0) {
        pj = ex2(s - m_ref);                                 // 0 for a row past the sequence's length
        p_row[row] = pj;
      }
      __syncthreads();                                       // the weights are rewritten
    }
    l_thr += pj;
    if (tid < kRopeSumThreads) {
      // ---- o' += sum_j p_j V'[j][8 vc .. 8 vc + 7] over this thread's rows (row-major tile, 16 bytes a row)
      const unsigned char* v_chunk = Vs + 16 * pv_c;
#pragma unroll 2
      for (int r = r_lo; r < r_hi; ++r) {
        const uint4 v = *reinterpret_cast<const uint4*>(v_chunk + r * rowb_v);
        const float pr = p_row[r];
        const unsigned long long p2 = pack2(pr, pr);
        o_acc[0] = fma2p(p2, pack2(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u)), o_acc[0]);
        o_acc[1] = fma2p(p2, pack2(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u)), o_acc[1]);
        o_acc[2] = fma2p(p2, pack2(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xffff0000u)), o_acc[2]);
        o_acc[3] = fma2p(p2, pack2(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xffff0000u)), o_acc[3]);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&hdr->v_free);              // this warp has read its rows of the V' tile
    } else {
      // ---- meanwhile the two issuing threads: K'(i + 3) into the buffer X(i + 1) was lifted from (that lift went out
      // a tile ago), and X(i + 2) into the accumulator every thread has just read (its rows were requested a tile ago)
      if (tid == kRopeRequester && live && i + 3 < nt_cta) {
        live = mbar_wait(&hdr->x_full[(i + 1) & 1], ((i + 1) >> 1) & 1u, p.status);
        if (live) fetch_k(i + 3);
      }
      if (tid == kRopeLifter && live && i + 2 < nt_cta) live = issue_lift(i + 2);
      __syncwarp();
    }
  }

  // ---- the piece's partial: m, l (sum over the rows), o'
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l_thr += __shfl_xor_sync(0xffffffffu, l_thr, o);
  __syncthreads();                                           // every thread is through with the V' tile
  if (lane == 0 && hf == 0) hdr->red[warp] = l_thr;
  // add up the row groups (the V' tile's shared memory is free: its last copy was waited for, or the launch gave up)
  float* o_red = reinterpret_cast<float*>(Vs);
  if (ok && pv_on) {
    float* dst = o_red + pv_g * hd.rp_v + 8 * pv_c;
#pragma unroll
    for (int k = 0; k < 4; ++k) unpack2(o_acc[k], dst[2 * k], dst[2 * k + 1]);
  }
  __syncthreads();
  if (tid == 0) {
    part[0] = m_ref;
    part[1] = (hdr->red[0] + hdr->red[1]) + (hdr->red[2] + hdr->red[3]);
  }
  if (tid < hd.rp_v) {
    float o = 0.f;
    if (ok)
      for (int k = 0; k < row_groups; ++k) o += o_red[k * hd.rp_v + tid];
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
  const int hq = unit / p.B, b = unit - hq * p.B;
  const int h = hq / p.group;
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
    out[b * p.out_stride_b + static_cast<int64_t>(hq) * p.d_head + t] = __float2bfloat16_rn(y);
  }
}

}  // namespace

size_t decode_rope_smem_bytes(int max_rp_k, int max_rp_v, int d_head) {
  const int k16 = (max_rp_k + 15) & ~15;
  // header, U^K image, two K' tiles in swizzled atom columns of 64 elements, V' tile
  return kRopeHeaderBytes + rope_kb(d_head * k16 * 2) + 2 * static_cast<size_t>((k16 + 63) >> 6) * kRopeAtom +
         rope_kb(kTile * max_rp_v * 2);
}

cudaError_t launch_decode_rope(const RopeDecodeParams& p, size_t smem, cudaStream_t s, uint64_t* launches) {
  static size_t configured[8][kMaxDevices] = {};
  auto run = [&](auto kernel, size_t (&done)[kMaxDevices]) -> cudaError_t {
    const cudaError_t ec = ensure_dynamic_smem(kernel, smem, done);
    if (ec != cudaSuccess) return ec;
    kernel<<<dim3(p.B * p.H * p.group, p.splits), kRopeThreads, smem, s>>>(p);
    return cudaGetLastError();
  };
  const bool paged = p.pages.table != nullptr, wide = p.d_head == 128, inter = p.interleaved != 0;
  const int which = (paged ? 4 : 0) + (wide ? 2 : 0) + (inter ? 1 : 0);
  cudaError_t e;
  switch (which) {
    case 0: e = run(decode_rope_kernel<false, 0, false>, configured[0]); break;
    case 1: e = run(decode_rope_kernel<true, 0, false>, configured[1]); break;
    case 2: e = run(decode_rope_kernel<false, 64, false>, configured[2]); break;
    case 3: e = run(decode_rope_kernel<true, 64, false>, configured[3]); break;
    case 4: e = run(decode_rope_kernel<false, 0, true>, configured[4]); break;
    case 5: e = run(decode_rope_kernel<true, 0, true>, configured[5]); break;
    case 6: e = run(decode_rope_kernel<false, 64, true>, configured[6]); break;
    default: e = run(decode_rope_kernel<true, 64, true>, configured[7]); break;
  }
  ++*launches;
  if (e != cudaSuccess) return e;
  rope_combine_kernel<<<p.B * p.H * p.group, 128, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
