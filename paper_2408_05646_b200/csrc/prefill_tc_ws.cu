// Warp-specialised causal rank-r prefill attention on the tensor cores (tcgen05 + TMEM).
//
// Same mathematics as prefill_tc.cu (S = Q'K'^T, online softmax, O' = P V', lift through (U^V)^T), but
// organised so that the tensor pipe, the loads and the softmax run concurrently.  One CTA per SM owns
// 256 query rows of one (sequence, head) unit as two 128-row tiles A and B:
//   * two loader warps stream the K'/V' tiles of the unit from the rank-r cache into a ring of shared
//     memory stages with 16-byte cp.async copies that place every chunk in the canonical core-matrix
//     layout (each K'/V' tile is fetched once for both query tiles);
//   * one thread of the MMA warp issues, for every key tile, PV_A, S_A(next), PV_B, S_B(next); every
//     group is followed by a tcgen05.commit onto the mbarrier that its consumer waits on;
//   * two softmax warpgroups (4 warps each, one thread per query row) alternate with the tensor pipe:
//     while group A turns S_A into P_A, the pipe works for group B, and vice versa.
// TMEM (512 columns): S_A, S_B (128 each), O'_A, O'_B (up to 128 each).  Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kSoftmaxWarps = 8;
constexpr int kMmaWarp = 8;
constexpr int kLoadWarp0 = 9;
constexpr int kLoadWarps = 2;
constexpr int kSIssueWarp = 11;               // issues the S products; kMmaWarp issues the PV products
constexpr int kWsThreads = (kSoftmaxWarps + 1 + kLoadWarps + 1) * 32;
constexpr int kMaxStages = 3;

struct __align__(16) WsHeader {
  unsigned long long kv_full[kMaxStages], kv_empty[kMaxStages];
  unsigned long long q_full;
  unsigned long long s_full[2], p_full[2], o_done[2];
  unsigned long long lift_done;
  uint32_t tmem_base;
  int abort_flag;
};

// One loader warp's share of a canonical tile: 16-byte chunks (row, c) for the index range it owns.
// Two neighbouring lanes fetch the two halves of a 32-byte piece of a row.
__device__ __forceinline__ void load_tile_async(unsigned char* dst, const __nv_bfloat16* src, int rp, int rows_valid,
                                                int nch, int loader, int lane) {
  const int src_chunks = rp >> 3;
  const int group_stride = nch << 7;
  for (int idx = loader * 32 + lane; idx < kTile * nch; idx += kLoadWarps * 32) {
    const int c = ((idx >> 8) << 1) + (idx & 1), row = (idx >> 1) & (kTile - 1);
    const bool live = row < rows_valid && c < src_chunks;
    const void* g = live ? static_cast<const void*>(src + static_cast<int64_t>(row) * rp + c * 8) : src;
    cp_async16(dst + chunk_off(row, c, group_stride), g, live ? 16u : 0u);
  }
}

__global__ void __launch_bounds__(kWsThreads, 1) prefill_tc_ws_kernel(const PrefillParams p, int stages) {
  extern __shared__ __align__(1024) unsigned char smem[];
  WsHeader* hdr = reinterpret_cast<WsHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const int qblk = gridDim.y - 1 - blockIdx.y;              // late (long) query blocks first
  const int t0 = qblk * 2 * kTile;
  const int rpk16 = (hd.rp_k + 15) & ~15, rpv16 = (hd.rp_v + 15) & ~15;
  const int nch_k = rpk16 >> 3, nch_v = rpv16 >> 3;
  const int grp_k = nch_k << 7, grp_v = nch_v << 7, grp_p = (kTile >> 3) << 7;
  const int q_bytes = kTile * rpk16 * 2, k_bytes = q_bytes, v_bytes = kTile * rpv16 * 2;
  const int stage_bytes = k_bytes + v_bytes;

  unsigned char* tiles = smem + 1024;
  unsigned char* Qs = tiles;                                 // Q_A, Q_B
  unsigned char* ring = Qs + 2 * q_bytes;                    // stages x (K tile, V tile)
  unsigned char* Ps = ring + stages * stage_bytes;           // P_A, P_B (128 x 128 bf16 each)
  const int p_bytes = kTile * kTile * 2;

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 512);
  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(&hdr->kv_full[s], kLoadWarps);
      mbar_init(&hdr->kv_empty[s], 1);
    }
    mbar_init(&hdr->q_full, kLoadWarps);
    for (int x = 0; x < 2; ++x) {
      mbar_init(&hdr->s_full[x], 1);
      mbar_init(&hdr->p_full[x], kTile);
      mbar_init(&hdr->o_done[x], 1);
    }
    mbar_init(&hdr->lift_done, 1);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  volatile int* abort_flag = &hdr->abort_flag;

  // key tiles each query tile needs (tile B starts 128 rows later, so it needs one more in general)
  int n_tiles[2];
  for (int x = 0; x < 2; ++x) {
    const int tx = t0 + x * kTile;
    n_tiles[x] = tx < p.T ? (p.len0 + min(p.T, tx + kTile) + kTile - 1) / kTile : 0;
  }
  const int n_max_tiles = max(n_tiles[0], n_tiles[1]);
  const int n_keys = p.len0 + min(p.T, t0 + 2 * kTile);      // rows of K'/V' the CTA may touch
  const int total_rows = p.B * p.T;

  if (warp >= kLoadWarp0 && warp < kLoadWarp0 + kLoadWarps) {
    // ------------------------------------------------------------------ loaders
    const int ld = warp - kLoadWarp0;
    const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.qp) +
                              static_cast<int64_t>(hd.lr_k_off) * total_rows +
                              (static_cast<int64_t>(b) * p.T + t0) * hd.rp_k;
    const __nv_bfloat16* Kg = reinterpret_cast<const __nv_bfloat16*>(p.cache + hd.k_off) +
                              static_cast<int64_t>(b) * p.n_max * hd.rp_k;
    const __nv_bfloat16* Vg = reinterpret_cast<const __nv_bfloat16*>(p.cache + hd.v_off) +
                              static_cast<int64_t>(b) * p.n_max * hd.rp_v;
    for (int x = 0; x < 2; ++x) {
      const int q_rows = max(0, min(kTile, p.T - t0 - x * kTile));
      load_tile_async(Qs + x * q_bytes, q_rows > 0 ? Qg + static_cast<int64_t>(x) * kTile * hd.rp_k : Qg, hd.rp_k,
                      q_rows, nch_k, ld, lane);
    }
    cp_async_commit();
    // Copy groups in issue order: group 0 = the Q tiles, group j + 1 = key tile j.  `signalled` groups have
    // been announced on their barrier; a group may be announced once cp.async.wait_group says it landed.
    int committed = 1, signalled = 0;
    auto announce = [&](int upto) {                          // groups [signalled, upto) have landed
      fence_async_smem();
      __syncwarp();
      if (lane == 0)
        for (int g = signalled; g < upto; ++g) mbar_arrive(g == 0 ? &hdr->q_full : &hdr->kv_full[(g - 1) % stages]);
      signalled = max(signalled, upto);
    };
    bool ok = true;
    for (int j = 0; j < n_max_tiles; ++j) {
      const int stage = j % stages;
      if (j >= stages) {
        // everything issued so far must be announced before blocking on a free stage: the MMA warp frees
        // stages only after it has seen the tiles that are still in flight here
        cp_async_wait<0>();
        announce(committed);
        if (lane == 0) ok = mbar_wait(&hdr->kv_empty[stage], ((j / stages) - 1) & 1u, p.status) && !*abort_flag;
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;   // one decision for the whole warp
        if (!ok) { *abort_flag = 1; break; }
      }
      const int key0 = j * kTile;
      const int k_valid = min(kTile, n_keys - key0);
      unsigned char* st = ring + stage * stage_bytes;
      load_tile_async(st, Kg + static_cast<int64_t>(key0) * hd.rp_k, hd.rp_k, k_valid, nch_k, ld, lane);
      load_tile_async(st + k_bytes, Vg + static_cast<int64_t>(key0) * hd.rp_v, hd.rp_v, k_valid, nch_v, ld, lane);
      cp_async_commit();
      ++committed;
      cp_async_wait<1>();                                    // everything but the newest group has landed
      announce(committed - 1);
    }
    cp_async_wait<0>();
    if (ok) announce(committed);
  } else if (warp == kMmaWarp || warp == kSIssueWarp) {
    // ------------------------------------------------------------------ MMA issuers
    // Two threads feed the tensor pipe so that their per-instruction latencies overlap: one issues the
    // PV products, the other the S products of the next key tile.  Both start a tile's work when the
    // softmax group has written P (which also means it has consumed S).  Descriptors are built once
    // and advanced by adding 16-byte units to their address field.
    if (lane == 0) {
      const bool pv_role = warp == kMmaWarp;
      const uint32_t idesc_s = instr_desc(kTile, false);
      const uint32_t idesc_o = instr_desc(rpv16, true);
      const uint32_t qa = smem_u32(Qs), ra = smem_u32(ring), pa = smem_u32(Ps);
      const uint64_t dq[2] = {smem_desc(qa, 128, grp_k), smem_desc(qa + q_bytes, 128, grp_k)};
      const uint64_t dp[2] = {smem_desc(pa, 128, grp_p), smem_desc(pa + p_bytes, 128, grp_p)};
      const uint64_t dk0 = smem_desc(ra, 128, grp_k);                 // K tile of stage 0 (K-major B operand)
      const uint64_t dv0 = smem_desc(ra + k_bytes, grp_v, 128);       // V tile of stage 0 (MN-major B operand)
      const uint64_t stage_step = static_cast<uint64_t>(stage_bytes >> 4);
      const uint64_t v_step = static_cast<uint64_t>((2 * grp_v) >> 4); // 16 keys = two 8-row groups
      const int ks_steps = rpk16 >> 4;
      const uint32_t ts[2] = {tmem, tmem + kTile}, to[2] = {tmem + 256, tmem + 256 + kTile};
      auto issue_s = [&](int x, int stage) {                 // S_x = Q_x K^T, contraction over the rank
        uint64_t a = dq[x], bk = dk0 + stage * stage_step;
        for (int s = 0; s < ks_steps; ++s, a += 16, bk += 16) mma_ss(ts[x], a, bk, idesc_s, s > 0);
        mma_commit(&hdr->s_full[x]);
      };
      bool ok = true;
      if (!pv_role) {
        ok = mbar_wait(&hdr->q_full, 0, p.status) && mbar_wait(&hdr->kv_full[0], 0, p.status);
        if (ok) {
          tc_fence_after();
          for (int x = 0; x < 2; ++x)
            if (n_tiles[x] > 0) issue_s(x, 0);
        }
      }
      int stage = 0, nstage = stages > 1 ? 1 : 0;            // ring slots of key tiles j and j + 1
      uint32_t nparity = stages > 1 ? 0u : 1u;               // kv_full parity of tile j + 1
      for (int j = 0; j < n_max_tiles && ok; ++j) {
        for (int x = 0; x < 2 && ok; ++x) {
          if (j >= n_tiles[x]) continue;
          if (!pv_role && j + 1 >= n_tiles[x]) continue;     // no further S product for this tile
          ok = mbar_wait(&hdr->p_full[x], j & 1u, p.status) && !*abort_flag;
          if (!ok) break;
          tc_fence_after();
          if (pv_role) {
            uint64_t a = dp[x], bv = dv0 + stage * stage_step;
#pragma unroll
            for (int s = 0; s < kTile / 16; ++s, a += 16, bv += v_step)   // O'_x += P_x V_j over the 128 keys
              mma_ss(to[x], a, bv, idesc_o, j > 0 || s > 0);
            mma_commit(&hdr->o_done[x]);
          } else {
            ok = mbar_wait(&hdr->kv_full[nstage], nparity, p.status);
            if (!ok) break;
            tc_fence_after();
            issue_s(x, nstage);
          }
        }
        // the PV products are the last readers of a stage (its S products completed before the softmax ran)
        if (ok && pv_role) mma_commit(&hdr->kv_empty[stage]);
        stage = nstage;
        if (++nstage == stages) { nstage = 0; nparity ^= 1u; }
      }
      // the last commit's arrival must have landed before the CTA may leave
      if (ok && pv_role)
        ok = mbar_wait(&hdr->kv_empty[(n_max_tiles - 1) % stages], ((n_max_tiles - 1) / stages) & 1u, p.status);
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ softmax warpgroups
    const int x = warp >> 2;                                 // 0 = tile A, 1 = tile B
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + x * kTile;
    const uint32_t tO = tmem + lane_base + 256 + x * kTile;
    unsigned char* Px = Ps + x * p_bytes;
    const int tx = t0 + x * kTile;
    const int my_pos = p.len0 + tx + row;                    // last key this thread's query sees
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles[x] && ok; ++j) {
      const int key0 = j * kTile;
      ok = mbar_wait(&hdr->s_full[x], j & 1u, p.status);
      ok = __all_sync(0xffffffffu, ok && !*abort_flag);      // one decision for the whole warp
      if (!ok) break;
      tc_fence_after();
      const bool diag = key0 + kTile - 1 > p.len0 + tx;      // some (row, key) pair of the tile is masked
      // pass 1: row maximum, 64 columns per TMEM round trip
      float row_max = -INFINITY;
#pragma unroll 1
      for (int c0 = 0; c0 < kTile; c0 += 64) {
        uint32_t r[64];
        tmem_ld64(tS + c0, r);
        tmem_wait_ld();
        if (diag) {
#pragma unroll
          for (int i = 0; i < 64; ++i)
            if (key0 + c0 + i <= my_pos) row_max = fmaxf(row_max, __uint_as_float(r[i]));
        } else {
#pragma unroll
          for (int i = 0; i < 64; ++i) row_max = fmaxf(row_max, __uint_as_float(r[i]));
        }
      }
      row_max *= p.scale_log2;                               // the scale is positive: max and scale commute
      // Lazy reference: the exponentials use m_run, which follows the true maximum only when that has grown
      // by more than 8 (a factor 256 that fp32 sums and bf16 P absorb); O' is rescaled only then.
      float alpha = 1.f;
      if (row_max > m_run + 8.f) {
        alpha = ex2(m_run - row_max);
        m_run = row_max;
      }
      if (j > 0) {                                           // P_x and O'_x are free once PV_x(j-1) is done
        ok = mbar_wait(&hdr->o_done[x], (j - 1) & 1u, p.status);
        ok = __all_sync(0xffffffffu, ok && !*abort_flag);
        if (!ok) break;
        tc_fence_after();
      }
      // pass 2: exponentials, row sum, P as bf16 into the A-operand tile
      float row_sum = 0.f;
      const float neg_m = -m_run;
#pragma unroll 1
      for (int c0 = 0; c0 < kTile; c0 += 64) {
        uint32_t r[64];
        tmem_ld64(tS + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          // P is cut to bf16 by truncation with integer ops, and the row sum adds the truncated values, so
          // numerator and denominator of the softmax use identical weights.
          uint32_t pt[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float e = ex2(fmaf(__uint_as_float(r[g * 8 + i]), p.scale_log2, neg_m));
            if (diag && key0 + c0 + g * 8 + i > my_pos) e = 0.f;
            pt[i] = __float_as_uint(e) & 0xffff0000u;
            row_sum += __uint_as_float(pt[i]);
          }
          uint4 w;
          w.x = __byte_perm(pt[0], pt[1], 0x7632); w.y = __byte_perm(pt[2], pt[3], 0x7632);
          w.z = __byte_perm(pt[4], pt[5], 0x7632); w.w = __byte_perm(pt[6], pt[7], 0x7632);
          *reinterpret_cast<uint4*>(Px + chunk_off(row, (c0 >> 3) + g, grp_p)) = w;
        }
      }
      l_run = l_run * alpha + row_sum;
      if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {  // rescale this row of O' (rare after the first tiles)
#pragma unroll 1
        for (int h0 = 0; h0 < rpv16; h0 += 64) {             // up to 64 columns per round trip
          uint32_t r[64];
#pragma unroll
          for (int c0 = 0; c0 < 64; c0 += 16)
            if (h0 + c0 < rpv16) tmem_ld16(tO + h0 + c0, *reinterpret_cast<uint32_t(*)[16]>(&r[c0]));
          tmem_wait_ld();
#pragma unroll
          for (int c0 = 0; c0 < 64; c0 += 16)
            if (h0 + c0 < rpv16) {
#pragma unroll
              for (int i = 0; i < 16; ++i) r[c0 + i] = __float_as_uint(__uint_as_float(r[c0 + i]) * alpha);
              tmem_st16(tO + h0 + c0, *reinterpret_cast<const uint32_t(*)[16]>(&r[c0]));
            }
        }
        tmem_wait_st();
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(&hdr->p_full[x]);
    }
    if (ok && n_tiles[x] > 0) {
      ok = mbar_wait(&hdr->o_done[x], (n_tiles[x] - 1) & 1u, p.status);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
    }
    if (!ok) *abort_flag = 1;

    // ---- epilogue part 1 (after every role is done with the main loop)
    tc_fence_before();
    __syncthreads();                                         // #1
    const bool run = !*abort_flag && n_tiles[x] > 0;
    const float inv_l = 1.f / l_run;
    const bool lowrank = (p.flags & 0x2u) != 0;
    const int q_valid = min(kTile, p.T - tx);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.out);
    unsigned char* Oh = tiles + x * 2 * v_bytes;             // O' hi and lo of this tile, [128][rpv16] each
    unsigned char* Ol = Oh + v_bytes;
    if (run) {
      tc_fence_after();
      __nv_bfloat16* dst_lr = out + b * p.out_stride_b + static_cast<int64_t>(tx + row) * p.out_stride_t + hd.lr_v_off;
      for (int c0 = 0; c0 < rpv16; c0 += 16) {
        uint32_t r[16];
        tmem_ld16(tO + c0, r);
        tmem_wait_ld();
        if (lowrank) {
          if (row < q_valid)
            for (int i = 0; i < 16; ++i)
              if (c0 + i < hd.rp_v) dst_lr[c0 + i] = __float2bfloat16_rn(__uint_as_float(r[i]) * inv_l);
        } else {
          uint32_t hi[8], lo[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float x0 = __uint_as_float(r[2 * i]) * inv_l, x1 = __uint_as_float(r[2 * i + 1]) * inv_l;
            const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
            hi[i] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
            lo[i] = pack_bf16(x0 - __bfloat162float(h0), x1 - __bfloat162float(h1));
          }
          *reinterpret_cast<uint4*>(Oh + chunk_off(row, c0 >> 3, grp_v)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(Oh + chunk_off(row, (c0 >> 3) + 1, grp_v)) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
          *reinterpret_cast<uint4*>(Ol + chunk_off(row, c0 >> 3, grp_v)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          *reinterpret_cast<uint4*>(Ol + chunk_off(row, (c0 >> 3) + 1, grp_v)) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        }
      }
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();                                         // #2
    if (run && !lowrank) {                                   // the lifted rows come back through S_x's columns
      bool ok2 = mbar_wait(&hdr->lift_done, 0, p.status);
      ok2 = __all_sync(0xffffffffu, ok2);
      tc_fence_after();
      if (ok2) {
        __nv_bfloat16* dst = out + b * p.out_stride_b + static_cast<int64_t>(tx + row) * p.out_stride_t +
                             static_cast<int64_t>(h) * p.d_head;
        for (int c0 = 0; c0 < p.d_head; c0 += 16) {
          uint32_t r[16];
          tmem_ld16(tS + c0, r);
          tmem_wait_ld();
          if (row < q_valid) {
            uint4 w0, w1;
            w0.x = pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1]));
            w0.y = pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3]));
            w0.z = pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5]));
            w0.w = pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7]));
            w1.x = pack_bf16(__uint_as_float(r[8]), __uint_as_float(r[9]));
            w1.y = pack_bf16(__uint_as_float(r[10]), __uint_as_float(r[11]));
            w1.z = pack_bf16(__uint_as_float(r[12]), __uint_as_float(r[13]));
            w1.w = pack_bf16(__uint_as_float(r[14]), __uint_as_float(r[15]));
            *reinterpret_cast<uint4*>(dst + c0) = w0;
            *reinterpret_cast<uint4*>(dst + c0 + 8) = w1;
          }
        }
      }
    }
    tc_fence_before();
    __syncthreads();                                         // #3
    if (warp == 0) tmem_dealloc(tmem, 512);
    return;
  }

  // ---- MMA and loader warps: epilogue
  tc_fence_before();
  __syncthreads();                                           // #1
  const bool lowrank = (p.flags & 0x2u) != 0;
  const bool run = !*abort_flag && !lowrank;
  unsigned char* Uh = tiles + 4 * v_bytes;                   // lift image of U^V: [d_head][rpv16] hi, then lo
  const int img16 = p.d_head * rpv16 * 2 / 16;               // 16-byte words per image
  if (run) {
    const uint4* Ug = reinterpret_cast<const uint4*>(p.basis + hd.uvl16_off);
    for (int idx = tid - kMmaWarp * 32; idx < 2 * img16; idx += (2 + kLoadWarps) * 32)
      reinterpret_cast<uint4*>(Uh)[idx] = __ldg(Ug + idx);
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();                                           // #2
  if (run && warp == kMmaWarp && lane == 0) {
    tc_fence_after();
    const uint32_t idesc_l = instr_desc(p.d_head, false);
    const uint32_t uh = smem_u32(Uh), ul = uh + img16 * 16;
    for (int x = 0; x < 2; ++x) {
      if (n_tiles[x] == 0) continue;
      const uint32_t oh = smem_u32(tiles + x * 2 * v_bytes), ol = oh + v_bytes;
      bool acc = false;
      for (int pass = 0; pass < 3; ++pass) {                 // hi*hi + lo*hi + hi*lo
        const uint32_t a = pass == 1 ? ol : oh, bb = pass == 2 ? ul : uh;
        for (int s = 0; s < rpv16 / 16; ++s) {
          mma_ss(tmem + x * kTile, smem_desc(a + s * 256, 128, grp_v), smem_desc(bb + s * 256, 128, grp_v), idesc_l, acc);
          acc = true;
        }
      }
    }
    mma_commit(&hdr->lift_done);
  }
  tc_fence_before();
  __syncthreads();                                           // #3
}

}  // namespace

// Stages of the K'/V' ring that fit beside the two Q tiles and the two P tiles (0 = does not fit).
int prefill_tc_ws_stages(int max_rp_k, int max_rp_v, int d_head, size_t* smem_bytes) {
  const size_t k16 = (max_rp_k + 15) & ~15, v16 = (max_rp_v + 15) & ~15;
  const size_t fixed = 1024 + 2 * kTile * k16 * 2 + 2 * kTile * kTile * 2;
  const size_t stage = kTile * (k16 + v16) * 2;
  const size_t limit = 227 * 1024;
  int stages = 0;
  for (int s = kMaxStages; s >= 2; --s)
    if (fixed + s * stage <= limit) { stages = s; break; }
  if (stages == 0) return 0;
  const size_t total = fixed + stages * stage;
  const size_t epilogue = 1024 + 4 * kTile * v16 * 2 + 2 * static_cast<size_t>(d_head) * v16 * 2;
  if (epilogue > total) return 0;
  *smem_bytes = total;
  return stages;
}

cudaError_t launch_prefill_tc_ws(const PrefillParams& p, int stages, size_t smem, cudaStream_t s, uint64_t* launches) {
  static size_t configured = 0;     // largest dynamic shared-memory size opted into so far
  if (smem > configured) {
    const cudaError_t e = cudaFuncSetAttribute(prefill_tc_ws_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  dim3 grid(p.B * p.H, (p.T + 2 * kTile - 1) / (2 * kTile));
  prefill_tc_ws_kernel<<<grid, kWsThreads, smem, s>>>(p, stages);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
