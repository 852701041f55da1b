// Warp-specialised causal rank-r prefill attention on the tensor cores (tcgen05 + TMEM).
//
// Same mathematics as prefill_tc.cu (S = Q'K'^T, online softmax, O' = P V', lift through (U^V)^T), but
// organised so that the tensor pipe, the loads and the softmax run concurrently.  One CTA per SM owns
// 256 query rows of one (sequence, head) unit as two 128-row tiles A and B and walks the key axis in
// tiles of 64 rows:
//   * one thread streams the K'/V' tiles of the unit from the rank-r cache into a ring of shared memory
//     stages by TMA (tensor maps of the cache slabs, 64 x 64 boxes in the 128-byte swizzled layout the
//     MMA descriptors name; each tile is fetched once for both query tiles).  Elements past the rank
//     and rows past the capacity arrive as zeros;
//   * two threads feed the tensor pipe, one per query tile: PV of key tile j when the softmax group has
//     written P(j), then S of tile j + 3 into the buffer that P(j) occupied; every group of MMAs is
//     followed by a tcgen05.commit onto the mbarrier that its consumer waits on;
//   * two softmax warpgroups (4 warps each, one thread per query row = one TMEM lane), one per query
//     tile.  S is double-buffered in TMEM (2 x 64 columns per group), so the S product of key tile
//     j + 1 runs while the group turns tile j into P; a 64-key row fits in registers, and the row of
//     tile j + 1 is fetched from TMEM while the exponentials of tile j run (the softmax warps take
//     registers from the other warps for that).  P(j) (bf16) goes into the first 32 columns of the
//     buffer that S(j + 1) has just left and is the A operand of the PV product straight from TMEM: it
//     never touches shared memory.  A buffer thus cycles S(t) -> registers -> P(t-1) -> PV(t-1) -> S(t+2).
// TMEM (512 columns): S_A[2], S_B[2] (64 columns each, P aliased), O'_A, O'_B (up to 128 each).
// Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kKeys = 64;                     // key rows per tile
constexpr int kAtomBytes = kKeys * 128;       // one swizzled atom column of a K'/V' tile: 64 rows x 64 elements
constexpr int kSoftmaxWarps = 8;
constexpr int kMmaWarp = 8;                   // issues the MMAs of query tile A (and the lift)
constexpr int kLoadWarp = 9;                  // lane 0 issues the TMA copies
constexpr int kMmaWarpB = 10;                 // issues the MMAs of query tile B
constexpr int kWsThreads = 12 * 32;           // 8 softmax warps, two MMA issuers, TMA producer, one spare warp
constexpr int kRegsSoftmax = 224, kRegsOther = 56;   // registers per thread after the reallocation (launch: 168)
constexpr int kMaxStages = 8;

struct __align__(16) WsHeader {
  unsigned long long kv_full[kMaxStages], kv_empty[kMaxStages];
  unsigned long long q_full;
  unsigned long long s_full[2][2];            // [query tile][buffer]: S product of a key tile complete
  unsigned long long p_full[2][2];            // [query tile][buffer]: P written over S, O' rescaled if needed
  unsigned long long o_done[2][2];            // [query tile][buffer]: PV product of a key tile complete (P consumed)
  unsigned long long lift_done;
  uint32_t tmem_base;
  int abort_flag;
};

// One thread's share of a canonical (no swizzle) Q' tile of 128 rows, loaded by the 128 threads of a softmax
// group: 16-byte chunks (row, c); two neighbouring lanes fetch the two halves of a 32-byte piece of a row.
__device__ __forceinline__ void load_q_tile_async(unsigned char* dst, const __nv_bfloat16* src, int rp, int rows_valid,
                                                  int nch, int t) {
  const int src_chunks = rp >> 3;
  const int group_stride = nch << 7;
  for (int idx = t; idx < kTile * nch; idx += kTile) {
    const int c = ((idx / (2 * kTile)) << 1) + (idx & 1), row = (idx >> 1) & (kTile - 1);
    const bool live = row < rows_valid && c < src_chunks;
    const void* g = live ? static_cast<const void*>(src + static_cast<int64_t>(row) * rp + c * 8) : src;
    cp_async16(dst + chunk_off(row, c, group_stride), g, live ? 16u : 0u);
  }
}

// One row of a 64-key tile: exponentials relative to the reference `neg_m` (= -m, log2 domain), their sum,
// and P as 32 bf16 pairs (round to nearest) in `pk`.  DIAG: keys past `my_pos` get weight zero.  TRACK: also
// returns the row maximum of the raw scores (for the lazy reference check).
template <bool DIAG, bool TRACK>
__device__ __forceinline__ float exp_row(const uint32_t (&r)[64], float scale, float neg_m, int key0, int my_pos,
                                         uint32_t (&pk)[32], float* raw_max) {
  float sum0 = 0.f, sum1 = 0.f;
  float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    const int c = 2 * i;
    const float s0 = __uint_as_float(r[c]), s1 = __uint_as_float(r[c + 1]);
    if (TRACK) mx[i & 3] = max3(mx[i & 3], s0, s1);
    float y0, y1;
    fma2(y0, y1, s0, s1, scale, neg_m);
    float e0 = ex2(y0), e1 = ex2(y1);
    if (DIAG) {
      if (key0 + c > my_pos) e0 = 0.f;
      if (key0 + c + 1 > my_pos) e1 = 0.f;
    }
    add2(sum0, sum1, e0, e1);
    pk[i] = pack_bf16(e0, e1);
  }
  if (TRACK) *raw_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
  return sum0 + sum1;
}

// S = Q' K'^T for one query tile and one key tile: KS steps of 16 rank elements.  K' sits in atom columns of
// 64 elements (8192 bytes each); a step advances 32 bytes along the swizzled rows.
template <int KS>
__device__ __forceinline__ void issue_s(uint32_t d_tmem, uint64_t dq, uint64_t dk, uint32_t idesc) {
#pragma unroll
  for (int s = 0; s < KS; ++s)
    mma_ss(d_tmem, dq + 16 * s, dk + (s >> 2) * (kAtomBytes >> 4) + (s & 3) * 2, idesc, s > 0);
}
__device__ __forceinline__ void issue_s_steps(int ks, uint32_t d_tmem, uint64_t dq, uint64_t dk, uint32_t idesc) {
  switch (ks) {
    case 1: issue_s<1>(d_tmem, dq, dk, idesc); break;
    case 2: issue_s<2>(d_tmem, dq, dk, idesc); break;
    case 3: issue_s<3>(d_tmem, dq, dk, idesc); break;
    case 4: issue_s<4>(d_tmem, dq, dk, idesc); break;
    case 5: issue_s<5>(d_tmem, dq, dk, idesc); break;
    case 6: issue_s<6>(d_tmem, dq, dk, idesc); break;
    case 7: issue_s<7>(d_tmem, dq, dk, idesc); break;
    default: issue_s<8>(d_tmem, dq, dk, idesc); break;
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
  const int grp_k = nch_k << 7, grp_v = nch_v << 7;
  // K'/V' tiles: atom columns of 64 rank elements, each [64 keys][128 bytes] with the 128-byte swizzle
  const int q_bytes = kTile * rpk16 * 2, k_bytes = ((rpk16 + 63) >> 6) * kAtomBytes, v_bytes = ((rpv16 + 63) >> 6) * kAtomBytes;
  const int o_bytes = kTile * rpv16 * 2;                     // an O' tile of the epilogue
  const int stage_bytes = k_bytes + v_bytes;

  unsigned char* tiles = smem + 1024;
  unsigned char* Qs = tiles;                                 // Q_A, Q_B
  unsigned char* ring = Qs + 2 * q_bytes;                    // stages x (K tile, V tile)

  // key tiles each query tile needs (tile B starts 128 rows later, so it needs two more in general)
  int n_tiles[2];
  for (int x = 0; x < 2; ++x) {
    const int tx = t0 + x * kTile;
    n_tiles[x] = tx < p.T ? (p.len0 + min(p.T, tx + kTile) + kKeys - 1) / kKeys : 0;
  }
  const int n_max_tiles = max(n_tiles[0], n_tiles[1]);
  const int active_groups = (n_tiles[0] > 0) + (n_tiles[1] > 0);
  const int total_rows = p.B * p.T;

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 512);
  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(&hdr->kv_full[s], 1);                        // the producer's arrival; the copies add their bytes
      mbar_init(&hdr->kv_empty[s], active_groups);           // one arrival per query tile that the CTA works on
    }
    mbar_init(&hdr->q_full, kSoftmaxWarps * 32);
    for (int x = 0; x < 2; ++x) {
      for (int bb = 0; bb < 2; ++bb) {
        mbar_init(&hdr->s_full[x][bb], 1);
        mbar_init(&hdr->p_full[x][bb], kTile);
        mbar_init(&hdr->o_done[x][bb], 1);
      }
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


  if (warp >= kSoftmaxWarps) {
  reg_dealloc<kRegsOther>();
  if (warp == kLoadWarp) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const unsigned char* maps = static_cast<const unsigned char*>(p.tmaps) + static_cast<size_t>(h) * 256;
      const void* map_k = maps;
      const void* map_v = maps + 128;
      tensormap_acquire(map_k);
      tensormap_acquire(map_v);
      bool ok = true;
      int stage = 0;
      uint32_t empty_parity = 1;                             // parity of "the previous use of this stage is over"
      int issued = 0;                                        // tiles whose copies have been issued
      for (int j = 0; j < n_max_tiles; ++j) {
        if (j >= stages) {
          ok = mbar_wait(&hdr->kv_empty[stage], empty_parity, p.status) && !*abort_flag;
          if (!ok) { *abort_flag = 1; break; }
        }
        unsigned char* st = ring + stage * stage_bytes;
        mbar_arrive_expect_tx(&hdr->kv_full[stage], static_cast<uint32_t>(stage_bytes));
        for (int a = 0; a * 64 < rpk16; ++a) tma_load_3d(st + a * kAtomBytes, map_k, a * 64, j * kKeys, b, &hdr->kv_full[stage]);
        for (int a = 0; a * 64 < rpv16; ++a)
          tma_load_3d(st + k_bytes + a * kAtomBytes, map_v, a * 64, j * kKeys, b, &hdr->kv_full[stage]);
        ++issued;
        if (++stage == stages) { stage = 0; empty_parity ^= 1u; }
      }
      // Every copy issued has a consumer that waits for it (the S thread).  If the CTA gives up instead, its
      // copies in flight must land before it leaves: wait (bounded) for the newest fill of every stage.
      if (!ok || *abort_flag) {
        for (int s = 0; s < stages; ++s) {
          int last = -1;                                     // newest tile whose copies went to stage s
          for (int jj = s; jj < issued; jj += stages) last = jj;
          if (last >= 0) mbar_wait(&hdr->kv_full[s], (last / stages) & 1u, p.status);
        }
      }
    }
  } else if (warp == kMmaWarp || warp == kMmaWarpB) {
    // ------------------------------------------------------------------ MMA issuers, one per query tile
    // Per key tile j: PV(j) once the group has written P(j) (into the buffer S(j + 1) came from); then, once
    // PV(j) has read P out of that buffer, S(j + 3) into it.  S(0) and S(1) go out up front, S(2) when P(0)
    // is there (the group then holds S(0) in registers).  The two issuers share nothing but the tensor pipe
    // and the ring, so neither query tile waits for the other.
    if (lane == 0) {
      const int x = warp == kMmaWarpB ? 1 : 0;
      const int nt = n_tiles[x];
      const uint32_t idesc_s = instr_desc(kKeys, false);
      const uint32_t idesc_o = instr_desc(rpv16, true);
      const uint32_t ra = smem_u32(ring);
      const uint64_t dq = smem_desc(smem_u32(Qs) + x * q_bytes, 128, grp_k);
      const uint64_t dk0 = smem_desc_sw128(ra, 16, 1024);             // K tile of stage 0 (K-major B operand)
      const uint64_t dv0 = smem_desc_sw128(ra + k_bytes, kAtomBytes, 1024);   // V tile of stage 0 (MN-major B operand)
      const uint64_t stage_step = static_cast<uint64_t>(stage_bytes >> 4);
      const uint64_t v_step = static_cast<uint64_t>(2048 >> 4);       // 16 keys = two 8-row groups of 1024 bytes
      const int ks_steps = rpk16 >> 4;
      const uint32_t tSx = tmem + x * kTile, tOx = tmem + 256 + x * kTile;
      bool ok = true;
      if (nt > 0) ok = mbar_wait(&hdr->q_full, 0, p.status);
      // ring position of the next S product's key tile
      int s_stage = 0;
      uint32_t s_parity = 0;
      auto issue_s_tile = [&](int buf) {                     // S(tile at the ring position) into S buffer `buf`
        ok = mbar_wait(&hdr->kv_full[s_stage], s_parity, p.status);
        if (!ok) return;
        tc_fence_after();
        issue_s_steps(ks_steps, tSx + buf * kKeys, dq, dk0 + s_stage * stage_step, idesc_s);
        mma_commit(&hdr->s_full[x][buf]);
        if (++s_stage == stages) { s_stage = 0; s_parity ^= 1u; }
      };
      for (int j = 0; j < min(2, nt) && ok; ++j) issue_s_tile(j);
      int stage = 0;
      for (int j = 0; j < nt && ok; ++j) {
        const int buf = j & 1;
        const uint32_t buf_parity = (j >> 1) & 1u;           // phase of tile j on the barriers of its buffer
        ok = mbar_wait(&hdr->p_full[x][buf], buf_parity, p.status) && !*abort_flag;
        if (!ok) break;
        tc_fence_after();
        if (j == 0 && nt > 2) {
          issue_s_tile(0);
          if (!ok) break;
        }
        const uint32_t tP = tSx + (buf ^ 1) * kKeys;         // P: 64 bf16 per lane in 32 columns
        const uint64_t bv = dv0 + stage * stage_step;
#pragma unroll
        for (int s = 0; s < kKeys / 16; ++s)                 // O'_x += P_x V_j over the 64 keys
          mma_ts(tOx, tP + 8 * s, bv + s * v_step, idesc_o, j > 0 || s > 0);
        mma_commit(&hdr->o_done[x][buf]);
        mma_commit(&hdr->kv_empty[stage]);                   // PV is this tile's last reader of the stage
        if (++stage == stages) stage = 0;
        if (j + 3 < nt) {
          ok = mbar_wait(&hdr->o_done[x][buf], buf_parity, p.status) && !*abort_flag;
          if (!ok) break;
          issue_s_tile(buf ^ 1);
        }
      }
      // Key tiles that only the other query tile reads still need this tile's arrival on their stage, one
      // phase at a time: wait until the previous use of the stage is over, then arrive.
      for (int j = nt; j < n_max_tiles && ok && nt > 0; ++j) {
        if (j >= stages) ok = mbar_wait(&hdr->kv_empty[j % stages], ((j / stages) - 1) & 1u, p.status) && !*abort_flag;
        if (ok) mbar_arrive(&hdr->kv_empty[j % stages]);
      }
      // the last commits' arrivals must have landed before the CTA may leave
      if (ok && nt > 0) ok = mbar_wait(&hdr->kv_empty[(n_max_tiles - 1) % stages], ((n_max_tiles - 1) / stages) & 1u, p.status);
      if (!ok) *abort_flag = 1;
    }
  }

  // ---- MMA and loader warps: epilogue
  tc_fence_before();
  __syncthreads();                                           // #1
  const bool lowrank = (p.flags & 0x2u) != 0;
  const bool run = !*abort_flag && !lowrank;
  unsigned char* Uh = tiles + 4 * o_bytes;                   // lift image of U^V: [d_head][rpv16] hi, then lo
  const int img16 = p.d_head * rpv16 * 2 / 16;               // 16-byte words per image
  if (run) {
    const uint4* Ug = reinterpret_cast<const uint4*>(p.basis + hd.uvl16_off);
    for (int idx = tid - kMmaWarp * 32; idx < 2 * img16; idx += kWsThreads - kSoftmaxWarps * 32)
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
      const uint32_t oh = smem_u32(tiles + x * 2 * o_bytes), ol = oh + o_bytes;
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
  return;
  }

  reg_alloc<kRegsSoftmax>();
  {
    // ------------------------------------------------------------------ softmax warpgroups
    const int x = warp >> 2;                                 // 0 = tile A, 1 = tile B
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + x * kTile;        // S buffers at +0 and +64
    const uint32_t tO = tmem + lane_base + 256 + x * kTile;
    const int tx = t0 + x * kTile;
    const int my_pos = p.len0 + tx + row;                    // last key this thread's query sees
    {                                                        // this group's Q' tile (zeros past the prompt's end)
      const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.qp) +
                                static_cast<int64_t>(hd.lr_k_off) * total_rows + static_cast<int64_t>(b) * p.T * hd.rp_k;
      const int q_rows = max(0, min(kTile, p.T - tx));
      load_q_tile_async(Qs + x * q_bytes, q_rows > 0 ? Qg + static_cast<int64_t>(tx) * hd.rp_k : Qg, hd.rp_k, q_rows,
                        nch_k, row);
      cp_async_commit();
      cp_async_wait<0>();
      fence_async_smem();
      mbar_arrive(&hdr->q_full);
    }
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    const int nt = n_tiles[x];
    // One key tile: `cur` holds this thread's row of S(j); the row of S(j + 1) is requested into `nxt` before
    // the arithmetic starts and awaited before P(j) goes out over the buffer it came from.
    auto tile = [&](const uint32_t (&cur)[64], uint32_t (&nxt)[64], int j) {
      const int key0 = j * kKeys, buf = j & 1;
      const bool has_next = j + 1 < nt;
      if (has_next) {
        ok = mbar_wait(&hdr->s_full[x][buf ^ 1], ((j + 1) >> 1) & 1u, p.status);
        ok = __all_sync(0xffffffffu, ok && !*abort_flag);    // one decision for the whole warp
        if (!ok) return;
        tc_fence_after();
        tmem_ld64(tS + (buf ^ 1) * kKeys, nxt);
      }
      const uint32_t tP = tS + (buf ^ 1) * kKeys;            // P(j) goes where S(j + 1) was
      const bool diag = key0 + kKeys - 1 > p.len0 + tx;      // some (row, key) pair of the tile is masked
      // Lazy reference: the exponentials use m_run, which follows the true maximum only when that has grown
      // by more than 8 (a factor 256 that fp32 sums and bf16 P absorb); O' is rescaled only then.
      float alpha = 1.f, row_sum;
      uint32_t pk[32];
      if (j == 0 || diag) {                                  // maximum first, then the exponentials
        float row_max = -INFINITY;
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (!diag || key0 + i <= my_pos) row_max = fmaxf(row_max, __uint_as_float(cur[i]));
        row_max *= p.scale_log2;                             // the scale is positive: max and scale commute
        if (row_max > m_run + 8.f) {
          alpha = ex2(m_run - row_max);
          m_run = row_max;
        }
        row_sum = diag ? exp_row<true, false>(cur, p.scale_log2, -m_run, key0, my_pos, pk, nullptr)
                       : exp_row<false, false>(cur, p.scale_log2, -m_run, key0, my_pos, pk, nullptr);
      } else {                                               // exponentials against the old reference, maximum on the side
        float raw_max;
        row_sum = exp_row<false, true>(cur, p.scale_log2, -m_run, key0, my_pos, pk, &raw_max);
        const float row_max = raw_max * p.scale_log2;
        if (__any_sync(0xffffffffu, row_max > m_run + 8.f)) { // the reference moved for some row: once more
          if (row_max > m_run + 8.f) {
            alpha = ex2(m_run - row_max);
            m_run = row_max;
          }
          row_sum = exp_row<false, false>(cur, p.scale_log2, -m_run, key0, my_pos, pk, nullptr);
        }
      }
      if (has_next) {
        tmem_wait_ld();                                      // S(j + 1) is in registers: its buffer may take P(j)
      } else if (j >= 2) {                                   // no S(j + 1) whose arrival implies it: PV_x(j-2) has read P(j-2)
        ok = mbar_wait(&hdr->o_done[x][buf], ((j - 2) >> 1) & 1u, p.status);
        ok = __all_sync(0xffffffffu, ok && !*abort_flag);
        if (!ok) return;
        tc_fence_after();
      }
      tmem_st16(tP, *reinterpret_cast<const uint32_t(*)[16]>(&pk[0]));
      tmem_st16(tP + 16, *reinterpret_cast<const uint32_t(*)[16]>(&pk[16]));
      l_run = l_run * alpha + row_sum;
      if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {  // rescale this row of O' (rare after the first tiles)
        ok = mbar_wait(&hdr->o_done[x][buf ^ 1], ((j - 1) >> 1) & 1u, p.status);   // PV_x(j-1) has added to O'
        ok = __all_sync(0xffffffffu, ok && !*abort_flag);
        if (!ok) return;
        tc_fence_after();
#pragma unroll 1
        for (int h0 = 0; h0 < rpv16; h0 += 16) {
          uint32_t o[16];
          tmem_ld16(tO + h0, o);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
          tmem_st16(tO + h0, o);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&hdr->p_full[x][buf]);
    };
    {
      uint32_t ra[64], rb[64];
      if (nt > 0) {
        ok = mbar_wait(&hdr->s_full[x][0], 0, p.status);
        ok = __all_sync(0xffffffffu, ok && !*abort_flag);
        if (ok) {
          tc_fence_after();
          tmem_ld64(tS, ra);
          tmem_wait_ld();
        }
      }
      for (int j = 0; j < nt && ok; j += 2) {
        tile(ra, rb, j);
        if (ok && j + 1 < nt) tile(rb, ra, j + 1);
      }
    }
    if (ok && n_tiles[x] > 0) {
      ok = mbar_wait(&hdr->o_done[x][(n_tiles[x] - 1) & 1], ((n_tiles[x] - 1) >> 1) & 1u, p.status);
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
    unsigned char* Oh = tiles + x * 2 * o_bytes;             // O' hi and lo of this tile, [128][rpv16] each
    unsigned char* Ol = Oh + o_bytes;
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
  }
}

}  // namespace

// Stages of the K'/V' ring that fit beside the two Q tiles (0 = does not fit).
int prefill_tc_ws_stages(int max_rp_k, int max_rp_v, int d_head, size_t* smem_bytes) {
  const size_t k16 = (max_rp_k + 15) & ~15, v16 = (max_rp_v + 15) & ~15;
  const size_t fixed = 1024 + 2 * kTile * k16 * 2;
  const size_t stage = (((k16 + 63) >> 6) + ((v16 + 63) >> 6)) * static_cast<size_t>(kAtomBytes);
  const size_t limit = 227 * 1024;
  int stages = 0;
  for (int s = kMaxStages; s >= 3; --s)   // the S products run three key tiles ahead of the PV products
    if (fixed + s * stage <= limit) { stages = s; break; }
  if (stages == 0) return 0;
  const size_t total = fixed + stages * stage;
  const size_t epilogue = 1024 + 4 * kTile * v16 * 2 + 2 * static_cast<size_t>(d_head) * v16 * 2;
  if (epilogue > total) return 0;
  *smem_bytes = total;
  return stages;
}

cudaError_t launch_prefill_tc_ws(const PrefillParams& p, int stages, size_t smem, cudaStream_t s, uint64_t* launches) {
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(prefill_tc_ws_kernel, smem, configured);
  if (ec != cudaSuccess) return ec;
  dim3 grid(p.B * p.H, (p.T + 2 * kTile - 1) / (2 * kTile));
  prefill_tc_ws_kernel<<<grid, kWsThreads, smem, s>>>(p, stages);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
