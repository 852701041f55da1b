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
//   * two threads feed the tensor pipe, one per query tile.  S is double-buffered in TMEM (2 x 64
//     columns per query tile): S(j + 1) is computed while the softmax works on S(j).  Per key tile j the
//     issuer waits for P(j), issues O' += P(j) V'(j), and once that product has read P(j) issues S(j + 2)
//     into the buffer P(j) occupied; every group of MMAs is followed by a tcgen05.commit onto the
//     mbarrier its consumer waits on;
//   * sixteen softmax warps, four per scheduler, so that the fixed latencies of one warp's instruction
//     stream are covered by the others.  A query tile has two warpgroups: a thread owns one query row
//     (= one TMEM lane) and one half of the tile's 64 keys.  Per key tile it loads its 32 scores, takes
//     their maximum, agrees with the other half of its row on the softmax reference through one
//     reducing barrier (the reference moves only when some row's maximum grew by more than 8 in the
//     log2 domain; only then do the halves exchange maxima through shared memory and rescale O'),
//     computes 32 exponentials and writes P (bf16) IN PLACE over the first 32 columns of the S buffer,
//     from where it is the A operand of the PV product: P never touches shared memory.
//     The ALiBi bias (per-head slope) is added to the scaled scores in a second instantiation.
// TMEM (512 columns): S_A[2], S_B[2] (64 columns each, P aliased), O'_A, O'_B (up to 128 each).
// Every wait is bounded.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kKeys = 64;                     // key rows per tile
constexpr int kHalfKeys = kKeys / 2;          // keys per softmax thread and tile
constexpr int kAtomBytes = kKeys * 128;       // one swizzled atom column of a K'/V' tile: 64 rows x 64 elements
constexpr int kSoftmaxWarps = 16;             // warpgroups 0,1: query tile A (keys 0..31, 32..63); 2,3: tile B
constexpr int kMmaWarp = 16;                  // issues the MMAs of query tile A (and the lift)
constexpr int kLoadWarp = 17;                 // lane 0 issues the TMA copies
constexpr int kMmaWarpB = 18;                 // issues the MMAs of query tile B
constexpr int kWsThreads = 20 * 32;           // 16 softmax warps, two MMA issuers, TMA producer, one spare warp
// Registers per thread after the reallocation: the CTA is launched with 640 x 96; the last warpgroup keeps 40,
// the softmax warpgroups take 104: 128 x 40 + 512 x 104 = 58 368 <= 61 440.
constexpr int kRegsSoftmax = 104, kRegsOther = 40;
static_assert(128 * kRegsOther + 512 * kRegsSoftmax <= kWsThreads * 96, "register split exceeds the launch");
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
  float exch[2][2][kTile];                    // [query tile][half][row]: row maxima (main loop), row sums (epilogue)
};
static_assert(sizeof(WsHeader) <= 3072, "header outgrew its area");
constexpr int kHeaderBytes = 3072;            // tiles start here (1024-byte aligned for the swizzled layout)

// One thread's share of a canonical (no swizzle) Q' tile of 128 rows, loaded by the 256 threads of a query tile:
// 16-byte chunks (row, c); two neighbouring lanes fetch the two halves of a 32-byte piece of a row.
__device__ __forceinline__ void load_q_tile_async(unsigned char* dst, const __nv_bfloat16* src, int rp, int rows_valid,
                                                  int nch, int t) {
  const int src_chunks = rp >> 3;
  const int group_stride = nch << 7;
  for (int idx = t; idx < kTile * nch; idx += 2 * kTile) {
    const int c = ((idx / (2 * kTile)) << 1) + (idx & 1), row = (idx >> 1) & (kTile - 1);
    const bool live = row < rows_valid && c < src_chunks;
    const void* g = live ? static_cast<const void*>(src + static_cast<int64_t>(row) * rp + c * 8) : src;
    cp_async16(dst + chunk_off(row, c, group_stride), g, live ? 16u : 0u);
  }
}

// Barrier of the 256 softmax threads of one query tile that also ORs a predicate over them.
__device__ __forceinline__ bool tile_barrier_or(int id, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, %2, 256, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out)
      : "r"(pred ? 1u : 0u), "r"(id)
      : "memory");
  return out != 0;
}
__device__ __forceinline__ void tile_barrier(int id) { asm volatile("bar.sync %0, 256;" ::"r"(id) : "memory"); }

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

template <bool ALIBI>
__global__ void __launch_bounds__(kWsThreads, 1) prefill_tc_ws_kernel(const PrefillParams p, int stages) {
  extern __shared__ __align__(1024) unsigned char smem[];
  WsHeader* hdr = reinterpret_cast<WsHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int unit = blockIdx.x;
  const int h = unit / p.B, b = unit - h * p.B;
  const HeadInfo hd = p.heads[h];
  const int qblk = gridDim.y - 1 - blockIdx.y;              // late (long) query blocks first
  const int len0 = p.len0 - (p.deficit != nullptr ? __ldg(p.deficit + b) : 0);   // rows this sequence held before the call
  const int t0 = qblk * 2 * kTile;
  // width and place of this head's query and key rows: the rank-r rows, or the override of the rotary prompt path
  const int rp_k = p.k_width ? p.k_width : hd.rp_k;
  const int q_off = p.k_width ? h * p.k_width : hd.lr_k_off;
  const int rpk16 = (rp_k + 15) & ~15, rpv16 = (hd.rp_v + 15) & ~15;
  const int nch_k = rpk16 >> 3, nch_v = rpv16 >> 3;
  const int grp_k = nch_k << 7, grp_v = nch_v << 7;
  // K'/V' tiles: atom columns of 64 rank elements, each [64 keys][128 bytes] with the 128-byte swizzle
  const int q_bytes = kTile * rpk16 * 2, k_bytes = ((rpk16 + 63) >> 6) * kAtomBytes, v_bytes = ((rpv16 + 63) >> 6) * kAtomBytes;
  const int o_bytes = kTile * rpv16 * 2;                     // an O' tile of the epilogue
  const int stage_bytes = k_bytes + v_bytes;

  unsigned char* tiles = smem + kHeaderBytes;
  unsigned char* Qs = tiles;                                 // Q_A, Q_B
  unsigned char* ring = Qs + 2 * q_bytes;                    // stages x (K tile, V tile)

  // key tiles each query tile needs (tile B starts 128 rows later, so it needs two more in general)
  int n_tiles[2];
  for (int x = 0; x < 2; ++x) {
    const int tx = t0 + x * kTile;
    n_tiles[x] = tx < p.T ? (len0 + min(p.T, tx + kTile) + kKeys - 1) / kKeys : 0;
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
        mbar_init(&hdr->p_full[x][bb], 2 * kTile);           // both halves of every row
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
      const void* map_k = p.tmaps_k ? static_cast<const void*>(static_cast<const unsigned char*>(p.tmaps_k) + static_cast<size_t>(h) * 128)
                                    : static_cast<const void*>(maps);
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
    // S(0) and S(1) go out up front.  Per key tile j: O' += P(j) V'(j) once both halves of every row have
    // written P(j) over S(j); then, once that product has read P(j), S(j + 2) into the same buffer.  The two
    // issuers share nothing but the tensor pipe and the ring, so neither query tile waits for the other.
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
        const uint32_t tP = tSx + buf * kKeys;               // P(j): 64 bf16 per lane in the first 32 columns of S(j)
        const uint64_t bv = dv0 + stage * stage_step;
#pragma unroll
        for (int s = 0; s < kKeys / 16; ++s)                 // O'_x += P_x V_j over the 64 keys
          mma_ts(tOx, tP + 8 * s, bv + s * v_step, idesc_o, j > 0 || s > 0);
        mma_commit(&hdr->o_done[x][buf]);
        mma_commit(&hdr->kv_empty[stage]);                   // PV is this tile's last reader of the stage
        if (++stage == stages) stage = 0;
        if (j + 2 < nt) {
          ok = mbar_wait(&hdr->o_done[x][buf], buf_parity, p.status) && !*abort_flag;
          if (!ok) break;
          issue_s_tile(buf);
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
    for (int idx = tid - kSoftmaxWarps * 32; idx < 2 * img16; idx += kWsThreads - kSoftmaxWarps * 32)
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
    const int x = warp >> 3;                                 // 0 = tile A, 1 = tile B
    const int hf = (warp >> 2) & 1;                          // which half of a tile's 64 keys
    const int row = (warp & 3) * 32 + lane;
    const int bar_id = 1 + x;                                // named barrier of this query tile's 256 threads
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + x * kTile;        // S buffers at +0 and +64
    const uint32_t tO = tmem + lane_base + 256 + x * kTile;
    const int tx = t0 + x * kTile;
    const int my_pos = len0 + tx + row;                    // last key this thread's query sees
    {                                                        // this tile's Q' (zeros past the prompt's end)
      const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.qp) +
                                static_cast<int64_t>(q_off) * total_rows + static_cast<int64_t>(b) * p.T * rp_k;
      const int q_rows = max(0, min(kTile, p.T - tx));
      load_q_tile_async(Qs + x * q_bytes, q_rows > 0 ? Qg + static_cast<int64_t>(tx) * rp_k : Qg, rp_k, q_rows,
                        nch_k, hf * kTile + row);
      cp_async_commit();
      cp_async_wait<0>();
      fence_async_smem();
      mbar_arrive(&hdr->q_full);
    }
    // columns of O' (and of the lifted output) each half of a row looks after in the rescale and the epilogue
    const int o_split = ((rpv16 >> 4) + 1) / 2 * 16;
    const int o_lo = hf ? o_split : 0, o_hi = hf ? rpv16 : o_split;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    const int nt = n_tiles[x];
    const float slope2 = ALIBI ? hd.alibi_slope2 : 0.f;

    // The 256 threads of a query tile meet at named barriers, which have no time limit: every decision to leave
    // the loop is therefore taken through a reducing barrier, so that all of them leave after the same tile.
    for (int j = 0; j < nt; ++j) {
      const int buf = j & 1;
      const int key0 = j * kKeys + hf * kHalfKeys;           // first key of this thread's half
      const uint32_t tSb = tS + buf * kKeys;
      const bool waited = mbar_wait(&hdr->s_full[x][buf], (j >> 1) & 1u, p.status);
      const bool diag = j * kKeys + kKeys - 1 > len0 + tx; // some (row, key) pair of the tile is masked
      uint32_t r[kHalfKeys];
      float cand = -INFINITY;                                // this half-row's largest score, scaled (log2 domain)
      if (waited) {
        tc_fence_after();
        tmem_ld16(tSb + hf * kHalfKeys, *reinterpret_cast<uint32_t(*)[16]>(&r[0]));
        tmem_ld16(tSb + hf * kHalfKeys + 16, *reinterpret_cast<uint32_t(*)[16]>(&r[16]));
        tmem_wait_ld();
        if (ALIBI) {
          // scaled score plus the bias slope * (key - position), kept in place of the raw score
          float off = slope2 * static_cast<float>(key0 - my_pos);
#pragma unroll
          for (int c = 0; c < kHalfKeys; ++c) {
            r[c] = __float_as_uint(fmaf(__uint_as_float(r[c]), p.scale_log2, off));
            off += slope2;
          }
        }
        if (diag) {
#pragma unroll
          for (int c = 0; c < kHalfKeys; ++c)
            if (key0 + c <= my_pos) cand = fmaxf(cand, __uint_as_float(r[c]));
        } else {
          float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
          for (int c = 0; c < kHalfKeys; c += 4) {
            mx0 = max3(mx0, __uint_as_float(r[c]), __uint_as_float(r[c + 1]));
            mx1 = max3(mx1, __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
          }
          cand = fmaxf(mx0, mx1);
        }
        if (!ALIBI) cand *= p.scale_log2;                    // the scale is positive: max and scale commute
      }
      // Lazy reference: it follows the row maximum only when that has grown by more than 8 (a factor 256 that
      // fp32 sums and bf16 P absorb).  One reducing barrier tells whether any row of the tile needs it; it also
      // orders the other half's loads of S before this half's stores of P into the same columns.
      float alpha = 1.f;
      if (tile_barrier_or(bar_id, !waited || cand > m_run + 8.f || *abort_flag != 0)) {
        hdr->exch[x][hf][row] = cand;
        if (tile_barrier_or(bar_id, !waited || *abort_flag != 0)) {   // a wait gave up somewhere: all 256 leave here
          ok = false;
          break;
        }
        const float row_max = fmaxf(cand, hdr->exch[x][hf ^ 1][row]);  // both halves take the same decision
        if (row_max > m_run + 8.f) {
          alpha = ex2(m_run - row_max);
          m_run = row_max;
        }
        l_run *= alpha;
        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {          // rescale this half's columns of the row of O'
          const bool got = mbar_wait(&hdr->o_done[x][buf ^ 1], ((j - 1) >> 1) & 1u, p.status);   // PV(j-1) has added to O'
          if (__all_sync(0xffffffffu, got)) {
            tc_fence_after();
#pragma unroll 1
            for (int h0 = o_lo; h0 < o_hi; h0 += 16) {
              uint32_t o[16];
              tmem_ld16(tO + h0, o);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              tmem_st16(tO + h0, o);
            }
          } else {
            *abort_flag = 1;                                 // seen by every thread of the tile at the next barrier
          }
        }
      }
      // exponentials against the reference, their sum, P as bf16 pairs
      uint32_t pk[kHalfKeys / 2];
      float sum0 = 0.f, sum1 = 0.f;
      const float neg_m = -m_run;
#pragma unroll
      for (int i = 0; i < kHalfKeys / 2; ++i) {
        const int c = 2 * i;
        float y0, y1;
        if (ALIBI) {
          y0 = __uint_as_float(r[c]) + neg_m;
          y1 = __uint_as_float(r[c + 1]) + neg_m;
        } else {
          fma2(y0, y1, __uint_as_float(r[c]), __uint_as_float(r[c + 1]), p.scale_log2, neg_m);
        }
        float e0 = ex2(y0), e1 = ex2(y1);
        if (diag) {
          if (key0 + c > my_pos) e0 = 0.f;
          if (key0 + c + 1 > my_pos) e1 = 0.f;
        }
        add2(sum0, sum1, e0, e1);
        pk[i] = pack_bf16(e0, e1);
      }
      l_run += sum0 + sum1;
      tmem_st16(tSb + hf * (kHalfKeys / 2), pk);             // in place: P(j) takes the first 32 columns of S(j)
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&hdr->p_full[x][buf]);
    }
    if (ok && nt > 0) {
      ok = mbar_wait(&hdr->o_done[x][(nt - 1) & 1], ((nt - 1) >> 1) & 1u, p.status);
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
    }
    if (!ok) *abort_flag = 1;
    hdr->exch[x][hf][row] = l_run;                           // the two halves' sums share the reference

    // ---- epilogue part 1 (after every role is done with the main loop)
    tc_fence_before();
    __syncthreads();                                         // #1
    const bool run = !*abort_flag && n_tiles[x] > 0;
    const float inv_l = 1.f / (hdr->exch[x][0][row] + hdr->exch[x][1][row]);
    const bool lowrank = (p.flags & 0x2u) != 0;
    const int q_valid = min(kTile, p.T - tx);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.out);
    unsigned char* Oh = tiles + x * 2 * o_bytes;             // O' hi and lo of this tile, [128][rpv16] each
    unsigned char* Ol = Oh + o_bytes;
    if (run) {
      tc_fence_after();
      __nv_bfloat16* dst_lr = out + b * p.out_stride_b + static_cast<int64_t>(tx + row) * p.out_stride_t + hd.lr_v_off;
      for (int c0 = o_lo; c0 < o_hi; c0 += 16) {             // this half's columns of the row
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
        const int d_split = ((p.d_head >> 4) + 1) / 2 * 16;  // this half's share of the d_head output columns
        const int d_lo = hf ? d_split : 0, d_hi = hf ? p.d_head : d_split;
        for (int c0 = d_lo; c0 < d_hi; c0 += 16) {
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
  const size_t fixed = kHeaderBytes + 2 * kTile * k16 * 2;
  const size_t stage = (((k16 + 63) >> 6) + ((v16 + 63) >> 6)) * static_cast<size_t>(kAtomBytes);
  const size_t limit = 227 * 1024;
  int stages = 0;
  for (int s = kMaxStages; s >= 3; --s)   // the S products run two key tiles ahead of the PV products
    if (fixed + s * stage <= limit) { stages = s; break; }
  if (stages == 0) return 0;
  const size_t total = fixed + stages * stage;
  const size_t epilogue = kHeaderBytes + 4 * kTile * v16 * 2 + 2 * static_cast<size_t>(d_head) * v16 * 2;
  if (epilogue > total) return 0;
  *smem_bytes = total;
  return stages;
}

cudaError_t launch_prefill_tc_ws(const PrefillParams& p, int stages, size_t smem, bool alibi, cudaStream_t s,
                                 uint64_t* launches) {
  static size_t configured[2][kMaxDevices] = {};
  const cudaError_t ec = alibi ? ensure_dynamic_smem(prefill_tc_ws_kernel<true>, smem, configured[1])
                               : ensure_dynamic_smem(prefill_tc_ws_kernel<false>, smem, configured[0]);
  if (ec != cudaSuccess) return ec;
  dim3 grid(p.B * p.H, (p.T + 2 * kTile - 1) / (2 * kTile));
  if (alibi) prefill_tc_ws_kernel<true><<<grid, kWsThreads, smem, s>>>(p, stages);
  else prefill_tc_ws_kernel<false><<<grid, kWsThreads, smem, s>>>(p, stages);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
