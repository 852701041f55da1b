// Prefill-side projections as one persistent, pipelined tensor-core kernel (tcgen05 + TMA):
//   Q' = Q U^K,  K' = K U^K,  V' = V U^V        (the r-wide factors of Eq. 6 of the paper)
// Same arithmetic as project_tc_kernel (token rows = bf16 A operand, fp32 basis = B operand split into bf16
// high + low parts, two products accumulated in fp32), different schedule.  The work items are
// (head, which of Q/K/V, tile of 128 tokens of one sequence), laid end to end with the tiles of one
// (head, which) pair adjacent; each CTA (one per SM) owns a contiguous range of them, so the basis images stay
// in shared memory for a whole run of tiles instead of being fetched again per tile.
//   warp 0, one thread: TMA producer.  A token tile arrives as two boxes of 64 elements x 128 rows in the
//     128-byte swizzled layout (tensor maps of q, k, v are kernel parameters, encoded by the host per call);
//     rows past T arrive as zeros.  The basis images come as one bulk copy when the basis changes.
//   warp 1, one thread: MMA issuer, accumulators double-buffered in TMEM.
//   warps 2-5: epilogue, one thread per token row: TMEM -> bf16 -> an output tile in shared memory; the rows of a
//     tile are adjacent in the cache slab (K', V') or the Q' scratch, so the tile leaves as one bulk store.
// The loads of the next tiles, the products of this one and the stores of the previous one overlap.
#include <cuda.h>   // CUtensorMap only
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

constexpr int kPsThreads = 192;
constexpr int kPsMaxStages = 4;
constexpr int kAtomBytesA = kTile * 128;        // one atom column of the token tile: 128 rows of 128 bytes

// Shared -> global bulk copy (both 16-byte aligned, size a multiple of 16) in this thread's bulk group.
__device__ __forceinline__ void bulk_store(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>                                // at most N of this thread's groups still read their source
__device__ __forceinline__ void bulk_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); }
// Barrier of the 128 epilogue threads that also tells each of them whether `ok` held for all.
__device__ __forceinline__ bool epilogue_sync_all(bool ok) {
  uint32_t all;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "barrier.red.and.pred q, 2, 128, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(all)
      : "r"(ok ? 1u : 0u)
      : "memory");
  return all != 0;
}

struct PsHeader {
  unsigned long long x_full[kPsMaxStages];
  unsigned long long x_empty[kPsMaxStages];
  unsigned long long acc_full[2];
  unsigned long long acc_empty[2];
  unsigned long long u_full;
  uint32_t tmem_base;
  int abort_flag;
};

// Position in the flat order of work items (pair = head * 3 + which, then sequence, then tile of the sequence);
// set up with divisions once per CTA and role, advanced by increments.
struct PsItem {
  int h, which, b, tt;      // which: 0 = Q, 1 = K, 2 = V; tt: tile of the sequence
  __device__ __forceinline__ void init(int64_t w, int tiles, int tps) {
    const int pair = static_cast<int>(w / tiles);
    const int tile = static_cast<int>(w - static_cast<int64_t>(pair) * tiles);
    h = pair / 3;
    which = pair - h * 3;
    b = tile / tps;
    tt = tile - b * tps;
  }
  __device__ __forceinline__ void next(int B, int tps) {
    if (++tt == tps) {
      tt = 0;
      if (++b == B) {
        b = 0;
        if (++which == 3) { which = 0; ++h; }
      }
    }
  }
};

template <int KS>               // contraction steps of 16 elements: d_head / 16 (4 or 8)
__global__ void __launch_bounds__(kPsThreads, 1)
project_tc_stream_kernel(const ProjectTcParams p, const __grid_constant__ CUtensorMap map_q,
                         const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                         int stages, uint32_t ncols, int u_bytes_max, int o_bytes_max) {
  extern __shared__ __align__(1024) unsigned char smem[];
  PsHeader* hdr = reinterpret_cast<PsHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tps = (p.T + kTile - 1) / kTile;                 // tiles per sequence
  const int tiles = p.B * tps;
  const int64_t total = 3ll * p.H * tiles;
  const int64_t w_begin = total * blockIdx.x / gridDim.x, w_end = total * (blockIdx.x + 1) / gridDim.x;
  const int n_items = static_cast<int>(w_end - w_begin);
  const int atoms = p.d_head >> 6;                           // 64-element atom columns per token row
  const int x_bytes = atoms * kAtomBytesA;
  const int grp_d = (p.d_head >> 3) << 7;                    // bytes per 8-row group of a canonical basis image

  unsigned char* Xring = smem + 1024;                        // stages x [atoms][128 rows][128 bytes], swizzled
  unsigned char* Us = Xring + stages * x_bytes;              // basis image, high part then low part

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 2 * ncols);
  if (tid == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(&hdr->x_full[s], 1);
      mbar_init(&hdr->x_empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&hdr->acc_full[a], 1);
      mbar_init(&hdr->acc_empty[a], kTile);
    }
    mbar_init(&hdr->u_full, 1);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  volatile int* abort_flag = &hdr->abort_flag;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && n_items > 0) {
      uint64_t keep;                                         // the images are read again by later CTAs and calls
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
      bool ok = true;
      int stage = 0, issued = 0;
      uint32_t empty_parity = 1;                             // parity of "the previous use of this stage is over"
      int prev_stage = 0;
      uint32_t prev_parity = 0;                              // phase in which the previous tile's stage is released
      int cur_h = -1, cur_v = -1, u_loads = 0;
      PsItem it;
      it.init(w_begin, tiles, tps);
      for (int i = 0; i < n_items; ++i, it.next(p.B, tps)) {
        const int is_v = it.which == 2;
        if (it.h != cur_h || is_v != cur_v) {
          // the products of every earlier tile have read the old image once the newest tile's stage is released
          if (i > 0) {
            ok = mbar_wait(&hdr->x_empty[prev_stage], prev_parity, p.status) && !*abort_flag;
            if (!ok) break;
          }
          const HeadInfo hd = p.heads[it.h];
          const int rp16 = ((is_v ? hd.rp_v : hd.rp_k) + 15) & ~15;
          const uint32_t u_bytes = static_cast<uint32_t>(2 * rp16 * p.d_head * 2);
          mbar_arrive_expect_tx(&hdr->u_full, u_bytes);
          bulk_load(Us, p.basis + (is_v ? hd.uvt16_off : hd.ukt16_off), u_bytes, &hdr->u_full, keep);
          ++u_loads;
          cur_h = it.h;
          cur_v = is_v;
        }
        if (i >= stages) {
          ok = mbar_wait(&hdr->x_empty[stage], empty_parity, p.status) && !*abort_flag;
          if (!ok) break;
        }
        const CUtensorMap* map = it.which == 0 ? &map_q : (it.which == 1 ? &map_k : &map_v);
        unsigned char* st = Xring + stage * x_bytes;
        mbar_arrive_expect_tx(&hdr->x_full[stage], static_cast<uint32_t>(x_bytes));
        for (int a = 0; a < atoms; ++a)
          tma_load_3d(st + a * kAtomBytesA, map, it.h * p.d_head + a * 64, it.tt * kTile, it.b, &hdr->x_full[stage]);
        ++issued;
        prev_stage = stage;
        prev_parity = empty_parity ^ 1u;
        if (++stage == stages) { stage = 0; empty_parity ^= 1u; }
      }
      // If the CTA gives up, its copies in flight must land before it leaves: wait (bounded) for the newest
      // fill of every stage and for the basis image.
      if (!ok || *abort_flag) {
        *abort_flag = 1;
        for (int s = 0; s < stages; ++s) {
          int last = -1;
          for (int jj = s; jj < issued; jj += stages) last = jj;
          if (last >= 0) mbar_wait(&hdr->x_full[s], (last / stages) & 1u, p.status);
        }
        if (u_loads > 0) mbar_wait(&hdr->u_full, (u_loads - 1) & 1u, p.status);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n_items > 0) {
      bool ok = true;
      int stage = 0;
      uint32_t full_parity = 0, u_parity = 0;
      int cur_h = -1, cur_v = -1;
      // descriptors of stage 0 / the high image; a step, a stage or the low image only moves the start address
      const uint64_t a0 = smem_desc_sw128(smem_u32(Xring), 16, 1024);
      const uint64_t b0 = smem_desc(smem_u32(Us), 128, grp_d);
      const uint64_t stage_step = static_cast<uint64_t>(x_bytes >> 4);
      uint64_t lo_step = 0;                                  // from the high to the low image of the current basis
      uint32_t idesc = 0;
      PsItem it;
      it.init(w_begin, tiles, tps);
      for (int i = 0; i < n_items && ok; ++i, it.next(p.B, tps)) {
        const int is_v = it.which == 2;
        if (it.h != cur_h || is_v != cur_v) {
          ok = mbar_wait(&hdr->u_full, u_parity, p.status) && !*abort_flag;
          if (!ok) break;
          u_parity ^= 1u;
          const HeadInfo hd = p.heads[it.h];
          const int rp16 = ((is_v ? hd.rp_v : hd.rp_k) + 15) & ~15;
          idesc = instr_desc(rp16, false);
          lo_step = static_cast<uint64_t>((rp16 * p.d_head * 2) >> 4);
          cur_h = it.h;
          cur_v = is_v;
        }
        const int acc = i & 1;
        if (i >= 2) {
          ok = mbar_wait(&hdr->acc_empty[acc], ((i >> 1) - 1) & 1u, p.status) && !*abort_flag;
          if (!ok) break;
        }
        ok = mbar_wait(&hdr->x_full[stage], full_parity, p.status) && !*abort_flag;
        if (!ok) break;
        tc_fence_after();
        const uint64_t a_st = a0 + stage * stage_step;
        const uint32_t d_tmem = tmem + acc * ncols;
#pragma unroll
        for (int s = 0; s < KS; ++s)                         // contraction over d_head, 16 elements per step
          mma_ss(d_tmem, a_st + ((s >> 2) * (kAtomBytesA >> 4) + (s & 3) * 2), b0 + s * 16, idesc, s > 0);
#pragma unroll
        for (int s = 0; s < KS; ++s)                         // the low part of the basis on top
          mma_ss(d_tmem, a_st + ((s >> 2) * (kAtomBytesA >> 4) + (s & 3) * 2), b0 + lo_step + s * 16, idesc, true);
        mma_commit(&hdr->x_empty[stage]);                    // the tile (and the image) have been read
        mma_commit(&hdr->acc_full[acc]);
        if (++stage == stages) { stage = 0; full_parity ^= 1u; }
      }
      if (!ok) *abort_flag = 1;
    }
  } else {
    // ------------------------------------------------------------------ epilogue, thread = token row
    const int quarter = warp & 3;                            // the TMEM lanes this warp may read
    const int row = quarter * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
    const int64_t total_rows = static_cast<int64_t>(p.B) * p.T;
    const bool issuer = warp == 2 && lane == 0;              // the thread that sends the finished tiles out
    unsigned char* Obuf = Us + u_bytes_max;                  // two output tiles, [128 rows][rp] bf16 each
    bool ok = true;
    PsItem it;
    it.init(w_begin, tiles, tps);
    for (int i = 0; i < n_items; ++i, it.next(p.B, tps)) {
      const HeadInfo hd = p.heads[it.h];
      const bool is_v = it.which == 2;
      const int rp = is_v ? hd.rp_v : hd.rp_k;
      const int rp16 = (rp + 15) & ~15;
      const int acc = i & 1;
      ok = mbar_wait(&hdr->acc_full[acc], (i >> 1) & 1u, p.status) && !*abort_flag;
      // The rows of a tile are adjacent in the destination (rows t0.. of one sequence in a slab or in the Q'
      // scratch), so the tile is put together in shared memory and leaves as one bulk store.  The buffer of
      // tile i served tile i - 2: its store must have read the buffer before anyone writes there again.
      unsigned char* ob = Obuf + acc * o_bytes_max;
      if (issuer) bulk_store_wait_read<1>();
      ok = epilogue_sync_all(ok);                            // one decision for the whole group: nobody is left at a barrier
      if (!ok) break;
      tc_fence_after();
      const uint32_t src = tmem + acc * ncols + lane_base;
      unsigned char* orow = ob + row * rp * 2;
      for (int c0 = 0; c0 < rp16; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(src + c0, v);
        tmem_wait_ld();
        uint4 w0, w1;
        w0.x = pack_bf16(__uint_as_float(v[0]), __uint_as_float(v[1]));
        w0.y = pack_bf16(__uint_as_float(v[2]), __uint_as_float(v[3]));
        w0.z = pack_bf16(__uint_as_float(v[4]), __uint_as_float(v[5]));
        w0.w = pack_bf16(__uint_as_float(v[6]), __uint_as_float(v[7]));
        w1.x = pack_bf16(__uint_as_float(v[8]), __uint_as_float(v[9]));
        w1.y = pack_bf16(__uint_as_float(v[10]), __uint_as_float(v[11]));
        w1.z = pack_bf16(__uint_as_float(v[12]), __uint_as_float(v[13]));
        w1.w = pack_bf16(__uint_as_float(v[14]), __uint_as_float(v[15]));
        *reinterpret_cast<uint4*>(orow + c0 * 2) = w0;
        if (c0 + 8 < rp) *reinterpret_cast<uint4*>(orow + c0 * 2 + 16) = w1;
      }
      tc_fence_before();
      mbar_arrive(&hdr->acc_empty[acc]);
      fence_async_smem();                                    // the rows above, before the bulk store reads them
      epilogue_sync();
      if (issuer) {
        const int t0 = it.tt * kTile;
        const int rows_valid = min(kTile, p.T - t0);
        char* dst;
        if (it.which == 0)
          dst = p.qp + (static_cast<int64_t>(hd.lr_k_off) * total_rows + (static_cast<int64_t>(it.b) * p.T + t0) * rp) * 2;
        else
          dst = p.cache + (is_v ? hd.v_off : hd.k_off) + (static_cast<int64_t>(it.b) * p.n_max + p.row0 + t0) * rp * 2;
        bulk_store(dst, ob, static_cast<uint32_t>(rows_valid * rp * 2));
      }
    }
    if (issuer) bulk_store_wait_all();                       // every store issued has completed before the CTA leaves
    if (!ok) *abort_flag = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 2 * ncols);
}

}  // namespace

// Shared memory of the kernel for a layer whose widest padded rank is max_rp; *stages gets the ring depth
// (0 when not even two stages fit).
size_t project_tc_stream_smem(int max_rp, int d_head, int* stages) {
  const int rp16 = (max_rp + 15) & ~15;
  const size_t u_bytes = 2ull * rp16 * d_head * 2;             // basis images
  const size_t o_bytes = 2ull * kTile * rp16 * 2;              // two output tiles
  const size_t x_bytes = static_cast<size_t>(d_head >> 6) * kAtomBytesA;
  const size_t budget = 227 * 1024;
  int s = kPsMaxStages;
  while (s >= 2 && 1024 + s * x_bytes + u_bytes + o_bytes > budget) --s;
  *stages = s >= 2 ? s : 0;
  return 1024 + s * x_bytes + u_bytes + o_bytes;
}

cudaError_t launch_project_tc_stream(const ProjectTcParams& p, const void* maps_qkv, int max_rp, int sm_count,
                                     cudaStream_t s, uint64_t* launches) {
  int stages = 0;
  const size_t smem = project_tc_stream_smem(max_rp, p.d_head, &stages);
  if (stages < 2) return cudaErrorInvalidConfiguration;
  auto kernel = p.d_head == 128 ? project_tc_stream_kernel<8> : project_tc_stream_kernel<4>;
  static size_t configured[2][kMaxDevices] = {};   // per kernel instance
  const cudaError_t ec = ensure_dynamic_smem(kernel, smem, configured[p.d_head == 128 ? 1 : 0]);
  if (ec != cudaSuccess) return ec;
  const CUtensorMap* maps = static_cast<const CUtensorMap*>(maps_qkv);
  const int64_t total = 3ll * p.H * p.B * ((p.T + kTile - 1) / kTile);
  const int grid = static_cast<int>(total < sm_count ? total : sm_count);
  const int rp16 = (max_rp + 15) & ~15;
  uint32_t ncols = 32;                                       // TMEM columns per accumulator: a power of two
  while (static_cast<int>(ncols) < rp16) ncols <<= 1;
  kernel<<<grid, kPsThreads, smem, s>>>(p, maps[0], maps[1], maps[2], stages, ncols, 2 * rp16 * p.d_head * 2,
                                        kTile * rp16 * 2);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
