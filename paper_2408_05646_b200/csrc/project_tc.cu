// Prefill-side projections on the tensor cores (tcgen05): for 128 prompt tokens of one head at a time,
//   Q' = Q U^K,  K' = K U^K,  V' = V U^V        (the r-wide factors of Eq. 6 of the paper)
// K' and V' go to rows row0.. of the rank-r cache, Q' to the prefill scratch.  The token rows are the
// bf16 A operand; the basis, an fp32 matrix, is the B operand split into bf16 high + low parts whose
// canonical shared-memory images are prepared once at create time, so each output is the sum of two
// tensor-core products accumulated in fp32 (about 2^-17 relative error from the split).  blockIdx.z
// selects which of the three projections the CTA performs.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

__global__ void __launch_bounds__(kThreads) project_tc_kernel(const ProjectTcParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  TcSmemHeader* hdr = reinterpret_cast<TcSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int h = blockIdx.y, which = blockIdx.z;               // which: 0 = Q, 1 = K, 2 = V
  const HeadInfo hd = p.heads[h];
  const bool is_v = which == 2;
  const int rp = is_v ? hd.rp_v : hd.rp_k;
  const int rp16 = (rp + 15) & ~15;
  const int nch_d = p.d_head >> 3;                            // 16-byte chunks along d_head
  const int grp_d = nch_d << 7;                               // bytes per 8-row group of a d_head-wide tile
  const int total_rows = p.B * p.T;
  const int r0 = blockIdx.x * kTile;
  const int rows_valid = min(kTile, total_rows - r0);

  unsigned char* Xs = smem + 1024;                            // [128 tokens][d_head] bf16, canonical
  unsigned char* Uh = Xs + kTile * p.d_head * 2;              // [rp16][d_head] bf16 high part of U^T
  unsigned char* Ul = Uh + rp16 * p.d_head * 2;               // low part

  uint32_t ncols = 32;
  while (ncols < static_cast<uint32_t>(rp16)) ncols <<= 1;
  if (warp == 0) tmem_alloc(&hdr->tmem_base, ncols);
  if (tid == 0) {
    mbar_init(&hdr->bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }

  // token rows -> canonical A tile (rows past the end are zero)
  const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(which == 0 ? p.q : (which == 1 ? p.k : p.v));
  for (int idx = tid; idx < kTile * nch_d; idx += kThreads) {
    const int c = idx >> 7, row = idx & (kTile - 1);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < rows_valid) {
      const int r = r0 + row, b = r / p.T, t = r - b * p.T;
      v = __ldg(reinterpret_cast<const uint4*>(X + b * p.stride_b + t * p.stride_t + static_cast<int64_t>(h) * p.d_head) + c);
    }
    *reinterpret_cast<uint4*>(Xs + chunk_off(row, c, grp_d)) = v;
  }
  // the basis images are already in canonical order: straight copy (high part, then low part)
  const uint4* Ug = reinterpret_cast<const uint4*>(p.basis + (is_v ? hd.uvt16_off : hd.ukt16_off));
  const int img16 = rp16 * p.d_head * 2 / 16;                 // 16-byte words per image
  for (int idx = tid; idx < 2 * img16; idx += kThreads) reinterpret_cast<uint4*>(Uh)[idx] = __ldg(Ug + idx);
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  if (tid == 0) {
    const uint32_t idesc = instr_desc(rp16, false);
    const uint32_t xa = smem_u32(Xs), uh = smem_u32(Uh), ul = smem_u32(Ul);
    bool acc = false;
    for (int pass = 0; pass < 2; ++pass)
      for (int s = 0; s < p.d_head / 16; ++s) {               // contraction over d_head
        mma_ss(tmem, smem_desc(xa + s * 256, 128, grp_d), smem_desc((pass ? ul : uh) + s * 256, 128, grp_d), idesc, acc);
        acc = true;
      }
    mma_commit(&hdr->bar);
  }
  const bool ok = mbar_wait(&hdr->bar, 0, p.status);
  tc_fence_after();
  if (!__syncthreads_or(!ok)) {
    // this thread's token row -> bf16 -> destination row (rp elements, contiguous)
    const int r = r0 + tid;
    __nv_bfloat16* dst = nullptr;
    if (tid < rows_valid) {
      const int b = r / p.T, t = r - b * p.T;
      if (which == 0)
        dst = reinterpret_cast<__nv_bfloat16*>(p.qp) + static_cast<int64_t>(hd.lr_k_off) * total_rows +
              static_cast<int64_t>(r) * rp;
      else
        dst = reinterpret_cast<__nv_bfloat16*>(p.cache + (is_v ? hd.v_off : hd.k_off)) +
              (static_cast<int64_t>(b) * p.n_max + p.row0 + t) * rp;
    }
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    for (int c0 = 0; c0 < rp16; c0 += 16) {
      uint32_t v[16];
      tmem_ld16(tmem + lane_base + c0, v);
      tmem_wait_ld();
      if (dst != nullptr) {
        uint4 w0, w1;
        w0.x = pack_bf16(__uint_as_float(v[0]), __uint_as_float(v[1]));
        w0.y = pack_bf16(__uint_as_float(v[2]), __uint_as_float(v[3]));
        w0.z = pack_bf16(__uint_as_float(v[4]), __uint_as_float(v[5]));
        w0.w = pack_bf16(__uint_as_float(v[6]), __uint_as_float(v[7]));
        w1.x = pack_bf16(__uint_as_float(v[8]), __uint_as_float(v[9]));
        w1.y = pack_bf16(__uint_as_float(v[10]), __uint_as_float(v[11]));
        w1.z = pack_bf16(__uint_as_float(v[12]), __uint_as_float(v[13]));
        w1.w = pack_bf16(__uint_as_float(v[14]), __uint_as_float(v[15]));
        *reinterpret_cast<uint4*>(dst + c0) = w0;
        if (c0 + 8 < rp) *reinterpret_cast<uint4*>(dst + c0 + 8) = w1;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, ncols);
}

}  // namespace

cudaError_t launch_project_tc(const ProjectTcParams& p, int max_rp, cudaStream_t s, uint64_t* launches) {
  const int rp16 = (max_rp + 15) & ~15;
  const size_t smem = 1024 + static_cast<size_t>(kTile) * p.d_head * 2 + 2ull * rp16 * p.d_head * 2;
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(project_tc_kernel, smem, configured);
  if (ec != cudaSuccess) return ec;
  dim3 grid((p.B * p.T + kTile - 1) / kTile, p.H, 3);
  project_tc_kernel<<<grid, kThreads, smem, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
