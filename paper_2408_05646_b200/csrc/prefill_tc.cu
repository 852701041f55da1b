// Causal rank-r prefill attention on the 5th-generation tensor cores (tcgen05, accumulators in TMEM):
//   S = Q' K'^T  (contraction over the rank, r_k),  P = softmax rows of mask(S / sqrt(d_h)),
//   O' = P V'    (contraction over the keys),       out = (O' / l) (U^V)^T        (Eq. 7 + causal mask)
// bf16 operands, fp32 accumulation.  One CTA owns 128 query rows of one (sequence, head) unit and walks
// the key axis in tiles of 128 rows.  Q', K', V' tiles are staged in shared memory in the canonical
// no-swizzle core-matrix layout (8 rows x 16 bytes per core matrix) that tcgen05.mma reads through
// shared-memory descriptors; K' is the K-major B operand of the first product and V', in the same
// physical layout, the MN-major B operand of the second.  One thread issues the MMAs; each of the 128
// threads owns one query row (= one TMEM lane) for the softmax, writes its row of P as bf16 into shared
// memory (A operand of the second product) and rescales its row of O' in TMEM when the running max
// grows.  The lift through (U^V)^T is a third tensor-core product with both operands split into
// bf16 high + low parts (three products), which keeps it at fp32-class accuracy.
#include <cuda_bf16.h>

#include "internal.h"
#include "tc_common.cuh"

namespace ea {
namespace {

using namespace tc;

// ---------------------------------------------------------------- the kernel

__global__ void __launch_bounds__(kThreads) prefill_tc_kernel(const PrefillParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  TcSmemHeader* hdr = reinterpret_cast<TcSmemHeader*>(smem);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int unit = blockIdx.x;
  const int h = unit / p.B, b = unit - h * p.B;
  const int len0 = p.len0 - (p.deficit != nullptr ? __ldg(p.deficit + b) : 0);   // rows this sequence held before the call
  const HeadInfo hd = p.heads[h];
  const int qblk = gridDim.y - 1 - blockIdx.y;              // late (long) query blocks first
  const int t0 = qblk * kTile;
  const int rpk16 = (hd.rp_k + 15) & ~15, rpv16 = (hd.rp_v + 15) & ~15;
  const int nch_k = rpk16 >> 3, nch_v = rpv16 >> 3;
  const int grp_k = nch_k << 7, grp_v = nch_v << 7, grp_p = (kTile >> 3) << 7;

  // shared-memory carve-up (1 KB header, then tiles)
  unsigned char* Qs = smem + 1024;
  unsigned char* Ks = Qs + kTile * rpk16 * 2;
  unsigned char* Vs = Ks + kTile * rpk16 * 2;
  unsigned char* Ps = Vs + kTile * rpv16 * 2;

  if (warp == 0) tmem_alloc(&hdr->tmem_base, 256);
  if (tid == 0) {
    mbar_init(&hdr->bar, 1);
    hdr->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = hdr->tmem_base;
  const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
  const uint32_t tS = tmem + lane_base;                      // S (and later the lifted output): columns 0..127
  const uint32_t tO = tmem + lane_base + 128;                // O': columns 128..128+rpv16
  uint32_t phase = 0;

  const int total_rows = p.B * p.T;
  const int q_valid = min(kTile, p.T - t0);
  const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.qp) +
                            static_cast<int64_t>(hd.lr_k_off) * total_rows +
                            (static_cast<int64_t>(b) * p.T + t0) * hd.rp_k;
  const __nv_bfloat16* Kg = reinterpret_cast<const __nv_bfloat16*>(p.cache + hd.k_off) +
                            static_cast<int64_t>(b) * p.n_max * hd.rp_k;
  const __nv_bfloat16* Vg = reinterpret_cast<const __nv_bfloat16*>(p.cache + hd.v_off) +
                            static_cast<int64_t>(b) * p.n_max * hd.rp_v;
  load_tile(Qs, Qg, hd.rp_k, q_valid, nch_k, tid);

  const int my_pos = len0 + t0 + tid;                      // last key this thread's query sees
  const float slope2 = hd.alibi_slope2;                      // ALiBi: slope * (key - query position), log2 domain
  const int n_keys = len0 + min(p.T, t0 + kTile);          // keys the block needs
  const int n_tiles = (n_keys + kTile - 1) / kTile;
  const uint32_t idesc_s = instr_desc(kTile, false);
  const uint32_t idesc_o = instr_desc(rpv16, true);
  float m_run = -INFINITY, l_run = 0.f;
  bool ok = true;

  for (int j = 0; j < n_tiles && ok; ++j) {
    const int key0 = j * kTile;
    const int k_valid = min(kTile, n_keys - key0);
    load_tile(Ks, Kg + static_cast<int64_t>(key0) * hd.rp_k, hd.rp_k, k_valid, nch_k, tid);
    load_tile(Vs, Vg + static_cast<int64_t>(key0) * hd.rp_v, hd.rp_v, k_valid, nch_v, tid);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t qa = smem_u32(Qs), ka = smem_u32(Ks);
      for (int s = 0; s < rpk16 / 16; ++s)                   // S = Q' K'^T, contraction over the rank
        mma_ss(tmem, smem_desc(qa + s * 256, 128, grp_k), smem_desc(ka + s * 256, 128, grp_k), idesc_s, s > 0);
      mma_commit(&hdr->bar);
    }
    ok = mbar_wait(&hdr->bar, phase, p.status);
    phase ^= 1u;
    tc_fence_after();
    if (__syncthreads_or(!ok)) { ok = false; break; }

    // ---- softmax of this thread's row: pass 1 = max, pass 2 = exponentials, sum and P
    const bool diag = key0 + kTile - 1 > len0 + t0;        // some (row, key) pair of the tile is masked
    float row_max = -INFINITY;
#pragma unroll 1
    for (int c0 = 0; c0 < kTile; c0 += 16) {
      uint32_t r[16];
      tmem_ld16(tS + c0, r);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        float s = fmaf(__uint_as_float(r[i]), p.scale_log2, slope2 * static_cast<float>(key0 + c0 + i - my_pos));
        if (diag && key0 + c0 + i > my_pos) s = -INFINITY;
        row_max = fmaxf(row_max, s);
      }
    }
    const float m_new = fmaxf(m_run, row_max);               // finite: key 0 is visible to every query
    const float alpha = ex2(m_run - m_new);
    float row_sum = 0.f;
#pragma unroll 1
    for (int c0 = 0; c0 < kTile; c0 += 16) {
      uint32_t r[16];
      tmem_ld16(tS + c0, r);
      tmem_wait_ld();
      float pr[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        float s = fmaf(__uint_as_float(r[i]), p.scale_log2, slope2 * static_cast<float>(key0 + c0 + i - my_pos)) - m_new;
        if (diag && key0 + c0 + i > my_pos) s = -INFINITY;
        pr[i] = ex2(s);
        row_sum += pr[i];
      }
      uint4 w0, w1;
      w0.x = pack_bf16(pr[0], pr[1]);   w0.y = pack_bf16(pr[2], pr[3]);
      w0.z = pack_bf16(pr[4], pr[5]);   w0.w = pack_bf16(pr[6], pr[7]);
      w1.x = pack_bf16(pr[8], pr[9]);   w1.y = pack_bf16(pr[10], pr[11]);
      w1.z = pack_bf16(pr[12], pr[13]); w1.w = pack_bf16(pr[14], pr[15]);
      *reinterpret_cast<uint4*>(Ps + chunk_off(tid, c0 >> 3, grp_p)) = w0;
      *reinterpret_cast<uint4*>(Ps + chunk_off(tid, (c0 >> 3) + 1, grp_p)) = w1;
    }
    l_run = l_run * alpha + row_sum;
    m_run = m_new;
    // ---- rescale this thread's row of O' when a running max in the warp grew
    if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
      for (int c0 = 0; c0 < rpv16; c0 += 16) {
        uint32_t r[16];
        tmem_ld16(tO + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
        tmem_st16(tO + c0, r);
      }
      tmem_wait_st();
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t pa = smem_u32(Ps), va = smem_u32(Vs);
      for (int s = 0; s < kTile / 16; ++s)                   // O' += P V', contraction over the 128 keys
        mma_ss(tmem + 128, smem_desc(pa + s * 256, 128, grp_p), smem_desc(va + s * 2 * grp_v, grp_v, 128), idesc_o,
               j > 0 || s > 0);
      mma_commit(&hdr->bar);
    }
    ok = mbar_wait(&hdr->bar, phase, p.status);
    phase ^= 1u;
    tc_fence_after();
    if (__syncthreads_or(!ok)) { ok = false; break; }
  }

  // ---- epilogue: out = (O' / l) (U^V)^T with hi/lo split bf16 operands (three tensor-core products)
  if (ok) {
    const float inv_l = 1.f / l_run;
    const bool lowrank = (p.flags & 0x2u) != 0;
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.out);
    if (lowrank) {
      __nv_bfloat16* dst = out + b * p.out_stride_b + static_cast<int64_t>(t0 + tid) * p.out_stride_t + hd.lr_v_off;
      for (int c0 = 0; c0 < rpv16; c0 += 16) {               // the TMEM loads are warp-collective: no divergence
        uint32_t r[16];
        tmem_ld16(tO + c0, r);
        tmem_wait_ld();
        if (tid < q_valid) {
          for (int i = 0; i < 16; ++i)
            if (c0 + i < hd.rp_v) dst[c0 + i] = __float2bfloat16_rn(__uint_as_float(r[i]) * inv_l);
        }
      }
    } else {
      // A operands: O' hi and lo as [128][rpv16] K-major tiles; B operands: U^V hi and lo as [d_head][rpv16]
      unsigned char* Oh = Qs;
      unsigned char* Ol = Oh + kTile * rpv16 * 2;
      unsigned char* Uh = Ol + kTile * rpv16 * 2;
      unsigned char* Ul = Uh + kTile * rpv16 * 2;
      for (int c0 = 0; c0 < rpv16; c0 += 16) {
        uint32_t r[16];
        tmem_ld16(tO + c0, r);
        tmem_wait_ld();
        uint32_t hi[8], lo[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float x0 = __uint_as_float(r[2 * i]) * inv_l, x1 = __uint_as_float(r[2 * i + 1]) * inv_l;
          const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
          hi[i] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
          lo[i] = pack_bf16(x0 - __bfloat162float(h0), x1 - __bfloat162float(h1));
        }
        *reinterpret_cast<uint4*>(Oh + chunk_off(tid, c0 >> 3, grp_v)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(Oh + chunk_off(tid, (c0 >> 3) + 1, grp_v)) = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        *reinterpret_cast<uint4*>(Ol + chunk_off(tid, c0 >> 3, grp_v)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        *reinterpret_cast<uint4*>(Ol + chunk_off(tid, (c0 >> 3) + 1, grp_v)) = make_uint4(lo[4], lo[5], lo[6], lo[7]);
      }
      // U^V (d_head x rp_v fp32, row-major) -> hi / lo tiles, rows = d (the N index), chunks along the rank
      const float* U = p.basis + hd.uv_off;
      for (int idx = tid; idx < kTile * nch_v; idx += kThreads) {
        const int c = idx >> 7, d = idx & (kTile - 1);
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float x0 = 0.f, x1 = 0.f;
          const int col = c * 8 + 2 * i;
          if (d < p.d_head && col < hd.rp_v) x0 = __ldg(U + d * hd.rp_v + col);
          if (d < p.d_head && col + 1 < hd.rp_v) x1 = __ldg(U + d * hd.rp_v + col + 1);
          const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
          hi[i] = pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
          lo[i] = pack_bf16(x0 - __bfloat162float(h0), x1 - __bfloat162float(h1));
        }
        *reinterpret_cast<uint4*>(Uh + chunk_off(d, c, grp_v)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(Ul + chunk_off(d, c, grp_v)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      }
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
        const uint32_t idesc_l = instr_desc(p.d_head, false);
        const uint32_t oh = smem_u32(Oh), ol = smem_u32(Ol), uh = smem_u32(Uh), ul = smem_u32(Ul);
        bool acc = false;
        for (int pass = 0; pass < 3; ++pass) {               // hi*hi + lo*hi + hi*lo
          const uint32_t a = pass == 1 ? ol : oh, bb = pass == 2 ? ul : uh;
          for (int s = 0; s < rpv16 / 16; ++s) {
            mma_ss(tmem, smem_desc(a + s * 256, 128, grp_v), smem_desc(bb + s * 256, 128, grp_v), idesc_l, acc);
            acc = true;
          }
        }
        mma_commit(&hdr->bar);
      }
      ok = mbar_wait(&hdr->bar, phase, p.status);
      phase ^= 1u;
      tc_fence_after();
      if (!__syncthreads_or(!ok)) {
        __nv_bfloat16* dst = out + b * p.out_stride_b + static_cast<int64_t>(t0 + tid) * p.out_stride_t +
                             static_cast<int64_t>(h) * p.d_head;
        for (int c0 = 0; c0 < p.d_head; c0 += 16) {
          uint32_t r[16];
          tmem_ld16(tS + c0, r);
          tmem_wait_ld();
          if (tid < q_valid) {
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
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
}

}  // namespace

size_t prefill_tc_smem_bytes(int max_rp_k, int max_rp_v) {
  const size_t k16 = (max_rp_k + 15) & ~15, v16 = (max_rp_v + 15) & ~15;
  const size_t loop = 2 * kTile * k16 * 2 + kTile * v16 * 2 + kTile * kTile * 2;   // Q, K, V, P
  const size_t lift = 4 * kTile * v16 * 2;                                          // O' hi/lo, U hi/lo
  return 1024 + (loop > lift ? loop : lift);
}

cudaError_t launch_prefill_tc(const PrefillParams& p, int max_rp_k, int max_rp_v, cudaStream_t s,
                              uint64_t* launches) {
  const size_t smem = prefill_tc_smem_bytes(max_rp_k, max_rp_v);
  static size_t configured[kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(prefill_tc_kernel, smem, configured);
  if (ec != cudaSuccess) return ec;
  dim3 grid(p.B * p.H, (p.T + kTile - 1) / kTile);
  prefill_tc_kernel<<<grid, kThreads, smem, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
