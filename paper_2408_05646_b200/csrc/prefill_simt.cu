// Causal rank-r prefill attention on the CUDA cores (any shape, any dtype the library supports):
//   O'[t] = Softmax( mask(Q'[t] K'^T / sqrt(d_h)) ) V' ,  out[t] = O'[t] (U^V)^T        (Eq. 7 + causal mask)
// Q' comes from a scratch buffer (already projected), K' and V' from the rank-r cache, so the rows
// attended are exactly the ones later decode steps will read.  Four threads share one query row
// (each holds a quarter of q' and of o'), a CTA covers 32 query rows and walks the key axis in
// tiles of 32 rows staged in shared memory as fp32, with an online softmax in base 2.
#include <cuda_bf16.h>

#include "internal.h"

namespace ea {
namespace {

constexpr int kQRows = 32;
constexpr int kKeyTile = 32;
constexpr int kThreads = kQRows * 4;

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// CW = upper bound of columns per thread (a quarter of the padded rank, rounded up to 8).
template <typename T, int CW>
__global__ void __launch_bounds__(kThreads) prefill_simt_kernel(const PrefillParams p) {
  extern __shared__ __align__(16) float sm[];
  const int unit = blockIdx.x;
  const int h = unit / p.B, b = unit - h * p.B;
  const int len0 = p.len0 - (p.deficit != nullptr ? __ldg(p.deficit + b) : 0);   // rows this sequence held before the call
  const HeadInfo hd = p.heads[h];
  const int rpk = hd.rp_k, rpv = hd.rp_v;
  const int cwk = rpk >> 2, cwv = rpv >> 2;           // rp is a multiple of 8 -> quarters are even
  float* Ks = sm;                                     // [kKeyTile][rpk]
  float* Vs = Ks + kKeyTile * rpk;                    // [kKeyTile][rpv]
  float* Os = Vs + kKeyTile * rpv;                    // [kQRows][rpv]
  const int qblk = gridDim.y - 1 - blockIdx.y;        // heavy (late) query blocks first
  const int tid = threadIdx.x;
  const int qr = tid >> 2, sub = tid & 3;
  const int t = qblk * kQRows + qr;                   // query index inside the call
  const bool live = t < p.T;
  const int total_rows = p.B * p.T;

  float q[CW], o[CW];
#pragma unroll
  for (int c = 0; c < CW; ++c) { q[c] = 0.f; o[c] = 0.f; }
  if (live) {
    const T* qp = reinterpret_cast<const T*>(p.qp) + static_cast<int64_t>(hd.lr_k_off) * total_rows +
                  (static_cast<int64_t>(b) * p.T + t) * rpk + sub * cwk;
#pragma unroll
    for (int c = 0; c < CW; ++c)
      if (c < cwk) q[c] = to_f<T>(qp[c]) * p.scale_log2;
  }
  float m = -INFINITY, l = 0.f;
  const int my_last = len0 + t;                                      // last key this query sees
  const int blk_last = len0 + min(p.T - 1, qblk * kQRows + kQRows - 1);
  const T* Kslab = reinterpret_cast<const T*>(p.cache + hd.k_off);
  const T* Vslab = reinterpret_cast<const T*>(p.cache + hd.v_off);

  for (int j0 = 0; j0 <= blk_last; j0 += kKeyTile) {
    const int nk = min(kKeyTile, blk_last + 1 - j0);
    __syncthreads();
    const int64_t prow = physical_row(p.pages, b, p.n_max, j0);     // a key tile of 32 rows lies inside one page
    for (int idx = tid; idx < nk * rpk; idx += kThreads) Ks[idx] = to_f<T>(Kslab[prow * rpk + idx]);
    for (int idx = tid; idx < nk * rpv; idx += kThreads) Vs[idx] = to_f<T>(Vslab[prow * rpv + idx]);
    __syncthreads();
    for (int j = 0; j < nk; ++j) {
      const float* kr = Ks + j * rpk + sub * cwk;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int c = 0; c < CW; c += 2)
        if (c < cwk) {
          const float2 kv = *reinterpret_cast<const float2*>(kr + c);
          s0 = fmaf(q[c], kv.x, s0);
          s1 = fmaf(q[c + 1], kv.y, s1);
        }
      float s = s0 + s1;
      s += __shfl_xor_sync(0xffffffffu, s, 1);
      s += __shfl_xor_sync(0xffffffffu, s, 2);
      s = fmaf(hd.alibi_slope2, static_cast<float>(j0 + j - my_last), s);   // ALiBi: slope * (key - query position)
      if (live && j0 + j <= my_last) {
        if (s > m) {
          const float c0 = ex2(m - s);
          l *= c0;
#pragma unroll
          for (int c = 0; c < CW; ++c) o[c] *= c0;
          m = s;
        }
        const float pr = ex2(s - m);
        l += pr;
        const float* vr = Vs + j * rpv + sub * cwv;
#pragma unroll
        for (int c = 0; c < CW; c += 2)
          if (c < cwv) {
            const float2 vv = *reinterpret_cast<const float2*>(vr + c);
            o[c] = fmaf(pr, vv.x, o[c]);
            o[c + 1] = fmaf(pr, vv.y, o[c + 1]);
          }
      }
    }
  }

  const float inv = live ? 1.f / l : 0.f;
  T* out = static_cast<T*>(p.out);
  if (p.flags & 0x2u) {   // rank-space output
    if (live) {
      T* dst = out + b * p.out_stride_b + t * p.out_stride_t + hd.lr_v_off + sub * cwv;
#pragma unroll
      for (int c = 0; c < CW; ++c)
        if (c < cwv) dst[c] = from_f<T>(o[c] * inv);
    }
    return;
  }
#pragma unroll
  for (int c = 0; c < CW; ++c)
    if (c < cwv) Os[qr * rpv + sub * cwv + c] = o[c] * inv;
  __syncthreads();
  if (live) {
    const float* Ut = p.basis + hd.uvt_off;     // (U^V)^T : rpv x d_head
    const float* orow = Os + qr * rpv;
    T* dst = out + b * p.out_stride_b + t * p.out_stride_t + static_cast<int64_t>(h) * p.d_head;
    for (int d = sub; d < p.d_head; d += 4) {
      float y = 0.f;
      for (int c = 0; c < rpv; ++c) y = fmaf(orow[c], __ldg(Ut + c * p.d_head + d), y);
      dst[d] = from_f<T>(y);
    }
  }
}

template <typename T>
cudaError_t launch_t(const PrefillParams& p, cudaStream_t s) {
  dim3 grid(p.B * p.H, (p.T + kQRows - 1) / kQRows);
  // the widest head bounds the shared-memory tiles and the per-thread column count
  const size_t smem = (static_cast<size_t>(kKeyTile) * 2 + kQRows) * p.max_rp * sizeof(float);
  const int cw = (p.max_rp / 4 + 7) / 8 * 8;
  switch (cw) {
    case 8: prefill_simt_kernel<T, 8><<<grid, kThreads, smem, s>>>(p); break;
    case 16: prefill_simt_kernel<T, 16><<<grid, kThreads, smem, s>>>(p); break;
    case 24: prefill_simt_kernel<T, 24><<<grid, kThreads, smem, s>>>(p); break;
    default: prefill_simt_kernel<T, 32><<<grid, kThreads, smem, s>>>(p); break;
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill_simt(const PrefillParams& p, int dtype, cudaStream_t s, uint64_t* launches) {
  ++*launches;
  return dtype == 0 ? launch_t<__nv_bfloat16>(p, s) : launch_t<float>(p, s);
}

}  // namespace ea
