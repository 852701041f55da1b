// Projection of new key/value rows onto the head bases and append to the rank-r cache:
// k' = k U^K, v' = v U^V (the r-wide factor of Eq. 6 of the paper), written at rows
// row0..row0+T-1 of the cache (Section 2: K <- Concat(K, k), V <- Concat(V, v)).
// Also the prefill-side projection Q' = Q U^K into a scratch buffer.
//
// One CTA handles a run of (sequence, token) rows of one head.  The input rows are staged in shared
// memory as fp32; thread c owns output column c (K' columns first, then V' columns), reads its
// column of U from global memory (coalesced across the CTA, L2 resident) and accumulates eight rows
// at a time in registers.
#include <cuda_bf16.h>

#include "internal.h"

namespace ea {
namespace {

constexpr int kProjThreads = 256;
constexpr int kRowBlock = 8;

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// rows_per_cta rows starting at blockIdx.x * rows_per_cta of the flattened (b, t) index, head blockIdx.y.
template <typename T, bool kQueryOnly>
__global__ void __launch_bounds__(kProjThreads) project_rows_kernel(const ProjectParams p, char* qp_out,
                                                                   int rows_per_cta) {
  extern __shared__ __align__(16) float xs[];   // [2][rows_per_cta][d_head]  (k rows, then v rows)
  const int h = blockIdx.y;
  const HeadInfo hd = p.heads[h];
  const int d_head = p.d_head;
  const int total_rows = p.B * p.T;
  const int r0 = blockIdx.x * rows_per_cta;
  const int nrows = min(rows_per_cta, total_rows - r0);
  const int tid = threadIdx.x;
  const T* k = static_cast<const T*>(p.k);
  const T* v = static_cast<const T*>(p.v);
  float* ks = xs;
  float* vs = xs + static_cast<size_t>(rows_per_cta) * d_head;

  for (int idx = tid; idx < nrows * d_head; idx += kProjThreads) {
    const int r = idx / d_head, d = idx - r * d_head;
    const int row = r0 + r;
    const int b = row / p.T, t = row - b * p.T;
    const int64_t src = b * p.stride_b + t * p.stride_t + static_cast<int64_t>(h) * d_head + d;
    ks[idx] = to_f<T>(k[src]);
    if (!kQueryOnly) vs[idx] = to_f<T>(v[src]);
  }
  __syncthreads();

  const int ncol = kQueryOnly ? hd.rp_k : hd.rp_k + hd.rp_v;
  for (int c = tid; c < ncol; c += kProjThreads) {
    const bool is_k = c < hd.rp_k;
    const int col = is_k ? c : c - hd.rp_k;
    const int rp = is_k ? hd.rp_k : hd.rp_v;
    const float* U = p.basis + (is_k ? hd.uk_off : hd.uv_off) + col;
    const float* x = is_k ? ks : vs;
    for (int rb = 0; rb < nrows; rb += kRowBlock) {
      float acc[kRowBlock];
#pragma unroll
      for (int i = 0; i < kRowBlock; ++i) acc[i] = 0.f;
      for (int d = 0; d < d_head; d += 4) {
        const float u0 = __ldg(U + (d + 0) * rp), u1 = __ldg(U + (d + 1) * rp);
        const float u2 = __ldg(U + (d + 2) * rp), u3 = __ldg(U + (d + 3) * rp);
#pragma unroll
        for (int i = 0; i < kRowBlock; ++i) {
          if (rb + i < nrows) {
            const float4 xv = *reinterpret_cast<const float4*>(x + (rb + i) * d_head + d);
            acc[i] = fmaf(xv.x, u0, acc[i]);
            acc[i] = fmaf(xv.y, u1, acc[i]);
            acc[i] = fmaf(xv.z, u2, acc[i]);
            acc[i] = fmaf(xv.w, u3, acc[i]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < kRowBlock; ++i) {
        if (rb + i < nrows) {
          const int row = r0 + rb + i;
          const int b = row / p.T, t = row - b * p.T;
          if (kQueryOnly) {
            T* dst = reinterpret_cast<T*>(qp_out) + static_cast<int64_t>(hd.lr_k_off) * total_rows +
                     static_cast<int64_t>(row) * rp + col;
            *dst = from_f<T>(acc[i]);
          } else {
            const int64_t crow = physical_row(p.pages, b, p.n_max, p.row0 - (p.deficit ? p.deficit[b] : 0) + t);
            T* dst = reinterpret_cast<T*>(p.cache + (is_k ? hd.k_off : hd.v_off)) + crow * rp + col;
            *dst = from_f<T>(acc[i]);
          }
        }
      }
    }
  }
}

// Rows already in the rank-r space (merged W^K', W^V'): copy them into the cache.
template <typename T>
__global__ void __launch_bounds__(256) copy_lowrank_rows_kernel(const ProjectParams p) {
  const int h = blockIdx.y;
  const HeadInfo hd = p.heads[h];
  const int row = blockIdx.x;
  const int b = row / p.T, t = row - b * p.T;
  const T* k = static_cast<const T*>(p.k);
  const T* v = static_cast<const T*>(p.v);
  const int64_t crow = physical_row(p.pages, b, p.n_max, p.row0 - (p.deficit ? p.deficit[b] : 0) + t);
  for (int c = threadIdx.x; c < hd.rp_k + hd.rp_v; c += blockDim.x) {
    const bool is_k = c < hd.rp_k;
    const int col = is_k ? c : c - hd.rp_k;
    const int r = is_k ? hd.r_k : hd.r_v;
    const int rp = is_k ? hd.rp_k : hd.rp_v;
    const int width = is_k ? p.lr_k_width : p.lr_v_width;   // packed rows are contiguous [B][T][width]
    const T* src = (is_k ? k : v) + (static_cast<int64_t>(b) * p.T + t) * width + (is_k ? hd.lr_k_off : hd.lr_v_off);
    T* dst = reinterpret_cast<T*>(p.cache + (is_k ? hd.k_off : hd.v_off)) + crow * rp;
    dst[col] = col < r ? src[col] : from_f<T>(0.f);
  }
}

// Query rows already in the rank-r space (merged W^Q'): packed [B][T][width] into the per-head Q' scratch.
template <typename T>
__global__ void __launch_bounds__(128) scatter_q_lowrank_kernel(const QProjectParams p, int width) {
  const int h = blockIdx.y;
  const HeadInfo hd = p.heads[h];
  const int row = blockIdx.x;                      // flattened (b, t)
  const int64_t total_rows = static_cast<int64_t>(p.B) * p.T;
  const T* src = static_cast<const T*>(p.q) + static_cast<int64_t>(row) * width + hd.lr_k_off;
  T* dst = reinterpret_cast<T*>(p.qp) + static_cast<int64_t>(hd.lr_k_off) * total_rows + static_cast<int64_t>(row) * hd.rp_k;
  for (int c = threadIdx.x; c < hd.rp_k; c += blockDim.x) dst[c] = c < hd.r_k ? src[c] : from_f<T>(0.f);
}

int pick_rows_per_cta(int total_rows, int H) {
  // enough CTAs to cover the chip when few rows arrive (decode), larger tiles otherwise
  int rows = 32;
  while (rows > 1 && static_cast<long long>((total_rows + rows - 1) / rows) * H < 296) rows >>= 1;
  return rows;
}

}  // namespace

cudaError_t launch_project_append(const ProjectParams& p, int dtype, cudaStream_t s, uint64_t* launches) {
  const int total_rows = p.B * p.T;
  if (p.flags & 0x4u) {
    dim3 grid(total_rows, p.H);
    if (dtype == 0) copy_lowrank_rows_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(p);
    else copy_lowrank_rows_kernel<float><<<grid, 256, 0, s>>>(p);
    ++*launches;
    return cudaGetLastError();
  }
  const int rows = pick_rows_per_cta(total_rows, p.H);
  dim3 grid((total_rows + rows - 1) / rows, p.H);
  const size_t smem = 2ull * rows * p.d_head * sizeof(float);
  if (dtype == 0)
    project_rows_kernel<__nv_bfloat16, false><<<grid, kProjThreads, smem, s>>>(p, nullptr, rows);
  else
    project_rows_kernel<float, false><<<grid, kProjThreads, smem, s>>>(p, nullptr, rows);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_q_scatter(const QProjectParams& q, int lr_k_width, int dtype, cudaStream_t s, uint64_t* launches) {
  dim3 grid(q.B * q.T, q.H);
  if (dtype == 0) scatter_q_lowrank_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>(q, lr_k_width);
  else scatter_q_lowrank_kernel<float><<<grid, 128, 0, s>>>(q, lr_k_width);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_q_project(const QProjectParams& q, int dtype, cudaStream_t s, uint64_t* launches) {
  ProjectParams p{};
  p.heads = q.heads; p.basis = q.basis; p.k = q.q; p.v = q.q; p.cache = nullptr;
  p.stride_b = q.stride_b; p.stride_t = q.stride_t;
  p.B = q.B; p.T = q.T; p.H = q.H; p.d_head = q.d_head; p.n_max = 0; p.row0 = 0; p.flags = 0;
  const int total_rows = p.B * p.T;
  const int rows = pick_rows_per_cta(total_rows, p.H);
  dim3 grid((total_rows + rows - 1) / rows, p.H);
  const size_t smem = 2ull * rows * p.d_head * sizeof(float);
  if (dtype == 0)
    project_rows_kernel<__nv_bfloat16, true><<<grid, kProjThreads, smem, s>>>(p, q.qp, rows);
  else
    project_rows_kernel<float, true><<<grid, kProjThreads, smem, s>>>(p, q.qp, rows);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
