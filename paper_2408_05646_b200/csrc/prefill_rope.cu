// Causal prompt attention of the RoPE variant (Section 4.3 of the paper applied to the prefill phase of Section 2)
// on the CUDA cores: the prompt path of a layer with rotary position embedding.
//
//   score(t, j) = RoPE_{len0+t}(q_t) . RoPE_j(k'_j (U^K)^T) / sqrt(d_h),   out_t = Softmax_j<=len0+t(score) V' (U^V)^T
//
// The queries stay full rank; every cached low-dimensional key is taken back to d_h dimensions through (U^K)^T
// and rotated by its position (row j of the cache = position j); the value side is the rank-r path unchanged.
// The rows attended are the ones the call has just appended (un-rotated keys projected by eigen_attn_append_kv's
// kernel), so that the generation phase finds the cache Section 4.3 expects.
//
// A CTA covers 32 query rows (four threads per row, each a quarter of d_h) and walks the key axis in tiles of 32
// rows.  Per tile: the rank-r rows are staged as fp32, thread d lifts all 32 rows' coordinate d (one pass over
// row d of U^K, 32 accumulators), pairs are rotated in place (the tile's base angle per pair is reduced in double
// precision once per tile, the row offset inside the tile comes from a table built once per CTA, the two are
// combined by the angle-addition formulas), then scores, an online softmax in base 2 and the weighted sum of
// value rows as in the plain CUDA-core prefill kernel.  fp32 throughout; this is the functional path, not a
// tensor-core one.
#include <cuda_bf16.h>

#include "internal.h"

namespace ea {
namespace {

constexpr int kQRows = 32;
constexpr int kKeyTile = 32;
constexpr int kThreads = kQRows * 4;
constexpr double kTwoPi = 6.283185307179586476925286766559;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// cos and sin of pos * freq with the product reduced to [-pi, pi] in double precision
__device__ __forceinline__ void cos_sin_of(double pos, double freq, float* c, float* s) {
  double a = pos * freq;
  a -= kTwoPi * rint(a / kTwoPi);
  sincosf(static_cast<float>(a), s, c);
}

template <int CWV>   // upper bound of value columns per thread (a quarter of the padded rank, rounded up to 8)
__global__ void __launch_bounds__(kThreads) prefill_rope_kernel(const PrefillParams p) {
  extern __shared__ __align__(16) float sm[];
  const int unit = blockIdx.x;
  const int h = unit / p.B, b = unit - h * p.B;
  const int len0 = p.len0 - (p.deficit != nullptr ? __ldg(p.deficit + b) : 0);   // rows this sequence held before the call
  const HeadInfo hd = p.heads[h];
  const int rpk = hd.rp_k, rpv = hd.rp_v, dh = p.d_head, half = dh >> 1, dq = dh >> 2;
  const int cwv = rpv >> 2;
  float* Kraw = sm;                                   // [32][rpk]   rank-r key rows of the tile
  float* Ks = Kraw + kKeyTile * rpk;                  // [32][dh]    lifted, then rotated keys
  float* Vs = Ks + kKeyTile * dh;                     // [32][rpv]
  float* Os = Vs + kKeyTile * rpv;                    // [32][rpv]
  float* tab = Os + kQRows * rpv;                     // [32][half][2]  cos, sin of (row offset) * freq
  float* base_cs = tab + kKeyTile * half * 2;         // [half][2]      cos, sin of (tile start) * freq
  const int qblk = gridDim.y - 1 - blockIdx.y;        // heavy (late) query blocks first
  const int tid = threadIdx.x;
  const int qr = tid >> 2, sub = tid & 3;
  const int t = qblk * kQRows + qr;                   // query index inside the call
  const bool live = t < p.T;
  const bool inter = p.rope_interleaved != 0;

  for (int idx = tid; idx < kKeyTile * half; idx += kThreads) {
    const int l = idx / half, i = idx - l * half;
    cos_sin_of(static_cast<double>(l), p.inv_freq[i], &tab[2 * idx], &tab[2 * idx + 1]);
  }
  // this thread's quarter of the rotated query, scaled into the base-2 domain
  float q[32], o[CWV];
#pragma unroll
  for (int c = 0; c < 32; ++c) q[c] = 0.f;
#pragma unroll
  for (int c = 0; c < CWV; ++c) o[c] = 0.f;
  if (live) {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q_raw) + b * p.q_stride_b + t * p.q_stride_t +
                              static_cast<int64_t>(h) * dh;
    const double pos = static_cast<double>(len0 + t);
#pragma unroll
    for (int c = 0; c < 32; ++c)
      if (c < dq) {
        const int d = sub * dq + c;
        const int i = inter ? d >> 1 : (d < half ? d : d - half);           // pair index
        const bool is_a = inter ? (d & 1) == 0 : d < half;
        const int partner = inter ? d ^ 1 : (d < half ? d + half : d - half);
        float cs, sn;
        cos_sin_of(pos, p.inv_freq[i], &cs, &sn);
        const float x = __bfloat162float(qg[d]), y = __bfloat162float(qg[partner]);
        q[c] = (is_a ? x * cs - y * sn : y * sn + x * cs) * p.scale_log2;
      }
  }
  float m = -INFINITY, l = 0.f;
  const int my_last = len0 + t;                                      // last key this query sees
  const int blk_last = len0 + min(p.T - 1, qblk * kQRows + kQRows - 1);
  const __nv_bfloat16* Kslab = reinterpret_cast<const __nv_bfloat16*>(p.cache + hd.k_off);
  const __nv_bfloat16* Vslab = reinterpret_cast<const __nv_bfloat16*>(p.cache + hd.v_off);
  const float* U = p.basis + hd.uk_off;                                // U^K: d_head x rp_k, row d = coordinates of e_d

  for (int j0 = 0; j0 <= blk_last; j0 += kKeyTile) {
    const int nk = min(kKeyTile, blk_last + 1 - j0);
    __syncthreads();
    const int64_t prow = physical_row(p.pages, b, p.n_max, j0);
    for (int idx = tid; idx < nk * rpk; idx += kThreads) Kraw[idx] = __bfloat162float(Kslab[prow * rpk + idx]);
    for (int idx = tid; idx < nk * rpv; idx += kThreads) Vs[idx] = __bfloat162float(Vslab[prow * rpv + idx]);
    if (tid < half) cos_sin_of(static_cast<double>(j0), p.inv_freq[tid], &base_cs[2 * tid], &base_cs[2 * tid + 1]);
    __syncthreads();
    // ---- lift: coordinate d of k'_row (U^K)^T for the 32 rows (rows past nk read stale finite numbers, never used)
    if (tid < dh) {
      float acc[kKeyTile];
#pragma unroll
      for (int r = 0; r < kKeyTile; ++r) acc[r] = 0.f;
      const float* Ud = U + static_cast<size_t>(tid) * rpk;
      for (int c = 0; c < rpk; ++c) {
        const float u = __ldg(Ud + c);
#pragma unroll
        for (int r = 0; r < kKeyTile; ++r) acc[r] = fmaf(Kraw[r * rpk + c], u, acc[r]);
      }
#pragma unroll
      for (int r = 0; r < kKeyTile; ++r) Ks[r * dh + tid] = acc[r];
    }
    __syncthreads();
    // ---- rotate pair i of row r by (j0 + r) * freq_i: angle addition of the tile's base and the row offset
    for (int idx = tid; idx < nk * half; idx += kThreads) {
      const int r = idx / half, i = idx - r * half;
      const int da = inter ? 2 * i : i, db = inter ? 2 * i + 1 : i + half;
      const float c0 = base_cs[2 * i], s0 = base_cs[2 * i + 1], cl = tab[2 * idx], sl = tab[2 * idx + 1];
      const float cs = c0 * cl - s0 * sl, sn = s0 * cl + c0 * sl;
      const float a = Ks[r * dh + da], bb = Ks[r * dh + db];
      Ks[r * dh + da] = a * cs - bb * sn;
      Ks[r * dh + db] = a * sn + bb * cs;
    }
    __syncthreads();
    for (int j = 0; j < nk; ++j) {
      const float* kr = Ks + j * dh + sub * dq;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int c = 0; c < 32; c += 2)
        if (c < dq) {
          const float2 kv = *reinterpret_cast<const float2*>(kr + c);
          s0 = fmaf(q[c], kv.x, s0);
          s1 = fmaf(q[c + 1], kv.y, s1);
        }
      float s = s0 + s1;
      s += __shfl_xor_sync(0xffffffffu, s, 1);
      s += __shfl_xor_sync(0xffffffffu, s, 2);
      if (live && j0 + j <= my_last) {
        if (s > m) {
          const float c0 = ex2(m - s);
          l *= c0;
#pragma unroll
          for (int c = 0; c < CWV; ++c) o[c] *= c0;
          m = s;
        }
        const float pr = ex2(s - m);
        l += pr;
        const float* vr = Vs + j * rpv + sub * cwv;
#pragma unroll
        for (int c = 0; c < CWV; c += 2)
          if (c < cwv) {
            const float2 vv = *reinterpret_cast<const float2*>(vr + c);
            o[c] = fmaf(pr, vv.x, o[c]);
            o[c + 1] = fmaf(pr, vv.y, o[c + 1]);
          }
      }
    }
  }

  const float inv = live ? 1.f / l : 0.f;
  __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.out);
  if (p.flags & 0x2u) {   // rank-space output
    if (live) {
      __nv_bfloat16* dst = out + b * p.out_stride_b + t * p.out_stride_t + hd.lr_v_off + sub * cwv;
#pragma unroll
      for (int c = 0; c < CWV; ++c)
        if (c < cwv) dst[c] = __float2bfloat16_rn(o[c] * inv);
    }
    return;
  }
#pragma unroll
  for (int c = 0; c < CWV; ++c)
    if (c < cwv) Os[qr * rpv + sub * cwv + c] = o[c] * inv;
  __syncthreads();
  if (live) {
    const float* Ut = p.basis + hd.uvt_off;     // (U^V)^T : rpv x d_head
    const float* orow = Os + qr * rpv;
    __nv_bfloat16* dst = out + b * p.out_stride_b + t * p.out_stride_t + static_cast<int64_t>(h) * dh;
    for (int d = sub; d < dh; d += 4) {
      float y = 0.f;
      for (int c = 0; c < rpv; ++c) y = fmaf(orow[c], __ldg(Ut + c * dh + d), y);
      dst[d] = __float2bfloat16_rn(y);
    }
  }
}

// ---- the same prompt on the tensor cores: what the attention kernel needs is prepared once per call
//
// With the full-rank rotated queries Qr_t = RoPE_{len0+t}(q_t) and the lifted, rotated keys Kr_j = RoPE_j(k'_j (U^K)^T)
// written out (16-bit, d_head wide), score(t, j) = Qr_t . Kr_j / sqrt(d_h) is an ordinary causal attention product
// over d_head-wide rows with rank-r values: the warp-specialised tensor-core kernel runs it unchanged, its key
// operand coming from these rows instead of the cache.  The keys are prepared by the tensor-core kernel of
// rope_lift_tc.cu, the queries here.

// Qr of one prompt token of one sequence, all heads: [h][b * T + t][d_head] (the layout the attention kernel reads)
__global__ void __launch_bounds__(256) rope_rotate_queries_kernel(const PrefillParams p) {
  __shared__ float cs[128];                           // cos, sin of the token's position times every frequency
  const int row = blockIdx.x;                         // b * T + t
  const int b = row / p.T, t = row - b * p.T;
  const int dh = p.d_head, half = dh >> 1;
  const int pos = p.len0 - (p.deficit != nullptr ? __ldg(p.deficit + b) : 0) + t;
  if (threadIdx.x < half) cos_sin_of(static_cast<double>(pos), p.inv_freq[threadIdx.x], &cs[2 * threadIdx.x], &cs[2 * threadIdx.x + 1]);
  __syncthreads();
  const bool inter = p.rope_interleaved != 0;
  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(p.q_raw) + b * p.q_stride_b + t * p.q_stride_t;
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(const_cast<char*>(p.qp));
  const int64_t total_rows = static_cast<int64_t>(p.B) * p.T;
  for (int idx = threadIdx.x; idx < p.H * half; idx += 256) {
    const int h = idx / half, i = idx - h * half;
    const int da = inter ? 2 * i : i, db = inter ? 2 * i + 1 : i + half;
    const float a = __bfloat162float(q[h * dh + da]), bb = __bfloat162float(q[h * dh + db]);
    const float c = cs[2 * i], s_ = cs[2 * i + 1];
    __nv_bfloat16* o = out + (static_cast<int64_t>(h) * total_rows + row) * dh;
    o[da] = __float2bfloat16_rn(a * c - bb * s_);
    o[db] = __float2bfloat16_rn(a * s_ + bb * c);
  }
}

}  // namespace

cudaError_t launch_rope_prompt_prepare(const PrefillParams& p, int max_rp_k, int sm_count, cudaStream_t s, uint64_t* launches) {
  const cudaError_t e = launch_rope_lift_tc(p, max_rp_k, sm_count, s, launches);   // Kr of every row held after the call
  if (e != cudaSuccess) return e;
  rope_rotate_queries_kernel<<<p.B * p.T, 256, 0, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_prefill_rope(const PrefillParams& p, int max_rp_k, int max_rp_v, cudaStream_t s, uint64_t* launches) {
  dim3 grid(p.B * p.H, (p.T + kQRows - 1) / kQRows);
  const int half = p.d_head / 2;
  const size_t smem = (static_cast<size_t>(kKeyTile) * (max_rp_k + p.d_head + max_rp_v) + static_cast<size_t>(kQRows) * max_rp_v +
                       static_cast<size_t>(kKeyTile) * half * 2 + half * 2) * sizeof(float);
  const int cw = (max_rp_v / 4 + 7) / 8 * 8;
  auto kernel = cw <= 8 ? prefill_rope_kernel<8> : cw <= 16 ? prefill_rope_kernel<16> : cw <= 24 ? prefill_rope_kernel<24>
                                                                                                   : prefill_rope_kernel<32>;
  static size_t configured[4][kMaxDevices] = {};
  const cudaError_t ec = ensure_dynamic_smem(kernel, smem, configured[cw <= 8 ? 0 : cw <= 16 ? 1 : cw <= 24 ? 2 : 3]);
  if (ec != cudaSuccess) return ec;
  kernel<<<grid, kThreads, smem, s>>>(p);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ea
