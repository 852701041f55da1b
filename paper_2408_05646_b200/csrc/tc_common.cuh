// Device-side building blocks shared by the tcgen05 kernels: mbarrier and fence wrappers, TMEM
// allocation and access, MMA issue, shared-memory matrix descriptors and the canonical no-swizzle tile.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "internal.h"

namespace ea {
namespace tc {

constexpr int kTile = 128;                 // query rows per CTA = key rows per tile = MMA M
constexpr int kThreads = 128;
constexpr uint64_t kWaitBoundNs = 2000000000ull;

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(void* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead of reading.
__device__ __forceinline__ void cp_async16(void* dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ bool mbar_try_wait(void* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(void* bar, uint32_t parity, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    // a wait that already gave up anywhere on this handle ends every other one: the launch drains in
    // one bound, not in one bound per wait
    if (*reinterpret_cast<volatile int*>(status) == kStatusTimeout) return false;
    if (global_ns() - t0 > kWaitBoundNs) {
      atomicExch(status, kStatusTimeout);
      return false;
    }
  }
}
// One arrival that also announces `bytes` of asynchronous copies which will complete on the barrier.
__device__ __forceinline__ void mbar_arrive_expect_tx(void* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// TMA: one box of a 3-D tensor map (in global memory) at element coordinates (x, y, z) into shared memory;
// the bytes of the whole box, zero fill included, complete on the barrier.  x * element size must be a
// multiple of 16 bytes.
__device__ __forceinline__ void tma_load_3d(void* dst, const void* tmap, int x, int y, int z, void* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}
// One contiguous asynchronous copy global -> shared (both 16-byte aligned, size a multiple of 16) that completes
// on the barrier; the data is read once, so L2 is told to evict it first.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, void* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
// Orders earlier writes of a tensor map through ordinary stores or copies before its use by TMA.
__device__ __forceinline__ void tensormap_acquire(const void* tmap) {
  asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(tmap) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(void* dst_smem, uint32_t ncols) {   // one full warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
               "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {  // one full warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem], M = 128, K = 16, bf16 x bf16 -> f32; issued by one thread.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       bool accumulate) {
  // (no lane mask operand: the issuing lane shares its scheduler with arithmetic warps, and every register the
  // instruction names is one more move into the uniform file to wait an issue slot for)
  const uint32_t acc = accumulate ? 1u : 0u;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}
// Same with the A operand in TMEM: lane = row, two bf16 per 32-bit column, 8 columns per K = 16 step.
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                       bool accumulate) {
  const uint32_t acc = accumulate ? 1u : 0u;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}
// The mbarrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(void* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

#define EA_R16(r, o) "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), \
  "=r"(r[o + 6]), "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]),               \
  "=r"(r[o + 12]), "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15])
#define EA_W16(r, o) "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]),       \
  "r"(r[o + 6]), "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]), "r"(r[o + 12]),      \
  "r"(r[o + 13]), "r"(r[o + 14]), "r"(r[o + 15])

// 16 consecutive fp32 columns of this thread's TMEM lane (warp w reads lanes 32w..32w+31).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : EA_R16(r, 0)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
      ::EA_W16(r, 0),
      "r"(taddr)
      : "memory");
}
// 8 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
// 64 consecutive columns: four loads in flight before the caller waits once.
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t (&r)[64]) {
#pragma unroll
  for (int k = 0; k < 4; ++k) tmem_ld16(taddr + 16 * k, *reinterpret_cast<uint32_t(*)[16]>(&r[16 * k]));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Register reallocation between the warpgroups of a CTA: every warp of a warpgroup executes the same one.
template <int N>
__device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Three-input maximum and two-wide fp32 arithmetic (one instruction for a pair of lanes' values).
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// (y0, y1) = (x0, x1) * s + m
__device__ __forceinline__ void fma2(float& y0, float& y1, float x0, float x1, float s, float m) {
  asm("{\n\t.reg .b64 a, b, c, d;\n\t"
      "mov.b64 a, {%2, %3};\n\tmov.b64 b, {%4, %4};\n\tmov.b64 c, {%5, %5};\n\t"
      "fma.rn.f32x2 d, a, b, c;\n\tmov.b64 {%0, %1}, d;\n\t}"
      : "=f"(y0), "=f"(y1)
      : "f"(x0), "f"(x1), "f"(s), "f"(m));
}
// (s0, s1) += (x0, x1)
__device__ __forceinline__ void add2(float& s0, float& s1, float x0, float x1) {
  asm("{\n\t.reg .b64 a, b, d;\n\t"
      "mov.b64 a, {%0, %1};\n\tmov.b64 b, {%2, %3};\n\tadd.rn.f32x2 d, a, b;\n\tmov.b64 {%0, %1}, d;\n\t}"
      : "+f"(s0), "+f"(s1)
      : "f"(x0), "f"(x1));
}
// The same on values kept packed in 64-bit registers (low word = first lane).
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2p(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add2p(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long mul2p(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  const __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// ---------------------------------------------------------------- descriptors

// Shared-memory matrix descriptor, no swizzle: start address, leading-dimension byte offset (LBO),
// stride-dimension byte offset (SBO), all in units of 16 bytes; bits 46-47 hold the descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return static_cast<uint64_t>((saddr >> 4) & 0x3FFFu) | (static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         (static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// Same for the 128-byte swizzle (bits 61-63 = 2): rows of 128 bytes whose 16-byte chunks are permuted by
// chunk ^= row % 8; tiles must start on a 1024-byte boundary.  K-major operands: SBO = stride between
// 8-row groups, LBO unused.  MN-major operands: LBO = stride between 64-element atoms along MN, SBO =
// stride between 8-row groups along K.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return smem_desc(saddr, lbo_bytes, sbo_bytes) | (2ull << 61);
}
// Byte offset of chunk c (16 bytes) of row `row` inside a 128-byte-swizzled atom column of dense rows.
__device__ __forceinline__ uint32_t sw128_off(int row, int c) {
  return static_cast<uint32_t>((row << 7) + ((c ^ (row & 7)) << 4));
}
// Instruction descriptor, kind::f16: f32 accumulator, bf16 A and B, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(kTile >> 4) << 24);
}

// The same with fp16 A and B (format fields 0): for operands a kernel writes itself and wants three more mantissa
// bits in than bf16 gives (both operands of one product always have the same type).
__host__ __device__ constexpr uint32_t instr_desc_f16(int n) {
  return (1u << 4) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kTile >> 4) << 24);
}

// Canonical tile: chunk (row, c) of 16 bytes lives at (row/8) * group_stride + c * 128 + (row%8) * 16,
// i.e. the core matrices of an 8-row group are contiguous.
__device__ __forceinline__ uint32_t chunk_off(int row, int c, int group_stride) {
  return static_cast<uint32_t>((row >> 3) * group_stride + (c << 7) + ((row & 7) << 4));
}

// Copies `rows_valid` rows of a row-major bf16 matrix (row pitch `rp` elements) into a canonical tile of
// 128 rows x `nch` chunks; rows and chunks past the source are zero.
__device__ __forceinline__ void load_tile(unsigned char* dst, const __nv_bfloat16* src, int rp, int rows_valid,
                                          int nch, int tid) {
  const int src_chunks = rp >> 3;
  const int group_stride = nch << 7;
  for (int idx = tid; idx < kTile * nch; idx += kThreads) {
    const int c = idx >> 7, row = idx & (kTile - 1);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < rows_valid && c < src_chunks)
      v = __ldg(reinterpret_cast<const uint4*>(src + static_cast<int64_t>(row) * rp) + c);
    *reinterpret_cast<uint4*>(dst + chunk_off(row, c, group_stride)) = v;
  }
}

// Moves a tile of 128 rows from row-major form (row pitch `rowb` bytes, a multiple of 16) into the canonical
// core-matrix layout, by four warps.  A warp instruction takes a block of 8 rows x 4 chunks: lane = (row % 8) +
// 8 * (chunk % 4).  For pitches of 32 bytes modulo 64 (ranks 48, 80, 112) both the reads and the writes then spread
// evenly over the banks; lane = row would read with an 8-way conflict.
__device__ __forceinline__ void relayout_tile(unsigned char* dst, const unsigned char* src, int rowb, int group_stride,
                                              int warp, int lane) {
  const int chunks = rowb >> 4;
  const int blocks = 16 * ((chunks + 3) >> 2);               // 16 row groups x quads of chunks
  const int r8 = lane & 7, cc = lane >> 3;
  for (int b0 = warp; b0 < blocks; b0 += 16) {               // four blocks in flight per warp
    uint4 tmp[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int b = b0 + 4 * u, c = ((b >> 4) << 2) + cc, row = ((b & 15) << 3) + r8;
      if (b < blocks && c < chunks) tmp[u] = *reinterpret_cast<const uint4*>(src + row * rowb + (c << 4));
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int b = b0 + 4 * u, c = ((b >> 4) << 2) + cc, row = ((b & 15) << 3) + r8;
      if (b < blocks && c < chunks) *reinterpret_cast<uint4*>(dst + chunk_off(row, c, group_stride)) = tmp[u];
    }
  }
}

struct __align__(16) TcSmemHeader {
  unsigned long long bar;
  uint32_t tmem_base;
  int abort_flag;
};

}  // namespace tc
}  // namespace ea
