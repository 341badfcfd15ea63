// 5th-generation tensor core primitives (tcgen05, sm_100a): shared-memory matrix descriptors,
// instruction descriptors, tensor-memory (TMEM) allocation, asynchronous MMA issue, completion
// through an mbarrier with a bounded wait, and TMEM -> register loads.
//
// Operands live in shared memory as bf16 in the canonical no-swizzle layout: 8 x 8 "core matrices"
// of 128 contiguous bytes (8 rows of 16 bytes).  One image of a matrix X, img(i, j), serves every
// role a product can ask of it, selected by the descriptor alone:
//   A = X      K-major A      B = X^T (B(k,n) = X[n][k])   K-major B
//   A = X^T    MN-major A     B = X   (B(k,n) = X[k][n])   MN-major B
#pragma once
#include "ln_common.cuh"

namespace ln {
namespace umma {

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// element offset of (i, j) in the image of a matrix with `cols` columns (cols % 8 == 0)
__device__ __forceinline__ int img(int i, int j, int cols) { return ((i >> 3) * (cols >> 3) + (j >> 3)) * 64 + (i & 7) * 8 + (j & 7); }

// 64-bit shared-memory matrix descriptor (no swizzle).  lbo: byte stride between core matrices along
// K, sbo: along M/N.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of sm_100
  return d;
}

// Descriptor of K-step `ks` (16 elements of K per MMA) of an image with `cols` columns.
//   kmajor = true : rows of the image are M/N, columns are K   (A = X, or B = X^T)
//   kmajor = false: rows of the image are K, columns are M/N   (A = X^T, or B = X)
__device__ __forceinline__ uint64_t operand_desc(const bf16* image, int cols, bool kmajor, int ks) {
  const uint32_t row_group = (uint32_t)(cols >> 3) * 128;          // bytes between 8-row groups of the image
  if (kmajor) return smem_desc(s32(image) + (uint32_t)ks * 256, 128, row_group);
  return smem_desc(s32(image) + (uint32_t)ks * 2 * row_group, row_group, 128);
}

// Instruction descriptor, kind::f16: fp32 accumulate, bf16 operands, M = 128 (accumulator row r in TMEM lane r) or
// M = 64 (row r in lane 32 (r / 16) + r % 16: each warp quarter holds 16 rows in its first 16 lanes).
__device__ __forceinline__ uint32_t instr_desc(int N, bool a_mn_major, bool b_mn_major, int M = 128) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A * B for one K-step; issued by ONE thread.
__device__ __forceinline__ void mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate ? 1u : 0u) : "memory");
}
// Arrive on `mbar` when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void commit(unsigned long long* mbar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(mbar)) : "memory");
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// shared-memory writes of this thread (generic proxy) become visible to the tensor core (async proxy)
__device__ __forceinline__ void fence_smem_to_mma() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(unsigned long long* mbar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(mbar)), "r"(count));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// Bounded wait for phase `parity`; returns false if the limit ran out (the caller records an error
// and carries on: results are then wrong but nothing spins for ever).
__device__ __forceinline__ bool mbar_wait(unsigned long long* mbar, uint32_t parity, int limit = 1 << 22) {
  uint32_t done = 0;
  for (int it = 0; it < limit && !done; ++it)
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(s32(mbar)), "r"(parity) : "memory");
  return done != 0;
}

// Bulk copy global -> shared of `bytes` (a multiple of 16, both addresses 16-byte aligned) by ONE thread; the
// bytes are counted on `mbar`, which must have been told to expect them (expect_tx) beforehand.
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* mbar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(mbar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, unsigned long long* mbar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(s32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(s32(mbar)) : "memory");
}

// Bulk copy shared -> global by ONE thread, as one bulk group; bulk_store_wait_read() returns once every group this
// thread issued has finished READING shared memory (the buffer may then be overwritten).
__device__ __forceinline__ void bulk_store(void* dst_gmem, const void* src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_gmem), "r"(s32(src_smem)), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// TMEM allocation (whole warp; ncols a power of two in [32, 512]); the base address lands in *slot.
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, int ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(slot)), "r"(ncols));
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, int ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(ncols));
}

// 32 consecutive fp32 columns of this thread's TMEM lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(r[q]);
}
// TMEM address of (lane quarter of this warp, column)
__device__ __forceinline__ uint32_t tmem_addr(uint32_t base, int col) {
  return base + ((uint32_t)(((threadIdx.x >> 5) & 3) * 32) << 16) + (uint32_t)col;
}

}  // namespace umma
}  // namespace ln
