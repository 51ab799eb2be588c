// Thin inline-PTX layer over the Blackwell (sm_100a) tensor-core path: tensor memory
// (TMEM) allocation and access, tcgen05.mma issue with shared-memory / TMEM operands,
// commit-to-mbarrier, and the shared-memory operand layout used by the refresh kernel.
#pragma once
#include <cstdint>

namespace tc5 {

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier -----------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
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

// One non-blocking look at the barrier (try_wait may suspend the thread for a while before it answers; this does not).
__device__ __forceinline__ bool mbar_test_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait: gives up after `max_polls` polls (each poll may itself block for a
// hardware-defined time slice) and reports failure instead of spinning for ever.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, uint32_t max_polls) {
  for (uint32_t i = 0; i < max_polls; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

// ---- TMA (bulk tensor copies into this CTA's shared memory, completing on an mbarrier; one CTA, one destination) ----
// The issuing thread announces the bytes of the copy it is about to start (this is also its arrival).
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Tiled load of one box; x is the innermost coordinate (x * element size must be a multiple of 16 bytes).
__device__ __forceinline__ void tma_load_3d(uint32_t dst_smem, const void *tmap, int32_t x, int32_t y, int32_t z,
                                            uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          dst_smem),
      "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst_smem, const void *tmap, int32_t x, int32_t y, int32_t z, int32_t w,
                                            uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(
          dst_smem),
      "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar))
      : "memory");
}

// ---- proxies and tcgen05 fences -------------------------------------------------------------
// Generic-proxy shared-memory writes -> visible to the tensor core (async proxy).
__device__ __forceinline__ void fence_smem_to_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- tensor memory --------------------------------------------------------------------------
// One full warp allocates `ncols` (power of two, 32..512) columns; the base address lands in *dst_smem.
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// 32 lanes x 32 consecutive columns: thread i of the warp gets lane (base lane + i), columns c..c+31.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,"
      "%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
// 32 lanes x 16 consecutive columns.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,"
      "%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- operands -------------------------------------------------------------------------------
// fp32 -> tf32.  The tensor cores read a tf32 operand from an fp32 container by ignoring the low
// 13 mantissa bits, so adding half a tf32 ulp to the bit pattern beforehand turns that truncation
// into round-to-nearest (ties away).  Plain integer arithmetic: cvt.rna.tf32.f32 was measured to
// cost an order of magnitude more issue time on this part.
// tf32_pre(x): container whose truncation is the rounded value (for operands only tensor cores read).
__device__ __forceinline__ uint32_t tf32_pre(float x) { return __float_as_uint(x) + 0x1000u; }
// to_tf32(x): the rounded value itself, low 13 bits cleared.
__device__ __forceinline__ uint32_t to_tf32(float x) { return (__float_as_uint(x) + 0x1000u) & 0xFFFFE000u; }

// Shared-memory operand tiles use the 128-byte-swizzle canonical layout.  A tile of R rows
// and 32*NB tf32 columns is stored as NB blocks of [R rows][128 bytes]; inside a block the
// 16-byte chunk j of row r sits at chunk position j ^ (r & 7).  Blocks start 1024-byte aligned.
// These tiles are used as K-major operands (rows = M or N index, columns = K).  A tf32 MN-major
// operand would need a different swizzle (128-byte swizzle on 32-byte units), so a matrix that is
// consumed in both orientations is stored twice.
__device__ __forceinline__ uint32_t sw128_offset(uint32_t rows, uint32_t r, uint32_t col) {
  const uint32_t blk = col >> 5, cin = col & 31;
  return blk * rows * 128u + r * 128u + ((((cin >> 2) ^ (r & 7u)) << 4) | ((cin & 3u) << 2));
}

// The same canonical K-major layout for 16-bit elements: 64 columns per 128-byte row.  `col` must be a multiple of 4
// (8 bytes) for the 8-byte accesses made here.
__device__ __forceinline__ uint32_t sw128_offset_bf16(uint32_t rows, uint32_t r, uint32_t col) {
  const uint32_t blk = col >> 6, cin = col & 63;
  return blk * rows * 128u + r * 128u + ((((cin >> 3) ^ (r & 7u)) << 4) | ((cin & 7u) << 1));
}

// MN-major tf32 operand tiles (rows = K index, the M or N index contiguous along a row): the tensor core accepts one
// swizzle for them, the 128-byte swizzle on 32-byte units.  A tile of R rows (the K index) and 32*NB tf32 columns is
// stored as NB blocks of [R rows][128 bytes]; inside a block the 32-byte unit u of row r sits at unit position
// u ^ (r & 3).  Blocks start 1024-byte aligned.  `col` must be a multiple of 4 (a 16-byte vector).
__device__ __forceinline__ uint32_t mn32_offset(uint32_t rows, uint32_t r, uint32_t col) {
  const uint32_t blk = col >> 5, cin = col & 31;
  return blk * rows * 128u + r * 128u + ((((cin >> 3) ^ (r & 3u)) << 5) | (((cin >> 2) & 1u) << 4));
}

constexpr uint64_t kDescSw128 = (uint64_t{1} << 46) | (uint64_t{2} << 61);  // version 1, SWIZZLE_128B

// K-major: 8-row groups are 1024 bytes apart (SBO); LBO is not used with swizzling.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t smem_addr) {
  return kDescSw128 | (uint64_t{(smem_addr & 0x3FFFFu) >> 4}) | (uint64_t{1} << 16) | (uint64_t{1024 >> 4} << 32);
}
// MN-major, 128-byte swizzle on 32-byte units: groups of 4 K rows are 512 bytes apart (SBO), blocks of 32 elements
// along M/N are `block_bytes` apart (LBO).  `smem_addr` points at the first K row of the slice.
constexpr uint64_t kDescSw128Base32 = (uint64_t{1} << 46) | (uint64_t{1} << 61);  // version 1, SWIZZLE_128B_BASE32B
__device__ __forceinline__ uint64_t desc_mn32(uint32_t smem_addr, uint32_t block_bytes) {
  return kDescSw128Base32 | (uint64_t{(smem_addr & 0x3FFFFu) >> 4}) | (uint64_t{block_bytes >> 4} << 16) |
         (uint64_t{512 >> 4} << 32);
}
// Instruction descriptor, kind::tf32, fp32 accumulation.
__host__ __device__ constexpr uint32_t idesc_tf32(uint32_t M, uint32_t N, bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | (2u << 7) | (2u << 10) | (uint32_t(a_mn_major) << 15) | (uint32_t(b_mn_major) << 16) |
         ((N >> 3) << 17) | ((M >> 4) << 24);
}

// Instruction descriptor, kind::f16 with bf16 operands (both K-major), fp32 accumulation.
__host__ __device__ constexpr uint32_t idesc_bf16(uint32_t M, uint32_t N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((N >> 3) << 17) | ((M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem], bf16 operands; one K = 16 slice.
__device__ __forceinline__ void mma_ss_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(uint32_t(accumulate))
      : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]; one K = 8 slice.  Issued by a single thread.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(uint32_t(accumulate))
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]; A is M lanes x 8 columns at a_tmem.
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(uint32_t(accumulate))
      : "memory");
}
// All MMAs issued so far by this thread arrive on `bar` when they have completed.
__device__ __forceinline__ void mma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

}  // namespace tc5
