// Inline-PTX wrappers for sm_100a shared by the tensor-core kernels of librosaq: mbarriers, bulk and
// tensor copies, tcgen05 (allocation, MMA, commit, TMEM load/store), cluster helpers.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace rosaq {

// ---------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One poll of a barrier phase.  The suspend-time hint lets the hardware park the thread (up to about
// a microsecond, woken as soon as the phase completes) instead of returning at once: warps that wait
// then stop competing for issue slots with the warps that work.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(1000u)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// 3-D view {64 channels, tokens, 64-channel block} of the activations: one instruction fetches both
// 64-channel halves of a group (issuing a TMA costs the single producer lane a few hundred cycles)
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int tok, int blk) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::
          "r"(dst),
      "l"(map), "r"(bar), "r"(0), "r"(tok), "r"(blk)
      : "memory");
}
// The column count is an immediate on purpose: with a register operand the tools cannot see how much
// tensor memory a CTA takes and assume all 512 columns, which limits the kernel to one CTA per SM.
template <uint32_t kCols>
__device__ __forceinline__ void tmem_alloc(uint32_t holder_smem) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "n"(kCols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
template <uint32_t kCols>
__device__ __forceinline__ void tmem_dealloc(uint32_t addr) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "n"(kCols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]; fp16 inputs, fp32 accumulate.  The MMAs of one unit are
// emitted as one block of back-to-back instructions sharing their predicates: issued one by one from
// separate statements they cost the issuing thread about 100 cycles each, in a block about 45.
// A advances by 8 TMEM columns (16 input channels) per MMA; B by 32 bytes inside a 64-channel
// swizzle row (descriptor address field + 2), b_hi is the descriptor of the second 64-channel half.
__device__ __forceinline__ void tc_mma8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_lo, uint64_t b_hi,
                                           uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b64 t;\n\t.reg .b32 a;\n\t"
      "setp.ne.b32 p, %5, 0;\n\tsetp.eq.b32 q, 0, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %4, p;\n\t"
      "add.u32 a, %1, 8;\n\tadd.u64 t, %2, 2;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 16;\n\tadd.u64 t, %2, 4;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 24;\n\tadd.u64 t, %2, 6;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 32;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [a], %3, %4, q;\n\t"
      "add.u32 a, %1, 40;\n\tadd.u64 t, %3, 2;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 48;\n\tadd.u64 t, %3, 4;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 56;\n\tadd.u64 t, %3, 6;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [a], t, %4, q;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_lo), "l"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// ---- CTA pairs (cta_group::2): two CTAs of a cluster, ranks 2j and 2j + 1, drive one MMA stream
template <uint32_t kCols>
__device__ __forceinline__ void tmem_alloc_pair(uint32_t holder_smem) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "n"(kCols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
template <uint32_t kCols>
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "n"(kCols) : "memory");
}
// commit whose arrival is delivered to the barrier at the same offset in every CTA of `mask`
__device__ __forceinline__ void tc_commit_mc(uint32_t bar, uint32_t mask) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
      "h"((unsigned short)mask)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// load whose bytes are counted on a barrier of the pair's leader (a shared::cluster address); no multicast
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t lead_bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::
          "r"(dst),
      "l"(map), "r"(lead_bar), "r"(c0), "r"(c1)
      : "memory");
}
// 3-D form of the same: {64 channels, tokens, 64-channel block}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *map, uint32_t lead_bar, int tok, int blk) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::
          "r"(dst),
      "l"(map), "r"(lead_bar), "r"(0), "r"(tok), "r"(blk)
      : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(1000u)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tc_mma8_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_lo, uint64_t b_hi,
                                                uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b64 t;\n\t.reg .b32 a;\n\t"
      "setp.ne.b32 p, %5, 0;\n\tsetp.eq.b32 q, 0, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %4, p;\n\t"
      "add.u32 a, %1, 8;\n\tadd.u64 t, %2, 2;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 16;\n\tadd.u64 t, %2, 4;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 24;\n\tadd.u64 t, %2, 6;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 32;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], [a], %3, %4, q;\n\t"
      "add.u32 a, %1, 40;\n\tadd.u64 t, %3, 2;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 48;\n\tadd.u64 t, %3, 4;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], [a], t, %4, q;\n\t"
      "add.u32 a, %1, 56;\n\tadd.u64 t, %3, 6;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], [a], t, %4, q;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_lo), "l"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t *r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(
          taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t *r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t *r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void grid_dep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lop_and_or(uint32_t a, uint32_t mask, uint32_t orv) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(a), "r"(mask), "r"(orv));  // (a & mask) | orv
  return r;
}
__device__ __forceinline__ uint32_t h2_sub_mul(uint32_t v, uint32_t sub, uint32_t mul) {
  __half2 r = __hmul2(__hsub2(*reinterpret_cast<__half2 *>(&v), *reinterpret_cast<__half2 *>(&sub)),
                      *reinterpret_cast<__half2 *>(&mul));
  return *reinterpret_cast<uint32_t *>(&r);
}

// K-major, 128-byte-swizzled shared-memory operand: 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_b_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr >> 4) & 0x3fff) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

}  // namespace rosaq
