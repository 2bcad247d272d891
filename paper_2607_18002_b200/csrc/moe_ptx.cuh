// Inline-PTX wrappers for the sm_100a features the persistent kernel uses: mbarriers, tiled
// and gather4 TMA loads, tcgen05 (UMMA) issue / commit / TMEM loads, proxy fences and
// scoped loads and stores.
#pragma once
#include <cuda.h>
#include <stdint.h>

namespace moe {

__device__ __forceinline__ unsigned smem_u32(const void* p) {
  return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(void* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(void* bar, unsigned n) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(n) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try(void* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// non-blocking test of a phase (try_wait may suspend the thread for a while)
__device__ __forceinline__ bool mbar_test(void* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tma_tile_2d(void* dst, const CUtensorMap* tm, int x, int y,
                                            void* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4];" ::"r"(smem_u32(dst)),
      "l"(tm), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
// L2 prefetch of one tensor-map box: no shared memory, no barrier
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* tm, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tm), "r"(x),
               "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_gather4(void* dst, const CUtensorMap* tm, int x, int4 rows,
                                            void* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(smem_u32(dst)),
      "l"(tm), "r"(x), "r"(rows.x), "r"(rows.y), "r"(rows.z), "r"(rows.w), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(void* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(unsigned d_tmem, unsigned long long adesc,
                                            unsigned long long bdesc, unsigned idesc,
                                            unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_mma_f8(unsigned d_tmem, unsigned long long adesc,
                                          unsigned long long bdesc, unsigned idesc,
                                          unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_st32(unsigned taddr, const unsigned (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
      "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
      "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
      "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tc_wait_st() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_ld32(unsigned taddr, unsigned (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
        "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]),
        "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_ld16(unsigned taddr, unsigned (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
        "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]),
        "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}
__device__ __forceinline__ void prefetch_l1(const void* p) {
  asm volatile("prefetch.global.L1 [%0];" ::"l"(p));
}
__device__ __forceinline__ void cp_async_16(unsigned dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
// the mbarrier receives one arrival when all cp.async issued so far by this thread have landed
__device__ __forceinline__ void cp_async_arrive_noinc(void* bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait_group() {
  asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.wait_all;" ::: "memory");
}
__device__ __forceinline__ void fence_async_proxy_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void fence_async_proxy() {
  asm volatile("fence.proxy.async;" ::: "memory");
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_acquire_sys(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_sys(unsigned* p, unsigned v) {
  asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_volatile(const int* p) {
  return *reinterpret_cast<const volatile int*>(p);
}

// UMMA shared-memory descriptor of a K-major operand whose rows are row_bytes (64 or 128)
// wide and swizzled with the matching pattern; 8-row groups lie 8 * row_bytes apart.
__device__ __forceinline__ unsigned long long umma_desc(unsigned saddr, unsigned row_bytes) {
  unsigned long long d = (unsigned long long)((saddr & 0x3ffffu) >> 4);
  d |= 1ull << 16;                                   // leading byte offset (unused for swizzled K-major)
  d |= (unsigned long long)((8u * row_bytes) >> 4) << 32;   // stride byte offset between 8-row groups
  d |= 1ull << 46;                                   // descriptor version (sm_100)
  d |= (row_bytes == 128u ? 2ull : 4ull) << 61;      // SWIZZLE_128B : SWIZZLE_64B
  return d;
}
// instruction descriptor: D fp32, A/B bf16, both K-major, M = 128, N = 256
constexpr unsigned kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);



// ------------------------------------------------------------------ CTA pairs (cluster of two)
__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {      // every thread of both CTAs
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ unsigned map_to_cta(const void* p, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(unsigned cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(unsigned cluster_addr, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// the same two without cluster-scope release: for pipeline barriers whose data moves by TMA or cp.async
__device__ __forceinline__ void mbar_arrive_remote(unsigned cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_remote(unsigned cluster_addr, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// wait that synchronises with arrivals made by the other CTA of the pair
__device__ __forceinline__ bool mbar_try_cluster(void* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void st_cluster_v4(unsigned cluster_addr, uint4 v) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// tiled TMA load by either CTA of a pair; the transaction bytes go to the barrier at `bar_cluster_addr`
// (the pair leader's), the data to this CTA's own shared memory
__device__ __forceinline__ void tma_tile_2d_pair(void* dst, const CUtensorMap* tm, int x, int y, unsigned bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(smem_u32(dst)),
      "l"(reinterpret_cast<unsigned long long>(tm)), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
// one MMA of the pair: M = 256 or 128 rows split over the two CTAs, both halves of B read from the two CTAs
__device__ __forceinline__ void tc_mma2_bf16(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,
                                             unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the barrier at the same shared-memory offset in both CTAs once the pair's MMAs so far retire
__device__ __forceinline__ void tc_commit_pair(void* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}

// ---- warp-uniform issue: the whole warp executes these, one elected lane issues the instruction.
// Their operands then stay warp-uniform for the compiler (no per-thread staging of descriptors),
// which keeps the issue loops of the MMA and producer warps short.
__device__ __forceinline__ void tc_mma2_bf16_elect(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,
                                                   unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .b32 r;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair_elect(void* bar) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t.reg .b32 r;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "@e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}" ::"r"(smem_u32(bar)),
      "h"((unsigned short)3)
      : "memory");
}
__device__ __forceinline__ void tma_tile_2d_pair_elect(unsigned dst_smem, const CUtensorMap* tm, int x, int y, unsigned bar_cluster_addr) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t.reg .b32 r;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "@e cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n\t}" ::"r"(dst_smem),
      "l"(reinterpret_cast<unsigned long long>(tm)), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_addr_elect(unsigned cluster_addr, unsigned bytes) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t.reg .b32 r;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "@e mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;\n\t}" ::"r"(cluster_addr), "r"(bytes)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_n_elect(void* bar, unsigned n) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t.reg .b32 r;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "@e mbarrier.arrive.shared::cta.b64 _, [%0], %1;\n\t}" ::"r"(smem_u32(bar)), "r"(n)
      : "memory");
}

// All loads and barrier arrivals of one k-block by one CTA of a pair, as ONE instruction group under a
// single election: expect_tx on the leader's stage barrier, up to two weight boxes, up to two
// activation boxes, the stand-in arrivals (tiles without a gather) and the go-ahead for the gather warps.
// Flags select what is issued; everything is warp-uniform.
__device__ __forceinline__ void pair_issue_kblock(unsigned bar, unsigned tx, unsigned standin_bar, unsigned standin_n,
                                                  unsigned sB, const CUtensorMap* tmw, int x, int wy0, int wy1, unsigned has_w1,
                                                  unsigned sA, const CUtensorMap* tma, int ay, unsigned a_boxes,
                                                  unsigned go_bar, unsigned has_go) {
  asm volatile(
      "{\n\t.reg .pred e, pw1, pa1, pa2, pgo, pst;\n\t.reg .b32 r, sB1, sA1, ay1;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "setp.ne.and.b32 pw1, %9, 0, e;\n\t"
      "setp.ge.and.u32 pa1, %13, 1, e;\n\t"
      "setp.ge.and.u32 pa2, %13, 2, e;\n\t"
      "setp.ne.and.b32 pgo, %15, 0, e;\n\t"
      "setp.ne.and.b32 pst, %3, 0, e;\n\t"
      "add.u32 sB1, %4, 8192;\n\t"
      "add.u32 sA1, %10, 4096;\n\t"
      "add.s32 ay1, %12, 32;\n\t"
      "@e mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;\n\t"
      "@pst mbarrier.arrive.shared::cta.b64 _, [%2], %3;\n\t"
      "@e cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%4], [%5, {%6, %7}], [%0];\n\t"
      "@pw1 cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [sB1], [%5, {%6, %8}], [%0];\n\t"
      "@pa1 cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%10], [%11, {%6, %12}], [%0];\n\t"
      "@pa2 cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [sA1], [%11, {%6, ay1}], [%0];\n\t"
      "@pgo mbarrier.arrive.shared::cta.b64 _, [%14];\n\t}"
      ::"r"(bar), "r"(tx), "r"(standin_bar), "r"(standin_n),
        "r"(sB), "l"(reinterpret_cast<unsigned long long>(tmw)), "r"(x), "r"(wy0), "r"(wy1), "r"(has_w1),
        "r"(sA), "l"(reinterpret_cast<unsigned long long>(tma)), "r"(ay), "r"(a_boxes),
        "r"(go_bar), "r"(has_go)
      : "memory");
}

// One k-block of the pair's MMAs as ONE instruction group: the next stage's barrier is tested first and
// the result is only read after the four MMAs and the commit have been issued, so that the barrier's
// shared-memory round trip hides behind the issue of the MMAs.  Whole warp, warp-uniform operands; one
// elected lane issues the MMAs and the commit.  Returns whether the next stage is already full.
__device__ __forceinline__ bool pair_mma_kblock(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,
                                                unsigned idesc, unsigned accumulate_first, unsigned empty_bar,
                                                unsigned next_full_bar, unsigned next_parity) {
  unsigned ready;
  asm volatile(
      "{\n\t.reg .pred e, p0, p1, pn;\n\t.reg .b32 r;\n\t.reg .b16 m;\n\t.reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
      "mov.b16 m, 3;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 pn, [%7], %8;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\t"
      "setp.eq.b32 p1, 0, 0;\n\t"
      "add.u64 a1, %2, 2;\n\tadd.u64 a2, %2, 4;\n\tadd.u64 a3, %2, 6;\n\t"
      "add.u64 b1, %3, 2;\n\tadd.u64 b2, %3, 4;\n\tadd.u64 b3, %3, 6;\n\t"
      "@e tcgen05.mma.cta_group::2.kind::f16 [%1], %2, %3, %4, p0;\n\t"
      "@e tcgen05.mma.cta_group::2.kind::f16 [%1], a1, b1, %4, p1;\n\t"
      "@e tcgen05.mma.cta_group::2.kind::f16 [%1], a2, b2, %4, p1;\n\t"
      "@e tcgen05.mma.cta_group::2.kind::f16 [%1], a3, b3, %4, p1;\n\t"
      "@e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%6], m;\n\t"
      "selp.u32 %0, 1, 0, pn;\n\t}"
      : "=r"(ready)
      : "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate_first), "r"(empty_bar),
        "r"(next_full_bar), "r"(next_parity)
      : "memory");
  return ready != 0;
}
// One e4m3 k-block (128 elements = four 32-element MMAs) into a fresh partial buffer, then the two
// commits (partial full, stage empty), as one group.  Whole warp, warp-uniform operands; one elected
// lane issues: instructions issued from a divergent single-lane branch cost about 100 clocks each.
__device__ __forceinline__ void f8_mma_kblock(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,
                                              unsigned idesc, unsigned pfull_bar, unsigned empty_bar) {
  asm volatile(
      "{\n\t.reg .pred e, p0, p1;\n\t.reg .b32 r;\n\t.reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "setp.ne.b32 p0, 0, 0;\n\t"
      "setp.eq.b32 p1, 0, 0;\n\t"
      "add.u64 a1, %1, 2;\n\tadd.u64 a2, %1, 4;\n\tadd.u64 a3, %1, 6;\n\t"
      "add.u64 b1, %2, 2;\n\tadd.u64 b2, %2, 4;\n\tadd.u64 b3, %2, 6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], a1, b1, %3, p1;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], a2, b2, %3, p1;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], a3, b3, %3, p1;\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%4];\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%5];\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(pfull_bar), "r"(empty_bar)
      : "memory");
}
// The loads of one k-block of the single-CTA kernel as ONE group: expect_tx, the two halves of the
// weight tile and (down tiles) the box of packed intermediate rows.  Whole warp, warp-uniform
// operands; one elected lane issues.
__device__ __forceinline__ void single_issue_kblock(unsigned bar, unsigned tx, unsigned sB0, unsigned sB1,
                                                    const CUtensorMap* tmw, int x, int wy0, int wy1, unsigned sA,
                                                    const CUtensorMap* tma, int ay, unsigned has_a) {
  asm volatile(
      "{\n\t.reg .pred e, pa;\n\t.reg .b32 r;\n\t"
      "elect.sync r|e, 0xffffffff;\n\t"
      "setp.ne.and.b32 pa, %11, 0, e;\n\t"
      "@e mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t"
      "@e cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%2], [%4, {%5, %6}], [%0];\n\t"
      "@e cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%3], [%4, {%5, %7}], [%0];\n\t"
      "@pa cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%8], [%9, {%5, %10}], [%0];\n\t}"
      ::"r"(bar), "r"(tx), "r"(sB0), "r"(sB1), "l"(reinterpret_cast<unsigned long long>(tmw)), "r"(x), "r"(wy0),
        "r"(wy1), "r"(sA), "l"(reinterpret_cast<unsigned long long>(tma)), "r"(ay), "r"(has_a)
      : "memory");
}
}  // namespace moe
