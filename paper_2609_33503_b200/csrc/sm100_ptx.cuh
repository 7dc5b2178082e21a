// Thin inline-PTX wrappers for the Blackwell (sm_100a) primitives the kernels use: mbarrier, TMA
// tiled loads (never multicast), tensor memory (TMEM) management, tcgen05.mma / ld / st / commit,
// and the shared-memory / instruction descriptors of the 5th-generation tensor cores.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace relaxkv {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Three-input maximum (one instruction on sm_100).
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Packed fp32 pairs (one instruction for two elements): d = a * b + c and d += a.
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1) {
  asm("{\n\t.reg .b64 ra, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rd, {%0, %1};\n\tadd.rn.f32x2 rd, rd, ra;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "+f"(d0), "+f"(d1) : "f"(a0), "f"(a1));
}

// Per-warpgroup register re-allocation (all four warps of the warpgroup must execute it).
template <int N> __device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// ---- mbarrier -----------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}

// Bounded wait: gives up after `limit_ns`, or as soon as another thread of the block has given up
// (*abort_flag != 0).  Returns false in that case; the caller leaves its loop and goes to teardown.
constexpr uint64_t kWaitLimitNs = 400ull * 1000 * 1000;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if ((it & 63u) == 0u && global_timer_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
  }
}

// ---- TMA (tiled, this CTA only) ---------------------------------------------------------------
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// ---- untiled bulk copies (this GPU's memory only, never multicast): whole rows global -> shared -> global ---------
// Both addresses 16-byte aligned, size a multiple of 16 bytes.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes) : "memory");
}
// Commits this thread's bulk stores and waits until they have READ their shared-memory source (it may then be reused
// or the block may exit; the global writes complete on their own).
__device__ __forceinline__ void bulk_store_commit_and_drain() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// ---- tensor memory ------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols) {   // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {                                    // whole warp
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {         // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (base lane + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// ---- tcgen05.mma (issued by one thread) -----------------------------------------------------------
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier receives one arrival once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// ---- batched issue: several tcgen05.mma from ONE asm statement ------------------------------------------
// The issuing thread is a single lane, so every instruction it spends on descriptor arithmetic delays
// the next MMA.  A descriptor's low word holds the (address >> 4); stepping along K only adds a small
// constant to it, so a whole K-loop is emitted as add / mov.b64 / mma triples with immediates.
//   lo word: (smem address >> 4) | (leading byte offset >> 4) << 16      hi word: see desc_hi_sw128()
__host__ __device__ constexpr uint32_t desc_hi_sw128(uint32_t sbo_bytes) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);        // stride offset | version | 128B swizzle
}
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
  return ((smem_addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}

#define RELAXKV_MMA_SS_STEP(OFF, PRED)                                                         \
  "add.u32 ta, %1, " #OFF ";\n\tadd.u32 tb, %2, " #OFF ";\n\t"                                    \
  "mov.b64 da, {ta, %3};\n\tmov.b64 db, {tb, %3};\n\t"                                           \
  "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, " #PRED ";\n\t"

// D[tmem] = A[smem] * B[smem] over K = 64 * HALVES (both operands K-major, 128B swizzle, halves 16 KB apart
// for A when a_half_step16 = 1024 and for B when the same): the first MMA overwrites D.
template <int HALVES>
__device__ __forceinline__ void mma_ss_kloop(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc) {
  if (HALVES == 2) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 ta, tb;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p0, 0, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        RELAXKV_MMA_SS_STEP(0, p0) RELAXKV_MMA_SS_STEP(2, p1) RELAXKV_MMA_SS_STEP(4, p1) RELAXKV_MMA_SS_STEP(6, p1)
        RELAXKV_MMA_SS_STEP(1024, p1) RELAXKV_MMA_SS_STEP(1026, p1) RELAXKV_MMA_SS_STEP(1028, p1) RELAXKV_MMA_SS_STEP(1030, p1)
        "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b32 ta, tb;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p0, 0, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        RELAXKV_MMA_SS_STEP(0, p0) RELAXKV_MMA_SS_STEP(2, p1) RELAXKV_MMA_SS_STEP(4, p1) RELAXKV_MMA_SS_STEP(6, p1)
        "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
  }
}

// D[tmem] (+)= A[smem] * B[smem] for four K steps of 16 inside one 64-element (128-byte) swizzled K block.
// acc_first = 0 makes the first MMA overwrite D.
__device__ __forceinline__ void mma_ss_4steps(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                              uint32_t acc_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b32 ta, tb;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      RELAXKV_MMA_SS_STEP(0, p0) RELAXKV_MMA_SS_STEP(2, p1) RELAXKV_MMA_SS_STEP(4, p1) RELAXKV_MMA_SS_STEP(6, p1)
      "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc_first) : "memory");
}

#define RELAXKV_MMA_TS_STEP(AOFF, BOFF, PRED)                                                  \
  "add.u32 ta, %1, " #AOFF ";\n\tadd.u32 tb, %2, " #BOFF ";\n\t"                                  \
  "mov.b64 db, {tb, %3};\n\t"                                                                  \
  "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %4, " #PRED ";\n\t"

// D[tmem] (+)= A[tmem] * B[smem] for four K steps of 16: A advances 8 columns, B (MN-major, 128B swizzle)
// 2048 bytes per step.  acc_first = 0 makes the first MMA overwrite D.
__device__ __forceinline__ void mma_ts_4steps(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                              uint32_t acc_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b32 ta, tb;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      RELAXKV_MMA_TS_STEP(0, 0, p0) RELAXKV_MMA_TS_STEP(8, 128, p1) RELAXKV_MMA_TS_STEP(16, 256, p1) RELAXKV_MMA_TS_STEP(24, 384, p1)
      "}" ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc_first) : "memory");
}

// ---- CTA pairs (cta_group::2): one MMA instruction drives the tensor cores of two SMs ----------------------
// A cluster of two CTAs; rank 0 (the leader) issues.  For M = 256 each CTA supplies 128 rows of A (its own shared
// memory or TMEM, same offsets in both), HALF of B's N rows from its own shared memory, and receives its 128 rows
// of D (all N columns) in its own TMEM.  alloc / dealloc are executed by one warp of EACH CTA.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync() {      // every thread of both CTAs
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cta address -> the same offset in CTA `rank` of the cluster (a shared::cluster address)
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// One arrival on a barrier of another CTA of the cluster.  Default qualifiers (release at CTA scope): a cluster-scope
// release on every arrival measured ~2x slower kernels (each arrival then waits for the thread's earlier writes to
// become visible cluster-wide); the data handed over here lives in tensor memory or was written by TMA and is ordered
// by tcgen05.fence / the mbarrier's own completion.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// bounded wait on a barrier that also receives arrivals from the other CTA of the cluster
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if (*abort_flag) return false;
    if ((it & 63u) == 0u && global_timer_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
  }
}
__device__ __forceinline__ void tmem_alloc2(uint32_t smem_result, uint32_t ncols) {   // whole warp, in each CTA
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// One arrival on the barrier at this offset in every CTA of `mask`, once all MMAs issued so far have completed.
// (A commit with cluster multicast, not a multicast copy: nothing is loaded.)
__device__ __forceinline__ void mma_commit2_mc(uint32_t bar, uint16_t mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
#define RELAXKV_MMA2_SS_STEP(AOFF, BOFF, PRED)                                               \
  "add.u32 ta, %1, " #AOFF ";\n\tadd.u32 tb, %2, " #BOFF ";\n\t"                                  \
  "mov.b64 da, {ta, %3};\n\tmov.b64 db, {tb, %3};\n\t"                                           \
  "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, " #PRED ";\n\t"
// D[tmem] = A[smem] * B[smem] over K = 128 (two 64-element halves; A's halves 16 KB apart, B's 8 KB: this CTA's
// 64 of the tile's 128 N rows): the first MMA overwrites D.
__device__ __forceinline__ void mma2_ss_kloop(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b32 ta, tb;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p0, 0, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      RELAXKV_MMA2_SS_STEP(0, 0, p0) RELAXKV_MMA2_SS_STEP(2, 2, p1) RELAXKV_MMA2_SS_STEP(4, 4, p1) RELAXKV_MMA2_SS_STEP(6, 6, p1)
      RELAXKV_MMA2_SS_STEP(1024, 512, p1) RELAXKV_MMA2_SS_STEP(1026, 514, p1) RELAXKV_MMA2_SS_STEP(1028, 516, p1)
      RELAXKV_MMA2_SS_STEP(1030, 518, p1)
      "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem] for four K steps of 16 inside one 64-element swizzled K block (both K-major).
__device__ __forceinline__ void mma2_ss_4steps(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                               uint32_t acc_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b32 ta, tb;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      RELAXKV_MMA2_SS_STEP(0, 0, p0) RELAXKV_MMA2_SS_STEP(2, 2, p1) RELAXKV_MMA2_SS_STEP(4, 4, p1) RELAXKV_MMA2_SS_STEP(6, 6, p1)
      "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc_first) : "memory");
}
#define RELAXKV_MMA2_TS_STEP(AOFF, BOFF, PRED)                                               \
  "add.u32 ta, %1, " #AOFF ";\n\tadd.u32 tb, %2, " #BOFF ";\n\t"                                  \
  "mov.b64 db, {tb, %3};\n\t"                                                                  \
  "tcgen05.mma.cta_group::2.kind::f16 [%0], [ta], db, %4, " #PRED ";\n\t"
// D[tmem] (+)= A[tmem] * B[smem] for four K steps of 16: A advances 8 columns, B (MN-major) 2048 bytes per step.
__device__ __forceinline__ void mma2_ts_4steps(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                               uint32_t acc_first) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b32 ta, tb;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
      RELAXKV_MMA2_TS_STEP(0, 0, p0) RELAXKV_MMA2_TS_STEP(8, 128, p1) RELAXKV_MMA2_TS_STEP(16, 256, p1) RELAXKV_MMA2_TS_STEP(24, 384, p1)
      "}" ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc_first) : "memory");
}

// ---- descriptors ------------------------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle, tiles whose 8-row groups are 1024 bytes apart.
//   K-major operand  (rows of 64 bf16 = 128 B):       lbo ignored (1),  sbo = 1024
//   MN-major operand (64 contiguous MN elements per K row): lbo = bytes between 64-element MN blocks,
//                                                           sbo = 1024 (between groups of 8 K rows)
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr >> 4) & 0x3FFFu);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;      // descriptor version of this architecture
  d |= 2ull << 61;      // 128-byte swizzle
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, dense.
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int m, int n, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(b_mn_major) << 16) |
         (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

}  // namespace ptx
}  // namespace relaxkv
