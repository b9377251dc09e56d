// Blackwell (sm_100a) primitives used by the kernels: mbarriers with bounded waits, TMA tile loads,
// tensor memory (TMEM) allocation and access, tcgen05 matrix-multiply issue, and the shared-memory /
// instruction descriptors those need.  Inline PTX only.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rbs {

// Kernels receive a pointer to the library's device status word: 0 = fine; otherwise the code of the
// first bounded wait that gave up (read back by rbs_device_status()).

enum : unsigned int {
  kWaitTmaFull = 1, kWaitStageFree = 2, kWaitMmaDone = 3, kWaitTmemFree = 4, kWaitPReady = 5, kWaitOReady = 6,
  kWaitSelfTest = 7,
};

// ------------------------------------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Waits for the phase with the given parity to complete.  Bounded: after kSpinLimit failed probes the
// wait gives up, records `code` in the device status word and returns false; callers then drain and exit.
constexpr uint32_t kSpinLimit = 1u << 24;
__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, unsigned int* status, unsigned int code,
                                                uint32_t limit) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 2048) __nanosleep(64);
    // once any wait anywhere has given up, the launch is lost: stop waiting everywhere
    if ((it & 255u) == 255u && *reinterpret_cast<volatile unsigned int*>(status) != 0u) return false;
  }
  atomicCAS(status, 0u, code);
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned int* status, unsigned int code) {
  return mbar_wait_limit(bar, parity, status, code, kSpinLimit);
}

// Debug build (-DRBS_DEBUG): index checks in the kernels.  A failing check records 0x100 + its site in the device
// status word (first failure wins), the caller skips the access and the kernel runs on: no trap, the context stays
// usable and rbs_device_status reports RBS_ERR_DEBUG_CHECK with the site.  In the release build the macro is the
// constant `true` and its condition is not even compiled.
enum DebugSite : unsigned int {
  kDbgStatsRow = 1,        // block statistics: output row past the end of centroid / radius
  kDbgSelectScore = 2,     // selector: score slot past the end of the row's L arrays in shared memory
  kDbgSelectPerm = 3,      // selector: block index of an accumulator row outside the padded row count
  kDbgSelectMask = 4,      // selector: mask word past the end of the mask
  kDbgSelectTmem = 5,      // selector: accumulator columns past the allocated tensor memory
  kDbgSelectCentroid = 6,  // selector: centroid row of a tile past the padded centroid arrays
  kDbgPrefillBlock = 7,    // attention: key sub-block after the query tile or past the sequence
  kDbgPrefillTile = 8,     // attention: query tile outside this call's queries
  kDbgPrefillPart = 9,     // attention: partial-result slot outside the workspace
  kDbgPrefillLse = 10,     // attention: lse index past the end
};
#ifdef RBS_DEBUG
__device__ __forceinline__ bool dbg_record(bool cond, unsigned int* status, unsigned int site) {
  if (!cond) atomicCAS(status, 0u, 0x100u + site);
  return cond;
}
#define RBS_DBG_OK(cond, status, site) ::rbs::dbg_record((cond), (status), (site))
#else
#define RBS_DBG_OK(cond, status, site) true
#endif

// ------------------------------------------------------------------------------------------- TMA
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
// 4-D tiled load: coordinates innermost first.  c0 * sizeof(element) must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
// 4-D tiled load with an L2 eviction-priority hint (policy from make_policy_evict_first): for data read exactly once.
__device__ __forceinline__ uint64_t make_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                                 int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}
// 4-D tiled store from shared memory (rows past the tensor's extent are clipped); completion through bulk groups.
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all bulk groups of this thread have finished reading their shared-memory source
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// generic-proxy writes to shared memory -> visible to the async proxy (TMA / tcgen05 operand reads)
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ------------------------------------------------------------------------------------------- TMEM
// Allocation is a warp-wide operation; the base address lands in shared memory.  ncols: power of two >= 32.
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Each thread of the warp reads 32 consecutive 32-bit columns of its own lane (lane = 32 * (warp % 4) + laneid).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// ------------------------------------------------------------------------------------------- tcgen05.mma
// Shared-memory matrix descriptor for a tile stored as 128-byte rows with the 128-byte swizzle
// (what a TMA load with CU_TENSOR_MAP_SWIZZLE_128B of a 64-element bf16 inner box produces).
//   K-major operand  (rows = M or N index, 64 K-elements per row):  sbo = bytes between 8-row groups.
//   MN-major operand (rows = K index, 64 MN-elements per row):      lbo = bytes between 64-element MN groups,
//                                                                    sbo = bytes between 8-row K groups.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3ffff) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fff) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3fff) << 32;
  d |= static_cast<uint64_t>(1) << 46;   // descriptor version of this architecture
  d |= static_cast<uint64_t>(2) << 61;   // 128-byte swizzle
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M x N tile, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t idesc_bf16_f32(int M, int N, bool b_mn_major) {
  return (1u << 4)                                  // accumulator fp32
         | (1u << 7) | (1u << 10)                   // A, B = bf16
         | (static_cast<uint32_t>(b_mn_major) << 16)
         | (static_cast<uint32_t>(N >> 3) << 17)
         | (static_cast<uint32_t>(M >> 4) << 24);
}
// The *_elect forms are called by a whole converged warp: one elected lane issues, the control flow and
// the operands stay warp-uniform (so they can live in uniform registers instead of being moved there
// for every instruction, which costs the issuing thread tens of cycles per MMA).
__device__ __forceinline__ void mma_ss_elect(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_ts_elect(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit_elect(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar) : "memory");
}
// Batched issue by a converged warp: one election, then the MMAs of a whole step back to back and the commit.
// S[d_tmem] = A B^T over K = 128 for two K-major operands stored as two 64-column panels `panel` bytes apart
// (8 MMAs of K = 16; descriptor address field advances by 32 bytes per step inside a panel).  The first MMA
// overwrites the accumulator unless `accumulate_first`; `bar` != 0: commit to that mbarrier afterwards.
__device__ __forceinline__ void mma_ss_k128_commit_elect(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                         uint32_t a_panel_bytes, uint32_t b_panel_bytes, uint32_t bar,
                                                         uint32_t accumulate_first = 0) {
  const uint64_t pa = static_cast<uint64_t>(a_panel_bytes >> 4), pb = static_cast<uint64_t>(b_panel_bytes >> 4);
  asm volatile(
      "{\n\t.reg .pred e, pt, pf;\n\t.reg .b64 a, b, a1, b1;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.eq.u32 pt, 0, 0;\n\t"
      "setp.ne.u32 pf, %7, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n\t"
      "add.u64 a, %1, 2;\n\t add.u64 b, %2, 2;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "add.u64 a, %1, 4;\n\t add.u64 b, %2, 4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "add.u64 a, %1, 6;\n\t add.u64 b, %2, 6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "add.u64 a1, %1, %4;\n\t add.u64 b1, %2, %6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a1, b1, %3, pt;\n\t"
      "add.u64 a, a1, 2;\n\t add.u64 b, b1, 2;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "add.u64 a, a1, 4;\n\t add.u64 b, b1, 4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "add.u64 a, a1, 6;\n\t add.u64 b, b1, 6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "setp.ne.u32 pf, %5, 0;\n\t"
      "and.pred pf, pf, e;\n\t"
      "@pf tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%5];\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "l"(pa), "r"(bar), "l"(pb), "r"(accumulate_first) : "memory");
}
// The same for one 64-column panel of each operand (K = 64: 4 MMAs of K = 16).
__device__ __forceinline__ void mma_ss_k64_commit_elect(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                        uint32_t bar, uint32_t accumulate_first) {
  asm volatile(
      "{\n\t.reg .pred e, pt, pf;\n\t.reg .b64 a, b;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.eq.u32 pt, 0, 0;\n\t"
      "setp.ne.u32 pf, %5, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n\t"
      "add.u64 a, %1, 2;\n\t add.u64 b, %2, 2;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "add.u64 a, %1, 4;\n\t add.u64 b, %2, 4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "add.u64 a, %1, 6;\n\t add.u64 b, %2, 6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, pt;\n\t"
      "setp.ne.u32 pf, %4, 0;\n\t"
      "and.pred pf, pf, e;\n\t"
      "@pf tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%4];\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(bar), "r"(accumulate_first) : "memory");
}
// O[d_tmem] (+)= P V for 64 keys: A = P from tensor memory (8 columns per K = 16 step from a_tmem), B = V as an
// MN-major operand whose descriptor advances by `kstep16` (in 16-byte units) per step.  4 MMAs; the first one
// overwrites the accumulator when `accumulate_first` is 0.  `bar` != 0: commit to that mbarrier afterwards.
__device__ __forceinline__ void mma_ts_k64_elect(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t kstep16, uint32_t accumulate_first, uint32_t bar) {
  const uint64_t ks = static_cast<uint64_t>(kstep16);
  asm volatile(
      "{\n\t.reg .pred e, pt, p0, c;\n\t.reg .b64 b;\n\t.reg .b32 a;\n\t"
      "elect.sync _|e, 0xffffffff;\n\t"
      "setp.eq.u32 pt, 0, 0;\n\t"
      "setp.ne.u32 p0, %5, 0;\n\t"
      "setp.ne.u32 c, %6, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p0;\n\t"
      "add.u32 a, %1, 8;\n\t add.u64 b, %2, %4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
      "add.u32 a, %1, 16;\n\t add.u64 b, b, %4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
      "add.u32 a, %1, 24;\n\t add.u64 b, b, %4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [a], b, %3, pt;\n\t"
      "and.pred c, c, e;\n\t"
      "@c tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%6];\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "l"(ks), "r"(accumulate_first), "r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]; one thread issues.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Makes the mbarrier complete one arrival when all tcgen05.mma issued so far by this thread have finished.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// ------------------------------------------------------------------------------------------- registers, packed math
// Register re-allocation is a warpgroup-wide operation: all four warps of an aligned group of 128 threads
// must execute the same one.
template <int N>
__device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// two fp32 values in one 64-bit register, processed by one instruction
__device__ __forceinline__ uint64_t f2_pack(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

__device__ __forceinline__ uint64_t f2_add_rm(uint64_t a, uint64_t b) {   // round toward -inf
  uint64_t d;
  asm("add.rm.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// 2^x for two values on the FMA pipe instead of the special-function unit (which is the scarce unit in
// the softmax): x = n + f with n = floor(x), 2^f by a degree-3 minimax polynomial on [0, 1) (relative
// error 7.5e-5), then n is added into the exponent field.  Inputs are clamped to x >= -126; x <= 127.
__device__ __forceinline__ void exp2_poly_x2(uint64_t x2, float& r0, float& r1) {
  constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23: its float spacing is 1
  float x0, x1;
  f2_unpack(x2, x0, x1);
  const uint64_t xc = f2_pack(fmaxf(x0, -126.0f), fmaxf(x1, -126.0f));
  const uint64_t t = f2_add_rm(xc, f2_pack(kMagic, kMagic));                  // low mantissa bits = floor(x)
  const uint64_t fl = f2_add(t, f2_pack(-kMagic, -kMagic));                   // floor(x), exact
  const uint64_t f = f2_fma(fl, f2_pack(-1.0f, -1.0f), xc);                   // x - floor(x) in [0, 1)
  uint64_t pl = f2_fma(f, f2_pack(0.0780242234f, 0.0780242234f), f2_pack(0.2260672301f, 0.2260672301f));
  pl = f2_fma(pl, f, f2_pack(0.6958336830f, 0.6958336830f));
  pl = f2_fma(pl, f, f2_pack(0.9999251962f, 0.9999251962f));
  float p0, p1, t0, t1;
  f2_unpack(pl, p0, p1);
  f2_unpack(t, t0, t1);
  r0 = __int_as_float(__float_as_int(p0) + (__float_as_int(t0) << 23));
  r1 = __int_as_float(__float_as_int(p1) + (__float_as_int(t1) << 23));
}

// Same idea without the clamp, for callers that know -126 <= x <= 127, and with a degree-4 polynomial
// (relative error 2.6e-6).  Everything runs on the FMA pipe: the exponent is added with an integer multiply-add.
__device__ __forceinline__ void exp2_poly4_x2(uint64_t x2, float& r0, float& r1) {
  constexpr float kMagic = 12582912.0f;
  const uint64_t t = f2_add_rm(x2, f2_pack(kMagic, kMagic));
  const uint64_t fl = f2_add(t, f2_pack(-kMagic, -kMagic));
  const uint64_t f = f2_fma(fl, f2_pack(-1.0f, -1.0f), x2);
  uint64_t pl = f2_fma(f, f2_pack(0.0135341408f, 0.0135341408f), f2_pack(0.0520114899f, 0.0520114899f));
  pl = f2_fma(pl, f, f2_pack(0.2414427549f, 0.2414427549f));
  pl = f2_fma(pl, f, f2_pack(0.6930038333f, 0.6930038333f));
  pl = f2_fma(pl, f, f2_pack(1.0000026226f, 1.0000026226f));
  float p0, p1, t0, t1;
  f2_unpack(pl, p0, p1);
  f2_unpack(t, t0, t1);
  int b0, b1;
  asm("mad.lo.s32 %0, %1, 8388608, %2;" : "=r"(b0) : "r"(__float_as_int(t0)), "r"(__float_as_int(p0)));
  asm("mad.lo.s32 %0, %1, 8388608, %2;" : "=r"(b1) : "r"(__float_as_int(t1)), "r"(__float_as_int(p1)));
  r0 = __int_as_float(b0);
  r1 = __int_as_float(b1);
}

}  // namespace rbs
