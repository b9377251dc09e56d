// Shared device/host helpers of the RBS prefill library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include <nvtx3/nvToolsExt.h>

#include "rbs.h"

struct CUtensorMap_st;

namespace rbs {

constexpr int kHeadDim = 128;
constexpr float kLog2e = 1.4426950408889634f;

// Shape-derived sizes used by every entry point.
struct Dims {
  int L, N, Hq, Hkv, d, B, M, W, G;
};

inline Dims make_dims(const rbs_shape& s) {
  Dims x;
  x.L = s.batch; x.N = s.seqlen; x.Hq = s.n_q_heads; x.Hkv = s.n_kv_heads; x.d = s.head_dim; x.B = s.block;
  x.M = s.block > 0 ? (s.seqlen + s.block - 1) / s.block : 0;   // a short last block counts
  x.W = (x.M + 31) / 32;
  x.G = s.n_kv_heads > 0 ? s.n_q_heads / s.n_kv_heads : 0;
  return x;
}

// Host-side argument checks shared by the entry points.
rbs_status check_shape(const rbs_shape* shape);
rbs_status check_tensor(const rbs_tensor& t);
struct Dims;
// A query chunk must start on a block boundary, lie inside the sequence, and may end inside a block only at the
// end of the sequence.
rbs_status check_chunk(const Dims& x, int q_start_block, int n_q_tokens);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace carve-up of rbs_select (all offsets 256-byte aligned).
struct SelectWorkspace {
  size_t off_chi, off_clo, off_g, off_cn, off_perm, off_counts, bytes;
  int Mpad;  // centroid rows per (l, hk) in the bf16 copies, multiple of 128
};
SelectWorkspace select_workspace(const Dims& x);

// Workspace carve-up of rbs_sparse_prefill's row-length-aware schedule (blocks of 128 and 256), sized for the whole
// sequence so that it also serves every chunked call: the work items, the list of split rows and the partial
// results of their parts.  n_rows = 128-row query tiles of the sequence.
struct PrefillWorkspace {
  size_t off_items, off_splits, off_part_o, off_part_ml, bytes;
};
PrefillWorkspace prefill_workspace(int L, int Hq, int Hkv, int n_rows, int G);

// Workspace of rbs_select_box (0 for shapes it does not support).
size_t select_box_workspace_bytes(const Dims& x);

// TMA tensor map over a bf16 [L][N][H][d] tensor with arbitrary (16-byte aligned) strides; box = box_d x box_t.
rbs_status make_tmap_lthd(::CUtensorMap_st* out, const void* ptr, int L, int N, int H, int d, int64_t sb, int64_t st,
                          int64_t sh, int box_d, int box_t, bool swizzle128);
rbs_status make_tmap_2d(::CUtensorMap_st* out, const void* ptr, int64_t rows, int cols, int box_cols, int box_rows);
// Number of SMs of the current device (looked up once per device).
int sm_count();
// Device address, on the current device, of the status word that bounded waits report to (nullptr if it cannot be
// obtained).  Looked up once per device, with that device current: an address taken on one GPU means nothing on another.
unsigned int* device_status_ptr();
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) only when this (kernel, device) has not yet been given at least
// `bytes`: the attribute is per device and sticky, and the call is not free on the per-layer path.
rbs_status ensure_dynamic_smem(const void* kernel, size_t bytes);

// A value per CUDA device, filled on first use by `make(device, &value)` (true = success; failures are not cached).
// The table itself is plain host logic: it never touches CUDA, so it is also exercised without a GPU.
template <typename T, int kMaxDevices = 64>
class PerDevice {
 public:
  template <typename Make>
  bool get(int device, T* out, Make make) {
    if (device < 0 || device >= kMaxDevices) return false;
    std::lock_guard<std::mutex> guard(lock_);
    if (!have_[device]) {
      T v{};
      if (!make(device, &v)) return false;
      value_[device] = v;
      have_[device] = true;
    }
    *out = value_[device];
    return true;
  }

 private:
  std::mutex lock_;
  bool have_[kMaxDevices] = {};
  T value_[kMaxDevices] = {};
};

// Named range around an entry point's host work, visible in NVIDIA's timeline tools (a no-op when none is attached).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

#define RBS_CUDA_OK(expr)                               \
  do {                                                  \
    cudaError_t _e = (expr);                            \
    if (_e != cudaSuccess) return RBS_ERR_CUDA;         \
  } while (0)

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fast_log2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src));
}
// 16-byte copy that writes zeros instead when `valid` is false (nothing is read from `src` then)
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, bool valid) {
  const uint32_t n = valid ? 16u : 0u;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Byte offset of 16-byte chunk `chunk` (0..15) of row `row` inside a [rows][128] bf16 tile whose rows
// are 256 bytes, with the chunk index XOR-ed by the row so that ldmatrix reads hit distinct banks.
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return static_cast<uint32_t>(row * 256 + ((chunk ^ (row & 7)) << 4));
}

}  // namespace rbs
