// Host helper: builds TMA tensor maps through the driver entry point obtained from the runtime
// (the library does not link against the driver library, so it loads on machines without one).
#include "rbs_common.cuh"
#include "rbs_sm100.cuh"
#include "rbs_selftest.h"

namespace rbs {

static __device__ unsigned int g_device_status = 0;

static bool current_device(int* dev) { return cudaGetDevice(dev) == cudaSuccess; }

unsigned int* device_status_ptr() {
  static PerDevice<unsigned int*> table;
  int dev = -1;
  if (!current_device(&dev)) return nullptr;
  unsigned int* p = nullptr;
  const bool ok = table.get(dev, &p, [](int, unsigned int** out) {
    void* q = nullptr;   // the symbol's address on the device that is current now
    if (cudaGetSymbolAddress(&q, g_device_status) != cudaSuccess || q == nullptr) return false;
    *out = static_cast<unsigned int*>(q);
    return true;
  });
  return ok ? p : nullptr;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor addressed as ptr[l*sb + t*st + h*sh + j], viewed by TMA as 4-D (j, h, t, l).
// Box = box_d x 1 x box_t x 1 elements.  swizzle128: 128-byte swizzle (box_d must be 64), else none.
rbs_status make_tmap_lthd(CUtensorMap* out, const void* ptr, int L, int N, int H, int d, int64_t sb, int64_t st,
                          int64_t sh, int box_d, int box_t, bool swizzle128) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return RBS_ERR_CUDA;
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(N),
                        static_cast<cuuint64_t>(L)};
  if (sb == 0) sb = st * N;  // batch of one: any valid stride
  cuuint64_t strides[3] = {static_cast<cuuint64_t>(sh) * 2, static_cast<cuuint64_t>(st) * 2,
                           static_cast<cuuint64_t>(sb) * 2};
  cuuint32_t box[4] = {static_cast<cuuint32_t>(box_d), 1, static_cast<cuuint32_t>(box_t), 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? RBS_OK : RBS_ERR_CUDA;
}

// Row-major bf16 matrix [rows][cols] (cols contiguous); box = box_cols x box_rows, 128-byte swizzle.
rbs_status make_tmap_2d(CUtensorMap* out, const void* ptr, int64_t rows, int cols, int box_cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return RBS_ERR_CUDA;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? RBS_OK : RBS_ERR_CUDA;
}

int sm_count() {
  static PerDevice<int> table;
  int dev = -1, n = 0;
  if (!current_device(&dev)) return 148;
  const bool ok = table.get(dev, &n, [](int d, int* out) {
    return cudaDeviceGetAttribute(out, cudaDevAttrMultiProcessorCount, d) == cudaSuccess && *out > 0;
  });
  return ok ? n : 148;
}

rbs_status ensure_dynamic_smem(const void* kernel, size_t bytes) {
  struct Key { const void* fn; int dev; size_t bytes; };
  static std::mutex lock;
  static Key seen[256];
  static int n_seen = 0;
  int dev = -1;
  if (!current_device(&dev)) return RBS_ERR_CUDA;
  std::lock_guard<std::mutex> guard(lock);
  Key* slot = nullptr;
  for (int k = 0; k < n_seen; ++k)
    if (seen[k].fn == kernel && seen[k].dev == dev) { slot = &seen[k]; break; }
  if (slot != nullptr && slot->bytes >= bytes) return RBS_OK;
  RBS_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)));
  if (slot == nullptr && n_seen < 256) slot = &seen[n_seen++];
  if (slot != nullptr) { slot->fn = kernel; slot->dev = dev; slot->bytes = bytes; }
  return RBS_OK;
}

// One CTA, one thread: waits on an mbarrier that nothing ever arrives on, with the given probe limit.
#ifdef RBS_DEBUG
// one thread runs a debug check that fails by construction (the "index" 1 against a bound of 1)
__global__ void selftest_debug_check_kernel(unsigned int* status, unsigned int* skipped) {
  const int index = 1, bound = 1;
  if (RBS_DBG_OK(index < bound, status, 0xffu)) *skipped = 0u;   // the guarded "access"
  else *skipped = 1u;
}
#endif

__global__ void selftest_wait_kernel(unsigned int* status, unsigned int spin_limit, unsigned int* gave_up) {
  __shared__ __align__(8) uint64_t bar;
  mbar_init(smem_u32(&bar), 1);
  mbar_fence_init();
  const bool ok = mbar_wait_limit(smem_u32(&bar), 0, status, kWaitSelfTest, spin_limit);
  *gave_up = ok ? 0u : 1u;
}

}  // namespace rbs

extern "C" rbs_status rbs_device_status(void* stream, unsigned int* code_out, int clear) {
  unsigned int code = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return RBS_ERR_CUDA;
  if (cudaMemcpyFromSymbol(&code, rbs::g_device_status, sizeof(code)) != cudaSuccess) return RBS_ERR_CUDA;
  if (clear && code != 0) {
    unsigned int zero = 0;
    if (cudaMemcpyToSymbol(rbs::g_device_status, &zero, sizeof(zero)) != cudaSuccess) return RBS_ERR_CUDA;
  }
  if (code_out) *code_out = code;
  return code == 0 ? RBS_OK : (code >= 0x100u ? RBS_ERR_DEBUG_CHECK : RBS_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// self-tests (include/rbs_selftest.h)
// ---------------------------------------------------------------------------------------------
extern "C" int rbs_selftest_device_table(void) {
  // the per-device table with a fake lookup: every device gets its own value, looked up exactly once; a failed
  // lookup is not remembered; out-of-range devices are refused
  rbs::PerDevice<long, 8> table;
  int calls[8] = {0};
  bool fail_next = true;
  auto make = [&](int dev, long* out) {
    ++calls[dev];
    if (dev == 5 && fail_next) { fail_next = false; return false; }
    *out = 1000 + 7 * dev;
    return true;
  };
  long v = 0;
  const int order[] = {3, 0, 3, 7, 0, 3};
  for (int dev : order) {
    if (!table.get(dev, &v, make) || v != 1000 + 7 * dev) return 1;
  }
  if (calls[3] != 1 || calls[0] != 1 || calls[7] != 1 || calls[1] != 0) return 2;
  if (table.get(5, &v, make)) return 3;                 // first lookup fails and must not be cached
  if (!table.get(5, &v, make) || v != 1035 || calls[5] != 2) return 4;
  if (table.get(-1, &v, make) || table.get(8, &v, make)) return 5;
  return 0;
}

extern "C" rbs_status rbs_selftest_wait_timeout(unsigned int spin_limit, unsigned int* gave_up, void* stream) {
  if (gave_up == nullptr || spin_limit == 0 || spin_limit > (1u << 16)) return RBS_ERR_INVALID_ARG;
  unsigned int* status = rbs::device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  rbs::selftest_wait_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(status, spin_limit, gave_up);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

extern "C" rbs_status rbs_selftest_debug_check(unsigned int* skipped, void* stream) {
#ifdef RBS_DEBUG
  if (skipped == nullptr) return RBS_ERR_INVALID_ARG;
  unsigned int* status = rbs::device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  rbs::selftest_debug_check_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(status, skipped);
  return cudaGetLastError() == cudaSuccess ? RBS_OK : RBS_ERR_CUDA;
#else
  (void)skipped; (void)stream;
  return RBS_ERR_UNSUPPORTED;   // the release build has no device-side checks
#endif
}
