// Host helper: builds TMA tensor maps through the driver entry point obtained from the runtime
// (the library does not link against the driver library, so it loads on machines without one).
#include "rbs_common.cuh"
#include "rbs_sm100.cuh"

namespace rbs {

static __device__ unsigned int g_device_status = 0;

unsigned int* device_status_ptr() {
  static unsigned int* p = nullptr;
  if (p == nullptr) {
    void* q = nullptr;
    if (cudaGetSymbolAddress(&q, g_device_status) != cudaSuccess) return nullptr;
    p = static_cast<unsigned int*>(q);
  }
  return p;
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
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
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
  return code == 0 ? RBS_OK : RBS_ERR_TIMEOUT;
}
