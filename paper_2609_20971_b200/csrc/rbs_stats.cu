// rbs_block_stats: one HBM stream over K.  Each CTA owns one (batch, KV head, key block) tile of
// B rows x 128 bf16, holds it in registers, and produces the centroid and the radius from that single read.
#include "rbs_common.cuh"

namespace rbs {

constexpr int kStatsThreads = 256;

// Thread t owns 16-byte chunk (t % 16) of rows (t / 16) + 16 j, j < B / 16.
template <int B>
__global__ void __launch_bounds__(kStatsThreads)
block_stats_kernel(const __nv_bfloat16* __restrict__ K, int64_t sb, int64_t st, int64_t sh, int M, int Hkv,
                   float* __restrict__ centroid, float* __restrict__ radius) {
  constexpr int R = B / 16;  // rows per thread
  __shared__ float s_part[kStatsThreads / 32][kHeadDim];
  __shared__ float s_max[kStatsThreads / 32];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunk = tid & 15, r0 = tid >> 4;
  // KV head fastest so that neighbouring CTAs read neighbouring 256-byte rows of the same tokens.
  int idx = blockIdx.x;
  const int hk = idx % Hkv; idx /= Hkv;
  const int b = idx % M;
  const int l = idx / M;

  const __nv_bfloat16* base = K + l * sb + (static_cast<int64_t>(b) * B + r0) * st + hk * sh + chunk * 8;
  uint4 v[R];
#pragma unroll
  for (int j = 0; j < R; ++j) v[j] = __ldg(reinterpret_cast<const uint4*>(base + static_cast<int64_t>(16 * j) * st));

  float acc[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) acc[k] = 0.f;
#pragma unroll
  for (int j = 0; j < R; ++j) {
    acc[0] += bf16lo(v[j].x); acc[1] += bf16hi(v[j].x);
    acc[2] += bf16lo(v[j].y); acc[3] += bf16hi(v[j].y);
    acc[4] += bf16lo(v[j].z); acc[5] += bf16hi(v[j].z);
    acc[6] += bf16lo(v[j].w); acc[7] += bf16hi(v[j].w);
  }
#pragma unroll
  for (int k = 0; k < 8; ++k) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], 16);
  if (lane < 16) {
    float4* p = reinterpret_cast<float4*>(&s_part[warp][chunk * 8]);
    p[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    p[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
  }
  __syncthreads();
  float cen[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) cen[k] = 0.f;
#pragma unroll
  for (int w = 0; w < kStatsThreads / 32; ++w) {
    const float4* p = reinterpret_cast<const float4*>(&s_part[w][chunk * 8]);
    float4 a = p[0], c = p[1];
    cen[0] += a.x; cen[1] += a.y; cen[2] += a.z; cen[3] += a.w;
    cen[4] += c.x; cen[5] += c.y; cen[6] += c.z; cen[7] += c.w;
  }
#pragma unroll
  for (int k = 0; k < 8; ++k) cen[k] *= (1.0f / B);
  const int64_t blk = (static_cast<int64_t>(l) * Hkv + hk) * M + b;
  if (tid < 16) {
    float4* out = reinterpret_cast<float4*>(centroid + blk * kHeadDim + chunk * 8);
    out[0] = make_float4(cen[0], cen[1], cen[2], cen[3]);
    out[1] = make_float4(cen[4], cen[5], cen[6], cen[7]);
  }

  // radius^2 = max over rows of sum_j (k_j - c_j)^2, difference form
  float rmax = 0.f;
#pragma unroll
  for (int j = 0; j < R; ++j) {
    float d0 = bf16lo(v[j].x) - cen[0], d1 = bf16hi(v[j].x) - cen[1];
    float d2 = bf16lo(v[j].y) - cen[2], d3 = bf16hi(v[j].y) - cen[3];
    float d4 = bf16lo(v[j].z) - cen[4], d5 = bf16hi(v[j].z) - cen[5];
    float d6 = bf16lo(v[j].w) - cen[6], d7 = bf16hi(v[j].w) - cen[7];
    float s = d0 * d0;
    s = fmaf(d1, d1, s); s = fmaf(d2, d2, s); s = fmaf(d3, d3, s);
    s = fmaf(d4, d4, s); s = fmaf(d5, d5, s); s = fmaf(d6, d6, s); s = fmaf(d7, d7, s);
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    s += __shfl_xor_sync(0xffffffffu, s, 8);
    rmax = fmaxf(rmax, s);
  }
  rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, 16));
  if (lane == 0) s_max[warp] = rmax;
  __syncthreads();
  if (tid == 0) {
    float m = s_max[0];
#pragma unroll
    for (int w = 1; w < kStatsThreads / 32; ++w) m = fmaxf(m, s_max[w]);
    radius[blk] = sqrtf(m);
  }
}

}  // namespace rbs

extern "C" rbs_status rbs_block_stats(const rbs_shape* shape, rbs_tensor K, rbs_stats stats, void* stream) {
  using namespace rbs;
  rbs_status st = check_shape(shape);
  if (st != RBS_OK) return st;
  st = check_tensor(K);
  if (st != RBS_OK) return st;
  if (stats.centroid == nullptr || stats.radius == nullptr) return RBS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(stats.centroid) % 16 != 0) return RBS_ERR_INVALID_ARG;
  Dims x = make_dims(*shape);
  const long long n_tiles = static_cast<long long>(x.L) * x.Hkv * x.M;
  if (n_tiles > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16* k = static_cast<const __nv_bfloat16*>(K.ptr);
  dim3 grid(static_cast<unsigned>(n_tiles));
  if (x.B == 128)
    block_stats_kernel<128><<<grid, kStatsThreads, 0, s>>>(k, K.stride_batch, K.stride_token, K.stride_head, x.M, x.Hkv,
                                                            stats.centroid, stats.radius);
  else
    block_stats_kernel<64><<<grid, kStatsThreads, 0, s>>>(k, K.stride_batch, K.stride_token, K.stride_head, x.M, x.Hkv,
                                                           stats.centroid, stats.radius);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}
