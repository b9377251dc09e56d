// Group-shared selection masks: union over the query heads of a KV group (a variant outside the paper's
// per-head selector, see rbs.h).
#include "rbs_common.cuh"

namespace rbs {

constexpr int kUnionThreads = 1024;

// One CTA per (batch, KV head): ORs the G mask rows word by word, writes the union back to all G heads, counts
// the kept pairs and writes the group's density.  Mask bits are only ever set for causal pairs, so the popcount
// of a word is its number of kept pairs.
__global__ void __launch_bounds__(kUnionThreads)
group_union_kernel(uint32_t* __restrict__ mask, float* __restrict__ density, int Hq, int G, int Mq, int W, int q0) {
  const int kv = blockIdx.x;                 // l * Hkv + hk
  const int Hkv = Hq / G;
  const int l = kv / Hkv, hk = kv % Hkv;
  const int64_t head_words = static_cast<int64_t>(Mq) * W;
  uint32_t* base = mask + (static_cast<int64_t>(l) * Hq + static_cast<int64_t>(hk) * G) * head_words;
  unsigned long long cnt = 0;
  for (int64_t w = threadIdx.x; w < head_words; w += kUnionThreads) {
    uint32_t u = 0;
    for (int g = 0; g < G; ++g) u |= base[g * head_words + w];
    for (int g = 0; g < G; ++g) base[g * head_words + w] = u;
    cnt += __popc(u);
  }
  __shared__ unsigned long long red[kUnionThreads / 32];
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = cnt;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long total = 0;
    for (int i = 0; i < kUnionThreads / 32; ++i) total += red[i];
    const double pairs = static_cast<double>(Mq) * static_cast<double>(q0) + 0.5 * static_cast<double>(Mq) * static_cast<double>(Mq + 1);
    const float d = static_cast<float>(static_cast<double>(total) / pairs);
    for (int g = 0; g < G; ++g) density[l * Hq + hk * G + g] = d;
  }
}

}  // namespace rbs

extern "C" rbs_status rbs_mask_group_union(const rbs_shape* shape, int q_start_block, int n_q_tokens, uint32_t* mask,
                                           float* density, void* stream) {
  using namespace rbs;
  rbs_status st = check_shape(shape);
  if (st != RBS_OK) return st;
  if (mask == nullptr || density == nullptr) return RBS_ERR_INVALID_ARG;
  Dims x = make_dims(*shape);
  if (n_q_tokens < 0) { q_start_block = 0; n_q_tokens = x.N; }
  if ((st = check_chunk(x, q_start_block, n_q_tokens)) != RBS_OK) return st;
  const int Mq = (n_q_tokens + x.B - 1) / x.B;
  group_union_kernel<<<x.L * x.Hkv, kUnionThreads, 0, static_cast<cudaStream_t>(stream)>>>(mask, density, x.Hq, x.G, Mq,
                                                                                           x.W, q_start_block);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}
