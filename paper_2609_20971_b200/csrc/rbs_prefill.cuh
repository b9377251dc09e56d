// Parameters and mask walkers shared by the attention kernels.
#pragma once

#include "rbs_common.cuh"
#include "rbs_sm100.cuh"

namespace rbs {

struct PrefillParams {
  const __nv_bfloat16* Q; int64_t qsb, qst, qsh;
  const __nv_bfloat16* K; int64_t ksb, kst, ksh;
  const __nv_bfloat16* V; int64_t vsb, vst, vsh;
  __nv_bfloat16* O; int64_t osb, ost, osh;
  const uint32_t* mask;  // nullptr: dense
  float* lse;            // nullable
  int M, W, L, Hq, G, N;
  int R;   // 128-row tiles per block (tensor-core path): block / 128
  int q0, Mq, Nq;   // this call's queries: first query block (global index), number of blocks, number of tokens
  int band_rows;    // 128-row query tiles per band of the tile order (tensor-core path)
  float scale_log2;
  // Row-length-aware schedule (null: tiles in their static order, one CTA per tile).  One int4 per CTA:
  // x = position of the tile in its group's static order (-1: nothing to do), [y, z) = range of 128-key sub-blocks
  // this item attends, w = slot of its partial result (-1: the item is a whole row and writes O itself).
  const int4* items;
  int items_per_group;
  float* part_o;    // [slot][128 rows][128] unnormalised O of a part, fp32
  float* part_ml;   // [slot][2][128]        running maximum (log2 units) and row sum of a part
};

// Rows longer than this many 128-key sub-blocks are cut into parts of equal length that run as separate CTAs and are
// merged afterwards; the cut depends only on the row itself, so a row is treated the same in every call.
constexpr int kSplitCap = 256;
constexpr int kSplitMaxParts = 4;      // parts per split row
constexpr int kSplitRowsPerGroup = 8;  // split rows per (band, batch, KV head) group: its longest ones
constexpr int kSplitSlotsPerGroup = kSplitRowsPerGroup * kSplitMaxParts;
constexpr int kExtraItemsPerGroup = kSplitRowsPerGroup * (kSplitMaxParts - 1);

// next selected key block after `cur` (cur = -1 to start), restricted to b <= i; -1 when exhausted
__device__ __forceinline__ int next_block(const uint32_t* __restrict__ row, int cur, int i) {
  int b = cur + 1;
  if (row == nullptr) return b <= i ? b : -1;
  while (b <= i) {
    uint32_t w = __ldg(row + (b >> 5)) >> (b & 31);
    if (w) {
      b += __ffs(w) - 1;
      return b <= i ? b : -1;
    }
    b = (b | 31) + 1;
  }
  return -1;
}

// Tensor-core path, blocks of R x 128 tokens: the kernel works on 128-row query tiles T and 128-key sub-blocks kb.
// Sub-block kb belongs to mask block kb / R; tile T (of query block T / R) attends sub-blocks kb <= T of the selected
// blocks, kb == T being the diagonal one.  Returns the next sub-block after `cur` (-1 to start), or -1.
__device__ __forceinline__ int next_kb(const uint32_t* __restrict__ row, int cur, int i, int R, int T) {
  int kb = cur + 1;
  if (kb > T) return -1;
  const int b = kb / R;
  const int nb = next_block(row, b - 1, i);   // first selected block >= b
  if (nb < 0) return -1;
  if (nb != b) kb = nb * R;
  return kb <= T ? kb : -1;
}

// A half-row of P whose sum reaches this value makes the row adopt the half's exact maximum (the lazy running maximum
// of the tensor-core kernels).
constexpr float kSumLimit = 16384.0f;

rbs_status launch_prefill_pair(const PrefillParams& p, const rbs_tensor& Q, const rbs_tensor& K, const rbs_tensor& V, int Hkv,
                               int mode, cudaStream_t s);

}  // namespace rbs
