// rbs_select: rescue coefficients (Eq. beta), dual-branch block scores (Eq. base_score, rescue_score,
// block_aggregation), per-branch relative thresholds, forced blocks, union, bit-packed mask, density.
//
// Scoring works on the transposed product  X^T = C . Q_i^T  (centroids are the M-dimension, the tokens of
// the query block the N-dimension) so that the sum over tokens needed by the aggregation runs along the
// accumulator row of one centroid.  Centroids are fed to the tensor cores as bf16 hi + bf16 lo
// (two accumulating products) so that the logit keeps ~16 mantissa bits of the fp32 centroid.
// Scores are kept per block as log2-sum-exp2, L = log2 sum_t 2^(z_t); the relative threshold
// S >= alpha max S becomes L >= log2(alpha) + max L (the common shift of Eq. block_aggregation cancels).
#include "rbs_common.cuh"
#include "rbs_sm100.cuh"
#include "rbs_score.cuh"

namespace rbs {

// ---------------------------------------------------------------------------------------------
// 1. per (l, KV head): sort radii, quantiles, beta, g = r * beta
// ---------------------------------------------------------------------------------------------
constexpr int kCoeffThreads = 1024;

// Besides beta, the kernel fixes the ORDER in which the scoring kernels see the blocks of each 128-row centroid tile:
// inside a tile the rows with r_b beta_b = 0 (at least half of all blocks: every radius at or below the median) come
// first, the others after them (the other way round in odd tiles).  perm[pos] = block index, gs[pos] = r_b beta_b scale
// (log2 units per unit of query norm) in that order.  A scoring warp whose 32 rows all have gs = 0 then needs no
// second exponential per logit, because S_rescue = S_base there; without the partition hardly any warp would qualify.
__global__ void __launch_bounds__(kCoeffThreads)
rescue_coeff_kernel(const float* __restrict__ radius, int M, int P /* pow2 >= M */, float scale_log2,
                    float* __restrict__ beta, float* __restrict__ rq, float* __restrict__ gs, int* __restrict__ perm,
                    int Mpad, int beta_mode /* 0: Eq. (beta), 1: beta = 0, 2: beta = 1 */) {
  extern __shared__ float s_sorted[];
  __shared__ float s_q[2];
  __shared__ unsigned short s_zero[8192 / 32];   // per group of 32 rows: how many have gs = 0
  const int hd = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const float* r = radius + static_cast<int64_t>(hd) * M;
  for (int idx = tid; idx < P; idx += kCoeffThreads) s_sorted[idx] = idx < M ? r[idx] : __int_as_float(0x7f800000);
  __syncthreads();
  for (int k = 2; k <= P; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int idx = tid; idx < P; idx += kCoeffThreads) {
        const int ixj = idx ^ j;
        if (ixj > idx) {
          const float a = s_sorted[idx], c = s_sorted[ixj];
          const bool asc = (idx & k) == 0;
          if ((a > c) == asc) { s_sorted[idx] = c; s_sorted[ixj] = a; }
        }
      }
      __syncthreads();
    }
  }
  if (tid < 2) {
    // quantile(p): linear interpolation between order statistics at position p (M - 1)
    const double p = tid == 0 ? 0.5 : 0.9;
    const double x = p * static_cast<double>(M - 1);
    const int lo = static_cast<int>(floor(x));
    const int hi = min(lo + 1, M - 1);
    const double a = static_cast<double>(s_sorted[lo]), c = static_cast<double>(s_sorted[hi]);
    const float q = static_cast<float>(a + (x - lo) * (c - a));
    s_q[tid] = q;
    rq[hd * 2 + tid] = q;
  }
  __syncthreads();
  const float r_low = s_q[0], r_high = s_q[1];
  const bool live = r_high > r_low;
  const float inv = live ? 1.0f / (r_high - r_low) : 0.f;
  auto coeff = [&](int idx) -> float {   // r_b beta_b scale of block idx (0 for padding rows); also writes beta
    if (idx >= M) return 0.f;
    const float rb = r[idx];
    float bt = live ? fminf(fmaxf((rb - r_low) * inv, 0.f), 1.f) : 0.f;
    if (beta_mode == 1) bt = 0.f;
    if (beta_mode == 2) bt = 1.f;
    beta[static_cast<int64_t>(hd) * M + idx] = bt;
    return rb * bt * scale_log2;
  };
  // Mpad is a multiple of 128 and the loops below step by the CTA size, so every warp stays whole
  for (int idx = tid; idx < Mpad; idx += kCoeffThreads) {
    const uint32_t z = __ballot_sync(0xffffffffu, coeff(idx) == 0.f);
    if (lane == 0) s_zero[idx >> 5] = static_cast<unsigned short>(__popc(z));
  }
  __syncthreads();
  for (int idx = tid; idx < Mpad; idx += kCoeffThreads) {
    const float g = coeff(idx);
    const bool zero = g == 0.f;
    const uint32_t z = __ballot_sync(0xffffffffu, zero);
    const int tile = idx >> 7, w_in_tile = (idx >> 5) & 3;
    int zeros_tile = 0, zeros_before = 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int c = s_zero[tile * 4 + w];
      zeros_tile += c;
      if (w < w_in_tile) zeros_before += c;
    }
    zeros_before += __popc(z & ((1u << lane) - 1u));
    const int before = idx & 127;                       // rows of the tile in front of this one
    int pos = zero ? zeros_before : zeros_tile + (before - zeros_before);
    // odd tiles are laid out the other way round, so that the warp that gets the rows without a rescue term (half the
    // exponentials) in one tile gets the expensive rows in the next: over a query block's tiles the warps even out
    if (tile & 1) pos = 127 - pos;
    const int64_t dst = static_cast<int64_t>(hd) * Mpad + tile * 128 + pos;
    gs[dst] = g;
    perm[dst] = idx;
  }
}

// ---------------------------------------------------------------------------------------------
// 2. fp32 centroid -> bf16 hi + bf16 lo, rows padded to Mpad with zeros
// ---------------------------------------------------------------------------------------------
__global__ void split_centroid_kernel(const float* __restrict__ centroid, const int* __restrict__ perm, int M, int Mpad,
                                      int64_t n_rows_padded, float scale_log2, __nv_bfloat16* __restrict__ chi,
                                      __nv_bfloat16* __restrict__ clo, float* __restrict__ cnorm) {
  // One thread per 4 elements, one warp per row of the bf16 copies.  Row `row` holds block perm[row] of its
  // (batch, KV head), multiplied by log2(e)/sqrt(d) so that the tensor-core product is the scaled logit in log2 units;
  // also writes the row's L2 norm (of the scaled centroid).
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t row = t / (kHeadDim / 4);
  const int c4 = static_cast<int>(t % (kHeadDim / 4));
  if (row >= n_rows_padded) return;   // whole warps: the grid covers rows in units of 32 threads
  const int64_t hd = row / Mpad;
  const int b = perm[row];
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (b < M) v = *reinterpret_cast<const float4*>(centroid + (hd * M + b) * kHeadDim + c4 * 4);
  v.x *= scale_log2; v.y *= scale_log2; v.z *= scale_log2; v.w *= scale_log2;
  const __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y);
  const __nv_bfloat16 h2 = __float2bfloat16_rn(v.z), h3 = __float2bfloat16_rn(v.w);
  const float l0 = v.x - __bfloat162float(h0), l1 = v.y - __bfloat162float(h1);
  const float l2 = v.z - __bfloat162float(h2), l3 = v.w - __bfloat162float(h3);
  uint2 hi, lo;
  hi.x = static_cast<uint32_t>(__bfloat16_as_ushort(h0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h1)) << 16);
  hi.y = static_cast<uint32_t>(__bfloat16_as_ushort(h2)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h3)) << 16);
  lo.x = pack_bf16(l0, l1);
  lo.y = pack_bf16(l2, l3);
  *reinterpret_cast<uint2*>(chi + row * kHeadDim + c4 * 4) = hi;
  *reinterpret_cast<uint2*>(clo + row * kHeadDim + c4 * 4) = lo;
  float n2 = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
  if (c4 == 0) cnorm[row] = sqrtf(n2);
}

// ---------------------------------------------------------------------------------------------
// 3. scoring + thresholds + union + pack on the 5th-generation tensor cores, one CTA per
//    (batch, query head, query block), two CTAs per SM.
//   D[128 centroids x B tokens] (fp32, tensor memory) = C_hi . Q_i^T + C_lo . Q_i^T, 16 tcgen05.mma per tile.
//   One TMEM lane = one centroid, so the aggregation over the block's tokens is a per-thread loop over
//   the accumulator row: no cross-thread reduction at all.
// Warps 0-3: epilogue (TMEM lane = centroid row), warp 4: TMA producer, warp 5: MMA issuer and TMEM owner.
// Two TMEM accumulators let the MMAs of tile t+1 run under the epilogue of tile t.
// ---------------------------------------------------------------------------------------------
struct SelectParams {
  const __nv_bfloat16* Q; int64_t qsb, qst, qsh;
  // per padded centroid row, in the tile-partitioned order of rescue_coeff_kernel: bf16 hi / lo halves of the scaled
  // centroid, gs = r beta scale, norm of the scaled centroid, and the block index the row holds
  const __nv_bfloat16* chi; const __nv_bfloat16* clo; const float* gs; const float* cnorm; const int* perm;
  int M, Mpad, W, L, Hq, G, N;
  int q0, Mq, Nq;   // this call's queries: first query block (global index), number of blocks, number of tokens
  float scale_log2, t_base, t_rescue;  // thresholds as log2(alpha)
  int n_sink, n_local, n_recent;
  uint32_t* mask; uint32_t* dbg_base; uint32_t* dbg_rescue;
  unsigned int* counts;
};

constexpr int kTcThreads = 192;

template <int B>
__global__ void __launch_bounds__(kTcThreads, 2)
select_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmChi,
                 const __grid_constant__ CUtensorMap tmClo, const SelectParams p, unsigned int* status) {
  constexpr uint32_t kPanelC = 128 * 128;          // one 64-column panel of a 128-row centroid tile
  constexpr uint32_t kStage = 4 * kPanelC;         // hi panels 0,1 then lo panels 0,1
  constexpr uint32_t kPanelQ = B * 128;
  constexpr uint32_t kIdesc = idesc_bf16_f32(128, B, false);
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sC = smem;                                        // 64 KB
  unsigned char* sQ = sC + kStage;                                 // 2 panels
  float* sQn = reinterpret_cast<float*>(sQ + 2 * kPanelQ);         // B
  float* sRed = sQn + B;                                           // 32
  float* sLb = sRed + 32;
  __shared__ __align__(8) uint64_t bar_q, bar_cfull[2], bar_cempty[2], bar_tfull[2], bar_tempty[2];   // c*: [0] hi half, [1] lo half
  __shared__ uint32_t s_tmem;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per_i = p.L * p.Hq;
  const int il = p.Mq - 1 - static_cast<int>(blockIdx.x / per_i);   // query block inside this call's chunk
  const int i = p.q0 + il;                                            // its position in the sequence
  const int rem = static_cast<int>(blockIdx.x % per_i);
  const int l = rem / p.Hq, h = rem % p.Hq, hk = h / p.G;
  const int Hkv = p.Hq / p.G;
  const int n_tiles = i / 128 + 1;
  float* sLr = sLb + n_tiles * 128;
  const int crow0 = static_cast<int>((static_cast<int64_t>(l) * Hkv + hk) * p.Mpad);

  if (tid == 0) {
    mbar_init(smem_u32(&bar_q), 1);
    for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bar_cfull[s]), 1); mbar_init(smem_u32(&bar_cempty[s]), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&bar_tfull[s]), 1); mbar_init(smem_u32(&bar_tempty[s]), 4); }
    mbar_fence_init();
  }
  if (warp == 5) tmem_alloc(smem_u32(&s_tmem), 2 * B);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s_tmem;

  if (warp == 4) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmChi); tma_prefetch_desc(&tmClo);
      mbar_arrive_expect_tx(smem_u32(&bar_q), 2 * kPanelQ);
      tma_load_4d(smem_u32(sQ), &tmQ, smem_u32(&bar_q), 0, h, il * B, l);
      tma_load_4d(smem_u32(sQ + kPanelQ), &tmQ, smem_u32(&bar_q), 64, h, il * B, l);
      // the hi and lo halves of a centroid tile are separate pipeline slots: the hi half of the next tile is
      // fetched as soon as this tile's hi MMAs are done, i.e. under its lo MMAs and its epilogue
      const uint32_t dst = smem_u32(sC);
      for (int bt = 0; bt < n_tiles; ++bt) {
        if (bt > 0 && !mbar_wait(smem_u32(&bar_cempty[0]), (bt - 1) & 1, status, kWaitStageFree)) break;
        mbar_arrive_expect_tx(smem_u32(&bar_cfull[0]), kStage / 2);
        tma_load_2d(dst, &tmChi, smem_u32(&bar_cfull[0]), 0, crow0 + bt * 128);
        tma_load_2d(dst + kPanelC, &tmChi, smem_u32(&bar_cfull[0]), 64, crow0 + bt * 128);
        if (bt > 0 && !mbar_wait(smem_u32(&bar_cempty[1]), (bt - 1) & 1, status, kWaitStageFree)) break;
        mbar_arrive_expect_tx(smem_u32(&bar_cfull[1]), kStage / 2);
        tma_load_2d(dst + 2 * kPanelC, &tmClo, smem_u32(&bar_cfull[1]), 0, crow0 + bt * 128);
        tma_load_2d(dst + 3 * kPanelC, &tmClo, smem_u32(&bar_cfull[1]), 64, crow0 + bt * 128);
      }
    }
  } else if (warp == 5) {
    // ------------------------------- MMA issuer -------------------------------
    // The whole warp runs the loop; one elected lane issues the 16 MMAs of a tile in one go.
    {
      bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull));
      const uint64_t dchi = smem_desc_sw128(smem_u32(sC), 16, 1024);
      const uint64_t dclo = smem_desc_sw128(smem_u32(sC) + 2 * kPanelC, 16, 1024);
      const uint64_t dq = smem_desc_sw128(smem_u32(sQ), 16, 1024);
      for (int bt = 0; ok && bt < n_tiles; ++bt) {
        const int buf = bt & 1;
        ok = mbar_wait(smem_u32(&bar_cfull[0]), bt & 1, status, kWaitTmaFull);
        if (ok && bt >= 2) ok = mbar_wait(smem_u32(&bar_tempty[buf]), ((bt >> 1) - 1) & 1, status, kWaitTmemFree);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + buf * B;
        mma_ss_k128_commit_elect(d_tmem, dchi, dq, kIdesc, kPanelC, kPanelQ, smem_u32(&bar_cempty[0]), 0);
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_cfull[1]), bt & 1, status, kWaitTmaFull));
        if (!ok) break;
        tc_fence_after_sync();
        mma_ss_k128_commit_elect(d_tmem, dclo, dq, kIdesc, kPanelC, kPanelQ, smem_u32(&bar_cempty[1]), 1);
        mma_commit_elect(smem_u32(&bar_tfull[buf]));
      }
    }
    __syncwarp();
  } else {
    // ------------------------------- epilogue: one centroid row per thread -------------------------------
    const int row = warp * 32 + lane;
    bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull));
    const int n_tok = min(B, p.Nq - il * B);
    float qn_max, qn_spread;
    ok = query_norm_shifts<B, 128>(sQ, tid, n_tok, sQn, sRed, 1, ok, qn_max, qn_spread);   // sQn holds ||q_t|| - ||q||max
    for (int bt = 0; ok && bt < n_tiles; ++bt) {
      const int buf = bt & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_tfull[buf]), (bt >> 1) & 1, status, kWaitMmaDone));
      if (!ok) break;
      tc_fence_after_sync();
      const int prow = crow0 + bt * 128 + row;
      const int b = p.perm[prow];                 // the block this accumulator row belongs to
      const uint32_t taddr = tmem_base + buf * B + (static_cast<uint32_t>(warp * 32) << 16);
      float Lb, Lr;
      score_tile<B, true>(taddr, sQn, p.gs[prow], p.cnorm[prow], qn_max, qn_spread, n_tok, [&]() {
        tc_fence_before_sync();                   // hand the TMEM buffer back to the MMA warp
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bar_tempty[buf]));
      }, Lb, Lr);
      const bool causal = b <= i;
      if (RBS_DBG_OK(b >= 0 && b < p.Mpad, status, kDbgSelectPerm)) {
        sLb[b] = causal ? Lb : -INFINITY;
        sLr[b] = causal ? Lr : -INFINITY;
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == 5) tmem_dealloc(tmem_base, 2 * B);

  // row maxima over the causal candidates, thresholds, forced blocks, union, pack (all six warps)
  float mxb = -INFINITY, mxr = -INFINITY;
  for (int b = tid; b <= i; b += kTcThreads) { mxb = fmaxf(mxb, sLb[b]); mxr = fmaxf(mxr, sLr[b]); }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mxb = fmaxf(mxb, __shfl_xor_sync(0xffffffffu, mxb, o));
    mxr = fmaxf(mxr, __shfl_xor_sync(0xffffffffu, mxr, o));
  }
  if (lane == 0) { sRed[warp] = mxb; sRed[16 + warp] = mxr; }
  __syncthreads();
  mxb = sRed[0]; mxr = sRed[16];
#pragma unroll
  for (int w = 1; w < kTcThreads / 32; ++w) { mxb = fmaxf(mxb, sRed[w]); mxr = fmaxf(mxr, sRed[16 + w]); }
  const float thr_b = mxb + p.t_base, thr_r = mxr + p.t_rescue;
  const int64_t mrow = ((static_cast<int64_t>(l) * p.Hq + h) * p.Mq + il) * p.W;
  const bool all_forced = i >= p.M - p.n_recent;
  unsigned int cnt = 0;
  for (int w = warp; w < p.W; w += kTcThreads / 32) {
    const int b = w * 32 + lane;
    const bool valid = b <= i;
    bool kb = false, kr = false, kf = false;
    if (valid) {
      kb = sLb[b] >= thr_b;
      kr = sLr[b] >= thr_r;
      kf = all_forced || b < p.n_sink || b > i - p.n_local;
    }
    const uint32_t wb = __ballot_sync(0xffffffffu, kb), wr = __ballot_sync(0xffffffffu, kr);
    const uint32_t wf = __ballot_sync(0xffffffffu, kf);
    if (lane == 0 && RBS_DBG_OK(mrow >= 0 && mrow + w < static_cast<int64_t>(p.L) * p.Hq * p.Mq * p.W, status, kDbgSelectMask)) {
      const uint32_t word = wb | wr | wf;
      p.mask[mrow + w] = word;
      if (p.dbg_base) p.dbg_base[mrow + w] = wb;
      if (p.dbg_rescue) p.dbg_rescue[mrow + w] = wr;
      cnt += __popc(word);
    }
  }
  if (lane == 0 && cnt) atomicAdd(p.counts + l * p.Hq + h, cnt);
}

// ---------------------------------------------------------------------------------------------
// 3b. The same scoring as a persistent kernel, one CTA per SM, that serves TWO query heads of a KV group per work
//     item (l, KV head, query block, head pair).  The two heads score against the same centroids, so every centroid
//     tile is brought into shared memory once for both (half the L2 -> shared-memory traffic per score) and the
//     tensor core runs the two heads' products back to back (four accumulators in tensor memory: 2 heads x 2 buffers).
//     Warps 0-7 / 8-15: epilogue of head 0 / head 1.  A row of the accumulator (one centroid) is shared by two warps
//     with the same lane quarter of tensor memory: warp q reduces the first half of the block's tokens, warp q + 4
//     the second half and hands its two partial sums over through shared memory, so that every scheduler has four
//     epilogue warps to hide the latencies of the exponentials and of the tensor-memory loads behind one another.
//     Warp 16: TMA producer, which also fetches the NEXT item's two Q tiles while the current item is being scored;
//     warp 17: MMA issuer.  Each epilogue group keeps its running row maxima in registers and does its own threshold /
//     pack pass, during which the MMA warp is already filling the accumulators of the next item.
//     Work items are dealt round-robin, longest rows first.
// ---------------------------------------------------------------------------------------------
constexpr int kPairThreads = 576;
constexpr int kPairProducer = 16, kPairMma = 17;

// HALVES (blocks of 256): the two "heads" of an item are the two halves of 128 tokens of ONE head's query block; the
// sum over the block's tokens (Eq. block_aggregation) is then the sum of the two groups' sums, handed from the second
// group to the first like the token halves inside a group; the first group alone keeps the scores and writes the mask.
template <int B, bool HALVES>
__global__ void __launch_bounds__(kPairThreads, 1)
select_pair_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmChi,
                   const __grid_constant__ CUtensorMap tmClo, const SelectParams p, int n_items, int l_floats,
                   unsigned int* status) {
  constexpr uint32_t kPanelC = 128 * 128;          // one 64-column panel of a 128-row centroid tile
  constexpr uint32_t kStage = 4 * kPanelC;         // hi panels 0,1 then lo panels 0,1
  constexpr uint32_t kPanelQ = B * 128;
  constexpr uint32_t kQTile = 2 * kPanelQ;         // one head's Q tile
  // the two heads' tiles are ONE operand of 2 B rows: a product with N = 2 B reads the centroid panel from shared
  // memory once for both heads
  constexpr uint32_t kIdesc = idesc_bf16_f32(128, 2 * B, false);
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sC = smem;                                        // 64 KB
  unsigned char* sQ = sC + kStage;                                 // [slot 2][panel 2][head 2][kPanelQ]
  float* sQn = reinterpret_cast<float*>(sQ + 4 * kQTile);          // [head 2][B]
  float* sL = sQn + 2 * B;                                         // [head 2][branch 2][l_floats]
  __shared__ __align__(8) uint64_t bar_qfull[2], bar_qempty[2], bar_cfull[4], bar_cempty[4], bar_tfull[2][2], bar_tempty[2][2];
  __shared__ __align__(8) uint64_t bar_half[2][4][2];      // [head][lane quarter][tile parity]: second half's sums are there
  __shared__ __align__(8) float2 sHalf[2][4][2][32];       // the partial sums (base, rescue) of the second half
  __shared__ __align__(8) uint64_t bar_group[4][2];        // HALVES: the second group's sums are there
  __shared__ __align__(8) float2 sGroup[4][2][32];
  __shared__ float sRed[2][2][8], sRedQ[2][16], sQstat[2][2];
  __shared__ uint32_t s_tmem;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Hkv = p.Hq / p.G, GP = HALVES ? p.G : p.G / 2;   // items per (batch, KV head, query block)
  const int per_i = p.L * Hkv * GP;
  constexpr int QB = HALVES ? 2 * B : B;                     // tokens of a query block

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      // a Q slot is free once the item's last product has been read by the tensor core AND both epilogue groups have
      // taken their query norms from it (an item of one or two centroid tiles can be multiplied completely before the
      // epilogue groups even reach it: without their arrivals the slot would be refilled under them, and the full
      // barrier could run two phases ahead of a waiter, which a parity wait cannot tell from no progress)
      mbar_init(smem_u32(&bar_qfull[s]), 1); mbar_init(smem_u32(&bar_qempty[s]), 3);
      mbar_init(smem_u32(&bar_cfull[s]), 1); mbar_init(smem_u32(&bar_cempty[s]), 1);        // one pair per 64-column
      mbar_init(smem_u32(&bar_cfull[2 + s]), 1); mbar_init(smem_u32(&bar_cempty[2 + s]), 1);   // panel: hi 0, hi 1, lo 0, lo 1
      for (int hw = 0; hw < 2; ++hw) {
        mbar_init(smem_u32(&bar_tfull[hw][s]), 1); mbar_init(smem_u32(&bar_tempty[hw][s]), 8);
        for (int q = 0; q < 4; ++q) mbar_init(smem_u32(&bar_half[hw][q][s]), 1);
      }
      for (int q = 0; q < 4; ++q) mbar_init(smem_u32(&bar_group[q][s]), 1);
    }
    mbar_fence_init();
  }
  if (warp == kPairMma) tmem_alloc(smem_u32(&s_tmem), 4 * B);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s_tmem;

  // item w -> (query block of the chunk, batch, KV head, head pair); longest rows first
  auto decode = [&](int w, int& il, int& l, int& hk, int& h0) {
    il = p.Mq - 1 - w / per_i;
    int rem = w % per_i;
    const int pr = rem % GP; rem /= GP;
    hk = rem % Hkv; l = rem / Hkv;
    h0 = hk * p.G + (HALVES ? pr : 2 * pr);
  };
  // tensor-memory columns of the accumulator of group hw, buffer buf: the two groups' accumulators of a buffer side by
  // side (one product writes both; HALVES reads them as one row of 2 B tokens)
  auto acc_col = [](int hw, uint32_t buf) -> uint32_t { return (buf * 2 + hw) * B; };

  if (warp == kPairProducer) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmChi); tma_prefetch_desc(&tmClo);
      uint32_t nq = 0, nc = 0;     // Q loads (items) and centroid tiles issued so far
      bool ok = true;
      auto load_q = [&](int w) {
        int il, l, hk, h0;
        decode(w, il, l, hk, h0);
        const uint32_t slot = nq & 1;
        if (nq >= 2 && !mbar_wait(smem_u32(&bar_qempty[slot]), ((nq >> 1) - 1) & 1, status, kWaitStageFree)) { ok = false; return; }
        const uint32_t dst = smem_u32(sQ) + slot * 2 * kQTile, bar = smem_u32(&bar_qfull[slot]);
        mbar_arrive_expect_tx(bar, 2 * kQTile);
        for (int hw = 0; hw < 2; ++hw) {
          const int hq = HALVES ? h0 : h0 + hw, tok0 = HALVES ? il * QB + hw * B : il * B;
          tma_load_4d(dst + hw * kPanelQ, &tmQ, bar, 0, hq, tok0, l);
          tma_load_4d(dst + hw * kPanelQ + kQTile, &tmQ, bar, 64, hq, tok0, l);
        }
        ++nq;
      };
      int w = blockIdx.x;
      if (w < n_items) load_q(w);
      for (; ok && w < n_items; w += gridDim.x) {
        int il, l, hk, h0;
        decode(w, il, l, hk, h0);
        const int n_tiles = (p.q0 + il) / 128 + 1;
        const int crow0 = static_cast<int>((static_cast<int64_t>(l) * Hkv + hk) * p.Mpad);
        const uint32_t dst = smem_u32(sC);
        for (int bt = 0; ok && bt < n_tiles; ++bt, ++nc) {
          // The four 64-column panels of a centroid tile (hi 0, hi 1, lo 0, lo 1) are separate pipeline slots: a panel
          // of the NEXT tile is requested as soon as the products with that panel of this one are done, a quarter, a
          // half, ... of the tile's tensor work before its end.
          for (int q = 0; q < 4; ++q) {
            if (nc > 0 && !mbar_wait(smem_u32(&bar_cempty[q]), (nc - 1) & 1, status, kWaitStageFree)) { ok = false; break; }
            mbar_arrive_expect_tx(smem_u32(&bar_cfull[q]), kPanelC);
            tma_load_2d(dst + q * kPanelC, q < 2 ? &tmChi : &tmClo, smem_u32(&bar_cfull[q]), (q & 1) * 64, crow0 + bt * 128);
          }
          if (!ok) break;
          // the next item's Q tiles go out right behind this item's first centroid tile
          if (bt == 0 && w + static_cast<int>(gridDim.x) < n_items) load_q(w + gridDim.x);
        }
      }
    }
  } else if (warp == kPairMma) {
    // ------------------------------- MMA issuer -------------------------------
    const uint64_t dchi = smem_desc_sw128(smem_u32(sC), 16, 1024);
    uint32_t nt = 0, k = 0;      // centroid tiles and items processed so far
    bool ok = true;
    for (int w = blockIdx.x; ok && w < n_items; w += gridDim.x, ++k) {
      const int il = p.Mq - 1 - w / per_i;
      const int n_tiles = (p.q0 + il) / 128 + 1;
      const uint32_t slot = k & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_qfull[slot]), (k >> 1) & 1, status, kWaitTmaFull));
      const uint64_t dq = smem_desc_sw128(smem_u32(sQ) + slot * 2 * kQTile, 16, 1024);
      for (int bt = 0; ok && bt < n_tiles; ++bt, ++nt) {
        const uint32_t buf = nt & 1;
        ok = mbar_wait(smem_u32(&bar_cfull[0]), nt & 1, status, kWaitTmaFull);
        if (ok && nt >= 2) ok = mbar_wait(smem_u32(&bar_tempty[0][buf]), ((nt >> 1) - 1) & 1, status, kWaitTmemFree) &&
                                mbar_wait(smem_u32(&bar_tempty[1][buf]), ((nt >> 1) - 1) & 1, status, kWaitTmemFree);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d = tmem_base + acc_col(0, buf);
        constexpr uint64_t kPanelQ16 = kQTile >> 4, kPanelC16 = kPanelC >> 4;   // panel strides in descriptor units
        // panel q of the centroid tile times panel q & 1 of the two heads' Q tiles
        for (int q = 0; q < 4; ++q) {
          if (q > 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_cfull[q]), nt & 1, status, kWaitTmaFull));
            if (!ok) break;
            tc_fence_after_sync();
          }
          mma_ss_k64_commit_elect(d, dchi + q * kPanelC16, dq + (q & 1) * kPanelQ16, kIdesc, smem_u32(&bar_cempty[q]), q > 0);
        }
        if (!ok) break;
        mma_commit_elect(smem_u32(&bar_tfull[0][buf]));
        mma_commit_elect(smem_u32(&bar_tfull[1][buf]));
        if (bt == n_tiles - 1) mma_commit_elect(smem_u32(&bar_qempty[slot]));   // this item's Q tiles are free
      }
    }
    __syncwarp();
  } else {
    // ------------------------------- epilogue groups: one centroid row per pair of threads -------------------------------
    const int hw = warp >> 3, wq = warp & 3, half = (warp >> 2) & 1;   // head of the pair, lane quarter, token half
    const int wg = warp & 7;                                           // warp inside the group
    const int row = wq * 32 + lane;
    const int wtid = tid & 255;
    const int gbar = 1 + hw;                                           // named barrier of this group (256 threads)
    float* sQn_h = sQn + hw * B;
    float* sLb = sL + (hw * 2) * l_floats;
    float* sLr = sLb + l_floats;
    uint32_t nt = 0, k = 0;
    bool ok = true;
    for (int w = blockIdx.x; ok && w < n_items; w += gridDim.x, ++k) {
      int il, l, hk, h0;
      decode(w, il, l, hk, h0);
      const int i = p.q0 + il, h = HALVES ? h0 : h0 + hw;
      const int n_tiles = i / 128 + 1;
      const int crow0 = static_cast<int>((static_cast<int64_t>(l) * Hkv + hk) * p.Mpad);
      const uint32_t slot = k & 1;
      const unsigned char* q = sQ + slot * 2 * kQTile + hw * kPanelQ;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_qfull[slot]), (k >> 1) & 1, status, kWaitTmaFull));
      const int n_tok = HALVES ? max(0, min(B, p.Nq - il * QB - hw * B)) : min(B, p.Nq - il * B);   // of this group
      float qn_max, qn_spread;
      ok = query_norm_shifts<B, 256, kQTile>(q, wtid, n_tok, sQn_h, &sRedQ[hw][0], gbar, ok, qn_max, qn_spread);
      if (wtid == 0) mbar_arrive(smem_u32(&bar_qempty[slot]));      // the Q tile itself is not read again by this group
      if (HALVES) {
        // the norms' maximum and spread are those of the whole block of 2 B tokens: exchange with the other group
        if (wtid == 0) { sQstat[hw][0] = qn_max; sQstat[hw][1] = n_tok > 0 ? qn_max - qn_spread : INFINITY; }
        ok = group_all<512>(ok, 3);                                  // both groups (and a failed wait ends both)
        const float g_max = fmaxf(sQstat[0][0], sQstat[1][0]), g_min = fminf(sQstat[0][1], sQstat[1][1]);
        if (wtid < B) sQn_h[wtid] -= g_max - qn_max;                // shifts relative to the block's maximum
        qn_max = g_max;
        qn_spread = g_max - g_min;
        ok = group_all<512>(ok, 3);                                  // shifts written; sQstat may be rewritten by the next item
      }
      float mxb = -INFINITY, mxr = -INFINITY;     // running maxima of this thread's L values (causal blocks only)
      for (int bt = 0; ok && bt < n_tiles; ++bt, ++nt) {
        const uint32_t buf = nt & 1;
        // the row's constants are requested before the wait for the accumulator: their latency passes under it
        const int prow = crow0 + bt * 128 + row;
        const bool prow_ok = RBS_DBG_OK(prow >= 0 && prow < p.L * Hkv * p.Mpad, status, kDbgSelectCentroid);
        const float gs = prow_ok ? __ldg(p.gs + prow) : 0.f, cn = prow_ok ? __ldg(p.cnorm + prow) : 0.f;
        const int b_row = prow_ok ? __ldg(p.perm + prow) : 0x7fffffff;   // the block this accumulator row belongs to
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_tfull[hw][buf]), (nt >> 1) & 1, status, kWaitMmaDone));
        if (!ok) break;
        tc_fence_after_sync();
        (void)RBS_DBG_OK(acc_col(hw, buf) + B <= 4u * B, status, kDbgSelectTmem);
        const uint32_t taddr = tmem_base + acc_col(hw, buf) + (static_cast<uint32_t>(wq * 32) << 16);
        // the decisions of score_tile, identical in the two warps that share these rows
        const float mb = qn_max * cn * 1.0001f;
        const bool no_rescue = __all_sync(0xffffffffu, gs == 0.f);
        const bool cheap = __all_sync(0xffffffffu, mb <= 60.0f && fmaf(gs, qn_spread, 2.0f * mb) <= 120.0f);
        const uint32_t hbar = smem_u32(&bar_half[hw][wq][buf]);
        auto release = [&]() {                        // hand the TMEM buffer back to the MMA warp
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bar_tempty[hw][buf]));
        };
        const uint32_t gbar2 = smem_u32(&bar_group[wq][buf]);
        if (half == 1) {
          if (cheap) {
            float sb, sr;
            partial_sums<B, B / 2>(taddr, sQn_h, gs, -mb, no_rescue, n_tok, B / 2, sb, sr);
            sHalf[hw][wq][buf][lane] = make_float2(sb, sr);
          }
          release();                                  // (also orders the shared-memory writes before the arrival below)
          if (lane == 0) mbar_arrive(hbar);
        } else if (HALVES && hw == 1) {
          // second group, first token half: its group's sums go on to the first group
          float sb = 0.f, sr = 0.f;
          if (cheap) partial_sums<B, B / 2>(taddr, sQn_h, gs, -mb, no_rescue, n_tok, 0, sb, sr);
          ok = __all_sync(0xffffffffu, mbar_wait(hbar, (nt >> 1) & 1, status, kWaitPReady));
          if (cheap) {
            const float2 o = sHalf[hw][wq][buf][lane];
            sGroup[wq][buf][lane] = make_float2(sb + o.x, sr + o.y);
          }
          release();
          if (lane == 0) mbar_arrive(gbar2);
        } else {
          float Lb, Lr;
          if (cheap) {
            float sb, sr;
            partial_sums<B, B / 2>(taddr, sQn_h, gs, -mb, no_rescue, n_tok, 0, sb, sr);
            ok = __all_sync(0xffffffffu, mbar_wait(hbar, (nt >> 1) & 1, status, kWaitPReady));
            float2 o = sHalf[hw][wq][buf][lane];
            if (HALVES) {
              ok = __all_sync(0xffffffffu, ok && mbar_wait(gbar2, (nt >> 1) & 1, status, kWaitPReady));
              const float2 o2 = sGroup[wq][buf][lane];
              o.x += o2.x; o.y += o2.y;
            }
            // the buffer (and with it these slots of sHalf / sGroup) goes back only after the partners' sums have been taken
            release();
            Lb = mb + fast_log2(sb + o.x);
            Lr = no_rescue ? Lb : fmaf(qn_max, gs, mb) + fast_log2(sr + o.y);
          } else {
            // exact shifts: this warp takes the whole row alone (HALVES: both groups' accumulators, side by side)
            if (HALVES) {
              const int n_all = min(QB, p.Nq - il * QB);
              score_tile<QB, false>(taddr, sQn, gs, cn, qn_max, qn_spread, n_all, []() {}, Lb, Lr);
            } else {
              score_tile<B, false>(taddr, sQn_h, gs, cn, qn_max, qn_spread, n_tok, []() {}, Lb, Lr);
            }
            ok = __all_sync(0xffffffffu, mbar_wait(hbar, (nt >> 1) & 1, status, kWaitPReady));
            if (HALVES) ok = __all_sync(0xffffffffu, ok && mbar_wait(gbar2, (nt >> 1) & 1, status, kWaitPReady));
            release();
          }
          const int b = b_row;
          if (b > i) { Lb = -INFINITY; Lr = -INFINITY; }
          if (RBS_DBG_OK(b >= 0 && b < l_floats && b < p.Mpad, status, kDbgSelectPerm)) {
            sLb[b] = Lb;
            sLr[b] = Lr;
          }
          mxb = fmaxf(mxb, Lb);
          mxr = fmaxf(mxr, Lr);
        }
      }
      // row maxima over the causal candidates, thresholds, forced blocks, union, pack: this group alone
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        mxb = fmaxf(mxb, __shfl_xor_sync(0xffffffffu, mxb, o));
        mxr = fmaxf(mxr, __shfl_xor_sync(0xffffffffu, mxr, o));
      }
      if (lane == 0) { sRed[hw][0][wg] = mxb; sRed[hw][1][wg] = mxr; }
      ok = group_all<256>(ok, gbar);
      mxb = sRed[hw][0][0]; mxr = sRed[hw][1][0];
#pragma unroll
      for (int u = 1; u < 8; ++u) { mxb = fmaxf(mxb, sRed[hw][0][u]); mxr = fmaxf(mxr, sRed[hw][1][u]); }
      const float thr_b = mxb + p.t_base, thr_r = mxr + p.t_rescue;
      const int64_t mrow = ((static_cast<int64_t>(l) * p.Hq + h) * p.Mq + il) * p.W;
      const bool all_forced = i >= p.M - p.n_recent;
      unsigned int cnt = 0;
      for (int wd = wg; ok && !(HALVES && hw == 1) && wd < p.W; wd += 8) {
        const int b = wd * 32 + lane;
        const bool valid = b <= i;
        bool kb = false, kr = false, kf = false;
        if (valid) {
          kb = sLb[b] >= thr_b;
          kr = sLr[b] >= thr_r;
          kf = all_forced || b < p.n_sink || b > i - p.n_local;
        }
        const uint32_t wb = __ballot_sync(0xffffffffu, kb), wr = __ballot_sync(0xffffffffu, kr);
        const uint32_t wf = __ballot_sync(0xffffffffu, kf);
        if (lane == 0 && RBS_DBG_OK(mrow >= 0 && mrow + wd < static_cast<int64_t>(p.L) * p.Hq * p.Mq * p.W, status, kDbgSelectMask)) {
          const uint32_t word = wb | wr | wf;
          p.mask[mrow + wd] = word;
          if (p.dbg_base) p.dbg_base[mrow + wd] = wb;
          if (p.dbg_rescue) p.dbg_rescue[mrow + wd] = wr;
          cnt += __popc(word);
        }
      }
      if (lane == 0 && cnt) atomicAdd(p.counts + l * p.Hq + h, cnt);
      // the L arrays, norms and maxima may be overwritten after this; `ok` leaves it identical in the whole group, so
      // that its warps leave the item loop together (a group split over a named barrier would wait forever)
      ok = group_all<256>(ok, gbar);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == kPairMma) tmem_dealloc(tmem_base, 4 * B);
}

__global__ void density_kernel(const unsigned int* __restrict__ counts, int n, int q0, int Mq, float* __restrict__ density) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) {
    // causal pairs of query blocks q0 .. q0 + Mq - 1: sum of (i + 1)
    const double pairs = static_cast<double>(Mq) * static_cast<double>(q0) + 0.5 * static_cast<double>(Mq) * static_cast<double>(Mq + 1);
    density[t] = static_cast<float>(static_cast<double>(counts[t]) / pairs);
  }
}

template <int B>
static rbs_status launch_select_tc(const SelectParams& p, const rbs_tensor& Q, cudaStream_t s) {
  CUtensorMap tmQ, tmChi, tmClo;
  rbs_status st = make_tmap_lthd(&tmQ, Q.ptr, p.L, p.Nq, p.Hq, kHeadDim, Q.stride_batch, Q.stride_token, Q.stride_head, 64, B, true);
  if (st != RBS_OK) return st;
  const int64_t rows = static_cast<int64_t>(p.L) * (p.Hq / p.G) * p.Mpad;
  if ((st = make_tmap_2d(&tmChi, p.chi, rows, kHeadDim, 64, 128)) != RBS_OK) return st;
  if ((st = make_tmap_2d(&tmClo, p.clo, rows, kHeadDim, 64, 128)) != RBS_OK) return st;
  unsigned int* status = device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  const int n_tiles_max = (p.M + 127) / 128;
  const size_t smem = static_cast<size_t>(4) * 128 * 128 + 2 * static_cast<size_t>(B) * 128 +
                      (B + 32) * sizeof(float) + 2 * static_cast<size_t>(n_tiles_max) * 128 * sizeof(float);
  auto kern = select_tc_kernel<B>;
  if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem)) != RBS_OK) return st;
  const long long n_cta = static_cast<long long>(p.L) * p.Hq * p.Mq;
  if (n_cta > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  kern<<<static_cast<unsigned>(n_cta), kTcThreads, smem, s>>>(tmQ, tmChi, tmClo, p, status);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

// Shared memory of select_pair_kernel for M blocks; 0 when this shape has to stay on the one-head kernel
// (blocks of 256: two Q tiles of 64 KB each do not fit twice; an odd group size; very long rows).
template <int B>
static size_t pair_kernel_smem(const SelectParams& p, int* l_floats) {
  if (B <= 128 && p.G % 2 != 0) return 0;
  constexpr int BT = B > 128 ? 128 : B;     // tokens per Q tile (blocks of 256: two tiles of 128 of one head)
  *l_floats = (p.M + 127) / 128 * 128;
  const size_t bytes = static_cast<size_t>(4) * 128 * 128 + 4 * 2 * static_cast<size_t>(BT) * 128 + 2 * BT * sizeof(float) +
                       4 * static_cast<size_t>(*l_floats) * sizeof(float);
  return bytes <= 227 * 1024 - 8 * 1024 ? bytes : 0;   // up to 7 KB of static shared memory beside it
}

template <int B>
static rbs_status launch_select_pair(const SelectParams& p, const rbs_tensor& Q, size_t smem, int l_floats, cudaStream_t s) {
  CUtensorMap tmQ, tmChi, tmClo;
  constexpr bool kHalves = B > 128;
  constexpr int BT = kHalves ? 128 : B;
  rbs_status st = make_tmap_lthd(&tmQ, Q.ptr, p.L, p.Nq, p.Hq, kHeadDim, Q.stride_batch, Q.stride_token, Q.stride_head, 64, BT, true);
  if (st != RBS_OK) return st;
  const int64_t rows = static_cast<int64_t>(p.L) * (p.Hq / p.G) * p.Mpad;
  if ((st = make_tmap_2d(&tmChi, p.chi, rows, kHeadDim, 64, 128)) != RBS_OK) return st;
  if ((st = make_tmap_2d(&tmClo, p.clo, rows, kHeadDim, 64, 128)) != RBS_OK) return st;
  unsigned int* status = device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  auto kern = select_pair_kernel<BT, kHalves>;
  if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem)) != RBS_OK) return st;
  const long long n_items = static_cast<long long>(p.L) * (kHalves ? p.Hq : p.Hq / 2) * p.Mq;
  if (n_items > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  const int grid = static_cast<int>(n_items < sm_count() ? n_items : sm_count());
  kern<<<grid, kPairThreads, smem, s>>>(tmQ, tmChi, tmClo, p, static_cast<int>(n_items), l_floats, status);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

template <int B>
static rbs_status launch_select(const SelectParams& p, const rbs_tensor& Q, cudaStream_t s) {
  int l_floats = 0;
  const size_t smem = pair_kernel_smem<B>(p, &l_floats);
  if (smem != 0) return launch_select_pair<B>(p, Q, smem, l_floats, s);
  return launch_select_tc<B>(p, Q, s);
}

}  // namespace rbs

// q_start_block / n_q_tokens: the queries of this call are tokens [q_start_block * B, q_start_block * B + n_q_tokens)
// of the sequence; Q, mask and density cover only them (n_q_tokens < 0: the whole sequence).
static rbs_status select_impl(const rbs_shape* shape, int q_start_block, int n_q_tokens, rbs_tensor Q, rbs_stats stats, int beta_mode, float alpha_base,
                              float alpha_rescue, int n_sink, int n_local, int n_recent, uint32_t* mask,
                              float* density, uint32_t* dbg_base_mask, uint32_t* dbg_rescue_mask,
                              void* workspace, size_t workspace_bytes, void* stream) {
  using namespace rbs;
  rbs::NvtxRange nvtx_range("rbs_select");
  rbs_status st = check_shape(shape);
  if (st != RBS_OK) return st;
  st = check_tensor(Q);
  if (st != RBS_OK) return st;
  if (!stats.centroid || !stats.radius || !stats.beta || !stats.rq || !mask || !density) return RBS_ERR_INVALID_ARG;
  if (!(alpha_base > 0.f) || !(alpha_rescue > 0.f)) return RBS_ERR_INVALID_ARG;
  if (n_sink < 0 || n_local < 0 || n_recent < 0) return RBS_ERR_INVALID_ARG;
  Dims x = make_dims(*shape);
  if (n_q_tokens < 0) { q_start_block = 0; n_q_tokens = x.N; }
  if ((st = check_chunk(x, q_start_block, n_q_tokens)) != RBS_OK) return st;
  SelectWorkspace ws = select_workspace(x);
  if (workspace == nullptr || workspace_bytes < ws.bytes) return RBS_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return RBS_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned char* wsp = static_cast<unsigned char*>(workspace);
  __nv_bfloat16* chi = reinterpret_cast<__nv_bfloat16*>(wsp + ws.off_chi);
  __nv_bfloat16* clo = reinterpret_cast<__nv_bfloat16*>(wsp + ws.off_clo);
  float* gs = reinterpret_cast<float*>(wsp + ws.off_g);
  int* perm = reinterpret_cast<int*>(wsp + ws.off_perm);
  float* cnorm = reinterpret_cast<float*>(wsp + ws.off_cn);
  unsigned int* counts = reinterpret_cast<unsigned int*>(wsp + ws.off_counts);
  const float scale_log2 = kLog2e / sqrtf(static_cast<float>(x.d));

  int P = 1;
  while (P < x.M) P <<= 1;
  if (P < 2) P = 2;
  const size_t coeff_smem = static_cast<size_t>(P) * sizeof(float);
  RBS_CUDA_OK(cudaMemsetAsync(counts, 0, static_cast<size_t>(x.L) * x.Hq * sizeof(unsigned int), s));
  rescue_coeff_kernel<<<x.L * x.Hkv, kCoeffThreads, coeff_smem, s>>>(stats.radius, x.M, P, scale_log2, stats.beta,
                                                                     stats.rq, gs, perm, ws.Mpad, beta_mode);
  RBS_CUDA_OK(cudaGetLastError());
  const int64_t rows = static_cast<int64_t>(x.L) * x.Hkv * ws.Mpad;
  const int64_t n_thr = rows * (kHeadDim / 4);
  split_centroid_kernel<<<static_cast<unsigned>((n_thr + 255) / 256), 256, 0, s>>>(stats.centroid, perm, x.M, ws.Mpad, rows, scale_log2, chi, clo, cnorm);
  RBS_CUDA_OK(cudaGetLastError());

  SelectParams p;
  p.Q = static_cast<const __nv_bfloat16*>(Q.ptr); p.qsb = Q.stride_batch; p.qst = Q.stride_token; p.qsh = Q.stride_head;
  p.chi = chi; p.clo = clo; p.gs = gs; p.cnorm = cnorm; p.perm = perm;
  p.M = x.M; p.Mpad = ws.Mpad; p.W = x.W; p.L = x.L; p.Hq = x.Hq; p.G = x.G; p.N = x.N;
  p.q0 = q_start_block; p.Nq = n_q_tokens; p.Mq = (n_q_tokens + x.B - 1) / x.B;
  p.scale_log2 = scale_log2; p.t_base = log2f(alpha_base); p.t_rescue = log2f(alpha_rescue);
  p.n_sink = n_sink; p.n_local = n_local; p.n_recent = n_recent;
  p.mask = mask; p.dbg_base = dbg_base_mask; p.dbg_rescue = dbg_rescue_mask; p.counts = counts;
  if (x.B == 256) st = launch_select<256>(p, Q, s);
  else st = (x.B == 128) ? launch_select<128>(p, Q, s) : launch_select<64>(p, Q, s);
  if (st != RBS_OK) return st;
  const int nh = x.L * x.Hq;
  density_kernel<<<(nh + 127) / 128, 128, 0, s>>>(counts, nh, p.q0, p.Mq, density);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

extern "C" rbs_status rbs_select(const rbs_shape* shape, rbs_tensor Q, rbs_stats stats, float alpha_base,
                                 float alpha_rescue, int n_sink, int n_local, int n_recent, uint32_t* mask,
                                 float* density, uint32_t* dbg_base_mask, uint32_t* dbg_rescue_mask,
                                 void* workspace, size_t workspace_bytes, void* stream) {
  return select_impl(shape, -1, -1, Q, stats, 0, alpha_base, alpha_rescue, n_sink, n_local, n_recent, mask, density,
                     dbg_base_mask, dbg_rescue_mask, workspace, workspace_bytes, stream);
}

extern "C" rbs_status rbs_select_chunk(const rbs_shape* shape, int q_start_block, int n_q_tokens, rbs_tensor Q,
                                       rbs_stats stats, float alpha_base, float alpha_rescue, int n_sink, int n_local,
                                       int n_recent, uint32_t* mask, float* density, uint32_t* dbg_base_mask,
                                       uint32_t* dbg_rescue_mask, void* workspace, size_t workspace_bytes, void* stream) {
  if (n_q_tokens <= 0) return RBS_ERR_INVALID_ARG;
  return select_impl(shape, q_start_block, n_q_tokens, Q, stats, 0, alpha_base, alpha_rescue, n_sink, n_local, n_recent,
                     mask, density, dbg_base_mask, dbg_rescue_mask, workspace, workspace_bytes, stream);
}

extern "C" rbs_status rbs_select_variant(const rbs_shape* shape, rbs_tensor Q, rbs_stats stats, rbs_selector which,
                                         float alpha_base, float alpha_rescue, int n_sink, int n_local, int n_recent,
                                         uint32_t* mask, float* density, uint32_t* dbg_base_mask,
                                         uint32_t* dbg_rescue_mask, void* workspace, size_t workspace_bytes,
                                         void* stream) {
  constexpr float kDisabled = 2.0f;   // alpha > 1 empties a branch
  switch (which) {
    case RBS_SELECTOR_RBS:
      return select_impl(shape, -1, -1, Q, stats, 0, alpha_base, alpha_rescue, n_sink, n_local, n_recent, mask, density,
                         dbg_base_mask, dbg_rescue_mask, workspace, workspace_bytes, stream);
    case RBS_SELECTOR_CENTROID_ONLY:
      return select_impl(shape, -1, -1, Q, stats, 1, alpha_base, kDisabled, n_sink, n_local, n_recent, mask, density,
                         dbg_base_mask, dbg_rescue_mask, workspace, workspace_bytes, stream);
    case RBS_SELECTOR_FULL_L2:
      return select_impl(shape, -1, -1, Q, stats, 2, kDisabled, alpha_rescue, n_sink, n_local, n_recent, mask, density,
                         dbg_base_mask, dbg_rescue_mask, workspace, workspace_bytes, stream);
  }
  return RBS_ERR_INVALID_ARG;
}

// ---------------------------------------------------------------------------------------------
// rbs_select_static: the same selection for callers that cannot supply or allocate scratch memory.
// The scratch is this fixed device array.  Its name is only a host-side handle here: the kernels need the
// device address, which is looked up once per device (with that device current) and then reused.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_select_static_scratch[RBS_SELECT_STATIC_SCRATCH_BYTES];

#include <mutex>

extern "C" rbs_status rbs_select_static(const rbs_shape* shape, rbs_tensor Q, rbs_stats stats, float alpha_base,
                                        float alpha_rescue, int n_sink, int n_local, int n_recent, uint32_t* mask,
                                        float* density, uint32_t* dbg_base_mask, uint32_t* dbg_rescue_mask,
                                        void* stream) {
  using namespace rbs;
  constexpr int kMaxDevices = 64;
  static void* scratch_of_device[kMaxDevices] = {nullptr};
  static std::mutex lock;
  rbs_status st = check_shape(shape);
  if (st != RBS_OK) return st;
  // sizes beyond the fixed array are refused before anything touches the GPU
  if (select_workspace(make_dims(*shape)).bytes > RBS_SELECT_STATIC_SCRATCH_BYTES) return RBS_ERR_WORKSPACE;
  int dev = -1;
  RBS_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return RBS_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> guard(lock);
    if (scratch_of_device[dev] == nullptr) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_select_static_scratch) != cudaSuccess || p == nullptr) return RBS_ERR_CUDA;
      scratch_of_device[dev] = p;
    }
    scratch = scratch_of_device[dev];
  }
  return rbs_select(shape, Q, stats, alpha_base, alpha_rescue, n_sink, n_local, n_recent, mask, density,
                    dbg_base_mask, dbg_rescue_mask, scratch, RBS_SELECT_STATIC_SCRATCH_BYTES, stream);
}
