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

namespace rbs {

// ---------------------------------------------------------------------------------------------
// 1. per (l, KV head): sort radii, quantiles, beta, g = r * beta
// ---------------------------------------------------------------------------------------------
constexpr int kCoeffThreads = 1024;

__global__ void __launch_bounds__(kCoeffThreads)
rescue_coeff_kernel(const float* __restrict__ radius, int M, int P /* pow2 >= M */, float scale_log2,
                    float* __restrict__ beta, float* __restrict__ rq, float* __restrict__ g, int Mpad,
                    int beta_mode /* 0: Eq. (beta), 1: beta = 0, 2: beta = 1 */) {
  extern __shared__ float s_sorted[];
  __shared__ float s_q[2];
  const int hd = blockIdx.x, tid = threadIdx.x;
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
  for (int idx = tid; idx < Mpad; idx += kCoeffThreads) {
    float bt = 0.f, rb = 0.f;
    if (idx < M) {
      rb = r[idx];
      bt = live ? fminf(fmaxf((rb - r_low) * inv, 0.f), 1.f) : 0.f;
      if (beta_mode == 1) bt = 0.f;
      if (beta_mode == 2) bt = 1.f;
      beta[static_cast<int64_t>(hd) * M + idx] = bt;
    }
    g[static_cast<int64_t>(hd) * Mpad + idx] = rb * bt;
  }
}

// ---------------------------------------------------------------------------------------------
// 2. fp32 centroid -> bf16 hi + bf16 lo, rows padded to Mpad with zeros
// ---------------------------------------------------------------------------------------------
__global__ void split_centroid_kernel(const float* __restrict__ centroid, int M, int Mpad, int64_t n_rows_padded,
                                      __nv_bfloat16* __restrict__ chi, __nv_bfloat16* __restrict__ clo,
                                      float* __restrict__ cnorm) {
  // one thread per 4 elements, one warp per centroid row (also writes the row's L2 norm)
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t row = t / (kHeadDim / 4);
  const int c4 = static_cast<int>(t % (kHeadDim / 4));
  if (row >= n_rows_padded) return;   // whole warps: the grid covers rows in units of 32 threads
  const int64_t hd = row / Mpad;
  const int b = static_cast<int>(row % Mpad);
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (b < M) v = *reinterpret_cast<const float4*>(centroid + (hd * M + b) * kHeadDim + c4 * 4);
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
  const __nv_bfloat16* chi; const __nv_bfloat16* clo; const float* g; const float* cnorm;
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
    bool ok = mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull);
    for (int tok = tid; ok && tok < B; tok += 128) {   // raw query norms ||q_t||_2
      float s2 = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 v = *reinterpret_cast<const uint4*>(sQ + (c >> 3) * kPanelQ + tok * 128 + (((c & 7) ^ (tok & 7)) << 4));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float a = bf16lo(w[k]), c2 = bf16hi(w[k]);
          s2 = fmaf(a, a, s2);
          s2 = fmaf(c2, c2, s2);
        }
      }
      sQn[tok] = sqrtf(s2);
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");   // the four epilogue warps
    // largest query norm of the block: with it, ||q|| ||c_b|| bounds every logit of block b from above
    float qn_max = 0.f;
#pragma unroll
    for (int t = lane; t < B; t += 32) qn_max = fmaxf(qn_max, sQn[t]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) qn_max = fmaxf(qn_max, __shfl_xor_sync(0xffffffffu, qn_max, o));
    const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2);
    const int n_tok = min(B, p.Nq - il * B);
    for (int bt = 0; ok && bt < n_tiles; ++bt) {
      const int buf = bt & 1;
      ok = mbar_wait(smem_u32(&bar_tfull[buf]), (bt >> 1) & 1, status, kWaitMmaDone);
      if (!ok) break;
      tc_fence_after_sync();
      const int b = bt * 128 + row;
      const float gb = p.g[crow0 + b];            // r_b beta_b, unscaled
      const uint64_t gb2 = f2_pack(gb, gb);
      const uint32_t taddr = tmem_base + buf * B + (static_cast<uint32_t>(warp * 32) << 16);
      // Shift of the log-sum-exp.  Any value common to the block's tokens cancels; the Cauchy-Schwarz bounds
      // ||q||max ||c_b|| (base) and ||q||max (||c_b|| + r_b beta_b) (rescue) need no pass over the logits.  They are
      // used when small enough that no term can underflow (2^-126); otherwise the exact maxima are taken.
      float mb = qn_max * p.cnorm[crow0 + b] * p.scale_log2 * 1.0001f;
      float mr = fmaf(qn_max * gb, p.scale_log2 * 1.0001f, mb);
      const bool exact_shift = !__all_sync(0xffffffffu, mr <= 60.0f);
      if (exact_shift) {
      // pass 1: maxima of the raw logits x and of y = x + ||q|| r beta
      float mb0 = -INFINITY, mb1 = -INFINITY, mr0 = -INFINITY, mr1 = -INFINITY;
#pragma unroll 1
      for (int c0 = 0; c0 < B; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + c0, r);
        tmem_wait_ld();
        if (n_tok < B) {   // short last query block: tokens past the sequence end do not count
#pragma unroll
          for (int q = 0; q < 32; ++q)
            if (c0 + q >= n_tok) r[q] = 0xff800000u;   // -inf
        }
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float4 qn = *reinterpret_cast<const float4*>(sQn + c0 + j);
          float y0, y1, y2, y3;
          f2_unpack(f2_fma(f2_pack(qn.x, qn.y), gb2, f2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1]))), y0, y1);
          f2_unpack(f2_fma(f2_pack(qn.z, qn.w), gb2, f2_pack(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]))), y2, y3);
          mb0 = max3(mb0, __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
          mb1 = max3(mb1, __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
          mr0 = max3(mr0, y0, y1);
          mr1 = max3(mr1, y2, y3);
        }
      }
        mb = fmaxf(mb0, mb1) * p.scale_log2;   // log2 units
        mr = fmaxf(mr0, mr1) * p.scale_log2;
      }
      const uint64_t nmb2 = f2_pack(-mb, -mb), nmr2 = f2_pack(-mr, -mr);
      uint64_t sb2 = 0ull, sr2 = 0ull, sb2b = 0ull, sr2b = 0ull;
#pragma unroll 1
      for (int c0 = 0; c0 < B; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + c0, r);
        tmem_wait_ld();
        if (n_tok < B) {   // short last query block: tokens past the sequence end do not count
#pragma unroll
          for (int q = 0; q < 32; ++q)
            if (c0 + q >= n_tok) r[q] = 0xff800000u;   // -inf
        }
        if (c0 + 32 >= B) {   // accumulator fully read: hand the TMEM buffer back to the MMA warp
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bar_tempty[buf]));
        }
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float4 qn = *reinterpret_cast<const float4*>(sQn + c0 + j);
          const uint64_t x01 = f2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
          const uint64_t x23 = f2_pack(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
          float e0, e1, e2, e3, f0, f1, f2, f3;
          f2_unpack(f2_fma(x01, scale2, nmb2), e0, e1);
          f2_unpack(f2_fma(x23, scale2, nmb2), e2, e3);
          f2_unpack(f2_fma(f2_fma(f2_pack(qn.x, qn.y), gb2, x01), scale2, nmr2), f0, f1);
          f2_unpack(f2_fma(f2_fma(f2_pack(qn.z, qn.w), gb2, x23), scale2, nmr2), f2, f3);
          sb2 = f2_add(sb2, f2_pack(fast_exp2(e0), fast_exp2(e1)));
          sb2b = f2_add(sb2b, f2_pack(fast_exp2(e2), fast_exp2(e3)));
          sr2 = f2_add(sr2, f2_pack(fast_exp2(f0), fast_exp2(f1)));
          sr2b = f2_add(sr2b, f2_pack(fast_exp2(f2), fast_exp2(f3)));
        }
      }
      float a0, a1, a2, a3;
      f2_unpack(f2_add(sb2, sb2b), a0, a1);
      f2_unpack(f2_add(sr2, sr2b), a2, a3);
      const bool causal = b <= i;
      sLb[b] = causal ? mb + fast_log2(a0 + a1) : -INFINITY;
      sLr[b] = causal ? mr + fast_log2(a2 + a3) : -INFINITY;
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
    if (lane == 0) {
      const uint32_t word = wb | wr | wf;
      p.mask[mrow + w] = word;
      if (p.dbg_base) p.dbg_base[mrow + w] = wb;
      if (p.dbg_rescue) p.dbg_rescue[mrow + w] = wr;
      cnt += __popc(word);
    }
  }
  if (lane == 0 && cnt) atomicAdd(p.counts + l * p.Hq + h, cnt);
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

}  // namespace rbs

// q_start_block / n_q_tokens: the queries of this call are tokens [q_start_block * B, q_start_block * B + n_q_tokens)
// of the sequence; Q, mask and density cover only them (n_q_tokens < 0: the whole sequence).
static rbs_status select_impl(const rbs_shape* shape, int q_start_block, int n_q_tokens, rbs_tensor Q, rbs_stats stats, int beta_mode, float alpha_base,
                              float alpha_rescue, int n_sink, int n_local, int n_recent, uint32_t* mask,
                              float* density, uint32_t* dbg_base_mask, uint32_t* dbg_rescue_mask,
                              void* workspace, size_t workspace_bytes, void* stream) {
  using namespace rbs;
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
  float* g = reinterpret_cast<float*>(wsp + ws.off_g);
  float* cnorm = reinterpret_cast<float*>(wsp + ws.off_cn);
  unsigned int* counts = reinterpret_cast<unsigned int*>(wsp + ws.off_counts);
  const float scale_log2 = kLog2e / sqrtf(static_cast<float>(x.d));

  int P = 1;
  while (P < x.M) P <<= 1;
  if (P < 2) P = 2;
  const size_t coeff_smem = static_cast<size_t>(P) * sizeof(float);
  RBS_CUDA_OK(cudaMemsetAsync(counts, 0, static_cast<size_t>(x.L) * x.Hq * sizeof(unsigned int), s));
  rescue_coeff_kernel<<<x.L * x.Hkv, kCoeffThreads, coeff_smem, s>>>(stats.radius, x.M, P, scale_log2, stats.beta,
                                                                     stats.rq, g, ws.Mpad, beta_mode);
  RBS_CUDA_OK(cudaGetLastError());
  const int64_t rows = static_cast<int64_t>(x.L) * x.Hkv * ws.Mpad;
  const int64_t n_thr = rows * (kHeadDim / 4);
  split_centroid_kernel<<<static_cast<unsigned>((n_thr + 255) / 256), 256, 0, s>>>(stats.centroid, x.M, ws.Mpad, rows, chi, clo, cnorm);
  RBS_CUDA_OK(cudaGetLastError());

  SelectParams p;
  p.Q = static_cast<const __nv_bfloat16*>(Q.ptr); p.qsb = Q.stride_batch; p.qst = Q.stride_token; p.qsh = Q.stride_head;
  p.chi = chi; p.clo = clo; p.g = g; p.cnorm = cnorm;
  p.M = x.M; p.Mpad = ws.Mpad; p.W = x.W; p.L = x.L; p.Hq = x.Hq; p.G = x.G; p.N = x.N;
  p.q0 = q_start_block; p.Nq = n_q_tokens; p.Mq = (n_q_tokens + x.B - 1) / x.B;
  p.scale_log2 = scale_log2; p.t_base = log2f(alpha_base); p.t_rescue = log2f(alpha_rescue);
  p.n_sink = n_sink; p.n_local = n_local; p.n_recent = n_recent;
  p.mask = mask; p.dbg_base = dbg_base_mask; p.dbg_rescue = dbg_rescue_mask; p.counts = counts;
  if (x.B == 256) st = launch_select_tc<256>(p, Q, s);
  else st = (x.B == 128) ? launch_select_tc<128>(p, Q, s) : launch_select_tc<64>(p, Q, s);
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
