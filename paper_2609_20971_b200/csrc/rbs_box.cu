// rbs_select_box: the Quest-style comparison selector of the paper's ablation (Sec. 4.2; App. D.2, Eq. quest_box) in
// the same backend as rbs_select.  The block logit is the upper bound of the block's coordinate-wise box,
//     U_b(q) = sum_j max(q_j a_bj, q_j u_bj) = q . v_b + |q| . h_b,     v_b = (u_b + a_b) / 2,  h_b = (u_b - a_b) / 2,
// i.e. one dot product of length 2 d between [q, |q|] and [v_b, h_b]: four accumulating tensor-core products per tile
// (v and h each as bf16 hi + bf16 lo, like the centroids of rbs_select; |q| is exact in bf16).  The logits are
// aggregated over the query block's tokens by the shared per-block log-sum-exp (Eq. block_aggregation) and query block i
// keeps its ceil(density_param (i + 1)) best causal blocks, ties with the last kept score included, plus the forced ones.
#include "rbs_common.cuh"
#include "rbs_sm100.cuh"
#include "rbs_score.cuh"

namespace rbs {

// ---------------------------------------------------------------------------------------------
// fp32 box minima / maxima -> scaled centre and half-width, each as bf16 hi + bf16 lo, rows padded to Mpad with zeros.
// Output layout: [4][rows_padded][128] bf16 (v hi, v lo, h hi, h lo); bound[row] = sqrt(2) ||[v, h] scale||_2, so that
// ||q|| bound >= the scaled box logit of any query (Cauchy-Schwarz on the vector [q, |q|], whose norm is sqrt(2) ||q||).
// One warp per row, one thread per 4 columns.
// ---------------------------------------------------------------------------------------------
__global__ void box_split_kernel(const float* __restrict__ lo, const float* __restrict__ hi, int M, int Mpad,
                                 int64_t n_rows_padded, float scale_log2, __nv_bfloat16* __restrict__ out,
                                 float* __restrict__ bound) {
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t row = t / (kHeadDim / 4);
  const int c4 = static_cast<int>(t % (kHeadDim / 4));
  if (row >= n_rows_padded) return;
  const int64_t hd = row / Mpad;
  const int b = static_cast<int>(row % Mpad);
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f), u = a;
  if (b < M) {
    a = *reinterpret_cast<const float4*>(lo + (hd * M + b) * kHeadDim + c4 * 4);
    u = *reinterpret_cast<const float4*>(hi + (hd * M + b) * kHeadDim + c4 * 4);
  }
  const float hs = 0.5f * scale_log2;
  const float v[4] = {(u.x + a.x) * hs, (u.y + a.y) * hs, (u.z + a.z) * hs, (u.w + a.w) * hs};
  const float h[4] = {(u.x - a.x) * hs, (u.y - a.y) * hs, (u.z - a.z) * hs, (u.w - a.w) * hs};
  auto split = [&](const float (&x)[4], __nv_bfloat16* dst_hi, __nv_bfloat16* dst_lo) {
    uint32_t wh[2], wl[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const __nv_bfloat16 h0 = __float2bfloat16_rn(x[2 * k]), h1 = __float2bfloat16_rn(x[2 * k + 1]);
      wh[k] = static_cast<uint32_t>(__bfloat16_as_ushort(h0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h1)) << 16);
      wl[k] = pack_bf16(x[2 * k] - __bfloat162float(h0), x[2 * k + 1] - __bfloat162float(h1));
    }
    *reinterpret_cast<uint2*>(dst_hi) = make_uint2(wh[0], wh[1]);
    *reinterpret_cast<uint2*>(dst_lo) = make_uint2(wl[0], wl[1]);
  };
  const int64_t plane = n_rows_padded * kHeadDim, at = row * kHeadDim + c4 * 4;
  split(v, out + at, out + plane + at);
  split(h, out + 2 * plane + at, out + 3 * plane + at);
  float n2 = 0.f;
#pragma unroll
  for (int k = 0; k < 4; ++k) n2 += v[k] * v[k] + h[k] * h[k];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
  if (c4 == 0) bound[row] = sqrtf(2.0f * n2);
}

struct BoxParams {
  const float* bound;
  int M, Mpad, W, L, Hq, G, N, rows_padded;
  double delta;
  int n_sink, n_local, n_recent;
  uint32_t* mask; uint32_t* dbg_chosen;
  unsigned int* counts;
};

// order-preserving map of a float onto an unsigned integer
__device__ __forceinline__ uint32_t float_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ---------------------------------------------------------------------------------------------
// One CTA per (batch, query head, query block), one CTA per SM (the four operand slots of a tile take 128 KB).
// Warps 0-3: epilogue (TMEM lane = block row), warp 4: TMA producer, warp 5: MMA issuer and TMEM owner.
// ---------------------------------------------------------------------------------------------
constexpr int kBoxThreads = 192;

template <int B>
__global__ void __launch_bounds__(kBoxThreads, 1)
select_box_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmBox, const BoxParams p,
                  unsigned int* status) {
  constexpr uint32_t kPanelC = 128 * 128;          // one 64-column panel of a 128-row operand tile
  constexpr uint32_t kSlot = 2 * kPanelC;          // one of the four operands of a tile: v hi, v lo, h hi, h lo
  constexpr uint32_t kPanelQ = B * 128;
  constexpr uint32_t kIdesc = idesc_bf16_f32(128, B, false);
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sC = smem;                                        // 4 slots: 128 KB
  unsigned char* sQ = sC + 4 * kSlot;                              // Q, 2 panels
  unsigned char* sQa = sQ + 2 * kPanelQ;                           // |Q|, 2 panels
  float* sD = reinterpret_cast<float*>(sQa + 2 * kPanelQ);         // B: ||q_t|| - max
  float* sL = sD + B;                                              // one score per candidate block
  __shared__ __align__(8) uint64_t bar_q, bar_qa, bar_cfull[4], bar_cempty[4], bar_tfull[2], bar_tempty[2];
  __shared__ float sRed[32];
  __shared__ int sCount[kBoxThreads / 32];
  __shared__ uint32_t s_tmem;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per_i = p.L * p.Hq;
  const int i = p.M - 1 - static_cast<int>(blockIdx.x / per_i);       // query block, longest rows first
  const int rem = static_cast<int>(blockIdx.x % per_i);
  const int l = rem / p.Hq, h = rem % p.Hq, hk = h / p.G;
  const int Hkv = p.Hq / p.G;
  const int n_tiles = i / 128 + 1;
  const int crow0 = static_cast<int>((static_cast<int64_t>(l) * Hkv + hk) * p.Mpad);

  if (tid == 0) {
    mbar_init(smem_u32(&bar_q), 1);
    mbar_init(smem_u32(&bar_qa), 128);
    for (int s = 0; s < 4; ++s) { mbar_init(smem_u32(&bar_cfull[s]), 1); mbar_init(smem_u32(&bar_cempty[s]), 1); }
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
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmBox);
      mbar_arrive_expect_tx(smem_u32(&bar_q), 2 * kPanelQ);
      tma_load_4d(smem_u32(sQ), &tmQ, smem_u32(&bar_q), 0, h, i * B, l);
      tma_load_4d(smem_u32(sQ + kPanelQ), &tmQ, smem_u32(&bar_q), 64, h, i * B, l);
      bool ok = true;
      for (int bt = 0; ok && bt < n_tiles; ++bt) {
        for (int s = 0; s < 4; ++s) {
          if (bt > 0 && !mbar_wait(smem_u32(&bar_cempty[s]), (bt - 1) & 1, status, kWaitStageFree)) { ok = false; break; }
          const uint32_t dst = smem_u32(sC) + s * kSlot, bar = smem_u32(&bar_cfull[s]);
          mbar_arrive_expect_tx(bar, kSlot);
          tma_load_2d(dst, &tmBox, bar, 0, s * p.rows_padded + crow0 + bt * 128);
          tma_load_2d(dst + kPanelC, &tmBox, bar, 64, s * p.rows_padded + crow0 + bt * 128);
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------- MMA issuer -------------------------------
    bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull));
    const uint64_t dq = smem_desc_sw128(smem_u32(sQ), 16, 1024);
    const uint64_t dqa = smem_desc_sw128(smem_u32(sQa), 16, 1024);
    for (int bt = 0; ok && bt < n_tiles; ++bt) {
      const int buf = bt & 1;
      if (bt >= 2) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_tempty[buf]), ((bt >> 1) - 1) & 1, status, kWaitTmemFree));
      const uint32_t d_tmem = tmem_base + buf * B;
      for (int s = 0; ok && s < 4; ++s) {
        ok = mbar_wait(smem_u32(&bar_cfull[s]), bt & 1, status, kWaitTmaFull);
        if (ok && s == 2 && bt == 0) ok = mbar_wait(smem_u32(&bar_qa), 0, status, kWaitPReady);   // |Q| written
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t da = smem_desc_sw128(smem_u32(sC) + s * kSlot, 16, 1024);
        mma_ss_k128_commit_elect(d_tmem, da, s < 2 ? dq : dqa, kIdesc, kPanelC, kPanelQ, smem_u32(&bar_cempty[s]), s > 0);
      }
      if (ok) mma_commit_elect(smem_u32(&bar_tfull[buf]));
    }
    __syncwarp();
  } else {
    // ------------------------------- epilogue: one block row per thread -------------------------------
    const int row = warp * 32 + lane;
    bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull));
    // |Q|: the same tile with the sign bits cleared, in the same swizzled layout (an element-wise copy)
    for (int c = tid; ok && c < B * 16; c += 128) {
      const int tok = c >> 4, piece = c & 15;
      const uint32_t at = (piece >> 3) * kPanelQ + tok * 128 + ((piece & 7) << 4);
      uint4 v = *reinterpret_cast<const uint4*>(sQ + at);
      v.x &= 0x7fff7fffu; v.y &= 0x7fff7fffu; v.z &= 0x7fff7fffu; v.w &= 0x7fff7fffu;
      *reinterpret_cast<uint4*>(sQa + at) = v;
    }
    fence_proxy_async_smem();                      // these writes are read by the tensor core (async proxy)
    mbar_arrive(smem_u32(&bar_qa));
    const int n_tok = min(B, p.N - i * B);
    float qn_max, qn_spread;
    ok = query_norm_shifts<B, 128>(sQ, tid, n_tok, sD, sRed, 1, ok, qn_max, qn_spread);
    for (int bt = 0; ok && bt < n_tiles; ++bt) {
      const int buf = bt & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_tfull[buf]), (bt >> 1) & 1, status, kWaitMmaDone));
      if (!ok) break;
      tc_fence_after_sync();
      const int b = bt * 128 + row;
      const uint32_t taddr = tmem_base + buf * B + (static_cast<uint32_t>(warp * 32) << 16);
      float Lb, Lr;
      score_tile<B, true>(taddr, sD, 0.f, p.bound[crow0 + b], qn_max, qn_spread, n_tok, [&]() {
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bar_tempty[buf]));
      }, Lb, Lr);
      sL[b] = b <= i ? Lb : -INFINITY;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == 5) tmem_dealloc(tmem_base, 2 * B);

  // The k-th largest score of the row, k = ceil(delta (i + 1)), by bisection on the order-preserving integer image of
  // the scores: the largest t with #{b <= i : key_b >= t} >= k.  All six warps count.
  const int nb = i + 1;
  int k = static_cast<int>(ceil(p.delta * static_cast<double>(nb)));
  k = min(nb, max(1, k));
  uint32_t t_lo = 0u;                              // invariant: count(key >= t_lo) >= k
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t t_try = t_lo | (1u << bit);
    int c = 0;
    for (int b = tid; b < nb; b += kBoxThreads) c += float_key(sL[b]) >= t_try;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if (lane == 0) sCount[warp] = c;
    __syncthreads();
    int total = 0;
#pragma unroll
    for (int w = 0; w < kBoxThreads / 32; ++w) total += sCount[w];
    if (total >= k) t_lo = t_try;
    __syncthreads();
  }
  const int64_t mrow = ((static_cast<int64_t>(l) * p.Hq + h) * p.M + i) * p.W;
  const bool all_forced = i >= p.M - p.n_recent;
  unsigned int cnt = 0;
  for (int w = warp; w < p.W; w += kBoxThreads / 32) {
    const int b = w * 32 + lane;
    const bool valid = b <= i;
    bool kc = false, kf = false;
    if (valid) {
      kc = float_key(sL[b]) >= t_lo;
      kf = all_forced || b < p.n_sink || b > i - p.n_local;
    }
    const uint32_t wc = __ballot_sync(0xffffffffu, kc), wf = __ballot_sync(0xffffffffu, kf);
    if (lane == 0) {
      p.mask[mrow + w] = wc | wf;
      if (p.dbg_chosen) p.dbg_chosen[mrow + w] = wc;
      cnt += __popc(wc | wf);
    }
  }
  if (lane == 0 && cnt) atomicAdd(p.counts + l * p.Hq + h, cnt);
}

__global__ void box_density_kernel(const unsigned int* __restrict__ counts, int n, int M, float* __restrict__ density) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n) density[t] = static_cast<float>(static_cast<double>(counts[t]) / (0.5 * static_cast<double>(M) * static_cast<double>(M + 1)));
}

struct BoxWorkspace {
  size_t off_ops, off_bound, off_counts, bytes;
  int Mpad;
};

static BoxWorkspace box_workspace(const Dims& x) {
  BoxWorkspace w;
  w.Mpad = (x.M + 127) / 128 * 128;
  const size_t rows = static_cast<size_t>(x.L) * x.Hkv * w.Mpad;
  size_t off = 0;
  w.off_ops = off; off = align_up(off + 4 * rows * x.d * sizeof(__nv_bfloat16), 256);
  w.off_bound = off; off = align_up(off + rows * sizeof(float), 256);
  w.off_counts = off; off = align_up(off + static_cast<size_t>(x.L) * x.Hq * sizeof(unsigned int), 256);
  w.bytes = off;
  return w;
}

size_t select_box_workspace_bytes(const Dims& x) { return x.B <= 128 ? box_workspace(x).bytes : 0; }

template <int B>
static rbs_status launch_select_box(const BoxParams& p, const rbs_tensor& Q, const __nv_bfloat16* ops, cudaStream_t s) {
  CUtensorMap tmQ, tmBox;
  rbs_status st = make_tmap_lthd(&tmQ, Q.ptr, p.L, p.N, p.Hq, kHeadDim, Q.stride_batch, Q.stride_token, Q.stride_head, 64, B, true);
  if (st != RBS_OK) return st;
  if ((st = make_tmap_2d(&tmBox, ops, static_cast<int64_t>(4) * p.rows_padded, kHeadDim, 64, 128)) != RBS_OK) return st;
  unsigned int* status = device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  const size_t smem = static_cast<size_t>(8) * 128 * 128 + 4 * static_cast<size_t>(B) * 128 + B * sizeof(float) +
                      static_cast<size_t>(p.Mpad) * sizeof(float);
  if (smem > 227 * 1024 - 2048) return RBS_ERR_UNSUPPORTED;
  auto kern = select_box_kernel<B>;
  if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem)) != RBS_OK) return st;
  const long long n_cta = static_cast<long long>(p.L) * p.Hq * p.M;
  if (n_cta > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  kern<<<static_cast<unsigned>(n_cta), kBoxThreads, smem, s>>>(tmQ, tmBox, p, status);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

}  // namespace rbs

extern "C" rbs_status rbs_select_box(const rbs_shape* shape, rbs_tensor Q, rbs_box box, double density_param, int n_sink,
                                     int n_local, int n_recent, uint32_t* mask, float* density, uint32_t* dbg_chosen_mask,
                                     void* workspace, size_t workspace_bytes, void* stream) {
  using namespace rbs;
  rbs::NvtxRange nvtx_range("rbs_select_box");
  rbs_status st = check_shape(shape);
  if (st != RBS_OK) return st;
  if ((st = check_tensor(Q)) != RBS_OK) return st;
  if (box.lo == nullptr || box.hi == nullptr || mask == nullptr || density == nullptr) return RBS_ERR_INVALID_ARG;
  if (!(density_param > 0.0) || density_param > 1.0) return RBS_ERR_INVALID_ARG;
  if (n_sink < 0 || n_local < 0 || n_recent < 0) return RBS_ERR_INVALID_ARG;
  Dims x = make_dims(*shape);
  if (x.B > 128) return RBS_ERR_UNSUPPORTED;
  const BoxWorkspace ws = box_workspace(x);
  if (workspace == nullptr || workspace_bytes < ws.bytes || reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return RBS_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned char* wsp = static_cast<unsigned char*>(workspace);
  __nv_bfloat16* ops = reinterpret_cast<__nv_bfloat16*>(wsp + ws.off_ops);
  float* bound = reinterpret_cast<float*>(wsp + ws.off_bound);
  unsigned int* counts = reinterpret_cast<unsigned int*>(wsp + ws.off_counts);
  const float scale_log2 = kLog2e / sqrtf(static_cast<float>(x.d));
  RBS_CUDA_OK(cudaMemsetAsync(counts, 0, static_cast<size_t>(x.L) * x.Hq * sizeof(unsigned int), s));
  const int64_t rows = static_cast<int64_t>(x.L) * x.Hkv * ws.Mpad;
  const int64_t n_thr = rows * (kHeadDim / 4);
  box_split_kernel<<<static_cast<unsigned>((n_thr + 255) / 256), 256, 0, s>>>(box.lo, box.hi, x.M, ws.Mpad, rows, scale_log2, ops, bound);
  RBS_CUDA_OK(cudaGetLastError());
  BoxParams p;
  p.bound = bound;
  p.M = x.M; p.Mpad = ws.Mpad; p.W = x.W; p.L = x.L; p.Hq = x.Hq; p.G = x.G; p.N = x.N;
  p.rows_padded = static_cast<int>(rows);
  p.delta = density_param;
  p.n_sink = n_sink; p.n_local = n_local; p.n_recent = n_recent;
  p.mask = mask; p.dbg_chosen = dbg_chosen_mask; p.counts = counts;
  st = x.B == 128 ? launch_select_box<128>(p, Q, ops, s) : launch_select_box<64>(p, Q, ops, s);
  if (st != RBS_OK) return st;
  const int nh = x.L * x.Hq;
  box_density_kernel<<<(nh + 127) / 128, 128, 0, s>>>(counts, nh, x.M, density);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}
