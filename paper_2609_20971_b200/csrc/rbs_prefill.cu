// rbs_sparse_prefill: causal block-sparse attention over a bit-packed block mask (Sec. 3.3), dense when
// the mask is NULL (Eq. 1).  One CTA per (batch, query head, query block); it walks the set bits of its
// mask row, streams those K/V blocks through shared memory and keeps an online softmax in registers.
#include "rbs_common.cuh"

namespace rbs {

struct PrefillParams {
  const __nv_bfloat16* Q; int64_t qsb, qst, qsh;
  const __nv_bfloat16* K; int64_t ksb, kst, ksh;
  const __nv_bfloat16* V; int64_t vsb, vst, vsh;
  __nv_bfloat16* O; int64_t osb, ost, osh;
  const uint32_t* mask;  // nullptr: dense
  float* lse;            // nullable
  int M, W, L, Hq, G, N;
  float scale_log2;
};

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

template <int B>
__global__ void __launch_bounds__(B * 2, 1)
prefill_mma_kernel(const PrefillParams p) {
  constexpr int NT = B / 8;       // key n-tiles per block
  constexpr int NTHREADS = B * 2;  // one warp per 16 query rows
  constexpr int TILE = B * 256;    // bytes of a [B][128] bf16 tile
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sQ = smem;
  unsigned char* sK = sQ + TILE;       // 2 stages
  unsigned char* sV = sK + 2 * TILE;   // 2 stages
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gq = lane >> 2, tq = lane & 3;

  const int per_i = p.L * p.Hq;
  const int i = p.M - 1 - static_cast<int>(blockIdx.x / per_i);
  const int rem = static_cast<int>(blockIdx.x % per_i);
  const int l = rem / p.Hq, h = rem % p.Hq, hk = h / p.G;
  const uint32_t* mrow = p.mask ? p.mask + ((static_cast<int64_t>(l) * p.Hq + h) * p.M + i) * p.W : nullptr;

  const __nv_bfloat16* qbase = p.Q + l * p.qsb + static_cast<int64_t>(i) * B * p.qst + h * p.qsh;
  const __nv_bfloat16* kbase = p.K + l * p.ksb + hk * p.ksh;
  const __nv_bfloat16* vbase = p.V + l * p.vsb + hk * p.vsh;
  __nv_bfloat16* obase = p.O + l * p.osb + static_cast<int64_t>(i) * B * p.ost + h * p.osh;

  auto load_kv = [&](int b, int stage) {
    const __nv_bfloat16* ks = kbase + static_cast<int64_t>(b) * B * p.kst;
    const __nv_bfloat16* vs = vbase + static_cast<int64_t>(b) * B * p.vst;
    for (int c = tid; c < B * 16; c += NTHREADS) {
      const int row = c >> 4, chunk = c & 15;
      cp_async16(smem_u32(sK + stage * TILE + tile_off(row, chunk)), ks + static_cast<int64_t>(row) * p.kst + chunk * 8);
      cp_async16(smem_u32(sV + stage * TILE + tile_off(row, chunk)), vs + static_cast<int64_t>(row) * p.vst + chunk * 8);
    }
  };

  int b_cur = next_block(mrow, -1, i);
  const int row0 = warp * 16 + gq;  // this thread's first query row inside the block (second: +8)
  if (b_cur < 0) {                  // nothing retained: zero rows, lse = -inf
    for (int c = tid; c < B * 16; c += NTHREADS) {
      const int row = c >> 4, chunk = c & 15;
      *reinterpret_cast<uint4*>(obase + static_cast<int64_t>(row) * p.ost + chunk * 8) = make_uint4(0, 0, 0, 0);
    }
    if (p.lse && tid < B) p.lse[(static_cast<int64_t>(l) * p.Hq + h) * p.N + i * B + tid] = -INFINITY;
    return;
  }

  for (int c = tid; c < B * 16; c += NTHREADS) {
    const int row = c >> 4, chunk = c & 15;
    cp_async16(smem_u32(sQ + tile_off(row, chunk)), qbase + static_cast<int64_t>(row) * p.qst + chunk * 8);
  }
  load_kv(b_cur, 0);
  cp_async_commit();

  float acc_o[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n) { acc_o[n][0] = acc_o[n][1] = acc_o[n][2] = acc_o[n][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  uint32_t qf[8][4];
  bool q_loaded = false;
  int stage = 0;

  while (b_cur >= 0) {
    const int b_next = next_block(mrow, b_cur, i);
    if (b_next >= 0) {
      load_kv(b_next, stage ^ 1);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (!q_loaded) {
#pragma unroll
      for (int k16 = 0; k16 < 8; ++k16)
        ldmatrix_x4(qf[k16][0], qf[k16][1], qf[k16][2], qf[k16][3],
                    smem_u32(sQ + tile_off(warp * 16 + (lane & 15), 2 * k16 + (lane >> 4))));
      q_loaded = true;
    }
    const unsigned char* cK = sK + stage * TILE;
    const unsigned char* cV = sV + stage * TILE;

    float acc_s[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { acc_s[nt][0] = acc_s[nt][1] = acc_s[nt][2] = acc_s[nt][3] = 0.f; }
#pragma unroll
    for (int k16 = 0; k16 < 8; ++k16) {
#pragma unroll
      for (int ntp = 0; ntp < NT / 2; ++ntp) {
        uint32_t b0, b1, b2, b3;
        const int row = 16 * ntp + (lane & 7) + ((lane >> 4) << 3);
        ldmatrix_x4(b0, b1, b2, b3, smem_u32(cK + tile_off(row, 2 * k16 + ((lane >> 3) & 1))));
        mma_bf16_16816(acc_s[2 * ntp], qf[k16], b0, b1);
        mma_bf16_16816(acc_s[2 * ntp + 1], qf[k16], b2, b3);
      }
    }
    // scale into log2 units, causal mask on the diagonal block, online softmax
    const bool diag = b_cur == i;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float s = acc_s[nt][e] * p.scale_log2;
        if (diag) {
          const int key = nt * 8 + tq * 2 + (e & 1);
          const int qr = row0 + (e >> 1) * 8;
          if (key > qr) s = -INFINITY;
        }
        acc_s[nt][e] = s;
        mx[e >> 1] = fmaxf(mx[e >> 1], s);
      }
    }
    float corr[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float m_new = fmaxf(m_run[r], mx[r]);
      corr[r] = fast_exp2(m_run[r] - m_new);
      m_run[r] = m_new;
      l_run[r] *= corr[r];
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float pe = fast_exp2(acc_s[nt][e] - m_run[e >> 1]);
        acc_s[nt][e] = pe;
        l_run[e >> 1] += pe;
      }
    }
#pragma unroll
    for (int n = 0; n < 16; ++n) {
      acc_o[n][0] *= corr[0]; acc_o[n][1] *= corr[0];
      acc_o[n][2] *= corr[1]; acc_o[n][3] *= corr[1];
    }
    // O += P V
#pragma unroll
    for (int j = 0; j < B / 16; ++j) {
      uint32_t pa[4];
      pa[0] = pack_bf16(acc_s[2 * j][0], acc_s[2 * j][1]);
      pa[1] = pack_bf16(acc_s[2 * j][2], acc_s[2 * j][3]);
      pa[2] = pack_bf16(acc_s[2 * j + 1][0], acc_s[2 * j + 1][1]);
      pa[3] = pack_bf16(acc_s[2 * j + 1][2], acc_s[2 * j + 1][3]);
#pragma unroll
      for (int ndp = 0; ndp < 8; ++ndp) {
        uint32_t b0, b1, b2, b3;
        const int row = 16 * j + (lane & 7) + (((lane >> 3) & 1) << 3);
        ldmatrix_x4_trans(b0, b1, b2, b3, smem_u32(cV + tile_off(row, 2 * ndp + (lane >> 4))));
        mma_bf16_16816(acc_o[2 * ndp], pa, b0, b1);
        mma_bf16_16816(acc_o[2 * ndp + 1], pa, b2, b3);
      }
    }
    __syncthreads();  // stage may be overwritten by the next iteration's prefetch
    b_cur = b_next;
    stage ^= 1;
  }

  // finalize
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  const float inv0 = 1.0f / l_run[0], inv1 = 1.0f / l_run[1];
  __nv_bfloat16* o0 = obase + static_cast<int64_t>(row0) * p.ost;
  __nv_bfloat16* o1 = obase + static_cast<int64_t>(row0 + 8) * p.ost;
#pragma unroll
  for (int n = 0; n < 16; ++n) {
    *reinterpret_cast<uint32_t*>(o0 + n * 8 + tq * 2) = pack_bf16(acc_o[n][0] * inv0, acc_o[n][1] * inv0);
    *reinterpret_cast<uint32_t*>(o1 + n * 8 + tq * 2) = pack_bf16(acc_o[n][2] * inv1, acc_o[n][3] * inv1);
  }
  if (p.lse && tq == 0) {
    float* dst = p.lse + (static_cast<int64_t>(l) * p.Hq + h) * p.N + i * B;
    dst[row0] = (m_run[0] + fast_log2(l_run[0])) * 0.6931471805599453f;
    dst[row0 + 8] = (m_run[1] + fast_log2(l_run[1])) * 0.6931471805599453f;
  }
}

template <int B>
static rbs_status launch_prefill(const PrefillParams& p, cudaStream_t s) {
  const size_t smem = static_cast<size_t>(5) * B * 256;
  RBS_CUDA_OK(cudaFuncSetAttribute(prefill_mma_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  const long long n_cta = static_cast<long long>(p.L) * p.Hq * p.M;
  if (n_cta > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  prefill_mma_kernel<B><<<static_cast<unsigned>(n_cta), B * 2, smem, s>>>(p);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

}  // namespace rbs

extern "C" rbs_status rbs_sparse_prefill(const rbs_shape* shape, rbs_tensor Q, rbs_tensor K, rbs_tensor V,
                                         const uint32_t* mask, rbs_tensor O, float* lse, float softmax_scale,
                                         void* workspace, size_t workspace_bytes, void* stream) {
  using namespace rbs;
  (void)workspace; (void)workspace_bytes;
  rbs_status st = check_shape(shape);
  if (st != RBS_OK) return st;
  if ((st = check_tensor(Q)) != RBS_OK || (st = check_tensor(K)) != RBS_OK || (st = check_tensor(V)) != RBS_OK ||
      (st = check_tensor(O)) != RBS_OK)
    return st;
  if (softmax_scale < 0.f) return RBS_ERR_INVALID_ARG;
  Dims x = make_dims(*shape);
  PrefillParams p;
  p.Q = static_cast<const __nv_bfloat16*>(Q.ptr); p.qsb = Q.stride_batch; p.qst = Q.stride_token; p.qsh = Q.stride_head;
  p.K = static_cast<const __nv_bfloat16*>(K.ptr); p.ksb = K.stride_batch; p.kst = K.stride_token; p.ksh = K.stride_head;
  p.V = static_cast<const __nv_bfloat16*>(V.ptr); p.vsb = V.stride_batch; p.vst = V.stride_token; p.vsh = V.stride_head;
  p.O = static_cast<__nv_bfloat16*>(O.ptr); p.osb = O.stride_batch; p.ost = O.stride_token; p.osh = O.stride_head;
  p.mask = mask; p.lse = lse;
  p.M = x.M; p.W = x.W; p.L = x.L; p.Hq = x.Hq; p.G = x.G; p.N = x.N;
  const float scale = softmax_scale == 0.f ? 1.0f / sqrtf(static_cast<float>(x.d)) : softmax_scale;
  p.scale_log2 = scale * kLog2e;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return (x.B == 128) ? launch_prefill<128>(p, s) : launch_prefill<64>(p, s);
}
