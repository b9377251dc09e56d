// rbs_block_stats: one HBM stream over K.  Each warp owns one (batch, KV head, key block) tile of
// B rows x 128 bf16 at a time, brought into shared memory by TMA, and produces the centroid and the
// radius from that single read of K.
#include "rbs_common.cuh"
#include "rbs_sm100.cuh"

namespace rbs {

// ---------------------------------------------------------------------------------------------
// Every warp owns NS shared-memory slots used in turn, fetches its own tiles with TMA
// (two 128-byte-swizzled panels of 64 columns) and reduces them alone, so warps never wait for one
// another; with NS = 2 the next tile is already on its way while the current one is reduced.  Pass 1: lanes own 4 columns and walk the rows (column sums, no cross-lane traffic).
// Pass 2: lanes own rows and walk the columns (row distances, no cross-lane traffic); the swizzle
// keeps both access patterns free of bank conflicts.
// ---------------------------------------------------------------------------------------------
// With WPB = 2 (blocks of 256) two neighbouring warps share a block, 128 rows each: they exchange their column
// sums and their row maxima through shared memory (two bounded mbarrier rendezvous per block), so a block of 256
// streams like two blocks of 128 instead of needing a 64 KB slot per warp.
// BOX: the same read of K also gives the per-coordinate minima and maxima of each block (the statistics of the
// Quest-style comparison selector, App. D.2), written to box_lo / box_hi.
template <int B, int NW, int NS, int WPB, bool BOX>
__global__ void __launch_bounds__(NW * 32, 1)
block_stats_warp_kernel(const __grid_constant__ CUtensorMap tmK, int n_tiles, int M, int Hkv, int N,
                        float* __restrict__ centroid, float* __restrict__ radius, float* __restrict__ box_lo,
                        float* __restrict__ box_hi, unsigned int* status) {
  constexpr int RW = B / WPB;                 // rows of a block held by one warp
  constexpr uint32_t kPanel = RW * 128;      // bytes of one 64-column panel
  constexpr uint32_t kSlot = 2 * kPanel;
  constexpr int RJ = RW / 32;                 // rows per lane in pass 2
  constexpr int NG = NW / WPB;                // blocks in flight per CTA
  static_assert(NW % WPB == 0 && (WPB == 1 || WPB == 2), "warps per block");
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ __align__(8) uint64_t full_bar[NW * NS];
  // half of the warp's centroid (64 columns) at a time, re-read by every lane in pass 2; the whole of it would not
  // fit beside the tile slots
  __shared__ __align__(16) float s_cen[NW][kHeadDim / 2];
  __shared__ __align__(16) float s_sum[WPB == 2 ? NW : 1][kHeadDim];   // a warp's column sums, for its partner
  __shared__ float s_max[WPB == 2 ? NW : 1];
  __shared__ __align__(16) float s_lo[BOX && WPB == 2 ? NW : 1][kHeadDim], s_hi[BOX && WPB == 2 ? NW : 1][kHeadDim];
  __shared__ __align__(8) uint64_t pair_bar[NG];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t bar0 = smem_u32(&full_bar[warp * NS]);
  const uint32_t slot0 = smem_u32(smem) + warp * NS * kSlot;
  const int group = warp / WPB, part = warp % WPB;
  if (lane == 0) {
    for (int k = 0; k < NS; ++k) mbar_init(bar0 + 8 * k, 1);
    if (WPB == 2 && part == 0) mbar_init(smem_u32(&pair_bar[group]), 64);
    mbar_fence_init();
  }
  if (WPB == 2) __syncthreads(); else __syncwarp();

  const int stride = gridDim.x * NG;
  int t = group * gridDim.x + blockIdx.x;
  // K is read exactly once by this pass: its lines are marked evict-first in L2 so that they do not push out what the
  // following kernels re-read (29.5 against 30.9 us per 128 MiB layer)
  const uint64_t pol = make_policy_evict_first();
  auto issue = [&](int tile, int buf) {
    const uint32_t bar = bar0 + 8 * buf, slot = slot0 + buf * kSlot;
    int idx = tile;
    const int hk = idx % Hkv; idx /= Hkv;
    const int b = idx % M;
    const int l = idx / M;
    mbar_arrive_expect_tx(bar, kSlot);
    tma_load_4d_hint(slot, &tmK, bar, 0, hk, b * B + part * RW, l, pol);
    tma_load_4d_hint(slot + kPanel, &tmK, bar, 64, hk, b * B + part * RW, l, pol);
  };
  if (lane == 0) {
    for (int k = 0; k < NS; ++k)
      if (t + k * stride < n_tiles) issue(t + k * stride, k);
  }

  // pass-1 addressing: lane owns 8 bytes (4 columns): 16-byte chunk c16 = lane / 2, half = lane % 2
  const int c16 = lane >> 1, cp = c16 & 7;
  for (int it = 0; t < n_tiles; t += stride, ++it) {
    const int buf = it % NS;
    const uint32_t phase = (it / NS) & 1;
    const uint32_t slot = slot0 + buf * kSlot;
    const uint32_t p1_base = slot + (c16 >> 3) * kPanel + (lane & 1) * 8;
    if (!mbar_wait(bar0 + 8 * buf, phase, status, kWaitTmaFull)) break;
    int idx = t;
    const int hk = idx % Hkv; idx /= Hkv;
    const int b = idx % M;
    const int l = idx / M;
    // a short last block: TMA filled the rows past the sequence end with zeros; divide by its own size |K_b|
    const int rows_block = min(B, N - b * B);
    const int rows_valid = max(0, min(RW, rows_block - part * RW));   // of this warp's rows
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    float lo0 = INFINITY, lo1 = INFINITY, lo2 = INFINITY, lo3 = INFINITY;
    float hi0 = -INFINITY, hi1 = -INFINITY, hi2 = -INFINITY, hi3 = -INFINITY;
#pragma unroll 4
    for (int r8 = 0; r8 < RW; r8 += 8) {
#pragma unroll
      for (int rr = 0; rr < 8; ++rr) {
        uint32_t lo, hi;
        asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(lo), "=r"(hi)
                     : "r"(p1_base + (r8 + rr) * 128 + ((cp ^ rr) << 4)));
        a0 += bf16lo(lo); a1 += bf16hi(lo); a2 += bf16lo(hi); a3 += bf16hi(hi);
        if (BOX && r8 + rr < rows_valid) {   // the zero rows past the sequence end are not keys
          lo0 = fminf(lo0, bf16lo(lo)); lo1 = fminf(lo1, bf16hi(lo)); lo2 = fminf(lo2, bf16lo(hi)); lo3 = fminf(lo3, bf16hi(hi));
          hi0 = fmaxf(hi0, bf16lo(lo)); hi1 = fmaxf(hi1, bf16hi(lo)); hi2 = fmaxf(hi2, bf16lo(hi)); hi3 = fmaxf(hi3, bf16hi(hi));
        }
      }
    }
    const float inv_rows = 1.0f / static_cast<float>(rows_block);
    bool pair_ok = true;
    if (WPB == 2) {   // add the partner's column sums (rows past the sequence end arrived as zeros)
      reinterpret_cast<float4*>(s_sum[warp])[lane] = make_float4(a0, a1, a2, a3);
      if (BOX) {
        reinterpret_cast<float4*>(s_lo[warp])[lane] = make_float4(lo0, lo1, lo2, lo3);
        reinterpret_cast<float4*>(s_hi[warp])[lane] = make_float4(hi0, hi1, hi2, hi3);
      }
      mbar_arrive(smem_u32(&pair_bar[group]));
      pair_ok = mbar_wait(smem_u32(&pair_bar[group]), 0, status, kWaitStageFree);
      const float4 o = reinterpret_cast<const float4*>(s_sum[warp ^ 1])[lane];
      a0 += o.x; a1 += o.y; a2 += o.z; a3 += o.w;
      if (BOX) {
        const float4 ol = reinterpret_cast<const float4*>(s_lo[warp ^ 1])[lane], oh = reinterpret_cast<const float4*>(s_hi[warp ^ 1])[lane];
        lo0 = fminf(lo0, ol.x); lo1 = fminf(lo1, ol.y); lo2 = fminf(lo2, ol.z); lo3 = fminf(lo3, ol.w);
        hi0 = fmaxf(hi0, oh.x); hi1 = fmaxf(hi1, oh.y); hi2 = fmaxf(hi2, oh.z); hi3 = fmaxf(hi3, oh.w);
      }
    }
    const float4 cen = make_float4(a0 * inv_rows, a1 * inv_rows, a2 * inv_rows, a3 * inv_rows);
    const int64_t blk = (static_cast<int64_t>(l) * Hkv + hk) * M + b;
    const bool row_ok = RBS_DBG_OK(blk < n_tiles && b * B < N, status, kDbgStatsRow);
    if (part == 0 && row_ok) reinterpret_cast<float4*>(centroid + blk * kHeadDim)[lane] = cen;
    if (BOX && part == 0 && row_ok) {
      reinterpret_cast<float4*>(box_lo + blk * kHeadDim)[lane] = make_float4(lo0, lo1, lo2, lo3);
      reinterpret_cast<float4*>(box_hi + blk * kHeadDim)[lane] = make_float4(hi0, hi1, hi2, hi3);
    }

    float q[RJ];
#pragma unroll
    for (int j = 0; j < RJ; ++j) q[j] = 0.f;
    const uint32_t row_base = slot + lane * 128;
    const int sw = lane & 7;
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      if ((c & 7) == 0) {   // columns 64 (c / 8) .. +63 of the centroid live in lanes 16 (c / 8) .. +15
        __syncwarp();
        if ((lane >> 4) == (c >> 3)) reinterpret_cast<float4*>(s_cen[warp])[lane & 15] = cen;
        __syncwarp();
      }
      // centroid columns 8c..8c+7: two broadcast reads (all lanes, same address)
      const float4 ca = reinterpret_cast<const float4*>(s_cen[warp])[2 * (c & 7)];
      const float4 cb = reinterpret_cast<const float4*>(s_cen[warp])[2 * (c & 7) + 1];
      const uint32_t col = (c >> 3) * kPanel + (((c & 7) ^ sw) << 4);
#pragma unroll
      for (int j = 0; j < RJ; ++j) {
        uint32_t x0, x1, x2, x3;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3)
                     : "r"(row_base + j * 32 * 128 + col));
        float d;
        d = bf16lo(x0) - ca.x; q[j] = fmaf(d, d, q[j]);
        d = bf16hi(x0) - ca.y; q[j] = fmaf(d, d, q[j]);
        d = bf16lo(x1) - ca.z; q[j] = fmaf(d, d, q[j]);
        d = bf16hi(x1) - ca.w; q[j] = fmaf(d, d, q[j]);
        d = bf16lo(x2) - cb.x; q[j] = fmaf(d, d, q[j]);
        d = bf16hi(x2) - cb.y; q[j] = fmaf(d, d, q[j]);
        d = bf16lo(x3) - cb.z; q[j] = fmaf(d, d, q[j]);
        d = bf16hi(x3) - cb.w; q[j] = fmaf(d, d, q[j]);
      }
    }
    float rmax = 0.f;
#pragma unroll
    for (int j = 0; j < RJ; ++j)
      if (lane + 32 * j < rows_valid) rmax = fmaxf(rmax, q[j]);
    __syncwarp();   // every lane is done reading the slot
    if (lane == 0 && t + NS * stride < n_tiles) {
      fence_proxy_async_smem();
      issue(t + NS * stride, buf);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
    if (WPB == 2) {
      if (lane == 0) s_max[warp] = rmax;
      mbar_arrive(smem_u32(&pair_bar[group]));
      pair_ok = mbar_wait(smem_u32(&pair_bar[group]), 1, status, kWaitStageFree) && pair_ok;
      if (part == 0 && lane == 0 && row_ok) radius[blk] = sqrtf(fmaxf(rmax, s_max[warp ^ 1]));
      if (!__all_sync(0xffffffffu, pair_ok)) break;
    } else {
      if (lane == 0 && row_ok) radius[blk] = sqrtf(rmax);
    }
  }
}

template <int B, int NW, int NS, int WPB, bool BOX>
static rbs_status launch_stats_warp(const rbs_tensor& K, const Dims& x, const rbs_stats& stats, float* box_lo, float* box_hi,
                                    cudaStream_t s) {
  CUtensorMap tm;
  rbs_status st = make_tmap_lthd(&tm, K.ptr, x.L, x.N, x.Hkv, x.d, K.stride_batch, K.stride_token, K.stride_head,
                                 64, B / WPB, true);
  if (st != RBS_OK) return st;
  unsigned int* status = device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  const size_t smem = static_cast<size_t>(NW) * NS * (B / WPB) * 256;
  auto kern = block_stats_warp_kernel<B, NW, NS, WPB, BOX>;
  if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem)) != RBS_OK) return st;
  const long long n_tiles = static_cast<long long>(x.L) * x.Hkv * x.M;
  long long want = (n_tiles + NW / WPB - 1) / (NW / WPB);
  const int grid = static_cast<int>(want < sm_count() ? want : sm_count());
  kern<<<grid, NW * 32, smem, s>>>(tm, static_cast<int>(n_tiles), x.M, x.Hkv, x.N, stats.centroid, stats.radius, box_lo,
                                   box_hi, status);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

}  // namespace rbs

static rbs_status block_stats_impl(const rbs_shape* shape, rbs_tensor K, rbs_stats stats, float* box_lo, float* box_hi,
                                   void* stream) {
  using namespace rbs;
  rbs::NvtxRange nvtx_range("rbs_block_stats");
  rbs_status st = check_shape(shape);
  if (st != RBS_OK) return st;
  st = check_tensor(K);
  if (st != RBS_OK) return st;
  if (stats.centroid == nullptr || stats.radius == nullptr) return RBS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(stats.centroid) % 16 != 0) return RBS_ERR_INVALID_ARG;
  const bool box = box_lo != nullptr;
  if (box && (box_hi == nullptr || reinterpret_cast<uintptr_t>(box_lo) % 16 != 0 || reinterpret_cast<uintptr_t>(box_hi) % 16 != 0))
    return RBS_ERR_INVALID_ARG;
  Dims x = make_dims(*shape);
  const long long n_tiles = static_cast<long long>(x.L) * x.Hkv * x.M;
  if (n_tiles > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Shared memory holds 6 or 7 tiles of 32 KB.  Measured per 128K layer of 4 KV heads (128 MiB):
  //   B = 128: twelve warps in pairs, 64 rows and a 16 KB slot each   31.2 us   (seven warps, one 32 KB slot each:
  //            32.4 us; three warps with two 32 KB slots each: 46 us, compute-bound)
  //   B = 64:  seven warps with two 16 KB slots each used in turn      28.7 us   (fourteen single-slot warps: 31.1 us)
  //   B = 256: six warps in pairs, 128 rows and a 32 KB slot each      35.7 us   (three warps, 64 KB slots: 58 us)
  if (box) {
    if (x.B == 256) return launch_stats_warp<256, 6, 1, 2, true>(K, x, stats, box_lo, box_hi, s);
    if (x.B == 128) return launch_stats_warp<128, 12, 1, 2, true>(K, x, stats, box_lo, box_hi, s);
    return launch_stats_warp<64, 7, 2, 1, true>(K, x, stats, box_lo, box_hi, s);
  }
  if (x.B == 256) return launch_stats_warp<256, 6, 1, 2, false>(K, x, stats, nullptr, nullptr, s);
  if (x.B == 128) return launch_stats_warp<128, 12, 1, 2, false>(K, x, stats, nullptr, nullptr, s);
  return launch_stats_warp<64, 7, 2, 1, false>(K, x, stats, nullptr, nullptr, s);
}

extern "C" rbs_status rbs_block_stats(const rbs_shape* shape, rbs_tensor K, rbs_stats stats, void* stream) {
  return block_stats_impl(shape, K, stats, nullptr, nullptr, stream);
}

extern "C" rbs_status rbs_block_stats_box(const rbs_shape* shape, rbs_tensor K, rbs_stats stats, rbs_box box, void* stream) {
  if (box.lo == nullptr || box.hi == nullptr) return RBS_ERR_INVALID_ARG;
  return block_stats_impl(shape, K, stats, box.lo, box.hi, stream);
}
