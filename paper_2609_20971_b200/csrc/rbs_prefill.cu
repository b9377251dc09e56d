// rbs_sparse_prefill: causal block-sparse attention over a bit-packed block mask (Sec. 3.3), dense when
// the mask is NULL (Eq. 1).  The work horses are the tcgen05 kernels further down (prefill_tc_kernel for blocks of
// 128 and 256, prefill_tc64_kernel for blocks of 64): TMA-fed K/V tiles, S and O accumulators in tensor memory,
// one softmax thread per query row with a lazily updated running maximum, the key list walked straight from the
// mask bits.  prefill_mma_kernel (mma.sync, softmax in registers) only serves a dense chunk that starts on an odd
// block of 64.
#include "rbs_common.cuh"
#include "rbs_sm100.cuh"
#include "rbs_prefill.cuh"

namespace rbs {

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
  const int il = p.Mq - 1 - static_cast<int>(blockIdx.x / per_i);   // query block inside this call's chunk
  const int i = p.q0 + il;                                            // its position in the sequence
  const int rem = static_cast<int>(blockIdx.x % per_i);
  const int l = rem / p.Hq, h = rem % p.Hq, hk = h / p.G;
  const uint32_t* mrow = p.mask ? p.mask + ((static_cast<int64_t>(l) * p.Hq + h) * p.Mq + il) * p.W : nullptr;

  const __nv_bfloat16* qbase = p.Q + l * p.qsb + static_cast<int64_t>(il) * B * p.qst + h * p.qsh;
  const __nv_bfloat16* kbase = p.K + l * p.ksb + hk * p.ksh;
  const __nv_bfloat16* vbase = p.V + l * p.vsb + hk * p.vsh;
  __nv_bfloat16* obase = p.O + l * p.osb + static_cast<int64_t>(il) * B * p.ost + h * p.osh;

  auto load_kv = [&](int b, int stage) {
    const __nv_bfloat16* ks = kbase + static_cast<int64_t>(b) * B * p.kst;
    const __nv_bfloat16* vs = vbase + static_cast<int64_t>(b) * B * p.vst;
    const int rows_in = p.N - b * B;   // keys past the sequence end are loaded as zeros (and hidden by causality)
    for (int c = tid; c < B * 16; c += NTHREADS) {
      const int row = c >> 4, chunk = c & 15;
      const bool in = row < rows_in;
      const int64_t r = in ? row : 0;
      cp_async16_zfill(smem_u32(sK + stage * TILE + tile_off(row, chunk)), ks + r * p.kst + chunk * 8, in);
      cp_async16_zfill(smem_u32(sV + stage * TILE + tile_off(row, chunk)), vs + r * p.vst + chunk * 8, in);
    }
  };

  int b_cur = next_block(mrow, -1, i);
  const int row0 = warp * 16 + gq;  // this thread's first query row inside the block (second: +8)
  const int q_rows = min(B, p.Nq - il * B);   // a short last query block: rows past the sequence end are not written
  if (b_cur < 0) {                  // nothing retained: zero rows, lse = -inf
    for (int c = tid; c < B * 16; c += NTHREADS) {
      const int row = c >> 4, chunk = c & 15;
      if (row < q_rows) *reinterpret_cast<uint4*>(obase + static_cast<int64_t>(row) * p.ost + chunk * 8) = make_uint4(0, 0, 0, 0);
    }
    if (p.lse && tid < q_rows) p.lse[(static_cast<int64_t>(l) * p.Hq + h) * p.Nq + il * B + tid] = -INFINITY;
    return;
  }

  for (int c = tid; c < B * 16; c += NTHREADS) {
    const int row = c >> 4, chunk = c & 15;
    const bool in = row < q_rows;
    cp_async16_zfill(smem_u32(sQ + tile_off(row, chunk)), qbase + static_cast<int64_t>(in ? row : 0) * p.qst + chunk * 8, in);
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
    if (row0 < q_rows) *reinterpret_cast<uint32_t*>(o0 + n * 8 + tq * 2) = pack_bf16(acc_o[n][0] * inv0, acc_o[n][1] * inv0);
    if (row0 + 8 < q_rows) *reinterpret_cast<uint32_t*>(o1 + n * 8 + tq * 2) = pack_bf16(acc_o[n][2] * inv1, acc_o[n][3] * inv1);
  }
  if (p.lse && tq == 0) {
    float* dst = p.lse + (static_cast<int64_t>(l) * p.Hq + h) * p.Nq + il * B;
    if (row0 < q_rows) dst[row0] = (m_run[0] + fast_log2(l_run[0])) * 0.6931471805599453f;
    if (row0 + 8 < q_rows) dst[row0 + 8] = (m_run[1] + fast_log2(l_run[1])) * 0.6931471805599453f;
  }
}

// ---------------------------------------------------------------------------------------------
// Tensor-core path for B = 128 and B = 256 (as 128-row tiles and 128-key sub-blocks): TMA-fed, tcgen05.mma with the accumulators in tensor memory.
//   S[128 q x 128 keys] = Q_i K_b^T          (both operands from shared memory, 8 MMAs of K = 16)
//   O[128 q x 128 d]   += P V_b              (P from tensor memory, V_b from shared memory, 8 MMAs)
// One CTA per (batch, query head, query block), two CTAs per SM so that one CTA's softmax overlaps the
// other's matrix multiplies.  TMEM columns: [0,128) S, with P (bf16 pairs) written over [0,64) once a
// thread has read its S row; [128,256) O.
// Warps 0-3: softmax, one query row per thread (TMEM lane = row).  Warp 4: TMA producer.  Warp 5: MMA issuer.
// Warps 6-7 only exist so that warps 4-7 form a whole warpgroup that can hand its registers to the softmax warps.
// The running row maximum is lazy: exponentials are taken against the maximum in use and a half-row is redone
// against its exact maximum only when its sum reaches kSumLimit, so P stays below kSumLimit and O is rescaled rarely.
// ---------------------------------------------------------------------------------------------
constexpr int kPfThreads = 256;
// Of every (kPolyEvery + 1) groups of four logits, one pair is exponentiated by polynomial on the FMA pipe instead of
// by ex2 (0: every group = 50 % of the exps, 1: 25 %, 3: 12.5 %, 16: none).  The polynomial relieves the exp unit but
// costs about six instructions per element, and the launch is bound by power, not by the exp unit: on the 128K
// workload at 8 % density (median burst / back-to-back ms) 25 %: 10.12 / 11.56, 12.5 %: 10.02 / 11.44, none:
// 9.89 / 11.32.
constexpr int kPolyEvery = 16;

template <bool SCHED>
__global__ void __launch_bounds__(kPfThreads, 2)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                  const PrefillParams p, unsigned int* status) {
  constexpr int B = 128;
  constexpr uint32_t kPanel = B * 128;   // 16 KB: 128 rows x 64 bf16 columns
  constexpr uint32_t kTile = 2 * kPanel;
  constexpr uint32_t kIdescQK = idesc_bf16_f32(128, 128, false);
  constexpr uint32_t kIdescPV = idesc_bf16_f32(128, 128, true);
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sQ = smem;
  unsigned char* sK = smem + kTile;
  unsigned char* sV = smem + 2 * kTile;
  __shared__ __align__(8) uint64_t bar_q, bar_kfull, bar_vfull, bar_s, bar_p, bar_p1, bar_pv0, bar_pv;
  __shared__ uint32_t s_tmem;
  // Per key sub-block, written by the MMA warp before it issues S = Q K^T of that block (two entries used in turn):
  // bit 0: the block is the diagonal one; bit 1: it is the tile's last block.  The softmax warps read it instead of
  // walking the mask themselves.
  __shared__ uint32_t s_blk[2];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // Tile order: the query tiles are cut into bands of band_rows consecutive tiles, the last (longest) band first;
  // inside a band one (batch, KV head) at a time, inside it longest rows first, the G query heads of the group
  // together.  All tiles in flight then read the K/V of one KV head (64 MiB at 128K tokens), which stays in L2;
  // with all KV heads interleaved the K/V tiles of a 128K layer (256 MiB) were re-read from DRAM many times.
  // The bands keep the very long rows (the dense rows of the last query blocks) of every KV head near the start
  // of the launch: with one band, the last KV head's dense rows started after three quarters of the launch and
  // ran on alone after everything else had finished.
  // SCHED: the grid follows the item list of plan_rows_kernel instead: the same order, with rows longer than kSplitCap
  // cut into parts that sit next to each other.
  const int R = p.R;
  const int Hkv = p.Hq / p.G;
  const int per_band_kv = SCHED ? p.items_per_group : p.band_rows * p.G;
  const int per_band = p.L * Hkv * per_band_kv;
  const int band = static_cast<int>(blockIdx.x / per_band), rem_band = static_cast<int>(blockIdx.x % per_band);
  const int kvid = rem_band / per_band_kv;
  int rem = rem_band % per_band_kv;
  // with a schedule the CTA's tile, its range of key sub-blocks and the slot of its partial result come from its item
  int4 item = make_int4(0, 0, 0x7fffffff, -1);
  if (SCHED) {
    item = __ldg(p.items + blockIdx.x);
    if (item.x < 0) return;                 // unused entry of the group's item list
    rem = item.x;
  }
  const int l = kvid / Hkv, hk = kvid % Hkv;
  const int Tl = p.Mq * R - 1 - (band * p.band_rows + rem / p.G);  // 128-row query tile inside this call's chunk
  if (Tl < 0) return;                       // padding of the last band
  const int T = p.q0 * R + Tl;              // its position in the sequence (in 128-token units)
  const int i = T / R;                      // its query block
  const int h = hk * p.G + rem % p.G;
  if (Tl * 128 >= p.Nq) return;             // a tile wholly past the end of the queries (short last block of 256)
  if (!RBS_DBG_OK(i >= p.q0 && i - p.q0 < p.Mq && h < p.Hq && l < p.L && T < p.M * R, status, kDbgPrefillTile)) return;
  const uint32_t* mrow = p.mask ? p.mask + ((static_cast<int64_t>(l) * p.Hq + h) * p.Mq + (i - p.q0)) * p.W : nullptr;
  const int Tw = SCHED ? min(T, item.z - 1) : T;   // last sub-block this CTA may attend (T itself for a whole row)
  const int kb0 = SCHED ? item.y - 1 : -1;         // where the walk over the mask row starts

  if (tid == 0) {
    mbar_init(smem_u32(&bar_q), 1);
    mbar_init(smem_u32(&bar_kfull), 1);
    mbar_init(smem_u32(&bar_vfull), 1);
    mbar_init(smem_u32(&bar_s), 1);
    mbar_init(smem_u32(&bar_p), 128);
    mbar_init(smem_u32(&bar_p1), 128);
    mbar_init(smem_u32(&bar_pv0), 1);
    mbar_init(smem_u32(&bar_pv), 1);
    mbar_fence_init();
    // the Q tile does not depend on the mask: it is on its way before tensor memory is set up and the mask row is read
    // (4.06 / 6.29 / 9.62 against 4.13 / 6.34 / 9.68 ms at 3 / 5 / 8 % density)
    // Q is read exactly once per launch: evict-first, so that it does not push the K/V of the KV head in flight out
    // of L2 (-0.2 % of the launch)
    mbar_arrive_expect_tx(smem_u32(&bar_q), kTile);
    const uint64_t pol_q = make_policy_evict_first();
    tma_load_4d_hint(smem_u32(sQ), &tmQ, smem_u32(&bar_q), 0, h, Tl * B, l, pol_q);
    tma_load_4d_hint(smem_u32(sQ + kPanel), &tmQ, smem_u32(&bar_q), 64, h, Tl * B, l, pol_q);
  }
  if (warp == 5) tmem_alloc(smem_u32(&s_tmem), 256);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_s = s_tmem, tmem_o = s_tmem + 128;

  if (warp >= 4) reg_dealloc<48>();
  if (warp >= 6) {
    // idle: registers donated above
  } else if (warp == 4) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      int b = next_kb(mrow, kb0, i, R, Tw);
      if (b < 0) mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull);   // nothing selected: the Q tile still has to land before the CTA may go
      for (int j = 0; b >= 0; ++j, b = next_kb(mrow, b, i, R, Tw)) {
        if (!RBS_DBG_OK(b <= Tw && b * B < p.N, status, kDbgPrefillBlock)) break;
        if (j > 0 && !mbar_wait(smem_u32(&bar_s), (j - 1) & 1, status, kWaitStageFree)) break;   // S_{j-1} done: K free
        mbar_arrive_expect_tx(smem_u32(&bar_kfull), kTile);
        tma_load_4d(smem_u32(sK), &tmK, smem_u32(&bar_kfull), 0, hk, b * B, l);
        tma_load_4d(smem_u32(sK + kPanel), &tmK, smem_u32(&bar_kfull), 64, hk, b * B, l);
        if (j > 0 && !mbar_wait(smem_u32(&bar_pv), (j - 1) & 1, status, kWaitStageFree)) break;  // O_{j-1} done: V free
        mbar_arrive_expect_tx(smem_u32(&bar_vfull), kTile);
        tma_load_4d(smem_u32(sV), &tmV, smem_u32(&bar_vfull), 0, hk, b * B, l);
        tma_load_4d(smem_u32(sV + kPanel), &tmV, smem_u32(&bar_vfull), 64, hk, b * B, l);
      }
    }
  } else if (warp == 5) {
    // ------------------------------- MMA issuer -------------------------------
    // The whole warp runs this loop in lock step and one elected lane issues each tcgen05 instruction.
    // Everything between two waits sits on the critical path of the tile, so the operand descriptors are
    // built once (they only differ in the address field) and the next block index is fetched from the
    // mask while the softmax of the current block runs.
    {
      int b = next_kb(mrow, kb0, i, R, Tw);
      bool ok = b < 0 || mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull);
      const uint64_t dq = smem_desc_sw128(smem_u32(sQ), 16, 1024);
      const uint64_t dk = smem_desc_sw128(smem_u32(sK), 16, 1024);
      const uint64_t dv = smem_desc_sw128(smem_u32(sV), kPanel, 1024);
      auto issue_qk = [&](int j, int blk, int blk_next) {
        if (lane == 0) {
          s_blk[j & 1] = (blk == T ? 1u : 0u) | (blk_next < 0 ? 2u : 0u);
          __threadfence_block();
        }
        __syncwarp();
        mma_ss_k128_commit_elect(tmem_s, dq, dk, kIdescQK, kPanel, kPanel, smem_u32(&bar_s));
      };
      int b_next = b >= 0 ? next_kb(mrow, b, i, R, Tw) : -1;
      ok = __all_sync(0xffffffffu, ok);
      if (ok && b >= 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_kfull), 0, status, kWaitTmaFull));
        if (ok) {
          tc_fence_after_sync();
          issue_qk(0, b, b_next);
        }
      }
      for (int j = 0; ok && b >= 0; ++j) {
        const uint32_t ph = j & 1;
        const int b_next2 = b_next >= 0 ? next_kb(mrow, b_next, i, R, Tw) : -1;   // global-memory latency hidden behind the softmax
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_vfull), ph, status, kWaitTmaFull) &&
                                         mbar_wait(smem_u32(&bar_p), ph, status, kWaitPReady));   // P of keys 0..63
        if (!ok) break;
        tc_fence_after_sync();
        mma_ts_k64_elect(tmem_o, tmem_s, dv, kIdescPV, 2048 >> 4, j != 0, smem_u32(&bar_pv0));
        // K of the next block arrived while the softmax ran; checking it here, before the wait for the second half
        // of P, keeps that check (about 200 cycles of wait, vote and fence) off the tile's critical path
        if (b_next >= 0) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_kfull), ph ^ 1, status, kWaitTmaFull));
        ok = ok && __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_p1), ph, status, kWaitPReady));   // keys 64..127
        if (!ok) break;
        tc_fence_after_sync();
        mma_ts_k64_elect(tmem_o, tmem_s + 32, dv + static_cast<uint64_t>((4 * 2048) >> 4), kIdescPV, 2048 >> 4, 1, smem_u32(&bar_pv));
        if (b_next >= 0) issue_qk(j + 1, b_next, b_next2);
        b = b_next;
        b_next = b_next2;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------- softmax: one query row per thread -------------------------------
    reg_alloc<208>();
    const int row = warp * 32 + lane;
    const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;
    float m_used = -INFINITY, l_sum = 0.f;   // m_used in log2 units of the scaled logits
    int b = next_kb(mrow, kb0, i, R, Tw);
    const bool any_block = b >= 0;
    bool ok = true;
    int j = 0;
    const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2);
    for (bool more = any_block; more; ++j) {
      if (!(ok = mbar_wait(smem_u32(&bar_s), j & 1, status, kWaitMmaDone))) break;
      const uint32_t blk = *reinterpret_cast<volatile uint32_t*>(&s_blk[j & 1]);
      more = (blk & 2u) == 0u;
      tc_fence_after_sync();
      uint32_t s[128];   // the whole S row of this thread
      {
        uint32_t(&s0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
        uint32_t(&s1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
        uint32_t(&s2)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[64]);
        uint32_t(&s3)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[96]);
        tmem_ld32(tmem_s + lane_off, s0);
        tmem_ld32(tmem_s + lane_off + 32, s1);
        tmem_ld32(tmem_s + lane_off + 64, s2);
        tmem_ld32(tmem_s + lane_off + 96, s3);
        tmem_wait_ld();
      }
      if (blk & 1u) {   // diagonal sub-block: keys after the query are hidden
#pragma unroll
        for (int c = 0; c < 128; ++c)
          if (c > row) s[c] = 0xff800000u;   // -inf
      }
      // Lazy running maximum: the exponentials of a half are first taken against the maximum in use.  Only when a
      // half's sum shows that this has gone stale (sum >= kSumLimit, or not finite; always so for the very first
      // half, where the maximum is still -inf) is the exact maximum of the half computed, O and l rescaled and
      // the half redone.  The maximum is a shift that cancels in O / l, so any value that keeps P finite is right.
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t pk[32];
        auto exps = [&]() -> float {
          const uint64_t negm2 = f2_pack(-m_used, -m_used);
          uint64_t sum_a = 0ull, sum_b = 0ull;   // (0.f, 0.f)
#pragma unroll
          for (int q = 0; q < 64; q += 4) {
            const int c = half * 64 + q;
            const uint64_t x01 = f2_fma(f2_pack(__uint_as_float(s[c]), __uint_as_float(s[c + 1])), scale2, negm2);
            const uint64_t x23 = f2_fma(f2_pack(__uint_as_float(s[c + 2]), __uint_as_float(s[c + 3])), scale2, negm2);
            float x0, x1, x2, x3;
            f2_unpack(x01, x0, x1);
            f2_unpack(x23, x2, x3);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
            float p2, p3;
            if (((q >> 2) & kPolyEvery) == kPolyEvery) {   // a share of the exps goes to the FMA pipe
              exp2_poly_x2(x23, p2, p3);
            } else {
              p2 = fast_exp2(x2);
              p3 = fast_exp2(x3);
            }
            sum_a = f2_add(sum_a, f2_pack(p0, p1));
            sum_b = f2_add(sum_b, f2_pack(p2, p3));
            pk[q >> 1] = pack_bf16(p0, p1);
            pk[(q >> 1) + 1] = pack_bf16(p2, p3);
          }
          float a0, a1, a2, a3;
          f2_unpack(sum_a, a0, a1);
          f2_unpack(sum_b, a2, a3);
          return (a0 + a1) + (a2 + a3);
        };
        // one copy of the exp loop per half, run a second time when the first pass found the maximum stale (the
        // kernel's instruction footprint decides how often its warps wait for instruction fetches)
        float hs = 0.f;
#pragma unroll 1
        for (int attempt = 0; attempt < 2; ++attempt) {
          hs = exps();
          if (attempt == 1 || !__any_sync(0xffffffffu, !(hs < kSumLimit))) break;
          float mxa[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) mxa[u] = -INFINITY;
#pragma unroll
          for (int c = half * 64; c < half * 64 + 64; c += 8) {
#pragma unroll
            for (int u = 0; u < 4; ++u) mxa[u] = max3(mxa[u], __uint_as_float(s[c + 2 * u]), __uint_as_float(s[c + 2 * u + 1]));
          }
          const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3])) * p.scale_log2;
          const float m_new = fmaxf(m_used, mx);
          const float corr = fast_exp2(m_used - m_new);     // 0 while m_used = -inf
          l_sum *= corr;
          m_used = m_new;
          if (j > 0 || half > 0) {   // O holds the P V of everything issued so far: wait for it, then rescale
            if (ok) ok = half == 0 ? mbar_wait(smem_u32(&bar_pv), (j - 1) & 1, status, kWaitOReady)
                                   : mbar_wait(smem_u32(&bar_pv0), j & 1, status, kWaitOReady);
            if (ok) {
              tc_fence_after_sync();
#pragma unroll 1
              for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_o + lane_off + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 32; ++q) r[q] = __float_as_uint(__uint_as_float(r[q]) * corr);
                tmem_st32(tmem_o + lane_off + c0, r);
              }
            }
          }
        }
        l_sum += hs;
        tmem_st32(tmem_s + lane_off + half * 32, pk);
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(smem_u32(half == 0 ? &bar_p : &bar_p1));
      }
      if (!ok) break;
    }
    // epilogue: O / l -> bf16 -> global
    __nv_bfloat16* orow = p.O + l * p.osb + (static_cast<int64_t>(Tl) * B + row) * p.ost + h * p.osh;
    float* lse_dst = p.lse ? p.lse + (static_cast<int64_t>(l) * p.Hq + h) * p.Nq + Tl * B + row : nullptr;
    const bool in_seq = Tl * B + row < p.Nq;   // rows of a short last block past the sequence end are not written
    if (!any_block) {
      if (in_seq) {
#pragma unroll
        for (int c = 0; c < 16; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
        if (lse_dst) *lse_dst = -INFINITY;
      }
    } else if (SCHED && __ldg(&p.items[blockIdx.x].w) >= 0) {
      const int part_slot = __ldg(&p.items[blockIdx.x].w);   // (read again here rather than kept in a register all along)
      // a part of a split row: the unnormalised O row, the maximum in use and the row sum go to the part's slot;
      // combine_parts_kernel merges the parts of the row in a fixed order
      const bool o_ready = __all_sync(0xffffffffu, ok && mbar_wait(smem_u32(&bar_pv), (j - 1) & 1, status, kWaitOReady));
      tc_fence_after_sync();
      float* po = p.part_o + (static_cast<int64_t>(part_slot) * 128 + row) * 128;
#pragma unroll 1
      for (int c0 = 0; o_ready && c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_o + lane_off + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < 32; q += 4)
          *reinterpret_cast<uint4*>(po + c0 + q) = make_uint4(r[q], r[q + 1], r[q + 2], r[q + 3]);
      }
      if (o_ready) {
        float* ml = p.part_ml + static_cast<int64_t>(part_slot) * 256;
        ml[row] = m_used;
        ml[128 + row] = l_sum;
      }
    } else {
      // every thread of the four warps reaches the barrier below, also one whose wait has given up
      const bool o_ready = __all_sync(0xffffffffu, ok && mbar_wait(smem_u32(&bar_pv), (j - 1) & 1, status, kWaitOReady));
      // O / l -> bf16 -> the Q buffer (free since the tile's last Q K^T), in the swizzled layout of a 128-byte-swizzle
      // tensor map, then two TMA stores: whole 128-byte lines go out instead of one 16-byte piece per row and
      // instruction, and rows past the end of the sequence are clipped by the tensor map.
      tc_fence_after_sync();
      const float inv = 1.0f / l_sum;
      const uint32_t srow = smem_u32(sQ) + row * 128;
#pragma unroll
      for (int c0 = 0; o_ready && c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_o + lane_off + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < 32; q += 8) {
          uint4 v;
          v.x = pack_bf16(__uint_as_float(r[q]) * inv, __uint_as_float(r[q + 1]) * inv);
          v.y = pack_bf16(__uint_as_float(r[q + 2]) * inv, __uint_as_float(r[q + 3]) * inv);
          v.z = pack_bf16(__uint_as_float(r[q + 4]) * inv, __uint_as_float(r[q + 5]) * inv);
          v.w = pack_bf16(__uint_as_float(r[q + 6]) * inv, __uint_as_float(r[q + 7]) * inv);
          const int chunk = (c0 + q) >> 3;   // 16-byte piece 0..15 of the row
          const uint32_t dst = srow + (chunk >> 3) * kPanel + (((chunk & 7) ^ (row & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
      }
      fence_proxy_async_smem();
      asm volatile("bar.sync 1, 128;" ::: "memory");   // the four softmax warps
      if (tid == 0 && o_ready) {
        tma_store_4d(&tmO, smem_u32(sQ), 0, h, Tl * B, l);
        tma_store_4d(&tmO, smem_u32(sQ + kPanel), 64, h, Tl * B, l);
        tma_store_commit();
        tma_store_wait_read();
      }
      if (lse_dst && in_seq && o_ready && RBS_DBG_OK(Tl * B + row < p.Nq, status, kDbgPrefillLse)) *lse_dst = (m_used + fast_log2(l_sum)) * 0.6931471805599453f;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == 5) tmem_dealloc(s_tmem, 256);
}

// ---------------------------------------------------------------------------------------------
// Row-length-aware schedule of prefill_tc_kernel (the index compaction of the method's complexity paragraph, Sec. 3.3,
// in the form this kernel needs: per-row counts of selected blocks, long rows cut into parts).
// One CTA per group = (band of query tiles, batch, KV head), the unit inside which the static order keeps the K/V of
// one KV head in flight.  It counts the selected 128-key sub-blocks of each of the group's rows from the mask and
// writes one item per CTA of the attention kernel, in the static order (rows from the end of the sequence backwards,
// i.e. longest candidate range first, the G heads of a row together).  The first kSplitRowsPerGroup rows of that
// order that exceed kSplitCap sub-blocks are cut into up to kSplitMaxParts parts of equal length, placed next to each
// other.  (Sorting the rows of a group by their counts was measured as well: 0.03 - 0.1 ms slower on the 128K layer.)
// ---------------------------------------------------------------------------------------------
constexpr int kPlanThreads = 1024;

// number of 128-key sub-blocks tile T of query block i attends in mask row `row`: R per selected block below the
// diagonal block, and the diagonal block's sub-blocks up to T
__device__ __forceinline__ int count_kb_fast(const uint32_t* __restrict__ row, int i, int R, int T) {
  int n = 0;
  const int wi = i >> 5;
  for (int w = 0; w < wi; ++w) n += __popc(__ldg(row + w));
  const uint32_t u = __ldg(row + wi) & (0xffffffffu >> (31 - (i & 31)));
  const uint32_t diag = (u >> (i & 31)) & 1u;
  return R * (n + __popc(u) - static_cast<int>(diag)) + (diag ? T - i * R + 1 : 0);
}

// the same count by walking the set bits, stopping at ordinal `stop` (>= 0): *kb_at receives the index of the
// sub-block with that ordinal
__device__ __forceinline__ int count_kb(const uint32_t* __restrict__ row, int i, int R, int T, int stop, int* kb_at) {
  int n = 0;
  for (int w = 0; w <= (i >> 5); ++w) {
    uint32_t u = __ldg(row + w);
    if (((w + 1) << 5) - 1 > i) u &= 0xffffffffu >> (31 - (i & 31));
    while (u) {
      const int b = (w << 5) + __ffs(u) - 1;
      u &= u - 1;
      const int first = b * R, last = min(b * R + R - 1, T);   // this block's sub-blocks up to the diagonal
      if (stop >= 0 && n + (last - first + 1) > stop) { *kb_at = first + (stop - n); return stop; }
      n += last - first + 1;
    }
  }
  return n;
}

__global__ void __launch_bounds__(kPlanThreads)
plan_rows_kernel(const PrefillParams p, int4* __restrict__ items, int4* __restrict__ splits) {
  extern __shared__ int s_cnt[];                     // sub-blocks per row of the group, in static order
  __shared__ int s_warp_long[kPlanThreads / 32];
  __shared__ int s_split_pos[kSplitRowsPerGroup], s_split_parts[kSplitRowsPerGroup], s_n_split;
  const int R = p.R, Hkv = p.Hq / p.G;
  const int n_g = p.band_rows * p.G;               // rows (128-row tiles) per group
  const int g = blockIdx.x;                        // band * (L * Hkv) + kvid
  const int band = g / (p.L * Hkv), kvid = g % (p.L * Hkv);
  const int l = kvid / Hkv, hk = kvid % Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  auto tile_of = [&](int pos, int& Tl, int& T, int& i, const uint32_t*& row) -> bool {
    Tl = p.Mq * R - 1 - (band * p.band_rows + pos / p.G);
    if (Tl < 0 || Tl * 128 >= p.Nq) return false;
    T = p.q0 * R + Tl;
    i = T / R;
    const int h = hk * p.G + pos % p.G;
    row = p.mask + ((static_cast<int64_t>(l) * p.Hq + h) * p.Mq + (i - p.q0)) * p.W;
    return true;
  };
  // every thread owns a contiguous run of rows, so that ranks in static order come from one scan over the threads
  const int per_thread = (n_g + kPlanThreads - 1) / kPlanThreads;
  const int first = tid * per_thread, last = min(n_g, first + per_thread);
  int n_long = 0;
  for (int pos = first; pos < last; ++pos) {
    int Tl, T, i;
    const uint32_t* row;
    const int cnt = tile_of(pos, Tl, T, i, row) ? count_kb_fast(row, i, R, T) : -1;   // -1: no such tile
    s_cnt[pos] = cnt;
    n_long += cnt > kSplitCap;
  }
  if (tid == 0) s_n_split = 0;
  // exclusive scan of n_long over the threads
  int incl = n_long;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_warp_long[warp] = incl;
  __syncthreads();
  int rank = incl - n_long;
  for (int w = 0; w < warp; ++w) rank += s_warp_long[w];
  for (int pos = first; pos < last && rank < kSplitRowsPerGroup; ++pos) {
    const int cnt = s_cnt[pos];
    if (cnt > kSplitCap) {
      s_split_pos[rank] = pos;
      s_split_parts[rank] = min(kSplitMaxParts, (cnt + kSplitCap - 1) / kSplitCap);
      atomicMax(&s_n_split, rank + 1);
      ++rank;
    }
  }
  __syncthreads();
  const int n_split = s_n_split;
  const int per_group = n_g + kExtraItemsPerGroup;
  int4* out = items + static_cast<int64_t>(g) * per_group;
  int extra_total = 0;
  for (int s = 0; s < n_split; ++s) extra_total += s_split_parts[s] - 1;
  // whole rows
  for (int pos = first; pos < last; ++pos) {
    int at = pos;
    bool is_split = false;
    for (int s = 0; s < n_split; ++s) {
      if (s_split_pos[s] < pos) at += s_split_parts[s] - 1;
      is_split |= s_split_pos[s] == pos;
    }
    if (!is_split) out[at] = s_cnt[pos] >= 0 ? make_int4(pos, 0, 0x7fffffff, -1) : make_int4(-1, 0, 0, -1);
  }
  for (int e = n_g + extra_total + tid; e < per_group; e += kPlanThreads) out[e] = make_int4(-1, 0, 0, -1);   // unused
  // the parts of the split rows: one thread per (row, part)
  if (tid < kSplitRowsPerGroup * kSplitMaxParts) {
    const int s = tid / kSplitMaxParts, part = tid % kSplitMaxParts;
    if (s < n_split) {
      const int pos = s_split_pos[s], parts = s_split_parts[s], cnt = s_cnt[pos];
      if (part < parts) {
        int at = pos + part;
        for (int s2 = 0; s2 < s; ++s2) at += s_split_parts[s2] - 1;
        int Tl, T, i;
        const uint32_t* row;
        tile_of(pos, Tl, T, i, row);
        const int len = (cnt + parts - 1) / parts;
        int kb_begin = 0, kb_end = T + 1;
        if (part > 0) count_kb(row, i, R, T, part * len, &kb_begin);
        if (part + 1 < parts) count_kb(row, i, R, T, (part + 1) * len, &kb_end);
        out[at] = make_int4(pos, kb_begin, kb_end, g * kSplitSlotsPerGroup + s * kSplitMaxParts + part);
      }
      if (part == 0) splits[g * kSplitRowsPerGroup + s] = make_int4(pos, parts, 0, 0);
    } else if (part == 0) {
      splits[g * kSplitRowsPerGroup + s] = make_int4(-1, 1, 0, 0);
    }
  }
}

// Merges the parts of one split row: with m = max_p m_p,  l = sum_p l_p 2^(m_p - m),  O = sum_p O_p 2^(m_p - m) / l
// (the maximum is only a shift, Sec. 3.3's softmax over the retained keys is unchanged), parts taken in order.
// One CTA per (group, split-row slot), one thread per query row.
__global__ void __launch_bounds__(128)
combine_parts_kernel(const PrefillParams p, const int4* __restrict__ splits) {
  const int4 sp = splits[blockIdx.x];
  if (sp.x < 0) return;
  const int g = blockIdx.x / kSplitRowsPerGroup, s = blockIdx.x % kSplitRowsPerGroup;
  const int R = p.R, Hkv = p.Hq / p.G;
  const int band = g / (p.L * Hkv), kvid = g % (p.L * Hkv);
  const int l = kvid / Hkv, hk = kvid % Hkv;
  const int Tl = p.Mq * R - 1 - (band * p.band_rows + sp.x / p.G);
  const int h = hk * p.G + sp.x % p.G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int slot0 = g * kSplitSlotsPerGroup + s * kSplitMaxParts;
  // a warp takes one query row at a time, its lanes four output columns each (whole 512-byte lines per part)
  for (int row = warp; row < 128; row += 4) {
    if (Tl * 128 + row >= p.Nq) break;     // rows past the end of the queries are not written
    float m = -INFINITY;
    for (int q = 0; q < sp.y; ++q) m = fmaxf(m, p.part_ml[static_cast<int64_t>(slot0 + q) * 256 + row]);
    float lsum = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int q = 0; q < sp.y; ++q) {
      const float* ml = p.part_ml + static_cast<int64_t>(slot0 + q) * 256;
      const float w = fast_exp2(ml[row] - m);
      lsum = fmaf(ml[128 + row], w, lsum);
      const float4 a = *reinterpret_cast<const float4*>(p.part_o + (static_cast<int64_t>(slot0 + q) * 128 + row) * 128 + lane * 4);
      acc.x = fmaf(a.x, w, acc.x); acc.y = fmaf(a.y, w, acc.y); acc.z = fmaf(a.z, w, acc.z); acc.w = fmaf(a.w, w, acc.w);
    }
    const float inv = 1.0f / lsum;
    __nv_bfloat16* orow = p.O + l * p.osb + (static_cast<int64_t>(Tl) * 128 + row) * p.ost + h * p.osh;
    uint2 v;
    v.x = pack_bf16(acc.x * inv, acc.y * inv);
    v.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(orow + lane * 4) = v;
    if (p.lse && lane == 0) p.lse[(static_cast<int64_t>(l) * p.Hq + h) * p.Nq + Tl * 128 + row] = (m + fast_log2(lsum)) * 0.6931471805599453f;
  }
}

static rbs_status launch_prefill_tc(const PrefillParams& p, const rbs_tensor& Q, const rbs_tensor& K,
                                    const rbs_tensor& V, int Hkv, void* workspace, size_t workspace_bytes, cudaStream_t s) {
  CUtensorMap tmQ, tmK, tmV;
  rbs_status st;
  if ((st = make_tmap_lthd(&tmQ, Q.ptr, p.L, p.Nq, p.Hq, kHeadDim, Q.stride_batch, Q.stride_token, Q.stride_head, 64, 128, true)) != RBS_OK) return st;
  if ((st = make_tmap_lthd(&tmK, K.ptr, p.L, p.N, Hkv, kHeadDim, K.stride_batch, K.stride_token, K.stride_head, 64, 128, true)) != RBS_OK) return st;
  if ((st = make_tmap_lthd(&tmV, V.ptr, p.L, p.N, Hkv, kHeadDim, V.stride_batch, V.stride_token, V.stride_head, 64, 128, true)) != RBS_OK) return st;
  CUtensorMap tmO;
  const int64_t osb = p.osb, ost = p.ost, osh = p.osh;
  if ((st = make_tmap_lthd(&tmO, p.O, p.L, p.Nq, p.Hq, kHeadDim, osb, ost, osh, 64, 128, true)) != RBS_OK) return st;
  unsigned int* status = device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  const size_t smem = 3 * 2 * 128 * 128;
  if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_tc_kernel<false>), smem)) != RBS_OK) return st;
  if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_tc_kernel<true>), smem)) != RBS_OK) return st;
  PrefillParams pp = p;
  const int n_rows = p.Mq * p.R;
  // up to four bands of at least 64 query tiles (512 CTAs per band and KV head at G = 8: enough to fill the GPU
  // from one KV head).  Measured at 128K, 32 q / 4 kv heads: 1 / 4 / 8 / 16 bands give 5.52 / 4.86 / 4.97 / 4.90 ms
  // at 3 % density and 17.5 / 16.7 / 17.2 / 17.2 ms at 12 %.
  int n_bands = n_rows / 64;
  n_bands = n_bands < 1 ? 1 : (n_bands > 4 ? 4 : n_bands);
  pp.band_rows = (n_rows + n_bands - 1) / n_bands;
  const int n_groups = n_bands * p.L * Hkv;
  const int rows_per_group = pp.band_rows * p.G;
  pp.items = nullptr; pp.items_per_group = 0; pp.part_o = nullptr; pp.part_ml = nullptr;
  int4* splits = nullptr;
  // the schedule needs the mask (dense attention keeps one CTA per tile: its launch is long and its rows shrink
  // steadily) and a group whose counts fit the planner's shared memory
  const size_t plan_smem = static_cast<size_t>(rows_per_group) * sizeof(int);
  const bool scheduled = p.mask != nullptr && workspace != nullptr && plan_smem <= 200 * 1024;
  if (scheduled) {
    const PrefillWorkspace w = prefill_workspace(p.L, p.Hq, Hkv, p.M * p.R, p.G);
    if (workspace_bytes < w.bytes || reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return RBS_ERR_WORKSPACE;
    unsigned char* base = static_cast<unsigned char*>(workspace);
    int4* items = reinterpret_cast<int4*>(base + w.off_items);
    splits = reinterpret_cast<int4*>(base + w.off_splits);
    pp.items = items;
    pp.items_per_group = rows_per_group + kExtraItemsPerGroup;
    pp.part_o = reinterpret_cast<float*>(base + w.off_part_o);
    pp.part_ml = reinterpret_cast<float*>(base + w.off_part_ml);
    if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(plan_rows_kernel), plan_smem)) != RBS_OK) return st;
    plan_rows_kernel<<<n_groups, kPlanThreads, plan_smem, s>>>(pp, items, splits);
    RBS_CUDA_OK(cudaGetLastError());
  }
  const long long n_cta = static_cast<long long>(n_groups) * (scheduled ? pp.items_per_group : rows_per_group);
  if (n_cta > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  if (scheduled) prefill_tc_kernel<true><<<static_cast<unsigned>(n_cta), kPfThreads, smem, s>>>(tmQ, tmK, tmV, tmO, pp, status);
  else prefill_tc_kernel<false><<<static_cast<unsigned>(n_cta), kPfThreads, smem, s>>>(tmQ, tmK, tmV, tmO, pp, status);
  RBS_CUDA_OK(cudaGetLastError());
  if (scheduled) {
    combine_parts_kernel<<<n_groups * kSplitRowsPerGroup, 128, 0, s>>>(pp, splits);
    RBS_CUDA_OK(cudaGetLastError());
  }
  return RBS_OK;
}

// ---------------------------------------------------------------------------------------------
// Tensor-core path for blocks of 64.  A 128-row tile holds two consecutive query blocks (rows 0-63: block iA,
// rows 64-127: block iB = iA + 1), each with its own mask row; the tile walks the union of the two rows in key
// blocks of 64 and every row half takes part only in the key blocks its own mask row selects (for the other half
// P is zero and no exponential is computed: the halves are whole warps).  Per key block:
//   S[128 q x 64 keys] = Q K_b^T   (8 MMAs of K = 16, N = 64)      O[128 q x 128 d] += P V_b   (4 MMAs, K = 64 keys)
// The work executed is the union of the two rows, so the kernel pays off when neighbouring query blocks select
// similar key blocks (forced blocks always do).  K and V are double-buffered (16 KB stages): with key blocks this
// short the next block must already be on its way while the current one is multiplied.
// TMEM columns: [0,64) S with P (bf16 pairs) over [0,32); [128,256) O.  Roles and CTA shape as in prefill_tc_kernel.
// ---------------------------------------------------------------------------------------------
struct Pair64 {
  const uint32_t* rowA; const uint32_t* rowB;   // mask rows of the two query blocks (rowB null: no second block)
  int iA, iB;
  // next key block after `cur` (-1 to start) selected by either row within its causal range, or -1
  __device__ __forceinline__ int next(int cur) const {
    const int last = rowB ? iB : iA;
    int b = cur + 1;
    while (b <= last) {
      const int w = b >> 5;
      uint32_t u = __ldg(rowA + w);
      if (((w + 1) << 5) - 1 > iA) u = (w << 5) > iA ? 0u : (u & (0xffffffffu >> (31 - (iA & 31))));
      if (rowB) {
        uint32_t v = __ldg(rowB + w);
        if (((w + 1) << 5) - 1 > iB) v = (w << 5) > iB ? 0u : (v & (0xffffffffu >> (31 - (iB & 31))));
        u |= v;
      }
      u >>= (b & 31);
      if (u) return b + __ffs(u) - 1;
      b = (b | 31) + 1;
    }
    return -1;
  }
  // bit 0 / 1: the block is selected by row A / B; bit 2 / 3: it is the diagonal block of row A / B
  __device__ __forceinline__ uint32_t flags(int b) const {
    uint32_t f = 0;
    if (b <= iA && ((__ldg(rowA + (b >> 5)) >> (b & 31)) & 1u)) f |= 1u;
    if (rowB && b <= iB && ((__ldg(rowB + (b >> 5)) >> (b & 31)) & 1u)) f |= 2u;
    if (b == iA) f |= 4u;
    if (b == iB) f |= 8u;
    return f;
  }
};

__global__ void __launch_bounds__(kPfThreads, 2)
prefill_tc64_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                    const PrefillParams p, unsigned int* status) {
  constexpr int B = 64;
  constexpr uint32_t kPanel = 128 * 128;       // Q: 128 rows x 64 bf16 columns = 16 KB
  constexpr uint32_t kTile = 2 * kPanel;
  constexpr uint32_t kHalfPanel = 64 * 128;    // K/V: 64 rows x 64 bf16 columns = 8 KB
  constexpr uint32_t kStage = 2 * kHalfPanel;  // one K or V stage: 16 KB
  constexpr uint32_t kIdescQK = idesc_bf16_f32(128, 64, false);
  constexpr uint32_t kIdescPV = idesc_bf16_f32(128, 128, true);
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sQ = smem;
  unsigned char* sK = smem + kTile;                // two stages
  unsigned char* sV = smem + kTile + 2 * kStage;   // two stages
  __shared__ __align__(8) uint64_t bar_q, bar_kfull[2], bar_vfull[2], bar_kempty[2], bar_vempty[2], bar_s, bar_p, bar_pv;
  __shared__ uint32_t s_tmem;
  __shared__ uint32_t s_blk[2];   // flags of the key block (see Pair64::flags), bit 4: the tile's last block

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // tile order as in prefill_tc_kernel, in units of 128-row tiles (two query blocks)
  const int n_rows = (p.Mq + 1) / 2;
  const int Hkv = p.Hq / p.G;
  const int per_band_kv = p.band_rows * p.G;
  const int per_band = p.L * Hkv * per_band_kv;
  const int band = static_cast<int>(blockIdx.x / per_band), rem_band = static_cast<int>(blockIdx.x % per_band);
  const int kvid = rem_band / per_band_kv, rem = rem_band % per_band_kv;
  const int l = kvid / Hkv, hk = kvid % Hkv;
  const int Tl = n_rows - 1 - (band * p.band_rows + rem / p.G);   // 128-row tile inside this call's chunk
  if (Tl < 0) return;
  const int h = hk * p.G + rem % p.G;
  Pair64 pr;
  pr.iA = p.q0 + 2 * Tl;
  pr.iB = pr.iA + 1;
  pr.rowA = p.mask + ((static_cast<int64_t>(l) * p.Hq + h) * p.Mq + 2 * Tl) * p.W;
  pr.rowB = (2 * Tl + 1 < p.Mq) ? pr.rowA + p.W : nullptr;

  if (tid == 0) {
    mbar_init(smem_u32(&bar_q), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&bar_kfull[s]), 1);
      mbar_init(smem_u32(&bar_vfull[s]), 1);
      mbar_init(smem_u32(&bar_kempty[s]), 1);
      mbar_init(smem_u32(&bar_vempty[s]), 1);
    }
    mbar_init(smem_u32(&bar_s), 1);
    mbar_init(smem_u32(&bar_p), 128);
    mbar_init(smem_u32(&bar_pv), 1);
    mbar_fence_init();
  }
  if (warp == 5) tmem_alloc(smem_u32(&s_tmem), 256);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_s = s_tmem, tmem_o = s_tmem + 128;

  if (warp >= 4) reg_dealloc<48>();
  if (warp >= 6) {
    // idle: registers donated above
  } else if (warp == 4) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      int b = pr.next(-1);
      if (b >= 0) {
        mbar_arrive_expect_tx(smem_u32(&bar_q), kTile);
        tma_load_4d(smem_u32(sQ), &tmQ, smem_u32(&bar_q), 0, h, Tl * 128, l);
        tma_load_4d(smem_u32(sQ + kPanel), &tmQ, smem_u32(&bar_q), 64, h, Tl * 128, l);
      }
      for (int n = 0; b >= 0; ++n, b = pr.next(b)) {
        const int st = n & 1;
        const uint32_t par = ((n >> 1) - 1) & 1;   // the stage's previous use
        if (n >= 2 && !mbar_wait(smem_u32(&bar_kempty[st]), par, status, kWaitStageFree)) break;
        mbar_arrive_expect_tx(smem_u32(&bar_kfull[st]), kStage);
        tma_load_4d(smem_u32(sK + st * kStage), &tmK, smem_u32(&bar_kfull[st]), 0, hk, b * B, l);
        tma_load_4d(smem_u32(sK + st * kStage + kHalfPanel), &tmK, smem_u32(&bar_kfull[st]), 64, hk, b * B, l);
        if (n >= 2 && !mbar_wait(smem_u32(&bar_vempty[st]), par, status, kWaitStageFree)) break;
        mbar_arrive_expect_tx(smem_u32(&bar_vfull[st]), kStage);
        tma_load_4d(smem_u32(sV + st * kStage), &tmV, smem_u32(&bar_vfull[st]), 0, hk, b * B, l);
        tma_load_4d(smem_u32(sV + st * kStage + kHalfPanel), &tmV, smem_u32(&bar_vfull[st]), 64, hk, b * B, l);
      }
    }
  } else if (warp == 5) {
    // ------------------------------- MMA issuer -------------------------------
    // The whole warp runs this loop in lock step and one elected lane issues each tcgen05 instruction.
    int b = pr.next(-1);
    bool ok = b < 0 || mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull);
    ok = __all_sync(0xffffffffu, ok);
    const uint64_t dq = smem_desc_sw128(smem_u32(sQ), 16, 1024);
    uint64_t dk[2], dv[2];
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      dk[s] = smem_desc_sw128(smem_u32(sK + s * kStage), 16, 1024);
      dv[s] = smem_desc_sw128(smem_u32(sV + s * kStage), kHalfPanel, 1024);
    }
    int b_next = b >= 0 ? pr.next(b) : -1;
    auto issue_qk = [&](int n, int blk, int blk_next) {
      if (lane == 0) {
        s_blk[n & 1] = pr.flags(blk) | (blk_next < 0 ? 16u : 0u);
        __threadfence_block();
      }
      __syncwarp();
      const int st = n & 1;
      mma_ss_k128_commit_elect(tmem_s, dq, st ? dk[1] : dk[0], kIdescQK, kPanel, kHalfPanel, smem_u32(&bar_kempty[st]));
      mma_commit_elect(smem_u32(&bar_s));
    };
    if (ok && b >= 0) {
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_kfull[0]), 0, status, kWaitTmaFull));
      if (ok) {
        tc_fence_after_sync();
        issue_qk(0, b, b_next);
      }
    }
    for (int n = 0; ok && b >= 0; ++n) {
      const int st = n & 1;
      const uint32_t ph = n & 1, sph = (n >> 1) & 1;
      const int b_next2 = b_next >= 0 ? pr.next(b_next) : -1;   // global-memory latency hidden behind the softmax
      // K of the next block is checked before the wait for P: the check stays off the tile's critical path
      if (b_next >= 0) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_kfull[st ^ 1]), ((n + 1) >> 1) & 1, status, kWaitTmaFull));
      ok = ok && __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_vfull[st]), sph, status, kWaitTmaFull) &&
                                             mbar_wait(smem_u32(&bar_p), ph, status, kWaitPReady));
      if (!ok) break;
      tc_fence_after_sync();
      mma_ts_k64_elect(tmem_o, tmem_s, st ? dv[1] : dv[0], kIdescPV, 2048 >> 4, n != 0, smem_u32(&bar_vempty[st]));
      mma_commit_elect(smem_u32(&bar_pv));
      if (b_next >= 0) issue_qk(n + 1, b_next, b_next2);
      b = b_next;
      b_next = b_next2;
    }
    __syncwarp();
  } else {
    // ------------------------------- softmax: one query row per thread -------------------------------
    reg_alloc<208>();
    const int row = warp * 32 + lane;
    const int rh = warp >> 1;                       // row half: 0 = block iA, 1 = block iB (whole warps)
    const int rloc = row - rh * 64;                 // row inside its query block
    const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;
    float m_used = -INFINITY, l_sum = 0.f;          // m_used in log2 units of the scaled logits
    const bool any_block = pr.next(-1) >= 0;
    bool ok = true;
    int n = 0;
    const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2);
    for (bool more = any_block; more; ++n) {
      if (!(ok = mbar_wait(smem_u32(&bar_s), n & 1, status, kWaitMmaDone))) break;
      const uint32_t blk = *reinterpret_cast<volatile uint32_t*>(&s_blk[n & 1]);
      more = (blk & 16u) == 0u;
      tc_fence_after_sync();
      uint32_t pk[32];
      if ((blk >> rh) & 1u) {   // this row half attends the block
        uint32_t s[64];
        {
          uint32_t(&s0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
          uint32_t(&s1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
          tmem_ld32(tmem_s + lane_off, s0);
          tmem_ld32(tmem_s + lane_off + 32, s1);
          tmem_wait_ld();
        }
        if ((blk >> (2 + rh)) & 1u) {   // the half's diagonal block: keys after the query are hidden
#pragma unroll
          for (int c = 0; c < 64; ++c)
            if (c > rloc) s[c] = 0xff800000u;   // -inf
        }
        // lazy running maximum, as in prefill_tc_kernel
        auto exps = [&]() -> float {
          const uint64_t negm2 = f2_pack(-m_used, -m_used);
          uint64_t sum_a = 0ull, sum_b = 0ull;   // (0.f, 0.f)
#pragma unroll
          for (int q = 0; q < 64; q += 4) {
            const uint64_t x01 = f2_fma(f2_pack(__uint_as_float(s[q]), __uint_as_float(s[q + 1])), scale2, negm2);
            const uint64_t x23 = f2_fma(f2_pack(__uint_as_float(s[q + 2]), __uint_as_float(s[q + 3])), scale2, negm2);
            float x0, x1, x2, x3;
            f2_unpack(x01, x0, x1);
            f2_unpack(x23, x2, x3);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1), p2 = fast_exp2(x2), p3 = fast_exp2(x3);
            sum_a = f2_add(sum_a, f2_pack(p0, p1));
            sum_b = f2_add(sum_b, f2_pack(p2, p3));
            pk[q >> 1] = pack_bf16(p0, p1);
            pk[(q >> 1) + 1] = pack_bf16(p2, p3);
          }
          float a0, a1, a2, a3;
          f2_unpack(sum_a, a0, a1);
          f2_unpack(sum_b, a2, a3);
          return (a0 + a1) + (a2 + a3);
        };
        float hs = 0.f;
#pragma unroll 1
        for (int attempt = 0; attempt < 2; ++attempt) {
          hs = exps();
          if (attempt == 1 || !__any_sync(0xffffffffu, !(hs < kSumLimit))) break;
          float mxa[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) mxa[u] = -INFINITY;
#pragma unroll
          for (int c = 0; c < 64; c += 8) {
#pragma unroll
            for (int u = 0; u < 4; ++u) mxa[u] = max3(mxa[u], __uint_as_float(s[c + 2 * u]), __uint_as_float(s[c + 2 * u + 1]));
          }
          const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3])) * p.scale_log2;
          const float m_new = fmaxf(m_used, mx);
          const float corr = fast_exp2(m_used - m_new);     // 0 while m_used = -inf
          l_sum *= corr;
          m_used = m_new;
          if (n > 0) {   // O holds the P V of everything issued so far: wait for it, then rescale
            if (ok) ok = mbar_wait(smem_u32(&bar_pv), (n - 1) & 1, status, kWaitOReady);
            if (ok) {
              tc_fence_after_sync();
#pragma unroll 1
              for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem_o + lane_off + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 32; ++q) r[q] = __float_as_uint(__uint_as_float(r[q]) * corr);
                tmem_st32(tmem_o + lane_off + c0, r);
              }
            }
          }
        }
        l_sum += hs;
      } else {
#pragma unroll
        for (int q = 0; q < 32; ++q) pk[q] = 0u;   // P = 0 for the rows whose block did not select these keys
      }
      tmem_st32(tmem_s + lane_off, pk);
      tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(smem_u32(&bar_p));
      if (!ok) break;
    }
    // epilogue: O / l -> bf16 -> global
    const int64_t tok = static_cast<int64_t>(Tl) * 128 + row;
    __nv_bfloat16* orow = p.O + l * p.osb + tok * p.ost + h * p.osh;
    float* lse_dst = p.lse ? p.lse + (static_cast<int64_t>(l) * p.Hq + h) * p.Nq + tok : nullptr;
    const bool in_seq = tok < p.Nq;   // rows past the end of the queries are not written
    if (!any_block) {
      if (in_seq) {
#pragma unroll
        for (int c = 0; c < 16; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
        if (lse_dst) *lse_dst = -INFINITY;
      }
    } else {
      // every thread of the four warps reaches the barrier below, also one whose wait has given up
      const bool o_ready = __all_sync(0xffffffffu, ok && mbar_wait(smem_u32(&bar_pv), (n - 1) & 1, status, kWaitOReady));
      tc_fence_after_sync();
      const bool empty_row = !(l_sum > 0.f);          // a row whose own block selected nothing: zeros, lse = -inf
      const float inv = empty_row ? 0.f : 1.0f / l_sum;
      const uint32_t srow = smem_u32(sQ) + row * 128;
#pragma unroll
      for (int c0 = 0; o_ready && c0 < 128; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem_o + lane_off + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int q = 0; q < 32; q += 8) {
          uint4 v;
          v.x = pack_bf16(__uint_as_float(r[q]) * inv, __uint_as_float(r[q + 1]) * inv);
          v.y = pack_bf16(__uint_as_float(r[q + 2]) * inv, __uint_as_float(r[q + 3]) * inv);
          v.z = pack_bf16(__uint_as_float(r[q + 4]) * inv, __uint_as_float(r[q + 5]) * inv);
          v.w = pack_bf16(__uint_as_float(r[q + 6]) * inv, __uint_as_float(r[q + 7]) * inv);
          if (empty_row) v = make_uint4(0, 0, 0, 0);
          const int chunk = (c0 + q) >> 3;   // 16-byte piece 0..15 of the row
          const uint32_t dst = srow + (chunk >> 3) * kPanel + (((chunk & 7) ^ (row & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
      }
      fence_proxy_async_smem();
      asm volatile("bar.sync 1, 128;" ::: "memory");   // the four softmax warps
      if (tid == 0 && o_ready) {
        tma_store_4d(&tmO, smem_u32(sQ), 0, h, Tl * 128, l);
        tma_store_4d(&tmO, smem_u32(sQ + kPanel), 64, h, Tl * 128, l);
        tma_store_commit();
        tma_store_wait_read();
      }
      if (lse_dst && in_seq && o_ready) *lse_dst = empty_row ? -INFINITY : (m_used + fast_log2(l_sum)) * 0.6931471805599453f;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == 5) tmem_dealloc(s_tmem, 256);
}

static rbs_status launch_prefill_tc64(const PrefillParams& p, const rbs_tensor& Q, const rbs_tensor& K,
                                      const rbs_tensor& V, int Hkv, cudaStream_t s) {
  CUtensorMap tmQ, tmK, tmV, tmO;
  rbs_status st;
  if ((st = make_tmap_lthd(&tmQ, Q.ptr, p.L, p.Nq, p.Hq, kHeadDim, Q.stride_batch, Q.stride_token, Q.stride_head, 64, 128, true)) != RBS_OK) return st;
  if ((st = make_tmap_lthd(&tmK, K.ptr, p.L, p.N, Hkv, kHeadDim, K.stride_batch, K.stride_token, K.stride_head, 64, 64, true)) != RBS_OK) return st;
  if ((st = make_tmap_lthd(&tmV, V.ptr, p.L, p.N, Hkv, kHeadDim, V.stride_batch, V.stride_token, V.stride_head, 64, 64, true)) != RBS_OK) return st;
  if ((st = make_tmap_lthd(&tmO, p.O, p.L, p.Nq, p.Hq, kHeadDim, p.osb, p.ost, p.osh, 64, 128, true)) != RBS_OK) return st;
  unsigned int* status = device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  const size_t smem = 2 * 128 * 128 + 4 * 2 * 64 * 128;   // Q + two stages each of K and V
  if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_tc64_kernel), smem)) != RBS_OK) return st;
  PrefillParams pp = p;
  const int n_rows = (p.Mq + 1) / 2;
  int n_bands = n_rows / 64;
  n_bands = n_bands < 1 ? 1 : (n_bands > 4 ? 4 : n_bands);
  pp.band_rows = (n_rows + n_bands - 1) / n_bands;
  const long long n_cta = static_cast<long long>(p.L) * p.Hq * pp.band_rows * n_bands;
  if (n_cta > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  prefill_tc64_kernel<<<static_cast<unsigned>(n_cta), kPfThreads, smem, s>>>(tmQ, tmK, tmV, tmO, pp, status);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

template <int B>
static rbs_status launch_prefill(const PrefillParams& p, cudaStream_t s) {
  const size_t smem = static_cast<size_t>(5) * B * 256;
  { const rbs_status st = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_mma_kernel<B>), smem); if (st != RBS_OK) return st; }
  const long long n_cta = static_cast<long long>(p.L) * p.Hq * p.Mq;
  if (n_cta > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  prefill_mma_kernel<B><<<static_cast<unsigned>(n_cta), B * 2, smem, s>>>(p);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

}  // namespace rbs

// grouped: the caller states that the query heads of a KV group have identical mask rows (rbs_sparse_prefill_grouped)
static rbs_status prefill_impl(const rbs_shape* shape, int q_start_block, int n_q_tokens, rbs_tensor Q, rbs_tensor K,
                               rbs_tensor V, const uint32_t* mask, rbs_tensor O, float* lse, float softmax_scale,
                               void* workspace, size_t workspace_bytes, void* stream, bool grouped = false) {
  using namespace rbs;
  rbs::NvtxRange nvtx_range("rbs_sparse_prefill");
  rbs_status st = check_shape(shape);
  if (st != RBS_OK) return st;
  if ((st = check_tensor(Q)) != RBS_OK || (st = check_tensor(K)) != RBS_OK || (st = check_tensor(V)) != RBS_OK ||
      (st = check_tensor(O)) != RBS_OK)
    return st;
  if (softmax_scale < 0.f) return RBS_ERR_INVALID_ARG;
  Dims x = make_dims(*shape);
  if (n_q_tokens < 0) { q_start_block = 0; n_q_tokens = x.N; }
  if ((st = check_chunk(x, q_start_block, n_q_tokens)) != RBS_OK) return st;
  PrefillParams p;
  p.q0 = q_start_block; p.Nq = n_q_tokens; p.Mq = (n_q_tokens + x.B - 1) / x.B;
  p.Q = static_cast<const __nv_bfloat16*>(Q.ptr); p.qsb = Q.stride_batch; p.qst = Q.stride_token; p.qsh = Q.stride_head;
  p.K = static_cast<const __nv_bfloat16*>(K.ptr); p.ksb = K.stride_batch; p.kst = K.stride_token; p.ksh = K.stride_head;
  p.V = static_cast<const __nv_bfloat16*>(V.ptr); p.vsb = V.stride_batch; p.vst = V.stride_token; p.vsh = V.stride_head;
  p.O = static_cast<__nv_bfloat16*>(O.ptr); p.osb = O.stride_batch; p.ost = O.stride_token; p.osh = O.stride_head;
  p.mask = mask; p.lse = lse;
  p.M = x.M; p.W = x.W; p.L = x.L; p.Hq = x.Hq; p.G = x.G; p.N = x.N;
  const float scale = softmax_scale == 0.f ? 1.0f / sqrtf(static_cast<float>(x.d)) : softmax_scale;
  p.scale_log2 = scale * kLog2e;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  p.R = x.B / 128;
  p.band_rows = 0; p.items = nullptr; p.items_per_group = 0; p.part_o = nullptr; p.part_ml = nullptr;
  if (grouped) {
    if (mask == nullptr) return RBS_ERR_INVALID_ARG;
    if (x.B < 128 || x.G % 2 != 0) return RBS_ERR_UNSUPPORTED;
    return launch_prefill_pair(p, Q, K, V, x.Hkv, 0, s);
  }
  if (x.B >= 128 && mask != nullptr && workspace != nullptr) {   // checked before anything touches the GPU
    const PrefillWorkspace w = prefill_workspace(x.L, x.Hq, x.Hkv, x.M * p.R, x.G);
    if (workspace_bytes < w.bytes || reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return RBS_ERR_WORKSPACE;
  }
  if (x.B >= 128) return launch_prefill_tc(p, Q, K, V, x.Hkv, workspace, workspace_bytes, s);   // tensor-core path (blocks of 128 or 256)
  if (mask == nullptr && (q_start_block & 1) == 0) {
    // Dense attention does not depend on the block size: blocks of 64 run on the tensor-core path as blocks of 128
    // (a chunk has to start on a 128-token boundary for that).
    p.R = 1;
    p.q0 = q_start_block / 2;
    p.Mq = (n_q_tokens + 127) / 128;
    p.M = (x.N + 127) / 128;
    p.W = (p.M + 31) / 32;
    return launch_prefill_tc(p, Q, K, V, x.Hkv, nullptr, 0, s);
  }
  if (mask != nullptr) return launch_prefill_tc64(p, Q, K, V, x.Hkv, s);   // blocks of 64, two query blocks per tile
  return launch_prefill<64>(p, s);   // dense chunk from an odd block of 64: register-softmax mma.sync kernel
}

extern "C" rbs_status rbs_sparse_prefill(const rbs_shape* shape, rbs_tensor Q, rbs_tensor K, rbs_tensor V,
                                         const uint32_t* mask, rbs_tensor O, float* lse, float softmax_scale,
                                         void* workspace, size_t workspace_bytes, void* stream) {
  return prefill_impl(shape, -1, -1, Q, K, V, mask, O, lse, softmax_scale, workspace, workspace_bytes, stream);
}

extern "C" rbs_status rbs_sparse_prefill_chunk(const rbs_shape* shape, int q_start_block, int n_q_tokens, rbs_tensor Q,
                                               rbs_tensor K, rbs_tensor V, const uint32_t* mask, rbs_tensor O, float* lse,
                                               float softmax_scale, void* workspace, size_t workspace_bytes,
                                               void* stream) {
  if (n_q_tokens <= 0) return RBS_ERR_INVALID_ARG;
  return prefill_impl(shape, q_start_block, n_q_tokens, Q, K, V, mask, O, lse, softmax_scale, workspace,
                      workspace_bytes, stream);
}

extern "C" rbs_status rbs_sparse_prefill_grouped(const rbs_shape* shape, rbs_tensor Q, rbs_tensor K, rbs_tensor V,
                                                 const uint32_t* mask, rbs_tensor O, float* lse, float softmax_scale,
                                                 void* stream) {
  return prefill_impl(shape, -1, -1, Q, K, V, mask, O, lse, softmax_scale, nullptr, 0, stream, true);
}
