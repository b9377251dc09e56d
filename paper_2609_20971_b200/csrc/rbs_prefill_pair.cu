// Two query tiles per CTA over ONE stream of K/V tiles: the attention kernel for query tiles that attend the same
// key blocks --
//   mode 0 (heads): two query heads of a KV group at the same query tile, under group-shared masks
//                   (rbs_mask_group_union: every head of the group keeps the same key blocks);
//   mode 1 (rows):  two consecutive 128-row query tiles of one head: the two halves of a query block of 256, or two
//                   neighbouring tiles of dense attention (the second tile attends one key tile more, its diagonal).
// Each selected K/V tile is brought into shared memory once for both query tiles (half the TMA, L2 and shared-memory
// fill traffic per FLOP of prefill_tc_kernel, which runs the same two tiles as two CTAs with a K/V copy each), and the
// K/V tiles are double-buffered.  Measured on B200 the saving does not pay: the same tiles run about 25 % faster as two
// independent CTAs of prefill_tc_kernel (tensor pipe 63 % against 44 % busy on dense 32K; 50 against 63 ms under the
// group-shared mask of the 128K layer; starting tile B half a block behind tile A changes nothing), so only
// rbs_sparse_prefill_grouped uses this kernel and mode 1 is kept for measurement.  Per tile the chain is the one of prefill_tc_kernel:
//   S = Q K_b^T (tcgen05.mma, both operands in shared memory) -> softmax, one query row per thread, lazily updated
//   running maximum -> P (bf16 pairs over S in tensor memory) -> O += P V_b (P from tensor memory),
// with its own softmax warpgroup and its own MMA-issuing warp; the two chains meet only at the K/V stages.
// Warps 0-3 / 4-7: softmax of tile A / B.  Warp 8: TMA producer.  Warps 9 / 10: MMA issuer of tile A / B.  Warp 11: owns
// the tensor-memory allocation (and completes the warpgroup that hands its registers to the softmax warps).
// TMEM columns: [0,128) S_A, [128,256) O_A, [256,384) S_B, [384,512) O_B.  One CTA per SM.
#include "rbs_prefill.cuh"

namespace rbs {

constexpr int kPairPfThreads = 384;

struct PairParams {
  PrefillParams p;
  int mode;         // 0: head pairs, 1: row pairs
  int band_prows;   // pair rows per band of the tile order
  int n_prows;      // pair rows of the call
  int pcols;        // pairs per pair row and KV head: G / 2 (heads) or G (rows)
};

__global__ void __launch_bounds__(kPairPfThreads, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                    const PairParams pp, unsigned int* status) {
  const PrefillParams& p = pp.p;
  constexpr int B = 128;
  constexpr uint32_t kPanel = B * 128;   // 16 KB: 128 rows x 64 bf16 columns
  constexpr uint32_t kTile = 2 * kPanel;
  constexpr uint32_t kIdescQK = idesc_bf16_f32(128, 128, false);
  constexpr uint32_t kIdescPV = idesc_bf16_f32(128, 128, true);
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sQ = smem;                  // [2 tiles][kTile]
  unsigned char* sK = smem + 2 * kTile;      // [2 stages][kTile]
  unsigned char* sV = smem + 4 * kTile;      // [2 stages][kTile]
  __shared__ __align__(8) uint64_t bar_q, bar_kfull[2], bar_vfull[2], bar_kempty[2], bar_vempty[2];
  __shared__ __align__(8) uint64_t bar_s[2], bar_p[2], bar_p1[2], bar_pv0[2], bar_pv[2];   // per tile
  __shared__ uint32_t s_tmem;
  // per tile and key block (two entries used in turn), written by the tile's MMA warp before it issues S = Q K^T:
  // bit 0: the block is the tile's diagonal one; bit 1: it is the tile's last block
  __shared__ uint32_t s_blk[2][2];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // pair order: as the tile order of prefill_tc_kernel (bands of pair rows, the last band first; inside a band one
  // (batch, KV head) at a time, longest rows first, the pairs of a row together)
  const int R = p.R;
  const int Hkv = p.Hq / p.G;
  const int per_band_kv = pp.band_prows * pp.pcols;
  const int per_band = p.L * Hkv * per_band_kv;
  const int band = static_cast<int>(blockIdx.x / per_band), rem_band = static_cast<int>(blockIdx.x % per_band);
  const int kvid = rem_band / per_band_kv, rem = rem_band % per_band_kv;
  const int l = kvid / Hkv, hk = kvid % Hkv;
  const int prow = pp.n_prows - 1 - (band * pp.band_prows + rem / pp.pcols);
  if (prow < 0) return;                      // padding of the last band
  const int pcol = rem % pp.pcols;
  // the two tiles: head, tile index inside the call's chunk, tile index in the sequence
  int h0, h1, Tl0, Tl1;
  if (pp.mode == 0) {
    h0 = hk * p.G + 2 * pcol; h1 = h0 + 1;
    Tl0 = Tl1 = prow;
  } else {
    h0 = h1 = hk * p.G + pcol;
    Tl0 = 2 * prow; Tl1 = 2 * prow + 1;
  }
  const int T0 = p.q0 * R + Tl0, T1 = p.q0 * R + Tl1;
  const bool act0 = Tl0 < p.Mq * R && Tl0 * 128 < p.Nq, act1 = Tl1 < p.Mq * R && Tl1 * 128 < p.Nq;
  if (!act0 && !act1) return;
  const int n_act = (act0 ? 1 : 0) + (act1 ? 1 : 0);
  // the walk over the key tiles follows the tile that reaches furthest (B when it exists); a tile takes part in the
  // key tiles up to its own diagonal
  const int Tw = act1 ? T1 : T0, iw = Tw / R;
  const uint32_t* mrow = p.mask ? p.mask + ((static_cast<int64_t>(l) * p.Hq + (act1 ? h1 : h0)) * p.Mq + (iw - p.q0)) * p.W : nullptr;

  if (tid == 0) {
    mbar_init(smem_u32(&bar_q), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&bar_kfull[s]), 1); mbar_init(smem_u32(&bar_vfull[s]), 1);
      mbar_init(smem_u32(&bar_kempty[s]), n_act); mbar_init(smem_u32(&bar_vempty[s]), n_act);
      mbar_init(smem_u32(&bar_s[s]), 1);
      mbar_init(smem_u32(&bar_p[s]), 128); mbar_init(smem_u32(&bar_p1[s]), 128);
      mbar_init(smem_u32(&bar_pv0[s]), 1); mbar_init(smem_u32(&bar_pv[s]), 1);
    }
    mbar_fence_init();
  }
  if (warp == 11) tmem_alloc(smem_u32(&s_tmem), 512);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s_tmem;

  if (warp >= 8) reg_dealloc<48>();
  if (warp == 11) {
    // idle: registers donated above
  } else if (warp == 8) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
      int b = next_kb(mrow, -1, iw, R, Tw);
      if (b >= 0) {
        mbar_arrive_expect_tx(smem_u32(&bar_q), n_act * kTile);
        if (act0) {
          tma_load_4d(smem_u32(sQ), &tmQ, smem_u32(&bar_q), 0, h0, Tl0 * B, l);
          tma_load_4d(smem_u32(sQ + kPanel), &tmQ, smem_u32(&bar_q), 64, h0, Tl0 * B, l);
        }
        if (act1) {
          tma_load_4d(smem_u32(sQ + kTile), &tmQ, smem_u32(&bar_q), 0, h1, Tl1 * B, l);
          tma_load_4d(smem_u32(sQ + kTile + kPanel), &tmQ, smem_u32(&bar_q), 64, h1, Tl1 * B, l);
        }
      }
      for (int j = 0; b >= 0; ++j, b = next_kb(mrow, b, iw, R, Tw)) {
        const int st = j & 1;
        const uint32_t par = ((j >> 1) - 1) & 1;   // the stage's previous use
        if (j >= 2 && !mbar_wait(smem_u32(&bar_kempty[st]), par, status, kWaitStageFree)) break;
        mbar_arrive_expect_tx(smem_u32(&bar_kfull[st]), kTile);
        tma_load_4d(smem_u32(sK + st * kTile), &tmK, smem_u32(&bar_kfull[st]), 0, hk, b * B, l);
        tma_load_4d(smem_u32(sK + st * kTile + kPanel), &tmK, smem_u32(&bar_kfull[st]), 64, hk, b * B, l);
        if (j >= 2 && !mbar_wait(smem_u32(&bar_vempty[st]), par, status, kWaitStageFree)) break;
        mbar_arrive_expect_tx(smem_u32(&bar_vfull[st]), kTile);
        tma_load_4d(smem_u32(sV + st * kTile), &tmV, smem_u32(&bar_vfull[st]), 0, hk, b * B, l);
        tma_load_4d(smem_u32(sV + st * kTile + kPanel), &tmV, smem_u32(&bar_vfull[st]), 64, hk, b * B, l);
      }
    }
  } else if (warp == 9 || warp == 10) {
    // ------------------------------- MMA issuer of tile x -------------------------------
    // The whole warp runs the loop in lock step; one elected lane issues each tcgen05 instruction.  Key tile j of the
    // walk sits in stage j & 1; the tile takes part in the key tiles up to its diagonal, which are a prefix of the walk.
    const int x = warp - 9;
    if (x ? act1 : act0) {
      const int Tx = x ? T1 : T0;
      const uint32_t tmem_s = tmem_base + x * 256, tmem_o = tmem_s + 128;
      int b = next_kb(mrow, -1, iw, R, Tw);
      if (b > Tx) b = -1;
      bool ok = b < 0 || mbar_wait(smem_u32(&bar_q), 0, status, kWaitTmaFull);
      ok = __all_sync(0xffffffffu, ok);
      const uint64_t dq = smem_desc_sw128(smem_u32(sQ + x * kTile), 16, 1024);
      uint64_t dk[2], dv[2];
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        dk[s] = smem_desc_sw128(smem_u32(sK + s * kTile), 16, 1024);
        dv[s] = smem_desc_sw128(smem_u32(sV + s * kTile), kPanel, 1024);
      }
      auto next_own = [&](int cur) { const int nb = next_kb(mrow, cur, iw, R, Tw); return nb > Tx ? -1 : nb; };
      auto issue_qk = [&](int j, int blk, int blk_next) {
        if (lane == 0) {
          s_blk[x][j & 1] = (blk == Tx ? 1u : 0u) | (blk_next < 0 ? 2u : 0u);
          __threadfence_block();
        }
        __syncwarp();
        const int st = j & 1;
        mma_ss_k128_commit_elect(tmem_s, dq, st ? dk[1] : dk[0], kIdescQK, kPanel, kPanel, smem_u32(&bar_kempty[st]));
        mma_commit_elect(smem_u32(&bar_s[x]));
      };
      int b_next = b >= 0 ? next_own(b) : -1;
      if (ok && b >= 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_kfull[0]), 0, status, kWaitTmaFull));
        if (ok) {
          tc_fence_after_sync();
          issue_qk(0, b, b_next);
        }
      }
      for (int j = 0; ok && b >= 0; ++j) {
        const int st = j & 1;
        const uint32_t ph = j & 1, sph = (j >> 1) & 1;
        const int b_next2 = b_next >= 0 ? next_own(b_next) : -1;   // global-memory latency hidden behind the softmax
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_vfull[st]), sph, status, kWaitTmaFull) &&
                                         mbar_wait(smem_u32(&bar_p[x]), ph, status, kWaitPReady));   // P of keys 0..63
        if (!ok) break;
        tc_fence_after_sync();
        mma_ts_k64_elect(tmem_o, tmem_s, st ? dv[1] : dv[0], kIdescPV, 2048 >> 4, j != 0, smem_u32(&bar_pv0[x]));
        // K of the next key tile is checked before the wait for the second half of P: off the tile's critical path
        if (b_next >= 0) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_kfull[st ^ 1]), ((j + 1) >> 1) & 1, status, kWaitTmaFull));
        ok = ok && __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_p1[x]), ph, status, kWaitPReady));   // keys 64..127
        if (!ok) break;
        tc_fence_after_sync();
        mma_ts_k64_elect(tmem_o, tmem_s + 32, (st ? dv[1] : dv[0]) + static_cast<uint64_t>((4 * 2048) >> 4), kIdescPV, 2048 >> 4, 1,
                         smem_u32(&bar_vempty[st]));
        mma_commit_elect(smem_u32(&bar_pv[x]));
        if (b_next >= 0) issue_qk(j + 1, b_next, b_next2);
        b = b_next;
        b_next = b_next2;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------- softmax of tile x: one query row per thread -------------------------------
    reg_alloc<208>();
    const int x = warp >> 2, wq = warp & 3;
    if (x ? act1 : act0) {
      const int Tx = x ? T1 : T0, Tl = x ? Tl1 : Tl0, h = x ? h1 : h0;
      const uint32_t tmem_s = tmem_base + x * 256, tmem_o = tmem_s + 128;
      const int row = wq * 32 + lane;
      const uint32_t lane_off = static_cast<uint32_t>(wq * 32) << 16;
      float m_used = -INFINITY, l_sum = 0.f;   // m_used in log2 units of the scaled logits
      const int b_first = next_kb(mrow, -1, iw, R, Tw);
      const bool any_block = b_first >= 0 && b_first <= Tx;
      bool ok = true;
      int j = 0;
      const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2);
      for (bool more = any_block; more; ++j) {
        if (!(ok = mbar_wait(smem_u32(&bar_s[x]), j & 1, status, kWaitMmaDone))) break;
        const uint32_t blk = *reinterpret_cast<volatile uint32_t*>(&s_blk[x][j & 1]);
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
        if (blk & 1u) {   // diagonal key tile: keys after the query are hidden
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c > row) s[c] = 0xff800000u;   // -inf
        }
        // lazy running maximum, as in prefill_tc_kernel: exponentials against the maximum in use; a half whose sum
        // reaches kSumLimit (or is not finite: always so for the very first half) adopts its exact maximum, rescales
        // O and l, and is redone
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
              if (ok) ok = half == 0 ? mbar_wait(smem_u32(&bar_pv[x]), (j - 1) & 1, status, kWaitOReady)
                                     : mbar_wait(smem_u32(&bar_pv0[x]), j & 1, status, kWaitOReady);
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
          mbar_arrive(smem_u32(half == 0 ? &bar_p[x] : &bar_p1[x]));
        }
        if (!ok) break;
      }
      // epilogue: O / l -> bf16 -> global
      __nv_bfloat16* orow = p.O + l * p.osb + (static_cast<int64_t>(Tl) * B + row) * p.ost + h * p.osh;
      float* lse_dst = p.lse ? p.lse + (static_cast<int64_t>(l) * p.Hq + h) * p.Nq + Tl * B + row : nullptr;
      const bool in_seq = Tl * B + row < p.Nq;   // rows past the end of the queries are not written
      if (!any_block) {
        if (in_seq) {
#pragma unroll
          for (int c = 0; c < 16; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
          if (lse_dst) *lse_dst = -INFINITY;
        }
      } else {
        // every thread of the four warps reaches the barrier below, also one whose wait has given up
        const bool o_ready = __all_sync(0xffffffffu, ok && mbar_wait(smem_u32(&bar_pv[x]), (j - 1) & 1, status, kWaitOReady));
        // O / l -> bf16 -> the tile's Q buffer (free since its last Q K^T) in the swizzled layout, then two TMA stores
        tc_fence_after_sync();
        const float inv = 1.0f / l_sum;
        unsigned char* stage = sQ + x * kTile;
        const uint32_t srow = smem_u32(stage) + row * 128;
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
        asm volatile("bar.sync %0, 128;" ::"r"(1 + x) : "memory");   // this tile's four softmax warps
        if (wq == 0 && lane == 0 && o_ready) {
          tma_store_4d(&tmO, smem_u32(stage), 0, h, Tl * B, l);
          tma_store_4d(&tmO, smem_u32(stage + kPanel), 64, h, Tl * B, l);
          tma_store_commit();
          tma_store_wait_read();
        }
        if (lse_dst && in_seq && o_ready) *lse_dst = (m_used + fast_log2(l_sum)) * 0.6931471805599453f;
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == 11) tmem_dealloc(s_tmem, 512);
}

rbs_status launch_prefill_pair(const PrefillParams& p, const rbs_tensor& Q, const rbs_tensor& K, const rbs_tensor& V, int Hkv,
                               int mode, cudaStream_t s) {
  CUtensorMap tmQ, tmK, tmV, tmO;
  rbs_status st;
  if ((st = make_tmap_lthd(&tmQ, Q.ptr, p.L, p.Nq, p.Hq, kHeadDim, Q.stride_batch, Q.stride_token, Q.stride_head, 64, 128, true)) != RBS_OK) return st;
  if ((st = make_tmap_lthd(&tmK, K.ptr, p.L, p.N, Hkv, kHeadDim, K.stride_batch, K.stride_token, K.stride_head, 64, 128, true)) != RBS_OK) return st;
  if ((st = make_tmap_lthd(&tmV, V.ptr, p.L, p.N, Hkv, kHeadDim, V.stride_batch, V.stride_token, V.stride_head, 64, 128, true)) != RBS_OK) return st;
  if ((st = make_tmap_lthd(&tmO, p.O, p.L, p.Nq, p.Hq, kHeadDim, p.osb, p.ost, p.osh, 64, 128, true)) != RBS_OK) return st;
  unsigned int* status = device_status_ptr();
  if (status == nullptr) return RBS_ERR_CUDA;
  const size_t smem = 6 * 2 * 128 * 128;   // two Q tiles, two stages each of K and V
  if ((st = ensure_dynamic_smem(reinterpret_cast<const void*>(prefill_pair_kernel), smem)) != RBS_OK) return st;
  PairParams pp;
  pp.p = p;
  pp.mode = mode;
  const int n_rows = p.Mq * p.R;
  pp.n_prows = mode == 0 ? n_rows : (n_rows + 1) / 2;
  pp.pcols = mode == 0 ? p.G / 2 : p.G;
  int n_bands = pp.n_prows / 64;
  n_bands = n_bands < 1 ? 1 : (n_bands > 4 ? 4 : n_bands);
  pp.band_prows = (pp.n_prows + n_bands - 1) / n_bands;
  const long long n_cta = static_cast<long long>(p.L) * Hkv * pp.pcols * pp.band_prows * n_bands;
  if (n_cta > 0x7fffffffLL) return RBS_ERR_UNSUPPORTED;
  prefill_pair_kernel<<<static_cast<unsigned>(n_cta), kPairPfThreads, smem, s>>>(tmQ, tmK, tmV, tmO, pp, status);
  RBS_CUDA_OK(cudaGetLastError());
  return RBS_OK;
}

}  // namespace rbs
