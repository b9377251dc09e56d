// Device helpers shared by the block-scoring kernels (the RBS selector and the Quest-style box selector): the
// per-block log-sum-exp of Eq. block_aggregation from an accumulator row in tensor memory, the query norms that its
// shifts need, and a named barrier over one epilogue group.
#pragma once

#include "rbs_common.cuh"
#include "rbs_sm100.cuh"

namespace rbs {

// Barrier `id` over the NT threads of one epilogue group, returning whether `ok` held in all of them.
template <int NT>
__device__ __forceinline__ bool group_all(bool ok, int id) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"(static_cast<uint32_t>(ok)), "r"(id), "n"(NT) : "memory");
  return r != 0;
}

// Query norms of one Q tile (B tokens, 128-byte-swizzled panels of 64 columns in shared memory), by the NT threads
// of an epilogue group: sD[t] = ||q_t|| - max_t ||q_t|| (<= 0), and the maximum and the spread (max - min) of the norms
// over the block's n_tok real tokens.  `red` is 2 * NT / 32 floats of scratch.  Two group barriers.
// PANEL_STRIDE: bytes from the first panel of the tile to the second.
template <int B, int NT, uint32_t PANEL_STRIDE = B * 128>
__device__ __forceinline__ bool query_norm_shifts(const unsigned char* q, int wtid, int n_tok, float* sD, float* red,
                                                  int bar_id, bool ok, float& qn_max, float& qn_spread) {
  constexpr uint32_t kPanelQ = PANEL_STRIDE;
  constexpr int TPT = (B + NT - 1) / NT;   // tokens per thread
  constexpr int NWG = NT / 32;
  const int lane = wtid & 31, wq = wtid >> 5;
  float nrm[TPT];
  float mx = 0.f, mn = INFINITY;
#pragma unroll
  for (int u = 0; u < TPT; ++u) {
    const int tok = wtid + u * NT;
    nrm[u] = 0.f;
    if (ok && tok < B) {
      float s2[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};   // eight independent chains of 32 terms
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 v = *reinterpret_cast<const uint4*>(q + (c >> 3) * kPanelQ + tok * 128 + (((c & 7) ^ (tok & 7)) << 4));
        const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float a = bf16lo(wv[e]), c2 = bf16hi(wv[e]);
          s2[2 * e] = fmaf(a, a, s2[2 * e]);
          s2[2 * e + 1] = fmaf(c2, c2, s2[2 * e + 1]);
        }
      }
      nrm[u] = sqrtf(((s2[0] + s2[1]) + (s2[2] + s2[3])) + ((s2[4] + s2[5]) + (s2[6] + s2[7])));
      if (tok < n_tok) { mx = fmaxf(mx, nrm[u]); mn = fminf(mn, nrm[u]); }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
  }
  if (lane == 0) { red[wq] = mx; red[NWG + wq] = mn; }
  ok = group_all<NT>(ok, bar_id);
  qn_max = red[0];
  float qn_min = red[NWG];
#pragma unroll
  for (int u = 1; u < NWG; ++u) { qn_max = fmaxf(qn_max, red[u]); qn_min = fminf(qn_min, red[NWG + u]); }
  qn_spread = qn_max - qn_min;
#pragma unroll
  for (int u = 0; u < TPT; ++u) {
    const int tok = wtid + u * NT;
    if (tok < B) sD[tok] = nrm[u] - qn_max;
  }
  return group_all<NT>(ok, bar_id);
}

// Scores the 128 centroid rows of one tile against the B tokens of a query block, one row per thread, from the
// accumulator row at `taddr` in tensor memory, which holds x_t = q_t . c_b scale in log2 units (the scale is folded
// into the centroids).  With the shifts  m_b = ||q||max ||c_b scale||  (Cauchy-Schwarz: x_t <= m_b)  and
// m_r = m_b + ||q||max gs  the two exponents are
//     e_t = x_t - m_b                 (base branch, Eq. base_score)
//     f_t = e_t + gs (||q_t|| - ||q||max) = (x_t + ||q_t|| gs) - m_r     (rescue branch, Eq. rescue_score)
// both <= 0, one packed add and one packed multiply-add per pair of tokens; then L = m + log2 sum_t 2^(.)
// (Eq. block_aggregation as a per-block log-sum-exp; any shift common to the block's tokens cancels).
// The bounds are used as shifts only while no term can underflow: e_t >= -2 m_b, f_t >= -2 m_b - gs * spread of the
// norms.  Otherwise (warp-uniform decision) a first pass takes the exact maxima and each branch gets its own pass.
// A warp whose 32 rows all have gs = 0 computes no rescue exponentials: S_rescue = S_base there.
// `release()` is called once, when the accumulator has been read for the last time.
template <int B, bool PREFETCH, typename Release>
__device__ __forceinline__ void score_tile(uint32_t taddr, const float* __restrict__ sD, float gs, float cn, float qn_max,
                                           float qn_spread, int n_tok, Release release, float& Lb, float& Lr) {
  float mb = qn_max * cn * 1.0001f;
  const bool no_rescue = __all_sync(0xffffffffu, gs == 0.f);
  const bool cheap = __all_sync(0xffffffffu, mb <= 60.0f && fmaf(gs, qn_spread, 2.0f * mb) <= 120.0f);
  float shift_r = fmaf(qn_max, gs, mb);      // m_r
  float c_first = -mb, c_second = 0.f;
  int n_pass = 1;
  if (!cheap) {
    // exact maxima of x and of y = x + ||q_t|| gs
    float mb0 = -INFINITY, mb1 = -INFINITY, mr0 = -INFINITY, mr1 = -INFINITY;
    const uint64_t g2 = f2_pack(gs, gs), qm2 = f2_pack(qn_max, qn_max);
#pragma unroll 1
    for (int c0 = 0; c0 < B; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(taddr + c0, r);
      tmem_wait_ld();
      if (n_tok < B) {
#pragma unroll
        for (int qq = 0; qq < 32; ++qq)
          if (c0 + qq >= n_tok) r[qq] = 0xff800000u;   // -inf: tokens past the sequence end do not count
      }
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        const float4 d = *reinterpret_cast<const float4*>(sD + c0 + j);
        float y0, y1, y2, y3;
        f2_unpack(f2_fma(f2_add(f2_pack(d.x, d.y), qm2), g2, f2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1]))), y0, y1);
        f2_unpack(f2_fma(f2_add(f2_pack(d.z, d.w), qm2), g2, f2_pack(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]))), y2, y3);
        mb0 = max3(mb0, __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
        mb1 = max3(mb1, __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
        mr0 = max3(mr0, y0, y1);
        mr1 = max3(mr1, y2, y3);
      }
    }
    mb = fmaxf(mb0, mb1);
    shift_r = fmaxf(mr0, mr1);
    c_first = -mb;
    c_second = fmaf(qn_max, gs, -shift_r);     // e' = x + c  =>  e' + gs (||q_t|| - ||q||max) = y_t - max y
    n_pass = no_rescue ? 1 : 2;
  }
  const uint64_t g2 = f2_pack(gs, gs);
  float sum_b = 0.f, sum_r = 0.f;
#pragma unroll 1
  for (int pass = 0; pass < n_pass; ++pass) {
    const float c = pass == 0 ? c_first : c_second;
    const uint64_t c2 = f2_pack(c, c);
    const bool last = pass == n_pass - 1;
    uint64_t sb_a = 0ull, sb_b = 0ull, sr_a = 0ull, sr_b = 0ull;
    auto chunk = [&](uint32_t (&r)[32], int c0) {
      if (n_tok < B) {
#pragma unroll
        for (int qq = 0; qq < 32; ++qq)
          if (c0 + qq >= n_tok) r[qq] = 0xff800000u;   // -inf
      }
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        const uint64_t e01 = f2_add(f2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), c2);
        const uint64_t e23 = f2_add(f2_pack(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])), c2);
        float e0, e1, e2, e3;
        f2_unpack(e01, e0, e1);
        f2_unpack(e23, e2, e3);
        sb_a = f2_add(sb_a, f2_pack(fast_exp2(e0), fast_exp2(e1)));
        sb_b = f2_add(sb_b, f2_pack(fast_exp2(e2), fast_exp2(e3)));
        if (!no_rescue) {
          const float4 d = *reinterpret_cast<const float4*>(sD + c0 + j);
          float f0, f1, f2, f3;
          f2_unpack(f2_fma(f2_pack(d.x, d.y), g2, e01), f0, f1);
          f2_unpack(f2_fma(f2_pack(d.z, d.w), g2, e23), f2, f3);
          sr_a = f2_add(sr_a, f2_pack(fast_exp2(f0), fast_exp2(f1)));
          sr_b = f2_add(sr_b, f2_pack(fast_exp2(f2), fast_exp2(f3)));
        }
      }
    };
    if (PREFETCH) {
      uint32_t ra[32], rb[32];
      tmem_ld32(taddr, ra);
#pragma unroll 1
      for (int c0 = 0; c0 < B; c0 += 64) {
        tmem_wait_ld();
        tmem_ld32(taddr + c0 + 32, rb);          // on its way while the first 32 columns are reduced
        chunk(ra, c0);
        tmem_wait_ld();
        if (c0 + 64 < B) tmem_ld32(taddr + c0 + 64, ra);
        else if (last) release();                 // the accumulator has been read completely
        chunk(rb, c0 + 32);
      }
    } else {
#pragma unroll 1
      for (int c0 = 0; c0 < B; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + c0, r);
        tmem_wait_ld();
        if (last && c0 + 32 >= B) release();
        chunk(r, c0);
      }
    }
    float a0, a1, a2, a3;
    f2_unpack(f2_add(sb_a, sb_b), a0, a1);
    f2_unpack(f2_add(sr_a, sr_b), a2, a3);
    if (pass == 0) sum_b = a0 + a1;
    if (last) sum_r = a2 + a3;
  }
  Lb = mb + fast_log2(sum_b);
  Lr = no_rescue ? Lb : shift_r + fast_log2(sum_r);
}


// The single-pass case of score_tile for the columns [c_begin, c_begin + NC) of the accumulator row only:
// sum_t 2^(x_t + c) and sum_t 2^(x_t + c + gs (||q_t|| - ||q||max)) over those tokens.  The load of each chunk of 16
// columns is in flight while the chunk before it is reduced.
template <int B, int NC>
__device__ __forceinline__ void partial_sums(uint32_t taddr, const float* __restrict__ sD, float gs, float c, bool no_rescue,
                                             int n_tok, int c_begin, float& sum_b, float& sum_r) {
  static_assert(NC % 32 == 0, "chunks are taken in pairs");
  const uint64_t g2 = f2_pack(gs, gs), c2 = f2_pack(c, c);
  uint64_t sb_a = 0ull, sb_b = 0ull, sr_a = 0ull, sr_b = 0ull;
  auto chunk = [&](uint32_t (&r)[16], int c0) {
    if (n_tok < B) {
#pragma unroll
      for (int qq = 0; qq < 16; ++qq)
        if (c0 + qq >= n_tok) r[qq] = 0xff800000u;   // -inf: tokens past the sequence end do not count
    }
#pragma unroll
    for (int j = 0; j < 16; j += 4) {
      const uint64_t e01 = f2_add(f2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), c2);
      const uint64_t e23 = f2_add(f2_pack(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])), c2);
      float e0, e1, e2, e3;
      f2_unpack(e01, e0, e1);
      f2_unpack(e23, e2, e3);
      sb_a = f2_add(sb_a, f2_pack(fast_exp2(e0), fast_exp2(e1)));
      sb_b = f2_add(sb_b, f2_pack(fast_exp2(e2), fast_exp2(e3)));
      if (!no_rescue) {
        const float4 d = *reinterpret_cast<const float4*>(sD + c0 + j);
        float f0, f1, f2, f3;
        f2_unpack(f2_fma(f2_pack(d.x, d.y), g2, e01), f0, f1);
        f2_unpack(f2_fma(f2_pack(d.z, d.w), g2, e23), f2, f3);
        sr_a = f2_add(sr_a, f2_pack(fast_exp2(f0), fast_exp2(f1)));
        sr_b = f2_add(sr_b, f2_pack(fast_exp2(f2), fast_exp2(f3)));
      }
    }
  };
  uint32_t ra[16], rb[16];
  tmem_ld16(taddr + c_begin, ra);
#pragma unroll 1
  for (int c0 = c_begin; c0 < c_begin + NC; c0 += 32) {
    tmem_wait_ld();
    tmem_ld16(taddr + c0 + 16, rb);
    chunk(ra, c0);
    tmem_wait_ld();
    if (c0 + 32 < c_begin + NC) tmem_ld16(taddr + c0 + 32, ra);
    chunk(rb, c0 + 16);
  }
  float a0, a1, a2, a3;
  f2_unpack(f2_add(sb_a, sb_b), a0, a1);
  f2_unpack(f2_add(sr_a, sr_b), a2, a3);
  sum_b = a0 + a1;
  sum_r = a2 + a3;
}

}  // namespace rbs
