// One 64-token tile of the fp8 (e4m3) cache on one warp.
#pragma once

#include "common.cuh"

namespace pdattn {

// ------------------------------------------------------------------------------------------
// One 64-token tile on one warp, fp8 cache (e4m3 codes; head_dim D = 128 or 64).
// K tile: [64 tokens][D bytes] (one code per element; 128-byte swizzle at D = 128, 64-byte swizzle at D = 64:
// the 16-byte chunk index is XORed with the row's low three bits, or with bits 1-2 of the row, as the copy
// engine does it); V tile: per page [D][BS tokens]
// (V is stored transposed inside a page; with pages of 32 or 64 tokens the 16-byte rows that ldmatrix
// reads lie 32 or 64 bytes apart and collide two or four ways in the banks).  The codes are widened to fp16 in registers (exact) and both
// products run as fp16 MMAs; Q arrives as fp16 fragments and P is rounded to fp16 (11 bits, one term).
// ldmatrix moves 16-bit units, i.e. PAIRS of codes, so a lane receives four consecutive elements of
// the contraction dimension where the MMA fragment wants two plus two eight further on.  Both
// products therefore run with the contraction index permuted inside every block of 16:
//     k = 2t + i  <->  element 4t + i,     k = 2t + 8 + i  <->  element 4t + 2 + i      (t < 4, i < 2)
// For S^T = K.Q^T the index is the head dimension and the Q fragments are loaded in the same order.
// For O^T = V^T.P^T it is the token: P's rows must come in that order, which they do when row rho of
// the score MMA holds token pi(rho) of its 16-token group -- a matter of the row addresses handed to
// ldmatrix for K.
// ------------------------------------------------------------------------------------------
template <int D, int NT, int BS, bool TAIL>
__device__ __forceinline__ void compute_tile_f8(uint32_t sK, uint32_t sV, const uint32_t (&qf)[NT][D / 16][2],
                                                float (&acc)[NT][D / 16][4], float (&m)[NT][2], float (&l)[NT][2],
                                                float sl2, int n_left, uint32_t badmask, int lane,
                                                const int (&lag)[NT][2]) {
  constexpr int GROUPS = TILE / 16;
  const float NEG_INF = __int_as_float(0xff800000);
  const int n_valid = n_left < TILE ? n_left : TILE;
  const int l8 = lane & 7;
  const int mi = lane >> 3;
  // K: matrices (rows 0-7, chunk c), (rows 8-15, c), (rows 0-7, c+1), (rows 8-15, c+1); row rho <-> token pi(rho)
  const int rho = l8 + 8 * (mi & 1);
  const int k_tok = ((rho & 7) >> 1) * 4 + (rho & 1) + (rho >> 3) * 2;
  const int k_csel = mi >> 1;
  // V^T: matrices (d rows 0-7 of block jm), (8-15 of jm), (0-7 of jm+1), (8-15 of jm+1)
  const int v_drow = (mi >> 1) * 16 + (mi & 1) * 8 + l8;

  float sc[GROUPS][NT][4];
#pragma unroll
  for (int j = 0; j < GROUPS; ++j) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) sc[j][nt][0] = sc[j][nt][1] = sc[j][nt][2] = sc[j][nt][3] = 0.f;
    if (!TAIL || j * 16 < n_valid) {
      const int tok = j * 16 + k_tok;
      const uint32_t base = sK + tok * D;
#pragma unroll
      for (int cc = 0; cc < D / 32; ++cc) {
        const int ch = (cc * 2 + k_csel) ^ (D == 128 ? (tok & 7) : ((tok >> 1) & 3));
        uint32_t r[4];
        ldsm_x4(r, base + (ch << 4));
        {
          const uint32_t a[4] = {cvt_e4m3x2_f16x2(r[0]), cvt_e4m3x2_f16x2(r[1]), cvt_e4m3x2_f16x2(r[0] >> 16),
                                 cvt_e4m3x2_f16x2(r[1] >> 16)};
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) mma_f16(sc[j][nt], a, qf[nt][cc * 2][0], qf[nt][cc * 2][1]);
        }
        {
          const uint32_t a[4] = {cvt_e4m3x2_f16x2(r[2]), cvt_e4m3x2_f16x2(r[3]), cvt_e4m3x2_f16x2(r[2] >> 16),
                                 cvt_e4m3x2_f16x2(r[3] >> 16)};
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) mma_f16(sc[j][nt], a, qf[nt][cc * 2 + 1][0], qf[nt][cc * 2 + 1][1]);
        }
      }
    }
  }

  // ---- scale, mask: score rows g and g + 8 of a group hold tokens pi(g) and pi(g) + 2
  const int trow = lane >> 2;
  const int tok0 = (trow >> 1) * 4 + (trow & 1);
#pragma unroll
  for (int j = 0; j < GROUPS; ++j) {
    bool dead_page = false;
    if (badmask) dead_page = (badmask >> ((j * 16) / BS)) & 1u;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        float v = sc[j][nt][r] * sl2;
        if (TAIL) {
          const int tok = j * 16 + tok0 + ((r & 2) ? 2 : 0);
          if (tok >= n_left - lag[nt][r & 1]) v = NEG_INF;
        }
        if (dead_page) v = NEG_INF;
        sc[j][nt][r] = v;
      }
  }

  // ---- online softmax (as in compute_tile)
  float alpha[NT][2], muse[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      float mx = NEG_INF;
#pragma unroll
      for (int j = 0; j < GROUPS; ++j) mx = fmaxf(mx, fmaxf(sc[j][nt][e], sc[j][nt][e + 2]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
      const float m_new = fmaxf(m[nt][e], mx);
      const float mu = (m_new == NEG_INF) ? 0.f : m_new;
      alpha[nt][e] = fast_exp2(m[nt][e] - mu);
      muse[nt][e] = mu;
      m[nt][e] = m_new;
      l[nt][e] *= alpha[nt][e];
    }
  bool moved = false;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) moved |= (alpha[nt][0] != 1.f) | (alpha[nt][1] != 1.f);
  if (__any_sync(0xffffffffu, moved)) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int jm = 0; jm < D / 16; ++jm) {
        acc[nt][jm][0] *= alpha[nt][0];
        acc[nt][jm][1] *= alpha[nt][1];
        acc[nt][jm][2] *= alpha[nt][0];
        acc[nt][jm][3] *= alpha[nt][1];
      }
  }

  // ---- P = exp2(S - m) as fp16, transposed into the B-operand layout
  uint32_t pb[GROUPS][NT][2];
#pragma unroll
  for (int j = 0; j < GROUPS; ++j)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float p0 = fast_exp2(sc[j][nt][0] - muse[nt][0]);
      const float p1 = fast_exp2(sc[j][nt][1] - muse[nt][1]);
      const float p2 = fast_exp2(sc[j][nt][2] - muse[nt][0]);
      const float p3 = fast_exp2(sc[j][nt][3] - muse[nt][1]);
      l[nt][0] += p0 + p2;
      l[nt][1] += p1 + p3;
      pb[j][nt][0] = movmatrix_trans(pack_f16x2(p0, p1));
      pb[j][nt][1] = movmatrix_trans(pack_f16x2(p2, p3));
    }

  // ---- O^T += V^T . P^T : [D] x [8*NT heads], 16 tokens of a page per MMA step
#pragma unroll
  for (int j = 0; j < GROUPS; ++j) {
    if (!TAIL || j * 16 < n_valid) {
      // codes of tokens past the end may be anything (NaN codes too) while their P is 0: blank them
      uint32_t keep_mask = 0xffffffffu;
      if (TAIL) {
        const int keep = n_valid - (j * 16 + (lane & 3) * 4);   // of this lane's four tokens
        keep_mask = keep >= 4 ? 0xffffffffu : (keep <= 0 ? 0u : ((1u << (8 * keep)) - 1u));
      }
#pragma unroll
      for (int jp = 0; jp < D / 32; ++jp) {
        uint32_t r[4];
        ldsm_x4(r, sV + ((j * 16) / BS) * (D * BS) + (jp * 32 + v_drow) * BS + (j * 16) % BS);
        if (TAIL) {
          r[0] &= keep_mask;
          r[1] &= keep_mask;
          r[2] &= keep_mask;
          r[3] &= keep_mask;
        }
        {
          const uint32_t a[4] = {cvt_e4m3x2_f16x2(r[0]), cvt_e4m3x2_f16x2(r[1]), cvt_e4m3x2_f16x2(r[0] >> 16),
                                 cvt_e4m3x2_f16x2(r[1] >> 16)};
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) mma_f16(acc[nt][jp * 2], a, pb[j][nt][0], pb[j][nt][1]);
        }
        {
          const uint32_t a[4] = {cvt_e4m3x2_f16x2(r[2]), cvt_e4m3x2_f16x2(r[3]), cvt_e4m3x2_f16x2(r[2] >> 16),
                                 cvt_e4m3x2_f16x2(r[3] >> 16)};
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) mma_f16(acc[nt][jp * 2 + 1], a, pb[j][nt][0], pb[j][nt][1]);
        }
      }
    }
  }
}

}  // namespace pdattn
