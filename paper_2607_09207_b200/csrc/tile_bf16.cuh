// One 64-token tile of the bf16 cache on one warp: scores, online softmax, P.V (warp-level MMAs).
#pragma once

#include "common.cuh"

namespace pdattn {

// ------------------------------------------------------------------------------------------
// One 64-token tile on one warp
// ------------------------------------------------------------------------------------------
// after_k() is called right after the last read of the K tile, before_v() right before the first access to the V
// tile (with split stage halves the caller releases K in the one and waits for V in the other).
template <int D, int NT, int BS, bool TAIL, class AfterK, class BeforeV>
__device__ __forceinline__ void compute_tile(uint32_t sK, uint32_t sV, const uint32_t (&qf)[NT][D / 16][2],
                                             float (&acc)[NT][D / 16][4], float (&m)[NT][2], float (&l)[NT][2],
                                             float sl2, int n_left, uint32_t badmask, int lane,
                                             const int (&lag)[NT][2], AfterK after_k, BeforeV before_v) {
  // n_left: tokens of the sequence from this tile's first one on (>= TILE unless TAIL)
  const int n_valid = n_left < TILE ? n_left : TILE;
  using C = Cfg<D, NT, BS>;
  constexpr int GROUPS = TILE / 16;     // 16-token MMA groups per tile
  const float NEG_INF = __int_as_float(0xff800000);

  // per-lane pieces of the ldmatrix addresses
  const int l8 = lane & 7;
  const int mi = lane >> 3;
  // K (A operand, row-major [token][d]): matrices (tok 0-7,c), (tok 8-15,c), (tok 0-7,c+1), (tok 8-15,c+1)
  const int k_row = l8 + 8 * (mi & 1);
  const int k_csel = mi >> 1;
  // V (A operand = V^T via .trans): matrices (tok 0-7,c), (tok 0-7,c+1), (tok 8-15,c), (tok 8-15,c+1)
  const int v_row = l8 + 8 * (mi >> 1);
  const int v_csel = mi & 1;

  // ---- S^T = K . Q^T : [64 tokens] x [8*NT heads]
  float sc[GROUPS][NT][4];
#pragma unroll
  for (int j = 0; j < GROUPS; ++j) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) sc[j][nt][0] = sc[j][nt][1] = sc[j][nt][2] = sc[j][nt][3] = 0.f;
    if (!TAIL || j * 16 < n_valid) {
      const int page = (j * 16) / BS, row0 = (j * 16) % BS;
      const int row = row0 + k_row;
      const uint32_t base = sK + page * C::PAGE_BYTES + row * 128;
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const int half = kk >> 2;
        const int ch = ((kk & 3) * 2 + k_csel) ^ (row & 7);
        uint32_t a[4];
        ldsm_x4(a, base + half * C::HALF_BYTES + (ch << 4));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16(sc[j][nt], a, qf[nt][kk][0], qf[nt][kk][1]);
      }
    }
  }

  after_k();

  // ---- scale, mask
  const int trow = lane >> 2;
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
          // lag: tokens at the end of the context that this column's query token must not see (it sits
          // that many positions before the last one; 0 for plain decode)
          const int tok = j * 16 + trow + ((r & 2) ? 8 : 0);
          if (tok >= n_left - lag[nt][r & 1]) v = NEG_INF;
        }
        if (dead_page) v = NEG_INF;
        sc[j][nt][r] = v;
      }
  }

  // ---- online softmax: running max per head (2 heads per thread per N tile)
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
  if (__any_sync(0xffffffffu, moved)) {   // the running max rarely moves after the first tiles
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

  // ---- P = exp2(S - m), transposed into the B-operand layout.  bf16 keeps 8 bits of P, which is
  // not enough when a few tokens carry the weight (short contexts, peaked softmax), so P goes
  // to the tensor cores as hi + lo, two bf16 terms (16 bits of significand).
  uint32_t pb[GROUPS][NT][2], pl[GROUPS][NT][2];
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
      const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);
      const uint32_t l01 = pack_bf16x2(p0 - __uint_as_float(h01 << 16), p1 - __uint_as_float(h01 & 0xffff0000u));
      const uint32_t l23 = pack_bf16x2(p2 - __uint_as_float(h23 << 16), p3 - __uint_as_float(h23 & 0xffff0000u));
      pb[j][nt][0] = movmatrix_trans(h01);
      pb[j][nt][1] = movmatrix_trans(h23);
      pl[j][nt][0] = movmatrix_trans(l01);
      pl[j][nt][1] = movmatrix_trans(l23);
    }

  before_v();
  if (TAIL) {
    // Zero the V rows past the last valid token inside its 16-token group: P is 0 there, but
    // 0 * NaN would still poison the accumulator.
    const int g_last = (n_valid - 1) >> 4;
    const int r_beg = n_valid - (g_last << 4);   // 1..16
    const int nrows = 16 - r_beg;
    const int tok0 = (g_last << 4) + r_beg;
    for (int idx = lane; idx < nrows * (D / 8); idx += 32) {
      const int tok = tok0 + idx / (D / 8);
      const int ch = idx % (D / 8);
      const int page = tok / BS, row = tok % BS;
      const uint32_t a = sV + page * C::PAGE_BYTES + (ch >> 3) * C::HALF_BYTES + row * 128 + ((ch & 7) << 4);
      asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
    }
    __syncwarp();
  }

  // ---- O^T += V^T . P^T : [D] x [8*NT heads], K = 64 tokens
#pragma unroll
  for (int j = 0; j < GROUPS; ++j) {
    if (!TAIL || j * 16 < n_valid) {
      const int page = (j * 16) / BS, row0 = (j * 16) % BS;
      const int row = row0 + v_row;
      const uint32_t base = sV + page * C::PAGE_BYTES + row * 128;
#pragma unroll
      for (int jm = 0; jm < D / 16; ++jm) {
        const int half = jm >> 2;
        const int ch = ((jm & 3) * 2 + v_csel) ^ (row & 7);
        uint32_t a[4];
        ldsm_x4_trans(a, base + half * C::HALF_BYTES + (ch << 4));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          mma_bf16(acc[nt][jm], a, pb[j][nt][0], pb[j][nt][1]);
          mma_bf16(acc[nt][jm], a, pl[j][nt][0], pl[j][nt][1]);
        }
      }
    }
  }
}

}  // namespace pdattn
