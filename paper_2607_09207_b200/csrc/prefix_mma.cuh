// Shared-prefix kernel with warp-level MMAs (the tcgen05 kernel is in prefix_umma.cuh).
#pragma once

#include "common.cuh"
#include "tile_bf16.cuh"
#include "tile_fp8.cuh"

namespace pdattn {

// ------------------------------------------------------------------------------------------
// Shared-prefix kernel (GRPO groups): the samples of a group share their prompt pages, so the
// prompt's K/V tiles are streamed ONCE per (group, kv head) and scored against the query rows of
// all samples: group_size * G rows, eight per consumer warp.  Here every consumer warp works on
// every tile (its own rows), so there is nothing to merge across warps; at the end of a unit each
// warp writes the (m, l, acc) partial of its rows into the per-(sequence, kv head) prefix slots,
// which decode_kernel / combine_kernel fold into the sequence's result.  Units (group * Hkv + kv
// head) are never cut: CTA c takes units [ranges[c].x, ranges[c].y).
// ------------------------------------------------------------------------------------------
constexpr int MAX_PREFIX_ROWS = 8 * (PDATTN_NCW < 6 ? PDATTN_NCW : 6);   // eight query rows per consumer warp
struct PrefixParams {
  const __nv_bfloat16* q;
  const int32_t* block_table;
  const int32_t* prefix_tiles;   // per group
  int32_t* start_tiles;          // per sequence, written here for the decode kernel that follows
  float* pfx_partials;           // [seq][kv head][HP*(D+2)]
  int32_t* err;
  int S, Hq, Hkv, G, Gs, MB, NB;
  float scale_log2;
  int box5d;
  const float* k_scale;          // fp8 cache only (EB = 1): per KV head, value = scale * e4m3 code
  const float* v_scale;
  int2 ranges[160];
};

// EB: bytes per cache element (2 = bf16 through compute_tile, 1 = e4m3 codes through compute_tile_f8)
template <int D, int BS, int EB = 2>
__global__ void __launch_bounds__(Cfg<D, 1, BS, EB>::NTHREADS_BASE, 1)
prefix_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
              const __grid_constant__ PrefixParams P) {
  using C = Cfg<D, 1, BS, EB>;
  constexpr int NST = C::NSTAGES;
  constexpr int NCW = C::NCW;
  static_assert(NST % C::NPW == 0, "a slot is always refilled by the same producer warp");
  static_assert(NCW * 8 >= MAX_PREFIX_ROWS, "rows per CTA");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const uint32_t ring = raw + pad;
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + NST * C::STAGE_BYTES);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const float NEG_INF = __int_as_float(0xff800000);
  if (threadIdx.x == 0) {
    for (int i = 0; i < NST; ++i) {
      mbar_init(smem_u32(&ctrl->full[i]), 1);
      mbar_init(smem_u32(&ctrl->empty[i]), NCW);   // every consumer warp releases every tile
    }
    ctrl->abort = 0;
    fence_mbar_init();
  }
  __syncthreads();
  // per-sequence start tiles for the decode kernel
  for (int s = cta * blockDim.x + threadIdx.x; s < P.S; s += gridDim.x * blockDim.x)
    P.start_tiles[s] = P.prefix_tiles[s / P.Gs];

  const int2 range = P.ranges[cta];
  int it = 0;
  bool aborted = false;

  if (warp >= NCW) {
    // ---- producers
    const int pw = warp - NCW;
    bool any_bad = false;
    for (int u = range.x; u < range.y && !aborted; ++u) {
      const int gi = u / P.Hkv, g = u - gi * P.Hkv;
      const int pt = __ldg(P.prefix_tiles + gi);
      const int32_t* row = P.block_table + static_cast<int64_t>(gi) * P.Gs * P.MB;   // the group's first row
      const int npages = pt * C::PAGES;
      constexpr int TILES_PER_BATCH = 32 / C::PAGES;
      int ids_cur = (lane < npages) ? __ldg(row + lane) : 0;
      int ids_nxt = (32 + lane < npages) ? __ldg(row + 32 + lane) : 0;
      for (int t = 0; t < pt; ++t, ++it) {
        const int kb = t % TILES_PER_BATCH;
        if (kb == 0 && t != 0) {
          ids_cur = ids_nxt;
          const int nb = t * C::PAGES + 32;
          ids_nxt = (nb + lane < npages) ? __ldg(row + nb + lane) : 0;
        }
        if (C::NPW > 1 && it % C::NPW != pw) continue;
        const int slot = it % NST;
        const uint32_t phase = (it / NST) & 1;
        if (!mbar_wait(smem_u32(&ctrl->empty[slot]), phase ^ 1u)) {
          aborted = true;
          break;
        }
        const int j = lane % C::PAGES;
        int id = __shfl_sync(0xffffffffu, ids_cur, kb * C::PAGES + j);
        const bool bad = (lane < C::PAGES) && (id < 0 || id >= P.NB);
        const uint32_t badmask = __ballot_sync(0xffffffffu, bad);
        if (id < 0 || id >= P.NB) id = P.NB;
        const uint32_t bar = smem_u32(&ctrl->full[slot]);
        if (lane == 0) {
          ctrl->meta[slot] = badmask;
          mbar_arrive_expect_tx(bar, static_cast<uint32_t>(C::STAGE_BYTES));
        }
        __syncwarp();
        if (lane < 2 * C::PAGES) {
          const bool isV = lane >= C::PAGES;
          const uint32_t dst = ring + slot * C::STAGE_BYTES + (isV ? C::KV_BYTES : 0) + j * C::PAGE_BYTES;
          const CUtensorMap* tm = isV ? &tmV : &tmK;
          if (P.box5d) {
            tma_load_5d(dst, tm, 0, 0, 0, g, id, bar);
          } else {
#pragma unroll
            for (int h = 0; h < C::HALVES; ++h) tma_load_4d(dst + h * C::HALF_BYTES, tm, h * 64, 0, g, id, bar);
          }
        }
        any_bad |= (badmask != 0);
      }
    }
    if (lane == 0) {
      if (any_bad) atomicOr(P.err, ERR_BAD_PAGE);
      if (aborted) {
        atomicOr(P.err, ERR_TIMEOUT);
        atomicExch(&ctrl->abort, 1u);
      }
    }
    return;
  }

  // ---- consumers: warp w owns query rows [8w, 8w + 8) of the group's group_size * G rows
  const int R = P.Gs * P.G;
  const int no_lag[1][2] = {{0, 0}};
  const int hq0 = lane >> 2;
  const int qcol = (lane & 3) * 2;
  const bool has_rows = warp * 8 < R;
  for (int u = range.x; u < range.y; ++u) {
    const int gi = u / P.Hkv, g = u - gi * P.Hkv;
    const int pt = __ldg(P.prefix_tiles + gi);
    if (pt <= 0) continue;
    const int s0 = gi * P.Gs;
    uint32_t qf[1][D / 16][2];
    {
      const int r = warp * 8 + hq0;
      const bool live = r < R;
      const int j = live ? r / P.G : 0, h = live ? r - j * P.G : 0;
      const uint32_t* qp =
          reinterpret_cast<const uint32_t*>(P.q + (static_cast<int64_t>(s0 + j) * P.Hq + g * P.G + h) * D);
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        if constexpr (EB == 2) {
          qf[0][kk][0] = live ? __ldg(qp + (kk * 16 + qcol) / 2) : 0u;
          qf[0][kk][1] = live ? __ldg(qp + (kk * 16 + 8 + qcol) / 2) : 0u;
        } else {
          // fp16 fragments in the permuted order of compute_tile_f8: four consecutive elements per lane
          const uint32_t v0 = live ? __ldg(qp + (kk * 16 + qcol * 2) / 2) : 0u;
          const uint32_t v1 = live ? __ldg(qp + (kk * 16 + qcol * 2) / 2 + 1) : 0u;
          qf[0][kk][0] = pack_f16x2(__uint_as_float(v0 << 16), __uint_as_float(v0 & 0xffff0000u));
          qf[0][kk][1] = pack_f16x2(__uint_as_float(v1 << 16), __uint_as_float(v1 & 0xffff0000u));
        }
      }
    }
    // fp8 cache: the K scale of this KV head joins the softmax scale
    const float sl2 = EB == 1 ? P.scale_log2 * __ldg(P.k_scale + g) : P.scale_log2;
    float acc[1][D / 16][4];
    float m[1][2] = {{NEG_INF, NEG_INF}}, l[1][2] = {{0.f, 0.f}};
#pragma unroll
    for (int jm = 0; jm < D / 16; ++jm) acc[0][jm][0] = acc[0][jm][1] = acc[0][jm][2] = acc[0][jm][3] = 0.f;
    for (int t = 0; t < pt; ++t, ++it) {
      if (!aborted && *reinterpret_cast<volatile uint32_t*>(&ctrl->abort)) aborted = true;
      if (aborted) continue;
      const int slot = it % NST;
      const uint32_t phase = (it / NST) & 1;
      if (!mbar_wait(smem_u32(&ctrl->full[slot]), phase)) {
        aborted = true;
        if (lane == 0) {
          atomicOr(P.err, ERR_TIMEOUT);
          atomicExch(&ctrl->abort, 1u);
        }
        continue;
      }
      if (has_rows) {
        const uint32_t sK = ring + slot * C::STAGE_BYTES;
        if constexpr (EB == 2)
          compute_tile<D, 1, BS, false>(sK, sK + C::KV_BYTES, qf, acc, m, l, sl2, TILE, ctrl->meta[slot], lane, no_lag, [] {}, [] {});
        else
          compute_tile_f8<D, 1, BS, false>(sK, sK + C::KV_BYTES, qf, acc, m, l, sl2, TILE, ctrl->meta[slot], lane, no_lag);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[slot]));
    }
    if (has_rows && !aborted) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        float v = l[0][e];
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        l[0][e] = v;
      }
      const int drow = lane >> 2;
      const float vs = EB == 1 ? __ldg(P.v_scale + g) : 1.f;   // fp8 cache: the accumulator is linear in V
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int r = warp * 8 + qcol + e;
        if (r < R) {
          const int j = r / P.G, h = r - j * P.G;
          float* slotp = P.pfx_partials + (static_cast<int64_t>(s0 + j) * P.Hkv + g) * C::SLOT_FLOATS;
          if (lane < 4) {
            slotp[h] = m[0][e];
            slotp[C::HP + h] = l[0][e];
          }
          float* a = slotp + 2 * C::HP + h * D;
#pragma unroll
          for (int jm = 0; jm < D / 16; ++jm) {
            a[jm * 16 + drow] = acc[0][jm][e] * vs;
            a[jm * 16 + drow + 8] = acc[0][jm][2 + e] * vs;
          }
        }
      }
    }
  }
  if (aborted && lane == 0) atomicOr(P.err, ERR_TIMEOUT);
}

}  // namespace pdattn
