// decode_kernel: split-KV flash decoding.  One persistent CTA per SM walks a contiguous span of the batch's
// 64-token KV tiles.  Producer warps stream K/V pages from HBM into a shared-memory ring with TMA tensor
// copies (128-byte swizzle, one copy per page-head) signalled through mbarriers; the consumer warps each
// take whole tiles, compute S^T = K.Q^T and O^T += V^T.P^T with tensor-core MMAs (tokens on M, the packed
// GQA query rows of the KV head on N) and keep the online-softmax running max / sum in fp32.  At the end of
// a piece the warps' states are merged either by handing them down a chain of warps (default, no barrier)
// or all at once behind a consumer-wide barrier (template flag CHAIN).
#pragma once

#include "common.cuh"
#include "tile_bf16.cuh"
#include "tile_fp8.cuh"

namespace pdattn {

// ------------------------------------------------------------------------------------------
// Final merge of a cut unit inside the decode kernel.  The span table's merge words tell every warp that writes
// a partial (m, l, acc) of a cut unit which span c the unit starts in and which of the spans after it hold a
// piece.  The warp posts a job to its CTA's merge warp, which publishes the partial device-wide by taking a
// ticket on word c; the merge warp that draws a unit's last ticket -- whichever CTA it belongs to, no one
// waits -- merges all the pieces in ascending token order (the shared-prefix partial first when there is one)
// and writes the output rows.  The order of the sum is fixed by the span table, so the bits do not depend on
// who merges.  merge_cut_unit takes plain values only: a reference to the kernel parameters inside a function
// that is not inlined would turn every access into a generic load.
// ------------------------------------------------------------------------------------------
struct MergeJob {
  const float* partials;      // [span][2][SLOT_FLOATS]
  const float* pfx;           // this unit's shared-prefix partial, or null
  __nv_bfloat16* out;
  int c, hold_mask, n_parts;
  int s, g, G, T, Hq;
};
template <int D, int NT>
__device__ __noinline__ void merge_cut_unit(const MergeJob J, int own_slot, int lane) {
  constexpr int HP = 8 * NT;
  constexpr int SLOT_FLOATS = HP * (D + 2);
  const float NEG_INF = __int_as_float(0xff800000);
  // piece p: -1 the partial of the unit's leading tiles (shared prefix, written by an earlier kernel), 0 the one
  // of span c, p >= 1 the p-th follower that holds tiles; lane p keeps the address of piece p
  const int p0 = J.pfx ? -1 : 0;
  const float* mine = nullptr;
  if (lane == 0) mine = J.partials + (static_cast<int64_t>(J.c) * 2 + own_slot) * SLOT_FLOATS;
  else if (lane < J.n_parts) mine = J.partials + static_cast<int64_t>(J.c + 1 + __fns(J.hold_mask, 0, lane)) * 2 * SLOT_FLOATS;
  auto piece = [&](int p) -> const float* {
    const unsigned long long a = __shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(mine), p < 0 ? 0 : p);
    return p < 0 ? J.pfx : reinterpret_cast<const float*>(a);
  };
  // Pieces are taken two at a time and every load of a pair is issued before anything is computed:
  // one round trip to the L2 per pair, however loaded the memory system is.  Pairs are folded into the
  // running (M, Ls, a) like tiles into an online softmax; the order is fixed by the span table.
  const int R = J.G * J.T;
  constexpr int ITEMS = HP * (D / 4);
  constexpr int IPL = ITEMS / 32;                   // items per lane: item = (row h, four consecutive dims dq)
  constexpr int CH = 2;
  static_assert(ITEMS % 32 == 0 && HP <= 32, "merge layout");
  int h[IPL], dq[IPL];
  float M[IPL], Ls[IPL];
  float4 a[IPL];
#pragma unroll
  for (int j = 0; j < IPL; ++j) {
    const int idx = j * 32 + lane;
    h[j] = idx / (D / 4);
    dq[j] = idx % (D / 4);
    M[j] = NEG_INF;
    Ls[j] = 0.f;
    a[j] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll 1
  for (int pb = p0; pb < J.n_parts; pb += CH) {
    float pm[CH], pl[CH];                           // lane t < HP: m and l of row t of each piece of the group
    float4 v[CH][IPL];
    bool valid[CH];
#pragma unroll
    for (int q = 0; q < CH; ++q) {
      valid[q] = pb + q < J.n_parts;
      const float* part = piece(valid[q] ? pb + q : pb);
      pm[q] = __ldcg(part + (lane % HP));
      pl[q] = __ldcg(part + HP + (lane % HP));
#pragma unroll
      for (int j = 0; j < IPL; ++j) v[q][j] = __ldcg(reinterpret_cast<const float4*>(part + 2 * HP + h[j] * D + dq[j] * 4));
    }
#pragma unroll
    for (int j = 0; j < IPL; ++j) {
      float mq[CH], lq[CH];
      float Mn = M[j];
#pragma unroll
      for (int q = 0; q < CH; ++q) {
        mq[q] = __shfl_sync(0xffffffffu, pm[q], h[j]);
        lq[q] = __shfl_sync(0xffffffffu, pl[q], h[j]);
        if (valid[q]) Mn = fmaxf(Mn, mq[q]);
      }
      const float Mu = (Mn == NEG_INF) ? 0.f : Mn;
      const float fo = fast_exp2(M[j] - Mu);        // 0 for the first group (M = -inf)
      M[j] = Mn;
      Ls[j] *= fo;
      a[j].x *= fo;
      a[j].y *= fo;
      a[j].z *= fo;
      a[j].w *= fo;
#pragma unroll
      for (int q = 0; q < CH; ++q) {
        if (valid[q]) {
          const float f = fast_exp2(mq[q] - Mu);
          Ls[j] += lq[q] * f;
          a[j].x += v[q][j].x * f;
          a[j].y += v[q][j].y * f;
          a[j].z += v[q][j].z * f;
          a[j].w += v[q][j].w * f;
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < IPL; ++j) {
    if (h[j] < R) {   // row h = query token * G + head
      const float inv = Ls[j] > 0.f ? 1.f / Ls[j] : 0.f;
      uint2 o;
      o.x = pack_bf16x2(a[j].x * inv, a[j].y * inv);
      o.y = pack_bf16x2(a[j].z * inv, a[j].w * inv);
      const int qtok = h[j] / J.G;
      *reinterpret_cast<uint2*>(J.out + ((static_cast<int64_t>(J.s) * J.T + qtok) * J.Hq + J.g * J.G + (h[j] - qtok * J.G)) * D +
                                dq[j] * 4) = o;
    }
  }
}

// The merge warp of a CTA: takes the jobs the consumer warps post (one per partial written for a unit that the
// decode kernel merges itself), in order, and runs merge_cut_unit for each.  It is the only warp of the kernel
// that waits on global memory for a merge, and nothing waits for it: while the ring is full a dependent access
// to global memory takes several microseconds (it queues behind the CTA's own bulk copies), which a consumer
// warp cannot afford -- its ring slot would stay occupied.  Ends when every consumer warp has said it is done
// and the queue is empty.  Every wait is bounded.
template <int D, int NT>
__device__ __forceinline__ void merge_warp_loop(const DecodeParams& P, Ctrl* ctrl, int ncw, int lane) {
  constexpr int SLOT_FLOATS = 8 * NT * (D + 2);
  constexpr int BATCH = 4;          // jobs whose tickets are drawn together (one lane each)
  const unsigned long long t_start = globaltimer_ns();
  for (int next = 0;;) {
    bool have = false;
    for (;;) {
      if (ld_acquire_shared(&ctrl->mq_tag[next % MERGE_QUEUE]) == next + 1) {
        have = true;
        break;
      }
      if (ld_acquire_shared(&ctrl->mq_done) == ncw && ld_acquire_shared(&ctrl->mq_head) == next) break;
      if (*reinterpret_cast<volatile uint32_t*>(&ctrl->abort)) break;
      if (globaltimer_ns() - t_start > 4 * kWaitLimitNs) {   // the whole kernel is bounded well below this
        if (lane == 0) atomicOr(&P.hdr->err, ERR_TIMEOUT);
        break;
      }
      __nanosleep(64);
    }
    if (!have) return;
    // every job that is already there, up to BATCH: their round trips to global memory overlap
    int nj = 1;
    while (nj < BATCH && ld_acquire_shared(&ctrl->mq_tag[(next + nj) % MERGE_QUEUE]) == next + nj + 1) ++nj;
    int4 j = make_int4(0, 0, 0, 0);
    if (lane < nj) j = ctrl->mq_job[(next + lane) % MERGE_QUEUE];
    __syncwarp();
    if (lane == 0) st_release_shared(&ctrl->mq_tail, next + nj);   // the entries may be reused
    next += nj;
    // ---- tickets: the partials the consumer warps wrote (made visible to this warp by the queue's release /
    // acquire) are published device-wide before them, the other CTAs' partials are read after them
    int tot = 0;
    if (lane < nj) {
      // release: what this thread has observed so far (the posted partials) is visible device-wide before the
      // ticket; acquire: what the earlier ticket holders published is visible to the loads that follow (the
      // other lanes' loads are ordered behind this one by the warp-wide ballot below)
      asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(tot) : "l"(P.tickets + j.x), "r"(j.z) : "memory");
      tot += j.z;
    }
    const bool last = lane < nj && (tot & 0xffff) == 1 + __popc(j.y);
    if (last) P.tickets[j.x] = 0;                   // everyone has drawn: rearm for the next call
    uint32_t todo = __ballot_sync(0xffffffffu, last);
    while (todo) {
      const int i = __ffs(todo) - 1;
      todo &= todo - 1;
      const int c = __shfl_sync(0xffffffffu, j.x, i), mask = __shfl_sync(0xffffffffu, j.y, i);
      const int uw = __shfl_sync(0xffffffffu, j.w, i), own = __shfl_sync(0xffffffffu, tot, i) >> 16;
      const int unit = uw & 0x3fffffff;
      MergeJob J;
      J.partials = P.partials;
      J.pfx = (uw >> 30) ? P.pfx_partials + static_cast<int64_t>(unit) * SLOT_FLOATS : nullptr;
      J.out = P.out;
      J.c = c;
      J.hold_mask = mask;
      J.n_parts = 1 + __popc(mask);
      J.s = unit / P.Hkv;
      J.g = unit - J.s * P.Hkv;
      J.G = P.G;
      J.T = P.T;
      J.Hq = P.Hq;
      merge_cut_unit<D, NT>(J, own, lane);   // the piece in span c said which of its two slots it used
    }
  }
}

// The tenth warp of the short-piece instantiation (WIN; it never merges cut units itself): it stages the query rows of
// every piece, which is producer warp 0's job elsewhere.  In such batches a piece is a tile or two, the
// consumer warps step over pieces in a few hundred cycles (WindowWalker), and the producer that walked the spans piece
// by piece, staged every piece's rows and issued its third of the tiles set the pace of the CTA.  Walks the same
// spans in the same order as everybody else, 32 units at a time.
template <int D, int NT, int BS, int EB>
__device__ __forceinline__ void stage_queries_loop(const DecodeParams& P, Ctrl* ctrl, uint32_t qbuf, int lane) {
  using C = Cfg<D, NT, BS, EB>;
  const int nunits = P.S * P.Hkv;
  int it = 0, pcnt = 0;
  bool aborted = false;
  int span = blockIdx.x;
  for (int k = 0; span >= 0 && !aborted; ++k) {
    const SpanStart sp = P.use_ws_plan ? P.spans_ws[span] : P.spans[span];
    const int sp_end = P.use_ws_plan ? P.spans_ws[span + 1].flat : P.spans[span + 1].flat;
    WindowWalker walk{P.context_lens, P.start_tiles, P.Hkv, nunits, lane};
    walk.begin_span(sp.unit, sp.tile, sp_end - sp.flat);
    PieceWindow W;
    while (!aborted && walk.next(W, it)) {
      it += W.total;
      uint32_t m = __ballot_sync(0xffffffffu, W.take > 0);
      while (m) {
        const int wl = __ffs(m) - 1;
        m &= m - 1;
        const int unit = __shfl_sync(0xffffffffu, W.unit, wl);
        const int s = __shfl_sync(0xffffffffu, W.s, wl);
        const int g = unit - s * P.Hkv;
        const int qs = pcnt % C::QSLOTS;
        const uint32_t qphase = (pcnt / C::QSLOTS) & 1;
        if (!mbar_wait(smem_u32(&ctrl->q_empty[qs]), qphase ^ 1u)) {
          aborted = true;
          break;
        }
        if (lane == 0) {
          // the G rows of each of the T query tokens, packed: row = query token * G + head
          const uint32_t bytes = static_cast<uint32_t>(P.G) * D * 2;
          const uint32_t qb = smem_u32(&ctrl->q_full[qs]);
          ctrl->qseq[qs] = pcnt;
          mbar_arrive_expect_tx(qb, bytes * P.T);
          for (int qt = 0; qt < P.T; ++qt)
            bulk_load(qbuf + qs * C::Q_BYTES + qt * bytes,
                      P.q + ((static_cast<int64_t>(s) * P.T + qt) * P.Hq + g * P.G) * D, bytes, qb);
        }
        ++pcnt;
      }
    }
    if (aborted) break;
    span = read_span(ctrl, k + 1, aborted);
  }
  if (aborted && lane == 0) {
    atomicOr(&P.hdr->err, ERR_TIMEOUT);
    atomicExch(&ctrl->abort, 1u);
  }
}

// ------------------------------------------------------------------------------------------
// Consumer side of decode_kernel<.., CHAIN = true>: the variant for batches of many short pieces.
//
// Tiles are dealt to the consumer warps exactly as in the default variant (tile i of the CTA to warp
// i mod NCW), but the warps never meet at a barrier.  A piece of n tiles has min(n, NCW) classes
// (class c = the tiles c, c + NCW, ... of the piece, all on one warp).  A piece with one class is
// finished by its warp straight from registers.  Otherwise the running (m, l, acc) travels down the
// chain of classes through a hand-off slot in shared memory: class 0 writes its state, class c
// waits for its turn, folds the slot into its registers and writes the sum back, and the last class
// finishes the piece.  The order of the sum is the class order, whatever the timing.  Hand-off slot
// e serves the pieces with more than one class number e, e + HANDOFFS, ...; its turn word says
// which class of which of those pieces may touch it next.  Warps that hold no tile of a piece skip it
// (they do not even read its query rows), so up to NCW short pieces are in work at once.
// ------------------------------------------------------------------------------------------
template <int D, int NT, int BS, int EB, bool WIN>
__device__ __forceinline__ void consume_chain(const DecodeParams& P, const PlanParams& pp, Ctrl* ctrl, uint32_t ring,
                                              uint32_t qbuf, uint8_t* handoff, int warp, int lane) {
  using C = Cfg<D, NT, BS, EB>;
  constexpr int NST = C::NSTAGES;
  constexpr int NCW = C::NCW;
  constexpr int E = C::HANDOFFS;
  static_assert(E >= 1, "no room for a hand-off slot");
  const float NEG_INF = __int_as_float(0xff800000);
  const int nunits = P.S * P.Hkv;
  const int hq0 = lane >> 2;
  const int qcol = (lane & 3) * 2;
  const int drow = lane >> 2;
  const int R = P.G * P.T;          // query rows per unit: row = query token * G + head
  int lag[NT][2];                   // per score column of this lane: context tokens its query token must not see
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int row = nt * 8 + qcol + e;
      lag[nt][e] = row < R ? P.T - 1 - row / P.G : 0;
    }
  bool aborted = false;
  int it = 0, pcnt = 0, mcnt = 0;

  auto fail = [&]() {
    aborted = true;
    if (lane == 0) {
      atomicOr(&P.hdr->err, ERR_TIMEOUT);
      atomicExch(&ctrl->abort, 1u);
    }
  };

  int span = blockIdx.x;
  for (int k = 0; span >= 0; ++k) {
    const SpanStart sp = P.use_ws_plan ? P.spans_ws[span] : P.spans[span];
    const int sp_end = P.use_ws_plan ? P.spans_ws[span + 1].flat : P.spans[span + 1].flat;
    int first_unit = -1, first_tb = 0, own_unit = -1, own_slot = 0, piece_idx = 0;

    // ---- one piece that this warp holds a tile of (class `pos` of its n_cls classes)
    auto piece_body = [&](const Piece& pc, const int it0, const int p, const int mq, const int slot_idx, const int pos) {
      const int n_piece = pc.te - pc.tb;
      const int n_cls = n_piece < NCW ? n_piece : NCW;
      const bool multi = n_cls > 1;
      const bool complete = (pc.tb == 0 && pc.te == pc.nt);
      if (*reinterpret_cast<volatile uint32_t*>(&ctrl->abort)) {
        aborted = true;
        return;
      }

      // ---- packed query rows of this KV head as MMA B fragments, from the staged copy
      uint32_t qf[NT][D / 16][2];
      {
        const int qs = p % C::QSLOTS;
        if (!wait_q<C::QSLOTS>(ctrl, qs, p)) {
          fail();
          return;
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int head = nt * 8 + hq0;
          const bool live = head < R;
          if constexpr (EB == 2) {
            const uint32_t qa = qbuf + qs * C::Q_BYTES + (live ? head : 0) * (D * 2) + qcol * 2;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              uint32_t v0 = 0u, v1 = 0u;
              if (live) {
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v0) : "r"(qa + kk * 32) : "memory");
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v1) : "r"(qa + kk * 32 + 16) : "memory");
              }
              qf[nt][kk][0] = v0;
              qf[nt][kk][1] = v1;
            }
          } else {
            // fp16 fragments in the permuted order of compute_tile_f8: four consecutive elements per lane
            const uint32_t qa = qbuf + qs * C::Q_BYTES + (live ? head : 0) * (D * 2) + qcol * 4;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              uint32_t v0 = 0u, v1 = 0u;
              if (live) asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v0), "=r"(v1) : "r"(qa + kk * 32) : "memory");
              qf[nt][kk][0] = pack_f16x2(__uint_as_float(v0 << 16), __uint_as_float(v0 & 0xffff0000u));
              qf[nt][kk][1] = pack_f16x2(__uint_as_float(v1 << 16), __uint_as_float(v1 & 0xffff0000u));
            }
          }
        }
        __syncwarp();
        // the slot is free again once every class has its copy: class 0 also arrives for the warps
        // that hold no tile of the piece
        if (lane == 0) mbar_arrive_n(smem_u32(&ctrl->q_empty[qs]), pos == 0 ? NCW - n_cls + 1 : 1);
      }
      float acc[NT][D / 16][4];
      float m[NT][2], l[NT][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        m[nt][0] = m[nt][1] = NEG_INF;
        l[nt][0] = l[nt][1] = 0.f;
#pragma unroll
        for (int jm = 0; jm < D / 16; ++jm) acc[nt][jm][0] = acc[nt][jm][1] = acc[nt][jm][2] = acc[nt][jm][3] = 0.f;
      }

      // fp8 cache: the K scale of this KV head joins the softmax scale
      const float sl2 = EB == 1 ? P.scale_log2 * __ldg(P.k_scale + pc.g) : P.scale_log2;
      (void)sl2;
      // ---- this class's tiles
      for (int its = it0 + pos; its < it0 + n_piece; its += NCW) {
        const int slot = its % NST;
        if (!mbar_wait(smem_u32(&ctrl->full[slot]), (its / NST) & 1)) {
          fail();
          break;
        }
        const int t = pc.tb + (its - it0);
        const uint32_t sK = ring + slot * C::STAGE_BYTES;
        const uint32_t sV = sK + C::KV_BYTES;
        const uint32_t badmask = ctrl->meta[slot];
        const int n_left = pc.L - (pc.t0 + t) * TILE;
        if constexpr (EB == 2) {
          // split stage halves: the K half goes back to the producers as soon as the scores are computed, and
          // the V half is waited for only when the probabilities are ready
          auto after_k = [&]() {
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[slot]));
          };
          auto before_v = [&]() {
            if (!mbar_wait(smem_u32(&ctrl->full_v[slot]), (its / NST) & 1)) fail();
          };
          if (n_left - (P.T - 1) >= TILE) {   // every query token sees the whole tile
            compute_tile<D, NT, BS, false>(sK, sV, qf, acc, m, l, P.scale_log2, TILE, badmask, lane, lag, after_k, before_v);
          } else {
            compute_tile<D, NT, BS, true>(sK, sV, qf, acc, m, l, P.scale_log2, n_left, badmask, lane, lag, after_k, before_v);
            fence_proxy_async();   // our zero-fill stores must be ordered before the next TMA write
          }
          if (aborted) break;
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty_v[slot]));
          continue;
        } else {
          if (n_left - (P.T - 1) >= TILE) {
            compute_tile_f8<D, NT, BS, false>(sK, sV, qf, acc, m, l, sl2, TILE, badmask, lane, lag);
          } else {
            compute_tile_f8<D, NT, BS, true>(sK, sV, qf, acc, m, l, sl2, n_left, badmask, lane, lag);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[slot]));
      }
      if (aborted) return;
      if constexpr (EB == 1) {
        // the V scale of this KV head, once per piece: the accumulator is linear in V
        const float vs = __ldg(P.v_scale + pc.g);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int jm = 0; jm < D / 16; ++jm) {
            acc[nt][jm][0] *= vs;
            acc[nt][jm][1] *= vs;
            acc[nt][jm][2] *= vs;
            acc[nt][jm][3] *= vs;
          }
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          float v = l[nt][e];
          v += __shfl_xor_sync(0xffffffffu, v, 4);
          v += __shfl_xor_sync(0xffffffffu, v, 8);
          v += __shfl_xor_sync(0xffffffffu, v, 16);
          l[nt][e] = v;
        }

      // ---- the chain of classes
      if (multi) {
        const int e = mq % E;
        float4* row4 = reinterpret_cast<float4*>(handoff + e * C::HANDOFF_BYTES) + lane;   // row r: row4[r * 32]
        if (!wait_turn(ctrl, e, mq * 8 + pos)) {
          fail();
          return;
        }
        if (pos > 0) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const float4 ml = row4[nt * 32];
            const float M0 = fmaxf(ml.x, m[nt][0]), M1 = fmaxf(ml.y, m[nt][1]);
            const float mu0 = (M0 == NEG_INF) ? 0.f : M0, mu1 = (M1 == NEG_INF) ? 0.f : M1;
            const float fp0 = fast_exp2(ml.x - mu0), fp1 = fast_exp2(ml.y - mu1);
            const float fo0 = fast_exp2(m[nt][0] - mu0), fo1 = fast_exp2(m[nt][1] - mu1);
            m[nt][0] = M0;
            m[nt][1] = M1;
            l[nt][0] = ml.z * fp0 + l[nt][0] * fo0;
            l[nt][1] = ml.w * fp1 + l[nt][1] * fo1;
#pragma unroll
            for (int jm = 0; jm < D / 16; ++jm) {
              const float4 a = row4[(NT + nt * (D / 16) + jm) * 32];
              acc[nt][jm][0] = a.x * fp0 + acc[nt][jm][0] * fo0;
              acc[nt][jm][1] = a.y * fp1 + acc[nt][jm][1] * fo1;
              acc[nt][jm][2] = a.z * fp0 + acc[nt][jm][2] * fo0;
              acc[nt][jm][3] = a.w * fp1 + acc[nt][jm][3] * fo1;
            }
          }
        }
        if (pos < n_cls - 1) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            row4[nt * 32] = make_float4(m[nt][0], m[nt][1], l[nt][0], l[nt][1]);
#pragma unroll
            for (int jm = 0; jm < D / 16; ++jm)
              row4[(NT + nt * (D / 16) + jm) * 32] =
                  make_float4(acc[nt][jm][0], acc[nt][jm][1], acc[nt][jm][2], acc[nt][jm][3]);
          }
          __syncwarp();
          if (lane == 0) st_release_shared(&ctrl->turn[e], mq * 8 + pos + 1);
          return;
        }
        __syncwarp();   // the last class has read the slot: it now serves merge number mq + E
        if (lane == 0) st_release_shared(&ctrl->turn[e], (mq + E) * 8);
      }

      // ---- finish the piece from registers (one-class piece, or last class of the chain)
      if (complete && pc.t0 > 0) {
        // the unit's leading tiles were handled elsewhere (shared prefix): fold that partial in
        const float* pfx = P.pfx_partials + (static_cast<int64_t>(pc.s) * P.Hkv + pc.g) * C::SLOT_FLOATS;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int h0 = nt * 8 + qcol;
          const float pm0 = pfx[h0], pm1 = pfx[h0 + 1];
          const float M0 = fmaxf(pm0, m[nt][0]), M1 = fmaxf(pm1, m[nt][1]);
          const float mu0 = (M0 == NEG_INF) ? 0.f : M0, mu1 = (M1 == NEG_INF) ? 0.f : M1;
          const float fp0 = fast_exp2(pm0 - mu0), fp1 = fast_exp2(pm1 - mu1);
          const float fo0 = fast_exp2(m[nt][0] - mu0), fo1 = fast_exp2(m[nt][1] - mu1);
          m[nt][0] = M0;
          m[nt][1] = M1;
          l[nt][0] = pfx[C::HP + h0] * fp0 + l[nt][0] * fo0;
          l[nt][1] = pfx[C::HP + h0 + 1] * fp1 + l[nt][1] * fo1;
          const float* pa0 = pfx + 2 * C::HP + h0 * D + drow;
          const float* pa1 = pa0 + D;
#pragma unroll
          for (int jm = 0; jm < D / 16; ++jm) {
            acc[nt][jm][0] = pa0[jm * 16] * fp0 + acc[nt][jm][0] * fo0;
            acc[nt][jm][1] = pa1[jm * 16] * fp1 + acc[nt][jm][1] * fo1;
            acc[nt][jm][2] = pa0[jm * 16 + 8] * fp0 + acc[nt][jm][2] * fo0;
            acc[nt][jm][3] = pa1[jm * 16 + 8] * fp1 + acc[nt][jm][3] * fo1;
          }
        }
      }
      if (complete) {
        // bf16 output; neighbouring lanes swap one value so that each stores two adjacent elements
        const bool odd = drow & 1;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const float inv0 = l[nt][0] > 0.f ? 1.f / l[nt][0] : 0.f;
          const float inv1 = l[nt][1] > 0.f ? 1.f / l[nt][1] : 0.f;
          const int myh = nt * 8 + qcol + (odd ? 1 : 0);     // row = query token * G + head
          const int qtok = myh < R ? myh / P.G : 0;
          __nv_bfloat16* orow = P.out + ((static_cast<int64_t>(pc.s) * P.T + qtok) * P.Hq + pc.g * P.G + (myh - qtok * P.G)) * D +
                                (drow & ~1);
#pragma unroll
          for (int jm = 0; jm < D / 16; ++jm) {
            const float v0 = acc[nt][jm][0] * inv0, v1 = acc[nt][jm][1] * inv1;
            const float v2 = acc[nt][jm][2] * inv0, v3 = acc[nt][jm][3] * inv1;
            const float r0 = __shfl_xor_sync(0xffffffffu, odd ? v0 : v1, 4);
            const float r1 = __shfl_xor_sync(0xffffffffu, odd ? v2 : v3, 4);
            if (myh < R) {
              *reinterpret_cast<uint32_t*>(orow + jm * 16) = odd ? pack_bf16x2(r0, v1) : pack_bf16x2(v0, r0);
              *reinterpret_cast<uint32_t*>(orow + jm * 16 + 8) = odd ? pack_bf16x2(r1, v3) : pack_bf16x2(v2, r1);
            }
          }
        }
      } else {
        float* part = P.partials + (static_cast<int64_t>(span) * 2 + slot_idx) * C::SLOT_FLOATS;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int h0 = nt * 8 + qcol;
          if (drow == 0) {
            part[h0] = m[nt][0];
            part[h0 + 1] = m[nt][1];
            part[C::HP + h0] = l[nt][0];
            part[C::HP + h0 + 1] = l[nt][1];
          }
          float* a0 = part + 2 * C::HP + h0 * D + drow;
          float* a1 = a0 + D;
#pragma unroll
          for (int jm = 0; jm < D / 16; ++jm) {
            a0[jm * 16] = acc[nt][jm][0];
            a1[jm * 16] = acc[nt][jm][1];
            a0[jm * 16 + 8] = acc[nt][jm][2];
            a1[jm * 16 + 8] = acc[nt][jm][3];
          }
        }
        // the unit's last partial to be written triggers its final merge; this warp only posts the job
        if (C::MERGE_WARP && P.inkernel_max > 0) {
          const int back = pc.tb > 0 ? merge_back(sp.merge) : 0;
          if (back != kMergeTooLong) {
            const int c = span - back;
            const int32_t w = back == 0 ? sp.merge : (P.use_ws_plan ? P.spans_ws[c].merge : P.spans[c].merge);
            const int run = merge_run(w);
            if (run >= 1 && run <= P.inkernel_max) {
              __syncwarp();            // every lane's part of the partial is written ...
              if (lane == 0) {
                const int k = atomicAdd(&ctrl->mq_head, 1);
                bool room = k - ld_acquire_shared(&ctrl->mq_tail) < MERGE_QUEUE;
                if (!room) {
                  const unsigned long long t0 = globaltimer_ns();
                  while (!(room = k - ld_acquire_shared(&ctrl->mq_tail) < MERGE_QUEUE))
                    if (*reinterpret_cast<volatile uint32_t*>(&ctrl->abort) || globaltimer_ns() - t0 > kWaitLimitNs) break;
                }
                if (room) {
                  const bool has_pfx = P.start_tiles != nullptr && pc.t0 > 0;
                  ctrl->mq_job[k % MERGE_QUEUE] = make_int4(c, merge_hold_mask(w), 1 + (pc.tb == 0 ? (slot_idx << 16) : 0),
                                                            pc.unit | (has_pfx ? (1 << 30) : 0));
                  st_release_shared(&ctrl->mq_tag[k % MERGE_QUEUE], k + 1);   // ... before the job becomes visible
                } else {
                  atomicOr(&P.hdr->err, ERR_TIMEOUT);
                  atomicExch(&ctrl->abort, 1u);
                }
              }
            }
          }
        }
      }
    };

    if constexpr (WIN) {
      // ---- 32 units at a time: which pieces exist, which are this warp's (see WindowWalker)
      WindowWalker walk{P.context_lens, P.start_tiles, P.Hkv, nunits, lane};
      walk.begin_span(sp.unit, sp.tile, sp_end - sp.flat);
      PieceWindow W;
      while (walk.next(W, it)) {
        const bool has = W.take > 0;
        const int w_ncls = W.take < NCW ? W.take : NCW;
        int w_pos = warp - W.it0 % NCW;
        if (w_pos < 0) w_pos += NCW;
        const uint32_t m_has = __ballot_sync(0xffffffffu, has);
        const uint32_t m_multi = __ballot_sync(0xffffffffu, has && w_ncls > 1);
        uint32_t m_mine = __ballot_sync(0xffffffffu, has && w_pos < w_ncls);
        // the span's record: its first piece, and the unit that starts here and runs past the span's end
        if (piece_idx == 0 && m_has) {
          const int fl = __ffs(m_has) - 1;
          first_unit = __shfl_sync(0xffffffffu, W.unit, fl);
          first_tb = __shfl_sync(0xffffffffu, W.tb, fl);
        }
        const uint32_t m_own = __ballot_sync(0xffffffffu, has && W.tb == 0 && W.take < W.full);
        if (m_own) {
          const int ol = __ffs(m_own) - 1;
          own_unit = __shfl_sync(0xffffffffu, W.unit, ol);
          own_slot = (piece_idx + __popc(m_has & ((1u << ol) - 1u))) == 0 ? 0 : 1;
        }
        const int p_w = pcnt, mq_w = mcnt, pi_w = piece_idx;
        it += W.total;
        pcnt += __popc(m_has);
        mcnt += __popc(m_multi);
        piece_idx += __popc(m_has);
        while (m_mine) {
          const int wl = __ffs(m_mine) - 1;
          m_mine &= m_mine - 1;
          if (aborted) continue;
          const uint32_t below = (1u << wl) - 1u;
          Piece pc;
          pc.unit = __shfl_sync(0xffffffffu, W.unit, wl);
          pc.s = __shfl_sync(0xffffffffu, W.s, wl);
          pc.g = pc.unit - pc.s * P.Hkv;
          pc.L = __shfl_sync(0xffffffffu, W.L, wl);
          pc.t0 = __shfl_sync(0xffffffffu, W.t0, wl);
          pc.nt = __shfl_sync(0xffffffffu, W.full, wl);
          pc.tb = __shfl_sync(0xffffffffu, W.tb, wl);
          pc.te = pc.tb + __shfl_sync(0xffffffffu, W.take, wl);
          const int it0 = __shfl_sync(0xffffffffu, W.it0, wl);
          int pos = warp - it0 % NCW;     // this warp's class in the piece
          if (pos < 0) pos += NCW;
          piece_body(pc, it0, p_w + __popc(m_has & below), mq_w + __popc(m_multi & below),
                     (pi_w + __popc(m_has & below)) == 0 ? 0 : 1, pos);
        }
      }
    } else {
      Walker walk{P.context_lens, P.start_tiles, P.Hkv, nunits, sp.unit, sp.tile, sp_end - sp.flat};
      Piece pc;
      while (walk.next(pc)) {
        const int n_piece = pc.te - pc.tb;
        const int it0 = it;
        it += n_piece;
        const int p = pcnt++;
        const int n_cls = n_piece < NCW ? n_piece : NCW;
        const int mq = mcnt;            // number of this piece among those with more than one class
        if (n_cls > 1) ++mcnt;
        const bool complete = (pc.tb == 0 && pc.te == pc.nt);
        const int slot_idx = piece_idx == 0 ? 0 : 1;
        if (piece_idx == 0) {
          first_unit = pc.unit;
          first_tb = pc.tb;
        }
        if (!complete && pc.tb == 0) {
          own_unit = pc.unit;
          own_slot = slot_idx;
        }
        ++piece_idx;
        int pos = warp - it0 % NCW;     // this warp's class in the piece
        if (pos < 0) pos += NCW;
        if (pos >= n_cls || aborted) continue;
        piece_body(pc, it0, p, mq, slot_idx, pos);
      }
    }
    if (warp == 0 && lane == 0) P.rec[span] = make_int4(first_unit, first_tb, own_unit, own_slot);
    span = read_span(ctrl, k + 1, aborted);
  }
  if (aborted && lane == 0) atomicOr(&P.hdr->err, ERR_TIMEOUT);
  __syncwarp();
  if (C::MERGE_WARP && lane == 0) {
    __threadfence_block();
    atomicAdd(&ctrl->mq_done, 1);     // this warp posts no more merge jobs
  }
}

// ------------------------------------------------------------------------------------------
// The decode kernel.  PROBE = true builds the page-gather ceiling: identical span walk, page-id
// lookups and TMA ring, but the consumers release every tile untouched and nothing is written.
// CHAIN = true replaces the consumers' barrier-and-merge at the end of each piece by the chained
// hand-off of consume_chain (the producers are the same).
// ------------------------------------------------------------------------------------------
// WIN: the instantiation for batches of mostly one-tile pieces (chained merge, 8-row tiles, no in-kernel merge):
// every warp walks the spans 32 units at a time (WindowWalker) and the tenth warp stages the query rows.
template <int D, int NT, int BS, bool PROBE = false, bool CHAIN = false, int EB = 2, bool WIN = false>
__global__ void __launch_bounds__(Cfg<D, NT, BS, EB>::NTHREADS, 1)
decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
              const __grid_constant__ DecodeParams P) {
  using C = Cfg<D, NT, BS, EB>;
  static_assert(EB == 2 || CHAIN, "the fp8 cache path uses the chained merge");
  constexpr int NST = C::NSTAGES;
  constexpr int NCW = C::NCW;
  constexpr int NCT = C::NCT;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const uint32_t ring = raw + pad;                                        // NST stages, 1024-aligned
  const uint32_t qbuf = ring + NST * C::STAGE_BYTES;                       // [QSLOTS][HP][D] bf16
  float* sm_m = reinterpret_cast<float*>(smem + NST * C::STAGE_BYTES + C::QSLOTS * C::Q_BYTES);   // [NCW][HP]
  float* sm_l = sm_m + NCW * C::HP;                                        // [NCW][HP]
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(sm_l + NCW * C::HP);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const float NEG_INF = __int_as_float(0xff800000);

  if (threadIdx.x == 0) {
    for (int i = 0; i < NST; ++i) {
      mbar_init(smem_u32(&ctrl->full[i]), 1);
      mbar_init(smem_u32(&ctrl->empty[i]), 1);
      mbar_init(smem_u32(&ctrl->full_v[i]), 1);
      mbar_init(smem_u32(&ctrl->empty_v[i]), 1);
    }
    ctrl->abort = 0;
    ctrl->sq_pub = 0;
    for (int i = 0; i < 4; ++i) ctrl->prod_last[i] = -1;
    for (int i = 0; i < C::QSLOTS; ++i) {
      mbar_init(smem_u32(&ctrl->q_full[i]), 1);
      mbar_init(smem_u32(&ctrl->q_empty[i]), NCW);
      ctrl->qseq[i] = -1;
    }
    for (int i = 0; i < 8; ++i) ctrl->turn[i] = i * 8;   // slot i first serves merge number i, class 0
    ctrl->mq_head = ctrl->mq_tail = ctrl->mq_done = 0;
    for (int i = 0; i < MERGE_QUEUE; ++i) ctrl->mq_tag[i] = 0;
    fence_mbar_init();
  }
  __syncthreads();

  // This kernel is launched as a programmatic dependent of whatever precedes it on the stream (plan_kernel
  // with a device-side plan, else the previous step's last kernel): its set-up above runs while that kernel
  // drains; nothing in global memory is touched before it has completed and flushed.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const PlanParams pp = P.use_ws_plan ? P.hdr->plan : P.plan;
  const int nunits = P.S * P.Hkv;
  int it = 0;        // tile counter within this CTA: tile `it` uses ring slot it % NST
  int pcnt = 0;      // piece counter within this CTA: piece p's query rows use query slot p % QSLOTS
  bool aborted = false;

  // split stage halves: only where the consumers use them (chained merge over the bf16 cache)
  constexpr bool SPLIT = CHAIN && EB == 2 && !PROBE;
  if (C::MERGE_WARP && warp == NCW + C::NPW) {
    // ================= merge warp =================
    if constexpr (CHAIN && !PROBE && NT == 1) {
      if constexpr (WIN) stage_queries_loop<D, NT, BS, EB>(P, ctrl, qbuf, lane);
      else if (P.inkernel_max > 0) merge_warp_loop<D, NT>(P, ctrl, NCW, lane);
    }
    return;
  }
  if (warp >= NCW) {
    // ================= producer warp(s) =================
    const int pw = warp - NCW;
    constexpr int IDS_PER_BATCH = 32;
    constexpr int TILES_PER_BATCH = IDS_PER_BATCH / C::PAGES;
    constexpr int DRAW_AHEAD = PDATTN_DRAW_AHEAD;
    bool any_bad = false;
    int span = cta;
    for (int k = 0; span >= 0; ++k) {
      const SpanStart sp = P.use_ws_plan ? P.spans_ws[span] : P.spans[span];
      const int sp_end = P.use_ws_plan ? P.spans_ws[span + 1].flat : P.spans[span + 1].flat;
      // The next run-time span is drawn when this span has DRAW_AHEAD tiles left to issue: early enough to hide the
      // atomic's round trip (its result is only consumed after this span's tiles are issued), late enough that a
      // CTA does not sit on a reserved span for the length of a whole span while other CTAs run dry.
      int nxt = -1;
      bool drawn = !(pw == 0 && pp.n_dyn > 0);
      const int draw_at = it + (sp_end - sp.flat) - DRAW_AHEAD;
      auto maybe_draw = [&](int it_now) {
        if (!drawn && it_now >= draw_at) {
          drawn = true;
          if (lane == 0) {
            const int j = atomicAdd(&P.hdr->counter, 1);
            nxt = j < pp.n_dyn ? pp.n_static + j : -1;
          }
        }
      };
      maybe_draw(it);
      // ---- the tiles of one piece that this warp issues (`it`: the CTA's tile counter at the piece's first tile)
      auto issue_piece = [&](const Piece& pc) -> bool {
        const int32_t* row = P.block_table + static_cast<int64_t>(pc.s) * P.MB;
        const int npages = (pc.L + BS - 1) / BS;
        const int pbase = (pc.t0 + pc.tb) * C::PAGES;
        // A context length beyond what the table row can describe: the entries past the row's end are not
        // read (they belong to the next row, or lie past the allocation); their tokens count as a bad page.
        const int nread = min(npages, P.MB);
        auto page_id = [&](int idx) {
          int id = idx < npages ? -1 : 0;
          if (idx < nread) id = __ldg(row + idx);
          return id;
        };
        int ids_cur = page_id(pbase + lane);
        int ids_nxt = page_id(pbase + IDS_PER_BATCH + lane);
        for (int t = pc.tb; t < pc.te; ++t, ++it) {
          const int rel = t - pc.tb;
          const int kb = rel % TILES_PER_BATCH;
          if (kb == 0 && rel != 0) {
            ids_cur = ids_nxt;
            ids_nxt = page_id(pbase + rel * C::PAGES + IDS_PER_BATCH + lane);
          }
          maybe_draw(it);
          if (C::NPW > 1 && it % C::NPW != pw) continue;
          const int slot = it % NST;
          const uint32_t phase = (it / NST) & 1;
          if (NST % C::NPW != 0 && it >= NST) {
            // the slot's previous tile was issued by another producer: make sure it has been, so
            // that the parity wait below refers to that tile's release and not to an older one
            const int prev = it - NST;
            const int32_t* pl = &ctrl->prod_last[prev % C::NPW];
            if (ld_acquire_shared(pl) < prev) {
              const unsigned long long t0 = globaltimer_ns();
              while (ld_acquire_shared(pl) < prev) {
                if (globaltimer_ns() - t0 > kWaitLimitNs) {
                  aborted = true;
                  break;
                }
              }
              if (aborted) return false;
            }
          }
          if (!mbar_wait(smem_u32(&ctrl->empty[slot]), phase ^ 1u)) return false;
          const int np = min(C::PAGES, npages - (pc.t0 + t) * C::PAGES);
          const int j = lane % C::PAGES;
          int id = __shfl_sync(0xffffffffu, ids_cur, kb * C::PAGES + j);
          const bool bad = (lane < C::PAGES) && (j < np) && (id < 0 || id >= P.NB);
          const uint32_t badmask = __ballot_sync(0xffffffffu, bad);
          if (id < 0 || id >= P.NB) id = P.NB;   // out-of-bounds coordinate: TMA fills zeros, nothing is read
          if constexpr (SPLIT) {
            // K half and V half of the stage under their own barriers: the consumers hand the K half back
            // after the scores and the V half after the products
            const uint32_t bar_k = smem_u32(&ctrl->full[slot]);
            if (lane == 0) {
              ctrl->meta[slot] = badmask;
              mbar_arrive_expect_tx(bar_k, static_cast<uint32_t>(np) * C::PAGE_BYTES);
            }
            __syncwarp();
            if (lane < C::PAGES && j < np) {
              const uint32_t dst = ring + slot * C::STAGE_BYTES + j * C::PAGE_BYTES;
              if (P.box5d) {
                tma_load_5d(dst, &tmK, 0, 0, 0, pc.g, id, bar_k);
              } else {
#pragma unroll
                for (int h = 0; h < C::HALVES; ++h) tma_load_4d(dst + h * C::HALF_BYTES, &tmK, h * 64, 0, pc.g, id, bar_k);
              }
            }
            if (!mbar_wait(smem_u32(&ctrl->empty_v[slot]), phase ^ 1u)) return false;
            const uint32_t bar_v = smem_u32(&ctrl->full_v[slot]);
            if (lane == 0) mbar_arrive_expect_tx(bar_v, static_cast<uint32_t>(np) * C::PAGE_BYTES);
            __syncwarp();
            if (lane < C::PAGES && j < np) {
              const uint32_t dst = ring + slot * C::STAGE_BYTES + C::KV_BYTES + j * C::PAGE_BYTES;
              if (P.box5d) {
                tma_load_5d(dst, &tmV, 0, 0, 0, pc.g, id, bar_v);
              } else {
#pragma unroll
                for (int h = 0; h < C::HALVES; ++h) tma_load_4d(dst + h * C::HALF_BYTES, &tmV, h * 64, 0, pc.g, id, bar_v);
              }
            }
          } else {
          const uint32_t bar = smem_u32(&ctrl->full[slot]);
          if (lane == 0) {
            ctrl->meta[slot] = badmask;
            mbar_arrive_expect_tx(bar, static_cast<uint32_t>(np) * 2u * C::PAGE_BYTES);
          }
          __syncwarp();
          if (lane < 2 * C::PAGES && j < np) {
            const bool isV = lane >= C::PAGES;
            const uint32_t dst = ring + slot * C::STAGE_BYTES + (isV ? C::KV_BYTES : 0) + j * C::PAGE_BYTES;
            const CUtensorMap* tm = isV ? &tmV : &tmK;
            if (P.box5d) {
              tma_load_5d(dst, tm, 0, 0, 0, pc.g, id, bar);
            } else {
#pragma unroll
              for (int h = 0; h < C::HALVES; ++h) tma_load_4d(dst + h * C::HALF_BYTES, tm, h * 64, 0, pc.g, id, bar);
            }
          }
          }
          any_bad |= (badmask != 0);
          if (NST % C::NPW != 0) {
            __syncwarp();
            if (lane == 0) st_release_shared(&ctrl->prod_last[pw], it);
          }
        }
        return true;
      };
      if constexpr (WIN) {
        // 32 units at a time (see WindowWalker); the query rows are staged by the tenth warp
        WindowWalker walk{P.context_lens, P.start_tiles, P.Hkv, nunits, lane};
        walk.begin_span(sp.unit, sp.tile, sp_end - sp.flat);
        PieceWindow W;
        while (!aborted && walk.next(W, it)) {
          const int it_end = it + W.total;
          maybe_draw(it_end);
          int first = pw - W.it0 % C::NPW;          // the first tile of the lane's piece that is this warp's
          if (first < 0) first += C::NPW;
          uint32_t m_mine = __ballot_sync(0xffffffffu, W.take > 0 && first < W.take);
          while (m_mine && !aborted) {
            const int wl = __ffs(m_mine) - 1;
            m_mine &= m_mine - 1;
            Piece pc;
            pc.unit = __shfl_sync(0xffffffffu, W.unit, wl);
            pc.s = __shfl_sync(0xffffffffu, W.s, wl);
            pc.g = pc.unit - pc.s * P.Hkv;
            pc.L = __shfl_sync(0xffffffffu, W.L, wl);
            pc.t0 = __shfl_sync(0xffffffffu, W.t0, wl);
            pc.nt = __shfl_sync(0xffffffffu, W.full, wl);
            pc.tb = __shfl_sync(0xffffffffu, W.tb, wl);
            pc.te = pc.tb + __shfl_sync(0xffffffffu, W.take, wl);
            it = __shfl_sync(0xffffffffu, W.it0, wl);
            if (!issue_piece(pc)) aborted = true;
          }
          it = it_end;
        }
      } else {
        Walker walk{P.context_lens, P.start_tiles, P.Hkv, nunits, sp.unit, sp.tile, sp_end - sp.flat};
        Piece pc;
        while (!aborted && walk.next(pc)) {
          if (!PROBE && pw == 0) {
            // stage this piece's packed query rows; the consumers reach the piece several tiles later
            const int qs = pcnt % C::QSLOTS;
            const uint32_t qphase = (pcnt / C::QSLOTS) & 1;
            if (!mbar_wait(smem_u32(&ctrl->q_empty[qs]), qphase ^ 1u)) {
              aborted = true;
              break;
            }
            if (lane == 0) {
              // the G rows of each of the T query tokens, packed: row = query token * G + head
              const uint32_t bytes = static_cast<uint32_t>(P.G) * D * 2;
              const uint32_t qb = smem_u32(&ctrl->q_full[qs]);
              if (CHAIN) ctrl->qseq[qs] = pcnt;
              mbar_arrive_expect_tx(qb, bytes * P.T);
              for (int qt = 0; qt < P.T; ++qt)
                bulk_load(qbuf + qs * C::Q_BYTES + qt * bytes,
                          P.q + ((static_cast<int64_t>(pc.s) * P.T + qt) * P.Hq + pc.g * P.G) * D, bytes, qb);
            }
          }
          ++pcnt;
          if (!issue_piece(pc)) aborted = true;
        }
      }
      if (aborted) break;
      maybe_draw(draw_at);
      if (pw == 0) {
        if (lane == 0) {
          const int slot = k % SPAN_QUEUE;
          ctrl->sq_id[slot] = nxt;
          ctrl->sq_tag[slot] = k + 1;
          st_release_shared(&ctrl->sq_pub, k + 1);
        }
        __syncwarp();
      }
      span = read_span(ctrl, k + 1, aborted);
    }
    if (lane == 0) {
      if (any_bad) atomicOr(&P.hdr->err, ERR_BAD_PAGE);
      if (aborted) {
        atomicOr(&P.hdr->err, ERR_TIMEOUT);
        atomicExch(&ctrl->abort, 1u);
      }
      // this CTA draws no more run-time spans; the last CTA to say so rearms the counter for the next call
      if (pw == 0 && atomicAdd(&P.hdr->done, 1) == static_cast<int>(gridDim.x) - 1) {
        P.hdr->done = 0;
        P.hdr->counter = 0;
      }
    }
    return;
  }

  // ================= consumer warps =================
  const int ct = threadIdx.x;   // 0..NCT-1
  if (!PROBE) {
    // sequences with no context produce zeros
    for (int s = cta; s < P.S; s += gridDim.x) {
      if (__ldg(P.context_lens + s) <= 0) {
        uint32_t* o = reinterpret_cast<uint32_t*>(P.out + static_cast<int64_t>(s) * P.T * P.Hq * D);
        for (int i = ct; i < P.T * P.Hq * D / 2; i += NCT) o[i] = 0u;
      }
    }
  }
  const int hq0 = lane >> 2;         // B-operand column (head) this lane feeds
  const int qcol = (lane & 3) * 2;

  if constexpr (CHAIN) {
    consume_chain<D, NT, BS, EB, WIN>(P, pp, ctrl, ring, qbuf,
                             smem + NST * C::STAGE_BYTES + C::QSLOTS * C::Q_BYTES + C::ML_BYTES + C::CTRL_BYTES, warp,
                             lane);
    return;
  }

  const int R = P.G * P.T;          // query rows per unit: row = query token * G + head
  int lag[NT][2];                   // per score column of this lane: context tokens its query token must not see
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int row = nt * 8 + qcol + e;
      lag[nt][e] = row < R ? P.T - 1 - row / P.G : 0;
    }

  int span = cta;
  for (int k = 0; span >= 0; ++k) {
    const SpanStart sp = P.use_ws_plan ? P.spans_ws[span] : P.spans[span];
    const int sp_end = P.use_ws_plan ? P.spans_ws[span + 1].flat : P.spans[span + 1].flat;
    Walker walk{P.context_lens, P.start_tiles, P.Hkv, nunits, sp.unit, sp.tile, sp_end - sp.flat};
    Piece pc;
    int first_unit = -1, first_tb = 0, own_unit = -1, own_slot = 0, piece_idx = 0;

    while (walk.next(pc)) {
      const int w_first = it % NCW;   // warp that takes this piece's first tile
      // ---- packed query rows of this KV head as MMA B fragments, from the staged copy
      uint32_t qf[NT][D / 16][2];
      if constexpr (!PROBE) {
        const int qs = pcnt % C::QSLOTS;
        const uint32_t qphase = (pcnt / C::QSLOTS) & 1;
        bool have_q = !aborted;
        if (have_q && !mbar_wait(smem_u32(&ctrl->q_full[qs]), qphase)) {
          have_q = false;
          aborted = true;
          if (lane == 0) {
            atomicOr(&P.hdr->err, ERR_TIMEOUT);
            atomicExch(&ctrl->abort, 1u);
          }
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int head = nt * 8 + hq0;
          const bool live = have_q && head < R;
          const uint32_t qa = qbuf + qs * C::Q_BYTES + (live ? head : 0) * (D * 2) + qcol * 2;
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            uint32_t v0 = 0u, v1 = 0u;
            if (live) {
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v0) : "r"(qa + kk * 32) : "memory");
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v1) : "r"(qa + kk * 32 + 16) : "memory");
            }
            qf[nt][kk][0] = v0;
            qf[nt][kk][1] = v1;
          }
        }
        __syncwarp();
        if (have_q && lane == 0) mbar_arrive(smem_u32(&ctrl->q_empty[qs]));
      }
      ++pcnt;
      float acc[NT][D / 16][4];
      float m[NT][2], l[NT][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        m[nt][0] = m[nt][1] = NEG_INF;
        l[nt][0] = l[nt][1] = 0.f;
#pragma unroll
        for (int jm = 0; jm < D / 16; ++jm) acc[nt][jm][0] = acc[nt][jm][1] = acc[nt][jm][2] = acc[nt][jm][3] = 0.f;
      }

      // The slot of the piece's last tile is kept back after it has been consumed: it is where the
      // warps exchange their accumulators for the merge.  Every other slot is released at once, so
      // the producers keep streaming the next piece meanwhile.
      const int n_piece = pc.te - pc.tb;              // tiles in this piece
      const int it_last = it + n_piece - 1;           // ring index of the piece's last tile
      const int park_slot = it_last % NST;
      const int w_last = it_last % NCW;               // the warp that consumes it
      for (int t = pc.tb; t < pc.te; ++t, ++it) {
        if (it % NCW != warp) continue;
        if (!aborted && *reinterpret_cast<volatile uint32_t*>(&ctrl->abort)) aborted = true;
        if (aborted) continue;
        const int slot = it % NST;
        const uint32_t phase = (it / NST) & 1;
        if (!mbar_wait(smem_u32(&ctrl->full[slot]), phase)) {
          aborted = true;
          if (lane == 0) {
            atomicOr(&P.hdr->err, ERR_TIMEOUT);
            atomicExch(&ctrl->abort, 1u);
          }
          continue;
        }
        const uint32_t sK = ring + slot * C::STAGE_BYTES;
        const uint32_t sV = sK + C::KV_BYTES;
        const uint32_t badmask = ctrl->meta[slot];
        const int n_left = pc.L - (pc.t0 + t) * TILE;
        if (PROBE) {
          // ceiling probe: no math
        } else if (n_left - (P.T - 1) >= TILE) {   // every query token sees the whole tile
          compute_tile<D, NT, BS, false>(sK, sV, qf, acc, m, l, P.scale_log2, TILE, badmask, lane, lag, [] {}, [] {});
        } else {
          compute_tile<D, NT, BS, true>(sK, sV, qf, acc, m, l, P.scale_log2, n_left, badmask, lane, lag, [] {}, [] {});
          fence_proxy_async();   // our zero-fill stores must be ordered before the next TMA write
        }
        __syncwarp();
        if ((PROBE || t != pc.te - 1) && lane == 0) mbar_arrive(smem_u32(&ctrl->empty[slot]));
      }

      const bool complete = (pc.tb == 0 && pc.te == pc.nt);
      const int slot_idx = piece_idx == 0 ? 0 : 1;
      if constexpr (!PROBE) {
        // ---- merge the warp states of this piece
        constexpr int ACC_FLOATS = C::HP * C::ACC_STRIDE;                 // one parked accumulator
        constexpr int WPR = C::STAGE_BYTES / (ACC_FLOATS * 4) < NCW ? C::STAGE_BYTES / (ACC_FLOATS * 4) : NCW;
        constexpr int ROUNDS = (NCW + WPR - 1) / WPR;                     // warps are merged WPR at a time
        int pos = warp - w_first;                      // this warp's tiles are residue class `pos` of the piece
        if (pos < 0) pos += NCW;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            float v = l[nt][e];
            v += __shfl_xor_sync(0xffffffffu, v, 4);
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            l[nt][e] = v;
          }
        if (lane < 4) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const int h0 = nt * 8 + qcol;
            sm_m[pos * C::HP + h0] = m[nt][0];
            sm_m[pos * C::HP + h0 + 1] = m[nt][1];
            sm_l[pos * C::HP + h0] = l[nt][0];
            sm_l[pos * C::HP + h0 + 1] = l[nt][1];
          }
        }
        bar_consumers<NCT>();   // the last tile has been consumed: its slot is free for the exchange
        float* park = reinterpret_cast<float*>(smem + park_slot * C::STAGE_BYTES);
        const int n_cls = n_piece < NCW ? n_piece : NCW;   // residue classes that hold tiles
        float* part = P.partials + (static_cast<int64_t>(span) * 2 + slot_idx) * C::SLOT_FLOATS;
        constexpr int ITEMS = C::HP * (D / 4);
        constexpr int IPT = (ITEMS + NCT - 1) / NCT;        // merge items per thread
        float Mu_r[IPT], Ls_r[IPT], M_r[IPT];
        float4 a_r[IPT];
#pragma unroll
        for (int i = 0; i < IPT; ++i) {
          const int idx = ct + i * NCT;
          const int h = (idx < ITEMS ? idx : 0) / (D / 4);
          float M = NEG_INF;
          for (int c = 0; c < n_cls; ++c) M = fmaxf(M, sm_m[c * C::HP + h]);
          // A unit whose leading tiles were handled elsewhere (shared prefix) and whose remaining tiles
          // all lie in this span: fold that partial in here, first in the order, and finish the unit.
          const float* pfx = (complete && pc.t0 > 0)
                                 ? P.pfx_partials + (static_cast<int64_t>(pc.s) * P.Hkv + pc.g) * C::SLOT_FLOATS
                                 : nullptr;
          if (pfx) M = fmaxf(M, pfx[h]);
          M_r[i] = M;
          Mu_r[i] = (M == NEG_INF) ? 0.f : M;
          Ls_r[i] = 0.f;
          a_r[i] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (pfx && idx < ITEMS) {
            const int dq = idx % (D / 4);
            const float f = fast_exp2(pfx[h] - Mu_r[i]);
            Ls_r[i] = pfx[C::HP + h] * f;
            const float4 v = *reinterpret_cast<const float4*>(pfx + 2 * C::HP + h * D + dq * 4);
            a_r[i] = make_float4(v.x * f, v.y * f, v.z * f, v.w * f);
          }
        }
#pragma unroll
        for (int q = 0; q < ROUNDS; ++q) {
          if (pos >= q * WPR && pos < (q + 1) * WPR && pos < n_cls) {
            float* my = park + (pos - q * WPR) * ACC_FLOATS;
            const int drow = lane >> 2;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              const int h0 = nt * 8 + qcol;
#pragma unroll
              for (int jm = 0; jm < D / 16; ++jm) {
                my[h0 * C::ACC_STRIDE + jm * 16 + drow] = acc[nt][jm][0];
                my[(h0 + 1) * C::ACC_STRIDE + jm * 16 + drow] = acc[nt][jm][1];
                my[h0 * C::ACC_STRIDE + jm * 16 + drow + 8] = acc[nt][jm][2];
                my[(h0 + 1) * C::ACC_STRIDE + jm * 16 + drow + 8] = acc[nt][jm][3];
              }
            }
          }
          bar_consumers<NCT>();
          // residue classes in ascending order: the sum does not depend on which warp held which class
#pragma unroll
          for (int i = 0; i < IPT; ++i) {
            const int idx = ct + i * NCT;
            if (idx < ITEMS) {
              const int h = idx / (D / 4);
              const int dq = idx % (D / 4);
              for (int c = q * WPR; c < (q + 1) * WPR && c < n_cls; ++c) {
                const float f = fast_exp2(sm_m[c * C::HP + h] - Mu_r[i]);
                Ls_r[i] += sm_l[c * C::HP + h] * f;
                const float4 v =
                    *reinterpret_cast<const float4*>(park + (c - q * WPR) * ACC_FLOATS + h * C::ACC_STRIDE + dq * 4);
                a_r[i].x += v.x * f;
                a_r[i].y += v.y * f;
                a_r[i].z += v.z * f;
                a_r[i].w += v.w * f;
              }
            }
          }
          bar_consumers<NCT>();   // everyone has read this pass's accumulators
        }
        if (warp == w_last && !aborted) {
          fence_proxy_async();    // our stores into the slot are ordered before the TMA write that refills it
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[park_slot]));
        }
#pragma unroll
        for (int i = 0; i < IPT; ++i) {
          const int idx = ct + i * NCT;
          if (idx < ITEMS) {
            const int h = idx / (D / 4);
            const int dq = idx % (D / 4);
            const float4 a = a_r[i];
            if (complete) {
              if (h < R) {   // row h = query token * G + head
                const float inv = Ls_r[i] > 0.f ? 1.f / Ls_r[i] : 0.f;
                uint2 o;
                o.x = pack_bf16x2(a.x * inv, a.y * inv);
                o.y = pack_bf16x2(a.z * inv, a.w * inv);
                const int qtok = h / P.G;
                *reinterpret_cast<uint2*>(P.out + ((static_cast<int64_t>(pc.s) * P.T + qtok) * P.Hq + pc.g * P.G +
                                                   (h - qtok * P.G)) * D + dq * 4) = o;
              }
            } else {
              if (dq == 0) {
                part[h] = M_r[i];
                part[C::HP + h] = Ls_r[i];
              }
              *reinterpret_cast<float4*>(part + 2 * C::HP + h * D + dq * 4) = a;
            }
          }
        }
      }
      if (piece_idx == 0) {
        first_unit = pc.unit;
        first_tb = pc.tb;
      }
      if (!complete && pc.tb == 0) {
        own_unit = pc.unit;
        own_slot = slot_idx;
      }
      ++piece_idx;
    }
    if (ct == 0 && !PROBE) P.rec[span] = make_int4(first_unit, first_tb, own_unit, own_slot);
    span = read_span(ctrl, k + 1, aborted);
  }
  if (aborted && lane == 0) atomicOr(&P.hdr->err, ERR_TIMEOUT);
}

}  // namespace pdattn
