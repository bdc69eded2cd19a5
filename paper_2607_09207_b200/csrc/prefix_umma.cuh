// Shared-prefix kernel on the 5th-generation tensor cores (tcgen05, accumulators in tensor memory).
//
// The samples of a GRPO group share their prompt pages, so the prompt's K/V tiles are streamed once
// per (group, kv head) and scored against the query rows of all samples: R = group_size * G rows.
// That is the one dense contraction on this path (R = 40 rows against every 64-token tile), and
// with warp-level MMAs it is bound by shared-memory reads and the legacy tensor pipe, not by HBM.
// Here the whole tile is one tensor-core operand:
//
//   S[128 rows, 64 tokens]  = Q[128, d] . K^T          tcgen05.mma, A and B from shared memory
//   O[128 rows, d]         += P[128, 64] . V[64, d]    tcgen05.mma, A = P from tensor memory
//
// Rows R..127 of Q are zeros.  K and V tiles arrive by TMA exactly as in the other kernels (128-byte
// swizzle), laid out per 64-column block as [64 tokens][128 bytes]: K is a K-major B operand of the
// first product, V an MN-major B operand of the second, so V needs no transpose.  Row r lives in
// tensor-memory lane (r mod 4) * 32 + r / 4, which spreads the rows over the four softmax warps (a
// warp can only reach its own quarter of the lanes); one thread owns one row, so the online softmax
// needs no shuffles: it loads the row's 64 scores, updates max and sum, rescales O when the max
// moved, and stores P back to tensor memory as hi + lo bf16 (two MMAs; 8 bits of P are not enough
// under the stated tolerance).  S and P are double buffered so the tensor cores run tile t+1's
// scores while the softmax warps work on tile t.
//
// Warps: 0-3 softmax (128 threads), 4 MMA issue (one elected lane; the warp also owns the tensor
// memory allocation), 5-7 TMA producers.  Every wait is bounded; on expiry the CTA raises
// ERR_TIMEOUT, drains its tensor-core work, frees its tensor memory and returns.
#pragma once

#include "kernels.cuh"

namespace pdattn {

// ---- tcgen05 wrappers ------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t holder_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {   // the mbarrier gets one arrival when all MMAs issued so far are done
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[smem] . B[smem]
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
      : "memory");
}
// D[tmem] (+)= A[tmem] . B[smem]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p; }" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accum)
      : "memory");
}
// 32 consecutive columns of this thread's lane (lane = 32 * (warp % 4) + lane id)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::
          "r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// Shared-memory matrix descriptor for a 128-byte-swizzled operand (descriptor version 1): start
// address, leading-dimension and stride-dimension byte offsets, all in 16-byte units.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return static_cast<uint64_t>((saddr >> 4) & 0x3fffu) | (static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fffu) << 16) |
         (static_cast<uint64_t>((sbo_bytes >> 4) & 0x3fffu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M x N tile, operand majors (0 = K-major, 1 = MN-major).
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(a_mn_major) << 15) |
         (static_cast<uint32_t>(b_mn_major) << 16) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

// Bounded mbarrier wait that also gives up when the CTA's abort flag is up.
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t bar, uint32_t parity, const uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait_hint(bar, parity, PDATTN_WAIT_HINT_NS)) return true;
    if (*reinterpret_cast<const volatile uint32_t*>(abort_flag) || globaltimer_ns() - t0 > kWaitLimitNs) return false;
  }
}


#ifdef PDATTN_TRACE
#define TR_DECL long long tr_t = clock64(); long long tr_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#define TR_MARK(i) { const long long tr_n = clock64(); tr_acc[i] += tr_n - tr_t; tr_t = tr_n; }
#define TR_DUMP(base) if (blockIdx.x == 0 && lane == 0) { for (int tr_i = 0; tr_i < 8; ++tr_i) P.err[(base) + tr_i] = static_cast<int>(tr_acc[tr_i] >> 4); }
#else
#define TR_DECL
#define TR_MARK(i)
#define TR_DUMP(base)
#endif

constexpr int UMMA_ROWS = 128;              // rows of the MMA tile = tensor-memory lanes

template <int D, int BS>
struct UmmaCfg {
  static constexpr int HALVES = D / 64;                     // 64-column (128-byte) blocks per row
  static constexpr int HALF_TILE_BYTES = TILE * 128;        // one block of a K or V tile: [64 tokens][128 B]
  static constexpr int KV_BYTES = HALVES * HALF_TILE_BYTES;
  static constexpr int STAGE_BYTES = 2 * KV_BYTES;          // K tile then V tile
  static constexpr int Q_HALF_BYTES = UMMA_ROWS * 128;      // one block of Q: [128 rows][128 B]
  static constexpr int Q_BYTES = HALVES * Q_HALF_BYTES;
  static constexpr int PAGES = TILE / BS;
  static constexpr int BOX_BYTES = BS * 128;                // one TMA box: a page-head's 64-column block
#ifndef PDATTN_UMMA_ST64
#define PDATTN_UMMA_ST64 12
#endif
  static constexpr int NSTAGES = D == 64 ? PDATTN_UMMA_ST64 : 6;
  static constexpr int NPW = 3;                             // producer warps
  static constexpr int MMA_WARP = 8;                        // warps 0-7: two softmax groups; 8: MMA; 9-11: producers
  static constexpr int NTHREADS = (MMA_WARP + 1 + NPW) * 32;
  static constexpr int CTRL_BYTES = 384;
  static constexpr int ML_BYTES = UMMA_ROWS * 2 * 4;        // (m, l) of group 1's rows, handed to group 0
  static constexpr int DYN_BYTES = 1024 + NSTAGES * STAGE_BYTES + Q_BYTES + ML_BYTES + CTRL_BYTES;
  static constexpr int HP = 8;                              // heads per partial slot (G <= 8)
  static constexpr int SLOT_FLOATS = HP * (D + 2);          // same slots as decode_kernel reads
  // tensor-memory columns: S (2 x 64), P (2 x (hi 32 + lo 32)), O (2 x D)
  static constexpr int COL_S = 0, COL_P = 128, COL_O = 256, TMEM_COLS = 512;
  static_assert(DYN_BYTES <= 232448, "shared memory");
  static_assert(NSTAGES % NPW == 0, "a slot is always refilled by the same producer warp");
  static_assert(COL_O + 2 * D <= TMEM_COLS, "tensor memory");
};

struct UmmaCtrl {
  uint64_t full[12], empty[12];                // ring: TMA landed / tile's MMAs done
  uint64_t s_full[2], p_full[2], pv_done[2];    // per softmax group: scores ready / probabilities stored / O updated
  uint64_t s_free[2];                          // ... and: the group has its scores in registers
  uint64_t q_ready;                            // the unit's query rows are in shared memory
  uint64_t ml_ready;                           // group 1's (m, l) of the unit are in shared memory
  uint64_t o1_free;                            // group 0 has read group 1's accumulator of the unit
  uint64_t unit_done;                          // every P.V of the unit is done
  uint64_t drained;                            // all MMAs of this CTA are done
  uint32_t meta[12];                           // per stage: bit j set = page j of the tile had a bad id
  uint32_t abort;
  uint32_t tmem_base;
};
static_assert(sizeof(UmmaCtrl) <= 384, "control block");

// Tiles alternate between two softmax groups of four warps (tile i of the CTA goes to group i & 1), each
// with its own score / probability buffers and its own accumulator O_g, so two tiles are in work at once
// and a group has two tile times to turn its scores into probabilities.  At the end of a unit group 0
// merges the two states (m, l, O) and writes the partials.
template <int D, int BS>
__global__ void __launch_bounds__(UmmaCfg<D, BS>::NTHREADS, 1)
prefix_umma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                   const __grid_constant__ PrefixParams P) {
  using C = UmmaCfg<D, BS>;
  constexpr int NST = C::NSTAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const uint32_t ring = raw + pad;                                  // NST stages, 1024-aligned
  const uint32_t sQ = ring + NST * C::STAGE_BYTES;
  uint8_t* sQ_ptr = smem + NST * C::STAGE_BYTES;
  float2* sml = reinterpret_cast<float2*>(sQ_ptr + C::Q_BYTES);     // [128] (m, l) of group 1
  UmmaCtrl* ctrl = reinterpret_cast<UmmaCtrl*>(sQ_ptr + C::Q_BYTES + C::ML_BYTES);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const float NEG_INF = __int_as_float(0xff800000);

  if (threadIdx.x == 0) {
    for (int i = 0; i < NST; ++i) {
      mbar_init(smem_u32(&ctrl->full[i]), 1);
      mbar_init(smem_u32(&ctrl->empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&ctrl->s_full[i]), 1);
      mbar_init(smem_u32(&ctrl->p_full[i]), 128);
      mbar_init(smem_u32(&ctrl->pv_done[i]), 1);
      mbar_init(smem_u32(&ctrl->s_free[i]), 128);
    }
    mbar_init(smem_u32(&ctrl->q_ready), 128);
    mbar_init(smem_u32(&ctrl->ml_ready), 128);
    mbar_init(smem_u32(&ctrl->o1_free), 128);
    mbar_init(smem_u32(&ctrl->unit_done), 1);
    mbar_init(smem_u32(&ctrl->drained), 1);
    ctrl->abort = 0;
    fence_mbar_init();
  }
  if (warp < 4) {
    // rows that hold no query stay zero for the whole kernel
    const int lam = warp * 32 + lane;
#pragma unroll
    for (int h = 0; h < C::HALVES; ++h)
#pragma unroll
      for (int c = 0; c < 8; ++c)
        *reinterpret_cast<uint4*>(sQ_ptr + h * C::Q_HALF_BYTES + lam * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
  }
  if (warp == C::MMA_WARP) {
    tmem_alloc(smem_u32(&ctrl->tmem_base), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_base);
  const uint32_t tS = tbase + C::COL_S, tP = tbase + C::COL_P, tO = tbase + C::COL_O;

  // per-sequence start tiles for the decode kernel
  for (int s = cta * blockDim.x + threadIdx.x; s < P.S; s += gridDim.x * blockDim.x)
    P.start_tiles[s] = P.prefix_tiles[s / P.Gs];

  const int2 range = P.ranges[cta];
  const uint32_t* abort_flag = &ctrl->abort;

  if (warp > C::MMA_WARP) {
    // ================= producers: tile i is issued by producer i mod NPW into slot i mod NST
    const int pw = warp - C::MMA_WARP - 1;
    bool any_bad = false, aborted = false;
    int it = 0;
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
        if (it % C::NPW != pw) continue;
        const int slot = it % NST;
        const uint32_t phase = (it / NST) & 1;
        if (!mbar_wait_abortable(smem_u32(&ctrl->empty[slot]), phase ^ 1u, abort_flag)) {
          aborted = true;
          break;
        }
        const int j = lane % C::PAGES;
        int id = __shfl_sync(0xffffffffu, ids_cur, kb * C::PAGES + j);
        const bool bad = (lane < C::PAGES) && (id < 0 || id >= P.NB);
        const uint32_t badmask = __ballot_sync(0xffffffffu, bad);
        if (id < 0 || id >= P.NB) id = P.NB;   // out-of-bounds coordinate: TMA fills zeros, nothing is read
        const uint32_t bar = smem_u32(&ctrl->full[slot]);
        if (lane == 0) {
          ctrl->meta[slot] = badmask;
          mbar_arrive_expect_tx(bar, static_cast<uint32_t>(C::STAGE_BYTES));
        }
        __syncwarp();
        if (lane < 2 * C::PAGES) {
          const bool isV = lane >= C::PAGES;
          const uint32_t dst = ring + slot * C::STAGE_BYTES + (isV ? C::KV_BYTES : 0) + j * C::BOX_BYTES;
          const CUtensorMap* tm = isV ? &tmV : &tmK;
#pragma unroll
          for (int h = 0; h < C::HALVES; ++h) tma_load_4d(dst + h * C::HALF_TILE_BYTES, tm, h * 64, 0, g, id, bar);
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
  } else if (warp == C::MMA_WARP) {
    // ================= MMA issue: one elected lane
    if (lane == 0) {
      constexpr uint32_t ID_S = umma_idesc(UMMA_ROWS, TILE, 0, 0);   // Q (K-major) x K tile (K-major)
      constexpr uint32_t ID_O = umma_idesc(UMMA_ROWS, D, 0, 1);      // P (tensor memory) x V tile (MN-major)
      bool ok = true;
      int it = 0, ucnt = 0;
      TR_DECL
      // Descriptors are built once; per MMA only the start-address field (16-byte units, low bits) moves.
      // The issuing lane is a single thread running dependent code, so every instruction here is on
      // the critical path of the whole CTA.
      const uint64_t q_desc = umma_desc(sQ, 16, 1024);
      const uint64_t k_desc0 = umma_desc(ring, 16, 1024);
      const uint64_t v_desc0 = umma_desc(ring + C::KV_BYTES, C::HALF_TILE_BYTES, 1024);
      // scores of tile i into S[i & 1]
      auto issue_scores = [&](int i) -> bool {
        const int slot = i % NST;
        TR_MARK(3)
        if (!mbar_wait_abortable(smem_u32(&ctrl->full[slot]), (i / NST) & 1, abort_flag)) return false;
        TR_MARK(6)
        tc_fence_after();
        const uint64_t kd = k_desc0 + static_cast<uint64_t>(slot * (C::STAGE_BYTES >> 4));
        const uint32_t d_s = tS + (i & 1) * 64;
#pragma unroll
        for (int h = 0; h < C::HALVES; ++h)
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            umma_ss(d_s, q_desc + static_cast<uint64_t>((h * C::Q_HALF_BYTES + kk * 32) >> 4),
                    kd + static_cast<uint64_t>((h * C::HALF_TILE_BYTES + kk * 32) >> 4), ID_S, (h | kk) ? 1u : 0u);
        tc_commit(smem_u32(&ctrl->s_full[i & 1]));
        return true;
      };
      for (int u = range.x; u < range.y && ok; ++u) {
        const int pt = __ldg(P.prefix_tiles + u / P.Hkv);
        if (pt <= 0) continue;
        TR_MARK(0)
        ok = mbar_wait_abortable(smem_u32(&ctrl->q_ready), ucnt & 1, abort_flag);
        TR_MARK(1)
        ++ucnt;
        for (int t = 0; t < pt && ok; ++t, ++it) {
          const int b = it & 1;
          if (t == 0) {   // one tile for each group to start with
            ok = issue_scores(it);
            if (ok && pt > 1) ok = issue_scores(it + 1);
          }
          // As soon as the group has tile `it`'s scores in registers, its next tile's scores are computed
          // (while the group turns this tile's into probabilities).
          TR_MARK(0)
          if (ok && t + 2 < pt) {
            ok = mbar_wait_abortable(smem_u32(&ctrl->s_free[b]), (it >> 1) & 1, abort_flag);
            TR_MARK(2)
            tc_fence_after();
            if (ok) ok = issue_scores(it + 2);
            TR_MARK(3)
          }
          if (!ok) break;
          ok = mbar_wait_abortable(smem_u32(&ctrl->p_full[b]), (it >> 1) & 1, abort_flag);
          TR_MARK(4)
          if (!ok) break;
          tc_fence_after();
          const int slot = it % NST;
          const uint64_t vd0 = v_desc0 + static_cast<uint64_t>(slot * (C::STAGE_BYTES >> 4));
          const uint32_t d_o = tO + b * D, a_p = tP + b * 64;
          const uint32_t acc0 = t >= 2 ? 1u : 0u;   // the group's first tile of the unit starts its accumulator afresh
#pragma unroll
          for (int ks = 0; ks < TILE / 16; ++ks) {
            const uint64_t vd = vd0 + static_cast<uint64_t>((ks * 2048) >> 4);
            umma_ts(d_o, a_p + ks * 8, vd, ID_O, ks ? 1u : acc0);      // hi part of P
            umma_ts(d_o, a_p + 32 + ks * 8, vd, ID_O, 1u);             // lo part of P
          }
          TR_MARK(5)
          tc_commit(smem_u32(&ctrl->empty[slot]));    // K and V of this tile are free again
          tc_commit(smem_u32(&ctrl->pv_done[b]));
          if (t == pt - 1) tc_commit(smem_u32(&ctrl->unit_done));
          TR_MARK(7)
        }
      }
      TR_DUMP(16)
      if (!ok) {
        atomicOr(P.err, ERR_TIMEOUT);
        atomicExch(&ctrl->abort, 1u);
      }
      // nothing of this CTA may still be running on the tensor cores when the tensor memory goes back
      tc_commit(smem_u32(&ctrl->drained));
      mbar_wait(smem_u32(&ctrl->drained), 0);
    }
    __syncwarp();
  } else {
    // ================= softmax: group wg = warp / 4 takes the tiles i with (i & 1) == wg; in each group the
    // thread (quadrant q = warp % 4, lane) owns query row lane * 4 + q, tensor-memory lane q * 32 + lane
    const int wg = warp >> 2;
    const int qd = warp & 3;
    const int lam = qd * 32 + lane;
    const int r = lane * 4 + qd;
    const int R = P.Gs * P.G;
    const bool valid = r < R;
    const int rj = valid ? r / P.G : 0, rh = valid ? r - rj * P.G : 0;   // sample in the group, head in the KV group
    const uint32_t lane_addr = static_cast<uint32_t>(qd * 32) << 16;
    bool ok = true;
    auto fail = [&]() {
      ok = false;
      if (lane == 0) {
        atomicOr(P.err, ERR_TIMEOUT);
        atomicExch(&ctrl->abort, 1u);
      }
    };
    // warp-uniform wait: the tensor-memory loads and stores below need the whole warp
    auto wait_all = [&](uint64_t* bar, uint32_t parity) {
      return __all_sync(0xffffffffu, mbar_wait_abortable(smem_u32(bar), parity, abort_flag)) != 0;
    };
    // the query rows of unit u into shared memory, 128-byte swizzled like a K-major MMA operand
    auto stage_q = [&](int u) {
      if (valid) {
        const int gi = u / P.Hkv, g = u - gi * P.Hkv;
        const uint4* src = reinterpret_cast<const uint4*>(
            P.q + (static_cast<int64_t>(gi * P.Gs + rj) * P.Hq + g * P.G + rh) * D);
#pragma unroll
        for (int h = 0; h < C::HALVES; ++h)
#pragma unroll
          for (int c = 0; c < 8; ++c)
            *reinterpret_cast<uint4*>(sQ_ptr + h * C::Q_HALF_BYTES + lam * 128 + ((c ^ (lam & 7)) << 4)) =
                __ldg(src + h * 8 + c);
      }
      fence_proxy_async();   // the tensor cores read these rows through the async proxy
      mbar_arrive(smem_u32(&ctrl->q_ready));
    };
    auto next_unit = [&](int u) {
      for (++u; u < range.y; ++u)
        if (__ldg(P.prefix_tiles + u / P.Hkv) > 0) return u;
      return -1;
    };

    int it = 0, ucnt = 0;
    int u = next_unit(range.x - 1);
    if (u >= 0 && wg == 0) stage_q(u);
    TR_DECL
    while (u >= 0 && ok) {
      const int gi = u / P.Hkv, g = u - gi * P.Hkv;
      const int pt = __ldg(P.prefix_tiles + gi);
      float m = NEG_INF, l = 0.f;
      bool first = true;   // this group has not had a tile of the unit yet
      for (int t = 0; t < pt && ok; ++t, ++it) {
        if ((it & 1) != wg) continue;
        TR_MARK(0)
        if (!wait_all(&ctrl->s_full[wg], (it >> 1) & 1)) {
          fail();
          break;
        }
        TR_MARK(1)
        tc_fence_after();
        uint32_t sa[32], sb[32];
        tmem_ld32(tS + wg * 64 + lane_addr, sa);
        tmem_ld32(tS + wg * 64 + 32 + lane_addr, sb);
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(smem_u32(&ctrl->s_free[wg]));   // the score buffer can take this group's next tile
        TR_MARK(2)
        const uint32_t badmask = ctrl->meta[it % NST];
        float mx = NEG_INF;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          float x0 = __uint_as_float(sa[c]) * P.scale_log2, x1 = __uint_as_float(sb[c]) * P.scale_log2;
          if (badmask) {
            if ((badmask >> (c / BS)) & 1u) x0 = NEG_INF;
            if ((badmask >> ((32 + c) / BS)) & 1u) x1 = NEG_INF;
          }
          sa[c] = __float_as_uint(x0);
          sb[c] = __float_as_uint(x1);
          mx = fmaxf(mx, fmaxf(x0, x1));
        }
        // The reference value m only follows the running max when that grew by more than 2^8: P and O may
        // then exceed 1 by that factor (harmless in fp32 / bf16), and the pass over O in tensor memory that a
        // new reference costs becomes rare.  (m, l, O) stay consistent, which is all the merges need.
        const bool grow = first || mx > m + 8.f;
        const float m_new = grow ? fmaxf(m, mx) : m;
        const float mu = (m_new == NEG_INF) ? 0.f : m_new;
        const float alpha = grow ? fast_exp2(m - mu) : 1.f;
        m = m_new;
        TR_MARK(3)
        // this group's previous P.V must be done before its P buffers and its accumulator are touched
        if (it >= 2 && !wait_all(&ctrl->pv_done[wg], ((it - 2) >> 1) & 1)) {
          fail();
          break;
        }
        // ... and group 0 must have read group 1's accumulator of the previous unit
        if (wg == 1 && first && ucnt > 0 && !wait_all(&ctrl->o1_free, (ucnt - 1) & 1)) {
          fail();
          break;
        }
        tc_fence_after();
        TR_MARK(4)
        if (__any_sync(0xffffffffu, !first && alpha != 1.f)) {   // the running max rarely moves after the first tiles
#pragma unroll
          for (int q = 0; q < D / 32; ++q) {
            uint32_t o[32];
            tmem_ld32(tO + wg * D + q * 32 + lane_addr, o);
            tc_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
            tmem_st32(tO + wg * D + q * 32 + lane_addr, o);
          }
        }
        TR_MARK(5)
        // P = exp2(S - m) as hi + lo bf16; column c of a P block holds tokens 2c and 2c + 1
        float ls = 0.f;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t hi[16], lo[16];
#pragma unroll
          for (int c = 0; c < 16; ++c) {
#if defined(PDATTN_ABL) && PDATTN_ABL == 1
            hi[c] = 0x3f803f80u; lo[c] = 0u; ls += 2.f;
#else
            const float p0 = fast_exp2(__uint_as_float(hf ? sb[2 * c] : sa[2 * c]) - mu);
            const float p1 = fast_exp2(__uint_as_float(hf ? sb[2 * c + 1] : sa[2 * c + 1]) - mu);
            ls += p0 + p1;
            const uint32_t h01 = pack_bf16x2(p0, p1);
            hi[c] = h01;
            lo[c] = pack_bf16x2(p0 - __uint_as_float(h01 << 16), p1 - __uint_as_float(h01 & 0xffff0000u));
#endif
          }
          tmem_st16(tP + wg * 64 + hf * 16 + lane_addr, hi);
          tmem_st16(tP + wg * 64 + 32 + hf * 16 + lane_addr, lo);
        }
        l = l * alpha + ls;
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(smem_u32(&ctrl->p_full[wg]));
        TR_MARK(6)
        first = false;
      }
      if (!ok) break;
      // The group that had the unit's last tile has seen its scores: the query rows can make way for the
      // next unit's, whose first scores then run while the epilogue below reads the accumulators.
      const int un = next_unit(u);
      if (((it - 1) & 1) == wg && un >= 0) stage_q(un);
      if (wg == 1) {
        if (first && ucnt > 0 && !wait_all(&ctrl->o1_free, (ucnt - 1) & 1)) {   // no tile here: keep in step all the same
          fail();
          break;
        }
        sml[lam] = make_float2(m, l);
        mbar_arrive(smem_u32(&ctrl->ml_ready));
      } else {
        // (a barrier of its own, one phase per unit: group 0 does not follow every phase of group 1's
        // pv_done, and a parity wait cannot tell two phases apart)
        if (!wait_all(&ctrl->unit_done, ucnt & 1) || !wait_all(&ctrl->ml_ready, ucnt & 1)) {
          fail();
          break;
        }
        tc_fence_after();
        const float2 ml1 = sml[lam];
        const float M = fmaxf(m, ml1.x);
        const float Mu = (M == NEG_INF) ? 0.f : M;
        const bool has0 = m != NEG_INF, has1 = ml1.x != NEG_INF;   // a group without a tile holds stale data
        const float f0 = fast_exp2(m - Mu), f1 = fast_exp2(ml1.x - Mu);
        float* slotp = P.pfx_partials + (static_cast<int64_t>(gi * P.Gs + rj) * P.Hkv + g) * C::SLOT_FLOATS;
        if (valid) {
          slotp[rh] = M;
          slotp[C::HP + rh] = l * f0 + ml1.y * f1;
        }
#pragma unroll
        for (int q = 0; q < D / 32; ++q) {
          uint32_t o0[32], o1[32];
          tmem_ld32(tO + q * 32 + lane_addr, o0);
          tmem_ld32(tO + D + q * 32 + lane_addr, o1);
          tc_wait_ld();
          if (valid) {
            float4* dst = reinterpret_cast<float4*>(slotp + 2 * C::HP + rh * D + q * 32);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              float v[4];
#pragma unroll
              for (int e = 0; e < 4; ++e)
                v[e] = (has0 ? __uint_as_float(o0[4 * c + e]) * f0 : 0.f) + (has1 ? __uint_as_float(o1[4 * c + e]) * f1 : 0.f);
              dst[c] = make_float4(v[0], v[1], v[2], v[3]);
            }
          }
        }
        tc_fence_before();
        mbar_arrive(smem_u32(&ctrl->o1_free));
      }
      ++ucnt;
      u = un;
    }
    if (qd == 0) { TR_MARK(7) TR_DUMP(24 + wg * 8) }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == C::MMA_WARP) tmem_dealloc(tbase, C::TMEM_COLS);
}

}  // namespace pdattn
