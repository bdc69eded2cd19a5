// Shared-prefix kernel on the 5th-generation tensor cores (tcgen05, operands and accumulators in tensor memory).
//
// The samples of a GRPO group share their prompt pages, so the prompt's K/V tiles are streamed once
// per (group, kv head) and scored against the query rows of all samples: R = group_size * G rows.
// That is the one dense contraction on this path (R = 40 rows against every 64-token tile), and
// with warp-level MMAs it is bound by shared-memory reads and the legacy tensor pipe, not by HBM.
// Here the whole tile is one tensor-core operand (M = 128 lanes of tensor memory):
//
//   S[128, 64 tokens]  = Q[128, d] . K^T          A = Q from tensor memory, B = K tile from shared memory
//   O[128, d]         += P[128, 64] . V[64, d]    A = P from tensor memory, B = V tile from shared memory
//
// K and V tiles arrive by TMA as in the other kernels (128-byte swizzle), laid out per 64-column block as
// [64 tokens][128 bytes]: K is a K-major B operand of the first product, V an MN-major B operand of the
// second, so V needs no transpose.  Query row r occupies TWO lanes, rho = (r % 2) * 32 + r / 2 and rho + 64,
// with the same Q: both get the same scores, the first lane receives the bf16 head of P and the second
// the bf16 rest (8 bits of P are not enough under the stated tolerance), and ONE product P.V per 16 tokens
// yields the hi part and the lo part of O in the two lane halves while V is read once.
//
// Eight softmax warps in two teams of four.  Team tm takes the tiles whose number has parity tm and owns a
// score buffer, a probability buffer, an accumulator O_tm and a running (m, l) per row, so inside a unit the
// teams never wait for each other and their per-tile chains (barrier wait, tensor-memory load, exponentials,
// tensor-memory store, arrive) overlap; their states are merged at the end of the unit.  Warp w reaches lanes
// 32 * (w % 4) .. + 31 only (a hardware rule); the thread in a row's first lane and the one in its second lane
// both read the row's 64 scores and take the max themselves; each computes half of the row's exponentials and
// hands the other the part that lane stores (64 bytes each way through shared memory, one barrier of the
// team's four warps per tile); the first lane keeps the bf16 heads, the second the rests (both by
// truncation: no conversion instructions).  The scores stay unscaled: the scale enters through the exponent's
// multiply-add, its sign through the staged Q.
// The reference value of the online softmax only follows the running max when that grew by more than 2^8,
// so O in tensor memory is rarely rescaled.
// Two MMA-issuing threads in two warps (scores; P.V), because the tensor cores take an MMA of this size
// only about every 80-100 cycles from its issuing thread; two TMA producer warps.  Scores run two tiles
// ahead of the softmax (one buffer per team); the next unit's query rows are staged by the team that
// meets the unit's last tile, as soon as that tile's scores (the last use of the query buffer) are there.
// Every mbarrier wait is bounded; on expiry the CTA raises ERR_TIMEOUT, its waits fall through, the
// issuing threads drain their tensor-core work, the tensor memory is freed and the CTA returns.
#pragma once

#include <type_traits>

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

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
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
    if (*reinterpret_cast<const volatile uint32_t*>(abort_flag) || globaltimer_ns() - t0 > kWaitLimitNs) return false;
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait_hint(bar, parity, PDATTN_WAIT_HINT_NS)) return true;
  }
}

constexpr int UMMA_ROWS = 128;              // rows of the MMA tile = tensor-memory lanes
constexpr int UMMA_MAX_QUERY_ROWS = 64;     // query rows per unit (group_size * G): each occupies two lanes

template <int D, int BS>
struct UmmaCfg {
  static constexpr int HALVES = D / 64;                     // 64-column (128-byte) blocks per row
  static constexpr int HALF_TILE_BYTES = TILE * 128;        // one block of a K or V tile: [64 tokens][128 B]
  static constexpr int KV_BYTES = HALVES * HALF_TILE_BYTES;
  static constexpr int STAGE_BYTES = 2 * KV_BYTES;          // K tile then V tile
  static constexpr int PAGES = TILE / BS;
  static constexpr int BOX_BYTES = BS * 128;                // one TMA box: a page-head's 64-column block
  static constexpr int NSTAGES = 6;
  static constexpr int NPW = 2;                             // producer warps
  static constexpr int MMA_WARP = 8;                        // warps 0-7: softmax; 8, 9: MMA issue; 10, 11: producers
  static constexpr int NTHREADS = (MMA_WARP + 2 + NPW) * 32;
  static constexpr int CTRL_BYTES = 384;
  static constexpr int XS_BYTES = 6 * 64 * 4;               // the teams' m and the four partial row sums, at the end of a unit
  static constexpr int XP_BYTES = 2 * 64 * 128;             // per team and row: the parts of P the row's two lanes hand each other
  static constexpr int XO_BYTES = 64 * D * 2;               // the second lanes' rows of O as bf16, at the end of a unit
  static constexpr int DYN_BYTES = 1024 + NSTAGES * STAGE_BYTES + XS_BYTES + XO_BYTES + XP_BYTES + CTRL_BYTES;
  static constexpr int HP = 8;                              // heads per partial slot (G <= 8)
  static constexpr int SLOT_FLOATS = HP * (D + 2);          // same slots as decode_kernel reads
  // tensor-memory columns: Q (D/2), S (2 x 64), P (2 x 32), O (2 x D): one score buffer, probability buffer and
  // accumulator per softmax team
  static constexpr int QC = D / 2;                          // columns of a row of Q (two bf16 per column)
  static constexpr int COL_Q = 0, COL_S = QC, COL_P = COL_S + 128, COL_O = COL_P + 64, TMEM_COLS = 512;
  static_assert(DYN_BYTES <= 232448, "shared memory");
  static_assert(NSTAGES % NPW == 0, "a slot is always refilled by the same producer warp");
  static_assert(COL_O + 2 * D <= TMEM_COLS, "tensor memory");
};

struct UmmaCtrl {
  uint64_t full[8], empty[8];                  // ring: TMA landed / tile's MMAs done
  uint64_t s_full[2], s_free[2];               // per score buffer: scores ready / scores are in registers
  uint64_t p_full[2], pv_done[2];              // per probability buffer: stored / consumed and O updated
  uint64_t q_ready;                            // the unit's query rows are in tensor memory
  uint64_t unit_done;                          // every P.V of the unit is done
  uint64_t drained[2];                         // all MMAs of an issuing thread are done
  uint32_t meta[8];                            // per stage: bit j set = page j of the tile had a bad id
  uint32_t abort;
  uint32_t tmem_base;
};
static_assert(sizeof(UmmaCtrl) <= 384, "control block");

// Units of this CTA in order, skipping groups without shared tiles.
struct UnitCursor {
  int u, end, pt, t, i, n;   // unit, end of range, its tiles, tile in unit, tile of the CTA, unit ordinal
  const int32_t* prefix_tiles;
  int Hkv;
  __device__ __forceinline__ void seek() {
    while (u < end && (pt = __ldg(prefix_tiles + u / Hkv)) <= 0) ++u;
  }
  __device__ __forceinline__ bool valid() const { return u < end; }
  __device__ __forceinline__ void next_tile() {
    ++i;
    if (++t == pt) {
      t = 0;
      ++n;
      ++u;
      seek();
    }
  }
};

// The kernel (see the head of this file for the design).  Units = (group, kv head) with shared tiles, a
// contiguous range per CTA; the result of a unit is the partial (m, l, acc) of each of its query rows in
// the per-(sequence, kv head) prefix slots that decode_kernel and combine_kernel fold in.
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
  float* xs = reinterpret_cast<float*>(smem + NST * C::STAGE_BYTES);   // [m | l first lanes | l second lanes][2 teams][64 rows]
  float* xo = xs + 6 * 64;                                          // [64 rows][D] bf16
  uint4* xp = reinterpret_cast<uint4*>(smem + NST * C::STAGE_BYTES + C::XS_BYTES + C::XO_BYTES);   // [2 teams][64 rows][8]
  UmmaCtrl* ctrl = reinterpret_cast<UmmaCtrl*>(smem + NST * C::STAGE_BYTES + C::XS_BYTES + C::XO_BYTES + C::XP_BYTES);
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
      mbar_init(smem_u32(&ctrl->s_free[i]), 128);
      mbar_init(smem_u32(&ctrl->p_full[i]), 128);
      mbar_init(smem_u32(&ctrl->pv_done[i]), 1);
    }
    mbar_init(smem_u32(&ctrl->q_ready), 128);
    mbar_init(smem_u32(&ctrl->unit_done), 1);
    mbar_init(smem_u32(&ctrl->drained[0]), 1);
    mbar_init(smem_u32(&ctrl->drained[1]), 1);
    ctrl->abort = 0;
    fence_mbar_init();
  }
  if (warp == C::MMA_WARP) {
    tmem_alloc(smem_u32(&ctrl->tmem_base), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_base);
  const uint32_t tQ = tbase + C::COL_Q, tS = tbase + C::COL_S, tP = tbase + C::COL_P, tO = tbase + C::COL_O;

  // per-sequence start tiles for the decode kernel
  for (int s = cta * blockDim.x + threadIdx.x; s < P.S; s += gridDim.x * blockDim.x)
    P.start_tiles[s] = P.prefix_tiles[s / P.Gs];

  const int2 range = P.ranges[cta];
  const uint32_t* abort_flag = &ctrl->abort;

  if (warp > C::MMA_WARP + 1) {
    // ================= producers: tile i is issued by producer i mod NPW into slot i mod NST
    const int pw = warp - C::MMA_WARP - 2;
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
  } else if (warp >= C::MMA_WARP) {
    // ================= MMA issue.  The tensor cores take an MMA of this size about every 80-100 cycles from
    // the issuing thread, which runs dependent code; with sixteen and more MMAs, three commits and four waits
    // per tile one thread would be the bottleneck of the CTA, so the score products (this warp) and the
    // P.V products (the next warp) are issued by two threads.  They meet only through the barriers.
    if (lane == 0) {
      bool ok = true;
      if (warp == C::MMA_WARP) {
        constexpr uint32_t ID_S = umma_idesc(UMMA_ROWS, TILE, 0, 0);   // Q (tensor memory) x K tile (K-major)
        // the descriptor is built once; per MMA only the start-address field (16-byte units, low bits) moves
        const uint64_t k_desc0 = umma_desc(ring, 16, 1024);
        UnitCursor sc{range.x, range.y, 0, 0, 0, 0, P.prefix_tiles, P.Hkv};
        sc.seek();
        int slot = 0;
        uint32_t ring_phase = 0;
        while (sc.valid() && ok) {
          const int b = sc.i & 1;
          // score buffer b is free when the softmax threads have tile i - 2 in registers
          if (sc.i >= 2) ok = mbar_wait_abortable(smem_u32(&ctrl->s_free[b]), ((sc.i - 2) >> 1) & 1, abort_flag);
          if (ok && sc.t == 0) ok = mbar_wait_abortable(smem_u32(&ctrl->q_ready), sc.n & 1, abort_flag);
          if (ok) ok = mbar_wait_abortable(smem_u32(&ctrl->full[slot]), ring_phase, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint64_t kd = k_desc0 + static_cast<uint64_t>(slot * (C::STAGE_BYTES >> 4));
          const uint32_t d_s = tS + b * 64, a_q = tQ;
#pragma unroll
          for (int h = 0; h < C::HALVES; ++h)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_ts(d_s, a_q + h * 32 + kk * 8, kd + static_cast<uint64_t>((h * C::HALF_TILE_BYTES + kk * 32) >> 4),
                      ID_S, (h | kk) ? 1u : 0u);
          tc_commit(smem_u32(&ctrl->s_full[b]));
          sc.next_tile();
          if (++slot == NST) {
            slot = 0;
            ring_phase ^= 1u;
          }
        }
      } else {
        constexpr uint32_t ID_O = umma_idesc(UMMA_ROWS, D, 0, 1);      // P (tensor memory) x V tile (MN-major)
        const uint64_t v_desc0 = umma_desc(ring + C::KV_BYTES, C::HALF_TILE_BYTES, 1024);
        UnitCursor pc{range.x, range.y, 0, 0, 0, 0, P.prefix_tiles, P.Hkv};
        pc.seek();
        int slot = 0;
        while (pc.valid() && ok) {
          const int b = pc.i & 1;
          // (the tile has landed: the softmax threads saw its scores before they stored these probabilities)
          ok = mbar_wait_abortable(smem_u32(&ctrl->p_full[b]), (pc.i >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint64_t vd0 = v_desc0 + static_cast<uint64_t>(slot * (C::STAGE_BYTES >> 4));
          const uint32_t a_p = tP + b * 32;
          const uint32_t acc0 = pc.t > 1 ? 1u : 0u;   // a team's first tile of the unit starts its accumulator afresh
#pragma unroll
          for (int ks = 0; ks < TILE / 16; ++ks)
            umma_ts(tO + b * D, a_p + ks * 8, vd0 + static_cast<uint64_t>((ks * 2048) >> 4), ID_O, ks ? 1u : acc0);
          tc_commit(smem_u32(&ctrl->empty[slot]));    // K and V of this tile are free again (its scores are long done)
          tc_commit(smem_u32(&ctrl->pv_done[b]));
          if (pc.t == pc.pt - 1) tc_commit(smem_u32(&ctrl->unit_done));
          pc.next_tile();
          if (++slot == NST) slot = 0;
        }
      }
      if (!ok) {
        atomicOr(P.err, ERR_TIMEOUT);
        atomicExch(&ctrl->abort, 1u);
      }
      // nothing of this thread may still be running on the tensor cores when the tensor memory goes back
      const uint32_t dbar = smem_u32(&ctrl->drained[warp - C::MMA_WARP]);
      tc_commit(dbar);
      mbar_wait(dbar, 0);
    }
    __syncwarp();
  } else {
    // ================= softmax: two teams of four warps; team tm works on the tiles with (tile number & 1) == tm,
    // with its own score buffer, probability buffer, accumulator O_tm and running (m, l) per row, so the two
    // teams never wait for each other inside a unit and their per-tile chains of latencies (barrier wait,
    // tensor-memory load, exponentials, tensor-memory store, arrive) overlap.  Warp w reaches tensor-memory
    // lanes 32 * (w % 4) .. + 31; a row's first lane takes the bf16 heads of P, its second lane the rests, and
    // both compute the row's 64 probabilities themselves from the same scores (no exchange inside a tile).
    // The teams' states are merged at the end of a unit.  No thread leaves this path early: all meet at the
    // unit's barriers, so after a failed wait a thread carries on (its waits then return at once).
    const int qd = warp & 3;
    const int tm = warp >> 2;             // team
    const bool is_lo = (qd >> 1) != 0;    // second lane of the row: rests of P, lo part of O
    const int rho = (qd & 1) * 32 + lane; // row slot
    const int r = (rho & 31) * 2 + (rho >> 5);
    const int R = P.Gs * P.G;
    const bool valid = r < R;
    const int rj = valid ? r / P.G : 0, rh = valid ? r - rj * P.G : 0;   // sample in the group, head in the KV group
    const uint32_t lane_addr = static_cast<uint32_t>(qd * 32) << 16;
    const uint32_t tOt = tO + tm * D;     // this team's accumulator
    // the scores stay unscaled in registers (the scale is applied inside the exponent's multiply-add), so it
    // must not be negative: its sign goes into the staged query rows
    // (never exactly zero, so that a masked score, minus infinity, stays that under the multiply-add; a scale this
    // small gives the same probabilities as zero)
    const float sc = fmaxf(fabsf(P.scale_log2), 1e-30f);
    const uint32_t qflip = P.scale_log2 < 0.f ? 0x80008000u : 0u;
    auto wait_all = [&](uint64_t* bar, uint32_t parity) {   // warp-uniform: tensor-memory accesses need the whole warp
      if (!__all_sync(0xffffffffu, mbar_wait_abortable(smem_u32(bar), parity, abort_flag)) && lane == 0) {
        atomicOr(P.err, ERR_TIMEOUT);
        atomicExch(&ctrl->abort, 1u);
      }
    };
    auto all_barrier = [&]() { asm volatile("bar.sync 5, 256;" ::: "memory"); };
    auto team_barrier = [&]() { asm volatile("bar.sync %0, 128;" ::"r"(1 + tm) : "memory"); };
    auto q_row = [&](int u) {
      const int gi = u / P.Hkv, g = u - gi * P.Hkv;
      return P.q + (static_cast<int64_t>(gi * P.Gs + rj) * P.Hq + g * P.G + rh) * D;
    };
    // this thread's query row of unit u into the (single) query buffer, two bf16 per column; the caller knows
    // that every score product of the buffer's previous unit is done
    auto stage_q = [&](int u, int n) {
      uint32_t qv[C::QC];      // all loads first: under this kernel's own traffic even an L2 hit takes about a microsecond
#pragma unroll
      for (int c = 0; c < C::QC; ++c) qv[c] = 0u;
      if (valid) {
        const uint4* src = reinterpret_cast<const uint4*>(q_row(u));
#pragma unroll
        for (int c = 0; c < C::QC / 4; ++c) {
          const uint4 v = __ldg(src + c);
          qv[4 * c] = v.x ^ qflip;
          qv[4 * c + 1] = v.y ^ qflip;
          qv[4 * c + 2] = v.z ^ qflip;
          qv[4 * c + 3] = v.w ^ qflip;
        }
      }
#pragma unroll
      for (int c0 = 0; c0 < C::QC; c0 += 32) tmem_st32(tQ + c0 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(qv + c0));
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&ctrl->q_ready));
      (void)n;
    };

    UnitCursor uc{range.x, range.y, 0, 0, 0, 0, P.prefix_tiles, P.Hkv};
    uc.seek();
    if (uc.valid() && tm == 0) stage_q(uc.u, 0);
    float m = NEG_INF, l = 0.f;
    while (uc.valid()) {
      const int it = uc.i, t = uc.t, pt = uc.pt, n = uc.n, u = uc.u;
      UnitCursor nu = uc;      // where the cursor goes after this tile
      nu.next_tile();
      const bool last = t == pt - 1;
      if ((it & 1) == tm) {
        if (t < 2) {           // this team's first tile of the unit
          m = NEG_INF;
          l = 0.f;
          // the next unit's query rows towards L2, a whole unit before they are staged (under this kernel's own
          // traffic a load from DRAM takes several tiles' time)
          UnitCursor fu = uc;
          fu.t = pt - 1;
          fu.next_tile();
          if (fu.valid() && valid) asm volatile("prefetch.global.L2 [%0];" ::"l"(q_row(fu.u) + (is_lo ? D / 2 : 0)));
        }
        uint32_t sv[64];
        wait_all(&ctrl->s_full[tm], (it >> 1) & 1);
        tc_fence_after();
        tmem_ld32(tS + tm * 64 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(sv));
        tmem_ld32(tS + tm * 64 + 32 + lane_addr, *reinterpret_cast<uint32_t(*)[32]>(sv + 32));
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(smem_u32(&ctrl->s_free[tm]));   // the score buffer can take tile it + 2
        const uint32_t badmask = ctrl->meta[it % NST];
        if (badmask) {
#pragma unroll
          for (int k = 0; k < 64; ++k)
            if ((badmask >> (k / BS)) & 1u) sv[k] = __float_as_uint(NEG_INF);
        }
        // the row max of the raw scores, four independent chains of three-input max (the scale is not negative:
        // its sign went into the staged query rows)
        float m4[4] = {NEG_INF, NEG_INF, NEG_INF, NEG_INF};
#pragma unroll
        for (int k = 0; k < 64; k += 2)
          m4[(k >> 1) & 3] = max3(m4[(k >> 1) & 3], __uint_as_float(sv[k]), __uint_as_float(sv[k + 1]));
        const float mr = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        const float mx = (mr == NEG_INF) ? NEG_INF : mr * sc;
        // The reference value m only follows the running max when that grew by more than 2^8: P and O may
        // then exceed 1 by that factor (harmless in fp32 / bf16), and the pass over O in tensor memory that a
        // new reference costs becomes rare.  (m, l, O) stay consistent, which is all the merges need.
        const bool grow = t < 2 || mx > m + 8.f;
        const float m_new = grow ? fmaxf(m, mx) : m;
        const float mu = (m_new == NEG_INF) ? 0.f : m_new;
        const float alpha = grow ? fast_exp2(m - mu) : 1.f;
        m = m_new;
        // the product that read this team's probability buffer two tiles ago must be done; it is also the
        // latest product into this team's accumulator, and every thread of the team stored those probabilities
        // after it had read the exchange area below, which is therefore free again
        if (it >= 2) wait_all(&ctrl->pv_done[tm], ((it - 2) >> 1) & 1);
        // P = exp2(S * scale - m), split by truncation into a bf16 head (the row's first lane stores the heads)
        // and the bf16 head of what is left (its second lane stores those rests): 16 bits of P between them, and
        // no conversion instructions.  Each lane computes half of the row's exponentials -- the first lane tokens
        // 0-31, the second 32-63 -- and hands the other lane the part that lane stores, 64 bytes each way through
        // shared memory behind a barrier of the team's four warps.  A P column holds two tokens.
        uint32_t pk[32];
        float ls = 0.f, ls1 = 0.f;
        uint4* xq = xp + (tm * 64 + rho) * 8;      // this row's eight 16-byte chunks: rests of tokens 0-31, heads of 32-63
        auto head_and_rest = [&](int k0, int k, uint32_t& head, uint32_t& rest) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(sv[k0 + 2 * k]), sc, -mu));
          const float p1 = fast_exp2(fmaf(__uint_as_float(sv[k0 + 2 * k + 1]), sc, -mu));
          ls += p0;
          ls1 += p1;
          const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
          head = __byte_perm(b0, b1, 0x7632);
          const float r0 = p0 - __uint_as_float(b0 & 0xffff0000u), r1 = p1 - __uint_as_float(b1 & 0xffff0000u);
          rest = __byte_perm(__float_as_uint(r0), __float_as_uint(r1), 0x7632);
        };
        if (!is_lo) {
          uint32_t give[16];
#pragma unroll
          for (int k = 0; k < 16; ++k) head_and_rest(0, k, pk[k], give[k]);
#pragma unroll
          for (int c = 0; c < 4; ++c) xq[c ^ (rho & 7)] = make_uint4(give[4 * c], give[4 * c + 1], give[4 * c + 2], give[4 * c + 3]);
          team_barrier();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint4 w = xq[(4 + c) ^ (rho & 7)];
            pk[16 + 4 * c] = w.x;
            pk[16 + 4 * c + 1] = w.y;
            pk[16 + 4 * c + 2] = w.z;
            pk[16 + 4 * c + 3] = w.w;
          }
        } else {
          uint32_t give[16];
#pragma unroll
          for (int k = 0; k < 16; ++k) head_and_rest(32, k, give[k], pk[16 + k]);
#pragma unroll
          for (int c = 0; c < 4; ++c) xq[(4 + c) ^ (rho & 7)] = make_uint4(give[4 * c], give[4 * c + 1], give[4 * c + 2], give[4 * c + 3]);
          team_barrier();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint4 w = xq[c ^ (rho & 7)];
            pk[4 * c] = w.x;
            pk[4 * c + 1] = w.y;
            pk[4 * c + 2] = w.z;
            pk[4 * c + 3] = w.w;
          }
        }
        l = l * alpha + (ls + ls1);     // this lane's half of the row sum
        if (__any_sync(0xffffffffu, t >= 2 && alpha != 1.f)) {
          // new reference: scale this lane's row of O (rare: kept small rather than fast)
          tc_fence_after();
#pragma unroll 1
          for (int q = 0; q < D / 32; ++q) {
            uint32_t o[32];
            tmem_ld32(tOt + q * 32 + lane_addr, o);
            tc_wait_ld();
#pragma unroll
            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
            tmem_st32(tOt + q * 32 + lane_addr, o);
          }
        }
        tc_fence_after();
        tmem_st32(tP + tm * 32 + lane_addr, pk);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(smem_u32(&ctrl->p_full[tm]));
      }
      if (last) {
        // ---- the unit's result.  Four threads hold parts of a row: (team 0 | team 1) x (first lane | second lane),
        // each team with its own reference max.  A thread reaches both teams' accumulators in its own lane, so
        // only the second lanes' sums cross lanes (through shared memory, as bf16: they are 2^-8 of the first
        // lanes').  Each team takes half of the columns.
        const int gi = u / P.Hkv, g = u - gi * P.Hkv;
        const bool owner = (it & 1) == tm;
        if (!owner && nu.valid()) {
          // The team without the last tile has time now: it stages the next unit's query rows, once the last
          // tile's scores -- the last use of the query buffer -- are complete (it only observes that barrier).
          wait_all(&ctrl->s_full[tm ^ 1], (it >> 1) & 1);
          stage_q(nu.u, n + 1);
        }
        const bool mine = pt >= 2 || owner;     // a one-tile unit leaves the other team without a state
        // The teams' (m, l) are final as soon as their own last tile's softmax is done, so they are exchanged and
        // the common reference and the two factors computed while the unit's last products still run.
        if (!is_lo) xs[tm * 64 + rho] = mine ? m : NEG_INF;
        xs[128 + (is_lo ? 128 : 0) + tm * 64 + rho] = mine ? l : 0.f;
        all_barrier();
        const float m0 = xs[rho], m1 = xs[64 + rho];
        const float mt = fmaxf(m0, m1);
        const float mtu = (mt == NEG_INF) ? 0.f : mt;
        const float f0 = fast_exp2(m0 - mtu), f1 = fast_exp2(m1 - mtu);   // 0 for a team without a state
        // (read here, before the second barrier: after it nobody touches this area until the next unit writes it)
        const float lsum = (xs[128 + rho] + xs[256 + rho]) * f0 + (xs[192 + rho] + xs[320 + rho]) * f1;
        wait_all(&ctrl->unit_done, n & 1);
        tc_fence_after();
        const int c0 = tm * (D / 2);
        uint4* xrow = reinterpret_cast<uint4*>(xo) + rho * (D / 8);       // a row of bf16: D / 8 chunks of 16 bytes
        auto combined = [&](int q, float (&v)[32]) {   // columns c0 + 32 q .. + 31 of this lane, both teams, common reference
          uint32_t a[32], bb[32];
          tmem_ld32(tO + c0 + q * 32 + lane_addr, a);
          tmem_ld32(tO + D + c0 + q * 32 + lane_addr, bb);
          tc_wait_ld();
#pragma unroll
          for (int k = 0; k < 32; ++k)   // (an accumulator without a state may hold anything)
            v[k] = (f0 != 0.f ? __uint_as_float(a[k]) * f0 : 0.f) + (f1 != 0.f ? __uint_as_float(bb[k]) * f1 : 0.f);
        };
        float v[D / 64][32];
#pragma unroll
        for (int q = 0; q < D / 64; ++q) combined(q, v[q]);
        if (is_lo) {
#pragma unroll
          for (int q = 0; q < D / 64; ++q)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              xrow[((c0 + q * 32) / 8 + k) ^ (rho & (D / 8 - 1))] =
                  make_uint4(pack_bf16x2(v[q][8 * k], v[q][8 * k + 1]), pack_bf16x2(v[q][8 * k + 2], v[q][8 * k + 3]),
                             pack_bf16x2(v[q][8 * k + 4], v[q][8 * k + 5]), pack_bf16x2(v[q][8 * k + 6], v[q][8 * k + 7]));
        }
        all_barrier();
        if (!is_lo && valid) {
          float* slotp = P.pfx_partials + (static_cast<int64_t>(gi * P.Gs + rj) * P.Hkv + g) * C::SLOT_FLOATS;
#pragma unroll
          for (int q = 0; q < D / 64; ++q) {
            float4* dst = reinterpret_cast<float4*>(slotp + 2 * C::HP + rh * D + c0 + q * 32);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const uint4 w = xrow[((c0 + q * 32) / 8 + k) ^ (rho & (D / 8 - 1))];
              dst[2 * k] = make_float4(v[q][8 * k] + __uint_as_float(w.x << 16), v[q][8 * k + 1] + __uint_as_float(w.x & 0xffff0000u),
                                       v[q][8 * k + 2] + __uint_as_float(w.y << 16), v[q][8 * k + 3] + __uint_as_float(w.y & 0xffff0000u));
              dst[2 * k + 1] = make_float4(v[q][8 * k + 4] + __uint_as_float(w.z << 16), v[q][8 * k + 5] + __uint_as_float(w.z & 0xffff0000u),
                                           v[q][8 * k + 6] + __uint_as_float(w.w << 16), v[q][8 * k + 7] + __uint_as_float(w.w & 0xffff0000u));
            }
          }
          if (tm == 0) {
            slotp[rh] = mt;
            slotp[C::HP + rh] = lsum;
          }
        }
        // (no barrier here: the next unit's writes to the (m, l) area come after this unit's second barrier, which
        // every read of it precedes, and those to the bf16 rows after the next unit's first barrier)
      }
      uc = nu;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == C::MMA_WARP) tmem_dealloc(tbase, C::TMEM_COLS);
}

}  // namespace pdattn
