// Device code of libpdattn (sm_100a only).
//
//   decode_kernel  : split-KV flash decoding.  One persistent CTA per SM walks a contiguous span
//                    of the batch's 64-token KV tiles.  Producer warps stream K/V pages from HBM
//                    into a shared-memory ring with TMA tensor copies (128-byte swizzle, one copy
//                    per page-head) signalled through mbarriers; the consumer warps each take whole tiles, compute
//                    S^T = K.Q^T and O^T += V^T.P^T with bf16 tensor-core MMAs (tokens on M, the
//                    packed GQA query heads of the KV head on N) and keep the online-softmax
//                    running max / sum in fp32.  At the end of a piece the warps' states are merged
//                    either by handing them down a chain of warps (default, no barrier) or all at
//                    once behind a consumer-wide barrier (template flag CHAIN).
//   combine_kernel : merges the (m, l, acc) triples of units that a span boundary cut.
//   plan_kernel    : device-side twin of the host partitioner for callers without host lengths.
//
// No kernel waits on another CTA.  Every mbarrier wait is bounded (kWaitLimitNs); on expiry the
// CTA raises ERR_TIMEOUT in the error word, stops consuming and returns normally.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "partition.h"

#ifndef PDATTN_NCW
#define PDATTN_NCW 6
#endif
#ifndef PDATTN_WAIT_HINT_NS
#define PDATTN_WAIT_HINT_NS 20000   // suspend-time hint of a waiting mbarrier poll
#endif
#ifndef PDATTN_NPW
#define PDATTN_NPW 3              // producer warps (tile i is issued by producer i mod NPW)
#endif

namespace pdattn {

constexpr int TILE = kTileTokens;                // tokens per pipeline stage
constexpr int MAX_SPANS = 2048;                  // spans per call (static + run-time); sizes the workspace
constexpr int MAX_PARAM_SPANS = 768;             // spans that can travel in kernel parameters
constexpr int SPAN_QUEUE = 32;                   // in-CTA queue of run-time span ids
constexpr int MAX_STAGES = 14;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

enum : int { ERR_BAD_PAGE = 1, ERR_TIMEOUT = 2 };

// Workspace header (first 256 bytes of the workspace)
struct WsHeader {
  int32_t err;        // sticky error bits
  int32_t counter;    // next run-time span; zero between calls (combine_kernel resets it)
  PlanParams plan;    // written by plan_kernel
  int32_t pad[54];
};
static_assert(sizeof(WsHeader) == 256, "header size");

struct DecodeParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const int32_t* block_table;
  const int32_t* context_lens;
  const int32_t* start_tiles;   // per sequence: leading tiles this call skips (null = none)
  const float* pfx_partials;    // with start_tiles: [seq][kv head][HP*(D+2)] partial of the skipped tiles
  WsHeader* hdr;
  const SpanStart* spans_ws;  // spans written by plan_kernel (used when use_ws_plan)
  int4* rec;                // per-span record: (first_unit, first_tile, own_unit, own_slot)
  float* partials;          // [span][2][HP*(D+2)] fp32
  int S, Hq, Hkv, G, MB, NB;
  int T;                    // query tokens per sequence (1 = plain decode); T * G rows share a KV head's tiles
  const float* k_scale;     // fp8 cache only: per KV head, value = scale * e4m3 code
  const float* v_scale;
  float scale_log2;         // scale * log2(e)
  PlanParams plan;          // host plan (ignored when use_ws_plan)
  int use_ws_plan;
  int box5d;                // 1: the tensor maps are 5-D and one TMA op brings a whole page-head
  SpanStart spans[MAX_PARAM_SPANS + 1];
};

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t count) {   // counts as `count` arrivals
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// The same with a suspend-time hint (ns): the thread may sleep in hardware until the phase
// completes instead of spinning, which is where a waiting warp spends most of this kernel.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false when the limit expired.  The clock is read once per 64 polls only.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait_hint(bar, parity, PDATTN_WAIT_HINT_NS)) return true;
    if (globaltimer_ns() - t0 > kWaitLimitNs) return false;
  }
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// 4-D tiled TMA load (no multicast), completion counted in bytes on an mbarrier of this CTA.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, int w,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar)
      : "memory");
}
// Untiled bulk copy global -> shared (16-byte aligned addresses, size a multiple of 16)
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}
// 5-D variant: (dim-in-half, slot, half, kv head, page)
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3, int c4,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// two e4m3 codes (low 16 bits of v) to two fp16 values: exact
__device__ __forceinline__ uint32_t cvt_e4m3x2_f16x2(uint32_t v) {
  uint32_t r;
  const unsigned short h = static_cast<unsigned short>(v);
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(h));
  return r;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
template <int NCT>
__device__ __forceinline__ void bar_consumers() {   // named barrier 1: the NCT consumer threads
  asm volatile("bar.sync 1, %0;" ::"n"(NCT) : "memory");
}

// ------------------------------------------------------------------------------------------
// Shared-memory plan
// ------------------------------------------------------------------------------------------
template <int D, int NT, int BS, int EB = 2>   // EB: bytes per cache element (2 = bf16, 1 = fp8 codes)
struct Cfg {
  static constexpr int PAGES = TILE / BS;              // pages per tile
  static constexpr int HALVES = D * EB / 128;          // 128-byte column blocks per row
  static constexpr int HALF_BYTES = BS * 128;          // one TMA box: BS rows x 128 bytes
  static constexpr int PAGE_BYTES = BS * D * EB;
  static constexpr int KV_BYTES = TILE * D * EB;
  static constexpr int STAGE_BYTES = 2 * KV_BYTES;     // K tile then V tile
  static constexpr int HP = 8 * NT;                    // padded query heads per KV head
  static constexpr int KSTEPS = D / 16;
  // Consumer warp w owns the tiles with index = w (mod NCW) and tile i lives in ring slot i mod
  // NSTAGES.  NSTAGES is a multiple of NCW: then the tile that used a slot one ring turn earlier
  // belonged to the same warp, so a warp can never wait on a slot's next mbarrier phase while the
  // previous one is still pending (a parity wait cannot tell those apart).  Producer warps do not
  // have that property (tile i is issued by producer i mod NPW); they check the previous user's
  // progress word instead.
  // There is no separate merge scratch: at the end of a piece the ring slot of the piece's last
  // tile is kept back and the warps exchange their accumulators through it.
  static constexpr int ACC_STRIDE = D + 4;             // floats; keeps the parked stores conflict-free
  static constexpr int SMEM_MAX = 232448;              // 227 KB
  static constexpr int CTRL_BYTES = 768;
  static constexpr int NCW = PDATTN_NCW;                               // consumer warps
  static constexpr int ML_BYTES = NCW * HP * 2 * 4;
  static constexpr int QSLOTS = 4;                     // query rows of upcoming pieces, staged by producer 0
  static constexpr int Q_BYTES = HP * D * 2;           // one slot: the packed query heads of one KV head
  static constexpr int NSTAGES_FIT = (SMEM_MAX - 1024 - QSLOTS * Q_BYTES - ML_BYTES - CTRL_BYTES) / STAGE_BYTES;
  static constexpr int NSTAGES = (NSTAGES_FIT > MAX_STAGES ? MAX_STAGES : NSTAGES_FIT) / NCW * NCW;
  static constexpr int NCT = NCW * 32;                                 // consumer threads
  static constexpr int NPW = (NT == 2 && PDATTN_NPW > 2) ? 2 : PDATTN_NPW;   // producer warps (8 warps in all for 16-row tiles: 255 registers)
  static constexpr int NTHREADS = NCT + 32 * NPW;
  static constexpr int DYN_BYTES = 1024 + NSTAGES * STAGE_BYTES + QSLOTS * Q_BYTES + ML_BYTES + CTRL_BYTES;
  static constexpr int SLOT_FLOATS = HP * (D + 2);     // one partial: m[HP], l[HP], acc[HP][D]
  // Chained merge (decode_kernel with CHAIN): a warp's running (m, l, acc) of a piece in MMA fragment
  // order, one float4 per lane per row: NT rows of (m0, m1, l0, l1), then acc[nt][jm] -- 512 B a row.
  static constexpr int HANDOFF_BYTES = NT * (1 + D / 16) * 512;
  static constexpr int HANDOFFS_FIT = (SMEM_MAX - DYN_BYTES) / HANDOFF_BYTES;
  static constexpr int HANDOFFS = HANDOFFS_FIT > 8 ? 8 : HANDOFFS_FIT;   // pieces whose merge is under way
  static constexpr int CHAIN_DYN_BYTES = DYN_BYTES + HANDOFFS * HANDOFF_BYTES;
  static_assert(NSTAGES >= NCW && NSTAGES % NCW == 0, "ring/warp mapping");
  static_assert(HP * ACC_STRIDE * 4 <= STAGE_BYTES, "a parked accumulator must fit one stage");
  static_assert(DYN_BYTES <= SMEM_MAX, "shared memory");
  static_assert(TILE % BS == 0 && BS % 16 == 0, "block size");
};

struct Ctrl {                 // lives in the CTRL_BYTES area
  uint64_t full[MAX_STAGES];
  uint64_t empty[MAX_STAGES];
  uint32_t meta[MAX_STAGES];  // per stage: bit j set = page j of the tile had a bad id
  uint32_t abort;
  int32_t sq_pub;             // number of run-time span ids published so far
  int32_t sq_id[SPAN_QUEUE];  // k-th id (k >= 1) at [(k-1) % SPAN_QUEUE]; -1 = no more spans
  int32_t sq_tag[SPAN_QUEUE]; // k, to detect an overwritten entry
  int32_t prod_last[4];       // per producer warp: index of the last tile it issued (-1 = none)
  uint64_t q_full[4];         // query slot q holds the rows of piece p, p mod QSLOTS == q
  uint64_t q_empty[4];        // ... and every consumer warp has copied them to registers
  int32_t qseq[4];            // CHAIN: piece whose rows the producer last armed the query slot for
  int32_t turn[8];            // CHAIN: hand-off slot e is waiting for class (turn % 8) of merge number (turn / 8)
};
static_assert(sizeof(Ctrl) <= 768, "control block");

// ------------------------------------------------------------------------------------------
// The walk over a span: pieces = (unit, tile range) in order.  Every warp runs the same walk.
// ------------------------------------------------------------------------------------------
struct Piece {
  int unit, s, g, L, nt, tb, te;
  int t0;   // tiles of the sequence that are skipped (shared prefix handled elsewhere): tile t of the
            // piece is tile t0 + t of the sequence
};
struct Walker {
  const int32_t* ctx;
  const int32_t* start_tiles;   // per sequence, may be null (= 0)
  int Hkv, nunits, unit, tb, rem;
  int pf_unit = -1, pf_L = 0, pf_t0 = 0;   // the following unit's length and start, loaded one piece early
  __device__ __forceinline__ bool next(Piece& p) {
    while (rem > 0 && unit < nunits) {
      const int s = unit / Hkv;
      const bool hit = unit == pf_unit;
      const int L = hit ? pf_L : __ldg(ctx + s);
      const int t0 = hit ? pf_t0 : (start_tiles ? __ldg(start_tiles + s) : 0);
      if (unit + 1 < nunits) {
        pf_unit = unit + 1;
        pf_L = __ldg(ctx + (unit + 1) / Hkv);
        pf_t0 = start_tiles ? __ldg(start_tiles + (unit + 1) / Hkv) : 0;
      }
      const int nt_all = L > 0 ? (L + TILE - 1) / TILE : 0;
      const int nt = nt_all > t0 ? nt_all - t0 : 0;
      if (tb >= nt) {
        ++unit;
        tb = 0;
        continue;
      }
      p.unit = unit;
      p.s = s;
      p.g = unit - s * Hkv;
      p.L = L;
      p.nt = nt;
      p.t0 = t0;
      p.tb = tb;
      p.te = min(nt, tb + rem);
      rem -= p.te - p.tb;
      ++unit;
      tb = 0;
      return true;
    }
    return false;
  }
};

// ------------------------------------------------------------------------------------------
// One 64-token tile on one warp
// ------------------------------------------------------------------------------------------
template <int D, int NT, int BS, bool TAIL>
__device__ __forceinline__ void compute_tile(uint32_t sK, uint32_t sV, const uint32_t (&qf)[NT][D / 16][2],
                                             float (&acc)[NT][D / 16][4], float (&m)[NT][2], float (&l)[NT][2],
                                             float sl2, int n_left, uint32_t badmask, int lane,
                                             const int (&lag)[NT][2]) {
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

// ------------------------------------------------------------------------------------------
// One 64-token tile on one warp, fp8 cache (e4m3 codes; head_dim 128).
// K tile: [64 tokens][128 B] (one code per element, 128-byte swizzle); V tile: per page [128 d][BS tokens]
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
template <int NT, int BS, bool TAIL>
__device__ __forceinline__ void compute_tile_f8(uint32_t sK, uint32_t sV, const uint32_t (&qf)[NT][8][2],
                                                float (&acc)[NT][8][4], float (&m)[NT][2], float (&l)[NT][2],
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
      const uint32_t base = sK + tok * 128;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        const int ch = (cc * 2 + k_csel) ^ (tok & 7);
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
      for (int jm = 0; jm < 8; ++jm) {
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

  // ---- O^T += V^T . P^T : [128] x [8*NT heads], 16 tokens of a page per MMA step
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
      for (int jp = 0; jp < 4; ++jp) {
        uint32_t r[4];
        ldsm_x4(r, sV + ((j * 16) / BS) * (128 * BS) + (jp * 32 + v_drow) * BS + (j * 16) % BS);
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

// ------------------------------------------------------------------------------------------
// Span sequencing inside a CTA.  Every warp walks the same sequence of spans: first the CTA's
// static span, then run-time spans.  Lane 0 of producer warp 0 draws run-time spans from the
// global counter (one atomic per span, issued a whole span ahead of its use) and publishes the
// ids through a small shared-memory queue; every other warp reads them from there.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int ld_acquire_shared(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.cta.shared.b32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_shared(int32_t* p, int v) {
  asm volatile("st.release.cta.shared.b32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
// k-th span of this CTA (k >= 1), or -1 when there is none (or the bounded wait expired).
__device__ __forceinline__ int read_span(Ctrl* ctrl, int k, bool& aborted) {
  if (aborted) return -1;
  if (ld_acquire_shared(&ctrl->sq_pub) < k) {
    const unsigned long long t0 = globaltimer_ns();
    while (ld_acquire_shared(&ctrl->sq_pub) < k) {
      if (*reinterpret_cast<volatile uint32_t*>(&ctrl->abort) || globaltimer_ns() - t0 > kWaitLimitNs) {
        aborted = true;
        return -1;
      }
    }
  }
  const int slot = (k - 1) % SPAN_QUEUE;
  const int id = ctrl->sq_id[slot];
  if (ctrl->sq_tag[slot] != k) {   // the queue wrapped past a reader: cannot happen while warps stay
    aborted = true;                //  within a ring's worth of tiles of each other; fail loudly if it does
    return -1;
  }
  return id;
}

// Query slot `qs` holds the rows of piece `p`.  A parity wait alone cannot tell "piece p has landed"
// from "the slot's previous piece has not landed yet" (two phases apart look the same), and in the
// chained-merge variant a warp skips the pieces it holds no tile of.  The producer therefore
// records which piece it armed the slot for (before the arming arrive, which releases the record); a
// wait that returns while the record still names an older piece is repeated.
template <int QSLOTS>
__device__ __forceinline__ bool wait_q(Ctrl* ctrl, int qs, int p) {
  const uint32_t phase = (p / QSLOTS) & 1;
  const uint32_t bar = smem_u32(&ctrl->q_full[qs]);
  if (!mbar_wait(bar, phase)) return false;
  if (ld_acquire_shared(&ctrl->qseq[qs]) == p) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (ld_acquire_shared(&ctrl->qseq[qs]) == p && mbar_try_wait(bar, phase)) return true;
    if (*reinterpret_cast<volatile uint32_t*>(&ctrl->abort) || globaltimer_ns() - t0 > kWaitLimitNs) return false;
  }
}
// Bounded wait until a hand-off slot's turn word reaches `want`.
__device__ __forceinline__ bool wait_turn(Ctrl* ctrl, int e, int want) {
  if (ld_acquire_shared(&ctrl->turn[e]) == want) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (ld_acquire_shared(&ctrl->turn[e]) == want) return true;
    if (*reinterpret_cast<volatile uint32_t*>(&ctrl->abort) || globaltimer_ns() - t0 > kWaitLimitNs) return false;
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
template <int D, int NT, int BS, int EB>
__device__ __forceinline__ void consume_chain(const DecodeParams& P, const PlanParams& pp, Ctrl* ctrl, uint32_t ring,
                                              uint32_t qbuf, uint8_t* handoff, int warp, int lane) {
  using C = Cfg<D, NT, BS, EB>;
  static_assert(EB == 2 || (EB == 1 && D == 128), "the fp8 cache path is built for head_dim 128");
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
    Walker walk{P.context_lens, P.start_tiles, P.Hkv, nunits, sp.unit, sp.tile, sp_end - sp.flat};
    Piece pc;
    int first_unit = -1, first_tb = 0, own_unit = -1, own_slot = 0, piece_idx = 0;

    while (walk.next(pc)) {
      const int n_piece = pc.te - pc.tb;
      const int it0 = it;
      it += n_piece;
      const int p = pcnt++;
      const int n_cls = n_piece < NCW ? n_piece : NCW;
      const bool multi = n_cls > 1;
      const int mq = mcnt;            // number of this piece among those with more than one class
      if (multi) ++mcnt;
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
      if (*reinterpret_cast<volatile uint32_t*>(&ctrl->abort)) {
        aborted = true;
        continue;
      }

      // ---- packed query rows of this KV head as MMA B fragments, from the staged copy
      uint32_t qf[NT][D / 16][2];
      {
        const int qs = p % C::QSLOTS;
        if (!wait_q<C::QSLOTS>(ctrl, qs, p)) {
          fail();
          continue;
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
          if (n_left - (P.T - 1) >= TILE) {   // every query token sees the whole tile
            compute_tile<D, NT, BS, false>(sK, sV, qf, acc, m, l, P.scale_log2, TILE, badmask, lane, lag);
          } else {
            compute_tile<D, NT, BS, true>(sK, sV, qf, acc, m, l, P.scale_log2, n_left, badmask, lane, lag);
            fence_proxy_async();   // our zero-fill stores must be ordered before the next TMA write
          }
        } else {
          if (n_left - (P.T - 1) >= TILE) {
            compute_tile_f8<NT, BS, false>(sK, sV, qf, acc, m, l, sl2, TILE, badmask, lane, lag);
          } else {
            compute_tile_f8<NT, BS, true>(sK, sV, qf, acc, m, l, sl2, n_left, badmask, lane, lag);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->empty[slot]));
      }
      if (aborted) continue;
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
          continue;
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
          continue;
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
      }
    }
    if (warp == 0 && lane == 0) P.rec[span] = make_int4(first_unit, first_tb, own_unit, own_slot);
    span = read_span(ctrl, k + 1, aborted);
  }
  if (aborted && lane == 0) atomicOr(&P.hdr->err, ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------
// The decode kernel.  PROBE = true builds the page-gather ceiling: identical span walk, page-id
// lookups and TMA ring, but the consumers release every tile untouched and nothing is written.
// CHAIN = true replaces the consumers' barrier-and-merge at the end of each piece by the chained
// hand-off of consume_chain (the producers are the same).
// ------------------------------------------------------------------------------------------
template <int D, int NT, int BS, bool PROBE = false, bool CHAIN = false, int EB = 2>
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
    fence_mbar_init();
  }
  __syncthreads();

  const PlanParams pp = P.use_ws_plan ? P.hdr->plan : P.plan;
  const int nunits = P.S * P.Hkv;
  int it = 0;        // tile counter within this CTA: tile `it` uses ring slot it % NST
  int pcnt = 0;      // piece counter within this CTA: piece p's query rows use query slot p % QSLOTS
  bool aborted = false;

  if (warp >= NCW) {
    // ================= producer warp(s) =================
    const int pw = warp - NCW;
    constexpr int IDS_PER_BATCH = 32;
    constexpr int TILES_PER_BATCH = IDS_PER_BATCH / C::PAGES;
    bool any_bad = false;
    int span = cta;
    for (int k = 0; span >= 0; ++k) {
      // draw the next run-time span now; its id is only consumed after this span's tiles are issued
      int nxt = -1;
      if (pw == 0 && lane == 0 && pp.n_dyn > 0) {
        const int j = atomicAdd(&P.hdr->counter, 1);
        nxt = j < pp.n_dyn ? pp.n_static + j : -1;
      }
      const SpanStart sp = P.use_ws_plan ? P.spans_ws[span] : P.spans[span];
      const int sp_end = P.use_ws_plan ? P.spans_ws[span + 1].flat : P.spans[span + 1].flat;
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
        const int32_t* row = P.block_table + static_cast<int64_t>(pc.s) * P.MB;
        const int npages = (pc.L + BS - 1) / BS;
        const int pbase = (pc.t0 + pc.tb) * C::PAGES;
        int ids_cur = (pbase + lane < npages) ? __ldg(row + pbase + lane) : 0;
        int ids_nxt = (pbase + IDS_PER_BATCH + lane < npages) ? __ldg(row + pbase + IDS_PER_BATCH + lane) : 0;
        for (int t = pc.tb; t < pc.te; ++t, ++it) {
          const int rel = t - pc.tb;
          const int kb = rel % TILES_PER_BATCH;
          if (kb == 0 && rel != 0) {
            ids_cur = ids_nxt;
            const int nb = pbase + rel * C::PAGES + IDS_PER_BATCH;
            ids_nxt = (nb + lane < npages) ? __ldg(row + nb + lane) : 0;
          }
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
              if (aborted) break;
            }
          }
          if (!mbar_wait(smem_u32(&ctrl->empty[slot]), phase ^ 1u)) {
            aborted = true;
            break;
          }
          const int np = min(C::PAGES, npages - (pc.t0 + t) * C::PAGES);
          const int j = lane % C::PAGES;
          int id = __shfl_sync(0xffffffffu, ids_cur, kb * C::PAGES + j);
          const bool bad = (lane < C::PAGES) && (j < np) && (id < 0 || id >= P.NB);
          const uint32_t badmask = __ballot_sync(0xffffffffu, bad);
          if (id < 0 || id >= P.NB) id = P.NB;   // out-of-bounds coordinate: TMA fills zeros, nothing is read
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
          any_bad |= (badmask != 0);
          if (NST % C::NPW != 0) {
            __syncwarp();
            if (lane == 0) st_release_shared(&ctrl->prod_last[pw], it);
          }
        }
      }
      if (aborted) break;
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
    consume_chain<D, NT, BS, EB>(P, pp, ctrl, ring, qbuf,
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
          compute_tile<D, NT, BS, false>(sK, sV, qf, acc, m, l, P.scale_log2, TILE, badmask, lane, lag);
        } else {
          compute_tile<D, NT, BS, true>(sK, sV, qf, acc, m, l, P.scale_log2, n_left, badmask, lane, lag);
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
          bar_consumers<NCT>();   // everyone has read this round's accumulators
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
  int2 ranges[160];
};

template <int D, int BS>
__global__ void __launch_bounds__(Cfg<D, 1, BS>::NTHREADS, 1)
prefix_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
              const __grid_constant__ PrefixParams P) {
  using C = Cfg<D, 1, BS>;
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
        qf[0][kk][0] = live ? __ldg(qp + (kk * 16 + qcol) / 2) : 0u;
        qf[0][kk][1] = live ? __ldg(qp + (kk * 16 + 8 + qcol) / 2) : 0u;
      }
    }
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
        compute_tile<D, 1, BS, false>(sK, sK + C::KV_BYTES, qf, acc, m, l, P.scale_log2, TILE, ctrl->meta[slot], lane, no_lag);
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
            a[jm * 16 + drow] = acc[0][jm][e];
            a[jm * 16 + drow + 8] = acc[0][jm][2 + e];
          }
        }
      }
    }
  }
  if (aborted && lane == 0) atomicOr(P.err, ERR_TIMEOUT);
}

// ------------------------------------------------------------------------------------------
// KV append: the step on the input side of decode attention.  Block s writes the new token's K
// and V rows of every KV head into slot L_s % bs of page block_table[s, L_s / bs] and then
// advances context_lens[s].  One warp per KV head: lanes copy 16-byte chunks, K then V.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512)
append_kernel(const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
              __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
              const int32_t* __restrict__ block_table, int32_t* __restrict__ context_lens, int Hkv, int D, int bs,
              int MB, int NB, int64_t sb, int64_t sh, int64_t st, int32_t* err) {
  const int s = blockIdx.x;
  const int g = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int L = context_lens[s];
  __syncthreads();                       // every warp has read the old length before it is advanced
  if (L < 0 || L / bs >= MB) {
    if (threadIdx.x == 0 && err) atomicOr(err, ERR_BAD_PAGE);
    return;
  }
  const int page = block_table[static_cast<int64_t>(s) * MB + L / bs];
  if (page < 0 || page >= NB) {          // not dereferenced; the length is left as it was
    if (threadIdx.x == 0 && err) atomicOr(err, ERR_BAD_PAGE);
    return;
  }
  if (g < Hkv) {
    const int64_t dst = page * sb + g * sh + static_cast<int64_t>(L % bs) * st;
    const int64_t src = (static_cast<int64_t>(s) * Hkv + g) * D;
    const int chunks = D / 8;            // 16-byte chunks per row
    for (int c = lane; c < 2 * chunks; c += 32) {
      const bool isV = c >= chunks;
      const int cc = isV ? c - chunks : c;
      const uint4 v = *reinterpret_cast<const uint4*>((isV ? v_new : k_new) + src + cc * 8);
      *reinterpret_cast<uint4*>((isV ? v_cache : k_cache) + dst + cc * 8) = v;
    }
  }
  if (threadIdx.x == 0) context_lens[s] = L + 1;
}

// Read-only streaming ceiling: every thread block sums a contiguous slice with 16-byte loads.
__global__ void __launch_bounds__(512)
stream_read_kernel(const uint4* __restrict__ src, size_t n_vec, uint32_t* __restrict__ sink) {
  uint32_t acc = 0;
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
#pragma unroll 1
  for (; i + 3 * stride < n_vec; i += 4 * stride) {
    const uint4 a = __ldcs(src + i), b = __ldcs(src + i + stride), c = __ldcs(src + i + 2 * stride),
                d = __ldcs(src + i + 3 * stride);
    acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ d.x ^ d.y ^ d.z ^ d.w;
  }
  for (; i < n_vec; i += stride) {
    const uint4 a = __ldcs(src + i);
    acc ^= a.x ^ a.y ^ a.z ^ a.w;
  }
  if (acc == 0x9e3779b9u) *sink = acc;   // practically never: keeps the loads alive
}

// ------------------------------------------------------------------------------------------
// KV append into an fp8 cache: the new token's K and V rows (bf16) are divided by the KV head's scale,
// rounded to e4m3 (nearest even, saturating to the largest finite code) and written as codes: K as a
// row of the page [slot][d], V as a column of the transposed page [d][slot].  One block per sequence,
// one warp per KV head.  Same rules as append_kernel for bad pages and full rows.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512)
append_fp8_kernel(const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
                  uint8_t* __restrict__ k8, uint8_t* __restrict__ v8, const float* __restrict__ k_scale,
                  const float* __restrict__ v_scale, const int32_t* __restrict__ block_table,
                  int32_t* __restrict__ context_lens, int Hkv, int D, int bs, int MB, int NB, int32_t* err) {
  const int s = blockIdx.x;
  const int g = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int L = context_lens[s];
  __syncthreads();                       // every warp has read the old length before it is advanced
  if (L < 0 || L / bs >= MB) {
    if (threadIdx.x == 0 && err) atomicOr(err, ERR_BAD_PAGE);
    return;
  }
  const int page = block_table[static_cast<int64_t>(s) * MB + L / bs];
  if (page < 0 || page >= NB) {
    if (threadIdx.x == 0 && err) atomicOr(err, ERR_BAD_PAGE);
    return;
  }
  if (g < Hkv) {
    const int slot = L % bs;
    const float sk = k_scale[g], sv = v_scale[g];   // true divisions below: the code is decided in fp32
    const int64_t src = (static_cast<int64_t>(s) * Hkv + g) * D;
    uint8_t* kp = k8 + ((static_cast<int64_t>(page) * Hkv + g) * bs + slot) * D;
    uint8_t* vp = v8 + (static_cast<int64_t>(page) * Hkv + g) * D * bs + slot;
    for (int j = lane * 2; j < D; j += 64) {
      const float2 kf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(k_new + src + j));
      const float2 vf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(v_new + src + j));
      unsigned short kc, vc;
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(kc) : "f"(__fdiv_rn(kf.y, sk)), "f"(__fdiv_rn(kf.x, sk)));
      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(vc) : "f"(__fdiv_rn(vf.y, sv)), "f"(__fdiv_rn(vf.x, sv)));
      *reinterpret_cast<unsigned short*>(kp + j) = kc;
      vp[static_cast<int64_t>(j) * bs] = static_cast<uint8_t>(vc & 0xff);
      vp[static_cast<int64_t>(j + 1) * bs] = static_cast<uint8_t>(vc >> 8);
    }
  }
  if (threadIdx.x == 0) context_lens[s] = L + 1;
}

// ------------------------------------------------------------------------------------------
// Split-combine: block i merges the unit that started in span i and ran past its end.  The
// pieces live in the following spans (slot 0 of each follower), merged in ascending token order:
//   M = max m_c;  Lsum = sum l_c 2^(m_c - M);  out = bf16( sum acc_c 2^(m_c - M) / Lsum ).
// Block 0 also rearms the run-time span counter for the next call.
// ------------------------------------------------------------------------------------------
template <int D, int NT>
__global__ void __launch_bounds__(256)
combine_kernel(WsHeader* hdr, int n_spans_host, const int4* __restrict__ rec, const float* __restrict__ partials,
               __nv_bfloat16* __restrict__ out, int Hq, int Hkv, int G, const int32_t* __restrict__ start_tiles,
               const float* __restrict__ pfx_partials, int T) {
  constexpr int HP = 8 * NT;
  constexpr int SLOT_FLOATS = HP * (D + 2);
  const int c = blockIdx.x;
  // launched as a programmatic dependent of the decode kernel: nothing of that kernel may be read
  // before this returns (it waits for the kernel's completion and memory flush)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (c == 0 && threadIdx.x == 0) hdr->counter = 0;
  const int n_spans = n_spans_host >= 0 ? n_spans_host : hdr->plan.n_static + hdr->plan.n_dyn;
  if (c >= n_spans) return;
  const int4 r = rec[c];
  const int unit = r.z;
  if (unit < 0) return;
  // followers: later spans whose first piece continues `unit` (spans without tiles may sit between)
  __shared__ int n_follow;
  __shared__ int follow[MAX_SPANS];
  if (threadIdx.x == 0) {
    int n = 0;
    for (int cc = c + 1; cc < n_spans; ++cc) {
      const int4 rr = rec[cc];
      if (rr.x < 0) continue;                 // a span that holds no tile
      if (rr.x != unit || rr.y <= 0) break;
      follow[n++] = cc;
    }
    n_follow = n;
  }
  __syncthreads();
  const int np = n_follow + 1;
  const int s = unit / Hkv, g = unit - s * Hkv;
  // piece -1: the partial of the unit's leading tiles when those were handled elsewhere (shared prefix)
  const int p0 = (start_tiles && start_tiles[s] > 0) ? -1 : 0;
  auto piece = [&](int p) -> const float* {
    if (p < 0) return pfx_partials + static_cast<int64_t>(unit) * SLOT_FLOATS;
    return partials + (p == 0 ? static_cast<int64_t>(c) * 2 + r.w : static_cast<int64_t>(follow[p - 1]) * 2) * SLOT_FLOATS;
  };
  const float NEG_INF = __int_as_float(0xff800000);
  for (int idx = threadIdx.x; idx < HP * (D / 4); idx += blockDim.x) {
    const int h = idx / (D / 4);
    const int dq = idx % (D / 4);
    if (h >= G * T) continue;   // row h = query token * G + head
    float M = NEG_INF;
    for (int p = p0; p < np; ++p) M = fmaxf(M, piece(p)[h]);
    const float Mu = (M == NEG_INF) ? 0.f : M;
    float Ls = 0.f;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int p = p0; p < np; ++p) {
      const float* part = piece(p);
      const float f = fast_exp2(part[h] - Mu);
      Ls += part[HP + h] * f;
      const float4 v = *reinterpret_cast<const float4*>(part + 2 * HP + h * D + dq * 4);
      a.x += v.x * f;
      a.y += v.y * f;
      a.z += v.z * f;
      a.w += v.w * f;
    }
    const float inv = Ls > 0.f ? 1.f / Ls : 0.f;
    uint2 o;
    o.x = pack_bf16x2(a.x * inv, a.y * inv);
    o.y = pack_bf16x2(a.z * inv, a.w * inv);
    const int qtok = h / G;
    *reinterpret_cast<uint2*>(out + ((static_cast<int64_t>(s) * T + qtok) * Hq + g * G + (h - qtok * G)) * D + dq * 4) = o;
  }
}

// ------------------------------------------------------------------------------------------
// Device twin of the host partitioner (one block).  prefix: [2 * (S + 1)] ints of scratch:
// running cost, then running tile count, per sequence.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int block_scan_1024(int v, int* warp_sums, int lane, int wid) {
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) warp_sums[wid] = x;
  __syncthreads();
  if (wid == 0) {
    int w = warp_sums[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += y;
    }
    warp_sums[lane] = w;
  }
  __syncthreads();
  const int incl = x + (wid > 0 ? warp_sums[wid - 1] : 0);
  __syncthreads();
  return incl;
}

__global__ void __launch_bounds__(1024)
plan_kernel(const int32_t* __restrict__ context_lens, const int32_t* __restrict__ start_tiles, int S, int Hkv,
            int n_static, int n_dyn_max, int32_t* __restrict__ prefix, SpanStart* __restrict__ spans, WsHeader* hdr) {
  __shared__ int warp_sums[32];
  __shared__ int carry_c, carry_t;
  __shared__ PlanParams pp_s;
  int32_t* pcost = prefix;
  int32_t* ptile = prefix + (S + 1);
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) {
    carry_c = carry_t = 0;
    pcost[0] = ptile[0] = 0;
  }
  __syncthreads();
  for (int base = 0; base < S; base += 1024) {
    const int s = base + tid;
    int nt = 0;
    if (s < S) nt = static_cast<int>(seq_tiles(context_lens[s], start_tiles ? start_tiles[s] : 0));
    const int ic = block_scan_1024(static_cast<int>(seq_cost(nt, Hkv)), warp_sums, lane, wid) + carry_c;
    const int itl = block_scan_1024(nt * Hkv, warp_sums, lane, wid) + carry_t;
    if (s < S) {
      pcost[s + 1] = ic;
      ptile[s + 1] = itl;
    }
    __syncthreads();
    if (tid == 1023) {
      carry_c = ic;
      carry_t = itl;
    }
    __syncthreads();
  }
  if (tid == 0) {
    pp_s = make_plan_params(carry_c, carry_t, n_static, n_dyn_max);
    hdr->plan = pp_s;
  }
  __threadfence_block();
  __syncthreads();
  const PlanParams pp = pp_s;
  const int n_spans = pp.n_static + pp.n_dyn;
  const int total_cost = static_cast<int>(pp.cost_total);
  for (int c = tid; c <= n_spans; c += 1024) {
    SpanStart sp;
    sp.unit = S * Hkv;
    sp.tile = 0;
    sp.flat = pp.total;
    sp.pad = 0;
    const int x = static_cast<int>(span_cost_start(pp, c));
    if (c < n_spans && x < total_cost) {
      int lo = 0, hi = S;   // find s with pcost[s] <= x < pcost[s+1]
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pcost[mid] <= x) lo = mid; else hi = mid;
      }
      const int nt = static_cast<int>(seq_tiles(context_lens[lo], start_tiles ? start_tiles[lo] : 0));
      int k, tile;
      locate_in_seq(x - pcost[lo], nt, &k, &tile);
      sp.unit = lo * Hkv + k;
      sp.tile = tile;
      sp.flat = ptile[lo] + k * nt + tile;
    }
    spans[c] = sp;
  }
}

}  // namespace pdattn
