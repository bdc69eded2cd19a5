// Shared by every kernel of libpdattn (sm_100a only): constants, the workspace header and kernel parameters,
// PTX wrappers (mbarrier, TMA, ldmatrix, MMA, conversions), the shared-memory plan (Cfg, Ctrl), the walk over
// a span's pieces, and the in-CTA sequencing of spans and hand-off waits.
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
#ifndef PDATTN_DRAW_AHEAD
#define PDATTN_DRAW_AHEAD 12   // tiles left in a span when the producer draws the CTA's next run-time span
#endif
constexpr int MAX_PARAM_SPANS = 768;             // spans that can travel in kernel parameters
constexpr int SPAN_QUEUE = 32;                   // in-CTA queue of run-time span ids
constexpr int MAX_STAGES = 14;
constexpr int MERGE_QUEUE = 8;                  // entries of the in-CTA queue of merge jobs
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

enum : int { ERR_BAD_PAGE = 1, ERR_TIMEOUT = 2, ERR_TOO_LARGE = 4 };

// Workspace header (first 256 bytes of the workspace)
struct WsHeader {
  int32_t err;        // sticky error bits
  int32_t counter;    // next run-time span; zero between calls (the last CTA out resets it)
  PlanParams plan;    // written by plan_kernel
  int32_t done;       // CTAs of the running decode kernel whose span draws are over; zero between calls
  int32_t pad[53];
};
static_assert(sizeof(WsHeader) == 256, "header size");
// Behind the header: one ticket word per span, zero between calls.  Word c counts the partials written so far
// for the unit that starts in span c and runs past its end; the CTA that brings the count to the unit's number
// of pieces merges them and writes the output (no CTA ever waits for another).
constexpr int WS_TICKETS_OFFSET = 256;
constexpr int WS_TICKETS_BYTES = MAX_SPANS * 4;
constexpr int WS_CLEARED_BYTES = WS_TICKETS_OFFSET + WS_TICKETS_BYTES;   // what must be zero before the first call

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
  int32_t* tickets;         // [MAX_SPANS] ticket words (see WS_TICKETS_OFFSET)
  int inkernel_max;         // > 0: a cut unit whose followers all lie within this many spans after its first one is
                            // merged by the CTA that writes its last partial; 0: every cut unit is left to combine_kernel
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
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
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
  static constexpr int HALVES = D * EB / 128 > 0 ? D * EB / 128 : 1;   // copies per page-head with the rank-4 view
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
  static constexpr int CTRL_BYTES = 1280;
  static constexpr int NCW = PDATTN_NCW;                               // consumer warps
  static constexpr int ML_BYTES = NCW * HP * 2 * 4;
  static constexpr int QSLOTS = 4;                     // query rows of upcoming pieces, staged ahead of the consumers
  static constexpr int Q_BYTES = HP * D * 2;           // one slot: the packed query heads of one KV head
  static constexpr int NSTAGES_FIT = (SMEM_MAX - 1024 - QSLOTS * Q_BYTES - ML_BYTES - CTRL_BYTES) / STAGE_BYTES;
  static constexpr int NSTAGES = (NSTAGES_FIT > MAX_STAGES ? MAX_STAGES : NSTAGES_FIT) / NCW * NCW;
  static constexpr int NCT = NCW * 32;                                 // consumer threads
  static constexpr int NPW = (NT == 2 && PDATTN_NPW > 2) ? 2 : PDATTN_NPW;   // producer warps (8 warps in all for 16-row tiles: 255 registers)
  // One more warp (8-row tiles only: with 16-row tiles the consumers need every register a smaller block leaves
  // them) does the final merge of cut units: consumers post jobs to it through shared memory and never wait
  // on global memory for a merge themselves.
  static constexpr bool MERGE_WARP = NT == 1;
  static constexpr int NTHREADS_BASE = NCT + 32 * NPW;                      // consumers and producers
  static constexpr int NTHREADS = NTHREADS_BASE + (MERGE_WARP ? 32 : 0);    // decode_kernel's block
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
  uint64_t full[MAX_STAGES];    // the stage's tile has landed (with split halves: its K half)
  uint64_t empty[MAX_STAGES];   // ... and has been consumed
  uint64_t full_v[MAX_STAGES];  // split halves only: the V half, filled and released on its own
  uint64_t empty_v[MAX_STAGES];
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
  // queue of merge jobs from the consumer warps to the merge warp (CHAIN with Cfg::MERGE_WARP)
  int32_t mq_head;            // jobs claimed so far (shared-memory atomic)
  int32_t mq_tail;            // jobs the merge warp has taken over
  int32_t mq_done;            // consumer warps that will post no more jobs
  int32_t mq_tag[MERGE_QUEUE];   // job k has been written to entry k % MERGE_QUEUE when its tag is k + 1
  int4 mq_job[MERGE_QUEUE];   // (first span c, hold mask, ticket increment, unit | has-prefix flag << 30)
};
static_assert(sizeof(Ctrl) <= 1280, "control block");

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
// The same walk, 32 units at a time, for the short-piece instantiation of the chained-merge kernel.  A consumer warp works on
// the pieces it holds a tile of and has to step over all the others; with the one-piece-at-a-time Walker that step
// (a dependent load, tile arithmetic, bookkeeping) cost ≈ 700 cycles, and in a batch of one-tile pieces a warp
// steps over five pieces for every one it works on.  Here lane i looks at unit base + i: one lane-wide load of
// the lengths (fetched a window ahead), one warp scan of the tile counts, and a ballot tell the warp which of the
// 32 pieces are its own; only for those are the fields broadcast.
// ------------------------------------------------------------------------------------------
struct PieceWindow {
  // per lane (unit base + lane)
  int unit, s, L, t0, full;   // full: tiles of the unit that this call covers
  int tb, take;               // this span's piece of the unit: tiles [tb, tb + take) (take == 0: none)
  int it0;                    // CTA tile counter at the piece's first tile
  // uniform
  int total;                  // tiles of the whole window
};
struct WindowWalker {
  const int32_t* ctx;
  const int32_t* start_tiles;   // per sequence, may be null (= 0)
  int Hkv, nunits, lane;
  int base = 0, rem = 0, first = 0, tb0 = 0;
  int nL = 0, nT = 0, nS = 0;   // the window at `base`, fetched ahead
  __device__ __forceinline__ void fetch(int b) {
    const int u = b + lane;
    nS = u < nunits ? u / Hkv : 0;
    nL = u < nunits ? __ldg(ctx + nS) : 0;
    nT = (start_tiles && u < nunits) ? __ldg(start_tiles + nS) : 0;
  }
  __device__ __forceinline__ void begin_span(int unit, int tile, int count) {
    first = base = unit;
    tb0 = tile;
    rem = count;
    if (rem > 0) fetch(base);
  }
  // it: the CTA's tile counter before this window
  __device__ __forceinline__ bool next(PieceWindow& w, int it) {
    if (rem <= 0 || base >= nunits) return false;
    w.unit = base + lane;
    w.s = nS;
    w.L = nL;
    w.t0 = nT;
    const int all = w.L > 0 ? (w.L + TILE - 1) / TILE : 0;
    w.full = (w.unit < nunits && all > w.t0) ? all - w.t0 : 0;
    w.tb = w.unit == first ? tb0 : 0;
    const int avail = w.full > w.tb ? w.full - w.tb : 0;
    int incl = avail;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    const int excl = incl - avail;
    w.take = excl >= rem ? 0 : (rem - excl < avail ? rem - excl : avail);
    w.it0 = it + excl;
    const int sum = __shfl_sync(0xffffffffu, incl, 31);
    w.total = sum < rem ? sum : rem;
    rem -= w.total;
    base += 32;
    if (rem > 0 && base < nunits) fetch(base);   // used a whole window of work later
    return true;
  }
};

// ------------------------------------------------------------------------------------------
// Span sequencing inside a CTA.  Every warp walks the same sequence of spans: first the CTA's
// static span, then run-time spans.  Lane 0 of producer warp 0 draws run-time spans from the
// global counter (one atomic per span, issued a dozen tiles before the current span's last) and
// publishes the ids through a small shared-memory queue; every other warp reads them from there.
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
  if (ctrl->sq_tag[slot] != k) {   // the queue wrapped past a reader: cannot happen while a CTA draws fewer
    aborted = true;                //  run-time spans than the queue has entries; fail loudly if it does
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

}  // namespace pdattn
