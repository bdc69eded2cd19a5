// Partitioner shared by the host planner and its device twin.
//
// The batch is flattened into a stream of fixed-size token tiles, unit-major (unit = sequence *
// Hkv + kv_head; unit u has ceil(L_s / tile) tiles), and the stream is cut into contiguous spans:
//   - n_static spans, one per CTA;
//   - optionally n_dyn short spans over the last quarter of the stream, handed out at run time, in
//     stream order, to whichever CTA is free; they shrink along the stream (kTaper), so that the
//     ones handed out last are the cheapest.
// Spans are balanced by COST, not by tile count: a unit costs its tiles plus kPieceCostTiles for
// starting it (query rows, page-table row, merge of the warp states, output); a sweep of that
// constant on the 7B-shaped batch put the best value at 2.  In cost coordinates unit u covers
// [C_u, C_u + kPieceCostTiles + nt_u); a cut that falls into the start-up part moves to tile 0.
// A long sequence is thereby split over as many CTAs as its share of the work warrants, a CTA
// that finishes a short sequence carries on with the next one, and only span boundaries ever
// produce partial (m, l, acc) triples.  The cut points depend on the context lengths alone, so
// the result does not depend on which CTA takes which span.
#pragma once
#include <cstdint>

#ifdef __CUDACC__
#define PDATTN_HD __host__ __device__
#else
#define PDATTN_HD
#endif

namespace pdattn {

#ifndef PDATTN_TILE_TOKENS
#define PDATTN_TILE_TOKENS 64     // tokens per tile = per pipeline stage of the decode kernel
#endif
#ifndef PDATTN_PIECE_COST
#define PDATTN_PIECE_COST 2       // cost of starting a unit, in tiles
#endif
constexpr int kTileTokens = PDATTN_TILE_TOKENS;
constexpr int kPieceCostTiles = PDATTN_PIECE_COST;
constexpr int kMaxDynPerCta = 8;      // at most this many run-time spans per CTA
#ifndef PDATTN_DYN_EIGHTHS
#define PDATTN_DYN_EIGHTHS 2
#endif
constexpr int kDynEighths = PDATTN_DYN_EIGHTHS;   // share of the cost stream that is cut into run-time spans, in eighths
#ifndef PDATTN_TAPER
#define PDATTN_TAPER 3
#endif
constexpr int kTaper = PDATTN_TAPER;   // taper of the run-time spans, in quarters (0: equal spans)
constexpr int kMinDynCost = 8;        // a run-time span is never cheaper than this
constexpr int kStaticOnlyBelow = 16;  // less cost per CTA than this: no run-time spans

struct PlanParams {
  int n_static, n_dyn;
  int64_t cost_static;   // cost covered by the static spans
  int64_t cost_total;
  int total;             // all tiles
};

// One span: where it starts and the index of its first tile in the flattened stream.  Span i
// holds spans[i + 1].flat - spans[i].flat tiles, so the table has n_static + n_dyn + 1 entries.
// `merge` describes how the units that span boundaries cut are put together again (see span_merge_info).
struct SpanStart {
  int32_t unit, tile, flat, merge;
};

// Merge word of span k.  A unit that starts in span c and runs past its end is followed by a run of spans that
// begin inside it; each of those that holds tiles produces one partial (m, l, acc), as does span c itself.
//   bits  0..14  as first span of such a unit: bit r set = span c + 1 + r holds tiles (a partial will exist)
//   bits 16..20  ... the length of that run (0 = no unit runs past this span's end; kMergeTooLong = longer than
//                kMaxMergeRun: left to the combine kernel)
//   bits 24..28  as a span that begins inside a unit: how many spans back that unit's first span lies
//                (0 = this span begins at a unit's tile 0; kMergeTooLong = too far back)
constexpr int kMaxMergeRun = 15;
constexpr int kMergeTooLong = 31;
PDATTN_HD inline int merge_hold_mask(int32_t w) { return w & 0x7fff; }
PDATTN_HD inline int merge_run(int32_t w) { return (w >> 16) & 31; }
PDATTN_HD inline int merge_back(int32_t w) { return (w >> 24) & 31; }
// spans: the finished table of n_spans + 1 entries (unit, tile, flat valid)
PDATTN_HD inline int32_t span_merge_info(const SpanStart* spans, int n_spans, int k) {
  const int unit_k = spans[k].unit;
  int32_t w = 0;
  // backwards: the first span of the unit this span begins inside
  if (spans[k].tile > 0) {
    int d = 1;
    while (d <= kMaxMergeRun && k - d > 0 && spans[k - d].unit == unit_k && spans[k - d].tile > 0) ++d;
    // span k - d is now the nearest one that does not begin inside the unit, or we gave up
    const bool found = d <= kMaxMergeRun && !(spans[k - d].unit == unit_k && spans[k - d].tile > 0);
    w |= (found ? d : kMergeTooLong) << 24;
  }
  // forwards: the run of spans that begin inside the unit that holds the last tile of span k, if that unit starts
  // in span k (a unit that started earlier is described by its own first span)
  if (k + 1 < n_spans && spans[k + 1].tile > 0 && spans[k + 1].flat > spans[k].flat) {
    const int u = spans[k + 1].unit;
    const bool starts_here = spans[k].unit < u || (spans[k].unit == u && spans[k].tile == 0);
    if (starts_here) {
      int run = 0, mask = 0;
      while (k + 1 + run < n_spans && spans[k + 1 + run].unit == u && spans[k + 1 + run].tile > 0) {
        if (run < kMaxMergeRun && spans[k + 2 + run].flat > spans[k + 1 + run].flat) mask |= 1 << run;
        ++run;
        if (run > kMaxMergeRun) break;
      }
      w |= mask | ((run > kMaxMergeRun ? kMergeTooLong : run) << 16);
    }
  }
  return w;
}

PDATTN_HD inline PlanParams make_plan_params(int64_t total_cost, int64_t total_tiles, int n_static, int n_dyn_max) {
  PlanParams p;
  p.n_static = n_static;
  p.n_dyn = 0;
  p.cost_total = total_cost;
  p.cost_static = total_cost;
  p.total = static_cast<int>(total_tiles);
  if (n_dyn_max > 0 && total_cost >= static_cast<int64_t>(n_static) * kStaticOnlyBelow) {
    const int64_t cd = total_cost * kDynEighths / 8;
    int64_t d = (cd + n_dyn_max - 1) / n_dyn_max;
    // (the smallest span of the taper, (4 - kTaper) / 4 of the mean, is held to the minimum)
    if (d * (4 - kTaper) < kMinDynCost * 4) d = (kMinDynCost * 4 + 3 - kTaper) / (4 - kTaper);
    p.n_dyn = static_cast<int>((cd + d - 1) / d);
    p.cost_static = total_cost - cd;
  }
  return p;
}
// cost coordinate at which span i begins (i == n_static + n_dyn gives the end of the stream)
PDATTN_HD inline int64_t span_cost_start(const PlanParams& p, int i) {
  if (i <= p.n_static) return p.cost_static * i / p.n_static;
  // run-time spans shrink linearly from (4 + kTaper) / 4 of their mean cost to (4 - kTaper) / 4 of it: the CTAs draw
  // them in this order, so the ones that decide when the last CTA finishes are the small ones
  const int64_t j = i - p.n_static, n = p.n_dyn;
  return p.cost_static + (p.cost_total - p.cost_static) * (j * ((4 + kTaper) * n - kTaper * j)) / (4 * n * n);
}
// cost of one sequence: Hkv units of nt tiles each
PDATTN_HD inline int64_t seq_cost(int64_t nt, int hkv) { return nt > 0 ? (nt + kPieceCostTiles) * hkv : 0; }
// position `r` (cost units) inside a sequence of Hkv units of nt tiles -> (unit within sequence, tile)
PDATTN_HD inline void locate_in_seq(int64_t r, int64_t nt, int* k, int* tile) {
  const int64_t per = nt + kPieceCostTiles;
  *k = static_cast<int>(r / per);
  const int64_t pos = r % per;
  *tile = pos > kPieceCostTiles ? static_cast<int>(pos - kPieceCostTiles) : 0;
}

// spans: [n_static + n_dyn + 1] entries; at most max_spans + 1 are written and n_dyn is lowered
// to fit.  Returns false on invalid arguments.
// start_tiles (may be null): per sequence, leading tiles that this plan leaves out.
bool plan_spans(const int32_t* context_lens, const int32_t* start_tiles, int num_seqs, int num_kv_heads,
                int n_static, int dyn_per_cta, int max_spans, SpanStart* spans, PlanParams* plan);

// tiles of one sequence that a plan covers
PDATTN_HD inline int64_t seq_tiles(int64_t context_len, int64_t start_tile) {
  const int64_t all = context_len > 0 ? (context_len + kTileTokens - 1) / kTileTokens : 0;
  return all > start_tile ? all - start_tile : 0;
}

}  // namespace pdattn
