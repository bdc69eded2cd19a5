// Partitioner shared by the host planner and its device twin.
//
// The batch is flattened into a stream of fixed-size token tiles, unit-major (unit = sequence *
// Hkv + kv_head; unit u has ceil(L_s / tile) tiles), and the stream is cut into contiguous spans:
//   - n_static spans, one per CTA, cover the first three quarters of the stream in equal parts;
//   - n_dyn small spans cover the rest and are handed out at run time to whichever CTA finishes
//     first, because SMs do not all stream at the same speed.
// A long sequence is thereby split over as many CTAs as its share of the bytes warrants, a CTA
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
constexpr int kTileTokens = PDATTN_TILE_TOKENS;
constexpr int kMaxDynPerCta = 8;      // at most this many run-time spans per CTA
constexpr int kMinDynTiles = 4;       // a run-time span is never shorter than this
constexpr int kStaticOnlyBelow = 16;  // fewer tiles per CTA than this: no run-time spans

struct PlanParams {
  int n_static, n_dyn;
  int qs, rs;          // static span i holds qs + (i < rs) tiles
  int qd, rd;          // run-time span j holds qd + (j < rd) tiles
  int total_static;    // tiles covered by the static spans
  int total;           // all tiles
};

PDATTN_HD inline PlanParams make_plan_params(int64_t total_tiles, int n_static, int n_dyn_max) {
  PlanParams p;
  p.n_static = n_static;
  p.total = static_cast<int>(total_tiles);
  int64_t ts = total_tiles, td = 0;
  p.n_dyn = p.qd = p.rd = 0;
  if (n_dyn_max > 0 && total_tiles >= static_cast<int64_t>(n_static) * kStaticOnlyBelow) {
    td = total_tiles / 4;
    ts = total_tiles - td;
    int64_t d = (td + n_dyn_max - 1) / n_dyn_max;
    if (d < kMinDynTiles) d = kMinDynTiles;
    p.n_dyn = static_cast<int>((td + d - 1) / d);
    p.qd = static_cast<int>(td / p.n_dyn);
    p.rd = static_cast<int>(td % p.n_dyn);
  }
  p.qs = static_cast<int>(ts / n_static);
  p.rs = static_cast<int>(ts % n_static);
  p.total_static = static_cast<int>(ts);
  return p;
}
PDATTN_HD inline int span_len(const PlanParams& p, int i) {
  if (i < p.n_static) return p.qs + (i < p.rs ? 1 : 0);
  const int j = i - p.n_static;
  return p.qd + (j < p.rd ? 1 : 0);
}
// index of the span's first tile in the flattened stream
PDATTN_HD inline int span_start(const PlanParams& p, int i) {
  if (i < p.n_static) return i * p.qs + (i < p.rs ? i : p.rs);
  const int j = i - p.n_static;
  return p.total_static + j * p.qd + (j < p.rd ? j : p.rd);
}

// spans: [2 * (n_static + n_dyn)] = (unit0, tile0) per span; at most 2 * max_spans ints are
// written and n_dyn is lowered to fit.  Returns false on invalid arguments.
bool plan_spans(const int32_t* context_lens, int num_seqs, int num_kv_heads, int n_static, int dyn_per_cta,
                int max_spans, int32_t* spans, PlanParams* plan);

}  // namespace pdattn
