// Host partitioner: flattens the batch into a stream of fixed-size token tiles, unit-major
// (unit = sequence * Hkv + kv_head), and cuts the stream into n_ctas contiguous spans whose
// lengths differ by at most one tile.  A long sequence is thereby split over as many CTAs as
// its share of the bytes warrants, and a CTA that finishes a short sequence carries on with
// the next one, so only span boundaries ever produce partial (m, l, acc) triples.
#pragma once
#include <cstdint>

namespace pdattn {

#ifndef PDATTN_TILE_TOKENS
#define PDATTN_TILE_TOKENS 64     // tokens per tile = per pipeline stage of the decode kernel
#endif
constexpr int kTileTokens = PDATTN_TILE_TOKENS;

struct Plan {
  int64_t total_tiles;
  int tiles_q;   // every span holds tiles_q tiles ...
  int tiles_r;   // ... and the first tiles_r spans one more
};

// spans: [2 * n_ctas] = (unit0, tile0) per span.  Returns false on invalid arguments.
bool plan_spans(const int32_t* context_lens, int num_seqs, int num_kv_heads, int n_ctas,
                int32_t* spans, Plan* plan);

}  // namespace pdattn
