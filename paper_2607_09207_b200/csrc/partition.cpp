#include "partition.h"

namespace pdattn {

bool plan_spans(const int32_t* context_lens, const int32_t* start_tiles, int num_seqs, int num_kv_heads,
                int n_static, int dyn_per_cta, int max_spans, SpanStart* spans, PlanParams* plan) {
  if (num_seqs < 0 || num_kv_heads <= 0 || n_static <= 0 || max_spans < n_static || !spans || !plan) return false;
  if (dyn_per_cta < 0 || dyn_per_cta > kMaxDynPerCta) return false;
  if (num_seqs > 0 && !context_lens) return false;
  int64_t total = 0, cost = 0;
  for (int s = 0; s < num_seqs; ++s) {
    const int64_t nt = seq_tiles(context_lens[s], start_tiles ? start_tiles[s] : 0);
    total += nt * num_kv_heads;
    cost += seq_cost(nt, num_kv_heads);
  }
  if (total > INT32_MAX / 2) return false;
  int n_dyn_max = n_static * dyn_per_cta;
  if (n_dyn_max > max_spans - n_static) n_dyn_max = max_spans - n_static;
  const PlanParams p = make_plan_params(cost, total, n_static, n_dyn_max);
  *plan = p;
  const int n_spans = p.n_static + p.n_dyn;

  // One pass over the sequences, emitting span starts as the running cost passes them.
  int c = 0;
  int64_t cbase = 0;   // cost coordinate of the current sequence's start
  int64_t tbase = 0;   // flattened tile index of its first tile
  for (int s = 0; s < num_seqs && c < n_spans; ++s) {
    const int64_t nt = seq_tiles(context_lens[s], start_tiles ? start_tiles[s] : 0);
    const int64_t sc = seq_cost(nt, num_kv_heads);
    while (c < n_spans) {
      const int64_t x = span_cost_start(p, c);
      if (x >= cbase + sc) break;
      int k, tile;
      locate_in_seq(x - cbase, nt, &k, &tile);
      spans[c].unit = static_cast<int32_t>(static_cast<int64_t>(s) * num_kv_heads + k);
      spans[c].tile = tile;
      spans[c].flat = static_cast<int32_t>(tbase + static_cast<int64_t>(k) * nt + tile);
      spans[c].merge = 0;
      ++c;
    }
    cbase += sc;
    tbase += nt * num_kv_heads;
  }
  for (; c <= n_spans; ++c) {         // spans past the end of the stream, and the end marker
    spans[c].unit = num_seqs * num_kv_heads;
    spans[c].tile = 0;
    spans[c].flat = static_cast<int32_t>(total);
    spans[c].merge = 0;
  }
  for (int k = 0; k < n_spans; ++k) spans[k].merge = span_merge_info(spans, n_spans, k);
  return true;
}

}  // namespace pdattn
