#include "partition.h"

namespace pdattn {

bool plan_spans(const int32_t* context_lens, int num_seqs, int num_kv_heads, int n_static, int dyn_per_cta,
                int max_spans, int32_t* spans, PlanParams* plan) {
  if (num_seqs < 0 || num_kv_heads <= 0 || n_static <= 0 || max_spans < n_static || !spans || !plan) return false;
  if (dyn_per_cta < 0 || dyn_per_cta > kMaxDynPerCta) return false;
  if (num_seqs > 0 && !context_lens) return false;
  int64_t total = 0;
  for (int s = 0; s < num_seqs; ++s) {
    int64_t L = context_lens[s] > 0 ? context_lens[s] : 0;
    total += (L + kTileTokens - 1) / kTileTokens * num_kv_heads;
  }
  if (total > INT32_MAX) return false;
  int n_dyn_max = n_static * dyn_per_cta;
  if (n_dyn_max > max_spans - n_static) n_dyn_max = max_spans - n_static;
  const PlanParams p = make_plan_params(total, n_static, n_dyn_max);
  *plan = p;
  const int n_spans = p.n_static + p.n_dyn;

  // One pass over the sequences, emitting span starts as the running tile index passes them.
  int c = 0;
  int64_t base = 0;   // flattened index of the current sequence's first tile
  for (int s = 0; s < num_seqs && c < n_spans; ++s) {
    int64_t L = context_lens[s] > 0 ? context_lens[s] : 0;
    int64_t nt = (L + kTileTokens - 1) / kTileTokens;
    int64_t seq_tiles = nt * num_kv_heads;
    while (c < n_spans) {
      if (span_len(p, c) == 0) {            // only possible for trailing static spans of a tiny batch
        spans[2 * c] = num_seqs * num_kv_heads;
        spans[2 * c + 1] = 0;
        ++c;
        continue;
      }
      const int64_t start = span_start(p, c);
      if (start >= base + seq_tiles) break;
      const int64_t off = start - base;
      spans[2 * c] = static_cast<int32_t>(static_cast<int64_t>(s) * num_kv_heads + off / nt);
      spans[2 * c + 1] = static_cast<int32_t>(off % nt);
      ++c;
    }
    base += seq_tiles;
  }
  for (; c < n_spans; ++c) {
    spans[2 * c] = num_seqs * num_kv_heads;
    spans[2 * c + 1] = 0;
  }
  return true;
}

}  // namespace pdattn
