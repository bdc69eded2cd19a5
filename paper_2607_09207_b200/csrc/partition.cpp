#include "partition.h"

namespace pdattn {

bool plan_spans(const int32_t* context_lens, int num_seqs, int num_kv_heads, int n_ctas,
                int32_t* spans, Plan* plan) {
  if (num_seqs < 0 || num_kv_heads <= 0 || n_ctas <= 0 || !spans || !plan) return false;
  if (num_seqs > 0 && !context_lens) return false;
  int64_t total = 0;
  for (int s = 0; s < num_seqs; ++s) {
    int64_t L = context_lens[s] > 0 ? context_lens[s] : 0;
    total += (L + kTileTokens - 1) / kTileTokens * num_kv_heads;
  }
  if (total > INT32_MAX) return false;
  plan->total_tiles = total;
  plan->tiles_q = static_cast<int>(total / n_ctas);
  plan->tiles_r = static_cast<int>(total % n_ctas);

  // One pass over the sequences, emitting span starts as the running tile index passes them.
  int c = 0;
  int64_t next_start = 0;   // global tile index where span c begins
  int64_t base = 0;         // global tile index of the current sequence's first tile
  for (int s = 0; s < num_seqs && c < n_ctas; ++s) {
    int64_t L = context_lens[s] > 0 ? context_lens[s] : 0;
    int64_t nt = (L + kTileTokens - 1) / kTileTokens;
    int64_t seq_tiles = nt * num_kv_heads;
    while (c < n_ctas && next_start < base + seq_tiles) {
      int64_t off = next_start - base;
      spans[2 * c] = static_cast<int32_t>(static_cast<int64_t>(s) * num_kv_heads + off / nt);
      spans[2 * c + 1] = static_cast<int32_t>(off % nt);
      int len = plan->tiles_q + (c < plan->tiles_r ? 1 : 0);
      if (len == 0) break;          // only empty spans remain
      next_start += len;
      ++c;
    }
    base += seq_tiles;
  }
  for (; c < n_ctas; ++c) {         // spans with no tiles
    spans[2 * c] = num_seqs * num_kv_heads;
    spans[2 * c + 1] = 0;
  }
  return true;
}

}  // namespace pdattn
