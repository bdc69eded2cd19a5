/*
 * libpdattn -- paged decode attention for RL rollout on NVIDIA B200 (sm_100a).
 *
 * One call = one layer's attention for one autoregressive decode step of a whole rollout
 * batch: a single query token per sequence attends over that sequence's history in a paged
 * bf16 KV cache (the "autoregressive decoding" of the rollout stage, Section 2.1 and Section 2.3
 * of the paper; the cache's per-token size is the b_kv formula of Appendix A.1.2, and the cost
 * the paper models as linear in history tokens is the beta_hist * H_dec term of the same appendix).
 *
 *     out[s,h,:] = softmax_t( scale * <q[s,h,:], K_s[t, h/G, :]> ) . V_s[t, h/G, :],  t in [0, L_s)
 *
 * G = num_q_heads / num_kv_heads; token t of sequence s is slot t % block_size of physical page
 * block_table[s, t / block_size]; L_s = context_lens[s] counts the current token (its K/V are
 * already in the cache).  Scores and accumulation are fp32, the output is rounded to bf16
 * (nearest even).
 *
 * Conventions for every entry point
 *   - C ABI, no exceptions, no aborts: a negative pdattn_status reports failure.
 *   - Pointers marked DEVICE must be device memory of the current device, HOST ordinary host
 *     memory.  All memory is caller-owned; the library never allocates, frees or keeps device
 *     memory, creates no streams, and synchronises only where stated.
 *   - Work is enqueued on `stream`; outputs are valid once the stream reaches that point.
 *   - State.  Per thread: the binding made by pdattn_bind(), the events of pdattn_profile_events(), the
 *     launch count and the text of the last CUDA failure.  Process-wide: the five tuning settings
 *     pdattn_set_dynamic_spans / _merge_mode / _short_piece_path / _prefix_engine / _host_zero_copy (plain ints; set them
 *     before the threads that decode start, not concurrently with a call).
 */
#ifndef PDATTN_H_
#define PDATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int pdattn_status;
#define PDATTN_OK                   0
#define PDATTN_INVALID_ARG         (-1) /* null pointer, negative size, Hq % Hkv != 0, ...           */
#define PDATTN_UNSUPPORTED         (-2) /* head_dim not in {64,128}, block_size not in {16,32,64}, G > 16, or a
                                           cache stride that is not a multiple of 8 elements          */
#define PDATTN_WORKSPACE_TOO_SMALL (-3)
#define PDATTN_MISALIGNED          (-4) /* q / k_cache / v_cache / out not 16-byte aligned, or workspace /
                                           staging not 256-byte aligned                              */
#define PDATTN_NOT_BOUND           (-5) /* pdattn_decode() without pdattn_bind() on this thread       */
#define PDATTN_CUDA_ERROR          (-6) /* a CUDA call failed; text in pdattn_last_cuda_error()       */
#define PDATTN_BAD_PAGE_INDEX      (-7) /* reported by pdattn_check(): a used block_table entry was
                                           outside [0, num_blocks)                                   */
#define PDATTN_DEVICE_TIMEOUT      (-8) /* reported by pdattn_check(): a bounded wait inside a kernel
                                           gave up; that call's output is undefined                  */

typedef struct CUstream_st* pdattn_stream_t; /* a cudaStream_t */

/*
 * Size of the scratch area a decode call needs (the partial (m, l, acc) triples of split
 * sequences, the per-CTA work spans and one sticky error word).  Splitting exists because of the
 * length skew of rollout batches (Section 2.3: a few long responses dominate the decoding time), so
 * the size depends on the head shape and the SM count, not on the context lengths.  max_context_len is accepted
 * for forward compatibility and does not change the result today.  pinned_host_bytes (optional)
 * receives 0: no pinned staging is needed.
 */
pdattn_status pdattn_workspace_size(int num_seqs, int num_q_heads, int num_kv_heads, int head_dim,
                                    int block_size, int max_context_len,
                                    size_t* device_bytes, size_t* pinned_host_bytes);

/*
 * Clear the words of the workspace that must be zero before its first use (error word, span counter, the
 * ticket words of the in-kernel merge: the first 8448 bytes).  Call once after allocating a workspace, and at
 * will later while no call that uses the workspace is in flight; enqueued on `stream`.  workspace: DEVICE.
 */
pdattn_status pdattn_workspace_init(void* workspace, size_t workspace_bytes, pdattn_stream_t stream);

/* All arguments of one decode step.  Strides are in ELEMENTS; head_dim is contiguous. */
typedef struct {
  const void* q;                    /* DEVICE bf16 [num_seqs, num_q_heads, head_dim], dense          */
  const void* k_cache;              /* DEVICE bf16, element (page, kv_head, slot, j) at               */
  const void* v_cache;              /*   page*kv_block_stride + kv_head*kv_head_stride +              */
                                    /*   slot*kv_token_stride + j.  Both caches use the same strides. */
  void* out;                        /* DEVICE bf16 [num_seqs, num_q_heads, head_dim], dense          */
  const int32_t* block_table;       /* DEVICE int32 [num_seqs, max_blocks_per_seq], row-major.        */
                                    /*   Entries at or past ceil(L_s/block_size) are never read.      */
  const int32_t* context_lens;      /* DEVICE int32 [num_seqs]; L_s <= max_blocks_per_seq * block_size */
  const int32_t* context_lens_host; /* HOST copy of context_lens for the host partitioner, or NULL:   */
                                    /*   then a small planning kernel runs on the device instead.      */
                                    /*   Read during the call only.  Must equal the device array.      */
  int num_seqs, num_q_heads, num_kv_heads, head_dim, block_size;
  int max_blocks_per_seq;           /* row stride of block_table                                      */
  int num_blocks;                   /* pages in each pool; used entries must be in [0, num_blocks)    */
  int64_t kv_block_stride, kv_head_stride, kv_token_stride;
  float scale;                      /* multiplies q.k before the softmax                              */
  void* workspace;                  /* DEVICE, >= pdattn_workspace_size() bytes, 256-byte aligned     */
  size_t workspace_bytes;
} pdattn_args;

/*
 * The decode step (Section 2.3's decoding loop body, attention part).  Launches the split-KV
 * kernel and the split-combine kernel on `stream`; never synchronises.
 *   - num_seqs == 0: PDATTN_OK, nothing launched.  L_s == 0: out[s] = +0.
 *   - The same page may appear in many rows (shared prompt pages of a GRPO group) or twice in one.
 *   - Cache slots at or past L_s and pages no row references may hold anything (NaN included)
 *     and do not influence `out`.
 *   - A used block_table entry outside [0, num_blocks) is not dereferenced: its tokens are left
 *     out of the softmax and the workspace's sticky error word is set (see pdattn_check).
 *   - A context length beyond max_blocks_per_seq * block_size (more tokens than the table row can
 *     describe) is refused with PDATTN_INVALID_ARG when context_lens_host is given.  Without the host
 *     copy the entries past the row's end are never read: those tokens are treated like a bad page
 *     (left out, error word set).
 *   - The result is a pure function of the logical inputs: bit-identical from run to run, under
 *     any renumbering of physical pages, and for shared versus privately copied prefix pages.
 *   - Two calls that share a workspace must not overlap on the GPU.
 */
pdattn_status pdattn_decode_ex(const pdattn_args* args, pdattn_stream_t stream);

/*
 * Decode step for GRPO sample groups (Section 2.1: several responses are sampled per prompt and form
 * a prompt-level group; Section 7.1 uses 8 per prompt).  Sequences g*group_size .. (g+1)*group_size-1
 * form group g and share their first prefix_tiles[g] * 64 tokens: their block_table rows must hold
 * the SAME page ids for those tokens.  The shared tiles are then streamed from HBM once per group
 * and KV head and scored against the query rows of all samples (group_size * G rows at a time),
 * and every sequence continues with its own pages; results equal pdattn_decode_ex's definition
 * (within rounding: the summation order differs) and are bit-identical from run to run.
 *   prefix_tiles      DEVICE int32 [num_seqs / group_size]; prefix_tiles_host its HOST copy.
 *   Requirements: args->context_lens_host given; num_seqs a multiple of group_size; G <= 8 and
 *   group_size * G <= 64 (48 with pdattn_set_prefix_engine(0)), else PDATTN_UNSUPPORTED -- a larger
 *   group is passed as several groups of a divisor of its size with the same prefix_tiles entry (its
 *   shared tiles are then read once per part);
 *   every member of group g has context_len > prefix_tiles[g] * 64
 *   (it owns at least its current token); 0 is allowed (the group shares nothing).
 *   args->workspace must hold pdattn_grouped_workspace_size() bytes.
 * The caller vouches for the page ids being shared; if they are not, the group's first row is
 * used for the shared tiles of all its members.
 */
pdattn_status pdattn_grouped_workspace_size(int num_seqs, int num_q_heads, int num_kv_heads, int head_dim,
                                            int block_size, size_t* device_bytes);
pdattn_status pdattn_decode_grouped(const pdattn_args* args, int group_size, const int32_t* prefix_tiles,
                                    const int32_t* prefix_tiles_host, pdattn_stream_t stream);

/*
 * Decode step with several query tokens per sequence: the last num_query_tokens tokens of every
 * sequence are new (their K/V are already in the cache and counted in context_lens, as the single
 * current token is in pdattn_decode_ex), e.g. the rows of a speculative-verification or chunked step
 * of the rollout engine (Section 2.1 only says that rollouters decode autoregressively; the paper has
 * no counterpart for this variant).  Query token j (0 <= j < T) sits at position context_len - T + j
 * and attends to the keys at positions <= its own (causal among the new tokens):
 *   out[s, j, h, :] = softmax_t( scale * q[s, j, h, :] . K[t, h / G, :] ) . V[t, h / G, :],  t < context_len - (T - 1 - j)
 * Layouts: args->q and args->out are DEVICE bf16 [num_seqs, T, num_q_heads, head_dim], dense; all else
 * as in pdattn_decode_ex.  The T * G query rows of a KV head share its K/V tiles (read once).
 * A query token that sees no key (context_len < T - j) gets zeros.
 *   Requirements: T >= 1, T * G <= 16; args->workspace holds pdattn_multi_workspace_size() bytes
 *   (pdattn_workspace_size() is enough while T * G <= 8).  T = 1 is pdattn_decode_ex.
 *   PDATTN_UNSUPPORTED for T * G > 16.
 */
pdattn_status pdattn_multi_workspace_size(int num_seqs, int num_q_heads, int num_kv_heads, int head_dim,
                                          int block_size, int num_query_tokens, size_t* device_bytes);
pdattn_status pdattn_decode_multi(const pdattn_args* args, int num_query_tokens, pdattn_stream_t stream);

/*
 * Decode step over an fp8 KV cache.  Appendix A.1.2 gives the per-token KV footprint as
 * b_kv = 2 L H_kv d_head b_dtype / tp and the decode cost as beta_hist per history token read: with
 * one-byte cache elements both halve.  K and V are stored as e4m3 codes (1 sign, 4 exponent, 3 mantissa
 * bits, finite-only variant) with one fp32 scale per KV head: value = scale[kv head] * e4m3(code).
 *   args->k_cache   DEVICE uint8 [num_blocks, num_kv_heads, block_size, head_dim]
 *   args->v_cache   DEVICE uint8 [num_blocks, num_kv_heads, head_dim, block_size]   (V transposed inside a page)
 *   k_scale, v_scale  DEVICE fp32 [num_kv_heads]
 * Both pools dense (the stride fields of args are ignored); everything else as in pdattn_decode_ex,
 * including the treatment of bad page ids and of slots past the end (any code, NaN codes too).
 * The codes are widened exactly; q is rounded to fp16 for the products (values below 2^-14 lose bits) and
 * the softmax weights to fp16 (11 bits), accumulation in fp32; out is bf16.
 *   Requirements: head_dim 128 or 64, every page size of pdattn_decode_ex.  Workspace as for pdattn_decode_ex.
 */
pdattn_status pdattn_decode_fp8(const pdattn_args* args, const float* k_scale, const float* v_scale,
                                pdattn_stream_t stream);
/* The same with num_query_tokens new tokens per sequence: pdattn_decode_multi's definition and layouts
 * (q, out [num_seqs, T, num_q_heads, head_dim]; T * G <= 16; pdattn_multi_workspace_size) over the fp8 cache. */
pdattn_status pdattn_decode_fp8_multi(const pdattn_args* args, int num_query_tokens, const float* k_scale,
                                      const float* v_scale, pdattn_stream_t stream);

/*
 * pdattn_decode_grouped over the fp8 cache of pdattn_decode_fp8 (GRPO prompt groups, Section 2.1, with the one-byte
 * cache elements of Appendix A.1.2's b_dtype): same group rules, same workspace size, same layouts as
 * pdattn_decode_fp8.  The shared tiles are scored with warp-level MMAs on the widened codes, eight query rows per
 * warp, so group_size * G <= 48 (else PDATTN_UNSUPPORTED; pass a larger group as several smaller ones).
 */
pdattn_status pdattn_decode_grouped_fp8(const pdattn_args* args, int group_size, const int32_t* prefix_tiles,
                                        const int32_t* prefix_tiles_host, const float* k_scale, const float* v_scale,
                                        pdattn_stream_t stream);

/*
 * KV append into the fp8 cache of pdattn_decode_fp8 (same layouts): the rows k_new[s], v_new[s] (DEVICE
 * bf16 [num_seqs, num_kv_heads, head_dim]) are divided by their KV head's scale, rounded to e4m3 (nearest
 * even; magnitudes beyond the largest finite code 448 saturate to it) and written at position
 * context_lens[s], which then becomes context_lens[s] + 1.  Page rules and error reporting as in
 * pdattn_append_kv.  head_dim 128 or 64.
 */
pdattn_status pdattn_append_kv_fp8(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                   const float* k_scale, const float* v_scale, const int32_t* block_table,
                                   int32_t* context_lens, int num_seqs, int num_kv_heads, int head_dim,
                                   int block_size, int max_blocks_per_seq, int num_blocks, void* workspace,
                                   pdattn_stream_t stream);

/*
 * KV append: the step that precedes attention in the decoding loop (Section 2.3; the cache grows by
 * b_kv bytes per token and layer, Appendix A.1.2).  For every sequence s with t = context_lens[s]:
 * the rows k_new[s], v_new[s] (DEVICE bf16 [num_seqs, num_kv_heads, head_dim], dense) are written to
 * slot t % block_size of page block_table[s, t / block_size] of the caches (same strides as
 * pdattn_args), and context_lens[s] becomes t + 1 (DEVICE, updated in place).  The page must
 * already be in the table: page allocation stays with the caller.  A sequence whose target page id
 * is outside [0, num_blocks), or whose table row is full, is left untouched and, if `workspace`
 * (DEVICE, may be NULL) is given, its sticky error word is set (see pdattn_check).
 * Followed by pdattn_decode_ex with context_lens_host = NULL, a whole decode step needs no host
 * work that depends on the lengths.
 */
pdattn_status pdattn_append_kv(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                               const int32_t* block_table, int32_t* context_lens, int num_seqs,
                               int num_kv_heads, int head_dim, int block_size, int max_blocks_per_seq,
                               int num_blocks, int64_t kv_block_stride, int64_t kv_head_stride,
                               int64_t kv_token_stride, void* workspace, pdattn_stream_t stream);

/*
 * Thread-local binding of the arguments the short form below does not carry: the block table's row
 * stride and the pool size (the paged cache of Appendix A.1.2's b_kv bytes per token), the workspace,
 * and the optional host copy of the lengths.  context_lens_host may be NULL.  The pointers must stay
 * valid while bound.  (No pinned-host arguments: the library needs no pinned staging.)
 */
pdattn_status pdattn_bind(int max_blocks_per_seq, int num_blocks, void* workspace,
                          size_t workspace_bytes, const int32_t* context_lens_host);

/*
 * Short form of the decode step (the attention part of the rollout's decoding loop, Section 2.1 and
 * Section 2.3, with the arguments of the problem statement): dense caches
 * [num_blocks, num_kv_heads, block_size, head_dim]; everything else as pdattn_decode_ex with the values
 * bound on this thread.  PDATTN_NOT_BOUND without a binding.
 */
pdattn_status pdattn_decode(const void* q, const void* k_cache, const void* v_cache,
                            const int32_t* block_table, const int32_t* context_lens,
                            int num_seqs, int num_q_heads, int num_kv_heads, int head_dim,
                            int block_size, float scale, void* out, pdattn_stream_t stream);

/*
 * End-to-end form for a caller whose per-step inputs live in HOST memory (pinned for real
 * asynchrony): copies q, block_table and context_lens to the device staging area, runs
 * pdattn_decode_ex (host partitioner on context_lens_host = the given lengths), copies `out`
 * back.  All on `stream`; the caller synchronises.  The KV pools are resident device state.
 * staging: DEVICE, >= pdattn_host_staging_size() bytes, 256-byte aligned.
 * When q_host and out_host are both pinned, mapped host memory (cudaHostAlloc / cudaHostRegister; 16-byte
 * aligned) the kernels read q and write out in place over the bus instead of through the two copies --
 * same results bit for bit; out_host is complete once `stream` has been synchronised.
 * pdattn_set_host_zero_copy(0) always takes the copies; -1 (default) and 1: in place when possible.
 */
pdattn_status pdattn_set_host_zero_copy(int mode);
pdattn_status pdattn_host_staging_size(int num_seqs, int num_q_heads, int head_dim,
                                       int max_blocks_per_seq, size_t* device_bytes);
pdattn_status pdattn_decode_host(const void* q_host, const int32_t* block_table_host,
                                 const int32_t* context_lens_host, void* out_host,
                                 const void* k_cache, const void* v_cache,
                                 int num_seqs, int num_q_heads, int num_kv_heads, int head_dim,
                                 int block_size, int max_blocks_per_seq, int num_blocks, float scale,
                                 void* staging, size_t staging_bytes,
                                 void* workspace, size_t workspace_bytes, pdattn_stream_t stream);

/*
 * pdattn_decode_host over the fp8 cache of pdattn_decode_fp8: k_cache / v_cache are the DEVICE code pools in that
 * entry point's layouts, k_scale / v_scale DEVICE fp32 [num_kv_heads]; everything else as pdattn_decode_host
 * (the per-step inputs q, block_table, context_lens and the result `out` live in HOST memory; same staging size).
 */
pdattn_status pdattn_decode_host_fp8(const void* q_host, const int32_t* block_table_host,
                                     const int32_t* context_lens_host, void* out_host,
                                     const void* k_cache, const void* v_cache, const float* k_scale,
                                     const float* v_scale, int num_seqs, int num_q_heads, int num_kv_heads,
                                     int head_dim, int block_size, int max_blocks_per_seq, int num_blocks, float scale,
                                     void* staging, size_t staging_bytes,
                                     void* workspace, size_t workspace_bytes, pdattn_stream_t stream);

/*
 * The host partitioner on its own (no GPU needed).  It flattens the batch into a stream of
 * 64-token tiles, unit-major (unit = s * num_kv_heads + kv_head; unit u has ceil(L_s / 64)
 * tiles), and cuts it into contiguous spans so that long-tail sequences are spread over all SMs
 * (Section 2.3: a few long responses dominate the rollout).  Spans are balanced by cost: a unit
 * costs its tiles plus 2 for starting it, so a CTA that walks many short sequences gets fewer
 * tiles than one inside a long sequence.  n_static spans, one per CTA, cover the stream; with
 * dynamic_per_cta > 0 they cover only its first three quarters (by cost) and up to n_ctas *
 * dynamic_per_cta short spans cover the rest, taken at run time, in stream order, by whichever CTA is free;
 * their cost falls linearly along the stream from 1.75 to 0.25 of their mean, and there are no more of them
 * than keeps the smallest at 8 cost units.
 * spans: HOST int32 [4 * (max_spans + 1)], one (unit, tile, flat, merge) entry per span plus an end
 * marker: span i starts at tile `tile` of unit `unit`, which is tile number `flat` of the stream,
 * and holds flat[i + 1] - flat[i] tiles (possibly none).  n_static + n_dynamic <= max_spans.
 * `merge` says how a unit that span boundaries cut is put together again: bits 16-20 the number of spans
 * right behind span i that begin inside the unit that starts in span i and runs past its end (0 = none,
 * 31 = more than 15), bits 0-14 which of those hold tiles (each writes one partial), bits 24-28, for a span
 * that begins inside a unit, how many spans back that unit's first span lies (31 = more than 15).
 * The plan depends on the context lengths only, never on page ids.
 */
typedef struct {
  int n_static, n_dynamic;
  int total_tiles;
} pdattn_plan;
pdattn_status pdattn_plan_host(const int32_t* context_lens_host, int num_seqs, int num_kv_heads,
                               int n_ctas, int dynamic_per_cta, int max_spans, int32_t* spans,
                               pdattn_plan* plan);

/*
 * Process-wide tuning of the partitioner above: at most `per_cta` run-time spans per CTA (0..8; 0 = every
 * span is static).  -1 (default): 4 when the batch has at least 4 units (sequence x KV head) per CTA, else 0 --
 * run-time spans even out the finishing times of the CTAs when there are many units, and only lengthen
 * the merge of cut sequences when there are few long ones.  Results stay bit-identical from run to run for
 * a given setting and batch shape; different settings cut sequences at different tiles.
 */
pdattn_status pdattn_set_dynamic_spans(int per_cta);

/*
 * Process-wide choice of how partial online-softmax states (m, l, acc) are merged (the split-combine of the
 * split-KV method; no paper counterpart beyond the decoding step of Section 2.3).  Two places merge:
 *   - inside a CTA, at the end of a piece (a sequence's run of tiles inside one span), the states of its
 *     consumer warps: "chained" hands the state down a chain of warps through shared memory and no warp waits
 *     for the others, so several short pieces are in work at once; "barrier" makes all warps meet and sum
 *     together (same cost on long pieces, one barrier round per piece on batches of short contexts);
 *   - across CTAs, the partials of a sequence that span boundaries cut: either inside the decode kernel, by
 *     whichever CTA writes the unit's last partial (found with one atomic ticket per unit; no CTA waits for
 *     another; units cut into more than 16 consecutive spans are left to the combine kernel), or by the separate
 *     combine kernel launched behind it.
 * mode 1: chained + merge of cut units inside the decode kernel (one launch per step when every chain is short
 * enough and context_lens_host is given); mode 2: chained + combine kernel; mode 0: barrier + combine kernel;
 * -1 (default): 1 when context_lens_host is given and the batch averages at least 8 tiles (512 tokens) per
 * sequence and KV head, else 2 (on batches of short ragged sequences the in-kernel merge costs more than the
 * launch it saves).  In every mode the order of every sum is fixed by tile and span indices, so a setting's
 * results are bit-identical from run to run and under any renumbering of the physical pages.
 */
pdattn_status pdattn_set_merge_mode(int mode);

/*
 * Process-wide choice of the decode kernel's instantiation for batches of very short contexts (early in a rollout
 * most sequences are a tile or two long: Section 2.3's length skew seen from its short end; no paper counterpart).
 * In the short-piece instantiation every warp walks the work spans 32 sequences x KV heads at a time (one load of
 * the lengths, one warp scan, one ballot) instead of piece by piece, and a warp of its own stages the query rows.
 * It applies to the chained merge over a bf16 cache with at most 8 query rows per KV head and context_lens_host
 * given; cut sequences are merged by the combine kernel.  -1 (default): used below 1.5 tiles (96 tokens) per
 * sequence and KV head on average; 0: never; 1: whenever it applies.  Results are the same bits either way.
 */
pdattn_status pdattn_set_short_piece_path(int mode);

/*
 * Process-wide choice of the kernel that pdattn_decode_grouped runs over the shared prompt tiles.
 * 1: the tile products run on tcgen05 tensor cores with accumulators in tensor memory (all
 * group_size * G query rows of a group against a 64-token tile in one operand).  0: warp-level
 * MMAs, eight rows per warp.  -1 (default): 1.  The paper has no counterpart; both compute the same
 * partial (m, l, acc) per (sequence, KV head) and differ only in rounding order.
 */
pdattn_status pdattn_set_prefix_engine(int engine);

/*
 * Error report of the decode steps enqueued so far (no paper counterpart; the rollout loop of Section 2.3
 * would call it once per step or less).  Synchronises `stream`, reads and clears the workspace's sticky
 * error word (hence a non-const pointer).  Returns PDATTN_OK, PDATTN_BAD_PAGE_INDEX, PDATTN_DEVICE_TIMEOUT, or
 * PDATTN_UNSUPPORTED when the device-side planner refused a batch of more than 2^30 tiles (with
 * context_lens_host the call itself returns PDATTN_INVALID_ARG for such a batch); that call computed nothing.
 * workspace: DEVICE.
 */
pdattn_status pdattn_check(void* workspace, pdattn_stream_t stream);

/*
 * Decode step for callers that cannot give the library any scratch memory and cannot let it
 * allocate.  (The paper has no counterpart for this entry point; it is a deployment variant of
 * pdattn_decode_ex.)  Meant for hosts where every byte of device memory was handed to the
 * engine's KV-cache pool at start-up, so a cudaMalloc at decode time fails or fragments the pool,
 * and for plug-in contexts whose owner forbids device allocation inside the step function.
 *
 * Same computation, same arguments and same results as pdattn_decode_ex, except:
 *   - args->workspace and args->workspace_bytes are ignored.  The partial (m, l, acc) triples, the
 *     per-span records and the error word live in a 4 MiB array built into the library image; every
 *     GPU that loads the library holds that array until the process exits.
 *   - Limits: num_seqs <= 65536 and the layout must fit the 4 MiB (it does for every supported
 *     head configuration on a B200); otherwise PDATTN_WORKSPACE_TOO_SMALL is returned and
 *     pdattn_last_cuda_error() says how many bytes were needed.  Spans are always static.
 *   - status_out (DEVICE int32, optional): receives 0, or the error bits of this call
 *     (1 = a used block_table entry was out of range, 2 = a bounded wait expired), on `stream`.
 *   - The first call on a device looks up the array's device address (one-time set-up, no
 *     allocation); make that first call before any stream capture is begun.  The address is cached
 *     per device for the life of the process and does not survive a cudaDeviceReset.
 *   - All calls on a device share the one array and it keeps the previous call's contents (the
 *     library clears the words that must start at zero).  Two calls that overlap on the GPU, from
 *     different streams or threads, race on it: serialise them, or use pdattn_decode_ex with
 *     separate workspaces.
 * Calls no cudaMalloc / cudaFree and no allocating library routine.
 */
pdattn_status pdattn_decode_static_scratch(const pdattn_args* args, int32_t* status_out,
                                           pdattn_stream_t stream);

/*
 * Measurement aid (roofline accounting of the split-KV kernel, Appendix A.1.2's history-token
 * term being the bytes it moves): while two CUDA events are registered on this thread, every
 * decode call records `start` just before and `stop` just after the split-KV kernel on its
 * stream.  start / stop are cudaEvent_t handles owned by the caller; pass NULLs to stop.
 */
pdattn_status pdattn_profile_events(void* start_event, void* stop_event);

/*
 * Bandwidth ceilings for the same roofline accounting (no paper counterpart beyond the bytes of
 * Appendix A.1.2's per-token footprint): measurement aids, they compute nothing.
 *   pdattn_gather_probe      : the decode step's exact memory access stream (same partition, page
 *                              lookups and TMA ring) with the math and all output removed.
 *   pdattn_stream_read_probe : a plain sequential read of `bytes` bytes (16-byte aligned DEVICE
 *                              src); sink is 4 bytes of DEVICE scratch.
 */
pdattn_status pdattn_gather_probe(const pdattn_args* args, pdattn_stream_t stream);
pdattn_status pdattn_stream_read_probe(const void* src, size_t bytes, void* sink, pdattn_stream_t stream);

/*
 * Self-test of the kernels' failure path (no paper counterpart).  Every wait inside the kernels is bounded:
 * when a wait expires, the CTA sets the DEVICE_TIMEOUT bit of the workspace's error word and returns.
 * This call enqueues one warp that waits, for at most limit_us microseconds (1 .. 1,000,000), on a barrier
 * that nothing arrives on; afterwards pdattn_check(workspace) returns PDATTN_DEVICE_TIMEOUT once, and the
 * context and the workspace remain usable.
 */
pdattn_status pdattn_wait_limit_probe(void* workspace, int limit_us, pdattn_stream_t stream);

/* Number of kernels the last decode call on this thread launched (1 to 4: planner, shared-prefix kernel,
 * split-KV kernel, combine kernel, each only when it is needed). */
int pdattn_last_launch_count(void);

/* Fixed English text for a status code (no paper counterpart); never NULL, never freed. */
const char* pdattn_status_string(pdattn_status status);
const char* pdattn_last_cuda_error(void); /* thread-local text of the last CUDA failure */

#ifdef __cplusplus
}
#endif
#endif /* PDATTN_H_ */
