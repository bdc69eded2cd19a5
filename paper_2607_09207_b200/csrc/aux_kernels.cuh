// KV append (bf16 and fp8), stream-read probe, combine of cut units, device-side planner.
#pragma once

#include "common.cuh"

namespace pdattn {

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
  asm volatile("griddepcontrol.wait;" ::: "memory");   // a programmatic dependent of the kernel before it on the stream
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

// ------------------------------------------------------------------------------------------
// Host-resident step inputs: block s copies the used part of row s of a block table that lives in pinned,
// mapped host memory (ceil(L_s / bs) entries, the only ones a decode step reads) and the length itself into
// their device staging copies.  All loads are independent, so the whole batch costs about one round trip over
// the bus plus the bytes actually used, and the launch replaces two host-to-device copies of the full arrays.
// ------------------------------------------------------------------------------------------
constexpr int kGatherRows = 8;     // sequences per block of host_table_gather_kernel (one warp each)

// The fetches go through the bulk-copy engine (plain loads from host memory reach a small fraction of the
// bus rate): per block one bulk copy brings the kGatherRows lengths, then warp w brings the used part of its
// row into shared memory and sends it on to the device copy.  Needs MB % 4 == 0 (16-byte aligned rows) and
// num_seqs-padded length arrays are not assumed: the last block copies only the lengths that exist.
__global__ void __launch_bounds__(32 * kGatherRows)
host_table_gather_kernel(const int32_t* __restrict__ table_host, const int32_t* __restrict__ lens_host,
                         int32_t* __restrict__ table_dev, int32_t* __restrict__ lens_dev, int S, int MB, int bs,
                         int32_t* err) {
  extern __shared__ __align__(128) uint8_t gsm[];
  __shared__ __align__(16) int32_t lens_s[kGatherRows];
  __shared__ uint64_t bar_len, bar_row[kGatherRows];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int s0 = blockIdx.x * kGatherRows;
  const int nseq = min(kGatherRows, S - s0);
  const int row_bytes = MB * 4;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar_len), 1);
    for (int i = 0; i < kGatherRows; ++i) mbar_init(smem_u32(&bar_row[i]), 1);
    fence_mbar_init();
  }
  __syncthreads();
  asm volatile("griddepcontrol.wait;" ::: "memory");   // the staging copies may still be read by the step before
  const bool whole = nseq == kGatherRows;              // 32 bytes from a 32-byte aligned offset: one bulk copy
  if (threadIdx.x == 0) {
    if (whole) {
      mbar_arrive_expect_tx(smem_u32(&bar_len), kGatherRows * 4);
      bulk_load(smem_u32(lens_s), lens_host + s0, kGatherRows * 4, smem_u32(&bar_len));
    } else {
      for (int i = 0; i < nseq; ++i) lens_s[i] = *reinterpret_cast<const volatile int32_t*>(lens_host + s0 + i);
      mbar_arrive(smem_u32(&bar_len));
    }
  }
  bool ok = mbar_wait(smem_u32(&bar_len), 0);
  if (ok && warp < nseq) {
    const int s = s0 + warp;
    const int L = lens_s[warp];
    int n = L > 0 ? (L + bs - 1) / bs : 0;
    if (n > MB) n = MB;
    const uint32_t bytes = static_cast<uint32_t>((n * 4 + 15) & ~15);   // within the row: MB is a multiple of 4
    const uint32_t dst_s = smem_u32(gsm) + warp * row_bytes;
    if (bytes > 0) {
      if (lane == 0) {
        mbar_arrive_expect_tx(smem_u32(&bar_row[warp]), bytes);
        bulk_load(dst_s, table_host + static_cast<int64_t>(s) * MB, bytes, smem_u32(&bar_row[warp]));
      }
      ok = mbar_wait(smem_u32(&bar_row[warp]), 0);
      if (ok && lane == 0) {
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(
                         reinterpret_cast<uint64_t>(table_dev + static_cast<int64_t>(s) * MB)),
                     "r"(dst_s), "r"(bytes)
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
      }
    }
    if (lane == 0) lens_dev[s] = L;
  }
  if (!ok && lane == 0 && err) atomicOr(err, ERR_TIMEOUT);
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
  asm volatile("griddepcontrol.wait;" ::: "memory");   // a programmatic dependent of the kernel before it on the stream
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
// With inkernel_max > 0 the decode kernel has already merged every unit whose followers lie within
// inkernel_max spans of its first one; this kernel then only takes the longer chains.
// ------------------------------------------------------------------------------------------
template <int D, int NT>
__global__ void __launch_bounds__(256)
combine_kernel(WsHeader* hdr, int n_spans_host, const int4* __restrict__ rec, const float* __restrict__ partials,
               __nv_bfloat16* __restrict__ out, int Hq, int Hkv, int G, const int32_t* __restrict__ start_tiles,
               const float* __restrict__ pfx_partials, int T, int inkernel_max) {
  constexpr int HP = 8 * NT;
  constexpr int SLOT_FLOATS = HP * (D + 2);
  const int c = blockIdx.x;
  // launched as a programmatic dependent of the decode kernel: nothing of that kernel may be read
  // before this returns (it waits for the kernel's completion and memory flush)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int n_spans = n_spans_host >= 0 ? n_spans_host : hdr->plan.n_static + hdr->plan.n_dyn;
  if (c >= n_spans) return;
  const int4 r = rec[c];
  const int unit = r.z;
  if (unit < 0) return;
  // followers: later spans whose first piece continues `unit` (spans without tiles may sit between).
  // The block looks at blockDim.x span records at a time instead of walking them one dependent load after
  // the other: a long sequence can be cut by hundreds of spans.
  __shared__ int n_follow, first_break, run_len;
  __shared__ int follow[MAX_SPANS];
  if (threadIdx.x == 0) {
    n_follow = 0;
    run_len = n_spans - (c + 1);
  }
  for (int base = c + 1; base < n_spans; base += blockDim.x) {
    if (threadIdx.x == 0) first_break = blockDim.x;
    __syncthreads();
    const int cc = base + threadIdx.x;
    int4 rr = make_int4(-1, 0, 0, 0);
    if (cc < n_spans) rr = rec[cc];
    const bool past_end = cc >= n_spans;
    const bool empty = !past_end && rr.x < 0;                      // a span that holds no tile
    const bool cont = !past_end && rr.x == unit && rr.y > 0;       // its first piece continues the unit
    if (past_end || (!empty && !cont)) atomicMin(&first_break, static_cast<int>(threadIdx.x));
    __syncthreads();
    const int fb = first_break;
    // compact the continuing spans below the break, in order
    const bool take = cont && static_cast<int>(threadIdx.x) < fb;
    const int lane_id = threadIdx.x & 31, warp_id = threadIdx.x >> 5;
    __shared__ int warp_count[32];
    const uint32_t bal = __ballot_sync(0xffffffffu, take);
    if (lane_id == 0) warp_count[warp_id] = __popc(bal);
    __syncthreads();
    int before = n_follow;
    for (int w = 0; w < warp_id; ++w) before += warp_count[w];
    if (take) follow[before + __popc(bal & ((1u << lane_id) - 1u))] = cc;
    __syncthreads();
    if (threadIdx.x == 0) {
      int tot = 0;
      for (int w = 0; w < static_cast<int>(blockDim.x) / 32; ++w) tot += warp_count[w];
      n_follow += tot;
      if (fb < static_cast<int>(blockDim.x)) run_len = base - (c + 1) + fb;
    }
    __syncthreads();
    if (fb < static_cast<int>(blockDim.x)) break;
  }
  __syncthreads();
  // a short chain has been merged inside the decode kernel by the CTA that wrote its last partial
  if (inkernel_max > 0 && run_len <= inkernel_max) return;
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
#pragma unroll 8
    for (int p = p0; p < np; ++p) M = fmaxf(M, piece(p)[h]);   // independent loads: many in flight
    const float Mu = (M == NEG_INF) ? 0.f : M;
    float Ls = 0.f;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
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
            int n_static, int n_dyn_max, int32_t* __restrict__ prefix, SpanStart* __restrict__ spans, WsHeader* hdr,
            int with_merge_words) {
  __shared__ int warp_sums[32];
  __shared__ int carry_c, carry_t;
  __shared__ PlanParams pp_s;
  int32_t* pcost = prefix;
  int32_t* ptile = prefix + (S + 1);
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  // launched as a programmatic dependent of whatever precedes it on the stream (the KV append in a decode
  // loop): nothing may be read or written before that kernel has completed and flushed
  asm volatile("griddepcontrol.wait;" ::: "memory");
  __shared__ unsigned long long wide_cost;
  if (tid == 0) {
    carry_c = carry_t = 0;
    pcost[0] = ptile[0] = 0;
    wide_cost = 0ull;
  }
  __syncthreads();
  unsigned long long mine64 = 0ull;   // this thread's share of the total cost, in 64 bits (see the end of the kernel)
  for (int base = 0; base < S; base += 1024) {
    const int s = base + tid;
    int nt = 0;
    if (s < S) nt = static_cast<int>(seq_tiles(context_lens[s], start_tiles ? start_tiles[s] : 0));
    mine64 += static_cast<unsigned long long>(seq_cost(nt, Hkv));
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
  // The running sums above are 32-bit, like the host planner's tables; the host refuses a batch whose tile count
  // does not fit, and so does this kernel: the true total, in 64 bits, decides.
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mine64 += __shfl_xor_sync(0xffffffffu, mine64, o);
  if (lane == 0 && mine64) atomicAdd(&wide_cost, mine64);
  __syncthreads();
  if (wide_cost > static_cast<unsigned long long>(INT32_MAX / 2)) {
    // too large: an empty plan (nothing is computed) and an error bit for pdattn_check
    const PlanParams none = make_plan_params(0, 0, n_static, 0);
    if (tid == 0) {
      hdr->plan = none;
      atomicOr(&hdr->err, ERR_TOO_LARGE);
    }
    for (int c = tid; c <= n_static; c += 1024) {
      SpanStart sp;
      sp.unit = S * Hkv;
      sp.tile = sp.flat = sp.merge = 0;
      spans[c] = sp;
    }
    return;
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
    sp.merge = 0;
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
  // how the cut units are put together again: one word per span, from the finished table (only when the decode
  // kernel that follows merges cut units itself: the scan is a chain of dependent loads per span)
  if (!with_merge_words) return;
  __syncthreads();
  for (int c = tid; c < n_spans; c += 1024) spans[c].merge = span_merge_info(spans, n_spans, c);
}

// ------------------------------------------------------------------------------------------
// Self-test of the bounded wait: one warp waits on an mbarrier that nothing will ever arrive on, with the
// given limit, and reports the expiry through the workspace's sticky error word exactly as the kernels
// do.  The context stays usable: the kernel returns normally.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32)
wait_limit_probe_kernel(int32_t* err, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    fence_mbar_init();
  }
  __syncwarp();
  const uint32_t b = smem_u32(&bar);
  bool done = mbar_try_wait(b, 0);
  const unsigned long long t0 = globaltimer_ns();
  while (!done) {
    if (globaltimer_ns() - t0 > limit_ns) break;
#pragma unroll 1
    for (int i = 0; i < 16 && !done; ++i) done = mbar_try_wait_hint(b, 0, 1000);
  }
  if (!done && threadIdx.x == 0) atomicOr(err, ERR_TIMEOUT);
}

}  // namespace pdattn
