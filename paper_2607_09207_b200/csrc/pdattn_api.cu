// Host side of libpdattn: argument checks, the host partitioner call, TMA tensor maps, launches.
// No allocation, no synchronisation (except pdattn_check).  State: the process-wide pdattn_set_* settings, and per
// thread the pdattn_bind binding, the profiling events, the tensor-map cache and the last error text.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/pdattn.h"
#include "kernels.cuh"
#include "prefix_umma.cuh"
#include "partition.h"

namespace {

using namespace pdattn;

thread_local char g_cuda_err[256] = "";
thread_local int g_last_launches = 0;
thread_local cudaEvent_t g_prof_start = nullptr, g_prof_stop = nullptr;
// Process-wide settings (the pdattn_set_* calls); everything that belongs to one call travels in a CallDesc.
int g_dyn_per_cta = -1;                   // run-time spans per CTA (pdattn_set_dynamic_spans); -1: by batch shape
constexpr int kAutoDynPerCta = 4;         // ... then this many when the batch has at least kAutoDynUnits units per CTA
constexpr int kAutoDynUnits = 4;
int g_merge_mode = -1;                    // pdattn_set_merge_mode: -1 default (1 or 2 by batch shape), 0 barrier + combine kernel, 1 chained + merge
                                          // of cut units inside the decode kernel, 2 chained + combine kernel
constexpr int kAutoInKernelTiles = 8;      // mode -1: in-kernel merge from this many tiles per unit on average
constexpr int kInKernelMergeSpans = kMaxMergeRun;   // a cut unit followed by at most this many spans is merged inside the decode kernel
int g_host_zero_copy = -1;                // pdattn_set_host_zero_copy: -1 default (when possible), 0 never, 1 as -1
int g_prefix_engine = -1;                 // pdattn_set_prefix_engine: -1 default (tcgen05), 0 warp MMAs, 1 tcgen05
int g_short_path = -1;                    // pdattn_set_short_piece_path: -1 by batch shape, 0 never, 1 whenever it applies
constexpr int kAutoShortTilesX2 = 3;      // mode -1: the short-piece kernel below 1.5 tiles per unit on average
thread_local std::vector<int32_t> g_start_tiles_host;   // scratch of the grouped path (no call parameter lives here)

// What one decode call is, beyond the plain arguments: every entry point fills one of these and hands it to
// decode_common.
struct CallDesc {
  int query_tokens = 1;                         // pdattn_decode_multi
  bool probe = false;                           // pdattn_gather_probe: same walk and loads, no math, no output
  bool fp8 = false;                             // pdattn_decode_fp8: e4m3 codes, one scale per KV head
  const float* k_scale = nullptr;
  const float* v_scale = nullptr;
  int group_size = 0;                           // pdattn_decode_grouped: > 0, with the shared tiles per group
  const int32_t* prefix_tiles = nullptr;        //   device copy
  const int32_t* prefix_tiles_host = nullptr;   //   host copy
  bool static_scratch = false;                  // pdattn_decode_static_scratch: scratch is the built-in array
  int32_t* status_out = nullptr;                //   device word that receives the error word after the call
};

// What the launchers need to pick a kernel instantiation.
struct DevInfo;
struct LaunchCtx {
  int block_size;
  bool chain, probe, fp8;
  bool win;                 // the short-piece instantiation of the chained-merge kernel (8-row tiles, bf16 cache)
  DevInfo* di;
  cudaStream_t stream;
};

struct Binding {
  bool set = false;
  int max_blocks_per_seq = 0, num_blocks = 0;
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  const int32_t* context_lens_host = nullptr;
};
thread_local Binding g_bind;

pdattn_status cuda_fail(const char* what, cudaError_t e) {
  snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", what, cudaGetErrorString(e));
  return PDATTN_CUDA_ERROR;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- workspace layout ----------------------------------------------------------------------
struct WsLayout {
  size_t hdr, spans, rec, prefix, partials, total;
};
// max_spans: spans the span table, the records and the partial slots are sized for
WsLayout ws_layout(int num_seqs, int G, int head_dim, int max_spans = MAX_SPANS) {
  const int NT = G > 8 ? 2 : 1;
  const size_t slot_bytes = static_cast<size_t>(8 * NT) * (head_dim + 2) * 4;
  WsLayout w;
  w.hdr = 0;
  w.spans = WS_CLEARED_BYTES;   // header, then the ticket words
  w.rec = w.spans + align_up(static_cast<size_t>(max_spans + 1) * sizeof(SpanStart), 256);
  w.prefix = w.rec + align_up(static_cast<size_t>(max_spans) * sizeof(int4), 256);
  w.partials = w.prefix + align_up(static_cast<size_t>(num_seqs + 1) * 8, 256);
  w.total = w.partials + align_up(static_cast<size_t>(max_spans) * 2 * slot_bytes, 256);
  return w;
}

pdattn_status check_shape(int num_seqs, int Hq, int Hkv, int d, int bs) {
  if (num_seqs < 0 || Hq <= 0 || Hkv <= 0 || d <= 0 || bs <= 0) return PDATTN_INVALID_ARG;
  if (Hq % Hkv != 0) return PDATTN_INVALID_ARG;
  if (d != 64 && d != 128) return PDATTN_UNSUPPORTED;
  if (bs != 16 && bs != 32 && bs != 64) return PDATTN_UNSUPPORTED;
  if (Hq / Hkv > 16) return PDATTN_UNSUPPORTED;
  return PDATTN_OK;
}

// ---- per-device facts ------------------------------------------------------------------------
struct DevInfo {
  bool ready = false;
  int sm_count = 0;
  bool attr_set[2][2][3] = {};      // [D==128][NT==2][page size / 32]
  bool probe_attr_set[2][2][3] = {};
  bool chain_attr_set[2][2][3] = {};
  bool win_attr_set[2][3] = {};     // [D==128][page size / 32]
  bool fp8_attr_set[2][2][3] = {};  // [D==128][NT==2][page size / 32]
  bool prefix_fp8_attr_set[2][3] = {};
  bool prefix_attr_set[2][3] = {};  // [D==128][page size / 32]
  bool prefix_umma_attr_set[2][3] = {};
};
constexpr int kMaxDevices = 64;
DevInfo g_dev[kMaxDevices];
std::mutex g_dev_mu;

pdattn_status device_info(int* dev_out, DevInfo** info) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail("cudaGetDevice", e);
  if (dev < 0 || dev >= kMaxDevices) return PDATTN_UNSUPPORTED;
  DevInfo& di = g_dev[dev];
  if (!di.ready) {
    std::lock_guard<std::mutex> lk(g_dev_mu);
    if (!di.ready) {
      int sms = 0, major = 0;
      e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return cuda_fail("cudaDeviceGetAttribute", e);
      e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
      if (e != cudaSuccess) return cuda_fail("cudaDeviceGetAttribute", e);
      if (major != 10) {
        snprintf(g_cuda_err, sizeof g_cuda_err, "libpdattn is built for sm_100a only (device has major %d)", major);
        return PDATTN_CUDA_ERROR;
      }
      di.sm_count = sms;
      di.ready = true;
    }
  }
  *dev_out = dev;
  *info = &di;
  return PDATTN_OK;
}

// ---- TMA tensor maps ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

pdattn_status get_encode() {
  if (g_encode) return PDATTN_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return cuda_fail("cudaGetDriverEntryPoint", e);
  if (!fn || qres != cudaDriverEntryPointSuccess) {
    snprintf(g_cuda_err, sizeof g_cuda_err, "cuTensorMapEncodeTiled not available in this driver");
    return PDATTN_CUDA_ERROR;
  }
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return PDATTN_OK;
}

constexpr int kMapK8 = 81, kMapV8 = 82;   // "ranks" of the two fp8 views in make_map

struct MapKey {
  const void* ptr;
  int d, bs, hkv, nb, rank;
  int64_t sb, sh, st;
  bool operator==(const MapKey& o) const {
    return ptr == o.ptr && d == o.d && bs == o.bs && hkv == o.hkv && nb == o.nb && rank == o.rank && sb == o.sb &&
           sh == o.sh && st == o.st;
  }
};
struct MapCacheEntry {
  bool valid = false;
  MapKey key;
  CUtensorMap map;
};
thread_local MapCacheEntry g_maps[16];
thread_local int g_map_next = 0;

// View of a cache as a tensor for TMA, 128-byte swizzle, zero fill out of bounds.
//   rank 4: (dim, slot, kv head, page); one box = one 64-element column block of a page-head,
//           [64, block_size, 1, 1]: head_dim / 64 copies per page-head.
//   rank 5: (dim within column block, slot, column block, kv head, page); one box = a whole
//           page-head [64, block_size, 2, 1, 1], landing in shared memory column block by column
//           block exactly like two rank-4 boxes.  head_dim 128 only.
pdattn_status make_map(const void* ptr, int d, int bs, int hkv, int nb, int64_t sb, int64_t sh, int64_t st, int rank,
                       CUtensorMap* out) {
  MapKey key{ptr, d, bs, hkv, nb, rank, sb, sh, st};
  for (auto& e : g_maps)
    if (e.valid && e.key == key) {
      *out = e.map;
      return PDATTN_OK;
    }
  pdattn_status s = get_encode();
  if (s != PDATTN_OK) return s;
  const cuuint64_t nbu = static_cast<cuuint64_t>(nb > 0 ? nb : 1);
  CUtensorMap m;
  CUresult r;
  if (rank == kMapK8) {
    // fp8 K pool [pages, kv heads, slots, d] of one-byte codes: one box = a page-head, [d, block_size, 1, 1]
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(bs), static_cast<cuuint64_t>(hkv), nbu};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(bs) * d,
                             static_cast<cuuint64_t>(hkv) * bs * d};
    cuuint32_t box[4] = {static_cast<cuuint32_t>(d), static_cast<cuuint32_t>(bs), 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    // rows of d bytes: 128-byte swizzle at head_dim 128, 64-byte swizzle at head_dim 64
    r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, d == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (rank == kMapV8) {
    // fp8 V pool [pages, kv heads, d, slots] (transposed inside a page): a page-head is d * block_size
    // contiguous bytes and lands in shared memory in the same order, so it is described as rows of 256
    // bytes (8 requests per box; rows of block_size bytes would be 128), no swizzle
    const cuuint64_t rows = static_cast<cuuint64_t>(d) * bs / 256;
    cuuint64_t dims[4] = {256, rows, static_cast<cuuint64_t>(hkv), nbu};
    cuuint64_t strides[3] = {256, static_cast<cuuint64_t>(d) * bs, static_cast<cuuint64_t>(hkv) * d * bs};
    cuuint32_t box[4] = {256, static_cast<cuuint32_t>(rows), 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else if (rank == 5) {
    cuuint64_t dims[5] = {64, static_cast<cuuint64_t>(bs), static_cast<cuuint64_t>(d / 64),
                          static_cast<cuuint64_t>(hkv), nbu};
    cuuint64_t strides[4] = {static_cast<cuuint64_t>(st) * 2, 128, static_cast<cuuint64_t>(sh) * 2,
                             static_cast<cuuint64_t>(sb) * 2};
    cuuint32_t box[5] = {64, static_cast<cuuint32_t>(bs), static_cast<cuuint32_t>(d / 64), 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(bs), static_cast<cuuint64_t>(hkv), nbu};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(st) * 2, static_cast<cuuint64_t>(sh) * 2,
                             static_cast<cuuint64_t>(sb) * 2};
    cuuint32_t box[4] = {64, static_cast<cuuint32_t>(bs), 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) {
    snprintf(g_cuda_err, sizeof g_cuda_err, "cuTensorMapEncodeTiled (rank %d) failed with CUresult %d", rank,
             static_cast<int>(r));
    return PDATTN_CUDA_ERROR;
  }
  MapCacheEntry& e = g_maps[g_map_next];
  g_map_next = (g_map_next + 1) % 16;
  e.valid = true;
  e.key = key;
  e.map = m;
  *out = m;
  return PDATTN_OK;
}

// ---- launches ------------------------------------------------------------------------------------
// Launch that may begin while the kernel before it on the stream drains (programmatic dependent launch); the
// kernel itself waits (griddepcontrol.wait) before it touches global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t stream, bool dependent,
                             Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = dependent ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <int D, int NT, int BS>
pdattn_status launch_bs(const CUtensorMap& mk, const CUtensorMap& mv, const DecodeParams& P, int grid, int combine_grid,
                     int n_spans_host, const LaunchCtx& lc) {
  using C = Cfg<D, NT, BS>;
  DevInfo* di = lc.di;
  cudaStream_t stream = lc.stream;
  auto kern = decode_kernel<D, NT, BS>;
  bool& done = di->attr_set[D == 128][NT == 2][BS / 32];
  if (!done) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::DYN_BYTES);
    if (e != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", e);
    done = true;
  }
  if (lc.probe) {
    auto probe = decode_kernel<D, NT, BS, true>;
    cudaError_t pe = cudaFuncSetAttribute(probe, cudaFuncAttributeMaxDynamicSharedMemorySize, C::DYN_BYTES);
    if (pe != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", pe);
    probe<<<grid, C::NTHREADS, C::DYN_BYTES, stream>>>(mk, mv, P);
    pe = cudaGetLastError();
    if (pe != cudaSuccess) return cuda_fail("gather probe launch", pe);
    pe = cudaMemsetAsync(&P.hdr->counter, 0, 4, stream);   // the combine kernel normally rearms it
    if (pe != cudaSuccess) return cuda_fail("cudaMemsetAsync", pe);
    return PDATTN_OK;
  }
  // the kernel may be set up while its predecessor on the stream drains (and waits for it inside)
  const bool dependent = g_prof_start == nullptr;
  if (g_prof_start) cudaEventRecord(g_prof_start, stream);
  if (lc.fp8) {
    using C8 = Cfg<D, NT, BS, 1>;
    auto k8 = decode_kernel<D, NT, BS, false, true, 1>;
    bool& fdone = di->fp8_attr_set[D == 128][NT == 2][BS / 32];
    if (!fdone) {
      cudaError_t fe = cudaFuncSetAttribute(k8, cudaFuncAttributeMaxDynamicSharedMemorySize, C8::CHAIN_DYN_BYTES);
      if (fe != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", fe);
      fdone = true;
    }
    launch_dependent(k8, grid, C8::NTHREADS, C8::CHAIN_DYN_BYTES, stream, dependent, mk, mv, P);
  } else if (lc.chain && lc.win && NT == 1) {
    if constexpr (NT == 1) {
      auto win = decode_kernel<D, NT, BS, false, true, 2, true>;
      bool& wdone = di->win_attr_set[D == 128][BS / 32];
      if (!wdone) {
        cudaError_t we = cudaFuncSetAttribute(win, cudaFuncAttributeMaxDynamicSharedMemorySize, C::CHAIN_DYN_BYTES);
        if (we != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", we);
        wdone = true;
      }
      launch_dependent(win, grid, C::NTHREADS, C::CHAIN_DYN_BYTES, stream, dependent, mk, mv, P);
    }
  } else if (lc.chain) {
    auto chain = decode_kernel<D, NT, BS, false, true>;
    bool& cdone = di->chain_attr_set[D == 128][NT == 2][BS / 32];
    if (!cdone) {
      cudaError_t ce = cudaFuncSetAttribute(chain, cudaFuncAttributeMaxDynamicSharedMemorySize, C::CHAIN_DYN_BYTES);
      if (ce != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", ce);
      cdone = true;
    }
    launch_dependent(chain, grid, C::NTHREADS, C::CHAIN_DYN_BYTES, stream, dependent, mk, mv, P);
  } else {
    launch_dependent(kern, grid, C::NTHREADS, C::DYN_BYTES, stream, dependent, mk, mv, P);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail("decode_kernel launch", e);
  if (g_prof_stop) cudaEventRecord(g_prof_stop, stream);
  // Programmatic dependent launch: the combine grid is set up while the decode kernel drains and
  // waits (griddepcontrol.wait in the kernel) until that kernel has completed and flushed.
  if (combine_grid <= 0) return PDATTN_OK;   // every cut unit is merged inside the decode kernel
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(combine_grid);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = (g_prof_stop == nullptr) ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, combine_kernel<D, NT>, P.hdr, n_spans_host, static_cast<const int4*>(P.rec),
                         static_cast<const float*>(P.partials), P.out, P.Hq, P.Hkv, P.G, P.start_tiles,
                         P.pfx_partials, P.T, P.inkernel_max);
  if (e != cudaSuccess) return cuda_fail("combine_kernel launch", e);
  return PDATTN_OK;
}

template <int D, int BS, int EB>
pdattn_status launch_prefix_bs(const CUtensorMap& mk, const CUtensorMap& mv, const PrefixParams& X, int grid, DevInfo* di,
                            cudaStream_t stream) {
  using C = Cfg<D, 1, BS, EB>;
  const int smem = 1024 + C::NSTAGES * C::STAGE_BYTES + C::CTRL_BYTES;
  auto kern = prefix_kernel<D, BS, EB>;
  bool& done = EB == 1 ? di->prefix_fp8_attr_set[D == 128][BS / 32] : di->prefix_attr_set[D == 128][BS / 32];
  if (!done) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", e);
    done = true;
  }
  if (grid <= 0) return PDATTN_OK;
  kern<<<grid, C::NTHREADS_BASE, smem, stream>>>(mk, mv, X);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail("prefix_kernel launch", e);
  return PDATTN_OK;
}

template <int D, int BS>
pdattn_status launch_prefix_umma_bs(const CUtensorMap& mk, const CUtensorMap& mv, const PrefixParams& X, int grid, DevInfo* di,
                                    cudaStream_t stream) {
  using C = UmmaCfg<D, BS>;
  auto kern = prefix_umma_kernel<D, BS>;
  bool& done = di->prefix_umma_attr_set[D == 128][BS / 32];
  if (!done) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::DYN_BYTES);
    if (e != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", e);
    done = true;
  }
  if (grid <= 0) return PDATTN_OK;
  kern<<<grid, C::NTHREADS, C::DYN_BYTES, stream>>>(mk, mv, X);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail("prefix_umma_kernel launch", e);
  return PDATTN_OK;
}

template <int D, int NT>
pdattn_status launch(const CUtensorMap& mk, const CUtensorMap& mv, const DecodeParams& P, int grid, int combine_grid,
                     int n_spans_host, const LaunchCtx& lc) {
  return lc.block_size == 64   ? launch_bs<D, NT, 64>(mk, mv, P, grid, combine_grid, n_spans_host, lc)
         : lc.block_size == 32 ? launch_bs<D, NT, 32>(mk, mv, P, grid, combine_grid, n_spans_host, lc)
                               : launch_bs<D, NT, 16>(mk, mv, P, grid, combine_grid, n_spans_host, lc);
}
template <int D>
pdattn_status launch_prefix_umma(const CUtensorMap& mk, const CUtensorMap& mv, const PrefixParams& X, int grid,
                                 const LaunchCtx& lc) {
  return lc.block_size == 64   ? launch_prefix_umma_bs<D, 64>(mk, mv, X, grid, lc.di, lc.stream)
         : lc.block_size == 32 ? launch_prefix_umma_bs<D, 32>(mk, mv, X, grid, lc.di, lc.stream)
                               : launch_prefix_umma_bs<D, 16>(mk, mv, X, grid, lc.di, lc.stream);
}
template <int D>
pdattn_status launch_prefix(const CUtensorMap& mk, const CUtensorMap& mv, const PrefixParams& X, int grid,
                            const LaunchCtx& lc) {
  if (lc.fp8)
    return lc.block_size == 64   ? launch_prefix_bs<D, 64, 1>(mk, mv, X, grid, lc.di, lc.stream)
           : lc.block_size == 32 ? launch_prefix_bs<D, 32, 1>(mk, mv, X, grid, lc.di, lc.stream)
                                 : launch_prefix_bs<D, 16, 1>(mk, mv, X, grid, lc.di, lc.stream);
  return lc.block_size == 64   ? launch_prefix_bs<D, 64, 2>(mk, mv, X, grid, lc.di, lc.stream)
         : lc.block_size == 32 ? launch_prefix_bs<D, 32, 2>(mk, mv, X, grid, lc.di, lc.stream)
                               : launch_prefix_bs<D, 16, 2>(mk, mv, X, grid, lc.di, lc.stream);
}

pdattn_status decode_common(const pdattn_args* a, const CallDesc& cd, pdattn_stream_t stream_);

}  // namespace

extern "C" {

pdattn_status pdattn_workspace_size(int num_seqs, int num_q_heads, int num_kv_heads, int head_dim, int block_size,
                                    int max_context_len, size_t* device_bytes, size_t* pinned_host_bytes) {
  (void)max_context_len;
  if (!device_bytes) return PDATTN_INVALID_ARG;
  pdattn_status s = check_shape(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size);
  if (s != PDATTN_OK) return s;
  *device_bytes = ws_layout(num_seqs, num_q_heads / num_kv_heads, head_dim).total;
  if (pinned_host_bytes) *pinned_host_bytes = 0;
  return PDATTN_OK;
}

pdattn_status pdattn_workspace_init(void* workspace, size_t workspace_bytes, pdattn_stream_t stream) {
  if (!workspace || workspace_bytes < static_cast<size_t>(WS_CLEARED_BYTES)) return PDATTN_INVALID_ARG;
  // the header (error word, span counter) and the ticket words of the in-kernel merge start at zero
  cudaError_t e = cudaMemsetAsync(workspace, 0, WS_CLEARED_BYTES, reinterpret_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail("cudaMemsetAsync", e);
  return PDATTN_OK;
}

pdattn_status pdattn_append_kv(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                               const int32_t* block_table, int32_t* context_lens, int num_seqs, int num_kv_heads,
                               int head_dim, int block_size, int max_blocks_per_seq, int num_blocks,
                               int64_t kv_block_stride, int64_t kv_head_stride, int64_t kv_token_stride,
                               void* workspace, pdattn_stream_t stream) {
  if (num_seqs < 0 || num_kv_heads <= 0 || num_kv_heads > 16 || max_blocks_per_seq <= 0 || num_blocks <= 0)
    return PDATTN_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return PDATTN_UNSUPPORTED;
  if (block_size != 16 && block_size != 32 && block_size != 64) return PDATTN_UNSUPPORTED;
  if (num_seqs == 0) return PDATTN_OK;
  if (!k_new || !v_new || !k_cache || !v_cache || !block_table || !context_lens) return PDATTN_INVALID_ARG;
  if (kv_block_stride <= 0 || kv_head_stride <= 0 || kv_token_stride < head_dim) return PDATTN_INVALID_ARG;
  if ((kv_block_stride | kv_head_stride | kv_token_stride) % 8 != 0) return PDATTN_UNSUPPORTED;
  auto mis = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; };
  if (mis(k_new) || mis(v_new) || mis(k_cache) || mis(v_cache)) return PDATTN_MISALIGNED;
  cudaError_t e = launch_dependent(
      append_kernel, num_seqs, 32 * num_kv_heads, 0, reinterpret_cast<cudaStream_t>(stream), true,
      static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
      static_cast<__nv_bfloat16*>(k_cache), static_cast<__nv_bfloat16*>(v_cache), block_table, context_lens,
      num_kv_heads, head_dim, block_size, max_blocks_per_seq, num_blocks, kv_block_stride, kv_head_stride,
      kv_token_stride, static_cast<int32_t*>(workspace));
  if (e != cudaSuccess) return cuda_fail("append_kernel launch", e);
  return PDATTN_OK;
}

pdattn_status pdattn_set_dynamic_spans(int per_cta) {
  if (per_cta < -1 || per_cta > kMaxDynPerCta) return PDATTN_INVALID_ARG;
  g_dyn_per_cta = per_cta;
  return PDATTN_OK;
}

pdattn_status pdattn_append_kv_fp8(const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                                   const float* k_scale, const float* v_scale, const int32_t* block_table,
                                   int32_t* context_lens, int num_seqs, int num_kv_heads, int head_dim,
                                   int block_size, int max_blocks_per_seq, int num_blocks, void* workspace,
                                   pdattn_stream_t stream) {
  if (num_seqs < 0 || num_kv_heads <= 0 || num_kv_heads > 16 || max_blocks_per_seq <= 0 || num_blocks <= 0)
    return PDATTN_INVALID_ARG;
  if ((head_dim != 128 && head_dim != 64) || (block_size != 16 && block_size != 32 && block_size != 64))
    return PDATTN_UNSUPPORTED;
  if (num_seqs == 0) return PDATTN_OK;
  if (!k_new || !v_new || !k_cache || !v_cache || !k_scale || !v_scale || !block_table || !context_lens)
    return PDATTN_INVALID_ARG;
  auto mis = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; };
  if (mis(k_new) || mis(v_new) || mis(k_cache) || mis(v_cache)) return PDATTN_MISALIGNED;
  cudaError_t e = launch_dependent(
      append_fp8_kernel, num_seqs, 32 * num_kv_heads, 0, reinterpret_cast<cudaStream_t>(stream), true,
      static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
      static_cast<uint8_t*>(k_cache), static_cast<uint8_t*>(v_cache), k_scale, v_scale, block_table, context_lens,
      num_kv_heads, head_dim, block_size, max_blocks_per_seq, num_blocks, static_cast<int32_t*>(workspace));
  if (e != cudaSuccess) return cuda_fail("append_fp8_kernel launch", e);
  return PDATTN_OK;
}

pdattn_status pdattn_set_short_piece_path(int mode) {
  if (mode < -1 || mode > 1) return PDATTN_INVALID_ARG;
  g_short_path = mode;
  return PDATTN_OK;
}

pdattn_status pdattn_set_prefix_engine(int engine) {
  if (engine < -1 || engine > 1) return PDATTN_INVALID_ARG;
  g_prefix_engine = engine;
  return PDATTN_OK;
}

pdattn_status pdattn_set_merge_mode(int mode) {
  if (mode < -1 || mode > 2) return PDATTN_INVALID_ARG;
  g_merge_mode = mode;
  return PDATTN_OK;
}

pdattn_status pdattn_plan_host(const int32_t* context_lens_host, int num_seqs, int num_kv_heads, int n_ctas,
                               int dynamic_per_cta, int max_spans, int32_t* spans, pdattn_plan* plan_out) {
  if (!plan_out) return PDATTN_INVALID_ARG;
  PlanParams plan;
  if (!spans || max_spans < n_ctas) return PDATTN_INVALID_ARG;
  static_assert(sizeof(SpanStart) == 4 * sizeof(int32_t), "span table entries are four int32");
  if (!plan_spans(context_lens_host, nullptr, num_seqs, num_kv_heads, n_ctas, dynamic_per_cta, max_spans,
                  reinterpret_cast<SpanStart*>(spans), &plan))
    return PDATTN_INVALID_ARG;
  plan_out->n_static = plan.n_static;
  plan_out->n_dynamic = plan.n_dyn;
  plan_out->total_tiles = plan.total;
  return PDATTN_OK;
}

pdattn_status pdattn_decode_ex(const pdattn_args* a, pdattn_stream_t stream) {
  return decode_common(a, CallDesc{}, stream);
}

pdattn_status pdattn_multi_workspace_size(int num_seqs, int num_q_heads, int num_kv_heads, int head_dim, int block_size,
                                          int num_query_tokens, size_t* device_bytes) {
  if (!device_bytes) return PDATTN_INVALID_ARG;
  pdattn_status s = check_shape(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size);
  if (s != PDATTN_OK) return s;
  if (num_query_tokens < 1) return PDATTN_INVALID_ARG;
  const int G = num_q_heads / num_kv_heads;
  if (G * num_query_tokens > 16) return PDATTN_UNSUPPORTED;
  *device_bytes = ws_layout(num_seqs, G * num_query_tokens, head_dim).total;
  return PDATTN_OK;
}

pdattn_status pdattn_decode_multi(const pdattn_args* args, int num_query_tokens, pdattn_stream_t stream) {
  CallDesc cd;
  cd.query_tokens = num_query_tokens;
  return decode_common(args, cd, stream);
}

pdattn_status pdattn_decode_fp8_multi(const pdattn_args* args, int num_query_tokens, const float* k_scale,
                                      const float* v_scale, pdattn_stream_t stream) {
  if (!args || !k_scale || !v_scale) return PDATTN_INVALID_ARG;
  pdattn_args a = *args;
  // dense pools of one-byte codes; the stride fields are not used by this variant
  a.kv_token_stride = a.head_dim;
  a.kv_head_stride = static_cast<int64_t>(a.block_size) * a.head_dim;
  a.kv_block_stride = static_cast<int64_t>(a.num_kv_heads) * a.block_size * a.head_dim;
  CallDesc cd;
  cd.query_tokens = num_query_tokens;
  cd.fp8 = true;
  cd.k_scale = k_scale;
  cd.v_scale = v_scale;
  return decode_common(&a, cd, stream);
}

pdattn_status pdattn_decode_fp8(const pdattn_args* args, const float* k_scale, const float* v_scale,
                                pdattn_stream_t stream) {
  return pdattn_decode_fp8_multi(args, 1, k_scale, v_scale, stream);
}

pdattn_status pdattn_grouped_workspace_size(int num_seqs, int num_q_heads, int num_kv_heads, int head_dim,
                                            int block_size, size_t* device_bytes) {
  if (!device_bytes) return PDATTN_INVALID_ARG;
  pdattn_status s = check_shape(num_seqs, num_q_heads, num_kv_heads, head_dim, block_size);
  if (s != PDATTN_OK) return s;
  const int G = num_q_heads / num_kv_heads;
  const size_t base = ws_layout(num_seqs, G, head_dim).total;
  const size_t pfx = static_cast<size_t>(num_seqs) * num_kv_heads * (G > 8 ? 16 : 8) * (head_dim + 2) * 4;
  *device_bytes = base + align_up(static_cast<size_t>(num_seqs) * 4, 256) + align_up(pfx, 256);
  return PDATTN_OK;
}

pdattn_status pdattn_decode_grouped(const pdattn_args* args, int group_size, const int32_t* prefix_tiles,
                                    const int32_t* prefix_tiles_host, pdattn_stream_t stream) {
  if (!args || !prefix_tiles || !prefix_tiles_host) return PDATTN_INVALID_ARG;
  if (group_size <= 0) return PDATTN_INVALID_ARG;
  CallDesc cd;
  cd.group_size = group_size;
  cd.prefix_tiles = prefix_tiles;
  cd.prefix_tiles_host = prefix_tiles_host;
  return decode_common(args, cd, stream);
}

pdattn_status pdattn_bind(int max_blocks_per_seq, int num_blocks, void* workspace, size_t workspace_bytes,
                          const int32_t* context_lens_host) {
  if (max_blocks_per_seq <= 0 || num_blocks <= 0 || !workspace) return PDATTN_INVALID_ARG;
  g_bind.set = true;
  g_bind.max_blocks_per_seq = max_blocks_per_seq;
  g_bind.num_blocks = num_blocks;
  g_bind.workspace = workspace;
  g_bind.workspace_bytes = workspace_bytes;
  g_bind.context_lens_host = context_lens_host;
  return PDATTN_OK;
}

pdattn_status pdattn_decode(const void* q, const void* k_cache, const void* v_cache, const int32_t* block_table,
                            const int32_t* context_lens, int num_seqs, int num_q_heads, int num_kv_heads,
                            int head_dim, int block_size, float scale, void* out, pdattn_stream_t stream) {
  if (!g_bind.set) return PDATTN_NOT_BOUND;
  pdattn_args a;
  memset(&a, 0, sizeof a);
  a.q = q;
  a.k_cache = k_cache;
  a.v_cache = v_cache;
  a.out = out;
  a.block_table = block_table;
  a.context_lens = context_lens;
  a.context_lens_host = g_bind.context_lens_host;
  a.num_seqs = num_seqs;
  a.num_q_heads = num_q_heads;
  a.num_kv_heads = num_kv_heads;
  a.head_dim = head_dim;
  a.block_size = block_size;
  a.max_blocks_per_seq = g_bind.max_blocks_per_seq;
  a.num_blocks = g_bind.num_blocks;
  a.kv_token_stride = head_dim;
  a.kv_head_stride = static_cast<int64_t>(block_size) * head_dim;
  a.kv_block_stride = static_cast<int64_t>(num_kv_heads) * block_size * head_dim;
  a.scale = scale;
  a.workspace = g_bind.workspace;
  a.workspace_bytes = g_bind.workspace_bytes;
  return pdattn_decode_ex(&a, stream);
}

pdattn_status pdattn_host_staging_size(int num_seqs, int num_q_heads, int head_dim, int max_blocks_per_seq,
                                       size_t* device_bytes) {
  if (num_seqs < 0 || num_q_heads <= 0 || head_dim <= 0 || max_blocks_per_seq <= 0 || !device_bytes)
    return PDATTN_INVALID_ARG;
  const size_t qb = align_up(static_cast<size_t>(num_seqs) * num_q_heads * head_dim * 2, 256);
  const size_t tb = align_up(static_cast<size_t>(num_seqs) * max_blocks_per_seq * 4, 256);
  const size_t lb = align_up(static_cast<size_t>(num_seqs) * 4, 256);
  *device_bytes = 2 * qb + tb + lb;
  return PDATTN_OK;
}

pdattn_status pdattn_set_host_zero_copy(int mode) {
  if (mode < -1 || mode > 1) return PDATTN_INVALID_ARG;
  g_host_zero_copy = mode;
  return PDATTN_OK;
}

// The device-side address of pinned, mapped host memory (null for pageable or unknown memory).
static void* mapped_host_pointer(const void* p) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

static pdattn_status decode_host_common(const void* q_host, const int32_t* block_table_host,
                                        const int32_t* context_lens_host, void* out_host, const void* k_cache,
                                        const void* v_cache, int num_seqs, int num_q_heads, int num_kv_heads,
                                        int head_dim, int block_size, int max_blocks_per_seq, int num_blocks, float scale,
                                        void* staging, size_t staging_bytes, void* workspace, size_t workspace_bytes,
                                        const CallDesc& cd, pdattn_stream_t stream_) {
  if (num_seqs == 0) return PDATTN_OK;
  if (!q_host || !block_table_host || !context_lens_host || !out_host || !staging) return PDATTN_INVALID_ARG;
  size_t need = 0;
  pdattn_status s = pdattn_host_staging_size(num_seqs, num_q_heads, head_dim, max_blocks_per_seq, &need);
  if (s != PDATTN_OK) return s;
  if (staging_bytes < need) return PDATTN_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(staging) & 255) return PDATTN_MISALIGNED;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  const size_t q_bytes = static_cast<size_t>(num_seqs) * num_q_heads * head_dim * 2;
  const size_t t_bytes = static_cast<size_t>(num_seqs) * max_blocks_per_seq * 4;
  const size_t l_bytes = static_cast<size_t>(num_seqs) * 4;
  uint8_t* st = static_cast<uint8_t*>(staging);
  void* q_dev = st;
  void* out_dev = st + align_up(q_bytes, 256);
  void* bt_dev = st + 2 * align_up(q_bytes, 256);
  void* len_dev = st + 2 * align_up(q_bytes, 256) + align_up(t_bytes, 256);
  // q is read once and out written once per step: when both are pinned and mapped the kernels use them
  // in place (query rows arrive by bulk copy a few units ahead of their use, output rows are posted
  // writes), which takes both transfers out of the step's critical path
  bool in_place = false;
  if (g_host_zero_copy != 0) {
    void* qm = mapped_host_pointer(q_host);
    void* om = mapped_host_pointer(out_host);
    if (qm && om && !(reinterpret_cast<uintptr_t>(qm) & 15) && !(reinterpret_cast<uintptr_t>(om) & 15)) {
      q_dev = qm;
      out_dev = om;
      in_place = true;
    }
  }
  cudaError_t e;
  if (!in_place && (e = cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
    return cuda_fail("cudaMemcpyAsync(q)", e);
  // block_table and context_lens: when both are pinned and mapped, one small kernel fetches the lengths and the
  // used part of every table row over the bus (about a third of the table for a long-tailed batch); otherwise
  // two copies of the whole arrays
  const void* btm = g_host_zero_copy != 0 ? mapped_host_pointer(block_table_host) : nullptr;
  const void* lm = g_host_zero_copy != 0 ? mapped_host_pointer(context_lens_host) : nullptr;
  const size_t gather_smem = static_cast<size_t>(kGatherRows) * max_blocks_per_seq * 4;
  if (btm && lm && !(reinterpret_cast<uintptr_t>(btm) & 15) && !(reinterpret_cast<uintptr_t>(lm) & 31) &&
      max_blocks_per_seq % 4 == 0 && gather_smem <= 200 * 1024) {
    static bool attr_set[kMaxDevices] = {};
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return cuda_fail("cudaGetDevice", e);
    if (dev >= 0 && dev < kMaxDevices && !attr_set[dev]) {
      e = cudaFuncSetAttribute(host_table_gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
      if (e != cudaSuccess) return cuda_fail("cudaFuncSetAttribute", e);
      attr_set[dev] = true;
    }
    e = launch_dependent(host_table_gather_kernel, (num_seqs + kGatherRows - 1) / kGatherRows, 32 * kGatherRows,
                         gather_smem, stream, true, static_cast<const int32_t*>(btm), static_cast<const int32_t*>(lm),
                         static_cast<int32_t*>(bt_dev), static_cast<int32_t*>(len_dev), num_seqs, max_blocks_per_seq,
                         block_size, static_cast<int32_t*>(workspace));
    if (e != cudaSuccess) return cuda_fail("host_table_gather_kernel launch", e);
  } else {
    if ((e = cudaMemcpyAsync(bt_dev, block_table_host, t_bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
      return cuda_fail("cudaMemcpyAsync(block_table)", e);
    if ((e = cudaMemcpyAsync(len_dev, context_lens_host, l_bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
      return cuda_fail("cudaMemcpyAsync(context_lens)", e);
  }
  pdattn_args a;
  memset(&a, 0, sizeof a);
  a.q = q_dev;
  a.k_cache = k_cache;
  a.v_cache = v_cache;
  a.out = out_dev;
  a.block_table = static_cast<const int32_t*>(bt_dev);
  a.context_lens = static_cast<const int32_t*>(len_dev);
  a.context_lens_host = context_lens_host;
  a.num_seqs = num_seqs;
  a.num_q_heads = num_q_heads;
  a.num_kv_heads = num_kv_heads;
  a.head_dim = head_dim;
  a.block_size = block_size;
  a.max_blocks_per_seq = max_blocks_per_seq;
  a.num_blocks = num_blocks;
  a.kv_token_stride = head_dim;
  a.kv_head_stride = static_cast<int64_t>(block_size) * head_dim;
  a.kv_block_stride = static_cast<int64_t>(num_kv_heads) * block_size * head_dim;
  a.scale = scale;
  a.workspace = workspace;
  a.workspace_bytes = workspace_bytes;
  s = decode_common(&a, cd, stream_);
  if (s != PDATTN_OK) return s;
  if (!in_place && (e = cudaMemcpyAsync(out_host, out_dev, q_bytes, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
    return cuda_fail("cudaMemcpyAsync(out)", e);
  return PDATTN_OK;
}

pdattn_status pdattn_decode_host(const void* q_host, const int32_t* block_table_host,
                                 const int32_t* context_lens_host, void* out_host, const void* k_cache,
                                 const void* v_cache, int num_seqs, int num_q_heads, int num_kv_heads, int head_dim,
                                 int block_size, int max_blocks_per_seq, int num_blocks, float scale, void* staging,
                                 size_t staging_bytes, void* workspace, size_t workspace_bytes,
                                 pdattn_stream_t stream) {
  return decode_host_common(q_host, block_table_host, context_lens_host, out_host, k_cache, v_cache, num_seqs,
                            num_q_heads, num_kv_heads, head_dim, block_size, max_blocks_per_seq, num_blocks, scale,
                            staging, staging_bytes, workspace, workspace_bytes, CallDesc{}, stream);
}

pdattn_status pdattn_decode_host_fp8(const void* q_host, const int32_t* block_table_host,
                                     const int32_t* context_lens_host, void* out_host, const void* k_cache,
                                     const void* v_cache, const float* k_scale, const float* v_scale, int num_seqs,
                                     int num_q_heads, int num_kv_heads, int head_dim, int block_size,
                                     int max_blocks_per_seq, int num_blocks, float scale, void* staging,
                                     size_t staging_bytes, void* workspace, size_t workspace_bytes,
                                     pdattn_stream_t stream) {
  if (!k_scale || !v_scale) return PDATTN_INVALID_ARG;
  CallDesc cd;
  cd.fp8 = true;
  cd.k_scale = k_scale;
  cd.v_scale = v_scale;
  return decode_host_common(q_host, block_table_host, context_lens_host, out_host, k_cache, v_cache, num_seqs,
                            num_q_heads, num_kv_heads, head_dim, block_size, max_blocks_per_seq, num_blocks, scale,
                            staging, staging_bytes, workspace, workspace_bytes, cd, stream);
}

pdattn_status pdattn_decode_grouped_fp8(const pdattn_args* args, int group_size, const int32_t* prefix_tiles,
                                        const int32_t* prefix_tiles_host, const float* k_scale, const float* v_scale,
                                        pdattn_stream_t stream) {
  if (!args || !prefix_tiles || !prefix_tiles_host || !k_scale || !v_scale) return PDATTN_INVALID_ARG;
  if (group_size <= 0) return PDATTN_INVALID_ARG;
  pdattn_args a = *args;
  a.kv_token_stride = a.head_dim;
  a.kv_head_stride = static_cast<int64_t>(a.block_size) * a.head_dim;
  a.kv_block_stride = static_cast<int64_t>(a.num_kv_heads) * a.block_size * a.head_dim;
  CallDesc cd;
  cd.group_size = group_size;
  cd.prefix_tiles = prefix_tiles;
  cd.prefix_tiles_host = prefix_tiles_host;
  cd.fp8 = true;
  cd.k_scale = k_scale;
  cd.v_scale = v_scale;
  return decode_common(&a, cd, stream);
}

pdattn_status pdattn_check(void* workspace, pdattn_stream_t stream_) {
  if (!workspace) return PDATTN_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  int32_t word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) return cuda_fail("cudaMemcpyAsync", e);
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail("cudaStreamSynchronize", e);
  if (word == 0) return PDATTN_OK;
  // a failed call may have left ticket words and counters half-way: put all of them back to zero
  e = cudaMemsetAsync(workspace, 0, WS_CLEARED_BYTES, stream);
  if (e != cudaSuccess) return cuda_fail("cudaMemsetAsync", e);
  e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail("cudaStreamSynchronize", e);
  if (word & ERR_TIMEOUT) return PDATTN_DEVICE_TIMEOUT;
  if (word & ERR_TOO_LARGE) return PDATTN_UNSUPPORTED;   // the device-side planner refused the batch (tile count)
  return PDATTN_BAD_PAGE_INDEX;
}

}  // extern "C"

// ---- decode without any caller-provided or allocated scratch -----------------------------------
// The scratch of this variant is a fixed array inside the library image.  Every GPU that loads the
// library carries it until the process exits, and every call on a device shares it.
#define PDATTN_STATIC_SCRATCH_BYTES (4u << 20)
#define PDATTN_STATIC_SCRATCH_MAX_SEQS 65536
static __device__ __align__(256) unsigned char g_static_scratch[PDATTN_STATIC_SCRATCH_BYTES];

namespace {
void* g_static_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device
std::mutex g_static_scratch_mu;

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel can
// use; the device address has to be asked for, once per device, with that device current.
pdattn_status static_scratch_address(int dev, uint8_t** out) {
  std::lock_guard<std::mutex> lk(g_static_scratch_mu);
  if (!g_static_scratch_ptr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return cuda_fail("cudaGetSymbolAddress(static scratch)", e);
    if (!p || (reinterpret_cast<uintptr_t>(p) & 255)) {
      snprintf(g_cuda_err, sizeof g_cuda_err, "static scratch address is null or misaligned");
      return PDATTN_CUDA_ERROR;
    }
    g_static_scratch_ptr[dev] = p;
  }
  *out = static_cast<uint8_t*>(g_static_scratch_ptr[dev]);
  return PDATTN_OK;
}
}  // namespace

// ---- the one decode path -----------------------------------------------------------------------
namespace {

pdattn_status decode_common(const pdattn_args* a, const CallDesc& cd, pdattn_stream_t stream_) {
  g_last_launches = 0;
  if (!a) return PDATTN_INVALID_ARG;
  pdattn_status s = check_shape(a->num_seqs, a->num_q_heads, a->num_kv_heads, a->head_dim, a->block_size);
  if (s != PDATTN_OK) return s;
  if (a->num_seqs == 0) return PDATTN_OK;
  if (!a->q || !a->k_cache || !a->v_cache || !a->out || !a->block_table || !a->context_lens) return PDATTN_INVALID_ARG;
  if (!cd.static_scratch && !a->workspace) return PDATTN_INVALID_ARG;
  if (a->max_blocks_per_seq <= 0 || a->num_blocks <= 0) return PDATTN_INVALID_ARG;
  if (a->kv_block_stride <= 0 || a->kv_head_stride <= 0 || a->kv_token_stride < a->head_dim) return PDATTN_INVALID_ARG;
  if ((a->kv_block_stride | a->kv_head_stride | a->kv_token_stride) % 8 != 0) return PDATTN_UNSUPPORTED;
  auto mis = [](const void* p, size_t al) { return (reinterpret_cast<uintptr_t>(p) & (al - 1)) != 0; };
  if (mis(a->q, 16) || mis(a->k_cache, 16) || mis(a->v_cache, 16) || mis(a->out, 16)) return PDATTN_MISALIGNED;
  if (!cd.static_scratch && mis(a->workspace, 256)) return PDATTN_MISALIGNED;
  const int G = a->num_q_heads / a->num_kv_heads;
  const int T = cd.query_tokens;
  const bool grouped = cd.group_size > 0;
  const bool fp8 = cd.fp8;
  if (T < 1) return PDATTN_INVALID_ARG;
  if (G * T > 16 || (T > 1 && grouped)) return PDATTN_UNSUPPORTED;
  if (fp8 && cd.probe) return PDATTN_UNSUPPORTED;
  if (fp8 && (!cd.k_scale || !cd.v_scale)) return PDATTN_INVALID_ARG;
  if (cd.static_scratch && (grouped || fp8 || T != 1 || cd.probe)) return PDATTN_UNSUPPORTED;
  // a context longer than its block_table row can describe is refused here when the host knows the lengths;
  // without a host copy the kernel treats the tokens past the row as a bad page
  if (a->context_lens_host) {
    const int64_t row_tokens = static_cast<int64_t>(a->max_blocks_per_seq) * a->block_size;
    for (int sq = 0; sq < a->num_seqs; ++sq)
      if (a->context_lens_host[sq] > row_tokens) return PDATTN_INVALID_ARG;
  }

  // ---- scratch: the caller's workspace (checked before any CUDA call), or the array built into the library
  // (static spans only, sized by the CTA count).  Grouped calls keep two more arrays behind the ordinary layout.
  auto scratch_need = [&](const WsLayout& w, size_t* off_start, size_t* off_pfx) {
    const size_t pfx_bytes = static_cast<size_t>(a->num_seqs) * a->num_kv_heads * (G > 8 ? 16 : 8) * (a->head_dim + 2) * 4;
    *off_start = w.total;
    *off_pfx = *off_start + align_up(static_cast<size_t>(a->num_seqs) * 4, 256);
    return grouped ? *off_pfx + align_up(pfx_bytes, 256) : w.total;
  };
  WsLayout wl = ws_layout(a->num_seqs, G * T, a->head_dim, MAX_SPANS);
  size_t off_start = 0, off_pfx = 0;
  size_t need = scratch_need(wl, &off_start, &off_pfx);
  if (!cd.static_scratch && a->workspace_bytes < need) return PDATTN_WORKSPACE_TOO_SMALL;

  int dev = 0;
  DevInfo* di = nullptr;
  s = device_info(&dev, &di);
  if (s != PDATTN_OK) return s;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  int n_ctas = di->sm_count;
  if (n_ctas > MAX_SPANS / (1 + kMaxDynPerCta)) n_ctas = MAX_SPANS / (1 + kMaxDynPerCta);

  uint8_t* ws = static_cast<uint8_t*>(a->workspace);
  if (cd.static_scratch) {
    wl = ws_layout(a->num_seqs, G * T, a->head_dim, n_ctas);
    need = scratch_need(wl, &off_start, &off_pfx);
    if (a->num_seqs > PDATTN_STATIC_SCRATCH_MAX_SEQS || need > PDATTN_STATIC_SCRATCH_BYTES) {
      snprintf(g_cuda_err, sizeof g_cuda_err,
               "pdattn_decode_static_scratch: %d sequences need %zu bytes of scratch; the built-in array holds %u "
               "bytes and at most %d sequences",
               a->num_seqs, need, PDATTN_STATIC_SCRATCH_BYTES, PDATTN_STATIC_SCRATCH_MAX_SEQS);
      return PDATTN_WORKSPACE_TOO_SMALL;
    }
    s = static_scratch_address(dev, &ws);
    if (s != PDATTN_OK) return s;
    // The array still holds whatever the previous call left: the error word, the span counter and the
    // ticket words must start at zero; everything else is written before it is read.
    cudaError_t e = cudaMemsetAsync(ws, 0, WS_CLEARED_BYTES, stream);
    if (e != cudaSuccess) return cuda_fail("cudaMemsetAsync(static scratch header)", e);
  }

  const int32_t* start_tiles_host = nullptr;
  int n_groups = 0;
  const bool umma = g_prefix_engine != 0 && !fp8;   // which kernel takes the shared tiles of a grouped call
  if (grouped) {
    const int Gs = cd.group_size;
    // rows the kernel for the shared tiles takes per unit: 64 on tensor memory, 48 with warp MMAs (the only
    // kernel for the shared tiles of an fp8 cache)
    const int max_rows = umma ? UMMA_MAX_QUERY_ROWS : MAX_PREFIX_ROWS;
    if (G > 8 || Gs * G > max_rows) return PDATTN_UNSUPPORTED;
    if (!a->context_lens_host || a->num_seqs % Gs != 0) return PDATTN_INVALID_ARG;
    n_groups = a->num_seqs / Gs;
    g_start_tiles_host.resize(a->num_seqs);
    for (int sq = 0; sq < a->num_seqs; ++sq) {
      const int pt = cd.prefix_tiles_host[sq / Gs];
      // every member must own at least one token past the shared tiles
      if (pt < 0 || static_cast<int64_t>(pt) * kTileTokens >= a->context_lens_host[sq]) return PDATTN_INVALID_ARG;
      if (static_cast<int64_t>(pt) * kTileTokens / a->block_size > a->max_blocks_per_seq) return PDATTN_INVALID_ARG;
      g_start_tiles_host[sq] = pt;
    }
    start_tiles_host = g_start_tiles_host.data();
  }

  static_assert(sizeof(DecodeParams) + 2 * sizeof(CUtensorMap) <= 32000, "kernel parameters");
  DecodeParams P{};
  P.q = static_cast<const __nv_bfloat16*>(a->q);
  P.out = static_cast<__nv_bfloat16*>(a->out);
  P.block_table = a->block_table;
  P.context_lens = a->context_lens;
  P.start_tiles = nullptr;
  P.pfx_partials = nullptr;
  P.hdr = reinterpret_cast<WsHeader*>(ws + wl.hdr);
  P.spans_ws = reinterpret_cast<const SpanStart*>(ws + wl.spans);
  P.rec = reinterpret_cast<int4*>(ws + wl.rec);
  P.partials = reinterpret_cast<float*>(ws + wl.partials);
  P.S = a->num_seqs;
  P.Hq = a->num_q_heads;
  P.Hkv = a->num_kv_heads;
  P.G = G;
  P.T = T;
  P.MB = a->max_blocks_per_seq;
  P.NB = a->num_blocks;
  P.scale_log2 = a->scale * 1.4426950408889634f;
  P.use_ws_plan = 0;
  P.box5d = 0;
  P.k_scale = fp8 ? cd.k_scale : nullptr;
  P.v_scale = fp8 ? cd.v_scale : nullptr;
  P.tickets = reinterpret_cast<int32_t*>(ws + WS_TICKETS_OFFSET);
  // the final merge of cut units: inside the decode kernel with the chained merge (modes -1 and 1) and 8-row
  // tiles, in combine_kernel alone with the barrier merge (0), with 16-row tiles or when asked for (2)
  const bool chain = g_merge_mode != 0;
  P.inkernel_max = (chain && g_merge_mode != 2 && !cd.probe && G * T <= 8) ? kInKernelMergeSpans : 0;

  // Run-time spans even out the CTAs' finishing times when there are many units; with few long sequences
  // they only lengthen the chains the combine kernel walks.  The choice depends on the batch shape alone.
  const int dyn_per_cta =
      cd.static_scratch ? 0
      : g_dyn_per_cta >= 0
          ? g_dyn_per_cta
          : (static_cast<int64_t>(a->num_seqs) * a->num_kv_heads >= static_cast<int64_t>(kAutoDynUnits) * n_ctas
                 ? kAutoDynPerCta
                 : 0);
  int grid = n_ctas, combine_grid = 0, n_spans_host = -1;
  bool win = false;
  if (a->context_lens_host) {
    const int max_param_spans = cd.static_scratch ? n_ctas : MAX_PARAM_SPANS;
    if (!plan_spans(a->context_lens_host, start_tiles_host, a->num_seqs, a->num_kv_heads, n_ctas, dyn_per_cta,
                    max_param_spans, P.spans, &P.plan))
      return PDATTN_INVALID_ARG;
    n_spans_host = P.plan.n_static + P.plan.n_dyn;
    combine_grid = n_spans_host;
    // By default (mode -1) the decode kernel merges its cut units itself only for batches of long pieces (at
    // least kAutoInKernelTiles tiles per unit on average): measured, the warp that does those merges, merely by
    // being resident, costs a batch of short ragged sequences (4096 x U[50,400] tokens) 12 % while it gains
    // 1 - 2 % on the long-context configurations.
    if (g_merge_mode == -1 && P.plan.total < static_cast<int64_t>(kAutoInKernelTiles) * a->num_seqs * a->num_kv_heads)
      P.inkernel_max = 0;
    // Batches of mostly one-tile pieces (below 1.5 tiles per unit on average) take the short-piece instantiation:
    // every warp walks the spans 32 units at a time and the tenth warp stages the query rows instead of merging.
    if (chain && !fp8 && !cd.probe && G * T <= 8 &&
        (g_short_path == 1 ||
         (g_short_path == -1 && 2 * static_cast<int64_t>(P.plan.total) <
                                    static_cast<int64_t>(kAutoShortTilesX2) * a->num_seqs * a->num_kv_heads))) {
      win = true;
      P.inkernel_max = 0;
    }
    {
      // if every cut unit is short enough for the decode kernel's own merge (or no unit is cut at all, as in a
      // batch of one-tile sequences), combine_kernel has nothing to do and is not launched
      bool all_short = true;
      for (int k = 0; k < n_spans_host && all_short; ++k) all_short = merge_run(P.spans[k].merge) <= P.inkernel_max;
      if (all_short) combine_grid = 0;
    }
  } else {
    if (g_merge_mode == -1) P.inkernel_max = 0;   // lengths unknown here: combine_kernel is launched in any case
    P.use_ws_plan = 1;
    memset(&P.plan, 0, sizeof P.plan);
    const int n_dyn_max = n_ctas * dyn_per_cta;
    cudaError_t e = launch_dependent(plan_kernel, 1, 1024, 0, stream, true, a->context_lens,
                                     static_cast<const int32_t*>(nullptr), a->num_seqs, a->num_kv_heads, n_ctas, n_dyn_max,
                                     reinterpret_cast<int32_t*>(ws + wl.prefix),
                                     reinterpret_cast<SpanStart*>(ws + wl.spans), P.hdr, P.inkernel_max > 0 ? 1 : 0);
    if (e != cudaSuccess) return cuda_fail("plan_kernel launch", e);
    g_last_launches += 1;
    combine_grid = n_ctas + n_dyn_max;
  }

  // One TMA op per page-head (rank-5 view) when head_dim is 128; the rank-4 view otherwise, or if
  // the driver refuses the rank-5 encoding.
  static const bool force4d = getenv("PDATTN_BOX4D") != nullptr;
  CUtensorMap mk, mv;
  int rank = (a->head_dim == 128 && !force4d) ? 5 : 4;
  if (fp8) rank = kMapK8;
  s = make_map(a->k_cache, a->head_dim, a->block_size, a->num_kv_heads, a->num_blocks, a->kv_block_stride,
               a->kv_head_stride, a->kv_token_stride, rank, &mk);
  if (s != PDATTN_OK && rank == 5) {
    rank = 4;
    s = make_map(a->k_cache, a->head_dim, a->block_size, a->num_kv_heads, a->num_blocks, a->kv_block_stride,
                 a->kv_head_stride, a->kv_token_stride, rank, &mk);
  }
  if (s != PDATTN_OK) return s;
  s = make_map(a->v_cache, a->head_dim, a->block_size, a->num_kv_heads, a->num_blocks, a->kv_block_stride,
               a->kv_head_stride, a->kv_token_stride, fp8 ? kMapV8 : rank, &mv);
  if (s != PDATTN_OK) return s;
  P.box5d = rank == 5;
  const LaunchCtx lc{a->block_size, chain, cd.probe, fp8, win, di, stream};

  if (grouped) {
    // shared prompt tiles first: one pass per (group, kv head) for the query rows of all samples
    PrefixParams X;
    X.q = P.q;
    X.block_table = a->block_table;
    X.prefix_tiles = cd.prefix_tiles;
    X.start_tiles = reinterpret_cast<int32_t*>(ws + off_start);
    X.pfx_partials = reinterpret_cast<float*>(ws + off_pfx);
    X.err = &P.hdr->err;
    X.S = a->num_seqs;
    X.Hq = a->num_q_heads;
    X.Hkv = a->num_kv_heads;
    X.G = G;
    X.Gs = cd.group_size;
    X.MB = a->max_blocks_per_seq;
    X.NB = a->num_blocks;
    X.scale_log2 = P.scale_log2;
    X.box5d = P.box5d;
    X.k_scale = P.k_scale;
    X.v_scale = P.v_scale;
    // whole units, contiguous ranges of equal tile count (to within one unit)
    const int n_units = n_groups * a->num_kv_heads;
    int64_t total = 0;
    for (int gi = 0; gi < n_groups; ++gi) total += static_cast<int64_t>(cd.prefix_tiles_host[gi]) * a->num_kv_heads;
    int pgrid = n_ctas < 160 ? n_ctas : 160;
    if (pgrid > n_units) pgrid = n_units;
    int u = 0;
    int64_t done = 0;
    for (int c = 0; c < pgrid; ++c) {
      const int64_t target = total * (c + 1) / pgrid;
      const int u0 = u;
      while (u < n_units && (done < target || c == pgrid - 1)) {
        done += cd.prefix_tiles_host[u / a->num_kv_heads];
        ++u;
      }
      X.ranges[c] = make_int2(u0, u);
    }
    if (umma) {
      // tensor-memory kernel: its tiles are laid out per 64-column block, so it takes the rank-4 view
      CUtensorMap pk = mk, pv = mv;
      if (rank != 4) {
        s = make_map(a->k_cache, a->head_dim, a->block_size, a->num_kv_heads, a->num_blocks, a->kv_block_stride,
                     a->kv_head_stride, a->kv_token_stride, 4, &pk);
        if (s != PDATTN_OK) return s;
        s = make_map(a->v_cache, a->head_dim, a->block_size, a->num_kv_heads, a->num_blocks, a->kv_block_stride,
                     a->kv_head_stride, a->kv_token_stride, 4, &pv);
        if (s != PDATTN_OK) return s;
      }
      s = a->head_dim == 128 ? launch_prefix_umma<128>(pk, pv, X, pgrid, lc) : launch_prefix_umma<64>(pk, pv, X, pgrid, lc);
    } else {
      s = a->head_dim == 128 ? launch_prefix<128>(mk, mv, X, pgrid, lc) : launch_prefix<64>(mk, mv, X, pgrid, lc);
    }
    if (s != PDATTN_OK) return s;
    g_last_launches += 1;
    P.start_tiles = X.start_tiles;
    P.pfx_partials = X.pfx_partials;
  }

  const bool nt2 = G * T > 8;
  if (a->head_dim == 128)
    s = nt2 ? launch<128, 2>(mk, mv, P, grid, combine_grid, n_spans_host, lc)
            : launch<128, 1>(mk, mv, P, grid, combine_grid, n_spans_host, lc);
  else
    s = nt2 ? launch<64, 2>(mk, mv, P, grid, combine_grid, n_spans_host, lc)
            : launch<64, 1>(mk, mv, P, grid, combine_grid, n_spans_host, lc);
  if (s != PDATTN_OK) return s;
  if (!cd.probe) g_last_launches += combine_grid > 0 ? 2 : 1;
  if (cd.status_out) {
    cudaError_t e = cudaMemcpyAsync(cd.status_out, ws, 4, cudaMemcpyDeviceToDevice, stream);
    if (e != cudaSuccess) return cuda_fail("cudaMemcpyAsync(status_out)", e);
  }
  return PDATTN_OK;
}

}  // namespace

extern "C" pdattn_status pdattn_decode_static_scratch(const pdattn_args* a, int32_t* status_out,
                                                      pdattn_stream_t stream) {
  CallDesc cd;
  cd.static_scratch = true;
  cd.status_out = status_out;
  return decode_common(a, cd, stream);
}

extern "C" {

pdattn_status pdattn_gather_probe(const pdattn_args* args, pdattn_stream_t stream) {
  CallDesc cd;
  cd.probe = true;
  const pdattn_status s = decode_common(args, cd, stream);
  g_last_launches = 0;   // a probe is not a decode step
  return s;
}

pdattn_status pdattn_wait_limit_probe(void* workspace, int limit_us, pdattn_stream_t stream) {
  if (!workspace || limit_us < 1 || limit_us > 1000000) return PDATTN_INVALID_ARG;
  wait_limit_probe_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      &static_cast<WsHeader*>(workspace)->err, static_cast<unsigned long long>(limit_us) * 1000ull);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail("wait_limit_probe_kernel launch", e);
  return PDATTN_OK;
}

pdattn_status pdattn_stream_read_probe(const void* src, size_t bytes, void* sink, pdattn_stream_t stream) {
  if (!src || !sink || (reinterpret_cast<uintptr_t>(src) & 15)) return PDATTN_INVALID_ARG;
  int dev = 0;
  DevInfo* di = nullptr;
  pdattn_status s = device_info(&dev, &di);
  if (s != PDATTN_OK) return s;
  stream_read_kernel<<<di->sm_count * 4, 512, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(src), bytes / 16, static_cast<uint32_t*>(sink));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail("stream_read_kernel launch", e);
  return PDATTN_OK;
}

pdattn_status pdattn_profile_events(void* start_event, void* stop_event) {
  if ((start_event == nullptr) != (stop_event == nullptr)) return PDATTN_INVALID_ARG;
  g_prof_start = static_cast<cudaEvent_t>(start_event);
  g_prof_stop = static_cast<cudaEvent_t>(stop_event);
  return PDATTN_OK;
}

int pdattn_last_launch_count(void) { return g_last_launches; }

const char* pdattn_status_string(pdattn_status st) {
  switch (st) {
    case PDATTN_OK: return "ok";
    case PDATTN_INVALID_ARG: return "invalid argument";
    case PDATTN_UNSUPPORTED: return "unsupported shape or stride";
    case PDATTN_WORKSPACE_TOO_SMALL: return "workspace too small";
    case PDATTN_MISALIGNED: return "misaligned pointer";
    case PDATTN_NOT_BOUND: return "pdattn_bind was not called on this thread";
    case PDATTN_CUDA_ERROR: return "CUDA error";
    case PDATTN_BAD_PAGE_INDEX: return "block_table entry out of range";
    case PDATTN_DEVICE_TIMEOUT: return "bounded wait expired inside a kernel";
    default: return "unknown status";
  }
}

const char* pdattn_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
