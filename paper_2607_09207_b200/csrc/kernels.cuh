// Device code of libpdattn (sm_100a only), one header per part:
//   common.cuh       constants, kernel parameters, PTX wrappers, shared-memory plan, span walk and sequencing
//   tile_bf16.cuh    one 64-token tile on one warp, bf16 cache
//   tile_fp8.cuh     the same over an fp8 (e4m3) cache
//   decode.cuh       decode_kernel: persistent split-KV flash decoding (chained or barrier merge at piece end)
//   prefix_mma.cuh   prefix_kernel: shared prompt tiles of a GRPO group, warp-level MMAs
//   prefix_umma.cuh  prefix_umma_kernel: the same on tcgen05 with tensor-memory operands (included by the API file)
//   aux_kernels.cuh  append_kernel, append_fp8_kernel, stream_read_kernel, combine_kernel, plan_kernel
#pragma once

#include "common.cuh"
#include "tile_bf16.cuh"
#include "tile_fp8.cuh"
#include "decode.cuh"
#include "prefix_mma.cuh"
#include "aux_kernels.cuh"
