// Launch parameters shared by the split-KV kernels, the merge kernel and the host entry points.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

namespace puzzle {

struct alignas(64) DecodeParams {
  CUtensorMap tmK;  // u8 (or bf16) [num_blocks*Hkv*16 rows][one token row], box = one 16-token block
  CUtensorMap tmV;
  const __nv_bfloat16* q;
  const int32_t* block_table;
  const int32_t* seq_lens;
  const float* k_scale;
  const float* v_scale;
  float* part_o;
  float* part_lse;
  int32_t* dev_status;
  long long num_blocks;
  int batch, Hkv, max_blocks_per_seq, window;
  int num_splits;  // 0 = balanced schedule
  int oob_row;     // a row coordinate outside the tensor maps: loads from it return zeros
  float sm_scale_log2e;
};

struct MergeParams {
  const float* part_o;
  const float* part_lse;
  const int32_t* num_parts;  // explicit layout only
  const float* sinks;
  __nv_bfloat16* out;
  float* lse_out;
  int batch, Hq, D, S;
  // balanced layout: partial rows are addressed as (worker + sequence*Hkv + kv head)*8 + head-in-group
  int balanced;
  const int32_t* seq_lens;
  int Hkv, window, max_tokens, num_workers, tile;
};

// Shape of the two split-KV kernel variants: warps per CTA (each an independent worker), TMA stages per
// warp and tokens per tile (the unit of the schedule and of one pipeline stage).
constexpr int kDecodeWarpsFp8 = 12, kDecodeStagesFp8 = 2, kTileFp8 = 64;
constexpr int kDecodeWarpsBf16 = 12, kDecodeStagesBf16 = 2, kTileBf16 = 32;

// Launches the split-KV kernel for an FP8 (fp8 = true) or bf16 cache on `ctas` CTAs.  attr_done[2] caches,
// per variant, that the dynamic shared-memory limit of the kernel has been raised on the current device.
cudaError_t launch_decode_attn(const DecodeParams& P, bool fp8, int ctas, cudaStream_t s, bool* attr_done);

__global__ void attn_merge_kernel(const MergeParams P);
size_t attn_merge_smem_bytes(int batch, int balanced);

__global__ void kv_append_kernel(void* k_cache, void* v_cache, const __nv_bfloat16* k_new,
                                 const __nv_bfloat16* v_new, const int32_t* block_table, const int32_t* seq_lens,
                                 const float* k_scale, const float* v_scale, long long num_blocks, int batch, int Hkv,
                                 int max_blocks_per_seq, int kv_dtype, int32_t* dev_status);

__global__ void hbm_read_probe_kernel(const uint4* buf, size_t n16, unsigned long long* sink);

}  // namespace puzzle
