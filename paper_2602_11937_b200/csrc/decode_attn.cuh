// Launch parameters shared by the split-KV kernels, the merge kernel and the host entry points.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/puzzle_attn.h"

namespace puzzle {

struct alignas(64) DecodeParams {
  CUtensorMap tmK;  // rows of 128 bytes (two FP8 tokens or one bf16 token), box = one 16-token block of one KV head
  CUtensorMap tmV;
  const __nv_bfloat16* q;
  const int32_t* block_table;
  const int32_t* seq_lens;
  const float* k_scale;
  const float* v_scale;
  float* part_o;
  float* part_lse;
  int32_t* counters;   // [batch*Hkv] arrivals per (sequence, KV head); zero before and after every launch
  int32_t* cta_words;  // CTA-balanced kernel only: its CTA counter, buffer switch and the two speed buffers
  const float* sinks;  // [Hq] or null
  __nv_bfloat16* out;  // [batch][Hq][D]
  float* out_f32;      // when set, the merged rows are stored here as float32 instead (out is unused)
  float* lse_out;      // [batch][Hq] or null
  int32_t* dev_status;
  long long num_blocks;
  int batch, Hkv, max_blocks_per_seq, window;
  int num_splits;  // 0 = balanced schedule
  int n_q;         // multi-token kernel: query tokens per sequence in q / out ([batch][n_q][Hq][D]); else unused
  const int32_t* q_lens;  // multi-token kernel: real query tokens per sequence [batch], or null (= n_q)
  int oob_row;     // a row coordinate outside the tensor maps: loads from it return zeros
  int rows_per_block;  // tensor-map rows (128 bytes each) per (block, KV head): 8 (FP8) or 16 (bf16)
  float sm_scale_log2e;
};

struct MergeParams {
  const float* part_o;       // part k of row r starts at part_o + r * o_row_stride + k * o_part_stride
  const float* part_lse;     // part k of row r is part_lse[r * lse_row_stride + k * lse_part_stride]
  long long o_row_stride, o_part_stride, lse_row_stride, lse_part_stride;   // in floats
  const int32_t* num_parts;  // [batch] or null
  const float* sinks;
  __nv_bfloat16* out;
  float* lse_out;
  int batch, Hq, D, S;
};

// Shape of the two split-KV kernel variants: warps per CTA (each an independent worker), TMA stages per
// warp and tokens per tile (the unit of the schedule and of one pipeline stage).
constexpr int kDecodeWarpsFp8 = 12, kDecodeStagesFp8 = 2, kTileFp8 = 64;
constexpr int kDecodeWarpsBf16 = 12, kDecodeStagesBf16 = 2, kTileBf16 = 32;
// The CTA-balanced kernel keeps its schedule arrays beside the TMA rings and the deposit buffers in shared memory,
// which bounds the batch it takes.  Launches with at least kCtaRateMinTiles tiles per CTA note the speed of every
// CTA slot at the start of the workspace (before the arrival counters: a CTA counter, the buffer switch, two pad words, then two
// float buffers of one speed per CTA) and are cut by the speeds the launch before them noted.
constexpr int kCtaMaxBatch = 1024;
constexpr int kCtaMinTilesPerCta = 64;   // below this bound on the tiles per CTA the warp-scheduled kernel is used (more with short pairs)
constexpr int kCtaRateMinTiles = 256;
constexpr int kWholePairTiles = 4;       // up to this many tiles per (sequence, KV head) a pair goes to one warp whole
inline size_t cta_rate_words(int ctas) { return 4 + 2 * (size_t)ctas; }

// Launches the split-KV kernel for an FP8 (fp8 = true) or bf16 cache on `ctas` CTAs.  smem_limit[2] caches,
// per variant, the dynamic shared-memory limit set for the kernel on the current device (0 = not set yet).
cudaError_t launch_decode_attn(const DecodeParams& P, bool fp8, int ctas, cudaStream_t s, int* smem_limit);
// The CTA-balanced kernel (balanced schedule only, batch <= kCtaMaxBatch).  Its partial row blocks: one per
// (CTA, pair) meeting, ctas + batch*Hkv at most.
cudaError_t launch_decode_attn_cta(const DecodeParams& P, bool fp8, int ctas, cudaStream_t s, int* smem_limit);
// The kernel for launches in which no (sequence, KV head) has more than kWholePairTiles tiles (narrow windows, very
// short contexts): a group of four warps per pair, one tile each, combined in shared memory; no workspace use.
// smem_limit[2] as above.  It pays up to decode_attn_small_max_pairs(ctas) pairs; beyond, the warp-scheduled kernel
// with one split per pair keeps its TMA rings full.
cudaError_t launch_decode_attn_small(const DecodeParams& P, bool fp8, int ctas, cudaStream_t s, int* smem_limit);
int decode_attn_small_max_pairs(int ctas);
// The multi-token kernel (FP8 cache, balanced schedule): P.n_q, P.q_lens set; P.counters has one word per
// (sequence, token pair, KV head); partial rows: decode_attn_tokens_partial_rows(...).
cudaError_t launch_decode_attn_tokens(const DecodeParams& P, int ctas, cudaStream_t s, int* smem_limit);
size_t decode_attn_tokens_partial_rows(int ctas, int batch, int n_q, int Hkv);
size_t decode_attn_tokens_counters(int batch, int n_q, int Hkv);
constexpr int kTokMaxRows = 8192;   // (sequence, token pair) rows its shared-memory schedule holds

// The tensor-memory (tcgen05) kernel for the FP8 cache.  Its tensor maps view the cache as rows of 64 bytes
// (one token), box = 16 rows, 64-byte swizzle; P.rows_per_block is 16 and P.oob_row counts such rows.
cudaError_t launch_decode_attn_tc(const DecodeParams& P, int ctas, cudaStream_t s, int* smem_limit);
int decode_attn_tc_workers_per_cta();

// Host-visible argument checks of the decode-attention entry points (everything but the workspace).
puzzle_status check_decode_attn_args(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q,
                                     const void* out, int batch, int num_splits, bool tcgen05);

__global__ void attn_merge_kernel(const MergeParams P);

__global__ void kv_append_kernel(void* k_cache, void* v_cache, const __nv_bfloat16* k_new,
                                 const __nv_bfloat16* v_new, const int32_t* block_table, const int32_t* seq_lens,
                                 const float* k_scale, const float* v_scale, long long num_blocks, int batch, int Hkv,
                                 int max_blocks_per_seq, int kv_dtype, int32_t* dev_status);

__global__ void kv_append_tokens_kernel(void* k_cache, void* v_cache, const uint4* k_new, const uint4* v_new,
                                        const int32_t* new_lens, const int32_t* block_table, const int32_t* seq_lens,
                                        const float* k_scale, const float* v_scale, long long num_blocks, int batch,
                                        int n_new, int Hkv, int max_blocks_per_seq, int kv_dtype, int32_t* dev_status);
__global__ void hbm_read_probe_kernel(const uint4* buf, size_t n16, unsigned long long* sink);

// Max calibration (calibrate.cu).
cudaError_t launch_amax_update(const void* x, long long n_tokens, int Hkv, int D, float* amax, int sm_count,
                               cudaStream_t s);
cudaError_t launch_scales_from_amax(const float* amax, int Hkv, int pow2, float* scale, cudaStream_t s);
int calibrate_max_heads();

}  // namespace puzzle
