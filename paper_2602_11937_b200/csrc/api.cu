// Host side of the C ABI declared in include/puzzle_attn.h: argument checks, TMA descriptor
// encoding and kernel launches.  No allocation, no synchronisation, no state besides a launch counter.
#include <algorithm>
#include <atomic>
#include <cstring>

#include "common.cuh"
#include "decode_attn.cuh"

namespace puzzle {

static std::atomic<long long> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

struct DeviceInfo {
  int sm_count = 0;
  // per split-KV kernel (warp-scheduled FP8, bf16; tensor-memory FP8; CTA-balanced FP8, bf16); 0 = not raised yet
  int smem_limit[8] = {0, 0, 0, 0, 0, 0, 0, 0};   // [5]: the multi-token kernel, [6..7]: the small-launch kernel
};
DeviceInfo& device_info() {
  static DeviceInfo info[64];
  int dev = 0;
  cudaGetDevice(&dev);
  DeviceInfo& d = info[dev & 63];
  if (d.sm_count == 0) cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev);
  return d;
}

puzzle_status check_desc(const puzzle_layer_desc* d) {
  if (!d) return PUZZLE_ERR_NULL;
  if (d->num_q_heads <= 0 || d->num_kv_heads <= 0 || d->head_dim <= 0 || d->block_size <= 0 || d->window < 0)
    return PUZZLE_ERR_SHAPE;
  if (d->num_q_heads % d->num_kv_heads != 0) return PUZZLE_ERR_SHAPE;
  if (d->kv_dtype != PUZZLE_KV_FP8_E4M3 && d->kv_dtype != PUZZLE_KV_BF16) return PUZZLE_ERR_SHAPE;
  if (d->head_dim != kHeadDim || d->block_size != kBlock || d->num_q_heads != kGroup * d->num_kv_heads)
    return PUZZLE_ERR_UNSUPPORTED;
  return PUZZLE_OK;
}

puzzle_status check_view(const puzzle_layer_desc* d, const puzzle_kv_view* kv, int batch) {
  if (!kv || !kv->k_cache || !kv->v_cache || !kv->seq_lens) return PUZZLE_ERR_NULL;
  if (batch <= 0 || kv->num_blocks <= 0 || kv->max_blocks_per_seq <= 0) return PUZZLE_ERR_SHAPE;
  if (batch > kMaxBatch) return PUZZLE_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(kv->k_cache) & 15) || (reinterpret_cast<uintptr_t>(kv->v_cache) & 15))
    return PUZZLE_ERR_SHAPE;
  // rows of the 2-D view of the cache must fit a signed 32-bit TMA coordinate
  if (kv->num_blocks * d->num_kv_heads * (long long)kBlock >= (1ll << 31) - 64) return PUZZLE_ERR_UNSUPPORTED;
  if (!kv->block_table && (long long)batch * kv->max_blocks_per_seq > kv->num_blocks) return PUZZLE_ERR_SHAPE;
  return PUZZLE_OK;
}

// 2-D view of a cache as rows of 128 bytes: two FP8 tokens or one bf16 token per row, so that every TMA
// request is a full 128-byte line.  Box = one 16-token block of one KV head (8 or 16 rows), 128-byte swizzle.
// row_bytes = 64 (FP8 only): one token per row, 16 rows per block, 64-byte swizzle (the tensor-memory kernel's view).
bool make_cache_map(CUtensorMap* m, void* base, long long rows, int elem_bytes, int row_bytes = 128) {
  EncodeTiledFn enc = encode_tiled();
  if (!enc) return false;
  if (row_bytes == 64) {
    const cuuint64_t dims[2] = {64, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {64};
    const cuuint32_t box[2] = {64, (cuuint32_t)kBlock};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
  const cuuint64_t inner = 128 / elem_bytes;  // elements per row
  const cuuint64_t dims[2] = {inner, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {128};
  const cuuint32_t box[2] = {(cuuint32_t)inner, (cuuint32_t)(kBlock * kHeadDim * elem_bytes / 128)};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(m, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base,
                   dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int grid_ctas() { return device_info().sm_count > 0 ? device_info().sm_count : 1; }

int decode_warps(int kv_dtype) { return kv_dtype == PUZZLE_KV_FP8_E4M3 ? kDecodeWarpsFp8 : kDecodeWarpsBf16; }

// The workspace starts with the CTA-speed words of the CTA-balanced kernel, then one arrival counter per (sequence,
// KV head), then the partials.  Every completed call leaves the arrival counters at zero.  The counter block has room
// for kCounterFloor counters whatever the batch, so that up to that many (sequence, KV head) pairs the partials of
// one call never lie where another call's counters do: one prepared workspace then serves calls of different batch
// sizes one after the other.  Beyond the floor the layout follows the batch.
constexpr size_t kCounterFloor = 16384;
size_t cta_word_bytes() { return (cta_rate_words(grid_ctas()) * sizeof(int32_t) + 255) & ~(size_t)255; }
size_t counter_bytes(int batch, int Hkv) {
  const size_t n = std::max((size_t)batch * Hkv, kCounterFloor);
  return cta_word_bytes() + ((n * sizeof(int32_t) + 255) & ~(size_t)255);
}

// The balanced schedule runs on the CTA-balanced kernel when the batch fits its shared-memory schedule and the
// launch can be large: with at most a few tiles per warp (window layers, short contexts) a launch is a chain of
// latencies, which the warp-scheduled kernel's shorter set-up serves better.  The bound on the tiles comes from
// what the host knows: the window, or the length of a block-table row.
// Upper bound on the tiles of one (sequence, KV head) from what the host knows.
long long tiles_per_pair_bound(const puzzle_layer_desc* d, const puzzle_kv_view* kv) {
  const int tt = d->kv_dtype == PUZZLE_KV_FP8_E4M3 ? kTileFp8 : kTileBf16;
  long long per_pair = ((long long)kv->max_blocks_per_seq * kBlock + tt - 1) / tt;
  if (d->window > 0) per_pair = std::min<long long>(per_pair, (d->window + tt - 1) / tt + 1);
  return per_pair;
}

bool use_cta_kernel(const puzzle_layer_desc* d, const puzzle_kv_view* kv, int batch, int num_splits) {
  if (num_splits == PUZZLE_SCHED_CTA) return true;
  if (num_splits != 0 || batch > kCtaMaxBatch) return false;
  // What the CTA-balanced kernel wins (no tail, CTAs cut by speed) grows with the length of the launch and of the
  // pairs; what it costs (a longer set-up, a claim and a hand-over per piece) weighs most on many short pairs.
  // Measured crossovers, in tiles per CTA: 64 with pairs of 256 tiles or more, about 200 at 128 tiles per pair,
  // about 600 below.
  const long long per_pair = tiles_per_pair_bound(d, kv);
  const long long min_per_cta = per_pair >= 256 ? kCtaMinTilesPerCta : (per_pair >= 128 ? 200 : 600);
  return per_pair * batch * d->num_kv_heads >= min_per_cta * grid_ctas();
}

// The kernel a call of puzzle_decode_attn runs on.
enum class Kernel { kCta, kWarp, kWarpWholePairs, kSmall };
Kernel pick_kernel(const puzzle_layer_desc* d, const puzzle_kv_view* kv, int batch, int num_splits) {
  if (use_cta_kernel(d, kv, batch, num_splits)) return Kernel::kCta;
  // Narrow windows and short contexts: with at most kWholePairTiles tiles per (sequence, KV head) a pair is not cut
  // at all.  A group of four warps (few pairs) or one warp (many pairs, or the warp-scheduled kernel pinned) takes
  // it whole and stores the output itself, which drops the partial, the arrival and the merge (three dependent
  // trips through L2) from a launch that is a chain of latencies anyway.
  const bool whole_pairs = num_splits <= 0 && tiles_per_pair_bound(d, kv) <= kWholePairTiles;
  if (!whole_pairs) return Kernel::kWarp;
  if (num_splits == 0 && (long long)batch * d->num_kv_heads <= decode_attn_small_max_pairs(grid_ctas()))
    return Kernel::kSmall;
  return Kernel::kWarpWholePairs;
}

size_t workspace_floats(int batch, int Hkv, int num_splits, int kv_dtype) {
  size_t rows;
  if (num_splits == 0) {
    // one row block per (worker, pair) meeting of the warp-scheduled kernels (the CTA-balanced kernel needs one
    // per (CTA, pair) meeting only, the tensor-memory kernel one per (worker, pair) with fewer workers)
    rows = ((size_t)grid_ctas() * decode_warps(kv_dtype) + (size_t)batch * Hkv) * kGroup;
  } else {
    rows = (size_t)batch * Hkv * kGroup * num_splits;
  }
  return rows * (kHeadDim + 1);
}

}  // namespace

// Everything about a decode-attention call that the host can check, short of the workspace.
puzzle_status check_decode_attn_args(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q,
                                     const void* out, int batch, int num_splits, bool tcgen05) {
  puzzle_status st = check_desc(desc);
  if (st != PUZZLE_OK) return st;
  st = check_view(desc, kv, batch);
  if (st != PUZZLE_OK) return st;
  if (!q || !out) return PUZZLE_ERR_NULL;
  if (num_splits < PUZZLE_SCHED_WARP || num_splits > 65536) return PUZZLE_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(q) & 7) || (reinterpret_cast<uintptr_t>(out) & 15)) return PUZZLE_ERR_SHAPE;
  if (num_splits == PUZZLE_SCHED_CTA && (tcgen05 || batch > kCtaMaxBatch)) return PUZZLE_ERR_UNSUPPORTED;
  if (tcgen05 && desc->kv_dtype != PUZZLE_KV_FP8_E4M3) return PUZZLE_ERR_UNSUPPORTED;   // that kernel reads E4M3 codes only
  return PUZZLE_OK;
}

}  // namespace puzzle

using namespace puzzle;

extern "C" {

const char* puzzle_status_string(puzzle_status s) {
  switch (s) {
    case PUZZLE_OK: return "ok";
    case PUZZLE_ERR_NULL: return "a required pointer is NULL";
    case PUZZLE_ERR_SHAPE: return "inconsistent or out-of-range sizes";
    case PUZZLE_ERR_UNSUPPORTED: return "shape or dtype not supported by this build";
    case PUZZLE_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case PUZZLE_ERR_CUDA: return "a CUDA call or kernel launch failed";
  }
  return "unknown status";
}

int64_t puzzle_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* puzzle_decode_attn_kernel_name(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, int32_t batch,
                                           int32_t num_splits) {
  if (check_desc(desc) != PUZZLE_OK || !kv || batch <= 0 || batch > kMaxBatch || num_splits < PUZZLE_SCHED_WARP)
    return "invalid arguments";
  switch (pick_kernel(desc, kv, batch, num_splits)) {
    case Kernel::kCta: return "decode_attn_cta_kernel";
    case Kernel::kSmall: return "decode_attn_small_kernel";
    default: return "decode_attn_kernel";
  }
}

puzzle_status puzzle_kv_append(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* k_new,
                               const void* v_new, int32_t batch, int32_t* dev_status, void* stream) {
  puzzle_status st = check_desc(desc);
  if (st != PUZZLE_OK) return st;
  st = check_view(desc, kv, batch);
  if (st != PUZZLE_OK) return st;
  if (!k_new || !v_new) return PUZZLE_ERR_NULL;
  const long long threads = 2ll * batch * desc->num_kv_heads * (kHeadDim / 2);
  const int grid = (int)((threads + 255) / 256);
  const cudaError_t e = launch_dependent(
      kv_append_kernel, dim3(grid), dim3(256), 0, static_cast<cudaStream_t>(stream), kv->k_cache, kv->v_cache,
      static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new), kv->block_table,
      kv->seq_lens, kv->k_scale, kv->v_scale, kv->num_blocks, batch, desc->num_kv_heads, kv->max_blocks_per_seq,
      desc->kv_dtype, dev_status);
  count_launch();
  return e == cudaSuccess ? PUZZLE_OK : PUZZLE_ERR_CUDA;
}

puzzle_status puzzle_kv_append_tokens(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* k_new,
                                      const void* v_new, const int32_t* new_lens, int32_t batch, int32_t n_new,
                                      int32_t* dev_status, void* stream) {
  puzzle_status st = check_desc(desc);
  if (st != PUZZLE_OK) return st;
  st = check_view(desc, kv, batch);
  if (st != PUZZLE_OK) return st;
  if (!k_new || !v_new) return PUZZLE_ERR_NULL;
  if (n_new <= 0 || n_new > (1 << 20)) return PUZZLE_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(k_new) & 15) || (reinterpret_cast<uintptr_t>(v_new) & 15)) return PUZZLE_ERR_SHAPE;
  const long long per_seq = (long long)n_new * desc->num_kv_heads * (kHeadDim / 8);
  if (per_seq > 0x7fffffffll || batch > 65535) return PUZZLE_ERR_SHAPE;
  const dim3 grid((unsigned)((per_seq + 255) / 256), (unsigned)batch, 2);
  const cudaError_t e = launch_dependent(
      kv_append_tokens_kernel, grid, dim3(256), 0, static_cast<cudaStream_t>(stream), kv->k_cache, kv->v_cache,
      static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), new_lens, kv->block_table, kv->seq_lens,
      kv->k_scale, kv->v_scale, kv->num_blocks, batch, n_new, desc->num_kv_heads, kv->max_blocks_per_seq,
      desc->kv_dtype, dev_status);
  count_launch();
  return e == cudaSuccess ? PUZZLE_OK : PUZZLE_ERR_CUDA;
}

size_t puzzle_decode_attn_workspace_bytes(const puzzle_layer_desc* desc, int32_t batch, int32_t num_splits) {
  if (check_desc(desc) != PUZZLE_OK || batch <= 0 || batch > kMaxBatch || num_splits < PUZZLE_SCHED_WARP) return 0;
  return counter_bytes(batch, desc->num_kv_heads) +
         workspace_floats(batch, desc->num_kv_heads, num_splits > 0 ? num_splits : 0, desc->kv_dtype) * sizeof(float);
}

static puzzle_status decode_attn_impl(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q,
                                      const float* sinks, void* out, float* lse_out, int32_t batch,
                                      int32_t num_splits, void* workspace, size_t workspace_bytes,
                                      int32_t* dev_status, void* stream, bool tcgen05, bool out_f32 = false) {
  puzzle_status st = check_decode_attn_args(desc, kv, q, out, batch, num_splits, tcgen05);
  if (st != PUZZLE_OK) return st;
  const int Hkv = desc->num_kv_heads;
  const bool fp8 = desc->kv_dtype == PUZZLE_KV_FP8_E4M3;
  const size_t cbytes = counter_bytes(batch, Hkv);
  const int splits = num_splits > 0 ? num_splits : 0;   // the kernels know explicit splits (S) and balanced (0)
  const size_t pfloats = workspace_floats(batch, Hkv, splits, desc->kv_dtype);
  const size_t need = cbytes + pfloats * sizeof(float);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 15)) return PUZZLE_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  const int ctas = grid_ctas();
  const size_t rows = pfloats / (kHeadDim + 1);
  float* part_o = reinterpret_cast<float*>(static_cast<char*>(workspace) + cbytes);
  float* part_lse = part_o + rows * kHeadDim;

  DecodeParams P;
  std::memset(&P, 0, sizeof P);
  const int eb = fp8 ? 1 : 2;
  const bool tc = tcgen05;
  const int row_bytes = tc ? 64 : 128;
  const int rows_per_block = kBlock * kHeadDim * eb / row_bytes;
  const long long cache_rows = kv->num_blocks * Hkv * (long long)rows_per_block;
  if (!make_cache_map(&P.tmK, kv->k_cache, cache_rows, eb, row_bytes) ||
      !make_cache_map(&P.tmV, kv->v_cache, cache_rows, eb, row_bytes))
    return PUZZLE_ERR_CUDA;
  P.q = static_cast<const __nv_bfloat16*>(q);
  P.block_table = kv->block_table;
  P.seq_lens = kv->seq_lens;
  P.k_scale = kv->k_scale;
  P.v_scale = kv->v_scale;
  P.part_o = part_o;
  P.part_lse = part_lse;
  P.cta_words = static_cast<int32_t*>(workspace);
  P.counters = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + cta_word_bytes());
  P.sinks = sinks;
  P.out = out_f32 ? nullptr : static_cast<__nv_bfloat16*>(out);
  P.out_f32 = out_f32 ? static_cast<float*>(out) : nullptr;
  P.lse_out = lse_out;
  P.dev_status = dev_status;
  P.num_blocks = kv->num_blocks;
  P.batch = batch;
  P.Hkv = Hkv;
  P.max_blocks_per_seq = kv->max_blocks_per_seq;
  P.window = desc->window;
  P.num_splits = splits;
  P.oob_row = (int)cache_rows;
  P.rows_per_block = rows_per_block;
  P.sm_scale_log2e = desc->sm_scale * 1.4426950408889634f;

  cudaError_t le;
  if (tc) {
    le = launch_decode_attn_tc(P, ctas, s, device_info().smem_limit + 2);
  } else {
    switch (pick_kernel(desc, kv, batch, num_splits)) {
      case Kernel::kCta:
        le = launch_decode_attn_cta(P, fp8, ctas, s, device_info().smem_limit + 3);
        break;
      case Kernel::kSmall:
        le = launch_decode_attn_small(P, fp8, ctas, s, device_info().smem_limit + 6);
        break;
      case Kernel::kWarpWholePairs:
        P.num_splits = 1;
        le = launch_decode_attn(P, fp8, ctas, s, device_info().smem_limit);
        break;
      default:
        le = launch_decode_attn(P, fp8, ctas, s, device_info().smem_limit);
    }
  }
  if (le != cudaSuccess) return PUZZLE_ERR_CUDA;
  count_launch();

  return PUZZLE_OK;
}

puzzle_status puzzle_decode_attn(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q,
                                 const float* sinks, void* out, float* lse_out, int32_t batch, int32_t num_splits,
                                 void* workspace, size_t workspace_bytes, int32_t* dev_status, void* stream) {
  return decode_attn_impl(desc, kv, q, sinks, out, lse_out, batch, num_splits, workspace, workspace_bytes, dev_status,
                          stream, false);
}

puzzle_status puzzle_decode_attn_tcgen05(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q,
                                         const float* sinks, void* out, float* lse_out, int32_t batch,
                                         int32_t num_splits, void* workspace, size_t workspace_bytes,
                                         int32_t* dev_status, void* stream) {
  return decode_attn_impl(desc, kv, q, sinks, out, lse_out, batch, num_splits, workspace, workspace_bytes, dev_status,
                          stream, true);
}

// Device staging of one step whose inputs and result live in host memory: q, k_new, v_new, out, each padded to 256 bytes.
static size_t staging_part(size_t elems) { return (elems * sizeof(__nv_bfloat16) + 255) & ~(size_t)255; }

size_t puzzle_decode_step_host_staging_bytes(const puzzle_layer_desc* desc, int32_t batch) {
  if (check_desc(desc) != PUZZLE_OK || batch <= 0 || batch > kMaxBatch) return 0;
  const size_t qn = (size_t)batch * desc->num_q_heads * desc->head_dim, kn = (size_t)batch * desc->num_kv_heads * desc->head_dim;
  return 2 * staging_part(qn) + 2 * staging_part(kn);
}

puzzle_status puzzle_decode_step_host(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q_host,
                                      const void* k_new_host, const void* v_new_host, const float* sinks,
                                      void* out_host, int32_t batch, int32_t num_splits, void* staging,
                                      size_t staging_bytes, void* workspace, size_t workspace_bytes,
                                      int32_t* dev_status, void* stream) {
  if (!q_host || !k_new_host || !v_new_host || !out_host) return PUZZLE_ERR_NULL;
  const size_t need = puzzle_decode_step_host_staging_bytes(desc, batch);
  if (need == 0) return check_desc(desc) != PUZZLE_OK ? check_desc(desc) : PUZZLE_ERR_SHAPE;
  if (!staging || staging_bytes < need || (reinterpret_cast<uintptr_t>(staging) & 255)) return PUZZLE_ERR_WORKSPACE;
  const size_t qn = (size_t)batch * desc->num_q_heads * desc->head_dim, kn = (size_t)batch * desc->num_kv_heads * desc->head_dim;
  char* dq = static_cast<char*>(staging);
  char* dk = dq + staging_part(qn);
  char* dv = dk + staging_part(kn);
  char* dout = dv + staging_part(kn);
  // every host-visible error of the two device calls is found before the first copy is enqueued
  puzzle_status st = check_decode_attn_args(desc, kv, dq, dout, batch, num_splits, false);
  if (st != PUZZLE_OK) return st;
  if (!workspace || workspace_bytes < puzzle_decode_attn_workspace_bytes(desc, batch, num_splits) ||
      (reinterpret_cast<uintptr_t>(workspace) & 15))
    return PUZZLE_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t qb = qn * sizeof(__nv_bfloat16), kb = kn * sizeof(__nv_bfloat16);
  const char* hq = static_cast<const char*>(q_host);
  if (static_cast<const char*>(k_new_host) == hq + qb && static_cast<const char*>(v_new_host) == hq + qb + kb &&
      qb % 256 == 0 && kb % 256 == 0) {
    // the three inputs follow each other in host memory as they do in the staging area: one copy
    if (cudaMemcpyAsync(dq, q_host, qb + 2 * kb, cudaMemcpyHostToDevice, s) != cudaSuccess) return PUZZLE_ERR_CUDA;
  } else if (cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
             cudaMemcpyAsync(dk, k_new_host, kb, cudaMemcpyHostToDevice, s) != cudaSuccess ||
             cudaMemcpyAsync(dv, v_new_host, kb, cudaMemcpyHostToDevice, s) != cudaSuccess) {
    return PUZZLE_ERR_CUDA;
  }
  st = puzzle_kv_append(desc, kv, dk, dv, batch, dev_status, stream);
  if (st != PUZZLE_OK) return st;
  st = puzzle_decode_attn(desc, kv, dq, sinks, dout, nullptr, batch, num_splits, workspace, workspace_bytes, dev_status,
                          stream);
  if (st != PUZZLE_OK) return st;
  return cudaMemcpyAsync(out_host, dout, qn * sizeof(__nv_bfloat16), cudaMemcpyDeviceToHost, s) == cudaSuccess
             ? PUZZLE_OK
             : PUZZLE_ERR_CUDA;
}

puzzle_status puzzle_decode_attn_partial(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q,
                                         float* o_part, float* lse_part, int32_t batch, int32_t num_splits,
                                         void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                         void* stream) {
  if (!lse_part) return PUZZLE_ERR_NULL;
  return decode_attn_impl(desc, kv, q, nullptr, o_part, lse_part, batch, num_splits, workspace, workspace_bytes,
                          dev_status, stream, false, true);
}

// Room for the largest supported batch * ceil(n_q / 2) whatever the call's own, for the same reason as counter_bytes.
static size_t tokens_counter_bytes(int batch, int n_q, int Hkv) {
  const size_t n = std::max<size_t>(decode_attn_tokens_counters(batch, n_q, Hkv), (size_t)kTokMaxRows * Hkv);
  return (n * sizeof(int32_t) + 255) & ~(size_t)255;
}

size_t puzzle_decode_attn_tokens_workspace_bytes(const puzzle_layer_desc* desc, int32_t batch, int32_t n_q) {
  if (check_desc(desc) != PUZZLE_OK || batch <= 0 || n_q <= 0 || (long long)batch * ((n_q + 1) / 2) > kTokMaxRows)
    return 0;
  return tokens_counter_bytes(batch, n_q, desc->num_kv_heads) +
         decode_attn_tokens_partial_rows(grid_ctas(), batch, n_q, desc->num_kv_heads) * (kHeadDim + 1) * sizeof(float);
}

puzzle_status puzzle_decode_attn_tokens_workspace_init(const puzzle_layer_desc* desc, int32_t batch, int32_t n_q,
                                                       void* workspace, size_t workspace_bytes, void* stream) {
  puzzle_status st = check_desc(desc);
  if (st != PUZZLE_OK) return st;
  if (batch <= 0 || n_q <= 0 || (long long)batch * ((n_q + 1) / 2) > kTokMaxRows) return PUZZLE_ERR_SHAPE;
  const size_t cbytes = tokens_counter_bytes(batch, n_q, desc->num_kv_heads);
  if (!workspace || workspace_bytes < cbytes || (reinterpret_cast<uintptr_t>(workspace) & 15))
    return PUZZLE_ERR_WORKSPACE;
  return cudaMemsetAsync(workspace, 0, cbytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? PUZZLE_OK
                                                                                                  : PUZZLE_ERR_CUDA;
}

puzzle_status puzzle_decode_attn_tokens(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q,
                                        const int32_t* q_lens, const float* sinks, void* out, float* lse_out,
                                        int32_t batch, int32_t n_q, void* workspace, size_t workspace_bytes,
                                        int32_t* dev_status, void* stream) {
  puzzle_status st = check_decode_attn_args(desc, kv, q, out, batch, 0, false);
  if (st != PUZZLE_OK) return st;
  if (n_q <= 0 || (long long)batch * ((n_q + 1) / 2) > kTokMaxRows) return PUZZLE_ERR_SHAPE;
  if (desc->kv_dtype != PUZZLE_KV_FP8_E4M3) return PUZZLE_ERR_UNSUPPORTED;   // the bf16 cache goes one row per token
  const int Hkv = desc->num_kv_heads;
  const size_t need = puzzle_decode_attn_tokens_workspace_bytes(desc, batch, n_q);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 15)) return PUZZLE_ERR_WORKSPACE;
  const size_t cbytes = tokens_counter_bytes(batch, n_q, Hkv);
  const size_t rows = decode_attn_tokens_partial_rows(grid_ctas(), batch, n_q, Hkv);
  DecodeParams P;
  std::memset(&P, 0, sizeof P);
  const long long cache_rows = kv->num_blocks * Hkv * (long long)(kBlock * kHeadDim / 128);
  if (!make_cache_map(&P.tmK, kv->k_cache, cache_rows, 1) || !make_cache_map(&P.tmV, kv->v_cache, cache_rows, 1))
    return PUZZLE_ERR_CUDA;
  P.q = static_cast<const __nv_bfloat16*>(q);
  P.block_table = kv->block_table;
  P.seq_lens = kv->seq_lens;
  P.k_scale = kv->k_scale;
  P.v_scale = kv->v_scale;
  P.part_o = reinterpret_cast<float*>(static_cast<char*>(workspace) + cbytes);
  P.part_lse = P.part_o + rows * kHeadDim;
  P.counters = static_cast<int32_t*>(workspace);
  P.sinks = sinks;
  P.out = static_cast<__nv_bfloat16*>(out);
  P.lse_out = lse_out;
  P.dev_status = dev_status;
  P.num_blocks = kv->num_blocks;
  P.batch = batch;
  P.Hkv = Hkv;
  P.max_blocks_per_seq = kv->max_blocks_per_seq;
  P.window = desc->window;
  P.n_q = n_q;
  P.q_lens = q_lens;
  P.oob_row = (int)cache_rows;
  P.rows_per_block = kBlock * kHeadDim / 128;
  P.sm_scale_log2e = desc->sm_scale * 1.4426950408889634f;
  if (launch_decode_attn_tokens(P, grid_ctas(), static_cast<cudaStream_t>(stream), device_info().smem_limit + 5) !=
      cudaSuccess)
    return PUZZLE_ERR_CUDA;
  count_launch();
  return PUZZLE_OK;
}

puzzle_status puzzle_decode_attn_workspace_init(const puzzle_layer_desc* desc, int32_t batch, void* workspace,
                                                size_t workspace_bytes, void* stream) {
  puzzle_status st = check_desc(desc);
  if (st != PUZZLE_OK) return st;
  if (batch <= 0 || batch > kMaxBatch) return PUZZLE_ERR_SHAPE;
  const size_t cbytes = counter_bytes(batch, desc->num_kv_heads);
  if (!workspace || workspace_bytes < cbytes || (reinterpret_cast<uintptr_t>(workspace) & 15))
    return PUZZLE_ERR_WORKSPACE;
  return cudaMemsetAsync(workspace, 0, cbytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? PUZZLE_OK
                                                                                                  : PUZZLE_ERR_CUDA;
}

puzzle_status puzzle_kv_amax_update(const void* x, int64_t n_tokens, int32_t num_kv_heads, int32_t head_dim,
                                    float* amax, void* stream) {
  if (!amax || (!x && n_tokens > 0)) return PUZZLE_ERR_NULL;
  if (n_tokens < 0 || num_kv_heads <= 0 || num_kv_heads > calibrate_max_heads() || head_dim <= 0 || head_dim % 8)
    return PUZZLE_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(amax) & 3)) return PUZZLE_ERR_SHAPE;
  if (n_tokens == 0) return PUZZLE_OK;
  if (launch_amax_update(x, n_tokens, num_kv_heads, head_dim, amax, grid_ctas(), static_cast<cudaStream_t>(stream)) !=
      cudaSuccess)
    return PUZZLE_ERR_CUDA;
  count_launch();
  return PUZZLE_OK;
}

puzzle_status puzzle_kv_scales_from_amax(const float* amax, int32_t num_kv_heads, int32_t pow2, float* scale_out,
                                         void* stream) {
  if (!amax || !scale_out) return PUZZLE_ERR_NULL;
  if (num_kv_heads <= 0 || num_kv_heads > calibrate_max_heads()) return PUZZLE_ERR_SHAPE;
  if (launch_scales_from_amax(amax, num_kv_heads, pow2, scale_out, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return PUZZLE_ERR_CUDA;
  count_launch();
  return PUZZLE_OK;
}

puzzle_status puzzle_attn_merge_strided(const float* part_o, const float* part_lse, int64_t o_row_stride,
                                        int64_t o_part_stride, int64_t lse_row_stride, int64_t lse_part_stride,
                                        const int32_t* num_parts, const float* sinks, void* out, float* lse_out,
                                        int32_t batch, int32_t Hq, int32_t D, int32_t S, void* stream) {
  if (!part_o || !part_lse || !out) return PUZZLE_ERR_NULL;
  if (batch <= 0 || Hq <= 0 || S <= 0 || D <= 0) return PUZZLE_ERR_SHAPE;
  if (D % 64 != 0 || D > 512) return PUZZLE_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(part_o) & 7) || (reinterpret_cast<uintptr_t>(out) & 3)) return PUZZLE_ERR_SHAPE;
  if (o_row_stride < 0 || o_part_stride < 0 || lse_row_stride < 0 || lse_part_stride < 0 || (o_row_stride & 1) ||
      (o_part_stride & 1))
    return PUZZLE_ERR_SHAPE;   // partial rows are read two floats at a time
  MergeParams M;
  std::memset(&M, 0, sizeof M);
  M.part_o = part_o;
  M.part_lse = part_lse;
  M.o_row_stride = o_row_stride;
  M.o_part_stride = o_part_stride;
  M.lse_row_stride = lse_row_stride;
  M.lse_part_stride = lse_part_stride;
  M.num_parts = num_parts;
  M.sinks = sinks;
  M.out = static_cast<__nv_bfloat16*>(out);
  M.lse_out = lse_out;
  M.batch = batch;
  M.Hq = Hq;
  M.D = D;
  M.S = S;
  const long long rows = (long long)batch * Hq;
  attn_merge_kernel<<<(unsigned)((rows + kWarps - 1) / kWarps), kWarps * 32, 0, static_cast<cudaStream_t>(stream)>>>(M);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? PUZZLE_OK : PUZZLE_ERR_CUDA;
}

puzzle_status puzzle_attn_merge(const float* part_o, const float* part_lse, const int32_t* num_parts,
                                const float* sinks, void* out, float* lse_out, int32_t batch, int32_t Hq, int32_t D,
                                int32_t S, void* stream) {
  return puzzle_attn_merge_strided(part_o, part_lse, (int64_t)S * D, D, S, 1, num_parts, sinks, out, lse_out, batch, Hq,
                                   D, S, stream);
}

puzzle_status puzzle_hbm_read_probe(const void* buf, size_t bytes, uint64_t* sink, void* stream) {
  if (!buf || !sink) return PUZZLE_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(buf) & 15) || (bytes & 15) || bytes == 0) return PUZZLE_ERR_SHAPE;
  const int ctas = grid_ctas() * 4;
  hbm_read_probe_kernel<<<ctas, 512, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(buf), bytes / 16, reinterpret_cast<unsigned long long*>(sink));
  count_launch();
  return cudaGetLastError() == cudaSuccess ? PUZZLE_OK : PUZZLE_ERR_CUDA;
}

}  // extern "C"
