// Fused quantise-and-append of one new token per sequence into the paged KV cache.
// FP8: code = E4M3(RNE, saturating at +-448) of the IEEE float32 quotient x / scale[h]
// (FP8 KV with calibrated scales, paper Section "KV Quantization"); bf16 cache: a copy.
// One thread converts two adjacent channels of K or of V.
#include "common.cuh"
#include "decode_attn.cuh"

namespace puzzle {

__device__ __forceinline__ uint32_t encode_e4m3_pair(float y0, float y1) {
  uint32_t codes = f32x2_to_e4m3x2(y0, y1);
  // every NaN becomes the one canonical NaN code, whatever sign the division left on it
  if (y0 != y0) codes = (codes & 0xff00u) | 0x7fu;
  if (y1 != y1) codes = (codes & 0x00ffu) | 0x7f00u;
  return codes;
}

__global__ void __launch_bounds__(256) kv_append_kernel(void* k_cache, void* v_cache, const __nv_bfloat16* k_new,
                                                        const __nv_bfloat16* v_new, const int32_t* block_table,
                                                        const int32_t* seq_lens, const float* k_scale,
                                                        const float* v_scale, long long num_blocks, int batch,
                                                        int Hkv, int max_blocks_per_seq, int kv_dtype,
                                                        int32_t* dev_status) {
  const int pairs_per_tensor = batch * Hkv * (kHeadDim / 2);
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= 2 * pairs_per_tensor) return;
  const bool is_v = idx >= pairs_per_tensor;
  const int i = is_v ? idx - pairs_per_tensor : idx;
  const int d = (i % (kHeadDim / 2)) * 2;
  const int h = (i / (kHeadDim / 2)) % Hkv;
  const int b = i / ((kHeadDim / 2) * Hkv);

  const int len = seq_lens[b];
  if (len <= 0) return;
  if (len > max_blocks_per_seq * kBlock) {
    if (dev_status && d == 0 && h == 0 && !is_v) atomicOr(dev_status, (int)PUZZLE_DEV_SEQ_TOO_LONG);
    return;
  }
  const int pos = len - 1;
  const long long blk = block_table ? (long long)block_table[(size_t)b * max_blocks_per_seq + pos / kBlock]
                                    : (long long)b * max_blocks_per_seq + pos / kBlock;
  if (blk < 0 || blk >= num_blocks) {
    if (dev_status && d == 0 && h == 0 && !is_v) atomicOr(dev_status, (int)PUZZLE_DEV_BAD_BLOCK);
    return;
  }
  const size_t dst = ((size_t)(blk * Hkv + h) * kBlock + pos % kBlock) * kHeadDim + d;
  const __nv_bfloat16* src = (is_v ? v_new : k_new) + ((size_t)b * Hkv + h) * kHeadDim + d;
  const uint32_t two = *reinterpret_cast<const uint32_t*>(src);
  void* cache = is_v ? v_cache : k_cache;
  if (kv_dtype == PUZZLE_KV_BF16) {
    reinterpret_cast<uint32_t*>(cache)[dst / 2] = two;
  } else {
    const float* sp = is_v ? v_scale : k_scale;
    const float s = sp ? sp[h] : 1.f;
    const float y0 = __fdiv_rn(__uint_as_float(two << 16), s);
    const float y1 = __fdiv_rn(__uint_as_float(two & 0xffff0000u), s);
    reinterpret_cast<uint16_t*>(cache)[dst / 2] = (uint16_t)encode_e4m3_pair(y0, y1);
  }
}

// Read-only streaming probe: XOR-reduces the buffer so the loads cannot be dropped.
__global__ void __launch_bounds__(512) hbm_read_probe_kernel(const uint4* buf, size_t n16, unsigned long long* sink) {
  uint4 acc = make_uint4(0, 0, 0, 0);
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 3 * stride < n16; i += 4 * stride) {
    const uint4 a = __ldcs(buf + i), b = __ldcs(buf + i + stride), c = __ldcs(buf + i + 2 * stride),
                d = __ldcs(buf + i + 3 * stride);
    acc.x ^= a.x ^ b.x ^ c.x ^ d.x; acc.y ^= a.y ^ b.y ^ c.y ^ d.y;
    acc.z ^= a.z ^ b.z ^ c.z ^ d.z; acc.w ^= a.w ^ b.w ^ c.w ^ d.w;
  }
  for (; i < n16; i += stride) {
    const uint4 a = __ldcs(buf + i);
    acc.x ^= a.x; acc.y ^= a.y; acc.z ^= a.z; acc.w ^= a.w;
  }
  unsigned long long v = ((unsigned long long)(acc.x ^ acc.z) << 32) | (acc.y ^ acc.w);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v ^= __shfl_xor_sync(0xffffffffu, v, d);
  if ((threadIdx.x & 31) == 0 && v != 0x9e3779b97f4a7c15ull) atomicXor(sink, v);
}

}  // namespace puzzle
