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
  // No early release here: the decode kernel behind the append should find every SM free when its CTAs are placed, so
  // that CTA i lands on the same SM launch after launch (the CTA speeds it notes are speeds of SMs).
  grid_dependency_wait();
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

// Bulk form: n_new tokens per sequence (a prompt chunk, or several tokens of a multi-token step).  Token i of
// sequence b goes to position seq_lens[b] - new_lens[b] + i (seq_lens counted after the append).  One thread
// converts eight adjacent channels: a 16-byte load, an 8-byte (FP8) or 16-byte (bf16) store.
__global__ void __launch_bounds__(256) kv_append_tokens_kernel(void* k_cache, void* v_cache, const uint4* k_new,
                                                               const uint4* v_new, const int32_t* new_lens,
                                                               const int32_t* block_table, const int32_t* seq_lens,
                                                               const float* k_scale, const float* v_scale,
                                                               long long num_blocks, int batch, int n_new, int Hkv,
                                                               int max_blocks_per_seq, int kv_dtype,
                                                               int32_t* dev_status) {
  grid_dependency_wait();              // no early release, for the reason given in kv_append_kernel
  constexpr int kOct = kHeadDim / 8;   // 16-byte pieces per (token, head) row
  // grid: x over the (token, head, piece) of one sequence, y = sequence, z = K or V
  const int per_seq = n_new * Hkv * kOct;
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= per_seq) return;
  const int b = blockIdx.y;
  const bool is_v = blockIdx.z != 0;
  // piece fastest, then token, then head: a warp reads four 128-byte head rows and writes 256 contiguous bytes
  // of one cache block (FP8), so both sides move whole lines
  const int o = r % kOct;
  const int tok = (r / kOct) % n_new;
  const int h = r / (kOct * n_new);
  const long long i = (((long long)b * n_new + tok) * Hkv + h) * kOct + o;   // 16-byte piece of k_new / v_new

  const int len = seq_lens[b];
  const int nl = new_lens ? min(max(new_lens[b], 0), n_new) : n_new;
  const bool reporter = o == 0 && h == 0 && tok == 0 && !is_v;
  if (len > max_blocks_per_seq * kBlock) {
    if (dev_status && reporter) atomicOr(dev_status, (int)PUZZLE_DEV_SEQ_TOO_LONG);
    return;
  }
  const int pos = len - nl + tok;
  if (tok >= nl || pos < 0) return;   // a sequence shorter than its chunk keeps the chunk's last `len` tokens
  const long long blk = block_table ? (long long)block_table[(size_t)b * max_blocks_per_seq + pos / kBlock]
                                    : (long long)b * max_blocks_per_seq + pos / kBlock;
  if (blk < 0 || blk >= num_blocks) {
    if (dev_status && o == 0 && h == 0 && !is_v) atomicOr(dev_status, (int)PUZZLE_DEV_BAD_BLOCK);
    return;
  }
  const size_t dst = ((size_t)(blk * Hkv + h) * kBlock + pos % kBlock) * kHeadDim + 8 * o;   // in elements
  const uint4 x = __ldcs((is_v ? v_new : k_new) + i);
  void* cache = is_v ? v_cache : k_cache;
  if (kv_dtype == PUZZLE_KV_BF16) {
    reinterpret_cast<uint4*>(cache)[dst / 8] = x;
  } else {
    const float* sp = is_v ? v_scale : k_scale;
    const float s = sp ? sp[h] : 1.f;
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
    uint32_t c[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      c[k] = encode_e4m3_pair(__fdiv_rn(__uint_as_float(w[k] << 16), s), __fdiv_rn(__uint_as_float(w[k] & 0xffff0000u), s));
    reinterpret_cast<uint2*>(cache)[dst / 8] = make_uint2((c[0] & 0xffffu) | (c[1] << 16), (c[2] & 0xffffu) | (c[3] << 16));
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
