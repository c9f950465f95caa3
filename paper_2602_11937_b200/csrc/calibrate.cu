// Max calibration of the per-head KV scales (paper Section "KV Quantization": scales from max calibration,
// rounded up to a power of two): amax_h = max |x| over every token and channel of KV head h,
// scale_h = amax_h / 448 as an IEEE float32 quotient.
//
// amax_update streams a bf16 tensor [n_tokens][Hkv][D] once (HBM-bound: 2 bytes per element, 16-byte loads) and
// raises a float32 [Hkv] array of running maxima; non-negative floats order like their bit patterns, so the
// maxima are kept with integer atomicMax.  NaNs are skipped, infinities count.  scales_from_amax turns the
// maxima into scales.
#include "common.cuh"

namespace puzzle {

namespace {

constexpr int kCalThreads = 256;
constexpr int kMaxHeads = 64;

// Largest |value| (as float32 bits) among the eight bf16 of a 16-byte chunk, NaNs left out.
__device__ __forceinline__ uint32_t chunk_amax_bits(const uint4 v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  uint32_t m = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t lo = (w[i] << 16) & 0x7fff0000u, hi = w[i] & 0x7fff0000u;   // |x| as float32 bits
    if (lo <= 0x7f800000u) m = max(m, lo);
    if (hi <= 0x7f800000u) m = max(m, hi);
  }
  return m;
}

__global__ void __launch_bounds__(kCalThreads) amax_update_kernel(const uint4* __restrict__ x, long long n_chunks,
                                                                  int chunks_per_head_row, int Hkv,
                                                                  uint32_t* __restrict__ amax_bits) {
  __shared__ uint32_t s_amax[kMaxHeads];
  if (threadIdx.x < kMaxHeads) s_amax[threadIdx.x] = 0;
  __syncthreads();
  // A thread keeps the maximum of the head it is looking at in a register and hands it to shared memory when
  // the head changes; with a stride that is a multiple of one token's chunks the head never changes.
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long start = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  int head = -1;
  uint32_t m = 0;
  long long i = start;
  if (stride % ((long long)chunks_per_head_row * Hkv) == 0 && start < n_chunks) {
    // the common case: one head per thread for the whole pass, four independent loads per round
    head = (int)((start / chunks_per_head_row) % Hkv);
    for (; i + 3 * stride < n_chunks; i += 4 * stride) {
      const uint4 a = __ldcs(x + i), b = __ldcs(x + i + stride), c = __ldcs(x + i + 2 * stride),
                  d = __ldcs(x + i + 3 * stride);
      m = max(max(m, chunk_amax_bits(a)), max(chunk_amax_bits(b), max(chunk_amax_bits(c), chunk_amax_bits(d))));
    }
  }
  for (; i < n_chunks; i += stride) {
    const int h = (int)((i / chunks_per_head_row) % Hkv);
    if (h != head) {
      if (head >= 0 && m) atomicMax(&s_amax[head], m);
      head = h;
      m = 0;
    }
    m = max(m, chunk_amax_bits(__ldcs(x + i)));
  }
  if (head >= 0 && m) atomicMax(&s_amax[head], m);
  __syncthreads();
  if (threadIdx.x < Hkv && s_amax[threadIdx.x]) atomicMax(&amax_bits[threadIdx.x], s_amax[threadIdx.x]);
}

__global__ void scales_from_amax_kernel(const float* __restrict__ amax, int Hkv, int pow2, float* __restrict__ scale) {
  const int h = blockIdx.x * blockDim.x + threadIdx.x;
  if (h >= Hkv) return;
  const float a = amax[h];
  float s = 1.f;               // an all-zero head keeps scale 1
  if (a != 0.f) {
    s = __fdiv_rn(a, 448.f);
    if (pow2) {
      // smallest power of two >= s; the bit pattern of a positive float is monotonic, subnormals included
      const uint32_t u = __float_as_uint(s), e = u >> 23, man = u & 0x7fffffu;
      if (e == 0) {
        if (man & (man - 1)) s = __uint_as_float(1u << (32 - __clz(man)));
      } else if (e != 0xffu && man) {
        s = __uint_as_float((e + 1) << 23);
      }
    }
  }
  scale[h] = s;
}

}  // namespace

cudaError_t launch_amax_update(const void* x, long long n_tokens, int Hkv, int D, float* amax, int sm_count,
                               cudaStream_t s) {
  const int chunks_per_head_row = D / 8;
  const long long n_chunks = n_tokens * Hkv * chunks_per_head_row;
  if (n_chunks == 0) return cudaSuccess;
  long long blocks = (n_chunks + kCalThreads - 1) / kCalThreads;
  const long long cap = (long long)sm_count * 8;
  if (blocks > cap) blocks = cap;
  // keep the stride a multiple of one token's chunks when the grid allows it
  const long long token_chunks = (long long)Hkv * chunks_per_head_row;
  if (blocks > 1 && (blocks * kCalThreads) % token_chunks != 0) {
    long long b = blocks;
    while (b > 1 && (b * kCalThreads) % token_chunks != 0) --b;
    if ((b * kCalThreads) % token_chunks == 0) blocks = b;
  }
  amax_update_kernel<<<(int)blocks, kCalThreads, 0, s>>>(static_cast<const uint4*>(x), n_chunks, chunks_per_head_row,
                                                        Hkv, reinterpret_cast<uint32_t*>(amax));
  return cudaGetLastError();
}

cudaError_t launch_scales_from_amax(const float* amax, int Hkv, int pow2, float* scale, cudaStream_t s) {
  scales_from_amax_kernel<<<1, kMaxHeads, 0, s>>>(amax, Hkv, pow2, scale);
  return cudaGetLastError();
}

int calibrate_max_heads() { return kMaxHeads; }

}  // namespace puzzle
