// Log-sum-exp merge of split-KV partials, with the per-head sink logit folded in once.
//   M = max(sink, max_p lse_p);  Z = e^(sink-M) + sum_p e^(lse_p-M);  out = sum_p e^(lse_p-M) o_p / Z.
// One warp per (sequence, query head) row; a lane owns two adjacent channels of each 64-wide slab.
#include "common.cuh"
#include "decode_attn.cuh"

namespace puzzle {

__global__ void __launch_bounds__(kWarps * 32) attn_merge_kernel(const MergeParams P) {
  extern __shared__ int sched[];  // balanced layout only: cum[batch+1], lens[batch]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (P.balanced) build_schedule(sched, sched + P.batch + 1, P.seq_lens, P.batch, P.Hkv, P.window, P.max_tokens, P.tile, nullptr);

  const long long row = (long long)blockIdx.x * kWarps + warp;
  if (row >= (long long)P.batch * P.Hq) return;
  const int b = (int)(row / P.Hq), head = (int)(row % P.Hq);

  // where this row's parts live: index(k) = first + k*stride, k < count
  long long first;
  int count, stride;
  if (P.balanced) {
    const int* cum = sched;
    const int kvh = head / kGroup, g = head % kGroup;
    const int nt = (cum[b + 1] - cum[b]) / P.Hkv;
    const int T = cum[P.batch];
    const int q = (T + P.num_workers - 1) / P.num_workers;
    if (nt == 0) {
      first = 0; count = 0;
    } else {
      const int g0 = cum[b] + kvh * nt;
      const int w0 = g0 / q, w1 = (g0 + nt - 1) / q;
      first = ((long long)w0 + b * P.Hkv + kvh) * kGroup + g;
      count = w1 - w0 + 1;
    }
    stride = kGroup;
  } else {
    first = row * P.S;
    count = P.num_parts ? min(max(P.num_parts[b], 0), P.S) : P.S;
    stride = 1;
  }

  const float sink = P.sinks ? P.sinks[head] : -INFINITY;
  float M = sink;
  for (int k = lane; k < count; k += 32) M = fmaxf(M, P.part_lse[first + (long long)k * stride]);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, d));

  __nv_bfloat16* orow = P.out + row * P.D;
  if (M == -INFINITY) {  // nothing visible and no sink
    for (int d = 2 * lane; d < P.D; d += 64) *reinterpret_cast<__nv_bfloat162*>(orow + d) = __floats2bfloat162_rn(0.f, 0.f);
    if (P.lse_out && lane == 0) P.lse_out[row] = -INFINITY;
    return;
  }
  float Z = 0.f;
  for (int k = lane; k < count; k += 32) {
    const float l = P.part_lse[first + (long long)k * stride];
    if (l != -INFINITY) Z += __expf(l - M);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, d);
  if (sink != -INFINITY) Z += __expf(sink - M);  // the sink is one more softmax column, counted once
  const float invZ = 1.f / Z;

  for (int d = 2 * lane; d < P.D; d += 64) {
    float ax = 0.f, ay = 0.f;
    for (int k = 0; k < count; ++k) {
      const long long idx = first + (long long)k * stride;
      const float l = P.part_lse[idx];
      if (l == -INFINITY) continue;
      const float wgt = __expf(l - M);
      const float2 o = *reinterpret_cast<const float2*>(P.part_o + idx * P.D + d);
      ax += wgt * o.x;
      ay += wgt * o.y;
    }
    *reinterpret_cast<__nv_bfloat162*>(orow + d) = __floats2bfloat162_rn(ax * invZ, ay * invZ);
  }
  if (P.lse_out && lane == 0) P.lse_out[row] = M + __logf(Z);
}

size_t attn_merge_smem_bytes(int batch, int balanced) { return balanced ? (size_t)(2 * batch + 2) * sizeof(int) : 0; }

}  // namespace puzzle
