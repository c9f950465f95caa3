// Log-sum-exp merge of attention partials that came from outside the split-KV kernel (which merges its own
// partials itself), with the per-head sink logit folded in once.
//   M = max(sink, max_p lse_p);  Z = e^(sink-M) + sum_p e^(lse_p-M);  out = sum_p e^(lse_p-M) o_p / Z.
// One warp per (sequence, query head) row; a lane owns two adjacent channels of each 64-wide slab.
#include "common.cuh"
#include "decode_attn.cuh"

namespace puzzle {

__global__ void __launch_bounds__(kWarps * 32) attn_merge_kernel(const MergeParams P) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kWarps + warp;
  if (row >= (long long)P.batch * P.Hq) return;
  const int b = (int)(row / P.Hq), head = (int)(row % P.Hq);
  const float* lse_row = P.part_lse + row * P.lse_row_stride;
  const float* o_row = P.part_o + row * P.o_row_stride;
  const int count = P.num_parts ? min(max(P.num_parts[b], 0), P.S) : P.S;

  const float sink = P.sinks ? P.sinks[head] : -INFINITY;
  float M = sink;
  for (int k = lane; k < count; k += 32) M = fmaxf(M, lse_row[k * P.lse_part_stride]);
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
    const float l = lse_row[k * P.lse_part_stride];
    if (l != -INFINITY) Z += __expf(l - M);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) Z += __shfl_xor_sync(0xffffffffu, Z, d);
  if (sink != -INFINITY) Z += __expf(sink - M);  // the sink is one more softmax column, counted once
  const float invZ = 1.f / Z;

  for (int d = 2 * lane; d < P.D; d += 64) {
    float ax = 0.f, ay = 0.f;
    for (int k = 0; k < count; ++k) {
      const float l = lse_row[k * P.lse_part_stride];
      if (l == -INFINITY) continue;
      const float wgt = __expf(l - M);
      const float2 o = *reinterpret_cast<const float2*>(o_row + k * P.o_part_stride + d);
      ax += wgt * o.x;
      ay += wgt * o.y;
    }
    *reinterpret_cast<__nv_bfloat162*>(orow + d) = __floats2bfloat162_rn(ax * invZ, ay * invZ);
  }
  if (P.lse_out && lane == 0) P.lse_out[row] = M + __logf(Z);
}

}  // namespace puzzle
