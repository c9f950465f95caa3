// Pieces the split-KV kernels share: the tile schedule of a worker (a contiguous, evenly sized share of the
// batch's tile space, or explicit splits), and the log-sum-exp merge that the last arriving worker of a
// (sequence, KV head) performs.  Include after common.cuh and decode_attn.cuh, inside a translation unit only
// (everything here has internal linkage).
#pragma once

#include "common.cuh"
#include "decode_attn.cuh"

namespace puzzle {
namespace {

struct Segment {
  int b, kvh;
  int t, t_end;       // tiles [t, t_end) of sequence b (absolute tile index)
  int L, lo;          // visible keys [lo, L)
  int prow, pstride;  // partial row of query head 0 of the group, and the stride between heads
};

struct Cursor {
  int pos, end, step;
};

template <int TT>
__device__ __forceinline__ bool next_segment(Cursor& cur, Segment& s, const DecodeParams& P, const int* cum,
                                             const int* lens, int w) {
  if (cur.pos >= cur.end) return false;
  const int Hkv = P.Hkv;
  if (P.num_splits == 0) {
    const int g = cur.pos;
    int a = 0, z = P.batch;
    while (z - a > 1) {
      int mid = (a + z) >> 1;
      if (cum[mid] <= g) a = mid; else z = mid;
    }
    const int b = a;
    const int nt = (cum[b + 1] - cum[b]) / Hkv;
    const int r = g - cum[b];
    const int kvh = r / nt, tin = r - kvh * nt;
    const int L = lens[b];
    const int lo = (P.window > 0 && L > P.window) ? L - P.window : 0;
    int seg_end = cum[b] + (kvh + 1) * nt;
    if (seg_end > cur.end) seg_end = cur.end;
    s.b = b; s.kvh = kvh; s.L = L; s.lo = lo;
    s.t = lo / TT + tin;
    s.t_end = s.t + (seg_end - g);
    s.prow = (w + b * Hkv + kvh) * kGroup;
    s.pstride = 1;
    cur.pos = seg_end;
  } else {
    const int u = cur.pos;
    cur.pos += cur.step;
    const int S = P.num_splits;
    const int p = u / S, sp = u - p * S;
    const int b = p / Hkv, kvh = p - b * Hkv;
    const int nt = (cum[b + 1] - cum[b]) / Hkv;
    const int L = lens[b];
    const int lo = (P.window > 0 && L > P.window) ? L - P.window : 0;
    s.b = b; s.kvh = kvh; s.L = L; s.lo = lo;
    s.t = lo / TT + (int)(((long long)sp * nt) / S);
    s.t_end = lo / TT + (int)(((long long)(sp + 1) * nt) / S);
    s.prow = ((b * Hkv + kvh) * kGroup) * S + sp;
    s.pstride = S;
  }
  return true;
}

// Log-sum-exp merge of the `count` partials of one (sequence, KV head) by one warp: the quad of lanes with
// g = lane/4 owns query head g of the group, lane c = lane%4 of the quad owns channels 16c..16c+15.
//   M = max(sink, max_k lse_k);  Z = e^(sink-M) + sum_k e^(lse_k-M);  out = sum_k e^(lse_k-M) o_k / Z.
// Part k < count of head g is partial row first + g*hstride + k*kstride; parts count .. count+count2-1 form a
// second run, first2 + g*hstride + (k-count)*kstride2.  The partials were written by other SMs in this launch,
// so they are read past L1.
__device__ __noinline__ void merge_rows(const DecodeParams& P, int b, int kvh, long long first, int count,
                                        int kstride, int hstride, long long first2, int count2, int kstride2,
                                        int lane) {
  const int g = lane >> 2, c = lane & 3;
  const int Hq = P.Hkv * kGroup, head = kvh * kGroup + g;
  const long long row_out = (long long)b * Hq + head;
  const float sink = P.sinks ? P.sinks[head] : -INFINITY;
  const long long base = first + (long long)g * hstride, base2 = first2 + (long long)g * hstride;
  const int total = count + count2;
  auto row_of = [&](int k) { return k < count ? base + (long long)k * kstride : base2 + (long long)(k - count) * kstride2; };
  float M = -INFINITY;
  for (int k = c; k < total; k += 16) {  // four loads in flight per lane: with many parts this pass is L2 round trips too
    float l4[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) l4[j] = k + 4 * j < total ? __ldcg(P.part_lse + row_of(k + 4 * j)) : -INFINITY;
    M = fmaxf(fmaxf(M, fmaxf(l4[0], l4[1])), fmaxf(l4[2], l4[3]));
  }
  M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 1));
  M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 2));
  M = fmaxf(M, sink);
  float acc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = 0.f;
  float Z = 0.f;
  if (M != -INFINITY) {
    // four parts per round, every load of the round issued before the first use: the merge is a chain of
    // L2 round trips, so their number, not the arithmetic, sets its duration
    for (int k0 = 0; k0 < total; k0 += 4) {
      float l[4];
      float4 v[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool on = k0 + j < total;
        const long long idx = row_of(on ? k0 + j : k0);
        l[j] = on ? __ldcg(P.part_lse + idx) : -INFINITY;
        const float4* o = reinterpret_cast<const float4*>(P.part_o + idx * kHeadDim + 16 * c);
#pragma unroll
        for (int i = 0; i < 4; ++i) v[j][i] = __ldcg(o + i);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (l[j] == -INFINITY) continue;  // an empty part: its payload is undefined
        const float wgt = __expf(l[j] - M);
        Z += wgt;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          acc[4 * i + 0] += wgt * v[j][i].x; acc[4 * i + 1] += wgt * v[j][i].y;
          acc[4 * i + 2] += wgt * v[j][i].z; acc[4 * i + 3] += wgt * v[j][i].w;
        }
      }
    }
    if (sink != -INFINITY) Z += __expf(sink - M);  // the sink is one more softmax column, counted once
  }
  const float invZ = Z > 0.f ? 1.f / Z : 0.f;  // nothing visible and no sink: zeros
  if (P.out_f32) {  // a partial for a merge across devices keeps float32
    float4* dst = reinterpret_cast<float4*>(P.out_f32 + row_out * kHeadDim + 16 * c);
#pragma unroll
    for (int i = 0; i < 4; ++i)
      dst[i] = make_float4(acc[4 * i] * invZ, acc[4 * i + 1] * invZ, acc[4 * i + 2] * invZ, acc[4 * i + 3] * invZ);
  } else {
    uint32_t packed[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) packed[i] = f32x2_to_bf16x2(acc[2 * i] * invZ, acc[2 * i + 1] * invZ);
    uint4* dst = reinterpret_cast<uint4*>(P.out + row_out * kHeadDim + 16 * c);
    dst[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    dst[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
  }
  if (P.lse_out && c == 0) P.lse_out[row_out] = Z > 0.f ? M + __logf(Z) : -INFINITY;
}

// Called by a warp after it has stored its partial of (sequence b, KV head kvh): counts the arrival, and the
// warp that completes the set merges it and leaves the counter at zero for the next launch.
__device__ __forceinline__ void arrive_and_merge(const DecodeParams& P, int b, int kvh, const int* cum, int nW,
                                                 int lane) {
  const int p = b * P.Hkv + kvh;
  long long first;
  int count, kstride, hstride;
  if (P.num_splits == 0) {
    const int nt = (cum[b + 1] - cum[b]) / P.Hkv;
    const int T = cum[P.batch];
    const int q = (T + nW - 1) / nW;
    const int g0 = cum[b] + kvh * nt;
    const int w0 = g0 / q, w1 = (g0 + nt - 1) / q;
    first = ((long long)w0 + p) * kGroup;
    count = w1 - w0 + 1;
    kstride = kGroup;
    hstride = 1;
  } else {
    first = (long long)p * kGroup * P.num_splits;
    count = P.num_splits;
    kstride = 1;
    hstride = P.num_splits;
  }
  __threadfence();  // this lane's partial stores before the arrival
  __syncwarp();
  int last = 0;
  if (lane == 0) last = atomicAdd(P.counters + p, 1) == count - 1;
  last = __shfl_sync(0xffffffffu, last, 0);
  if (!last) return;
  __threadfence();  // the arrivals before the other warps' partials are read
  merge_rows(P, b, kvh, first, count, kstride, hstride, 0, 0, 0, lane);
  if (lane == 0) P.counters[p] = 0;
}


}  // namespace
}  // namespace puzzle
