// Decode attention for launches that are a chain of latencies, not a stream of bytes: window layers with a narrow
// window and very short contexts, where no (sequence, KV head) pair has more than four tiles (Section "Window
// attention for long-context inference": most layers of the searched architectures are of this kind).
//
// Such a launch has a few hundred pairs of two or three tiles each.  Its duration is the longest dependent chain in
// it, so this kernel keeps the chain short:
//  * no schedule is built: pair p belongs to a group of four warps, group p / gridDim.x (mod 3) of CTA p mod gridDim.x,
//    which reads the pair's length itself;
//  * warp i of the group takes tile i of the pair, so the tiles of a pair are computed side by side (one warp alone
//    needs about 1.5 us per tile: it has the SM's issue slots to itself but every instruction waits for the one
//    before it);
//  * the four running states meet in shared memory behind one named barrier of the group; its first warp combines
//    them, folds the sink in and stores the bf16 rows.  Nothing goes through the workspace.
// The arithmetic per tile is decode_tile.cuh's, the one of the two larger kernels.
#include <cuda.h>

#include <climits>

#include "common.cuh"
#include "decode_attn.cuh"
#include "decode_tile.cuh"

namespace puzzle {

namespace {

constexpr int kSmallWarps = 12;                         // warps per CTA
constexpr int kSmallGroup = kWholePairTiles;            // warps per group = tiles a pair can have
constexpr int kSmallGroups = kSmallWarps / kSmallGroup; // groups per CTA
static_assert(kSmallGroups * kSmallGroup == kSmallWarps, "whole groups");

__device__ __forceinline__ void group_barrier(int group) {
  asm volatile("bar.sync %0, %1;" ::"r"(1 + group), "r"(kSmallGroup * 32) : "memory");
}

}  // namespace

template <int TT, bool FP8>
__global__ void __launch_bounds__(kSmallWarps * 32, 1) decode_attn_small_kernel(const __grid_constant__ DecodeParams P) {
  constexpr int NW = kSmallWarps, GW = kSmallGroup;
  constexpr int NB = TT / kBlock;                       // blocks per tile
  constexpr int EB = FP8 ? 1 : 2;                       // bytes per cache element
  constexpr int BLOCK_BYTES = kBlock * kHeadDim * EB;   // one (block, KV head): 1 KiB or 2 KiB
  constexpr int STAGE_BYTES = 2 * NB * BLOCK_BYTES;     // K and V of one tile
  constexpr int kNotVisible = INT_MIN;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;  // this lane's query head within the group of heads / column quad
  const int group = warp / GW, wi = warp % GW;
  const uint32_t stage = smem_u32(smem) + warp * STAGE_BYTES;
  uint8_t* sp = smem + NW * STAGE_BYTES;
  const uint32_t bar = smem_u32(sp) + warp * 8;                       sp += NW * 8;
  sp += (16 - (NW * 8) % 16) % 16;
  float4* dep_o = reinterpret_cast<float4*>(sp);                      sp += NW * 4 * 32 * sizeof(float4);  // [warp][j][lane]
  float* dep_m = reinterpret_cast<float*>(sp);                        sp += NW * kGroup * sizeof(float);
  float* dep_l = reinterpret_cast<float*>(sp);

  if (lane == 0) {
    mbar_init(bar, 1);
    fence_mbar_init();
  }
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&P.tmK);
    tma_prefetch_desc(&P.tmV);
  }
  release_dependents();
  grid_dependency_wait();   // nothing above reads or writes global memory
  __syncwarp();

  LaneOffsets<FP8> lo;
  lo.init(lane);
  uint32_t phase = 0;
  const int pairs = P.batch * P.Hkv;

#pragma unroll 1
  for (int p = group * gridDim.x + blockIdx.x; p < pairs; p += kSmallGroups * gridDim.x) {  // the same p in a group
    const int b = p / P.Hkv, kvh = p - b * P.Hkv;
    bool too_long;
    const SeqRange r = seq_range(P.seq_lens[b], P.window, P.max_blocks_per_seq * kBlock, TT, too_long);
    if (too_long && P.dev_status && warp % GW == 0 && lane == 0) atomicOr(P.dev_status, (int)PUZZLE_DEV_SEQ_TOO_LONG);
    const int nt = min(r.ntile, GW);       // the host chose this kernel because no pair can have more tiles
    const bool have = wi < nt;

    TileState st;
    st.reset();
    float sink_g = -INFINITY, vs = 1.f;
    if (have) {
      const int t = r.tlo + wi;
      // ---- this warp's tile: table look-up by the lanes that own a block, copies issued by one lane
      int row = P.oob_row;
      if (lane < NB) {
        const int j = t * NB + lane;
        if ((j * kBlock < r.L) && (j * kBlock + kBlock > r.lo)) {
          const int phys = P.block_table ? P.block_table[(size_t)b * P.max_blocks_per_seq + j]
                                         : b * P.max_blocks_per_seq + j;
          if (phys >= 0 && phys < P.num_blocks) row = (phys * P.Hkv + kvh) * P.rows_per_block;
          else if (P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_BAD_BLOCK);
        }
      }
      int rows[NB];
#pragma unroll
      for (int i = 0; i < NB; ++i) rows[i] = __shfl_sync(0xffffffffu, row, i);
      if (elect_one()) {
        mbar_arrive_expect_tx(bar, STAGE_BYTES);
#pragma unroll
        for (int i = 0; i < NB; ++i) tma_load_2d(stage + i * BLOCK_BYTES, &P.tmK, 0, rows[i], bar);
#pragma unroll
        for (int i = 0; i < NB; ++i) tma_load_2d(stage + (NB + i) * BLOCK_BYTES, &P.tmV, 0, rows[i], bar);
      }
      // ---- query, scales and sink while the tile is in flight
      st.template load_query<FP8>(P.q + ((size_t)b * (P.Hkv * kGroup) + kvh * kGroup + g) * kHeadDim,
                                  P.k_scale && FP8 ? P.k_scale[kvh] : 1.f, P.sm_scale_log2e, c);
      st.reset();
      vs = P.v_scale && FP8 ? P.v_scale[kvh] : 1.f;
      if (wi == 0 && P.sinks) sink_g = P.sinks[kvh * kGroup + g];
      if (mbar_wait_bounded(bar, phase)) {
        const uint32_t kbase = stage, vbase = stage + NB * BLOCK_BYTES;
        const int tok0 = t * TT;
        if ((tok0 < r.lo) || (tok0 + TT > r.L))
          st.template tile<TT, FP8, true>(lo, kbase, vbase, tok0, r.lo, r.L, c);
        else
          st.template tile<TT, FP8, false>(lo, kbase, vbase, tok0, r.lo, r.L, c);
      } else {
        // the copy did not land in time: report it, contribute nothing, and keep in step with the group
        if (P.dev_status && lane == 0) atomicOr(P.dev_status, (int)PUZZLE_DEV_WAIT_EXPIRED);
        st.reset();
      }
      phase ^= 1u;
    } else if (wi == 0) {
      if (P.sinks) sink_g = P.sinks[kvh * kGroup + g];   // a pair without visible keys: the output is the sink's
    }

    float l_tot = st.l_run;
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 1);
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
    float m = st.m_ref;
    float o[8][2];
#pragma unroll
    for (int nd = 0; nd < 8; ++nd) {
      o[nd][0] = st.O[nd][0] + st.O[nd][2];
      o[nd][1] = st.O[nd][1] + st.O[nd][3];
    }

    if (nt > 1) {   // uniform in the group
      if (wi != 0 && have) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          dep_o[(warp * 4 + j) * 32 + lane] = make_float4(o[2 * j][0], o[2 * j][1], o[2 * j + 1][0], o[2 * j + 1][1]);
        if (c == 0) {
          dep_m[warp * kGroup + g] = m;
          dep_l[warp * kGroup + g] = l_tot;
        }
      }
      group_barrier(group);
      if (wi == 0) {
        float M = m;
        for (int u = warp + 1; u < warp + nt; ++u) M = fmaxf(M, dep_m[u * kGroup + g]);
        const float fo = m == -INFINITY ? 0.f : ex2(m - M);
        l_tot *= fo;
#pragma unroll
        for (int nd = 0; nd < 8; ++nd) { o[nd][0] *= fo; o[nd][1] *= fo; }
        for (int u = warp + 1; u < warp + nt; ++u) {
          const float mu = dep_m[u * kGroup + g];
          const float fu = mu == -INFINITY ? 0.f : ex2(mu - M);
          l_tot = fmaf(fu, dep_l[u * kGroup + g], l_tot);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float4 v = dep_o[(u * 4 + j) * 32 + lane];
            o[2 * j][0] = fmaf(fu, v.x, o[2 * j][0]); o[2 * j][1] = fmaf(fu, v.y, o[2 * j][1]);
            o[2 * j + 1][0] = fmaf(fu, v.z, o[2 * j + 1][0]); o[2 * j + 1][1] = fmaf(fu, v.w, o[2 * j + 1][1]);
          }
        }
        m = M;
      }
      group_barrier(group);   // the deposits have been read: the next pair of this group may overwrite them
    }

    if (wi == 0) {
      // ---- fold the sink in and store the rows of the pair's eight query heads
      const long long row_out = (long long)b * (P.Hkv * kGroup) + kvh * kGroup + g;
      const float s2 = sink_g * 1.4426950408889634f;
      const float M = fmaxf(l_tot > 0.f ? m : -INFINITY, s2);
      float f = 0.f, Z = 0.f;
      if (M != -INFINITY) {
        const float wa = l_tot > 0.f ? ex2(m - M) : 0.f;
        Z = l_tot * wa + (s2 == -INFINITY ? 0.f : ex2(s2 - M));
        f = wa * vs / Z;
      }
      if (P.out_f32) {
        float* dst = P.out_f32 + row_out * kHeadDim + 2 * c;
#pragma unroll
        for (int nd = 0; nd < 8; ++nd)
          *reinterpret_cast<float2*>(dst + 8 * nd) = make_float2(o[nd][0] * f, o[nd][1] * f);
      } else {
        __nv_bfloat16* dst = P.out + row_out * kHeadDim + 2 * c;
#pragma unroll
        for (int nd = 0; nd < 8; ++nd)
          *reinterpret_cast<uint32_t*>(dst + 8 * nd) = f32x2_to_bf16x2(o[nd][0] * f, o[nd][1] * f);
      }
      if (P.lse_out && c == 0) P.lse_out[row_out] = Z > 0.f ? (M + log2f(Z)) * 0.6931471805599453f : -INFINITY;
    }
  }
}

template <int TT, bool FP8>
static cudaError_t launch_small_variant(const DecodeParams& P, int ctas, cudaStream_t s, int& smem_limit) {
  auto kern = decode_attn_small_kernel<TT, FP8>;
  constexpr int STAGE_BYTES = 2 * (TT / kBlock) * kBlock * kHeadDim * (FP8 ? 1 : 2);
  const size_t need = 1024 + (size_t)kSmallWarps * STAGE_BYTES + kSmallWarps * 8 + 16 +
                      (size_t)kSmallWarps * 4 * 32 * sizeof(float4) + 2 * kSmallWarps * kGroup * sizeof(float);
  if (smem_limit == 0) {  // first launch of this variant on this device: raise its dynamic shared-memory limit
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    if (e != cudaSuccess) return e;
    smem_limit = (int)need;
  }
  return launch_dependent(kern, dim3(ctas), dim3(kSmallWarps * 32), need, s, P);
}

cudaError_t launch_decode_attn_small(const DecodeParams& P, bool fp8, int ctas, cudaStream_t s, int* smem_limit) {
  return fp8 ? launch_small_variant<kTileFp8, true>(P, ctas, s, smem_limit[0])
             : launch_small_variant<kTileBf16, false>(P, ctas, s, smem_limit[1]);
}

int decode_attn_small_max_pairs(int ctas) { return 2 * kSmallGroups * ctas; }

}  // namespace puzzle
