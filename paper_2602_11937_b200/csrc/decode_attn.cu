// Split-KV decode attention over a paged KV cache (FP8 E4M3 codes, or bf16), sm_100a: the warp-scheduled kernel.
//
// The paper's long-context decode is bound by KV-cache I/O (Section "Optimized
// Scenarios"); FP8 KV halves those bytes (Section "KV Quantization") and window
// layers bound them by W (Section "Window attention for long-context
// inference").  The kernel therefore streams each visible K/V byte from HBM
// exactly once and spends as few issue slots per byte as it can (decode_tile.cuh
// holds the arithmetic of a tile).
//
//  * Every warp is an independent worker with a private ring of TMA stages
//    (one stage = one tile of K blocks + V blocks).  Tiled TMA loads land each
//    16-token block swizzled so that ldmatrix reads it without bank conflicts;
//    completion is an mbarrier; the block-table entries of the next refill are
//    fetched one tile ahead so the lookup never stalls the math.
//  * Work is cut into tiles.  With explicit splits a warp takes whole (sequence, KV head, split) units; in the
//    balanced schedule the tile space of the whole batch is divided evenly over all warps (ragged contexts and
//    window layers included).  Each worker writes one float32 partial (o, lse) per (sequence, KV head) run it
//    touches; the worker whose partial completes a (sequence, KV head) merges all of them (log-sum-exp, sink
//    folded in once) and writes the bf16 output: one launch per layer, no waiting anywhere.
//
// The balanced schedule of decode_attn_cta.cu (work handed out per CTA and combined in shared memory) is the
// default for batches it has room for; this kernel serves explicit split counts and larger batches.
#include <cuda.h>

#include <type_traits>

#include <climits>

#include "common.cuh"
#include "decode_attn.cuh"
#include "decode_sched.cuh"
#include "decode_tile.cuh"

namespace puzzle {

namespace {

// Producer side of one warp.  Lane i < NB owns block i of a tile (NB blocks of 16 tokens per tile; the K copy and
// the V copy of a block share the row coordinate).  `phys` holds, per owning lane, the physical
// block of the NEXT tile to issue (kNotVisible: the block lies wholly outside [lo, L) and is fetched
// from a row outside the tensor map, which the TMA unit fills with zeros).  The table entry is loaded one
// tile ahead of its use.
template <int TT>
struct Producer {
  static constexpr int NB = TT / kBlock;
  static constexpr int kNotVisible = INT_MIN;
  Cursor cur;
  Segment seg;
  bool ok;
  int phys;

  __device__ __forceinline__ void skip_empty(const DecodeParams& P, const int* cum, const int* lens, int w) {
    while (ok && seg.t == seg.t_end) ok = next_segment<TT>(cur, seg, P, cum, lens, w);
  }
  __device__ __forceinline__ void lookup(const DecodeParams& P, int lane) {
    phys = kNotVisible;
    if (ok && lane < NB) {
      const int j = seg.t * NB + lane;
      if ((j * kBlock < seg.L) && (j * kBlock + kBlock > seg.lo))
        phys = P.block_table ? P.block_table[(size_t)seg.b * P.max_blocks_per_seq + j]
                             : seg.b * P.max_blocks_per_seq + j;
    }
  }
  __device__ __forceinline__ void start(Cursor c, const DecodeParams& P, const int* cum, const int* lens, int w,
                                        int lane) {
    cur = c;
    ok = next_segment<TT>(cur, seg, P, cum, lens, w);
    skip_empty(P, cum, lens, w);
    lookup(P, lane);
  }
  // Issues the pending tile into `stage_addr` and looks the next one up.  Returns false if nothing was pending.
  template <int BLOCK_BYTES>
  __device__ __forceinline__ bool issue(const DecodeParams& P, const int* cum, const int* lens, int w, int lane,
                                        uint32_t stage_addr, uint32_t bar) {
    if (!ok) return false;
    int row = P.oob_row;
    if (lane < NB) {
      if (phys >= 0 && phys < P.num_blocks) {
        row = (phys * P.Hkv + seg.kvh) * P.rows_per_block;
      } else if (phys != kNotVisible) {
        if (P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_BAD_BLOCK);
      }
    }
    // the copies are issued by one lane, which collects the row coordinates first: a TMA instruction takes
    // warp-uniform operands, so issuing from several lanes would be serialised lane by lane anyway
    int rows[NB];
#pragma unroll
    for (int i = 0; i < NB; ++i) rows[i] = __shfl_sync(0xffffffffu, row, i);
    if (elect_one()) {
      mbar_arrive_expect_tx(bar, 2 * NB * BLOCK_BYTES);
#pragma unroll
      for (int i = 0; i < NB; ++i) tma_load_2d(stage_addr + i * BLOCK_BYTES, &P.tmK, 0, rows[i], bar);
#pragma unroll
      for (int i = 0; i < NB; ++i) tma_load_2d(stage_addr + (NB + i) * BLOCK_BYTES, &P.tmV, 0, rows[i], bar);
    }
    if (++seg.t == seg.t_end) {
      ok = next_segment<TT>(cur, seg, P, cum, lens, w);
      skip_empty(P, cum, lens, w);
    }
    lookup(P, lane);
    return true;
  }
};

}  // namespace

// NW warps per CTA, NS stages per warp, TT tokens per tile; FP8 selects the E4M3 cache (else bf16).
template <int NW, int NS, int TT, bool FP8>
__global__ void __launch_bounds__(NW * 32, 1) decode_attn_kernel(const __grid_constant__ DecodeParams P) {
  constexpr int NB = TT / kBlock;                       // blocks per tile
  constexpr int EB = FP8 ? 1 : 2;                       // bytes per cache element
  constexpr int BLOCK_BYTES = kBlock * kHeadDim * EB;   // one (block, KV head): 1 KiB or 2 KiB
  constexpr int STAGE_BYTES = 2 * NB * BLOCK_BYTES;
  constexpr int PIPE_BYTES = NW * NS * STAGE_BYTES;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;  // this lane's query head within the group / column quad
  const uint32_t pipe = smem_u32(smem) + warp * (NS * STAGE_BYTES);
  const uint32_t bars = smem_u32(smem) + PIPE_BYTES + warp * (NS * 8);
  int* cum = reinterpret_cast<int*>(smem + PIPE_BYTES + NW * NS * 8);
  int* lens = cum + P.batch + 1;

  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NS; ++i) mbar_init(bars + 8 * i, 1);
    fence_mbar_init();
  }
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&P.tmK);
    tma_prefetch_desc(&P.tmV);
  }
  release_dependents();
  grid_dependency_wait();   // nothing above reads or writes global memory
  build_schedule(cum, lens, P.seq_lens, P.batch, P.Hkv, P.window, P.max_blocks_per_seq * kBlock, TT, P.dev_status);

  const int nW = gridDim.x * NW;
  const int w = blockIdx.x * NW + warp;
  Cursor cc;
  if (P.num_splits == 0) {
    const int T = cum[P.batch];
    const int q = (T + nW - 1) / nW;
    cc.pos = min(w * q, T);
    cc.end = min(cc.pos + q, T);
    cc.step = 0;
  } else {
    // Every worker takes one contiguous share of the units (sequence, KV head, split), shares in the order
    // warp 0 of every CTA, warp 1 of every CTA, ...: a launch with fewer units than workers still uses every SM, and
    // a worker meets only one or two (sequence, KV head) pairs.  (Handing units out round-robin made every worker
    // meet many pairs; a worker that had merged one fell behind, arrived last at each of its later pairs and so
    // had to merge those as well: with 128 splits one warp ended up with most merges of the launch.)
    const long long units = (long long)P.batch * P.Hkv * P.num_splits;
    const int wi = warp * gridDim.x + blockIdx.x;
    cc.pos = (int)(wi * units / nW);
    cc.end = (int)((wi + 1) * units / nW);
    cc.step = 1;
  }

  LaneOffsets<FP8> lo;
  lo.init(lane);

  Producer<TT> prod;
  prod.start(cc, P, cum, lens, w, lane);
  int inflight = 0;
#pragma unroll 1
  for (int i = 0; i < NS; ++i)
    if (prod.template issue<BLOCK_BYTES>(P, cum, lens, w, lane, pipe + i * STAGE_BYTES, bars + 8 * i)) ++inflight;

  int stage = 0;
  uint32_t phase = 0;
  bool failed = false;
  Segment cs;
#pragma unroll 1
  while (!failed && next_segment<TT>(cc, cs, P, cum, lens, w)) {
    if (cs.t == cs.t_end) {  // empty split: weight zero
      if (c == 0) P.part_lse[cs.prow + g * cs.pstride] = -INFINITY;
      arrive_and_merge(P, cs.b, cs.kvh, cum, nW, lane);
      continue;
    }
    TileState st;
    st.template load_query<FP8>(P.q + ((size_t)cs.b * (P.Hkv * kGroup) + cs.kvh * kGroup + g) * kHeadDim,
                                P.k_scale && FP8 ? P.k_scale[cs.kvh] : 1.f, P.sm_scale_log2e, c);
    st.reset();
    // one split per pair: this warp's result is final, so the sink is fetched while the tiles are in flight
    const float sink_g = (P.num_splits == 1 && P.sinks) ? P.sinks[cs.kvh * kGroup + g] : -INFINITY;

#pragma unroll 1
    for (int t = cs.t; t < cs.t_end; ++t) {
      if (!mbar_wait_bounded(bars + 8 * stage, phase)) {
        if (P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_WAIT_EXPIRED);
        failed = true;
        break;
      }
      --inflight;
      const uint32_t kbase = pipe + stage * STAGE_BYTES;
      const uint32_t vbase = kbase + NB * BLOCK_BYTES;
      const int tok0 = t * TT;
      if ((tok0 < cs.lo) || (tok0 + TT > cs.L))
        st.template tile<TT, FP8, true>(lo, kbase, vbase, tok0, cs.lo, cs.L, c);
      else
        st.template tile<TT, FP8, false>(lo, kbase, vbase, tok0, cs.lo, cs.L, c);

      // ---- refill this stage with the tile NS ahead
      __syncwarp();
      if (prod.template issue<BLOCK_BYTES>(P, cum, lens, w, lane, kbase, bars + 8 * stage)) ++inflight;
      if (++stage == NS) { stage = 0; phase ^= 1u; }
    }
    if (failed) break;

    // ---- partial (o, lse) of this run of tiles
    float l_tot = st.l_run;
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 1);
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
    const float vs = P.v_scale && FP8 ? P.v_scale[cs.kvh] : 1.f;
    if (P.num_splits == 1) {
      // the whole (sequence, KV head) was this warp's: fold the sink in and store the output, no partial, no arrival
      const long long row_out = (long long)cs.b * (P.Hkv * kGroup) + cs.kvh * kGroup + g;
      const float s2 = sink_g * 1.4426950408889634f;
      const float M = fmaxf(l_tot > 0.f ? st.m_ref : -INFINITY, s2);
      float f = 0.f, Z = 0.f;
      if (M != -INFINITY) {
        const float wa = l_tot > 0.f ? ex2(st.m_ref - M) : 0.f;
        Z = l_tot * wa + (s2 == -INFINITY ? 0.f : ex2(s2 - M));
        f = wa * vs / Z;
      }
      if (P.out_f32) {
        float* dst = P.out_f32 + row_out * kHeadDim + 2 * c;
#pragma unroll
        for (int nd = 0; nd < 8; ++nd)
          *reinterpret_cast<float2*>(dst + 8 * nd) =
              make_float2((st.O[nd][0] + st.O[nd][2]) * f, (st.O[nd][1] + st.O[nd][3]) * f);
      } else {
        __nv_bfloat16* dst = P.out + row_out * kHeadDim + 2 * c;
#pragma unroll
        for (int nd = 0; nd < 8; ++nd)
          *reinterpret_cast<uint32_t*>(dst + 8 * nd) =
              f32x2_to_bf16x2((st.O[nd][0] + st.O[nd][2]) * f, (st.O[nd][1] + st.O[nd][3]) * f);
      }
      if (P.lse_out && c == 0) P.lse_out[row_out] = Z > 0.f ? (M + log2f(Z)) * 0.6931471805599453f : -INFINITY;
      continue;
    }
    const float inv = l_tot > 0.f ? vs / l_tot : 0.f;
    const float lse = l_tot > 0.f ? (st.m_ref + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
    const size_t row = (size_t)cs.prow + (size_t)g * cs.pstride;
    float* po = P.part_o + row * kHeadDim + 2 * c;
#pragma unroll
    for (int nd = 0; nd < 8; ++nd)
      *reinterpret_cast<float2*>(po + 8 * nd) = make_float2((st.O[nd][0] + st.O[nd][2]) * inv, (st.O[nd][1] + st.O[nd][3]) * inv);
    if (c == 0) P.part_lse[row] = lse;
    arrive_and_merge(P, cs.b, cs.kvh, cum, nW, lane);
  }

  // sequences without any visible key have no tile and hence no worker in the balanced schedule
  if (!failed && P.num_splits == 0) {
    for (int p = w; p < P.batch * P.Hkv; p += nW) {
      const int b = p / P.Hkv;
      if (cum[b + 1] == cum[b]) merge_rows(P, b, p - b * P.Hkv, 0, 0, 0, 0, 0, 0, 0, lane);
    }
  }

  if (failed) {
    // give the copies still in flight a bounded chance to land before the CTA's shared memory is released
    for (int i = 0; i < inflight; ++i) {
      mbar_wait_bounded(bars + 8 * stage, phase);
      if (++stage == NS) { stage = 0; phase ^= 1u; }
    }
  }
}

template <int NW, int NS, int TT, bool FP8>
static size_t smem_bytes_of(int batch) {
  constexpr int STAGE_BYTES = 2 * (TT / kBlock) * kBlock * kHeadDim * (FP8 ? 1 : 2);
  return 1024 + (size_t)NW * NS * STAGE_BYTES + NW * NS * 8 + (size_t)(2 * batch + 2) * sizeof(int);
}

template <int NW, int NS, int TT, bool FP8>
static cudaError_t launch_variant(const DecodeParams& P, int ctas, cudaStream_t s, int& smem_limit) {
  auto kern = decode_attn_kernel<NW, NS, TT, FP8>;
  if (smem_limit == 0) {  // first launch of this variant on this device: raise its dynamic shared-memory limit
    int dev = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
    if (e != cudaSuccess) return e;
    smem_limit = optin;
  }
  const size_t need = smem_bytes_of<NW, NS, TT, FP8>(P.batch);
  if (need > (size_t)smem_limit) return cudaErrorInvalidValue;  // batch too large for the schedule arrays
  return launch_dependent(kern, dim3(ctas), dim3(NW * 32), need, s, P);
}

cudaError_t launch_decode_attn(const DecodeParams& P, bool fp8, int ctas, cudaStream_t s, int* smem_limit) {
  return fp8 ? launch_variant<kDecodeWarpsFp8, kDecodeStagesFp8, kTileFp8, true>(P, ctas, s, smem_limit[0])
             : launch_variant<kDecodeWarpsBf16, kDecodeStagesBf16, kTileBf16, false>(P, ctas, s, smem_limit[1]);
}

}  // namespace puzzle

