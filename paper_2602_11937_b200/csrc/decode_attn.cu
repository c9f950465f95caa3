// Split-KV decode attention over a paged KV cache (FP8 E4M3 codes, or bf16), sm_100a.
//
// The paper's long-context decode is bound by KV-cache I/O (Section "Optimized
// Scenarios"); FP8 KV halves those bytes (Section "KV Quantization") and window
// layers bound them by W (Section "Window attention for long-context
// inference").  The kernel therefore streams each visible K/V byte from HBM
// exactly once and spends as few issue slots per byte as it can:
//
//  * Every warp is an independent worker with a private ring of TMA stages
//    (one stage = one tile of K blocks + V blocks).  Tiled TMA loads land each
//    16-token block swizzled so that ldmatrix reads it without bank conflicts;
//    completion is an mbarrier; the block-table entries of the next refill are
//    fetched one tile ahead so the lookup never stalls the math.
//  * The tensor cores see f16 (FP8 cache) or bf16 (bf16 cache) operands.  E4M3
//    to f16 is exact and one pack-convert instruction per two elements; the
//    per-head scales factor out of both dot products, so dequantisation costs
//    nothing else.  The query is scaled by a power of two into f16 (exact).
//  * S^T = Q.K^T puts the 8 query heads of a KV-head group on accumulator rows,
//    so the softmax weights a lane computes are exactly the A-fragment
//    registers of the P.V product: no shuffle or shared-memory round trip
//    between the two products.  Rows 0-7 of P carry the high and rows 8-15 the
//    low half of an exact two-term split of each float32 weight, so P.V keeps
//    more than 16 significant bits at no extra MMA.
//  * The running maximum is only raised (and the accumulators rescaled) when a
//    tile exceeds it by more than 2^8; between such events a tile costs no
//    accumulator traffic at all.
//  * Work is cut into tiles; in the balanced schedule the tile space of the
//    whole batch is divided evenly over all workers (ragged contexts and window
//    layers included), each worker writing one float32 partial (o, lse) per
//    (sequence, KV head) run it touches.  The worker whose partial completes a
//    (sequence, KV head) merges all of them (log-sum-exp, sink folded in once)
//    and writes the bf16 output: one launch per layer, no waiting anywhere.
#include <cuda.h>

#include <type_traits>

#include <climits>

#include "common.cuh"
#include "decode_attn.cuh"
#include "decode_sched.cuh"

namespace puzzle {

#ifdef PUZZLE_TIMELINE
// Diagnostic build only (timeline.py): per warp of the FP8 kernel, nanosecond stamps of the kernel entry, the first
// tile's arrival and the end of the tile loop, and the SM it ran on; read back with puzzle_debug_timeline.
constexpr int kTimelineWarps = 4096;
__device__ unsigned long long g_timeline[kTimelineWarps][4];
__device__ __forceinline__ unsigned long long timeline_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
#define TIMELINE(x) x
#else
#define TIMELINE(x)
#endif

namespace {

constexpr float kLazyLog2 = 8.0f;  // weights stay below 2^8 relative to the reference maximum


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

// E4M3 -> f16 of the four codes in `r`: lo = codes 0,1; hi = codes 2,3.
__device__ __forceinline__ void e4m3x4_to_f16x2x2(uint32_t r, uint32_t& lo, uint32_t& hi) {
  asm("{\n\t.reg .b16 l, h;\n\t"
      "mov.b32 {l, h}, %2;\n\t"
      "cvt.rn.f16x2.e4m3x2 %0, l;\n\t"
      "cvt.rn.f16x2.e4m3x2 %1, h;\n\t}"
      : "=r"(lo), "=r"(hi)
      : "r"(r));
}
// D(16x8, f32) += A(16x16, f16, row) * B(16x8, f16, col)
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// The same with a zero C operand (first k-step of a chain): D is written, nothing has to be cleared first.
__device__ __forceinline__ void mma_f16_z(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void mma_bf16v_z(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void mma_bf16v(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}


}  // namespace

// NW warps per CTA, NS stages per warp, TT tokens per tile; FP8 selects the E4M3 cache (else bf16).
template <int NW, int NS, int TT, bool FP8>
__global__ void __launch_bounds__(NW * 32, 1) decode_attn_kernel(const __grid_constant__ DecodeParams P) {
  constexpr int NB = TT / kBlock;                       // blocks per tile
  constexpr int EB = FP8 ? 1 : 2;                       // bytes per cache element
  constexpr int BLOCK_BYTES = kBlock * kHeadDim * EB;   // one (block, KV head): 1 KiB or 2 KiB
  constexpr int STAGE_BYTES = 2 * NB * BLOCK_BYTES;
  constexpr int PIPE_BYTES = NW * NS * STAGE_BYTES;
  constexpr int NT = TT / 8;                            // 8-token n-tiles of S^T per tile

  TIMELINE(const unsigned long long tl_start = timeline_now(); unsigned long long tl_first = 0;)
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
    cc.pos = w;
    cc.end = P.batch * P.Hkv * P.num_splits;
    cc.step = nW;
  }

  // ---- lane-constant shared-memory offsets
  // FP8.  A block lands as 8 rows of 128 bytes (two tokens per row) under the 128-byte swizzle: the 16-byte
  // chunk q of token t sits at row t/2, chunk ((t&1)*4 + q) ^ (t/2 & 7).  K rows for ldmatrix.x4: a lane
  // supplies row i = lane&7 of chunk m = lane>>3.  The 8 rows of n-tile u (u = 0, 1) of a block are tokens
  // 4c' + 2(u ^ (c'>>1)) + e with i = 2c' + e: bank-conflict free under that swizzle, and the accumulator columns a lane owns (2c, 2c+1 of n-tiles 0 and 1) are the
  // k-columns 2c.., 2c+8.. of its P.V A-fragment.  V rows for ldmatrix.m16n16.x2.trans.b8: lane supplies
  // matrix row (lane&15) of block (lane>>4); rows 8..15 hold tokens (row ^ 2), so that the low half of each
  // returned register is always the lane's k-columns 2c, 2c+1 and the high half its k-columns 2c+8, 2c+9.
  // bf16.  Natural order: n-tile u of a block is tokens 8u..8u+7; the 128-byte swizzle is conflict free.
  uint32_t koff[2], vrow, vswz, vhalf = 0;
  if constexpr (FP8) {
    const int i = lane & 7, m = lane >> 3, ci = i >> 1, e = i & 1;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int tok = 4 * ci + 2 * (u ^ (ci >> 1)) + e;
      koff[u] = (tok >> 1) * 128 + (((((tok & 1) << 2) | m) ^ ((tok >> 1) & 7)) << 4);
    }
    const int vr = lane & 15, vt = vr < 8 ? vr : (vr ^ 2);
    vrow = (lane >> 4) * BLOCK_BYTES + (vt >> 1) * 128;
    vswz = (vt >> 1) & 7;
    vhalf = (vt & 1) << 2;
  } else {
    // K: matrices m = lane>>3 are chunks (4h + m) of tokens 8u + (lane&7); the chunk is XOR-ed with the row
    koff[0] = (lane & 7) * 128;            // + ((chunk ^ (lane & 7)) << 4) per use
    koff[1] = (8 + (lane & 7)) * 128;
    // V (ldmatrix.x4.trans): matrices 0,1 = tokens 0-7, 8-15 of dim chunk 2j; 2,3 = the same of chunk 2j+1
    vrow = (((lane >> 3) & 1) * 8 + (lane & 7)) * 128;
    vswz = lane & 7;                        // row & 7
  }

  // per-use lane-constant offsets, hoisted: inside the tile loop an address is stage base + one of these,
  // the block offset goes into the instruction as an immediate
  uint32_t kof[2][2], vof[4];
  if constexpr (FP8) {
    kof[0][0] = koff[0]; kof[1][0] = koff[1]; kof[0][1] = 0; kof[1][1] = 0;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) vof[ch] = vrow + (((vhalf | ch) ^ vswz) << 4);
  } else {
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
      for (int h = 0; h < 2; ++h) kof[u][h] = koff[u] + (((4 * h + (lane >> 3)) ^ (lane & 7)) << 4);
#pragma unroll
    for (int j = 0; j < 4; ++j) vof[j] = vrow + (((2 * j + (lane >> 4)) ^ vswz) << 4);
  }

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
    // ---- query of this (sequence, KV head) as A-fragments (rows 0-7 = heads, rows 8-15 unused)
    uint32_t qa[4][2];
    float alpha;
    {
      const __nv_bfloat16* qrow = P.q + ((size_t)cs.b * (P.Hkv * kGroup) + cs.kvh * kGroup + g) * kHeadDim;
      const float ks = P.k_scale && FP8 ? P.k_scale[cs.kvh] : 1.f;
      if constexpr (FP8) {
        // k-step s covers dims 16s..16s+15; its k-columns 2c, 2c+1 are dims 16s+4c, +1 and its k-columns
        // 2c+8, 2c+9 are dims 16s+4c+2, +3 (the order the K codes arrive in).  The row is scaled by a power
        // of two so that its largest magnitude lies in [1, 2): every bf16 value is then exact in f16.
        float qv[4][4];
        float amax = 0.f;
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const uint2 raw2 = *reinterpret_cast<const uint2*>(qrow + 16 * s + 4 * c);
          qv[s][0] = __uint_as_float(raw2.x << 16);
          qv[s][1] = __uint_as_float(raw2.x & 0xffff0000u);
          qv[s][2] = __uint_as_float(raw2.y << 16);
          qv[s][3] = __uint_as_float(raw2.y & 0xffff0000u);
#pragma unroll
          for (int k = 0; k < 4; ++k) amax = fmaxf(amax, fabsf(qv[s][k]));
        }
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
        int shift = 0;
        if (amax > 0.f) {
          shift = -((int)(__float_as_uint(amax) >> 23) - 127);  // amax * 2^shift in [1, 2)
          shift = max(-120, min(120, shift));
        }
        const float up = __uint_as_float((uint32_t)(127 + shift) << 23);
        const float down = __uint_as_float((uint32_t)(127 - shift) << 23);
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          qa[s][0] = f32x2_to_f16x2(qv[s][0] * up, qv[s][1] * up);
          qa[s][1] = f32x2_to_f16x2(qv[s][2] * up, qv[s][3] * up);
        }
        alpha = P.sm_scale_log2e * ks * down;
      } else {
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          qa[s][0] = *reinterpret_cast<const uint32_t*>(qrow + 16 * s + 2 * c);
          qa[s][1] = *reinterpret_cast<const uint32_t*>(qrow + 16 * s + 8 + 2 * c);
        }
        alpha = P.sm_scale_log2e;
      }
      alpha = fmaxf(alpha, 1e-30f);  // keeps (-inf) * alpha = -inf for masked keys
    }

    float m_ref = -INFINITY, l_run = 0.f;
    float O[8][4];  // [dim n-tile][row g: cols 2c, 2c+1 | row g+8: cols 2c, 2c+1]; rows g+8 carry the low P term
#pragma unroll
    for (int nd = 0; nd < 8; ++nd) O[nd][0] = O[nd][1] = O[nd][2] = O[nd][3] = 0.f;

#pragma unroll 1
    for (int t = cs.t; t < cs.t_end; ++t) {
      if (!mbar_wait_bounded(bars + 8 * stage, phase)) {
        if (P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_WAIT_EXPIRED);
        failed = true;
        break;
      }
      TIMELINE(if (tl_first == 0) tl_first = timeline_now();)
      --inflight;
      const uint32_t kbase = pipe + stage * STAGE_BYTES;
      const uint32_t vbase = kbase + NB * BLOCK_BYTES;
      const int tok0 = t * TT;
      const bool edge = (tok0 < cs.lo) || (tok0 + TT > cs.L);
      const uint32_t kb[2][2] = {{kbase + kof[0][0], kbase + kof[0][1]}, {kbase + kof[1][0], kbase + kof[1][1]}};
      const uint32_t vb[4] = {vbase + vof[0], vbase + vof[1], vbase + vof[2], vbase + vof[3]};
      // the tile's math, compiled twice: interior tiles carry none of the masking of edge tiles
      auto tile_math = [&](auto edge_tag) {
      constexpr bool EDGE = decltype(edge_tag)::value;

      // ---- S^T[head][token] = Q K^T (code products; the scales are folded into alpha)
      float sr[NT][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float sc[4];
        if constexpr (FP8) {
          uint32_t r[4];
          ldsm_x4(kb[nt & 1][0] + (nt >> 1) * BLOCK_BYTES, r[0], r[1], r[2], r[3]);
#pragma unroll
          for (int s = 0; s < 4; ++s) {
            uint32_t b0, b1;
            e4m3x4_to_f16x2x2(r[s], b0, b1);
            if (s == 0) mma_f16_z(sc, qa[s][0], 0u, qa[s][1], 0u, b0, b1);
            else mma_f16(sc, qa[s][0], 0u, qa[s][1], 0u, b0, b1);
          }
        } else {
#pragma unroll
          for (int h = 0; h < 2; ++h) {  // dims 32h .. 32h+31: chunks 4h .. 4h+3
            uint32_t r[4];
            ldsm_x4(kb[nt & 1][h] + (nt >> 1) * BLOCK_BYTES, r[0], r[1], r[2], r[3]);
            if (h == 0) mma_bf16v_z(sc, qa[2 * h][0], 0u, qa[2 * h][1], 0u, r[0], r[1]);
            else mma_bf16v(sc, qa[2 * h][0], 0u, qa[2 * h][1], 0u, r[0], r[1]);
            mma_bf16v(sc, qa[2 * h + 1][0], 0u, qa[2 * h + 1][1], 0u, r[2], r[3]);
          }
        }
        sr[nt][0] = sc[0];
        sr[nt][1] = sc[1];
      }
      if constexpr (EDGE) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int tk = tok0 + (nt >> 1) * kBlock + (FP8 ? 4 * c + 2 * ((nt & 1) ^ (c >> 1)) : 8 * (nt & 1) + 2 * c);
#pragma unroll
          for (int e = 0; e < 2; ++e)
            if (tk + e < cs.lo || tk + e >= cs.L) sr[nt][e] = -INFINITY;
        }
      }
      // ---- online softmax in base 2 against a lazily raised reference maximum
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) mx = fmaxf(mx, fmaxf(sr[nt][0], sr[nt][1]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx *= alpha;
      if (mx > m_ref + kLazyLog2 || m_ref == -INFINITY) {
        if (mx != -INFINITY) {
          const float corr = ex2(m_ref - mx);  // 0 on the first visible tile
          l_run *= corr;
#pragma unroll
          for (int nd = 0; nd < 8; ++nd) {
            O[nd][0] *= corr; O[nd][1] *= corr; O[nd][2] *= corr; O[nd][3] *= corr;
          }
          m_ref = mx;
        }
      }
      const float negm = (m_ref == -INFINITY) ? 0.f : -m_ref;
      uint32_t pa[NB][4];
#pragma unroll
      for (int blk = 0; blk < NB; ++blk) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const float p0 = ex2(fmaf(sr[2 * blk + u][0], alpha, negm));
          const float p1 = ex2(fmaf(sr[2 * blk + u][1], alpha, negm));
          l_run += p0 + p1;
          // exact split p = hi + lo: hi keeps the leading bits the 16-bit type holds, lo is the remainder
          if constexpr (FP8) {
            const float h0 = __uint_as_float(__float_as_uint(p0) & 0xffffe000u);
            const float h1 = __uint_as_float(__float_as_uint(p1) & 0xffffe000u);
            pa[blk][2 * u + 0] = f32x2_to_f16x2(h0, h1);
            pa[blk][2 * u + 1] = f32x2_to_f16x2(p0 - h0, p1 - h1);
          } else {
            const float h0 = __uint_as_float(__float_as_uint(p0) & 0xffff0000u);
            const float h1 = __uint_as_float(__float_as_uint(p1) & 0xffff0000u);
            pa[blk][2 * u + 0] = prmt(__float_as_uint(p0), __float_as_uint(p1), 0x7632u);
            pa[blk][2 * u + 1] = f32x2_to_bf16x2(p0 - h0, p1 - h1);
          }
        }
      }

      // ---- O[head][dim] += P V  (k = the 16 tokens of one block per MMA)
#pragma unroll
      for (int blk2 = 0; blk2 < NB / 2; ++blk2) {
        if constexpr (FP8) {
          uint32_t mlo = 0xffffffffu, mhi = 0xffffffffu;
          if constexpr (EDGE) {  // zero the V codes of tokens at or beyond L (they may hold anything, NaN codes included)
            const int n0 = cs.L - (tok0 + 32 * blk2 + 4 * c);
            const int n1 = n0 - kBlock;
            mlo = n0 >= 4 ? 0xffffffffu : (n0 <= 0 ? 0u : (1u << (8 * n0)) - 1u);
            mhi = n1 >= 4 ? 0xffffffffu : (n1 <= 0 ? 0u : (1u << (8 * n1)) - 1u);
            if (c >> 1) {  // this lane's registers hold its tokens in the order +2, +3, +0, +1
              mlo = prmt(mlo, 0u, 0x1032u);
              mhi = prmt(mhi, 0u, 0x1032u);
            }
          }
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t r0, r1, r2, r3;
            ldsm_x2_trans_b8(vb[ch] + blk2 * 2 * BLOCK_BYTES, r0, r1, r2, r3);
            if constexpr (EDGE) { r0 &= mlo; r1 &= mlo; r2 &= mhi; r3 &= mhi; }
            uint32_t b0, b1;
            e4m3x4_to_f16x2x2(r0, b0, b1);
            mma_f16(O[2 * ch], pa[2 * blk2][0], pa[2 * blk2][1], pa[2 * blk2][2], pa[2 * blk2][3], b0, b1);
            e4m3x4_to_f16x2x2(r1, b0, b1);
            mma_f16(O[2 * ch + 1], pa[2 * blk2][0], pa[2 * blk2][1], pa[2 * blk2][2], pa[2 * blk2][3], b0, b1);
            e4m3x4_to_f16x2x2(r2, b0, b1);
            mma_f16(O[2 * ch], pa[2 * blk2 + 1][0], pa[2 * blk2 + 1][1], pa[2 * blk2 + 1][2], pa[2 * blk2 + 1][3], b0,
                    b1);
            e4m3x4_to_f16x2x2(r3, b0, b1);
            mma_f16(O[2 * ch + 1], pa[2 * blk2 + 1][0], pa[2 * blk2 + 1][1], pa[2 * blk2 + 1][2],
                    pa[2 * blk2 + 1][3], b0, b1);
          }
        } else {
#pragma unroll
          for (int bb = 0; bb < 2; ++bb) {
            const int blk = 2 * blk2 + bb;
            uint32_t mlo = 0xffffffffu, mhi = 0xffffffffu;
            if constexpr (EDGE) {  // zero the V values of tokens at or beyond L
              const int n0 = cs.L - (tok0 + kBlock * blk + 2 * c);
              const int n1 = n0 - 8;
              mlo = n0 >= 2 ? 0xffffffffu : (n0 <= 0 ? 0u : 0xffffu);
              mhi = n1 >= 2 ? 0xffffffffu : (n1 <= 0 ? 0u : 0xffffu);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {  // dim chunks 2j, 2j+1 -> n-tiles 2j, 2j+1
              uint32_t r0, r1, r2, r3;
              ldsm_x4_trans(vb[j] + blk * BLOCK_BYTES, r0, r1, r2, r3);
              if constexpr (EDGE) { r0 &= mlo; r1 &= mhi; r2 &= mlo; r3 &= mhi; }
              mma_bf16v(O[2 * j], pa[blk][0], pa[blk][1], pa[blk][2], pa[blk][3], r0, r1);
              mma_bf16v(O[2 * j + 1], pa[blk][0], pa[blk][1], pa[blk][2], pa[blk][3], r2, r3);
            }
          }
        }
      }

      };  // tile_math
      if (edge) tile_math(std::true_type{}); else tile_math(std::false_type{});

      // ---- refill this stage with the tile NS ahead
      __syncwarp();
      if (prod.template issue<BLOCK_BYTES>(P, cum, lens, w, lane, kbase, bars + 8 * stage)) ++inflight;
      if (++stage == NS) { stage = 0; phase ^= 1u; }
    }
    if (failed) break;

    // ---- partial (o, lse) of this run of tiles
    float l_tot = l_run;
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 1);
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
    const float vs = P.v_scale && FP8 ? P.v_scale[cs.kvh] : 1.f;
    const float inv = l_tot > 0.f ? vs / l_tot : 0.f;
    const float lse = l_tot > 0.f ? (m_ref + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
    const size_t row = (size_t)cs.prow + (size_t)g * cs.pstride;
    float* po = P.part_o + row * kHeadDim + 2 * c;
#pragma unroll
    for (int nd = 0; nd < 8; ++nd)
      *reinterpret_cast<float2*>(po + 8 * nd) = make_float2((O[nd][0] + O[nd][2]) * inv, (O[nd][1] + O[nd][3]) * inv);
    if (c == 0) P.part_lse[row] = lse;
    arrive_and_merge(P, cs.b, cs.kvh, cum, nW, lane);
  }

  TIMELINE(if (FP8 && lane == 0 && w < kTimelineWarps) {
    unsigned smid;
    asm volatile("mov.u32 %0, %smid;" : "=r"(smid));
    g_timeline[w][0] = tl_start; g_timeline[w][1] = tl_first; g_timeline[w][2] = timeline_now(); g_timeline[w][3] = smid;
  })
  // sequences without any visible key have no tile and hence no worker in the balanced schedule
  if (!failed && P.num_splits == 0) {
    for (int p = w; p < P.batch * P.Hkv; p += nW) {
      const int b = p / P.Hkv;
      if (cum[b + 1] == cum[b]) merge_rows(P, b, p - b * P.Hkv, 0, 0, 0, 0, lane);
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
  kern<<<ctas, NW * 32, need, s>>>(P);
  return cudaGetLastError();
}

cudaError_t launch_decode_attn(const DecodeParams& P, bool fp8, int ctas, cudaStream_t s, int* smem_limit) {
  return fp8 ? launch_variant<kDecodeWarpsFp8, kDecodeStagesFp8, kTileFp8, true>(P, ctas, s, smem_limit[0])
             : launch_variant<kDecodeWarpsBf16, kDecodeStagesBf16, kTileBf16, false>(P, ctas, s, smem_limit[1]);
}

}  // namespace puzzle

#ifdef PUZZLE_TIMELINE
// Copies the stamps of the last FP8 launch to the host: unsigned long long [4096][4] (diagnostic build only).
extern "C" __attribute__((visibility("default"))) int puzzle_debug_timeline(unsigned long long* host_out) {
  return (int)cudaMemcpyFromSymbol(host_out, puzzle::g_timeline, sizeof(puzzle::g_timeline));
}
#endif
