// Split-KV decode attention over an FP8 (E4M3) paged KV cache, sm_100a.
//
// The paper's long-context decode is bound by KV-cache I/O (Section "Optimized
// Scenarios"); FP8 KV halves those bytes (Section "KV Quantization") and window
// layers bound them by W (Section "Window attention for long-context
// inference").  This kernel therefore streams each visible K/V byte from HBM
// exactly once and keeps everything else off the critical path:
//
//  * Every warp is an independent worker with a private ring of TMA stages
//    (64 tokens = 4 K blocks + 4 V blocks = 8 KiB per stage).  Tiled TMA loads
//    with the 64-byte swizzle land each 16-token x 64-byte block so that
//    ldmatrix reads it without bank conflicts; completion is an mbarrier.
//  * The E4M3 codes feed the tensor cores as they are (m16n8k32 e4m3 MMA), so
//    dequantisation costs no instruction per element: the per-head scales
//    factor out of both dot products.  The 8 query heads of a KV-head group
//    are the M rows; rows 0-7 hold the high and rows 8-15 the low E4M3 part of
//    an exact two-term split of the bf16 query (and of the softmax weights for
//    P.V), so no MMA row is wasted and the operands keep 8 significant bits.
//  * S^T = Q.K^T puts heads on accumulator rows, so the softmax weights a lane
//    computes are exactly the A-fragment registers of the P.V product: no
//    shuffles or shared-memory round trip between the two products.
//  * Work is cut into 64-token tiles; in the balanced schedule the tile space
//    of the whole batch is divided evenly over all workers (ragged contexts
//    and window layers included), each worker writing one float32 partial
//    (o, lse) per (sequence, KV head) run it touches.  A merge kernel combines.
#include <cuda.h>

#include "common.cuh"
#include "decode_attn.cuh"

namespace puzzle {

namespace {

constexpr int kStages = 3;
constexpr int kStageBytes = 8192;
constexpr int kPipeBytes = kWarps * kStages * kStageBytes;
constexpr float kPShift = 8.0f;  // softmax weights are scaled to (0, 2^8] before the E4M3 split

struct Segment {
  int b, kvh;
  int t, t_end;  // tiles [t, t_end) of sequence b (absolute tile index)
  int L, lo;     // visible keys [lo, L)
  int prow, pstride;  // partial row of query head 0 of the group, and the stride between heads
};

struct Cursor {
  int pos, end, step;
};

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
    s.t = lo / kTile + tin;
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
    s.t = lo / kTile + (int)(((long long)sp * nt) / S);
    s.t_end = lo / kTile + (int)(((long long)(sp + 1) * nt) / S);
    s.prow = ((b * Hkv + kvh) * kGroup) * S + sp;
    s.pstride = S;
  }
  return true;
}

// One lane per 1 KiB block copy: lanes 0-3 fetch the tile's K blocks, lanes 4-7 its V blocks.
// A block that lies wholly outside [lo, L), or whose table entry is invalid, is fetched from a
// row outside the tensor map, which the TMA unit fills with zeros.
__device__ __forceinline__ void issue_tile(const DecodeParams& P, const Segment& s, int t, uint32_t stage_addr,
                                           uint32_t bar, int lane) {
  if (lane == 0) mbar_arrive_expect_tx(bar, kStageBytes);
  __syncwarp();
  if (lane < 8) {
    const int j = t * (kTile / kBlock) + (lane & 3);
    const bool vis = (j * kBlock < s.L) && (j * kBlock + kBlock > s.lo);
    int row = P.oob_row;
    if (vis) {
      long long phys = P.block_table ? (long long)P.block_table[(size_t)s.b * P.max_blocks_per_seq + j]
                                     : (long long)s.b * P.max_blocks_per_seq + j;
      if (phys < 0 || phys >= P.num_blocks) {
        if (P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_BAD_BLOCK);
      } else {
        row = (int)((phys * P.Hkv + s.kvh) * kBlock);
      }
    }
    tma_load_2d(stage_addr + (lane >> 2) * 4096 + (lane & 3) * 1024, (lane >> 2) ? &P.tmV : &P.tmK, 0, row, bar);
  }
}

}  // namespace

__global__ void __launch_bounds__(kWarps * 32, 1) decode_attn_fp8_kernel(const __grid_constant__ DecodeParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;  // this lane's query head within the group / column quad
  const uint32_t pipe = smem_u32(smem) + warp * (kStages * kStageBytes);
  const uint32_t bars = smem_u32(smem) + kPipeBytes + warp * (kStages * 8);
  int* cum = reinterpret_cast<int*>(smem + kPipeBytes + kWarps * kStages * 8);
  int* lens = cum + P.batch + 1;

  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < kStages; ++i) mbar_init(bars + 8 * i, 1);
    fence_mbar_init();
  }
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&P.tmK);
    tma_prefetch_desc(&P.tmV);
  }
  build_schedule(cum, lens, P.seq_lens, P.batch, P.Hkv, P.window, P.max_blocks_per_seq * kBlock, P.dev_status);

  const int nW = gridDim.x * kWarps;
  const int w = blockIdx.x * kWarps + warp;
  Cursor pc;
  if (P.num_splits == 0) {
    const int T = cum[P.batch];
    const int q = (T + nW - 1) / nW;
    pc.pos = min(w * q, T);
    pc.end = min(pc.pos + q, T);
    pc.step = 0;
  } else {
    pc.pos = w;
    pc.end = P.batch * P.Hkv * P.num_splits;
    pc.step = nW;
  }
  Cursor cc = pc;

  // lane-constant shared-memory offsets
  // K rows for ldmatrix.x4: lane supplies row i = lane&7 of 16-byte chunk m = lane>>3.  The 8 rows of
  // n-tile u (u = 0, 1) of a block are tokens 4c' + 2(u ^ (c'>>1)) + e with i = 2c' + e: this order makes the
  // accumulator columns a lane owns the very tokens its P.V A-fragment bytes need, and is bank-conflict free
  // under the 64-byte swizzle.
  uint32_t koff[2];
  {
    const int i = lane & 7, m = lane >> 3, ci = i >> 1, e = i & 1;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int tok = 4 * ci + 2 * (u ^ (ci >> 1)) + e;
      koff[u] = tok * 64 + ((m ^ ((tok >> 1) & 3)) << 4);
    }
  }
  // V rows for ldmatrix.m16n16.x2.trans: lane supplies token row r = lane&15 of block (lane>>4).
  const uint32_t vrow = (lane >> 4) * 1024 + (lane & 15) * 64;
  const uint32_t vswz = ((lane & 15) >> 1) & 3;
  const uint32_t psel = (c >> 1) ? 0x1054u : 0x5410u;

  // producer: run ahead by kStages tiles
  Segment ps;
  bool p_ok = next_segment(pc, ps, P, cum, lens, w);
  while (p_ok && ps.t == ps.t_end) p_ok = next_segment(pc, ps, P, cum, lens, w);
  int inflight = 0;
#pragma unroll 1
  for (int i = 0; i < kStages; ++i) {
    if (p_ok) {
      issue_tile(P, ps, ps.t, pipe + i * kStageBytes, bars + 8 * i, lane);
      ++inflight;
      if (++ps.t == ps.t_end) {
        do p_ok = next_segment(pc, ps, P, cum, lens, w); while (p_ok && ps.t == ps.t_end);
      }
    }
  }

  int stage = 0;
  uint32_t phase = 0;
  bool failed = false;
  Segment cs;
#pragma unroll 1
  while (!failed && next_segment(cc, cs, P, cum, lens, w)) {
    if (cs.t == cs.t_end) {  // empty split: weight zero
      if (c == 0) P.part_lse[cs.prow + g * cs.pstride] = -INFINITY;
      continue;
    }
    // ---- query of this (sequence, KV head): exact two-term E4M3 split, rows 0-7 high, 8-15 low
    uint32_t qa[2][4];
    float alpha_hi, alpha_lo;
    {
      const __nv_bfloat16* qrow = P.q + ((size_t)cs.b * (P.Hkv * kGroup) + cs.kvh * kGroup + g) * kHeadDim;
      float qv[4][4];
      float amax = 0.f;
#pragma unroll
      for (int h = 0; h < 4; ++h) {  // h = 2*kstep + half: dims 16h + 4c .. +3
        const uint2 raw2 = *reinterpret_cast<const uint2*>(qrow + 16 * h + 4 * c);
        qv[h][0] = __uint_as_float(raw2.x << 16);
        qv[h][1] = __uint_as_float(raw2.x & 0xffff0000u);
        qv[h][2] = __uint_as_float(raw2.y << 16);
        qv[h][3] = __uint_as_float(raw2.y & 0xffff0000u);
#pragma unroll
        for (int k = 0; k < 4; ++k) amax = fmaxf(amax, fabsf(qv[h][k]));
      }
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
      amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
      int shift = 0;
      if (amax > 0.f) {
        shift = 7 - ((int)(__float_as_uint(amax) >> 23) - 127);  // amax * 2^shift in [128, 256)
        shift = max(-120, min(120, shift));
      }
      const float up = __uint_as_float((uint32_t)(127 + shift) << 23);
      const float down = __uint_as_float((uint32_t)(127 - shift) << 23);
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        uint32_t hi16[2], lo16[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const float x0 = qv[h][2 * k] * up, x1 = qv[h][2 * k + 1] * up;
          hi16[k] = f32x2_to_e4m3x2(x0, x1);
          const uint32_t back = e4m3x2_to_f16x2(hi16[k]);
          const float2 bf = __half22float2(*reinterpret_cast<const __half2*>(&back));
          lo16[k] = f32x2_to_e4m3x2((x0 - bf.x) * 16.f, (x1 - bf.y) * 16.f);
        }
        qa[h >> 1][(h & 1) * 2 + 0] = hi16[0] | (hi16[1] << 16);
        qa[h >> 1][(h & 1) * 2 + 1] = lo16[0] | (lo16[1] << 16);
      }
      const float ks = P.k_scale ? P.k_scale[cs.kvh] : 1.f;
      alpha_hi = P.sm_scale_log2e * ks * down;
      alpha_lo = alpha_hi * 0.0625f;
    }

    float m_run = -INFINITY, l_run = 0.f;
    float O[8][2];
#pragma unroll
    for (int nd = 0; nd < 8; ++nd) O[nd][0] = O[nd][1] = 0.f;

#pragma unroll 1
    for (int t = cs.t; t < cs.t_end; ++t) {
      if (!mbar_wait_bounded(bars + 8 * stage, phase)) {
        if (P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_WAIT_EXPIRED);
        failed = true;
        break;
      }
      --inflight;
      const uint32_t kbase = pipe + stage * kStageBytes;
      const uint32_t vbase = kbase + 4096;
      const int tok0 = t * kTile;
      const bool edge = (tok0 < cs.lo) || (tok0 + kTile > cs.L);

      // ---- S^T[head][token] = Q K^T  (raw code products; scales applied below)
      float tv[8][2];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        float sc[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t r0, r1, r2, r3;
        ldsm_x4(kbase + (nt >> 1) * 1024 + koff[nt & 1], r0, r1, r2, r3);
        mma_e4m3(sc, qa[0], r0, r1);
        mma_e4m3(sc, qa[1], r2, r3);
        tv[nt][0] = sc[0] * alpha_hi + sc[2] * alpha_lo;
        tv[nt][1] = sc[1] * alpha_hi + sc[3] * alpha_lo;
      }
      if (edge) {
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const int tk = tok0 + (nt >> 1) * kBlock + 4 * c + 2 * ((nt & 1) ^ (c >> 1));
#pragma unroll
          for (int e = 0; e < 2; ++e)
            if (tk + e < cs.lo || tk + e >= cs.L) tv[nt][e] = -INFINITY;
        }
      }
      // ---- online softmax (base 2), weights scaled to (0, 2^8]
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) mx = fmaxf(mx, fmaxf(tv[nt][0], tv[nt][1]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run, mx);
      const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
      const float corr = ex2(m_run - m_use);
      m_run = m_new;
      const float off = kPShift - m_use;
      float psum = 0.f;
      uint32_t pa[2][4];
#pragma unroll
      for (int blk = 0; blk < 4; ++blk) {
        uint32_t hi16[2], lo16[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const float p0 = ex2(tv[2 * blk + u][0] + off), p1 = ex2(tv[2 * blk + u][1] + off);
          psum += p0 + p1;
          const uint32_t h2 = f32x2_to_f16x2(p0, p1);
          hi16[u] = f16x2_to_e4m3x2(h2);
          const uint32_t back = e4m3x2_to_f16x2(hi16[u]);
          const __half2 rem = __hmul2(__hsub2(*reinterpret_cast<const __half2*>(&h2),
                                              *reinterpret_cast<const __half2*>(&back)),
                                      __float2half2_rn(16.f));
          lo16[u] = f16x2_to_e4m3x2(*reinterpret_cast<const uint32_t*>(&rem));
        }
        pa[blk >> 1][(blk & 1) * 2 + 0] = prmt(hi16[0], hi16[1], psel);
        pa[blk >> 1][(blk & 1) * 2 + 1] = prmt(lo16[0], lo16[1], psel);
      }
      l_run = l_run * corr + psum;

      // ---- O_tile^T[head][dim] = P V, accumulated from zero, then folded into the running sum
      float ot[8][4];
#pragma unroll
      for (int nd = 0; nd < 8; ++nd) ot[nd][0] = ot[nd][1] = ot[nd][2] = ot[nd][3] = 0.f;
#pragma unroll
      for (int kk = 0; kk < 2; ++kk) {
        uint32_t mlo = 0xffffffffu, mhi = 0xffffffffu;
        if (edge) {  // zero the V bytes of tokens at or beyond L (they may hold anything, NaN codes included)
          const int n0 = cs.L - (tok0 + 32 * kk + 4 * c);
          const int n1 = n0 - kBlock;
          mlo = n0 >= 4 ? 0xffffffffu : (n0 <= 0 ? 0u : (1u << (8 * n0)) - 1u);
          mhi = n1 >= 4 ? 0xffffffffu : (n1 <= 0 ? 0u : (1u << (8 * n1)) - 1u);
        }
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t r0, r1, r2, r3;
          ldsm_x2_trans_b8(vbase + kk * 2048 + vrow + ((ch ^ vswz) << 4), r0, r1, r2, r3);
          if (edge) { r0 &= mlo; r1 &= mlo; r2 &= mhi; r3 &= mhi; }
          mma_e4m3(ot[2 * ch], pa[kk], r0, r2);
          mma_e4m3(ot[2 * ch + 1], pa[kk], r1, r3);
        }
      }
#pragma unroll
      for (int nd = 0; nd < 8; ++nd) {
        O[nd][0] = O[nd][0] * corr + (ot[nd][0] + ot[nd][2] * 0.0625f);
        O[nd][1] = O[nd][1] * corr + (ot[nd][1] + ot[nd][3] * 0.0625f);
      }

      // ---- refill this stage with the tile kStages ahead
      __syncwarp();
      if (p_ok) {
        issue_tile(P, ps, ps.t, kbase, bars + 8 * stage, lane);
        ++inflight;
        if (++ps.t == ps.t_end) {
          do p_ok = next_segment(pc, ps, P, cum, lens, w); while (p_ok && ps.t == ps.t_end);
        }
      }
      if (++stage == kStages) { stage = 0; phase ^= 1u; }
    }
    if (failed) break;

    // ---- partial (o, lse) of this run of tiles
    float l_tot = l_run;
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 1);
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
    const float vs = P.v_scale ? P.v_scale[cs.kvh] : 1.f;
    const float inv = l_tot > 0.f ? vs / l_tot : 0.f;
    const float lse = l_tot > 0.f ? (m_run - kPShift + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
    const size_t row = (size_t)cs.prow + (size_t)g * cs.pstride;
    float* po = P.part_o + row * kHeadDim + 2 * c;
#pragma unroll
    for (int nd = 0; nd < 8; ++nd) *reinterpret_cast<float2*>(po + 8 * nd) = make_float2(O[nd][0] * inv, O[nd][1] * inv);
    if (c == 0) P.part_lse[row] = lse;
  }

  if (failed) {
    // give the copies still in flight a bounded chance to land before the CTA's shared memory is released
    for (int i = 0; i < inflight; ++i) {
      mbar_wait_bounded(bars + 8 * stage, phase);
      if (++stage == kStages) { stage = 0; phase ^= 1u; }
    }
  }
}

size_t decode_attn_fp8_smem_bytes(int batch) {
  return 1024 + kPipeBytes + kWarps * kStages * 8 + (size_t)(2 * batch + 2) * sizeof(int);
}

}  // namespace puzzle
