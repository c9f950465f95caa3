// The per-tile arithmetic of the split-KV kernels that use mma.sync: one warp, one tile of TT tokens of one KV
// head already in shared memory (K blocks followed by V blocks, each as the 128-byte-swizzled TMA box), the eight
// query heads of the group on the MMA rows.  Shared by the kernels in decode_attn.cu and decode_attn_cta.cu, which
// differ only in how tiles are handed to warps and how partial results leave them.  Include inside a
// translation unit only (internal linkage).
//
//  * The tensor cores see f16 (FP8 cache) or bf16 (bf16 cache) operands.  E4M3 to f16 is exact and one
//    pack-convert instruction per two elements; the per-head scales factor out of both dot products (Section "KV
//    Quantization": one scale per head), so dequantisation costs nothing else.  The query is scaled by a power of
//    two into f16 (exact).
//  * S^T = Q.K^T puts the 8 query heads of a KV-head group on accumulator rows, so the softmax weights a lane
//    computes are exactly the A-fragment registers of the P.V product: no shuffle or shared-memory round trip
//    between the two products.  Rows 0-7 of P carry the high and rows 8-15 the low half of an exact two-term
//    split of each float32 weight, so P.V keeps more than 16 significant bits at no extra MMA.
//  * The running maximum is only raised (and the accumulators rescaled) when a tile exceeds it by more than 2^8;
//    between such events a tile costs no accumulator traffic at all.
#pragma once

#include "common.cuh"
#include "decode_attn.cuh"

namespace puzzle {
namespace {

constexpr float kLazyLog2 = 8.0f;  // weights stay below 2^8 relative to the reference maximum

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

// Lane-constant shared-memory offsets of the ldmatrix reads of one stage.
//
// FP8.  A block lands as 8 rows of 128 bytes (two tokens per row) under the 128-byte swizzle: the 16-byte chunk q
// of token t sits at row t/2, chunk ((t&1)*4 + q) ^ (t/2 & 7).  K rows for ldmatrix.x4: a lane supplies row
// i = lane&7 of chunk m = lane>>3.  The 8 rows of n-tile u (u = 0, 1) of a block are tokens 4c' + 2(u ^ (c'>>1)) + e
// with i = 2c' + e: bank-conflict free under that swizzle, and the accumulator columns a lane owns (2c, 2c+1 of
// n-tiles 0 and 1) are the k-columns 2c.., 2c+8.. of its P.V A-fragment.  V rows for ldmatrix.m16n16.x2.trans.b8:
// lane supplies matrix row (lane&15) of block (lane>>4); rows 8..15 hold tokens (row ^ 2), so that the low half of
// each returned register is always the lane's k-columns 2c, 2c+1 and the high half its k-columns 2c+8, 2c+9.
// bf16.  Natural order: n-tile u of a block is tokens 8u..8u+7; the 128-byte swizzle is conflict free.
//
// Inside the tile loop an address is stage base + one of these; the block offset goes into the instruction as an
// immediate.
template <bool FP8>
struct LaneOffsets {
  uint32_t kof[2][2], vof[4];
  __device__ __forceinline__ void init(int lane) {
    constexpr int BLOCK_BYTES = kBlock * kHeadDim * (FP8 ? 1 : 2);
    if constexpr (FP8) {
      const int i = lane & 7, m = lane >> 3, ci = i >> 1, e = i & 1;
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int tok = 4 * ci + 2 * (u ^ (ci >> 1)) + e;
        kof[u][0] = (tok >> 1) * 128 + (((((tok & 1) << 2) | m) ^ ((tok >> 1) & 7)) << 4);
        kof[u][1] = 0;
      }
      const int vr = lane & 15, vt = vr < 8 ? vr : (vr ^ 2);
      const uint32_t vrow = (lane >> 4) * BLOCK_BYTES + (vt >> 1) * 128;
      const uint32_t vswz = (vt >> 1) & 7, vhalf = (vt & 1) << 2;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) vof[ch] = vrow + (((vhalf | ch) ^ vswz) << 4);
    } else {
      // K: matrices m = lane>>3 are chunks (4h + m) of tokens 8u + (lane&7); the chunk is XOR-ed with the row
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int h = 0; h < 2; ++h)
          kof[u][h] = (8 * u + (lane & 7)) * 128 + (((4 * h + (lane >> 3)) ^ (lane & 7)) << 4);
      // V (ldmatrix.x4.trans): matrices 0,1 = tokens 0-7, 8-15 of dim chunk 2j; 2,3 = the same of chunk 2j+1
      const uint32_t vrow = (((lane >> 3) & 1) * 8 + (lane & 7)) * 128, vswz = lane & 7;
#pragma unroll
      for (int j = 0; j < 4; ++j) vof[j] = vrow + (((2 * j + (lane >> 4)) ^ vswz) << 4);
    }
  }
};

// Running state of one warp over the tiles of one (sequence, KV head): the query as A-fragments (rows 0-7 =
// heads, rows 8-15 unused), the logit scale, the reference maximum (base-2 units), the lane's share of the row
// sum and the accumulator O[dim n-tile][row g: cols 2c, 2c+1 | row g+8: cols 2c, 2c+1]; rows g+8 carry the
// low P term, so the value of (head g, dim 8nd+2c+e) is O[nd][e] + O[nd][2+e].
struct TileState {
  uint32_t qa[4][2];
  float alpha;
  float m_ref, l_run;
  float O[8][4];

  __device__ __forceinline__ void reset() {
    m_ref = -INFINITY;
    l_run = 0.f;
#pragma unroll
    for (int nd = 0; nd < 8; ++nd) O[nd][0] = O[nd][1] = O[nd][2] = O[nd][3] = 0.f;
  }

  // Loads query row `qrow` (head g of the group; 64 bf16) for lane column c.  ks = K dequantisation scale.
  template <bool FP8>
  __device__ __forceinline__ void load_query(const __nv_bfloat16* qrow, float ks, float sm_scale_log2e, int c) {
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
      alpha = sm_scale_log2e * ks * down;
    } else {
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        qa[s][0] = *reinterpret_cast<const uint32_t*>(qrow + 16 * s + 2 * c);
        qa[s][1] = *reinterpret_cast<const uint32_t*>(qrow + 16 * s + 8 + 2 * c);
      }
      alpha = sm_scale_log2e;
    }
    alpha = fmaxf(alpha, 1e-30f);  // keeps (-inf) * alpha = -inf for masked keys
  }

  // One tile: kbase / vbase are the shared-memory addresses of its K and V blocks, tok0 its first token;
  // EDGE tiles mask the keys outside [lo, L), interior tiles carry none of that.
  template <int TT, bool FP8, bool EDGE>
  __device__ __forceinline__ void tile(const LaneOffsets<FP8>& lo_, uint32_t kbase, uint32_t vbase, int tok0, int lo,
                                       int L, int c) {
    constexpr int NB = TT / kBlock;
    constexpr int NT = TT / 8;
    constexpr int BLOCK_BYTES = kBlock * kHeadDim * (FP8 ? 1 : 2);
    const uint32_t kb[2][2] = {{kbase + lo_.kof[0][0], kbase + lo_.kof[0][1]},
                               {kbase + lo_.kof[1][0], kbase + lo_.kof[1][1]}};
    const uint32_t vb[4] = {vbase + lo_.vof[0], vbase + lo_.vof[1], vbase + lo_.vof[2], vbase + lo_.vof[3]};

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
          if (tk + e < lo || tk + e >= L) sr[nt][e] = -INFINITY;
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
          const int n0 = L - (tok0 + 32 * blk2 + 4 * c);
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
          mma_f16(O[2 * ch + 1], pa[2 * blk2 + 1][0], pa[2 * blk2 + 1][1], pa[2 * blk2 + 1][2], pa[2 * blk2 + 1][3],
                  b0, b1);
        }
      } else {
#pragma unroll
        for (int bb = 0; bb < 2; ++bb) {
          const int blk = 2 * blk2 + bb;
          uint32_t mlo = 0xffffffffu, mhi = 0xffffffffu;
          if constexpr (EDGE) {  // zero the V values of tokens at or beyond L
            const int n0 = L - (tok0 + kBlock * blk + 2 * c);
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
  }
};

}  // namespace
}  // namespace puzzle
