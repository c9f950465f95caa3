// Decode attention for several new tokens per sequence (a multi-token decode step, or a chunk of a prompt after
// its bulk append: the input half of the paper's fixed-length scenarios, Section "Optimized Scenarios") over the
// FP8 cache, sm_100a.
//
// The bytes of a step do not grow with the number of query tokens, only the arithmetic does, so query tokens are
// processed in pairs that share one pass over the K/V tiles: in the single-token kernels rows 8-15 of the
// S^T = Q.K^T MMA are empty; here they carry the eight heads of a second query token, so the tile's E4M3 -> f16
// converts and its S MMAs serve both tokens, and only the softmax and half of the P.V MMAs are paid per token
// (P.V with the same converted V fragments).  A pair of tokens (2j, 2j+1) of sequence b is one row of the schedule; a
// causal mask gives the earlier token one key fewer (and a window that starts one key earlier).  An odd last
// token is paired with itself.  Sequences with more than two new tokens take several rows, whose repeated reads
// of the same blocks are neighbours in the schedule and are served by L2.
//
// Everything else is the warp-scheduled kernel's design (decode_attn.cu): every warp an independent worker with
// a private ring of TMA stages, the tile space of all rows cut evenly over the workers, one float32 partial
// (o, lse) per (worker, row, KV head) and query head, merged by the worker whose arrival completes the (row, KV
// head).  Twelve warps of two stages, as there: the two tokens share one accumulator (see TileState2), which
// brings the kernel to 168 registers with a few spilled words outside the MMA stream; eight warps of three stages
// (190 registers, no spill) measured 5 % slower on two tokens and 10 % slower on four.
#include <cuda.h>

#include <climits>

#include "common.cuh"
#include "decode_attn.cuh"
#include "decode_tile.cuh"

namespace puzzle {
namespace {

constexpr int kTokWarps = 12, kTokStages = 2, kTokTile = 64;
constexpr int kPairRows = 2 * kGroup;  // partial rows per (worker, row, KV head): 8 heads of each of the two tokens

// One row of the schedule: query tokens t0 and t1 (= t0 + 1, or t0 again for an odd last token) of sequence b.
struct RowInfo {
  int b, t0, t1;
  int L, LA;     // keys [lo, L) are visible to t1, [loA, LA) to t0 (LA = L - (t1 - t0))
  int lo, loA;
  int tlo, ntile;  // tiles that cover [loA, L)
  bool present, too_long;
};
__device__ __forceinline__ RowInfo row_info(const DecodeParams& P, int r) {
  RowInfo i;
  const int npairs = (P.n_q + 1) >> 1;
  i.b = r / npairs;
  const int j = r - i.b * npairs;
  const int qlen = P.q_lens ? max(0, min(P.q_lens[i.b], P.n_q)) : P.n_q;
  i.t0 = 2 * j;
  i.present = i.t0 < qlen;
  i.t1 = min(i.t0 + 1, qlen - 1);
  const int max_tokens = P.max_blocks_per_seq * kBlock;
  const int len = P.seq_lens[i.b];
  i.too_long = len > max_tokens;
  const int Lb = len < 0 ? 0 : min(len, max_tokens);
  i.L = i.present ? max(0, Lb - qlen + i.t1 + 1) : 0;
  i.LA = max(0, i.L - (i.t1 - i.t0));
  i.lo = (P.window > 0 && i.L > P.window) ? i.L - P.window : 0;
  i.loA = (P.window > 0 && i.LA > P.window) ? i.LA - P.window : 0;
  i.tlo = i.loA / kTokTile;
  i.ntile = i.L > 0 ? (i.L + kTokTile - 1) / kTokTile - i.tlo : 0;
  return i;
}

struct TokSegment {
  int r, kvh;
  int t, t_end;  // tiles [t, t_end) of the row (absolute tile index)
  RowInfo row;
  int prow;      // first partial row of this (worker, row, KV head)
};

__device__ __forceinline__ bool next_tok_segment(int& pos, int end, TokSegment& s, const DecodeParams& P, const int* cum,
                                                 int rows, int w) {
  if (pos >= end) return false;
  int a = 0, z = rows;
  while (z - a > 1) {
    const int mid = (a + z) >> 1;
    if (cum[mid] <= pos) a = mid; else z = mid;
  }
  const int r = a;
  const int nt = (cum[r + 1] - cum[r]) / P.Hkv;
  const int rem = pos - cum[r];
  const int kvh = rem / nt, tin = rem - kvh * nt;
  int seg_end = cum[r] + (kvh + 1) * nt;
  if (seg_end > end) seg_end = end;
  s.r = r; s.kvh = kvh;
  s.row = row_info(P, r);
  s.t = s.row.tlo + tin;
  s.t_end = s.t + (seg_end - pos);
  s.prow = (w + r * P.Hkv + kvh) * kPairRows;
  pos = seg_end;
  return true;
}

// Running state of a warp over the tiles of one (row, KV head): as TileState in decode_tile.cuh, for two query
// tokens.  Token A (t0) sits on MMA rows 0-7, token B (t1) on rows 8-15 of S and of O; each has its own logit
// scale, reference maximum and row sum.  P.V runs twice per V fragment, with A = [P_A ; P_B] of the high terms and
// of the low terms of the exact two-term f16 split of P, both into the same accumulator (the single-token kernels
// put the low terms on rows 8-15 instead and add the two halves at the end).
struct TileState2 {
  uint32_t qa[4][4];
  float alpha[2], m_ref[2], l_run[2];
  float O[8][4];   // O[dim n-tile][token A: cols 2c, 2c+1 | token B: cols 2c, 2c+1] (rows g and g + 8 of the MMA)

  __device__ __forceinline__ void reset() {
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      m_ref[t] = -INFINITY;
      l_run[t] = 0.f;
    }
#pragma unroll
    for (int nd = 0; nd < 8; ++nd) O[nd][0] = O[nd][1] = O[nd][2] = O[nd][3] = 0.f;
  }

  // Query row of token `tok` (head g of the group, 64 bf16), scaled by a power of two into f16 exactly; see
  // TileState::load_query for the order of the dimensions.
  __device__ __forceinline__ void load_query(int tok, const __nv_bfloat16* qrow, float ks, float sm_scale_log2e, int c) {
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
      shift = -((int)(__float_as_uint(amax) >> 23) - 127);
      shift = max(-120, min(120, shift));
    }
    const float up = __uint_as_float((uint32_t)(127 + shift) << 23);
    const float down = __uint_as_float((uint32_t)(127 - shift) << 23);
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      qa[s][tok] = f32x2_to_f16x2(qv[s][0] * up, qv[s][1] * up);          // a0 / a1: k-columns 2c, 2c+1
      qa[s][2 + tok] = f32x2_to_f16x2(qv[s][2] * up, qv[s][3] * up);      // a2 / a3: k-columns 2c+8, 2c+9
    }
    alpha[tok] = fmaxf(sm_scale_log2e * ks * down, 1e-30f);
  }

  // One tile of 64 tokens for both query tokens.  EDGE tiles mask the keys outside [loA, LA) for token A and
  // outside [lo, L) for token B; V codes at or beyond L are cleared (keys in [LA, L) are real tokens).
  template <bool EDGE>
  __device__ __forceinline__ void tile(const LaneOffsets<true>& lo_, uint32_t kbase, uint32_t vbase, int tok0, int loA,
                                       int LA, int lo, int L, int c) {
    constexpr int TT = kTokTile, NB = TT / kBlock, NT = TT / 8, BLOCK_BYTES = kBlock * kHeadDim;
    const uint32_t kb[2] = {kbase + lo_.kof[0][0], kbase + lo_.kof[1][0]};
    const uint32_t vb[4] = {vbase + lo_.vof[0], vbase + lo_.vof[1], vbase + lo_.vof[2], vbase + lo_.vof[3]};

    // ---- S^T[head of A | head of B][token] = Q K^T
    float sr[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      uint32_t r[4];
      ldsm_x4(kb[nt & 1] + (nt >> 1) * BLOCK_BYTES, r[0], r[1], r[2], r[3]);
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        uint32_t b0, b1;
        e4m3x4_to_f16x2x2(r[s], b0, b1);
        if (s == 0) mma_f16_z(sr[nt], qa[s][0], qa[s][1], qa[s][2], qa[s][3], b0, b1);
        else mma_f16(sr[nt], qa[s][0], qa[s][1], qa[s][2], qa[s][3], b0, b1);
      }
    }
    if constexpr (EDGE) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int tk = tok0 + (nt >> 1) * kBlock + 4 * c + 2 * ((nt & 1) ^ (c >> 1));
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          if (tk + e < loA || tk + e >= LA) sr[nt][e] = -INFINITY;
          if (tk + e < lo || tk + e >= L) sr[nt][2 + e] = -INFINITY;
        }
      }
    }
    // ---- online softmax per token.  P is split exactly into a high and a low f16 term; both terms of both tokens
    // go through the same accumulator rows: A = [P_A ; P_B] (rows 0-7 | 8-15), once with the high and once with
    // the low terms, so O needs the registers of one token's two-term accumulator
    uint32_t pa_hi[NB][4], pa_lo[NB][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) mx = fmaxf(mx, fmaxf(sr[nt][2 * t], sr[nt][2 * t + 1]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx *= alpha[t];
      if (mx > m_ref[t] + kLazyLog2 || m_ref[t] == -INFINITY) {
        if (mx != -INFINITY) {
          const float corr = ex2(m_ref[t] - mx);
          l_run[t] *= corr;
#pragma unroll
          for (int nd = 0; nd < 8; ++nd) { O[nd][2 * t] *= corr; O[nd][2 * t + 1] *= corr; }
          m_ref[t] = mx;
        }
      }
      const float negm = (m_ref[t] == -INFINITY) ? 0.f : -m_ref[t];
#pragma unroll
      for (int blk = 0; blk < NB; ++blk) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const float p0 = ex2(fmaf(sr[2 * blk + u][2 * t], alpha[t], negm));
          const float p1 = ex2(fmaf(sr[2 * blk + u][2 * t + 1], alpha[t], negm));
          l_run[t] += p0 + p1;
          const float h0 = __uint_as_float(__float_as_uint(p0) & 0xffffe000u);
          const float h1 = __uint_as_float(__float_as_uint(p1) & 0xffffe000u);
          pa_hi[blk][2 * u + t] = f32x2_to_f16x2(h0, h1);
          pa_lo[blk][2 * u + t] = f32x2_to_f16x2(p0 - h0, p1 - h1);
        }
      }
    }
    // ---- O[token][head][dim] += P V: the converted V fragments serve both tokens
#pragma unroll
    for (int blk2 = 0; blk2 < NB / 2; ++blk2) {
      uint32_t mlo = 0xffffffffu, mhi = 0xffffffffu;
      if constexpr (EDGE) {
        const int n0 = L - (tok0 + 32 * blk2 + 4 * c);
        const int n1 = n0 - kBlock;
        mlo = n0 >= 4 ? 0xffffffffu : (n0 <= 0 ? 0u : (1u << (8 * n0)) - 1u);
        mhi = n1 >= 4 ? 0xffffffffu : (n1 <= 0 ? 0u : (1u << (8 * n1)) - 1u);
        if (c >> 1) {
          mlo = prmt(mlo, 0u, 0x1032u);
          mhi = prmt(mhi, 0u, 0x1032u);
        }
      }
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r0, r1, r2, r3;
        ldsm_x2_trans_b8(vb[ch] + blk2 * 2 * BLOCK_BYTES, r0, r1, r2, r3);
        if constexpr (EDGE) { r0 &= mlo; r1 &= mlo; r2 &= mhi; r3 &= mhi; }
        // two independent accumulators alternate, so that an MMA never waits for the one issued just before it
        uint32_t b0, b1, d0, d1;
        e4m3x4_to_f16x2x2(r0, b0, b1);
        e4m3x4_to_f16x2x2(r1, d0, d1);
        mma_f16(O[2 * ch], pa_hi[2 * blk2][0], pa_hi[2 * blk2][1], pa_hi[2 * blk2][2], pa_hi[2 * blk2][3], b0, b1);
        mma_f16(O[2 * ch + 1], pa_hi[2 * blk2][0], pa_hi[2 * blk2][1], pa_hi[2 * blk2][2], pa_hi[2 * blk2][3], d0, d1);
        mma_f16(O[2 * ch], pa_lo[2 * blk2][0], pa_lo[2 * blk2][1], pa_lo[2 * blk2][2], pa_lo[2 * blk2][3], b0, b1);
        mma_f16(O[2 * ch + 1], pa_lo[2 * blk2][0], pa_lo[2 * blk2][1], pa_lo[2 * blk2][2], pa_lo[2 * blk2][3], d0, d1);
        e4m3x4_to_f16x2x2(r2, b0, b1);
        e4m3x4_to_f16x2x2(r3, d0, d1);
        mma_f16(O[2 * ch], pa_hi[2 * blk2 + 1][0], pa_hi[2 * blk2 + 1][1], pa_hi[2 * blk2 + 1][2],
                pa_hi[2 * blk2 + 1][3], b0, b1);
        mma_f16(O[2 * ch + 1], pa_hi[2 * blk2 + 1][0], pa_hi[2 * blk2 + 1][1], pa_hi[2 * blk2 + 1][2],
                pa_hi[2 * blk2 + 1][3], d0, d1);
        mma_f16(O[2 * ch], pa_lo[2 * blk2 + 1][0], pa_lo[2 * blk2 + 1][1], pa_lo[2 * blk2 + 1][2],
                pa_lo[2 * blk2 + 1][3], b0, b1);
        mma_f16(O[2 * ch + 1], pa_lo[2 * blk2 + 1][0], pa_lo[2 * blk2 + 1][1], pa_lo[2 * blk2 + 1][2],
                pa_lo[2 * blk2 + 1][3], d0, d1);
      }
    }
  }
};

// Log-sum-exp merge of the `count` partials of one (row, KV head) by one warp, one token after the other: the
// quad of lanes g = lane / 4 owns query head g of the group, lane c of the quad channels 16c .. 16c + 15.  Part k
// of head g of token half h is partial row first + 8 h + g + 16 k.  The formula is merge_rows' (decode_sched.cuh).
__device__ __noinline__ void merge_tok_rows(const DecodeParams& P, const RowInfo row, int kvh, long long first, int count,
                                            int lane) {
  const int g = lane >> 2, c = lane & 3;
  const int Hq = P.Hkv * kGroup, head = kvh * kGroup + g;
  const float sink = P.sinks ? P.sinks[head] : -INFINITY;
  for (int h = 0; h < 2; ++h) {
    if (h == 1 && row.t1 == row.t0) break;  // an odd last token was paired with itself
    const long long row_out = ((long long)row.b * P.n_q + (h ? row.t1 : row.t0)) * Hq + head;
    const long long base = first + 8 * h + g;
    float M = -INFINITY;
    for (int k = c; k < count; k += 4) M = fmaxf(M, __ldcg(P.part_lse + base + (long long)k * kPairRows));
    M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 1));
    M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 2));
    M = fmaxf(M, sink);
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.f;
    float Z = 0.f;
    if (M != -INFINITY) {
      for (int k = 0; k < count; ++k) {
        const long long idx = base + (long long)k * kPairRows;
        const float l = __ldcg(P.part_lse + idx);
        if (l == -INFINITY) continue;  // an empty part: its payload is undefined
        const float4* o = reinterpret_cast<const float4*>(P.part_o + idx * kHeadDim + 16 * c);
        const float wgt = __expf(l - M);
        Z += wgt;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 v = __ldcg(o + i);
          acc[4 * i + 0] += wgt * v.x; acc[4 * i + 1] += wgt * v.y;
          acc[4 * i + 2] += wgt * v.z; acc[4 * i + 3] += wgt * v.w;
        }
      }
      if (sink != -INFINITY) Z += __expf(sink - M);  // the sink is one more softmax column, counted once
    }
    const float invZ = Z > 0.f ? 1.f / Z : 0.f;
    uint32_t packed[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) packed[i] = f32x2_to_bf16x2(acc[2 * i] * invZ, acc[2 * i + 1] * invZ);
    uint4* dst = reinterpret_cast<uint4*>(P.out + row_out * kHeadDim + 16 * c);
    dst[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    dst[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
    if (P.lse_out && c == 0) P.lse_out[row_out] = Z > 0.f ? M + __logf(Z) : -INFINITY;
  }
}

}  // namespace

__global__ void __launch_bounds__(kTokWarps * 32, 1) decode_attn_tokens_kernel(const __grid_constant__ DecodeParams P) {
  constexpr int NW = kTokWarps, NS = kTokStages, TT = kTokTile;
  constexpr int NB = TT / kBlock;
  constexpr int BLOCK_BYTES = kBlock * kHeadDim;
  constexpr int STAGE_BYTES = 2 * NB * BLOCK_BYTES;
  constexpr int PIPE_BYTES = NW * NS * STAGE_BYTES;
  constexpr int kNotVisible = INT_MIN;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const uint32_t pipe = smem_u32(smem) + warp * (NS * STAGE_BYTES);
  const uint32_t bars = smem_u32(smem) + PIPE_BYTES + warp * (NS * 8);
  int* cum = reinterpret_cast<int*>(smem + PIPE_BYTES + NW * NS * 8);
  const int rows = P.batch * ((P.n_q + 1) >> 1);

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
  // ---- schedule: tiles of every row, prefix sums
  for (int r = threadIdx.x; r < rows; r += blockDim.x) {
    const RowInfo i = row_info(P, r);
    if (i.too_long && P.dev_status && blockIdx.x == 0) atomicOr(P.dev_status, (int)PUZZLE_DEV_SEQ_TOO_LONG);
    cum[r + 1] = i.ntile * P.Hkv;
  }
  if (threadIdx.x == 0) cum[0] = 0;
  __syncthreads();
  if (threadIdx.x < 32) {
    int carry = 0;
    for (int base = 0; base < rows; base += 32) {
      const int i = base + lane;
      int v = i < rows ? cum[i + 1] : 0;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += u;
      }
      if (i < rows) cum[i + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();

  const int nW = gridDim.x * NW;
  const int w = blockIdx.x * NW + warp;
  const int T = cum[rows];
  const int share = (T + nW - 1) / nW;
  const int w_lo = min(w * share, T), w_hi = min(w_lo + share, T);

  LaneOffsets<true> lo;
  lo.init(lane);

  // ---- producer side: tiles of this worker's run, block-table entries fetched one tile ahead
  int p_pos = w_lo;
  TokSegment ps;
  bool p_ok = next_tok_segment(p_pos, w_hi, ps, P, cum, rows, w);
  int phys = kNotVisible;
  auto lookup = [&]() {
    phys = kNotVisible;
    if (p_ok && lane < NB) {
      const int j = ps.t * NB + lane;
      if ((j * kBlock < ps.row.L) && (j * kBlock + kBlock > ps.row.loA))
        phys = P.block_table ? P.block_table[(size_t)ps.row.b * P.max_blocks_per_seq + j]
                             : ps.row.b * P.max_blocks_per_seq + j;
    }
  };
  auto issue = [&](uint32_t stage_addr, uint32_t bar) -> bool {
    if (!p_ok) return false;
    int row = P.oob_row;
    if (lane < NB) {
      if (phys >= 0 && phys < P.num_blocks) {
        row = (phys * P.Hkv + ps.kvh) * P.rows_per_block;
      } else if (phys != kNotVisible) {
        if (P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_BAD_BLOCK);
      }
    }
    int rws[NB];
#pragma unroll
    for (int i = 0; i < NB; ++i) rws[i] = __shfl_sync(0xffffffffu, row, i);
    if (elect_one()) {
      mbar_arrive_expect_tx(bar, 2 * NB * BLOCK_BYTES);
#pragma unroll
      for (int i = 0; i < NB; ++i) tma_load_2d(stage_addr + i * BLOCK_BYTES, &P.tmK, 0, rws[i], bar);
#pragma unroll
      for (int i = 0; i < NB; ++i) tma_load_2d(stage_addr + (NB + i) * BLOCK_BYTES, &P.tmV, 0, rws[i], bar);
    }
    if (++ps.t == ps.t_end) p_ok = next_tok_segment(p_pos, w_hi, ps, P, cum, rows, w);
    lookup();
    return true;
  };
  lookup();
  int inflight = 0;
#pragma unroll 1
  for (int i = 0; i < NS; ++i)
    if (issue(pipe + i * STAGE_BYTES, bars + 8 * i)) ++inflight;

  int stage = 0;
  uint32_t phase = 0;
  bool failed = false;
  int c_pos = w_lo;
  TokSegment cs;
#pragma unroll 1
  while (!failed && next_tok_segment(c_pos, w_hi, cs, P, cum, rows, w)) {
    TileState2 st;
    const int Hq = P.Hkv * kGroup;
    const float ks = P.k_scale ? P.k_scale[cs.kvh] : 1.f;
    st.load_query(0, P.q + (((size_t)cs.row.b * P.n_q + cs.row.t0) * Hq + cs.kvh * kGroup + g) * kHeadDim, ks,
                  P.sm_scale_log2e, c);
    st.load_query(1, P.q + (((size_t)cs.row.b * P.n_q + cs.row.t1) * Hq + cs.kvh * kGroup + g) * kHeadDim, ks,
                  P.sm_scale_log2e, c);
    st.reset();
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
      if ((tok0 < cs.row.lo) || (tok0 + TT > cs.row.LA))
        st.tile<true>(lo, kbase, vbase, tok0, cs.row.loA, cs.row.LA, cs.row.lo, cs.row.L, c);
      else
        st.tile<false>(lo, kbase, vbase, tok0, cs.row.loA, cs.row.LA, cs.row.lo, cs.row.L, c);
      __syncwarp();
      if (issue(kbase, bars + 8 * stage)) ++inflight;
      if (++stage == NS) { stage = 0; phase ^= 1u; }
    }
    if (failed) break;

    // ---- partial (o, lse) of this run of tiles, both tokens
    const float vs = P.v_scale ? P.v_scale[cs.kvh] : 1.f;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      float l_tot = st.l_run[t];
      l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 1);
      l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
      const float inv = l_tot > 0.f ? vs / l_tot : 0.f;
      const size_t row = (size_t)cs.prow + 8 * t + g;
      float* po = P.part_o + row * kHeadDim + 2 * c;
#pragma unroll
      for (int nd = 0; nd < 8; ++nd)
        *reinterpret_cast<float2*>(po + 8 * nd) =
            make_float2(st.O[nd][2 * t] * inv, st.O[nd][2 * t + 1] * inv);
      if (c == 0) P.part_lse[row] = l_tot > 0.f ? (st.m_ref[t] + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
    }
    // ---- arrival; the warp that completes the (row, KV head) merges it and leaves the counter at zero
    {
      const int p = cs.r * P.Hkv + cs.kvh;
      const int nt = (cum[cs.r + 1] - cum[cs.r]) / P.Hkv;
      const int g0 = cum[cs.r] + cs.kvh * nt;
      const int w0 = g0 / share, w1 = (g0 + nt - 1) / share;
      __threadfence();
      __syncwarp();
      int last = 0;
      if (lane == 0) last = atomicAdd(P.counters + p, 1) == w1 - w0;
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) {
        __threadfence();
        merge_tok_rows(P, cs.row, cs.kvh, ((long long)w0 + p) * kPairRows, w1 - w0 + 1, lane);
        if (lane == 0) P.counters[p] = 0;
      }
    }
  }

  // rows whose tokens see no key at all have no tile and hence no worker: zeros (lse = sink) from here
  if (!failed) {
    for (int p = w; p < rows * P.Hkv; p += nW) {
      const int r = p / P.Hkv;
      if (cum[r + 1] == cum[r]) {
        const RowInfo i = row_info(P, r);
        if (i.present) merge_tok_rows(P, i, p - r * P.Hkv, 0, 0, lane);
      }
    }
  }
  if (failed) {
    for (int i = 0; i < inflight; ++i) {
      mbar_wait_bounded(bars + 8 * stage, phase);
      if (++stage == NS) { stage = 0; phase ^= 1u; }
    }
  }
}

// Arrival counters (one per (sequence, token pair, KV head)) and partial rows of the kernel for a batch of `batch`
// sequences with up to n_q query tokens each.
size_t decode_attn_tokens_counters(int batch, int n_q, int Hkv) { return (size_t)batch * ((n_q + 1) / 2) * Hkv; }
size_t decode_attn_tokens_partial_rows(int ctas, int batch, int n_q, int Hkv) {
  return ((size_t)ctas * kTokWarps + (size_t)batch * ((n_q + 1) / 2) * Hkv) * kPairRows;
}

cudaError_t launch_decode_attn_tokens(const DecodeParams& P, int ctas, cudaStream_t s, int* smem_limit) {
  if (*smem_limit == 0) {
    int dev = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(decode_attn_tokens_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
    if (e != cudaSuccess) return e;
    *smem_limit = optin;
  }
  const int rows = P.batch * ((P.n_q + 1) / 2);
  const size_t need = 1024 + (size_t)kTokWarps * kTokStages * 2 * (kTokTile / kBlock) * kBlock * kHeadDim +
                      kTokWarps * kTokStages * 8 + (size_t)(rows + 1) * sizeof(int);
  if (need > (size_t)*smem_limit) return cudaErrorInvalidValue;  // too many rows for the schedule array
  return launch_dependent(decode_attn_tokens_kernel, dim3(ctas), dim3(kTokWarps * 32), need, s, P);
}

}  // namespace puzzle
