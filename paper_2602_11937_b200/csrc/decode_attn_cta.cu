// Split-KV decode attention over a paged KV cache (FP8 E4M3 codes, or bf16), sm_100a: the CTA-balanced kernel,
// default for the balanced schedule (num_splits = 0).
//
// Long-context decode is bound by KV-cache I/O (Section "Optimized Scenarios"), so what is left to win once every
// byte is read exactly once is time in which part of the chip has nothing to read.  With an equal static share per
// warp the launch ends when the slowest warp of the slowest SM ends; SMs differ in speed by their place on the chip
// (the same ones are slow in every launch) and the warps of one SM by the luck of their memory requests.  This
// kernel balances at both levels:
//
//  * The tile space of the batch (every (sequence, KV head) pair is a run of tiles of TT tokens; ragged contexts
//    and window layers included) is cut into one contiguous range per CTA.  Inside a CTA the twelve warps do not
//    own fixed shares: a warp takes the next tiles of the CTA's range (up to 16, fewer towards its end) with one
//    compare-and-swap on a shared-memory counter whenever its own TMA ring runs dry, so the warps of an SM finish
//    together.  (Only the very first chunk of every warp is fixed at set-up, when all twelve lie in one pair.)
//  * On large launches every CTA notes how many tiles per cycle it managed; the next large launch on the same
//    workspace cuts the ranges in proportion to those speeds (clamped to 0.8 .. 1.25 of the mean), so that all SMs
//    finish together.  The speeds live at the start of the workspace, before the arrival counters; a fresh
//    workspace gives equal ranges.  They change how the work is cut, never what is computed.
//
// A "piece" is the part of one pair inside one CTA's range.  A warp that leaves a piece deposits its running
// (max, sum, accumulator) in a shared-memory buffer of its own and adds its tile count to the piece's counter; the
// warp whose count completes the piece combines the deposits (nobody waits for a lock) and either writes the bf16
// output directly (the piece is the whole pair: short contexts, window layers) or stores ONE float32 partial for
// the piece and counts an arrival for the pair; the last arrival merges the pair's partials (log-sum-exp, sink
// folded in once).  Per-tile arithmetic: decode_tile.cuh.
//
// In this kernel a warp's time is a chain of dependent instructions between tensor-core work (about 25 cycles per
// instruction with twelve warps on the SM), so everything on the hand-out path is counted in instructions: 16-byte
// shared-memory accesses by address, no locks, nothing that one warp does while eleven wait.
//
// Waiting: a warp waits on an mbarrier of its own TMA ring, for its own deposit buffer to be collected by the warp
// that completes an earlier piece, or for the counter slot of the piece sixteen pieces back; pieces complete in
// order of hand-out, so the earliest open piece never waits.  Every wait is bounded and flags
// PUZZLE_DEV_WAIT_EXPIRED.
#include <cuda.h>

#include <climits>

#include "common.cuh"
#include "decode_attn.cuh"
#include "decode_sched.cuh"
#include "decode_tile.cuh"

namespace puzzle {
namespace {

constexpr int kMaxChunk = 16;    // most tiles handed to a warp at a time
constexpr int kPieceSlots = 16;  // tile counters of open pieces; pieces k and k + 16 of a CTA share one

// Hand-out state of a CTA (shared memory); the first 16 bytes are read by one load.
struct alignas(16) CtaCtl {
  int pos, end, lo, p_first;  // next tile to hand out; the CTA's range [lo, end) of the tile space; its first pair
  long long t0;               // clock when the kernels before this one had completed
  int warps_left;             // warps still running: the last one notes the CTA's speed
  int use_rates;              // this launch is large enough to note (and use) CTA speeds
  int4 seed[2];               // the pair the range starts in, as a PairCache record: every warp starts from it
  int first_n, pad[3];        // > 0: warp w's first claim is the first_n tiles from lo + w * first_n (no counter involved)
};

// Per-warp memory of the pair its last claim fell into (most claims fall into the same one again).  Two int4.
struct alignas(16) PairCache {
  int ps, pe, b, kvh;     // the pair's run in the tile space; the pair
  int tbase, L, lo, pad;  // absolute index of its first tile; visible keys of the sequence
};

// What a warp holds after a claim, and what travels with every tile through the TMA ring.  Two int4.
struct alignas(16) TileDesc {
  int b, kvh, t, k;     // sequence, KV head, absolute tile index, number of the piece within the CTA's range
  int total, L, lo, n;  // tiles of the piece, visible keys [lo, L), tiles in this claim (claims only)
};

__device__ __forceinline__ int4 lds128_volatile(uint32_t a) {
  int4 v;
  asm volatile("ld.volatile.shared.v4.s32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(a)
               : "memory");
  return v;
}
__device__ __forceinline__ void sts128(uint32_t a, int4 v) {
  asm volatile("st.shared.v4.s32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ int atoms_cas32(uint32_t a, int cmp, int val) {
  int old;
  asm volatile("atom.shared.cas.b32 %0, [%1], %2, %3;" : "=r"(old) : "r"(a), "r"(cmp), "r"(val) : "memory");
  return old;
}

struct SeqTiles {
  int L, lo, tlo, nt;  // clamped length, first visible key, first tile, tiles (per KV head)
};
template <int TT>
__device__ __forceinline__ SeqTiles seq_tiles(const DecodeParams& P, int b) {
  bool too_long;
  const SeqRange r = seq_range(P.seq_lens[b], P.window, P.max_blocks_per_seq * kBlock, TT, too_long);
  SeqTiles s;
  s.L = r.L; s.lo = r.lo; s.tlo = r.tlo; s.nt = r.ntile;
  return s;
}

// Largest b in [0, batch) with cum[b] <= x, for 0 <= x < cum[batch].
__device__ __forceinline__ int seq_of(const int* cum, int batch, int x) {
  int a = 0, z = batch;
  while (z - a > 1) {
    const int mid = (a + z) >> 1;
    if (cum[mid] <= x) a = mid; else z = mid;
  }
  return a;
}

// A cut of the tile space at x (0 < x < T), moved onto the start or end of the pair it falls into when that is no
// further than `snap` tiles away (a short pair then stays within one CTA and needs no partial at all).  Cuts at
// different x stay different unless both land on a pair boundary, so a range that meets a pair holds one of its
// tiles at least.
__device__ __forceinline__ int snap_cut(const int* cum, int batch, int Hkv, int x, int snap) {
  const int b = seq_of(cum, batch, x);
  const int nt = (cum[b + 1] - cum[b]) / Hkv;
  const int r = x - cum[b];
  const int ps = cum[b] + (r / nt) * nt, pe = ps + nt;
  if (x - ps <= snap) return ps;
  if (pe - x <= snap) return pe;
  return x;
}

// Takes the next tiles for a warp (one thread) and writes them to the warp's claim record: n > 0 tiles of one
// piece; n = 0: nothing is left; n = -1: gave up.  ctl_a, pc_a, rec_a are shared-memory addresses.
template <int TT>
__device__ __noinline__ void claim_tiles(uint32_t ctl_a, const DecodeParams& P, const int* cum, uint32_t pc_a,
                                         uint32_t rec_a) {
  int4 v = lds128_volatile(ctl_a);  // pos, end, lo, p_first
  int4 c0 = lds128_volatile(pc_a), c1 = lds128_volatile(pc_a + 16);
  for (int tries = 0; tries < (1 << 20); ++tries) {
    const int pos = v.x;
    if (pos >= v.y) {
      sts128(rec_a + 16, make_int4(0, 0, 0, 0));
      return;
    }
    if (pos < c0.x || pos >= c0.y) {  // another pair than last time
      int b = c0.z;
      SeqTiles q;
      if (c0.y > c0.x && pos >= cum[b] && pos < cum[b + 1]) {
        // another KV head of the same sequence (seven pair changes in eight): its lengths are known, and neither
        // the search nor the trip to global memory for the length stands between this warp and its next copies
        q.nt = c0.y - c0.x; q.tlo = c1.x; q.L = c1.y; q.lo = c1.z;
      } else {
        b = seq_of(cum, P.batch, pos);
        q = seq_tiles<TT>(P, b);
      }
      const int kvh = (pos - cum[b]) / q.nt;
      c0 = make_int4(cum[b] + kvh * q.nt, cum[b] + (kvh + 1) * q.nt, b, kvh);
      c1 = make_int4(q.tlo, q.L, q.lo, 0);
      sts128(pc_a, c0);
      sts128(pc_a + 16, c1);
    }
    const int hi = min(c0.y, v.y);
    const int n = min(hi - pos, max(1, min(kMaxChunk, (v.y - pos) >> 4)));
    const int old = atoms_cas32(ctl_a, pos, pos + n);
    if (old == pos) {
      sts128(rec_a, make_int4(c0.z, c0.w, c1.x + (pos - c0.x), c0.z * P.Hkv + c0.w - v.w));
      sts128(rec_a + 16, make_int4(hi - max(c0.x, v.z), c1.y, c1.z, n));
      return;
    }
    v.x = old;  // another warp was faster: go on from where it left the counter
  }
  sts128(rec_a + 16, make_int4(0, 0, 0, -1));
}

// Spins (bounded) until *p == want.
__device__ __forceinline__ bool wait_for(const int* p, int want) {
  for (int i = 0; i < (1 << 22); ++i) {
    if (*reinterpret_cast<const volatile int*>(p) == want) return true;
    if (i > 4096) __nanosleep(32);
  }
  return false;
}

// Producer side of one warp: the tiles it has claimed and not yet issued, and the block-table entries of the next
// tile to issue (fetched one tile ahead of their use).  Lane i < NB owns block i of a tile.
template <int TT>
struct ClaimProducer {
  static constexpr int NB = TT / kBlock;
  static constexpr int kNotVisible = INT_MIN;
  TileDesc d;  // d.t = next tile to issue, d.n = tiles left in the claim
  int phys;

  __device__ __forceinline__ void lookup(const DecodeParams& P, int lane) {
    phys = kNotVisible;
    if (d.n > 0 && lane < NB) {
      const int j = d.t * NB + lane;
      if ((j * kBlock < d.L) && (j * kBlock + kBlock > d.lo))
        phys = P.block_table ? P.block_table[(size_t)d.b * P.max_blocks_per_seq + j] : d.b * P.max_blocks_per_seq + j;
    }
  }
  // All lanes call it; returns false when the claim gave up.
  __device__ __forceinline__ bool claim(uint32_t ctl_a, const DecodeParams& P, const int* cum, uint32_t pc_a,
                                        uint32_t rec_a, int lane) {
    if (lane == 0) claim_tiles<TT>(ctl_a, P, cum, pc_a, rec_a);
    __syncwarp();
    const int4 a = lds128_volatile(rec_a), z = lds128_volatile(rec_a + 16);
    __syncwarp();
    d.b = a.x; d.kvh = a.y; d.t = a.z; d.k = a.w;
    d.total = z.x; d.L = z.y; d.lo = z.z; d.n = z.w;
    if (d.n < 0) { d.n = 0; return false; }
    return true;
  }
  // Issues the pending tile into `stage_addr` (its description goes to desc_a) and prepares the next one.
  // Returns 1 if a tile was issued, 0 if nothing was pending, -1 if a claim gave up.
  template <int BLOCK_BYTES>
  __device__ __forceinline__ int issue(uint32_t ctl_a, const DecodeParams& P, const int* cum, uint32_t pc_a,
                                       uint32_t rec_a, int lane, uint32_t stage_addr, uint32_t bar, uint32_t desc_a) {
    if (d.n <= 0) return 0;
    int row = P.oob_row;
    if (lane < NB) {
      if (phys >= 0 && phys < P.num_blocks) {
        row = (phys * P.Hkv + d.kvh) * P.rows_per_block;
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
      sts128(desc_a, make_int4(d.b, d.kvh, d.t, d.k));
      sts128(desc_a + 16, make_int4(d.total, d.L, d.lo, 0));
      mbar_arrive_expect_tx(bar, 2 * NB * BLOCK_BYTES);
#pragma unroll
      for (int i = 0; i < NB; ++i) tma_load_2d(stage_addr + i * BLOCK_BYTES, &P.tmK, 0, rows[i], bar);
#pragma unroll
      for (int i = 0; i < NB; ++i) tma_load_2d(stage_addr + (NB + i) * BLOCK_BYTES, &P.tmV, 0, rows[i], bar);
    }
    ++d.t;
    bool ok = true;
    if (--d.n == 0) ok = claim(ctl_a, P, cum, pc_a, rec_a, lane);
    lookup(P, lane);
    return ok ? 1 : -1;
  }
};

// Number of CTA ranges that meet the run [ps, pe) of a pair, and the first of them.
__device__ __forceinline__ int ranges_of(const int* bound, int nC, int ps, int pe, int& c_first) {
  int a = 0, z = nC;  // largest c with bound[c] <= ps
  while (z - a > 1) {
    const int mid = (a + z) >> 1;
    if (bound[mid] <= ps) a = mid; else z = mid;
  }
  c_first = a;
  a = c_first + 1; z = nC;  // smallest i > c_first with bound[i] >= pe  (bound[nC] = T >= pe)
  while (a < z) {
    const int mid = (a + z) >> 1;
    if (bound[mid] >= pe) z = mid; else a = mid + 1;
  }
  return a - c_first;
}

}  // namespace

// NW warps per CTA, NS stages per warp, TT tokens per tile; FP8 selects the E4M3 cache (else bf16).
template <int NW, int NS, int TT, bool FP8>
__global__ void __launch_bounds__(NW * 32, 1) decode_attn_cta_kernel(const __grid_constant__ DecodeParams P) {
  constexpr int NB = TT / kBlock;                       // blocks per tile
  constexpr int EB = FP8 ? 1 : 2;                       // bytes per cache element
  constexpr int BLOCK_BYTES = kBlock * kHeadDim * EB;   // one (block, KV head): 1 KiB or 2 KiB
  constexpr int STAGE_BYTES = 2 * NB * BLOCK_BYTES;
  constexpr int PIPE_BYTES = NW * NS * STAGE_BYTES;
  static_assert(NW <= 32 && NW <= kPieceSlots, "one deposit buffer per warp, found by one ballot");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;  // this lane's query head within the group / column quad
  const int nC = gridDim.x;
  const uint32_t pipe = smem_u32(smem) + warp * (NS * STAGE_BYTES);
  uint8_t* sp = smem + PIPE_BYTES;
  const uint32_t bars = smem_u32(sp) + warp * (NS * 8);                   sp += NW * NS * 8;
  const uint32_t desc_a = smem_u32(sp) + warp * NS * sizeof(TileDesc);    sp += NW * NS * sizeof(TileDesc);
  const uint32_t rec_a = smem_u32(sp) + warp * sizeof(TileDesc);          sp += NW * sizeof(TileDesc);
  const uint32_t pc_a = smem_u32(sp) + warp * sizeof(PairCache);          sp += NW * sizeof(PairCache);
  float4* dep_o = reinterpret_cast<float4*>(sp);                          sp += NW * 4 * 32 * sizeof(float4);  // [warp][j][lane]
  float* dep_m = reinterpret_cast<float*>(sp);                            sp += NW * kGroup * sizeof(float);
  float* dep_l = reinterpret_cast<float*>(sp);                            sp += NW * kGroup * sizeof(float);
  int* dep_piece = reinterpret_cast<int*>(sp);                            sp += 32 * sizeof(int);
  int* pk_key = reinterpret_cast<int*>(sp);                               sp += kPieceSlots * sizeof(int);
  int* pk_done = reinterpret_cast<int*>(sp);                              sp += kPieceSlots * sizeof(int);
  CtaCtl& ctl = *reinterpret_cast<CtaCtl*>(sp);                           sp += sizeof(CtaCtl);
  static_assert(sizeof(CtaCtl) % 16 == 0, "the arrays behind it stay aligned");
  const uint32_t ctl_a = smem_u32(&ctl);
  int* bound = reinterpret_cast<int*>(sp);                                sp += ((nC + 1 + 3) & ~3) * sizeof(int);
  int* share = reinterpret_cast<int*>(sp);                                sp += ((nC + 1 + 3) & ~3) * sizeof(int);
  int* cum = reinterpret_cast<int*>(sp);

  // speeds of the CTA slots from earlier launches: two buffers, the valid one named by `epoch`
  int* cta_done = P.cta_words;
  int* epoch_p = cta_done + 1;
  float* rates = reinterpret_cast<float*>(cta_done + 4);

  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < NS; ++i) mbar_init(bars + 8 * i, 1);
    fence_mbar_init();
  }
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&P.tmK);
    tma_prefetch_desc(&P.tmV);
  }
  if (threadIdx.x < 32) dep_piece[threadIdx.x] = -1;
  if (threadIdx.x < kPieceSlots) { pk_key[threadIdx.x] = -1; pk_done[threadIdx.x] = 0; }
  if (threadIdx.x == 0) cum[0] = 0;
  release_dependents();
  grid_dependency_wait();   // nothing above reads or writes global memory
  if (threadIdx.x == 0) ctl.t0 = clock64();
  // ---- schedule, step 1: tiles of every sequence
  for (int b = threadIdx.x; b < P.batch; b += blockDim.x) {
    bool too_long;
    const SeqRange r = seq_range(P.seq_lens[b], P.window, P.max_blocks_per_seq * kBlock, TT, too_long);
    if (too_long && P.dev_status && blockIdx.x == 0) atomicOr(P.dev_status, (int)PUZZLE_DEV_SEQ_TOO_LONG);
    cum[b + 1] = r.ntile * P.Hkv;
  }
  // one warp turns the noted speeds into cumulative shares (fixed point, 4096 = the mean speed); without a full set
  // of speeds every CTA gets the same share
  if (warp == 1) {
    // both buffers are fetched together with the switch that names the valid one: one round trip, not two
    const int ep_word = __ldcg(epoch_p);
    float r[8], r_other[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int cc = i * 32 + lane;
      const bool on = cc < nC && i * 32 < nC;
      r[i] = on ? __ldcg(rates + cc) : -1.f;
      r_other[i] = on ? __ldcg(rates + nC + cc) : -1.f;
    }
    float sum = 0.f, mn = 1e30f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int cc = i * 32 + lane;
      if (ep_word & 1) r[i] = r_other[i];
      if (cc < nC) { sum += r[i]; mn = fminf(mn, r[i]); }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      sum += __shfl_xor_sync(0xffffffffu, sum, d);
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, d));
    }
    const bool have = mn > 0.f && nC <= 256;
    const float inv_mean = have ? (float)nC / sum : 0.f;
    int carry = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int cc = i * 32 + lane;
      int q = 0;
      if (cc < nC) q = have ? (int)(fminf(fmaxf(r[i] * inv_mean, 0.8f), 1.25f) * 4096.f) : 4096;
      int v = q;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += u;
      }
      if (cc < nC) share[cc + 1] = v + carry;  // cumulative share up to and including CTA cc
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
    if (lane == 0) share[0] = 0;
  }
  __syncthreads();
  // ---- step 2 (one warp): prefix sums
  if (threadIdx.x < 32) {
    int carry = 0;
    for (int base = 0; base < P.batch; base += 32) {
      const int i = base + lane;
      int v = i < P.batch ? cum[i + 1] : 0;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += u;
      }
      if (i < P.batch) cum[i + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();
  // ---- step 3: range boundaries of all CTAs (the merge needs them), and this CTA's hand-out state.
  // Large launches are cut in proportion to the CTA speeds; small ones evenly over as many CTAs as there are tiles.
  // Every CTA evaluates the same expressions on the same numbers, so all agree on the cuts.
  {
    const int T = cum[P.batch];
    const bool large = T / nC >= kCtaRateMinTiles && nC <= 256;
    const int nR = large ? nC : max(1, min(nC, T));
    const int snap = max(1, (T / nR) >> 5);
    const float per_share = (float)T / (float)share[nC];
    auto boundary = [&](int i) {
      if (i <= 0) return 0;
      if (i >= nR) return T;
      // small launches on up to 256 CTAs: i * T < 2^24 (fewer than kCtaRateMinTiles tiles per CTA)
      const int x = large ? min(T - 1, (int)((float)share[i] * per_share))
                          : (nC <= 256 ? (i * T) / nR : (int)(((long long)i * T) / nR));
      return x > 0 ? snap_cut(cum, P.batch, P.Hkv, x, snap) : 0;
    };
    for (int i = threadIdx.x; i <= nC; i += blockDim.x) bound[i] = boundary(i);
    // one thread of an otherwise idle warp works out this CTA's own range at the same time, the pair it starts in
    // (every warp's first claim falls into it) and, when the first chunk of all NW warps lies inside that pair, hands
    // those chunks out right here: twelve warps that start together would otherwise retry each other's
    // compare-and-swap
    if (threadIdx.x == 32 * (NW - 1)) {
      const int lo_c = boundary(blockIdx.x), end_c = boundary(blockIdx.x + 1);
      int pf = 0, first_n = 0;
      int4 s0 = make_int4(0, 0, 0, 0), s1 = make_int4(0, 0, 0, 0);
      if (lo_c < end_c) {
        const int b = seq_of(cum, P.batch, lo_c);
        const SeqTiles q = seq_tiles<TT>(P, b);
        const int kvh = (lo_c - cum[b]) / q.nt;
        pf = b * P.Hkv + kvh;
        s0 = make_int4(cum[b] + kvh * q.nt, cum[b] + (kvh + 1) * q.nt, b, kvh);
        s1 = make_int4(q.tlo, q.L, q.lo, 0);
        const int c0 = max(1, min(kMaxChunk, (end_c - lo_c) >> 4));
        if (min(s0.y, end_c) - lo_c >= NW * c0) first_n = c0;
      }
      ctl.lo = lo_c;
      ctl.end = end_c;
      ctl.pos = lo_c + NW * first_n;
      ctl.p_first = pf;
      ctl.seed[0] = s0;
      ctl.seed[1] = s1;
      ctl.first_n = first_n;
      ctl.warps_left = NW;
      ctl.use_rates = large ? 1 : 0;
    }
  }
  __syncthreads();

  LaneOffsets<FP8> lo;
  lo.init(lane);

  ClaimProducer<TT> prod;
  bool failed = false;
  {
    const int4 s0 = ctl.seed[0], s1 = ctl.seed[1];
    const int first_n = ctl.first_n;
    if (lane == 0) {
      sts128(pc_a, s0);
      sts128(pc_a + 16, s1);
    }
    if (first_n > 0) {  // this warp's share of the range's first tiles: the claim record written in place
      const int pos = ctl.lo + warp * first_n;
      prod.d.b = s0.z; prod.d.kvh = s0.w; prod.d.t = s1.x + (pos - s0.x); prod.d.k = 0;
      prod.d.total = min(s0.y, ctl.end) - max(s0.x, ctl.lo); prod.d.L = s1.y; prod.d.lo = s1.z; prod.d.n = first_n;
    } else {
      __syncwarp();
      failed = !prod.claim(ctl_a, P, cum, pc_a, rec_a, lane);
    }
  }
  prod.lookup(P, lane);
  int inflight = 0;
#pragma unroll 1
  for (int i = 0; i < NS && !failed; ++i) {
    const int r = prod.template issue<BLOCK_BYTES>(ctl_a, P, cum, pc_a, rec_a, lane, pipe + i * STAGE_BYTES,
                                                   bars + 8 * i, desc_a + i * sizeof(TileDesc));
    if (r != 0) ++inflight;
    if (r < 0) failed = true;
  }
  __syncwarp();

  int stage = 0;
  uint32_t phase = 0;
  int cur_k = -1, cur_b = 0, cur_kvh = 0, cur_total = 0, nacc = 0;
  TileState st;
  st.reset();

#pragma unroll 1
  for (;;) {
    // the next tile's description is known since the tile was issued: a change of piece (its hand-over, the new
    // query) is dealt with while the tile's bytes are still on their way
    int4 d0 = make_int4(0, 0, 0, -1), d1 = make_int4(0, 0, 0, 0);
    const bool more = inflight > 0;
    if (more) {
      d0 = lds128_volatile(desc_a + stage * sizeof(TileDesc));
      d1 = lds128_volatile(desc_a + stage * sizeof(TileDesc) + 16);
    }
    if (d0.w != cur_k) {
      // ---- the piece changes (or nothing is left): hand this warp's share of the old piece over
      if (cur_k >= 0) {
        // fetched now, used at the very end (only the warp that completes the piece needs them)
        const float vs = P.v_scale && FP8 ? __ldg(P.v_scale + cur_kvh) : 1.f;
        const float sink_g = P.sinks ? __ldg(P.sinks + cur_kvh * kGroup + g) : -INFINITY;
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
        bool complete = nacc == cur_total;
        if (!complete) {
          // deposit in this warp's buffer (free once the warp that completed its previous piece has read it)
          int ok = 1;
          if (lane == 0) ok = wait_for(dep_piece + warp, -1);
          ok = __shfl_sync(0xffffffffu, ok, 0);
          __syncwarp();
          if (!ok) { failed = true; break; }
#pragma unroll
          for (int j = 0; j < 4; ++j)
            dep_o[(warp * 4 + j) * 32 + lane] = make_float4(o[2 * j][0], o[2 * j][1], o[2 * j + 1][0], o[2 * j + 1][1]);
          if (c == 0) {
            dep_m[warp * kGroup + g] = m;
            dep_l[warp * kGroup + g] = l_tot;
          }
          __syncwarp();
          int last = 0;
          const int e = cur_k & (kPieceSlots - 1);
          if (lane == 0) {
            *reinterpret_cast<volatile int*>(dep_piece + warp) = cur_k;
            __threadfence_block();
            // the piece's tile counter: taken from the free state by whoever comes first
            last = -1;
            for (int i = 0; i < (1 << 22); ++i) {
              const int key = *reinterpret_cast<volatile int*>(pk_key + e);
              if (key == cur_k) { last = 0; break; }
              if (key == -1) {
                const int old = atomicCAS(pk_key + e, -1, cur_k);
                if (old == -1 || old == cur_k) { last = 0; break; }
              }
              if (i > 4096) __nanosleep(32);  // the piece sixteen back is still open
            }
            if (last == 0) last = atomicAdd(pk_done + e, nacc) + nacc == cur_total ? 1 : 0;
            __threadfence_block();
          }
          last = __shfl_sync(0xffffffffu, last, 0);
          __syncwarp();
          if (last < 0) { failed = true; break; }
          if (last) {
            // ---- every tile of the piece is accounted for: combine the other warps' deposits with this one
            const int pcs = lane < NW ? *reinterpret_cast<volatile int*>(dep_piece + lane) : -2;
            const unsigned mask = __ballot_sync(0xffffffffu, pcs == cur_k) & ~(1u << warp);
            float M = m;
            for (unsigned mm = mask; mm; mm &= mm - 1) M = fmaxf(M, dep_m[(__ffs(mm) - 1) * kGroup + g]);
            const float fo = m == -INFINITY ? 0.f : ex2(m - M);
            l_tot *= fo;
#pragma unroll
            for (int nd = 0; nd < 8; ++nd) { o[nd][0] *= fo; o[nd][1] *= fo; }
            for (unsigned mm = mask; mm; mm &= mm - 1) {
              const int u = __ffs(mm) - 1;
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
            __syncwarp();  // all lanes have read the deposits: release the buffers and the counter
            if (lane < NW && ((mask | (1u << warp)) >> lane & 1u)) *reinterpret_cast<volatile int*>(dep_piece + lane) = -1;
            if (lane == 0) {
              pk_done[e] = 0;
              __threadfence_block();
              *reinterpret_cast<volatile int*>(pk_key + e) = -1;
            }
            complete = true;
          }
        }
        if (complete) {
          // ---- this warp holds the whole piece: output, or one partial for the pair's merge
          const int p = ctl.p_first + cur_k;
          const int nt = (cum[cur_b + 1] - cum[cur_b]) / P.Hkv;
          const int ps = cum[cur_b] + cur_kvh * nt;
          int c_first = blockIdx.x;
          const int count = cur_total == nt ? 1 : ranges_of(bound, nC, ps, ps + nt, c_first);  // the whole pair is here
          if (count == 1) {
            const int head = cur_kvh * kGroup + g;
            const long long row_out = (long long)cur_b * (P.Hkv * kGroup) + head;
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
            if (P.lse_out && c == 0)
              P.lse_out[row_out] = Z > 0.f ? (M + log2f(Z)) * 0.6931471805599453f : -INFINITY;
          } else {
            const float inv = l_tot > 0.f ? vs / l_tot : 0.f;
            const size_t row = (size_t)(blockIdx.x + p) * kGroup + g;
            float* po = P.part_o + row * kHeadDim + 2 * c;
#pragma unroll
            for (int nd = 0; nd < 8; ++nd)
              *reinterpret_cast<float2*>(po + 8 * nd) = make_float2(o[nd][0] * inv, o[nd][1] * inv);
            if (c == 0) P.part_lse[row] = l_tot > 0.f ? (m + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
            __threadfence();  // this lane's partial stores before the arrival
            __syncwarp();
            int last = 0;
            if (lane == 0) last = atomicAdd(P.counters + p, 1) == count - 1;
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
              __threadfence();  // the arrivals before the other pieces' partials are read
              merge_rows(P, cur_b, cur_kvh, (long long)(c_first + p) * kGroup, count, kGroup, 1, 0, 0, 0, lane);
              if (lane == 0) P.counters[p] = 0;
            }
          }
        }
      }
      if (!more) break;
      cur_k = d0.w; cur_b = d0.x; cur_kvh = d0.y; cur_total = d1.x;
      nacc = 0;
      st.template load_query<FP8>(P.q + ((size_t)cur_b * (P.Hkv * kGroup) + cur_kvh * kGroup + g) * kHeadDim,
                                  P.k_scale && FP8 ? P.k_scale[cur_kvh] : 1.f, P.sm_scale_log2e, c);
      st.reset();
    }
    if (!more) break;
    if (!mbar_wait_bounded(bars + 8 * stage, phase)) {
      failed = true;
      break;
    }
    --inflight;
    const uint32_t kbase = pipe + stage * STAGE_BYTES;
    const uint32_t vbase = kbase + NB * BLOCK_BYTES;
    const int tok0 = d0.z * TT;
    if ((tok0 < d1.z) || (tok0 + TT > d1.y))
      st.template tile<TT, FP8, true>(lo, kbase, vbase, tok0, d1.z, d1.y, c);
    else
      st.template tile<TT, FP8, false>(lo, kbase, vbase, tok0, d1.z, d1.y, c);
    ++nacc;

    // ---- refill this stage with the next tile this warp holds
    __syncwarp();
    const int r = prod.template issue<BLOCK_BYTES>(ctl_a, P, cum, pc_a, rec_a, lane, kbase, bars + 8 * stage,
                                                   desc_a + stage * sizeof(TileDesc));
    if (r != 0) ++inflight;
    if (++stage == NS) { stage = 0; phase ^= 1u; }
    if (r < 0) { failed = true; break; }
  }

  // pairs without any visible key have no tile and hence no piece: zeros (lse = sink) from here
  if (!failed) {
    for (int p = blockIdx.x * NW + warp; p < P.batch * P.Hkv; p += nC * NW) {
      const int b = p / P.Hkv;
      if (cum[b + 1] == cum[b]) merge_rows(P, b, p - b * P.Hkv, 0, 0, 0, 0, 0, 0, 0, lane);
    }
  }

  if (failed) {
    if (lane == 0 && P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_WAIT_EXPIRED);
    // give the copies still in flight a bounded chance to land before the CTA's shared memory is released
    for (int i = 0; i < inflight; ++i) {
      mbar_wait_bounded(bars + 8 * stage, phase);
      if (++stage == NS) { stage = 0; phase ^= 1u; }
    }
  }

  // ---- the last warp of the CTA notes its speed for the next large launch; the last CTA switches the buffers
  if (lane == 0 && atomicSub(&ctl.warps_left, 1) == 1 && ctl.use_rates && !failed) {
    const int ep = *reinterpret_cast<const volatile int*>(epoch_p) & 1;
    const float cycles = (float)(clock64() - ctl.t0);
    // a CTA's speed varies by a few percent from launch to launch around a value that belongs to its place on the
    // chip; the running average keeps the latter
    const float now = (float)(ctl.end - ctl.lo) / fmaxf(cycles, 1.f), before = __ldcg(rates + ep * nC + blockIdx.x);
    rates[(1 - ep) * nC + blockIdx.x] = before > 0.f ? 0.875f * before + 0.125f * now : now;
    __threadfence();
    if (atomicAdd(cta_done, 1) == nC - 1) {
      *cta_done = 0;
      __threadfence();
      *reinterpret_cast<volatile int*>(epoch_p) = 1 - ep;
    }
  }
}

template <int NW, int NS, int TT, bool FP8>
static size_t cta_smem_bytes(int batch, int ctas) {
  constexpr int STAGE_BYTES = 2 * (TT / kBlock) * kBlock * kHeadDim * (FP8 ? 1 : 2);
  return 1024 + (size_t)NW * NS * STAGE_BYTES + NW * NS * 8 + (size_t)NW * NS * sizeof(TileDesc) +
         NW * sizeof(TileDesc) + NW * sizeof(PairCache) + (size_t)NW * 4 * 32 * sizeof(float4) +
         2 * NW * kGroup * sizeof(float) + 32 * sizeof(int) + 2 * kPieceSlots * sizeof(int) + sizeof(CtaCtl) +
         2 * (size_t)((ctas + 1 + 3) & ~3) * sizeof(int) + (size_t)(batch + 1) * sizeof(int);
}

template <int NW, int NS, int TT, bool FP8>
static cudaError_t launch_cta_variant(const DecodeParams& P, int ctas, cudaStream_t s, int& smem_limit) {
  auto kern = decode_attn_cta_kernel<NW, NS, TT, FP8>;
  if (smem_limit == 0) {  // first launch of this variant on this device: raise its dynamic shared-memory limit
    int dev = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
    if (e != cudaSuccess) return e;
    smem_limit = optin;
  }
  const size_t need = cta_smem_bytes<NW, NS, TT, FP8>(P.batch, ctas);
  if (need > (size_t)smem_limit) return cudaErrorInvalidValue;
  return launch_dependent(kern, dim3(ctas), dim3(NW * 32), need, s, P);
}

cudaError_t launch_decode_attn_cta(const DecodeParams& P, bool fp8, int ctas, cudaStream_t s, int* smem_limit) {
  return fp8 ? launch_cta_variant<kDecodeWarpsFp8, kDecodeStagesFp8, kTileFp8, true>(P, ctas, s, smem_limit[0])
             : launch_cta_variant<kDecodeWarpsBf16, kDecodeStagesBf16, kTileBf16, false>(P, ctas, s, smem_limit[1]);
}

}  // namespace puzzle
