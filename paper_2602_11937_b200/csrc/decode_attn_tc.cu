// Split-KV decode attention over an FP8 (E4M3) paged KV cache on the 5th-generation tensor cores
// (tcgen05 MMA with accumulators in tensor memory), sm_100a.
//
// Decode over a long context is bound by KV-cache I/O (paper, Section "Optimized Scenarios"); FP8 KV halves
// those bytes (Section "KV Quantization"), window layers bound them by W (Section "Window attention for
// long-context inference").  Here the E4M3 codes go from HBM to the tensor cores untouched:
//
//  * A CTA holds two independent workers ("groups") of ten warps: a copy warp, a warp whose lane 0 issues the
//    MMAs, and eight softmax warps.  A worker streams its share of the batch's tile space (tiles of 128 tokens
//    of one (sequence, KV head)) through a ring of TMA stages: K tile and V tile as eight 1 KiB blocks each,
//    64-byte swizzle, looked up in the block table.
//  * S = K Q^T: the K tile is the A operand as it landed (tokens on the 128 accumulator rows, K-major);
//    B holds the 8 query heads of the group twice, as the high and the low part of an exact two-term E4M3
//    split of the bf16 query.  The 128 x 16 result sits in tensor memory; a softmax thread reads the row of
//    ITS token for four of the heads (warps 0..3 of a worker take heads 0..3, warps 4..7 heads 4..7), so the
//    softmax needs no shuffle.
//  * The weights p = 2^(logit - m_ref) are split into four E4M3 terms (p = t1 + t2/16 + t3/256 + t4/4096,
//    15 significant bits), written token-major to shared memory, and O^T = V^T P accumulates in tensor memory
//    over the whole run of tiles: V is the A operand as it landed (MN-major), P the MN-major B operand.
//    The reference maximum m_ref is shared by the group and raised (accumulator rescaled in tensor memory)
//    only when a tile exceeds it by more than 2^8.
//  * At the end of a (sequence, KV head) run the group reads the accumulator, writes one float32 partial
//    (o, lse); the worker whose partial completes a (sequence, KV head) merges all of them and stores bf16.
//  Every wait is bounded, the barrier of a group's softmax warps included (an mbarrier with a poll limit that
//  also watches the abort flag, not a named barrier): a wait that runs out sets PUZZLE_DEV_WAIT_EXPIRED and the
//  abort flag, and every role then leaves its loop, whichever warp of a group notices first.
//
//  Copies and MMAs are issued under an elect.sync predicate with the whole warp in the loop: inside an
//  `if (lane == 0)` branch the compiler elects a lane and moves every operand to a uniform register per
//  instruction, which cost about 126 cycles per MMA and 100 per TMA box here.  Measured on B200 the kernel is now
//  bound by its softmax warps (about 1950 cycles per tile and worker, where HBM speed needs 1460), and it executes
//  about twice the instructions per token of the mma.sync kernel, so it stays behind it.
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "decode_attn.cuh"
#include "decode_sched.cuh"

namespace puzzle {

namespace {

constexpr int TT = 128;                    // tokens per tile
constexpr int NBLK = TT / kBlock;          // cache blocks per tile
constexpr int KV_TILE = TT * kHeadDim;     // bytes of a K (or V) tile
constexpr int STAGE = 2 * KV_TILE;         // K tile + V tile
constexpr int G = 2;                       // workers per CTA
constexpr int S = 5;                       // TMA stages per worker
constexpr int P_BYTES = TT * 32;           // one P tile: 128 tokens x (4 terms x 8 heads) codes
constexpr int Q_BYTES = 16 * 64;           // high and low query rows of the 8 heads
constexpr int GROUP_BYTES = S * STAGE + 2 * P_BYTES + Q_BYTES;
constexpr int SW = 8;                      // softmax warps per worker
constexpr int CW = 1;                      // copy warps per worker (1 or 3: box i of a tile belongs to copy warp i % CW)
constexpr int HW = CW + 1;                 // helper warps per worker: the copy warps and one that issues the MMAs
constexpr int kThreads = (HW * G + SW * G) * 32;
static_assert((HW * G) % 4 == 0, "softmax warp i must have i % 4 = its tensor-memory lane quadrant");
// Tensor memory of a worker (columns): S = K Q^T as two buffers of 16 columns, then O^T as 32 columns.
constexpr int kS = 0, kO = 32, kTmemCols = 64;
constexpr float kLazyLog2 = 8.0f;
constexpr unsigned kFull = 0xffffffffu;
static_assert(GROUP_BYTES % 1024 == 0, "stage bases must keep the swizzle alignment");

struct GroupCtl {
  uint64_t kv_full[S], kv_empty[S];
  uint64_t d1_full[2], d1_empty[2];
  uint64_t p_full[2], pv_done[2];
  uint64_t verdict[2];     // the softmax warps have posted whether the reference maximum covers their rows
  uint64_t q_full;
  uint64_t gsync;          // barrier of the group's softmax warps (one arrival per warp)
  float alpha[kGroup];     // logit scale per head in log2 units (k_scale and the query's power of two folded in)
  float xchg[4][kGroup];   // per-warp values exchanged inside the group (tile maxima, weight sums)
  int raise[2];            // by tile parity: some warp's rows exceed the reference by more than 2^8
  int pad[2];
};

struct CtaCtl {
  GroupCtl grp[G];
  uint32_t tmem_base;
  volatile int abort;
};

// ---------------------------------------------------------------- small PTX wrappers
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Non-blocking: has the phase with this parity completed?
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (16-byte units), layout type
// (0 = no swizzle, 4 = 64-byte swizzle), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)(layout & 7) << 61;
  return d;
}
// D[tmem] (+)= A[smem] * B[smem], E4M3 x E4M3 -> f32, issued by one thread.
__device__ __forceinline__ void umma_e4m3(uint32_t taddr, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(taddr), "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
               ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t f16x2_to_e4m3x2(uint32_t h2) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(r) : "r"(h2));
  return r;
}
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t codes) {
  uint32_t r;
  const uint16_t c = (uint16_t)codes;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(c));
  return r;
}
__device__ __forceinline__ uint32_t h2_sub_mul16(uint32_t a, uint32_t b) {  // (a - b) * 16, packed halves, exact here
  const __half2 d = __hsub2(*reinterpret_cast<const __half2*>(&a), *reinterpret_cast<const __half2*>(&b));
  const __half2 r = __hmul2(d, __float2half2_rn(16.f));
  return *reinterpret_cast<const uint32_t*>(&r);
}

// Four E4M3 terms of two weights: p = t1 + t2/16 + t3/256 + t4/4096 (each term two codes in the low 16 bits).
__device__ __forceinline__ void split_pair(float p0, float p1, uint32_t (&t)[4]) {
  const uint32_t ph = f32x2_to_f16x2(p0, p1);
  const float2 phf = __half22float2(*reinterpret_cast<const __half2*>(&ph));
  t[3] = f32x2_to_e4m3x2((p0 - phf.x) * 4096.f, (p1 - phf.y) * 4096.f);  // what f16 dropped
  t[0] = f16x2_to_e4m3x2(ph);
  const uint32_t r1 = h2_sub_mul16(ph, e4m3x2_to_f16x2(t[0]));
  t[1] = f16x2_to_e4m3x2(r1);
  const uint32_t r2 = h2_sub_mul16(r1, e4m3x2_to_f16x2(t[1]));
  t[2] = f16x2_to_e4m3x2(r2);
}

}  // namespace

__global__ void __launch_bounds__(kThreads, 1) decode_attn_tc_kernel(const __grid_constant__ DecodeParams P) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  CtaCtl* C = reinterpret_cast<CtaCtl*>(smem + G * GROUP_BYTES);
  int* cum = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(C) + ((sizeof(CtaCtl) + 15) & ~15));
  int* lens = cum + P.batch + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int Hkv = P.Hkv;

  // ---- set-up: barriers, tensor memory, schedule
  if (threadIdx.x == 0) {
    for (int g = 0; g < G; ++g) {
      GroupCtl* c = &C->grp[g];
      for (int i = 0; i < S; ++i) { mbar_init(smem_u32(&c->kv_full[i]), CW); mbar_init(smem_u32(&c->kv_empty[i]), 1); }
      for (int i = 0; i < 2; ++i) {
        mbar_init(smem_u32(&c->d1_full[i]), 1); mbar_init(smem_u32(&c->d1_empty[i]), SW);
        mbar_init(smem_u32(&c->p_full[i]), SW); mbar_init(smem_u32(&c->pv_done[i]), 1);
        mbar_init(smem_u32(&c->verdict[i]), SW);
        c->raise[i] = 0;
      }
      mbar_init(smem_u32(&c->q_full), SW);
      mbar_init(smem_u32(&c->gsync), SW);
    }
    C->abort = 0;
    fence_mbar_init();
    tma_prefetch_desc(&P.tmK);
    tma_prefetch_desc(&P.tmV);
  }
  if (warp == 0) {  // owns the tensor-memory allocation: 64 columns per worker
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 128;" ::"r"(smem_u32(&C->tmem_base))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  build_schedule(cum, lens, P.seq_lens, P.batch, Hkv, P.window, P.max_blocks_per_seq * kBlock, TT, P.dev_status);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = C->tmem_base;

  // first the helper warps, HW per worker (copy warps, then the MMA warp); then SW softmax warps per worker
  const int role = warp < HW * G ? ((warp % HW) == CW ? 1 : 0) : 2;
  const int g = role < 2 ? warp / HW : (warp - HW * G) / SW;
  const int cw = warp % HW;   // copy warp index within the worker
  GroupCtl* ctl = &C->grp[g];
  const uint32_t gbase = smem_u32(smem) + g * GROUP_BYTES;    // stages, then the two P tiles, then the query rows
  const uint32_t pbase = gbase + S * STAGE, qbase = pbase + 2 * P_BYTES;
  const int nW = (int)gridDim.x * G;
  const int w = blockIdx.x * G + g;
  Cursor cur;
  if (P.num_splits == 0) {
    const int T = cum[P.batch];
    const int q = (T + nW - 1) / nW;
    cur.pos = min(w * q, T);
    cur.end = min(cur.pos + q, T);
    cur.step = 0;
  } else {
    // one contiguous share of the units per worker, shares in the order worker 0 of every CTA, worker 1 of every
    // CTA: a worker meets one or two (sequence, KV head) pairs only (see decode_attn.cu on why not round-robin)
    const long long units = (long long)P.batch * Hkv * P.num_splits;
    const int wi = g * (int)gridDim.x + blockIdx.x;
    cur.pos = (int)(wi * units / nW);
    cur.end = (int)((wi + 1) * units / nW);
    cur.step = 1;
  }
  Segment seg;
  auto give_up = [&]() {
    if (P.dev_status) atomicOr(P.dev_status, (int)PUZZLE_DEV_WAIT_EXPIRED);
    C->abort = 1;
  };

  if (role == 0) {
    // =============================================================== copies
    // A warp's TMA copies are handled one after the other (about 140 cycles per 1 KiB box); with several copy
    // warps, box i of a tile (K blocks 0..7, V blocks 8..15) belongs to copy warp i % CW.
    // Block-table entries are fetched for four tiles at a time (lane = 8 * tile + block), one batch ahead of
    // the copies, so the copies of a tile never wait for a table lookup.
    auto lookup = [&](const Segment& sg, int t0) -> int {
      int row = P.oob_row;   // row coordinate of the block in the 64-byte-row view (outside the map: zeros)
      const int t = t0 + (lane >> 3);
      if (t < sg.t_end) {
        const int j = t * NBLK + (lane & 7);
        if ((j * kBlock < sg.L) && (j * kBlock + kBlock > sg.lo)) {
          const long long phys = P.block_table ? (long long)P.block_table[(size_t)sg.b * P.max_blocks_per_seq + j]
                                               : (long long)sg.b * P.max_blocks_per_seq + j;
          if (phys >= 0 && phys < P.num_blocks) row = (int)((phys * Hkv + sg.kvh) * kBlock);
          else if (P.dev_status && cw == 0) atomicOr(P.dev_status, (int)PUZZLE_DEV_BAD_BLOCK);
        }
      }
      return row;
    };
    constexpr int kMine = (2 * NBLK + CW - 1) / CW;
    const uint32_t my_bytes = (uint32_t)((2 * NBLK - cw + CW - 1) / CW) * 1024u;
    int n = 0;
    bool dead = false;
    while (!dead && next_segment<TT>(cur, seg, P, cum, lens, w)) {   // aborts are seen warp-wide below
      if (seg.t == seg.t_end) continue;
      int row_next = lookup(seg, seg.t);
      for (int t0 = seg.t; t0 < seg.t_end && !dead; t0 += 4) {
        const int row_cur = row_next;
        if (t0 + 4 < seg.t_end) row_next = lookup(seg, t0 + 4);
        const int nt = min(4, seg.t_end - t0);
        for (int i = 0; i < nt; ++i, ++n) {
          const int s = n % S;
          if (!__all_sync(kFull, !C->abort && mbar_wait_bounded(smem_u32(&ctl->kv_empty[s]), ((uint32_t)(n / S) & 1u) ^ 1u))) {
            if (!C->abort) give_up();
            dead = true;
            break;
          }
          int rows[kMine];
#pragma unroll
          for (int k = 0; k < kMine; ++k) rows[k] = __shfl_sync(kFull, row_cur, 8 * i + ((cw + CW * k) & 7));
          if (elect_one()) {
            const uint32_t bar = smem_u32(&ctl->kv_full[s]);
            const uint32_t dst = gbase + s * STAGE;
            mbar_arrive_expect_tx(bar, my_bytes);
#pragma unroll
            for (int k = 0; k < kMine; ++k) {
              const int box = cw + CW * k;
              if (box < 2 * NBLK) tma_load_2d(dst + box * 1024, box < NBLK ? &P.tmK : &P.tmV, 0, rows[k], bar);
            }
          }
          __syncwarp();
        }
      }
    }
  } else if (role == 1) {
    // =============================================================== MMA issue (one thread)
    // S = K Q^T runs up to two tiles ahead of the softmax warps (two accumulator buffers); O^T += V^T P of a
    // tile is issued as soon as its P is in shared memory.  The first S of a run is issued only once every
    // P.V of the runs before it has been issued: the softmax warps write the run's query rows after they have
    // finished the run before, which needs those products.
    {
      constexpr uint32_t kIdescQK = (1u << 4) | (2u << 17) | (8u << 24);   // f32; both K-major; N = 16, M = 128
      constexpr uint32_t kIdescPV = (1u << 4) | (1u << 15) | (1u << 16) | (4u << 17) | (4u << 24);  // MN-major; N = 32, M = 64
      const uint32_t td = tmem + g * kTmemCols;
      auto next_run = [&](Cursor& c, Segment& sg) {   // next (sequence, KV head) run that has tiles
        bool ok;
        do ok = next_segment<TT>(c, sg, P, cum, lens, w); while (ok && sg.t == sg.t_end);
        return ok;
      };
      Cursor qcur = cur, pcur = cur;
      Segment qseg, pseg;
      bool q_on = next_run(qcur, qseg), p_on = next_run(pcur, pseg);
      int qn = 0, qt = q_on ? qseg.t : 0, qsegno = 0;   // S = K Q^T: tiles issued, next tile, runs started
      int pn = 0, pt = p_on ? pseg.t : 0;               // O^T += V^T P likewise
      bool dead = false;
      while ((q_on || p_on) && !dead) {   // an abort raised elsewhere is seen by the warp-wide checks below
        while (q_on && qn < pn + 2 && (qt != qseg.t || qn == pn)) {
          const int s = qn % S, b = qn & 1;
          bool ok = true;
          if (qt == qseg.t) ok = mbar_wait_bounded(smem_u32(&ctl->q_full), (uint32_t)qsegno & 1u);
          ok = ok && mbar_wait_bounded(smem_u32(&ctl->kv_full[s]), (uint32_t)(qn / S) & 1u) &&
               mbar_wait_bounded(smem_u32(&ctl->d1_empty[b]), ((uint32_t)(qn >> 1) & 1u) ^ 1u);
          ok = __all_sync(kFull, ok && !C->abort);   // one decision for the warp: the issue below is warp-collective
          if (!ok) { if (!C->abort) give_up(); dead = true; break; }
          tc_fence_after();
          const uint32_t kaddr = gbase + s * STAGE;
          if (elect_one()) {
#pragma unroll
            for (int ks = 0; ks < 2; ++ks)   // 32 dims per MMA
              umma_e4m3(td + kS + 16 * b, smem_desc(kaddr + ks * 32, 16, 512, 4),
                        smem_desc(qbase + ks * 32, 16, 512, 4), kIdescQK, (uint32_t)ks);
            umma_commit(smem_u32(&ctl->d1_full[b]));
          }
          __syncwarp();
          ++qn;
          if (++qt == qseg.t_end) {
            ++qsegno;
            q_on = next_run(qcur, qseg);
            qt = q_on ? qseg.t : 0;
          }
        }
        if (dead || !p_on) continue;
        {
          const int s = pn % S, b = pn & 1;
          if (!__all_sync(kFull, mbar_wait_bounded(smem_u32(&ctl->p_full[b]), (uint32_t)(pn >> 1) & 1u) && !C->abort)) {
            if (!C->abort) give_up();
            break;
          }
          tc_fence_after();
          const uint32_t vaddr = gbase + s * STAGE + KV_TILE, paddr = pbase + b * P_BYTES;
          if (elect_one()) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)   // 32 tokens per MMA
              umma_e4m3(td + kO, smem_desc(vaddr + ks * 2048, 16, 512, 4),
                        smem_desc(paddr + ks * 1024, 256, 128, 0), kIdescPV, (pt == pseg.t && ks == 0) ? 0u : 1u);
            umma_commit(smem_u32(&ctl->pv_done[b]));
            umma_commit(smem_u32(&ctl->kv_empty[s]));   // the stage: its K was consumed before this P existed
          }
          __syncwarp();
          ++pn;
          if (++pt == pseg.t_end) {
            p_on = next_run(pcur, pseg);
            pt = p_on ? pseg.t : 0;
          }
        }
      }
    }
  } else {
    // =============================================================== softmax (8 warps: 128 token rows x 2 head halves)
    const int sw = warp - HW * G - SW * g;   // 0..7 within the group
    const int wq = sw & 3;                  // tensor-memory lane quadrant (= warp index mod 4)
    const int hh = sw >> 2;                 // which four heads of the group
    const int H0 = 4 * hh;
    const int row = 32 * wq + lane;         // token row of the tile this thread owns
    const int gi = sw * 32 + lane;          // 0..255 within the group
    const uint32_t td = tmem + g * kTmemCols + ((uint32_t)(32 * wq) << 16);
    int n = 0;
    bool dead = false;
    // Barrier of the group's eight softmax warps on an mbarrier, so that it has a limit like every other wait: a
    // warp that has left (its own wait ran out, or it saw the abort flag) lets the others run into the limit or
    // see the flag, never wait for ever.  False: leave.
    uint32_t gphase = 0;
    auto group_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->gsync));
      bool ok = false;
      for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (mbar_try_wait(smem_u32(&ctl->gsync), gphase)) { ok = true; break; }
        if (C->abort) break;
      }
      gphase ^= 1u;
      if (!ok) { give_up(); dead = true; }
      return ok;
    };
    while (!dead && !C->abort && next_segment<TT>(cur, seg, P, cum, lens, w)) {
      if (seg.t == seg.t_end) {  // empty split (explicit schedule): weight zero
        if (gi < kGroup) P.part_lse[seg.prow + gi * seg.pstride] = -INFINITY;
        __threadfence();
        if (!group_sync()) break;
        if (gi < 32) arrive_and_merge(P, seg.b, seg.kvh, cum, nW, lane);
        continue;
      }
      // ---- the query rows of this (sequence, KV head): exact E4M3 high + low parts, 64-byte swizzle.
      // Thread gi < 128: head gi/16, dims 4*(gi%16)..+3.  Row of head h: 8*(h/4) + h%4, its low part 4 rows on,
      // so that the eight columns of S a softmax thread needs are adjacent.
      if (gi < 128) {
        const int h = gi >> 4, part = gi & 15;
        const __nv_bfloat16* qrow = P.q + ((size_t)seg.b * (Hkv * kGroup) + seg.kvh * kGroup + h) * kHeadDim + 4 * part;
        const uint2 raw2 = *reinterpret_cast<const uint2*>(qrow);
        float x[4] = {__uint_as_float(raw2.x << 16), __uint_as_float(raw2.x & 0xffff0000u),
                      __uint_as_float(raw2.y << 16), __uint_as_float(raw2.y & 0xffff0000u)};
        float amax = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) amax = fmaxf(amax, __shfl_xor_sync(kFull, amax, d));
        int shift = 0;
        if (amax > 0.f) {
          shift = 7 - ((int)(__float_as_uint(amax) >> 23) - 127);   // amax * 2^shift in [128, 256)
          shift = max(-120, min(120, shift));
        }
        const float up = __uint_as_float((uint32_t)(127 + shift) << 23);
        uint32_t hi = 0, lo = 0;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const float x0 = x[2 * k] * up, x1 = x[2 * k + 1] * up;
          const uint32_t h16 = f32x2_to_e4m3x2(x0, x1);
          const uint32_t back = e4m3x2_to_f16x2(h16);
          const float2 bf = __half22float2(*reinterpret_cast<const __half2*>(&back));
          const uint32_t l16 = f32x2_to_e4m3x2((x0 - bf.x) * 16.f, (x1 - bf.y) * 16.f);
          hi |= h16 << (16 * k);
          lo |= l16 << (16 * k);
        }
        const uint32_t chunk = part >> 2, inner = (part & 3) * 4;
        const int r_hi = 8 * (h >> 2) + (h & 3), r_lo = r_hi + 4;
        uint8_t* qs = smem + g * GROUP_BYTES + S * STAGE + 2 * P_BYTES;
        *reinterpret_cast<uint32_t*>(qs + r_hi * 64 + ((chunk ^ ((r_hi >> 1) & 3)) << 4) + inner) = hi;
        *reinterpret_cast<uint32_t*>(qs + r_lo * 64 + ((chunk ^ ((r_lo >> 1) & 3)) << 4) + inner) = lo;
        if (part == 0) {
          const float ks = P.k_scale ? P.k_scale[seg.kvh] : 1.f;
          const float down = __uint_as_float((uint32_t)(127 - shift) << 23);
          ctl->alpha[h] = fmaxf(P.sm_scale_log2e * ks * down, 1e-30f);
        }
      }
      fence_proxy_async();    // the query rows are read by the tensor core
      if (!group_sync()) break;
      if (lane == 0) mbar_arrive(smem_u32(&ctl->q_full));
      float a_hi[4], a_lo[4], m_ref[4], l_run[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a_hi[i] = ctl->alpha[H0 + i];
        a_lo[i] = a_hi[i] * 0.0625f;
        m_ref[i] = -INFINITY;
        l_run[i] = 0.f;
      }

      bool d1_ready = false;   // the next tile's S was already seen complete (tested a tile ahead)
      for (int t = seg.t; t < seg.t_end; ++t, ++n) {
        const int b = n & 1;
        if (!d1_ready && !mbar_wait_bounded(smem_u32(&ctl->d1_full[b]), (uint32_t)(n >> 1) & 1u)) { give_up(); dead = true; break; }
        tc_fence_after();
        uint32_t r[8];
        tmem_ld8(td + kS + 16 * b + 8 * hh, r);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->d1_empty[b]));
        // ---- logits (log2 units); does the reference maximum still cover this warp's rows?
        const int tok = t * TT + row;
        float tl[4];
        bool fits = true;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          tl[i] = fmaf(__uint_as_float(r[4 + i]), a_lo[i], __uint_as_float(r[i]) * a_hi[i]);
          fits = fits && (tl[i] <= m_ref[i] + kLazyLog2);
        }
        if (t * TT < seg.lo || t * TT + TT > seg.L) {   // an edge tile: codes of keys outside [lo, L) may be anything
          if (tok < seg.lo || tok >= seg.L) {
#pragma unroll
            for (int i = 0; i < 4; ++i) tl[i] = -INFINITY;
            fits = true;
          }
        }
        // post this warp's verdict; the group's verdict is read only after the weights have been computed, so
        // nobody waits for a slower warp while it still has work of its own
        const bool warp_fits = __all_sync(kFull, fits);
        if (lane == 0) {
          if (!warp_fits) atomicOr(&ctl->raise[b], 1);
          __threadfence_block();
          mbar_arrive(smem_u32(&ctl->verdict[b]));
        }
        // state of the two buffers this tile still needs, tested now, used later
        const bool pv_ok = mbar_test(smem_u32(&ctl->pv_done[b]), ((uint32_t)(n >> 1) & 1u) ^ 1u);
        const bool d1_next = (t + 1 < seg.t_end) && mbar_test(smem_u32(&ctl->d1_full[b ^ 1]), (uint32_t)((n + 1) >> 1) & 1u);

        // ---- weights against the current reference (speculative), their four-term split: word k of pk holds
        // term k + 1 of this thread's four heads
        uint32_t pk[4];
        float l_add[4];
        auto weights = [&]() {
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const float m0 = (m_ref[2 * j] == -INFINITY) ? 0.f : m_ref[2 * j];
            const float m1 = (m_ref[2 * j + 1] == -INFINITY) ? 0.f : m_ref[2 * j + 1];
            const float p0 = ex2(tl[2 * j] - m0), p1 = ex2(tl[2 * j + 1] - m1);
            l_add[2 * j] = p0;
            l_add[2 * j + 1] = p1;
            uint32_t tm[4];
            split_pair(p0, p1, tm);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              if (j) pk[k] |= tm[k] << 16; else pk[k] = tm[k];
            }
          }
        };
        weights();

        // ---- the group's verdict
        if (!mbar_wait_bounded(smem_u32(&ctl->verdict[b]), (uint32_t)(n >> 1) & 1u)) { give_up(); dead = true; break; }
        if (*reinterpret_cast<volatile int*>(&ctl->raise[b]) != 0) {
          // rare: some row exceeds the reference by more than 2^8 (always so on the first tile of a run)
          float corr[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float mx = tl[i];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, d));
            if (lane == 0) ctl->xchg[wq][H0 + i] = mx;
          }
          if (!group_sync()) break;
          if (gi == 0) ctl->raise[b] = 0;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int h = H0 + i;
            const float mx = fmaxf(fmaxf(ctl->xchg[0][h], ctl->xchg[1][h]), fmaxf(ctl->xchg[2][h], ctl->xchg[3][h]));
            const float m_new = fmaxf(m_ref[i], mx);
            corr[i] = (m_ref[i] == -INFINITY) ? 0.f : ex2(m_ref[i] - m_new);   // m_new is finite or both are -inf
            if (m_new == -INFINITY) corr[i] = 1.f;
            m_ref[i] = m_new;
            l_run[i] *= corr[i];
          }
          if (t != seg.t) {
            // rescale this half's columns of the accumulator in tensor memory: every P.V issued so far (tile
            // n-1 was the last) is done
            if (!mbar_wait_bounded(smem_u32(&ctl->pv_done[(n - 1) & 1]), (uint32_t)((n - 1) >> 1) & 1u)) { give_up(); dead = true; break; }
            tc_fence_after();
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2) {   // the two 16-column halves (terms 1, 2 and terms 3, 4)
              uint32_t o[8];
              tmem_ld8(td + kO + 16 * c2 + 8 * hh, o);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr[i & 3]);
              tmem_st8(td + kO + 16 * c2 + 8 * hh, o);
            }
            tmem_wait_st();
            tc_fence_before();
          }
          if (!group_sync()) break;   // xchg / raise may be rewritten only after everyone has read them
          weights();       // again, against the raised reference
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) l_run[i] += l_add[i];

        // the P tile of two tiles ago must have been consumed
        if (!pv_ok && !mbar_wait_bounded(smem_u32(&ctl->pv_done[b]), ((uint32_t)(n >> 1) & 1u) ^ 1u)) { give_up(); dead = true; break; }
        if (tok >= seg.L) {
          // a key at or beyond L: its V codes may be anything (NaN codes included) and 0 * NaN is NaN; clear
          // the row (this thread's half of it; the swizzle permutes 16-byte pieces within a row)
          uint4* vr = reinterpret_cast<uint4*>(smem + g * GROUP_BYTES + (n % S) * STAGE + KV_TILE + row * 64 + 32 * hh);
          vr[0] = vr[1] = make_uint4(0, 0, 0, 0);
        }
        {
          // P row of a token: 16 bytes (terms 1, 2) and, 128 bytes on, 16 bytes (terms 3, 4); in each, byte
          // 8 * half + 4 * (term parity) + head % 4
          uint8_t* pt = smem + g * GROUP_BYTES + S * STAGE + b * P_BYTES + (row >> 3) * 256 + (row & 7) * 16 + 8 * hh;
          *reinterpret_cast<uint2*>(pt) = make_uint2(pk[0], pk[1]);
          *reinterpret_cast<uint2*>(pt + 128) = make_uint2(pk[2], pk[3]);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->p_full[b]));
        d1_ready = d1_next;
      }
      if (dead) break;

      // ---- end of the run: read O^T, finish the sums, store the partial
      if (!mbar_wait_bounded(smem_u32(&ctl->pv_done[(n - 1) & 1]), (uint32_t)((n - 1) >> 1) & 1u)) { give_up(); break; }
      tc_fence_after();
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float v = l_run[i];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(kFull, v, d);
        if (lane == 0) ctl->xchg[wq][H0 + i] = v;
      }
      if (!group_sync()) break;
      {
        uint32_t o0[8], o1[8];   // terms 1, 2 and terms 3, 4 of this half's heads
        tmem_ld8(td + kO + 8 * hh, o0);
        tmem_ld8(td + kO + 16 + 8 * hh, o1);
        tmem_wait_ld();
        tc_fence_before();
        const float vs = P.v_scale ? P.v_scale[seg.kvh] : 1.f;
        if (lane < 16) {   // this quadrant's 16 rows of O^T are dims 16*wq .. 16*wq + 15
          const int d = 16 * wq + lane;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int h = H0 + i;
            const float l_tot = ctl->xchg[0][h] + ctl->xchg[1][h] + ctl->xchg[2][h] + ctl->xchg[3][h];
            const float acc = __uint_as_float(o0[i]) + __uint_as_float(o0[4 + i]) * 0.0625f +
                              __uint_as_float(o1[i]) * (1.f / 256.f) + __uint_as_float(o1[4 + i]) * (1.f / 4096.f);
            const size_t prow = (size_t)seg.prow + (size_t)h * seg.pstride;
            P.part_o[prow * kHeadDim + d] = l_tot > 0.f ? acc * vs / l_tot : 0.f;
            if (d == 0) P.part_lse[prow] = l_tot > 0.f ? (m_ref[i] + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
          }
        }
      }
      __threadfence();
      if (!group_sync()) break;
      if (gi < 32) arrive_and_merge(P, seg.b, seg.kvh, cum, nW, lane);
    }
    // sequences without any visible key have no tile and hence no worker in the balanced schedule
    if (!dead && !C->abort && P.num_splits == 0 && gi < 32) {
      for (int p = w; p < P.batch * Hkv; p += nW) {
        const int b = p / Hkv;
        if (cum[b + 1] == cum[b]) merge_rows(P, b, p - b * Hkv, 0, 0, 0, 0, 0, 0, 0, lane);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 128;" ::"r"(tmem) : "memory");
  }
}

static size_t tc_smem_bytes(int batch) {
  return 1024 + (size_t)G * GROUP_BYTES + ((sizeof(CtaCtl) + 15) & ~(size_t)15) + (size_t)(2 * batch + 2) * sizeof(int);
}

cudaError_t launch_decode_attn_tc(const DecodeParams& P, int ctas, cudaStream_t s, int* smem_limit) {
  if (*smem_limit == 0) {
    int dev = 0, optin = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
    if (e != cudaSuccess) return e;
    *smem_limit = optin;
  }
  const size_t need = tc_smem_bytes(P.batch);
  if (need > (size_t)*smem_limit) return cudaErrorInvalidValue;
  decode_attn_tc_kernel<<<ctas, kThreads, need, s>>>(P);
  return cudaGetLastError();
}

int decode_attn_tc_workers_per_cta() { return G; }

}  // namespace puzzle
