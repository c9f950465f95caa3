// Shared device helpers of the decode-attention library: thin wrappers over the
// sm_100a PTX the kernels use (mbarrier, tiled TMA loads, ldmatrix, FP8
// conversions).  Header-only; no state.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/puzzle_attn.h"

namespace puzzle {

constexpr int kGroup = 8;     // query heads per KV head
constexpr int kHeadDim = 64;
constexpr int kBlock = 16;    // tokens per cache block
constexpr int kWarps = 8;     // warps per CTA of the merge kernel (one output row each)
constexpr int kMaxBatch = 4096;

void count_launch();

// --------------------------------------------- programmatic dependent launch --
// The append kernels and the mma.sync decode kernels are launched so that their CTAs may be placed on an SM as soon as
// the kernel before them on the stream lets go of it, instead of after that whole grid has drained and a launch
// latency on top.  A kernel launched this way calls grid_dependency_wait() before its first access to global memory:
// it returns once every earlier kernel on the stream has completed and its writes are visible, so nothing the caller
// (or an earlier call) produced is read early; all that runs ahead of it is the placement of the CTA and set-up that
// touches shared memory and kernel parameters only.  release_dependents() at the top of a decode kernel tells the
// kernel behind it (if it was launched this way) that its CTAs may be placed whenever there is room; a kernel that
// never calls it releases them when its last CTA exits.  Both are no-ops next to a kernel launched the ordinary way.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------- mbarrier --
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: returns false if the phase did not complete within the limit
// (each failed try_wait already suspends the thread for a hardware time slice).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 64) __nanosleep(64);
  }
  return false;
}

// True in exactly one lane of a converged warp (all 32 lanes must call it).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ------------------------------------------------------------- TMA (tiled) --
// 2-D tiled load global -> shared, completion counted in bytes on an mbarrier.
// crd0 (innermost, bytes for u8 maps) must keep crd0 * element size a multiple of 16.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, int crd0, int crd1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(crd0), "r"(crd1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}

// ---------------------------------------------------------------- ldmatrix --
// Four 8x8 matrices of 16-bit cells (= 8 rows x 16 bytes each); lanes 8m..8m+7
// give the row addresses of matrix m; lane l receives row l/4, bytes 4(l%4)..+3.
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// Two 16x16 byte matrices, transposed on the way in; lanes 0-15 give the rows
// of matrix 0, lanes 16-31 of matrix 1.  Lane l receives, per matrix, two
// registers: byte e of the first = mem[row 4(l%4)+e][byte l/4], of the second
// = mem[row 4(l%4)+e][byte l/4 + 8].
__device__ __forceinline__ void ldsm_x2_trans_b8(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                 uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m16n16.x2.trans.shared.b8 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// Four 8x8 b16 matrices, transposed (bf16 V tiles).
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                              uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

// ------------------------------------------------------------ conversions --
// Two floats -> two E4M3 codes (round to nearest even, saturate to +-448);
// the low byte holds `lo`, the high byte `hi`.
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t f32x2_to_f16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// ------------------------------------------------- tile schedule (shared) ---
// Visible key range of a sequence and the tiles (of `tile` tokens) that cover it.
struct SeqRange {
  int L;     // clamped length
  int lo;    // first visible key
  int tlo;   // first tile
  int ntile; // tiles covering [lo, L)
};
__device__ __forceinline__ SeqRange seq_range(int len, int window, int max_tokens, int tile, bool& too_long) {
  SeqRange r;
  too_long = len > max_tokens;
  r.L = len < 0 ? 0 : (len > max_tokens ? max_tokens : len);
  r.lo = (window > 0 && r.L > window) ? r.L - window : 0;
  r.tlo = r.lo / tile;
  r.ntile = r.L > 0 ? (r.L + tile - 1) / tile - r.tlo : 0;
  return r;
}

// Fills cum[0..batch] (exclusive prefix of ntile * Hkv) and lens[0..batch) in
// shared memory; every thread of the CTA must call it.  Ends with a CTA barrier.
__device__ __forceinline__ void build_schedule(int* cum, int* lens, const int32_t* seq_lens, int batch, int Hkv,
                                               int window, int max_tokens, int tile, int32_t* dev_status) {
  for (int b = threadIdx.x; b < batch; b += blockDim.x) {
    bool too_long;
    SeqRange r = seq_range(seq_lens[b], window, max_tokens, tile, too_long);
    if (too_long && dev_status && blockIdx.x == 0) atomicOr(dev_status, (int)PUZZLE_DEV_SEQ_TOO_LONG);
    lens[b] = r.L;
    cum[b + 1] = r.ntile * Hkv;
  }
  if (threadIdx.x == 0) cum[0] = 0;
  __syncthreads();
  if (threadIdx.x < 32) {
    int carry = 0;
    for (int base = 0; base < batch; base += 32) {
      int i = base + threadIdx.x;
      int v = i < batch ? cum[i + 1] : 0;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        int u = __shfl_up_sync(0xffffffffu, v, d);
        if ((int)threadIdx.x >= d) v += u;
      }
      if (i < batch) cum[i + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();
}

}  // namespace puzzle
