/*
 * puzzle_attn.h -- C ABI of the FP8-KV decode-attention library (sm_100a).
 *
 * One decode step of one attention layer of a gpt-oss-style grouped-query
 * model, as the paper's serving optimisations shape it:
 *
 *   - the KV cache is stored as FP8 (E4M3) with max-calibrated dequantisation
 *     scales (paper, Section "KV Quantization"); a bf16 cache is the comparison
 *     variant the paper measures against;
 *   - every layer is either full-context attention or window attention that
 *     sees only the most recent W tokens (paper, Section "Window attention for
 *     long-context inference"); which layers are which is the per-layer choice
 *     the architecture search makes (Section "Puzzle Optimization", "Blocks,
 *     subblocks, and search space");
 *   - decode is KV-cache-I/O bound (Section "Optimized Scenarios"), so the
 *     library streams every visible K/V byte exactly once per step.
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller, unless marked
 *     "host".  The two descriptor structs are read on the host during the call.
 *   - No device memory is allocated or freed by any call; what the library
 *     keeps between calls is host-side only (per device: its SM count, the
 *     shared-memory limit it has set on its kernels, the address of the
 *     built-in scratch array).  Work is enqueued on the CUDA stream passed as
 *     `stream` (a cudaStream_t cast to void*; NULL is the default stream) and
 *     the call returns without synchronising.  Stream order holds as usual: a
 *     kernel of the library reads or writes global memory only after all
 *     earlier work on its stream has completed (some are launched so that
 *     their thread blocks are placed, and set up shared memory, while the
 *     kernel before them drains; nothing else runs early).  The decode kernels
 *     in turn let a following kernel be placed early IF that kernel was
 *     launched with programmatic stream serialization; such a kernel must, as
 *     that attribute always requires, wait for its grid dependency before it
 *     reads what the library wrote.  Ordinary launches are unaffected.
 *   - The balanced schedule hands tiles of the cache to warps as they become
 *     free, so the order of the float32 sums can differ between two calls on the
 *     same inputs: outputs agree to rounding (the last bit of a bf16 value may
 *     differ), not bit for bit.  Appended cache bytes are always bit-exact.
 *   - Errors that the host can see (NULL required pointer, unsupported shape,
 *     workspace too small) return a code BEFORE anything is launched.  A CUDA
 *     launch error maps to PUZZLE_ERR_CUDA.  Errors only the device can see
 *     (a block-table entry outside [0, num_blocks), a sequence longer than its
 *     table row) set a bit in *dev_status, skip the access and never trap.
 *   - Shapes supported by this version: head_dim 64, block_size 16,
 *     num_q_heads == 8 * num_kv_heads, batch <= 4096.
 *
 * Cache layout (both K and V):  [num_blocks][num_kv_heads][block_size][head_dim]
 *   elements u8 (E4M3 codes) or bf16; one (block, KV head) is 1 KiB (FP8) or
 *   2 KiB (bf16) contiguous.  Base pointers must be 16-byte aligned.
 */
#ifndef PUZZLE_ATTN_H_
#define PUZZLE_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define PUZZLE_API __attribute__((visibility("default")))
#else
#define PUZZLE_API
#endif

typedef enum {
  PUZZLE_OK = 0,
  PUZZLE_ERR_NULL = 1,        /* a required pointer is NULL */
  PUZZLE_ERR_SHAPE = 2,       /* sizes inconsistent or out of range */
  PUZZLE_ERR_UNSUPPORTED = 3, /* valid but not built in this version */
  PUZZLE_ERR_WORKSPACE = 4,   /* workspace missing or too small */
  PUZZLE_ERR_CUDA = 5         /* a CUDA call or launch failed */
} puzzle_status;

typedef enum { PUZZLE_KV_FP8_E4M3 = 0, PUZZLE_KV_BF16 = 1 } puzzle_kv_dtype;

/* bits of *dev_status */
#define PUZZLE_DEV_BAD_BLOCK 1u  /* block-table entry outside [0, num_blocks) */
#define PUZZLE_DEV_SEQ_TOO_LONG 2u /* seq_len > max_blocks_per_seq * block_size (clamped) */
#define PUZZLE_DEV_WAIT_EXPIRED 4u /* a bounded wait on a copy ran out; results invalid */

/* One per layer: the layer's attention choice (host struct). */
typedef struct {
  int32_t num_q_heads;  /* 64 */
  int32_t num_kv_heads; /* 8; consecutive groups of 8 query heads share one KV head */
  int32_t head_dim;     /* 64 */
  int32_t block_size;   /* 16 tokens per cache block */
  int32_t window;       /* 0 = full context; W > 0 = the W most recent tokens, current one included */
  int32_t kv_dtype;     /* puzzle_kv_dtype */
  float sm_scale;       /* logit scale, 1/sqrt(head_dim) */
} puzzle_layer_desc;

/* One per layer: that layer's cache and how this batch maps onto it (host
 * struct holding device pointers). */
typedef struct {
  void* k_cache;              /* see "Cache layout" */
  void* v_cache;
  int64_t num_blocks;
  const int32_t* block_table; /* [batch][max_blocks_per_seq]; NULL = contiguous: block = b*max_blocks_per_seq + i.
                                 Entries for blocks that lie wholly outside the visible range are never read. */
  int32_t max_blocks_per_seq;
  const int32_t* seq_lens;    /* [batch], length AFTER this step's append; 0 is legal */
  const float* k_scale;       /* [num_kv_heads] dequantisation scales (x ~= code * scale); NULL = 1; FP8 only */
  const float* v_scale;
} puzzle_kv_view;

/* Max calibration of the per-head scales, step 1 (paper Section "KV Quantization": FP8 KV cache with
 * scales from max calibration).  Raises amax[h] to the largest |x| over every token and channel of KV
 * head h of this tensor: amax[h] = max(amax[h], max_{t,d} |x[t][h][d]|).  NaNs are skipped, infinities
 * count.  Call it once per chunk of calibration data; start from amax = 0.
 *   x: device, bf16 [n_tokens][num_kv_heads][head_dim], 16-byte aligned; head_dim a multiple of 8;
 *   amax: device, float32 [num_kv_heads], read and written (values must be >= 0);
 *   num_kv_heads <= 64.  n_tokens == 0 is legal and launches nothing.
 * Errors: PUZZLE_ERR_NULL, PUZZLE_ERR_SHAPE (sizes, alignment) before any launch. */
PUZZLE_API puzzle_status puzzle_kv_amax_update(const void* x, int64_t n_tokens, int32_t num_kv_heads,
                                 int32_t head_dim, float* amax, void* stream);

/* Max calibration, step 2: scale[h] = amax[h] / 448 as an IEEE float32 quotient (448 = largest E4M3
 * value), so that x / scale fills the E4M3 range; amax[h] == 0 gives scale 1.  pow2 != 0 rounds every
 * scale up to the next power of two (a power of two stays), as the paper does ("rounded the scales up
 * to a power of 2", same Section).  These are the dequantisation scales puzzle_kv_view carries
 * (x ~ code * scale).  amax and scale_out: device float32 [num_kv_heads]; they may be the same array. */
PUZZLE_API puzzle_status puzzle_kv_scales_from_amax(const float* amax, int32_t num_kv_heads, int32_t pow2,
                                 float* scale_out, void* stream);

/* Quantise-and-append of the new token's K and V (one token per sequence).
 * FP8: code = E4M3(round-to-nearest-even, saturating at +-448, of the float32
 * quotient x / scale[h]); NaN -> 0x7F.  bf16: the value is copied.  The token
 * lands at logical position seq_lens[b]-1 through the block table.  This is
 * the FP8 KV quantisation of Section "KV Quantization" applied at decode time.
 *   k_new, v_new: bf16 [batch][num_kv_heads][head_dim].
 *   dev_status: optional int32 device word, bits OR-ed in on device-side errors. */
PUZZLE_API puzzle_status puzzle_kv_append(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* k_new,
                               const void* v_new, int32_t batch, int32_t* dev_status, void* stream);

/* puzzle_kv_append for n_new tokens per sequence at once: a chunk of the prompt, or the tokens of a
 * multi-token decode step (the input half of the paper's fixed-length scenarios, Section "Optimized
 * Scenarios"; same quantisation, Section "KV Quantization").  Token i of sequence b lands at logical
 * position seq_lens[b] - new_lens[b] + i, seq_lens counted AFTER the append.
 *   k_new, v_new: device bf16 [batch][n_new][num_kv_heads][head_dim], 16-byte aligned;
 *   new_lens: device int32 [batch], tokens of each row that are real (clamped to [0, n_new]; the rest of
 *     the row is ignored), or NULL = n_new for every sequence.  Tokens that would land before position
 *     0 (new_lens[b] > seq_lens[b]) are skipped.
 * Errors and dev_status as puzzle_kv_append. */
PUZZLE_API puzzle_status puzzle_kv_append_tokens(const puzzle_layer_desc* desc, const puzzle_kv_view* kv,
                                 const void* k_new, const void* v_new, const int32_t* new_lens, int32_t batch,
                                 int32_t n_new, int32_t* dev_status, void* stream);

/* Values of num_splits below 1: the balanced schedule, with the kernel chosen by the library or pinned. */
#define PUZZLE_SCHED_AUTO 0
#define PUZZLE_SCHED_CTA (-1)
#define PUZZLE_SCHED_WARP (-2)

/* Bytes of scratch puzzle_decode_attn needs for this batch and split choice
 * (0 on invalid arguments).  num_splits <= 0 selects the balanced schedule.
 * The scratch serves the split-KV pass of the KV-I/O-bound decode (paper,
 * Section "Optimized Scenarios"): float32 partial (o, lse) rows, arrival
 * counters, and the speeds of the CTA slots noted by large launches (see
 * puzzle_decode_attn).  The paper does not describe a split-KV pass; the
 * partition and its merge follow the problem statement this library was built
 * to.  The size depends on the batch and the device's SM count, not on the
 * context length (the grid is persistent), so there is no max_seq_len argument. */
PUZZLE_API size_t puzzle_decode_attn_workspace_bytes(const puzzle_layer_desc* desc, int32_t batch, int32_t num_splits);

/* Prepares a freshly allocated workspace: zero-fills the CTA-speed words and
 * the arrival counters at its start on `stream`.  Call it once per workspace
 * before its first puzzle_decode_attn; every completed puzzle_decode_attn
 * leaves the counters at zero again.  The counter block has room for 16384
 * (sequence, KV head) pairs whatever `batch` is, and the partials start behind
 * it: a workspace prepared once serves calls of any batch with
 * batch * num_kv_heads <= 16384 and any split choice that fit it, one after
 * the other.  (A larger batch moves the partials: prepare the workspace for
 * that batch and use it for that batch only.)  Call it again after a step
 * whose *dev_status reported PUZZLE_DEV_WAIT_EXPIRED (that step stopped half
 * way).  The split-KV phase of Section "Optimized Scenarios"' KV-bound decode
 * needs these counters to know which worker finishes a (sequence, KV head). */
PUZZLE_API puzzle_status puzzle_decode_attn_workspace_init(const puzzle_layer_desc* desc, int32_t batch,
                                                           void* workspace, size_t workspace_bytes, void* stream);

/* Decode-step attention of one layer: for every sequence b and query head g
 * (KV head h = g / 8), over the visible keys j in [L - min(W, L), L) with
 * L = seq_lens[b] (all of [0, L) when window == 0):
 *     s_j = sm_scale * k_scale[h] * (q_g . Kcode_j),  M = max(max_j s_j, sink_g),
 *     Z = e^(sink_g - M) + sum_j e^(s_j - M),  out = v_scale[h] * sum_j e^(s_j - M) Vcode_j / Z.
 * Full vs window is the paper's per-layer choice (Section "Window attention for
 * long-context inference"); the sink is one extra softmax column per query head
 * that carries no value.  Internally ONE kernel: a split-KV pass writes float32
 * partial (o, lse) into the workspace, and the worker that completes a
 * (sequence, KV head) merges its partials by log-sum-exp and writes `out`.
 *   q: bf16 [batch][num_q_heads][head_dim], 8-byte aligned;  sinks: float32 [num_q_heads] or NULL (no sink);
 *   out: bf16 [batch][num_q_heads][head_dim], 16-byte aligned;  lse_out: float32 [batch][num_q_heads] or NULL;
 *   num_splits: 0 = balanced schedule (recommended); S >= 1 = every (sequence, KV head) context is
 *     cut into S equal runs of 64-token tiles.  The balanced schedule has three kernels and picks by
 *     what the host knows about the size of the launch (batch, window, block-table row length;
 *     puzzle_decode_attn_kernel_name tells which): large launches are cut into one range of tiles
 *     per CTA, handed out to its warps as they become free, in proportion to the speed each CTA
 *     showed in the previous large launch on this workspace; smaller ones, and mid-size ones made
 *     of many short contexts, are cut evenly over all warps, which has the shorter set-up; and
 *     when no (sequence, KV head) can have more than four tiles (narrow windows, very short
 *     contexts) nothing is cut: a group of four warps, or one warp when there are very many
 *     pairs, takes the pair whole and writes the output itself.  PUZZLE_SCHED_CTA and
 *     PUZZLE_SCHED_WARP pin the first or the second kernel (PUZZLE_SCHED_CTA needs batch <= 1024,
 *     else PUZZLE_ERR_UNSUPPORTED);
 *   workspace: device scratch of at least puzzle_decode_attn_workspace_bytes(...) bytes, 16-byte
 *     aligned, prepared once by puzzle_decode_attn_workspace_init; calls that share a workspace must
 *     not overlap on the GPU.  Besides partials and counters it keeps the CTA speeds between calls:
 *     they change how the next launch is cut, never its result beyond rounding;
 *   dev_status: optional int32 device word (see PUZZLE_DEV_*).
 * An empty context gives out = 0 and lse = sink (-inf without a sink). */
PUZZLE_API puzzle_status puzzle_decode_attn(const puzzle_layer_desc* desc, const puzzle_kv_view* kv, const void* q,
                                 const float* sinks, void* out, float* lse_out, int32_t batch,
                                 int32_t num_splits, void* workspace, size_t workspace_bytes,
                                 int32_t* dev_status, void* stream);

/* The same operation and contract as puzzle_decode_attn (same arguments, same workspace, same
 * results within the same tolerance), computed by a second kernel that feeds the E4M3 codes of the
 * cache straight to the 5th-generation tensor cores (tcgen05 MMA, accumulators in tensor memory):
 * S = K Q^T with the bf16 query split exactly into two E4M3 terms, O^T += V^T P with the softmax
 * weights split into four E4M3 terms.  FP8 caches only: a bf16 cache returns
 * PUZZLE_ERR_UNSUPPORTED and nothing is launched.  Tiles are 128 tokens (num_splits >= 1 cuts the
 * context into runs of 128-token tiles).  It is the slower of the two kernels on the workloads
 * measured so far and is kept as a validated alternative; puzzle_decode_attn is the default path.
 * (Paper: KV-cache I/O bounds decoding, Section "Optimized Scenarios"; FP8 KV cache, Section
 * "KV Quantization".) */
PUZZLE_API puzzle_status puzzle_decode_attn_tcgen05(const puzzle_layer_desc* desc, const puzzle_kv_view* kv,
                                 const void* q, const float* sinks, void* out, float* lse_out, int32_t batch,
                                 int32_t num_splits, void* workspace, size_t workspace_bytes,
                                 int32_t* dev_status, void* stream);

/* This device's share of a decode-step attention whose context is spread over several devices: the
 * same computation as puzzle_decode_attn over the keys THIS cache view holds, without any sink, with
 * the result left in float32 for a later merge:
 *   o_part[b][g][:] = sum_j e^(s_j - lse) v_j,  lse_part[b][g] = ln sum_j e^(s_j),  j over the visible keys
 * (zeros and -inf when the view holds no visible key).  Every device of a context-sharded layer calls
 * this on its slice of every sequence (seq_lens = tokens of the slice, its own block table), the
 * partials are exchanged (one all-gather of batch * Hq * (D + 1) floats per device), and
 * puzzle_attn_merge_strided applies the sink once.  (Paper: long-context decode is bound by KV-cache
 * I/O, Section "Optimized Scenarios"; serving sweeps tensor-parallel degree 1..8, paragraph "Inference
 * efficiency benchmarking"; the 8-GPU 64K/64K study, Section "B200 Inference Efficiency Case Study".
 * The paper does not describe context sharding itself.)
 *   o_part: device float32 [batch][Hq][D], 16-byte aligned; lse_part: device float32 [batch][Hq],
 *   required.  Other arguments, workspace and errors as puzzle_decode_attn.  A window counts back from
 *   the END of the slice, so a window layer is sharded only if the caller gives each device the window
 *   that remains on it (the same for every sequence), or keeps window layers on one device. */
PUZZLE_API puzzle_status puzzle_decode_attn_partial(const puzzle_layer_desc* desc, const puzzle_kv_view* kv,
                                 const void* q, float* o_part, float* lse_part, int32_t batch,
                                 int32_t num_splits, void* workspace, size_t workspace_bytes,
                                 int32_t* dev_status, void* stream);

/* One whole layer-step for a caller whose step inputs and result live in HOST memory: copies q, k_new and v_new to
 * the device, runs puzzle_kv_append and puzzle_decode_attn (the path of the paper's decode scenarios, Section
 * "Optimized Scenarios", with the FP8 append of Section "KV Quantization"), and copies the bf16 result back, all
 * enqueued on `stream`; the call returns without synchronising, so out_host is valid after the caller has
 * synchronised the stream.  The cache, block table, lengths, scales and sinks stay on the device as for the
 * other entry points.
 *   q_host: host bf16 [batch][num_q_heads][head_dim];  k_new_host, v_new_host: host bf16 [batch][num_kv_heads][head_dim];
 *   out_host: host bf16 [batch][num_q_heads][head_dim].  Pinned (page-locked) host memory keeps the copies
 *     asynchronous; pageable memory works but serialises with the host.  When k_new_host follows q_host and
 *     v_new_host follows k_new_host directly in memory (and the sizes are multiples of 256 bytes) the three travel
 *     as one copy;
 *   staging: device scratch of at least puzzle_decode_step_host_staging_bytes(desc, batch) bytes, 256-byte
 *     aligned, owned by the caller (the library allocates nothing); not to be shared by steps that overlap;
 *   num_splits, workspace, dev_status: as puzzle_decode_attn.
 * Host-visible errors are reported before the first copy is enqueued. */
PUZZLE_API size_t puzzle_decode_step_host_staging_bytes(const puzzle_layer_desc* desc, int32_t batch);
PUZZLE_API puzzle_status puzzle_decode_step_host(const puzzle_layer_desc* desc, const puzzle_kv_view* kv,
                                                 const void* q_host, const void* k_new_host, const void* v_new_host,
                                                 const float* sinks, void* out_host, int32_t batch, int32_t num_splits,
                                                 void* staging, size_t staging_bytes, void* workspace,
                                                 size_t workspace_bytes, int32_t* dev_status, void* stream);

/* Decode attention for up to n_q new tokens per sequence in one call: the tokens of a multi-token decode step, or
 * a chunk of a prompt after its bulk append (puzzle_kv_append_tokens), i.e. the input half of the paper's
 * fixed-length scenarios (Section "Optimized Scenarios"), on full and window layers (Section "Window attention for
 * long-context inference") over the FP8 cache (Section "KV Quantization").  Query token i of sequence b sits at
 * position p = seq_lens[b] - q_lens[b] + i (seq_lens counted AFTER the append of all q_lens[b] tokens) and is one
 * decode step of puzzle_decode_attn over the keys [p + 1 - min(W, p + 1), p] (all of [0, p] when window == 0): the
 * mask is causal.  Pairs of query tokens share one pass over the cache tiles, so two tokens cost little more than
 * one; the kernel is bound by KV bytes like the single-token one.
 *   q: bf16 [batch][n_q][num_q_heads][head_dim], 8-byte aligned;  q_lens: int32 [batch] real tokens per sequence
 *     (clamped to [0, n_q]), or NULL = n_q for all;  sinks as puzzle_decode_attn;
 *   out: bf16 [batch][n_q][num_q_heads][head_dim], 16-byte aligned: rows i < q_lens[b] are written, the others left
 *     as they are;  lse_out: float32 [batch][n_q][num_q_heads] or NULL;
 *   workspace: at least puzzle_decode_attn_tokens_workspace_bytes(desc, batch, n_q) bytes, 16-byte aligned,
 *     prepared once by puzzle_decode_attn_tokens_workspace_init (zero-fills its arrival counters; every completed
 *     call leaves them at zero); not to be shared with calls that overlap on the GPU;
 *   a token whose position would be negative (q_lens[b] > seq_lens[b]) sees no key: out = 0, lse = sink.
 * FP8 caches only (PUZZLE_ERR_UNSUPPORTED for bf16: give puzzle_decode_attn one batch row per query token instead);
 * batch * ceil(n_q / 2) <= 8192 (PUZZLE_ERR_SHAPE).  Errors and dev_status as puzzle_decode_attn. */
PUZZLE_API size_t puzzle_decode_attn_tokens_workspace_bytes(const puzzle_layer_desc* desc, int32_t batch, int32_t n_q);
PUZZLE_API puzzle_status puzzle_decode_attn_tokens_workspace_init(const puzzle_layer_desc* desc, int32_t batch,
                                                                  int32_t n_q, void* workspace, size_t workspace_bytes,
                                                                  void* stream);
PUZZLE_API puzzle_status puzzle_decode_attn_tokens(const puzzle_layer_desc* desc, const puzzle_kv_view* kv,
                                                   const void* q, const int32_t* q_lens, const float* sinks, void* out,
                                                   float* lse_out, int32_t batch, int32_t n_q, void* workspace,
                                                   size_t workspace_bytes, int32_t* dev_status, void* stream);

/* Size of the scratch array built into the library for puzzle_decode_attn_static. */
#define PUZZLE_STATIC_SCRATCH_BYTES (8u << 20)

/* puzzle_decode_attn without a workspace argument, for callers that cannot
 * allocate device memory where they call it: a server that gave all free HBM to
 * its KV-cache pool at start-up, code hosted inside another runtime whose
 * allocator it must not use, or a decode loop whose rules forbid cudaMalloc
 * because it stalls the whole device.  (The paper has no counterpart; this is a
 * deployment convenience.)  Results are those of puzzle_decode_attn, argument
 * for argument; inputs and outputs are still the caller's.
 *   - The scratch is a fixed PUZZLE_STATIC_SCRATCH_BYTES (8 MiB) array inside
 *     the library's device image; every GPU that loads the library holds it until
 *     the process exits.  A batch and split choice whose
 *     puzzle_decode_attn_workspace_bytes exceeds that size is refused with
 *     PUZZLE_ERR_WORKSPACE and nothing is launched (balanced schedule: batch up
 *     to about 280 on a 148-SM device; explicit splits: batch * num_splits up to
 *     about 500).
 *   - The call allocates and frees nothing.  The first call on each device looks
 *     up the array's device address (with that device current).  Make that first
 *     call at start-up: before any stream capture, and before the caller hands
 *     out the device's remaining memory, because the driver reserves the
 *     array's 8 MiB when it loads the library's device image, which can be as
 *     late as this first call.  From the second call on, free device memory
 *     does not change.
 *   - Argument errors are reported before anything is enqueued, as for every
 *     entry point: an invalid call neither clears nor touches the array.
 *   - All calls on a device share the one array.  Two calls that overlap on the
 *     GPU (different streams, no dependency between them) race on it and both
 *     results are undefined; order them.  The array keeps the previous call's
 *     contents; the part that must start at zero is cleared on `stream` by every
 *     call before its kernel. */
PUZZLE_API puzzle_status puzzle_decode_attn_static(const puzzle_layer_desc* desc, const puzzle_kv_view* kv,
                                                   const void* q, const float* sinks, void* out, float* lse_out,
                                                   int32_t batch, int32_t num_splits, int32_t* dev_status,
                                                   void* stream);

/* Log-sum-exp merge of partial attention results that came from elsewhere
 * (e.g. context shards on other GPUs; puzzle_decode_attn merges its own
 * partials itself).  It is the second half of the split-KV pass of the
 * KV-I/O-bound decode (paper, Section "Optimized Scenarios"); the paper does not
 * define the merge: the formula is the exact recombination of softmax partials,
 * with the per-head sink logit counted once.  For every row r = (b, g):
 *     M = max(sink_g, max_p lse_p),  Z = e^(sink_g - M) + sum_p e^(lse_p - M),
 *     out = sum_p e^(lse_p - M) o_p / Z,  lse_out = M + ln Z.
 *   part_o: float32 [batch][Hq][S][D];  part_lse: float32 [batch][Hq][S] (natural log; -inf = empty part);
 *   num_parts: int32 [batch] or NULL (= S for all);  sinks: float32 [Hq] or NULL;
 *   out: bf16 [batch][Hq][D];  lse_out: float32 [batch][Hq] or NULL.  D must be a multiple of 64, <= 512. */
PUZZLE_API puzzle_status puzzle_attn_merge(const float* part_o, const float* part_lse, const int32_t* num_parts,
                                const float* sinks, void* out, float* lse_out, int32_t batch, int32_t Hq,
                                int32_t D, int32_t S, void* stream);

/* puzzle_attn_merge (same passage, same formula) over partials laid out with strides (in floats), for the
 * exchange step of a context-sharded layer (serving over 1..8 GPUs: paper, paragraph "Inference efficiency
 * benchmarking"): part k of row r = b * Hq + g has
 * its D outputs at part_o + r * o_row_stride + k * o_part_stride and its lse at
 * part_lse[r * lse_row_stride + k * lse_part_stride].  An all-gather of per-device buffers
 * {o [batch][Hq][D], lse [batch][Hq]} is merged in place with o_row_stride = D,
 * o_part_stride = lse_part_stride = batch * Hq * (D + 1), lse_row_stride = 1 and
 * part_lse = part_o + batch * Hq * D.  o_row_stride and o_part_stride must be even, no stride negative
 * (PUZZLE_ERR_SHAPE).  Everything else as puzzle_attn_merge, which is this call with the strides of
 * a [batch][Hq][S][D] array. */
PUZZLE_API puzzle_status puzzle_attn_merge_strided(const float* part_o, const float* part_lse, int64_t o_row_stride,
                                 int64_t o_part_stride, int64_t lse_row_stride, int64_t lse_part_stride,
                                 const int32_t* num_parts, const float* sinks, void* out, float* lse_out,
                                 int32_t batch, int32_t Hq, int32_t D, int32_t S, void* stream);

/* Read-only streaming pass over `bytes` bytes at `buf` (16-byte aligned,
 * bytes a multiple of 16): the XOR of all words is written to *sink (device,
 * 8 bytes).  Not part of the method; it measures the read bandwidth the
 * attention kernel is bounded by on the device it runs on. */
PUZZLE_API puzzle_status puzzle_hbm_read_probe(const void* buf, size_t bytes, uint64_t* sink, void* stream);

/* Static description of a status code (host string, never NULL). */
PUZZLE_API const char* puzzle_status_string(puzzle_status s);

/* Which of the library's kernels puzzle_decode_attn would launch for these
 * arguments ("decode_attn_cta_kernel", "decode_attn_kernel",
 * "decode_attn_small_kernel"; host string, never NULL; "invalid arguments" when
 * the call would be refused).  The choice follows from desc, the batch, the
 * width of a block-table row and num_splits alone, so nothing is launched or
 * read on the device.  For logs and benchmarks that name what they time; the
 * paper has no counterpart (it does not describe kernels). */
PUZZLE_API const char* puzzle_decode_attn_kernel_name(const puzzle_layer_desc* desc, const puzzle_kv_view* kv,
                                                      int32_t batch, int32_t num_splits);

/* Number of kernels this library has launched from this process so far. */
PUZZLE_API int64_t puzzle_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PUZZLE_ATTN_H_ */
