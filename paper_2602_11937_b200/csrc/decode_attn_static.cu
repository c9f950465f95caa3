// puzzle_decode_attn_static: decode attention for callers that have no device memory to give.
//
// Some hosts of this library cannot allocate on the GPU at the point where they call it: a serving
// process that handed every free byte of HBM to its KV-cache pool at start-up, a plug-in that runs
// inside another runtime whose allocator it may not touch, a latency-critical loop whose rules forbid
// cudaMalloc because it synchronises the device.  For them the scratch that puzzle_decode_attn takes as
// `workspace` lives here, in a fixed array in the library's own device image.
#include <mutex>

#include "common.cuh"
#include "decode_attn.cuh"

namespace puzzle {
namespace {

constexpr size_t kStaticScratchBytes = PUZZLE_STATIC_SCRATCH_BYTES;

// One array per device that loads the library, held until the process exits.  In host code this name is
// only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the array on the current device, looked up once per device.
puzzle_status scratch_address(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PUZZLE_ERR_CUDA;
  std::lock_guard<std::mutex> hold(g_setup_lock);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return PUZZLE_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return PUZZLE_OK;
}

}  // namespace
}  // namespace puzzle

extern "C" puzzle_status puzzle_decode_attn_static(const puzzle_layer_desc* desc, const puzzle_kv_view* kv,
                                                   const void* q, const float* sinks, void* out, float* lse_out,
                                                   int32_t batch, int32_t num_splits, int32_t* dev_status,
                                                   void* stream) {
  using namespace puzzle;
  // argument errors first: an invalid call must not put the counter clear on the stream (it could zero the
  // counters under a call that is still running on another stream)
  puzzle_status st = check_decode_attn_args(desc, kv, q, out, batch, num_splits, false);
  if (st != PUZZLE_OK) return st;
  const size_t need = puzzle_decode_attn_workspace_bytes(desc, batch, num_splits);
  if (need == 0) return PUZZLE_ERR_SHAPE;
  if (need > kStaticScratchBytes) return PUZZLE_ERR_WORKSPACE;
  void* scratch = nullptr;
  st = scratch_address(&scratch);
  if (st != PUZZLE_OK) return st;
  // The array keeps whatever the previous call left.  Only the arrival counters must start at zero; a call
  // that ran to its end leaves them so, but one that was cut short does not, so they are cleared every time.
  st = puzzle_decode_attn_workspace_init(desc, batch, scratch, kStaticScratchBytes, stream);
  if (st != PUZZLE_OK) return st;
  return puzzle_decode_attn(desc, kv, q, sinks, out, lse_out, batch, num_splits, scratch, kStaticScratchBytes,
                            dev_status, stream);
}
