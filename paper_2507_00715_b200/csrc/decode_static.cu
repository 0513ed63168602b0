// earn_decode_attn_static: the decode step for callers that may not allocate device memory.
//
// Some hosts give a plug-in its input and output buffers and nothing else: an inference server whose
// memory pool belongs to the framework around it, or a latency-critical loop that cannot afford the
// device-wide synchronisation (and the possible out-of-memory failure) of cudaMalloc.  Such a caller
// cannot provide the workspace earn_decode_attn asks for.  This entry point carries its own: a
// fixed-size array in device memory that is part of the library image.  Every GPU that loads the
// library holds these EARN_STATIC_SCRATCH_BYTES until the process exits, whether the call is used or not.
//
// The array's name is only a host-side handle; the device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and handed to the ordinary decode path as its
// workspace.  Nothing here calls cudaMalloc, cudaFree or any allocating library routine.
#include <mutex>

#include "earn_common.cuh"

namespace earn {
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[EARN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device; resolved on the first call per device.
cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (p == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace earn

extern "C" earn_status_t earn_decode_attn_static(const earn_model_t* model, const earn_batch_t* batch, int32_t layer,
                                                 int32_t step, const void* q, const void* k_new, const void* v_new,
                                                 const void* k_full_or_null, const void* v_full_or_null,
                                                 const earn_cache_t* cache, void* o, earn_stream_t stream) {
  using namespace earn;
  // The ordinary decode call's argument checks come first: a bad model or batch must be turned away on the host
  // before its fields are used to size anything, and a rejected call must not have enqueued the clearing below.
  bool nothing_to_do = false;
  const earn_status_t checked = validate_decode(model, batch, layer, step, q, k_new, v_new, k_full_or_null,
                                                v_full_or_null, cache, o, &nothing_to_do);
  if (checked != EARN_OK || nothing_to_do) return checked;
  // the same layout earn_decode_attn expects from a caller's workspace: status block, split tickets, split partials
  const size_t need = earn_workspace_bytes(model, batch, cache->beams);
  if (need > (size_t)EARN_STATIC_SCRATCH_BYTES) return EARN_ERR_WORKSPACE;   // this batch needs more than the built-in scratch
  void* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return EARN_ERR_CUDA;
  // The array keeps whatever the previous call left.  The status block and the tickets must read zero when the
  // kernel starts; the partials behind them are always written before they are read.
  size_t head = workspace_head_bytes(*model, *batch, cache->beams);
  if (head > need) head = need;
  if (cudaMemsetAsync(scratch, 0, head, (cudaStream_t)stream) != cudaSuccess) return EARN_ERR_CUDA;
  return earn_decode_attn(model, batch, layer, step, q, k_new, v_new, k_full_or_null, v_full_or_null, cache, o, scratch,
                          (size_t)EARN_STATIC_SCRATCH_BYTES, stream);
}
