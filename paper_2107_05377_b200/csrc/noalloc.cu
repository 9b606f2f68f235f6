// Pooler + head for callers that cannot allocate device memory.
//
// mt_kernel_pooler_head needs a caller-provided scratch buffer (the tanh pooler features travel
// through it from the pooler launch to the head launch).  Some callers have nowhere to get one:
// code running inside a serving process whose device memory was handed out in full at start-up,
// plug-ins that are only given input and output pointers by their host, or code on a path where
// cudaMalloc is off limits because it synchronises the whole device.  For them this file keeps the
// scratch in a fixed array that lives in the library's device image, so the entry point below
// needs nothing but inputs and outputs.

#include <cstring>
#include <mutex>

#include "../../include/mt_bert.h"
#include "mt_kernels.h"

namespace {

// MT_STATIC_POOLER_MAX_FLOATS floats = 1 MiB, resident on every GPU that loads the library until
// the process exits.
static __device__ __align__(256) float g_pooled_scratch[MT_STATIC_POOLER_MAX_FLOATS];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float* g_scratch_address[kMaxDevices] = {};  // device address of the array, per device ordinal

// In host code `g_pooled_scratch` is only a handle for the runtime, not an address a kernel can use;
// the device address has to be asked for, once per device, with that device current.
cudaError_t scratch_for_current_device(float** out) {
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_address[dev] == nullptr) {
    float* ptr = nullptr;
    err = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_pooled_scratch);
    if (err != cudaSuccess) return err;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_address[dev] = ptr;
  }
  *out = g_scratch_address[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int mt_kernel_pooler_head_static(const void* d_hidden, const void* d_pool_w, const void* d_pool_b,
                                            const void* d_cls_w, const void* d_cls_b, float* d_logits, int32_t batch,
                                            int32_t seq, int32_t hidden, int32_t num_classes, int32_t logits_stride,
                                            int32_t col0, void* stream) {
  if (d_hidden == nullptr || d_pool_w == nullptr || d_pool_b == nullptr || d_cls_w == nullptr || d_cls_b == nullptr ||
      d_logits == nullptr || batch < 1 || seq < 1 || num_classes < 1 || col0 < 0 || logits_stride < col0 + num_classes)
    return MT_ERR_INVALID_ARG;
  if (hidden != 768 && hidden != 1024) return MT_ERR_UNSUPPORTED;
  // the built-in scratch holds batch * hidden floats at most
  if (static_cast<int64_t>(batch) * hidden > static_cast<int64_t>(MT_STATIC_POOLER_MAX_FLOATS)) return MT_ERR_SHAPE;
  float* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) return MT_ERR_CUDA;
  mt::HeadParams p;
  memset(&p, 0, sizeof(p));
  p.task[0] = {static_cast<const mt::bf16*>(d_hidden), static_cast<const mt::bf16*>(d_pool_w),
               static_cast<const mt::bf16*>(d_pool_b), static_cast<const mt::bf16*>(d_cls_w),
               static_cast<const mt::bf16*>(d_cls_b), num_classes, col0};
  p.logits = d_logits;
  // Every feature the head launch reads (rows < batch) is written by the pooler launch first, so
  // nothing left over from an earlier call needs clearing.
  p.pooled = scratch;
  p.n_tasks = 1; p.batch = batch; p.seq = seq; p.hidden = hidden; p.logits_stride = logits_stride;
  return mt::launch_pooler_head(p, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}
