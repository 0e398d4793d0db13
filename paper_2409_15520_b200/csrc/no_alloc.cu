// MP-LoRA linear for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need the layer:
// code running inside a framework whose allocator owns the whole device budget, plug-ins that
// are handed only their input and output buffers, or latency-critical loops where an
// allocation would synchronise the device.  For them the scratch that zo_mp_lora_linear
// normally receives from the caller lives here, in a fixed array in the library's device
// image.  Every GPU that loads the library carries these bytes until the process exits.
#include <mutex>

#include "../../include/zo.h"

namespace {

// Scratch of the no-allocation entry point (status word, down-projections U, base product).
static __device__ __align__(256) unsigned char g_static_scratch[ZO_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices];   // device address of the array, per device ordinal
std::mutex g_setup_mutex;

// The array's name is only a host-side handle; kernels need its device address, which differs
// per device.  Looked up once per device with that device current.
zo_status static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ZO_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ZO_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return ZO_OK;
}

}  // namespace

extern "C" zo_status zo_mp_lora_linear_static(void* cuda_stream, int32_t precision, const void* X,
                                              const void* W, const void* bias, const void* A,
                                              const float* B, void* Y, int32_t T, int32_t k_in,
                                              int32_t k_out, int32_t r, float scale, uint64_t seed,
                                              uint32_t tensor_id, int32_t q, float eps,
                                              int32_t x_replicated, uint32_t flags) {
  const size_t need = zo_mp_lora_scratch_bytes(precision, T, k_in, k_out, r, q, x_replicated);
  if (need == 0) return ZO_ERR_INVALID_ARG;
  if (need > (size_t)ZO_STATIC_SCRATCH_BYTES) return ZO_ERR_WORKSPACE;   // problem too large for the fixed array
  void* scratch = nullptr;
  const zo_status s = static_scratch(&scratch);
  if (s != ZO_OK) return s;
  // The status word at the head of the scratch is cleared by the call below; everything else
  // in the array is fully rewritten before it is read.
  return zo_mp_lora_linear(cuda_stream, precision, X, W, bias, A, B, Y, T, k_in, k_out, r, scale,
                           seed, tensor_id, q, eps, x_replicated, scratch,
                           (size_t)ZO_STATIC_SCRATCH_BYTES, flags);
}

// The status word of the last zo_mp_lora_linear_static call on the current device (it sits at the
// head of the fixed array, where the caller cannot read it).  One 4-byte copy on the given stream
// and a wait for that stream; nothing is allocated.
extern "C" zo_status zo_mp_lora_linear_static_status(void* cuda_stream, uint32_t* host_status) {
  if (!host_status) return ZO_ERR_INVALID_ARG;
  void* scratch = nullptr;
  const zo_status s = static_scratch(&scratch);
  if (s != ZO_OK) return s;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  uint32_t word = 0;
  if (cudaMemcpyAsync(&word, scratch, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return ZO_ERR_CUDA;
  *host_status = word;
  return (word & 1u) ? ZO_ERR_TIMEOUT : ZO_OK;   // bit 0: a bounded device-side wait ran out
}
