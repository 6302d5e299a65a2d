// kmq_linear_static_scratch: kmq_linear for callers that cannot hand over a scratch buffer.
//
// Some shapes of kmq_linear (long rows, more 16-row tiles than the GPU keeps resident) run the balanced kernel pair,
// which parks partial sums in global scratch memory between its two launches.  kmq_linear takes that scratch from the
// caller, who normally gets it from cudaMalloc or a framework allocator.  A caller that must not allocate -- code
// running inside a region where the allocator is locked or allocation is forbidden (a real-time control loop, a
// callback that may not block, a plug-in that was handed only its input and output buffers, a process whose memory
// was budgeted up front) -- can use this entry point instead: the scratch lives in a fixed array inside the library
// image, so nothing is allocated here, now or later.
#include <mutex>

#include "kmq_common.cuh"

namespace {

// The scratch itself: part of the library's device image, present on every GPU that loads the library until the
// process exits.  512 KiB covers the balanced kernel pair on GPUs with up to 160 SMs (3 * SMs * 1088 bytes).
constexpr size_t kStaticScratchBytes = 512u * 1024u;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel may use; the device
// address has to be asked for, once per device, with that device current.
void* static_scratch_address(cudaError_t* err) {
  constexpr int kMaxDevices = 64;
  static void* addr[kMaxDevices] = {};
  static std::mutex mu;
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= kMaxDevices) {
    *err = cudaErrorInvalidDevice;
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    void* p = nullptr;
    *err = cudaGetSymbolAddress(&p, g_static_scratch);
    if (*err != cudaSuccess) return nullptr;
    addr[dev] = p;
  }
  return addr[dev];
}

}  // namespace

extern "C" kmq_status kmq_linear_static_scratch(const uint32_t* packed, const uint16_t* codebooks, const uint16_t* x,
                                                uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, int layout,
                                                void* stream) {
  // 0 both for shapes that need no scratch and for invalid arguments: kmq_linear sorts those out
  const size_t need = kmq_workspace_bytes(N, K, bits, M, layout);
  if (need == 0) return kmq_linear(packed, codebooks, x, y, N, K, bits, M, layout, nullptr, 0, stream);
  if (need > kStaticScratchBytes) return KMQ_ERR_SCRATCH_LIMIT;
  cudaError_t err = cudaSuccess;
  void* scratch = static_scratch_address(&err);
  if (!scratch) return KMQ_ERR_CUDA;
  // Nothing in the scratch has to start at zero: the first launch writes every slot the second one reads.
  return kmq_linear(packed, codebooks, x, y, N, K, bits, M, layout, scratch, kStaticScratchBytes, stream);
}

extern "C" size_t kmq_static_scratch_capacity(void) { return kStaticScratchBytes; }
