// Measurement helpers (no counterpart in the paper): what a launch costs and how fast memory can be read on this GPU,
// measured with kernels of this library in the same way as the layer itself, so that the layer's timings can be
// set against them.
#include "kmq_common.cuh"

namespace kmq {
namespace {

// The fixed cost of one call: a kernel that does nothing, launched like the layer's kernels (programmatic
// dependent launch: wait for the previous kernel, release the next).
__global__ void probe_launch_kernel() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
}

// Read-only streaming: every thread folds 128-bit loads (no L1 allocation, as the layer reads its packed indices)
// into one word; the CTAs walk the buffer side by side, 8 loads in flight per thread.
__global__ void __launch_bounds__(256) probe_read_kernel(const uint4* __restrict__ buf, size_t n16,
                                                         uint32_t* __restrict__ out) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t acc = 0;
  for (; i + 7 * stride < n16; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = ldg_stream_u4(buf + i + u * stride);
#pragma unroll
    for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  for (; i < n16; i += stride) {
    const uint4 v = ldg_stream_u4(buf + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
  out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

}  // namespace
}  // namespace kmq

using namespace kmq;

extern "C" kmq_status kmq_probe_launch(void* stream) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1);
  cfg.blockDim = dim3(32);
  cfg.stream = (cudaStream_t)stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, probe_launch_kernel) == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

extern "C" size_t kmq_probe_read_out_bytes(void) {
  const DeviceInfo* di = device_info();
  return di ? (size_t)di->sm_count * 8 * 256 * sizeof(uint32_t) : 0;
}

extern "C" kmq_status kmq_probe_read(const void* buf, size_t bytes, void* out, void* stream) {
  if (!buf || !out) return KMQ_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(buf) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u)) return KMQ_ERR_ALIGN;
  const DeviceInfo* di = device_info();
  if (!di) return KMQ_ERR_CUDA;
  probe_read_kernel<<<di->sm_count * 8, 256, 0, (cudaStream_t)stream>>>(static_cast<const uint4*>(buf), bytes / 16,
                                                                         static_cast<uint32_t*>(out));
  return cudaGetLastError() == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}
