// extern "C" boundary of libkmq: argument validation and dispatch.
#include <mutex>

#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"
#include "kmq_table_layout.cuh"

namespace kmq {

const DeviceInfo* device_info() {
  constexpr int kMaxDevices = 64;
  static DeviceInfo cache[kMaxDevices];
  static bool valid[kMaxDevices] = {};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!valid[dev]) {
    int sms = 0, smem = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return nullptr;
    cache[dev].sm_count = sms;
    cache[dev].max_smem_optin = smem;
    valid[dev] = true;
  }
  return &cache[dev];
}

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool known_layout(int layout) {
  return layout == KMQ_LAYOUT_CANONICAL || layout == KMQ_LAYOUT_TUNED || layout == KMQ_LAYOUT_TABLE;
}
// b = 4 is stored identically in the tuned and the table layout
inline bool is_plane_layout(int layout, int bits) { return layout == KMQ_LAYOUT_TABLE && bits != 4; }

kmq_status check_shape(int64_t N, int64_t K, int bits, int64_t M) {
  if (bits != 1 && bits != 2 && bits != 4) return KMQ_ERR_BITS;
  const int64_t per = 32 / bits;
  if (N < 1 || M < 1 || K < per || (K % per) != 0) return KMQ_ERR_SHAPE;
  // keep every element count and byte offset inside int64 with room to spare
  if (N > (int64_t(1) << 31) || K > (int64_t(1) << 31) || M > (int64_t(1) << 24)) return KMQ_ERR_SHAPE;
  return KMQ_OK;
}

}  // namespace
}  // namespace kmq

using namespace kmq;

extern "C" {

int kmq_version(void) { return 100; }

const char* kmq_status_string(int status) {
  switch (status) {
    case KMQ_OK: return "ok";
    case KMQ_ERR_NULL: return "a required pointer is NULL";
    case KMQ_ERR_BITS: return "bits must be 1, 2 or 4";
    case KMQ_ERR_SHAPE: return "invalid shape (N, M >= 1; K a positive multiple of 32/bits)";
    case KMQ_ERR_ALIGN: return "device pointers must be 16-byte aligned";
    case KMQ_ERR_WORKSPACE: return "workspace missing or too small";
    case KMQ_ERR_LAYOUT: return "unknown packed layout";
    case KMQ_ERR_CUDA: return "CUDA runtime error";
    case KMQ_ERR_SCRATCH_LIMIT: return "the shape needs more scratch than the built-in static buffer holds";
    default: return "unknown status";
  }
}

size_t kmq_packed_bytes(int64_t N, int64_t K, int bits, int layout) {
  if (!known_layout(layout) || check_shape(N, K, bits, 1) != KMQ_OK) return 0;
  const int64_t wpr = K / (32 / bits);
  if (is_plane_layout(layout, bits)) return (size_t)table_total_bytes(N, K, bits);
  if (layout != KMQ_LAYOUT_CANONICAL) return (size_t)tuned_total_words(N, wpr) * 4u;
  return (size_t)N * (size_t)wpr * 4u;
}

int64_t kmq_packed_word_index(int64_t n, int64_t j, int64_t N, int64_t K, int bits, int layout) {
  if (!known_layout(layout) || check_shape(N, K, bits, 1) != KMQ_OK) return -1;
  const int64_t wpr = K / (32 / bits);
  if (n < 0 || n >= N || j < 0 || j >= wpr || is_plane_layout(layout, bits)) return -1;
  return layout != KMQ_LAYOUT_CANONICAL ? tuned_word_index(n, j, tuned_steps(wpr)) : n * wpr + j;
}

int kmq_packed_field_shift(int i, int bits, int layout) {
  if (!known_layout(layout) || (bits != 1 && bits != 2 && bits != 4) || i < 0 || i >= 32 / bits) return -1;
  if (is_plane_layout(layout, bits)) return -1;
  const bool tuned = layout != KMQ_LAYOUT_CANONICAL;
  return bits == 1 ? field_pos<1>(i, tuned) : bits == 2 ? field_pos<2>(i, tuned) : field_pos<4>(i, tuned);
}

int64_t kmq_packed_bit_index(int64_t n, int64_t k, int plane, int64_t N, int64_t K, int bits, int layout) {
  if (!known_layout(layout) || check_shape(N, K, bits, 1) != KMQ_OK) return -1;
  if (n < 0 || n >= N || k < 0 || k >= K || plane < 0 || plane >= bits) return -1;
  if (is_plane_layout(layout, bits))
    return table_byte_offset(n, k >> 3, plane, table_chunks(K), bits) * 8 + (k & 7);
  const int64_t per = 32 / bits, wpr = K / per;
  const int64_t word = layout != KMQ_LAYOUT_CANONICAL ? tuned_word_index(n, k / per, tuned_steps(wpr)) : n * wpr + k / per;
  return word * 32 + kmq_packed_field_shift((int)(k % per), bits, layout) + plane;
}

size_t kmq_workspace_bytes(int64_t N, int64_t K, int bits, int64_t M, int layout) {
  if (!known_layout(layout) || check_shape(N, K, bits, M) != KMQ_OK) return 0;
  return plan_linear(N, K, bits, M, layout).workspace;
}

int kmq_linear_num_launches(int64_t N, int64_t K, int bits, int64_t M, int layout) {
  if (!known_layout(layout) || check_shape(N, K, bits, M) != KMQ_OK) return 0;
  return plan_linear(N, K, bits, M, layout).launches;
}

int kmq_preferred_layout(int64_t N, int64_t K, int bits, int64_t M) {
  if (check_shape(N, K, bits, M) != KMQ_OK) return KMQ_LAYOUT_TUNED;
  return linear_lut_preferred(N, K, bits, M) ? KMQ_LAYOUT_TABLE : KMQ_LAYOUT_TUNED;
}

const char* kmq_linear_variant(int64_t N, int64_t K, int bits, int64_t M, int layout) {
  if (!known_layout(layout) || check_shape(N, K, bits, M) != KMQ_OK) return "invalid";
  return plan_linear(N, K, bits, M, layout).name;
}

kmq_status kmq_pack(const uint8_t* idx, int64_t N, int64_t K, int bits, int layout, uint32_t* packed, void* stream) {
  if (!idx || !packed) return KMQ_ERR_NULL;
  if (kmq_status s = check_shape(N, K, bits, 1)) return s;
  if (!known_layout(layout)) return KMQ_ERR_LAYOUT;
  if (!aligned16(idx) || !aligned16(packed)) return KMQ_ERR_ALIGN;
  return launch_pack(idx, N, K, bits, layout, packed, (cudaStream_t)stream) == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

kmq_status kmq_unpack(const uint32_t* packed, int64_t N, int64_t K, int bits, int layout, uint8_t* idx, void* stream) {
  if (!idx || !packed) return KMQ_ERR_NULL;
  if (kmq_status s = check_shape(N, K, bits, 1)) return s;
  if (!known_layout(layout)) return KMQ_ERR_LAYOUT;
  if (!aligned16(idx) || !aligned16(packed)) return KMQ_ERR_ALIGN;
  return launch_unpack(packed, N, K, bits, layout, idx, (cudaStream_t)stream) == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

namespace {

// Every check of kmq_linear that needs no GPU work; on success `plan` is the kernel variant to launch.
kmq_status check_linear_args(const uint32_t* packed, const uint16_t* codebooks, const uint16_t* x, const uint16_t* y,
                             int64_t N, int64_t K, int bits, int64_t M, int layout, const void* workspace,
                             size_t workspace_bytes, LinearPlan* plan) {
  if (!packed || !codebooks || !x || !y) return KMQ_ERR_NULL;
  if (kmq_status s = check_shape(N, K, bits, M)) return s;
  if (!known_layout(layout)) return KMQ_ERR_LAYOUT;
  if (!aligned16(packed) || !aligned16(codebooks) || !aligned16(x) || !aligned16(y)) return KMQ_ERR_ALIGN;
  if (!device_info()) return KMQ_ERR_CUDA;
  *plan = plan_linear(N, K, bits, M, layout);
  if (plan->workspace > 0) {
    if (!workspace || workspace_bytes < plan->workspace) return KMQ_ERR_WORKSPACE;
    if (!aligned16(workspace)) return KMQ_ERR_ALIGN;
  }
  return KMQ_OK;
}

}  // namespace

kmq_status kmq_linear(const uint32_t* packed, const uint16_t* codebooks, const uint16_t* x, uint16_t* y, int64_t N,
                      int64_t K, int bits, int64_t M, int layout, void* workspace, size_t workspace_bytes,
                      void* stream) {
  LinearPlan plan;
  if (kmq_status s = check_linear_args(packed, codebooks, x, y, N, K, bits, M, layout, workspace, workspace_bytes, &plan))
    return s;
  return launch_linear(plan, packed, codebooks, x, y, N, K, bits, M, layout, workspace, (cudaStream_t)stream) ==
                 cudaSuccess
             ? KMQ_OK
             : KMQ_ERR_CUDA;
}

kmq_status kmq_linear_host(const uint32_t* packed, const uint16_t* codebooks, const uint16_t* x_host, uint16_t* y_host,
                           int64_t N, int64_t K, int bits, int64_t M, int layout, uint16_t* x_dev, uint16_t* y_dev,
                           void* workspace, size_t workspace_bytes, void* stream) {
  if (!x_host || !y_host) return KMQ_ERR_NULL;
  // everything is validated before the first copy is enqueued: a failed check launches nothing
  LinearPlan plan;
  if (kmq_status s = check_linear_args(packed, codebooks, x_dev, y_dev, N, K, bits, M, layout, workspace,
                                       workspace_bytes, &plan))
    return s;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(x_dev, x_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) return KMQ_ERR_CUDA;
  if (launch_linear(plan, packed, codebooks, x_dev, y_dev, N, K, bits, M, layout, workspace, st) != cudaSuccess)
    return KMQ_ERR_CUDA;
  if (cudaMemcpyAsync(y_host, y_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KMQ_ERR_CUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

kmq_status kmq_linear_tcgen05(const uint32_t* packed, const uint16_t* codebooks, const uint16_t* x, uint16_t* y,
                              int64_t N, int64_t K, int bits, int64_t M, void* stream) {
  if (!packed || !codebooks || !x || !y) return KMQ_ERR_NULL;
  if (kmq_status s = check_shape(N, K, bits, M)) return s;
  if ((K * bits) % 128 != 0) return KMQ_ERR_SHAPE;
  if (!aligned16(packed) || !aligned16(codebooks) || !aligned16(x) || !aligned16(y)) return KMQ_ERR_ALIGN;
  if (!device_info()) return KMQ_ERR_CUDA;
  return launch_linear_umma(packed, codebooks, x, y, N, K, bits, M, (cudaStream_t)stream) == cudaSuccess ? KMQ_OK
                                                                                                        : KMQ_ERR_CUDA;
}

kmq_status kmq_device_error_flags(unsigned int* flags) {
  if (!flags) return KMQ_ERR_NULL;
  return read_device_error_flags(flags) == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA;
}

kmq_status kmq_dequant_to_bf16(const uint32_t* packed, const uint16_t* codebooks, uint16_t* W, int64_t N, int64_t K,
                               int bits, int layout, void* stream) {
  if (!packed || !codebooks || !W) return KMQ_ERR_NULL;
  if (kmq_status s = check_shape(N, K, bits, 1)) return s;
  if (!known_layout(layout)) return KMQ_ERR_LAYOUT;
  if (!aligned16(packed) || !aligned16(codebooks) || !aligned16(W)) return KMQ_ERR_ALIGN;
  return launch_dequant(packed, codebooks, W, N, K, bits, layout, (cudaStream_t)stream) == cudaSuccess ? KMQ_OK
                                                                                               : KMQ_ERR_CUDA;
}

}  // extern "C"
