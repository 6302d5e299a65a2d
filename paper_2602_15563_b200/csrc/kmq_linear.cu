// Host-side dispatch of kmq_linear: picks a kernel variant for (bits, M, N, K).
#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"

namespace kmq {

LinearPlan plan_linear(int64_t N, int64_t K, int bits, int64_t M) {
  (void)N; (void)K; (void)bits; (void)M;
  LinearPlan p;
  p.variant = kVariantGeneric;
  p.launches = 1;
  p.workspace = 0;
  p.split_k = 1;
  p.name = "generic_warp_per_row";
  return p;
}

cudaError_t launch_linear(const LinearPlan& plan, const uint32_t* packed, const uint16_t* cb, const uint16_t* x,
                          uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, void* workspace, cudaStream_t s) {
  (void)workspace;
  switch (plan.variant) {
    case kVariantGeneric:
    default:
      return launch_linear_generic(packed, cb, x, y, N, K, bits, M, s);
  }
}

}  // namespace kmq
