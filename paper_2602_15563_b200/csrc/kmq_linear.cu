// Host-side dispatch of kmq_linear: picks a kernel variant for (bits, M, N, K, layout).
#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"

namespace kmq {

LinearPlan plan_linear(int64_t N, int64_t K, int bits, int64_t M, int layout) {
  LinearPlan p;
  p.workspace = 0;
  p.split_k = 1;
  if (layout == KMQ_LAYOUT_TABLE && bits != 4) {
    if (!linear_lut_supports(N, K, bits, M)) {
      p.variant = kVariantUnsupported;
      p.launches = 0;
      p.name = "unsupported";
      return p;
    }
    p.variant = kVariantLut;
    p.workspace = linear_lut_scratch_bytes(N, K, bits);
    p.launches = (int)(p.workspace ? 2 * M : M);
    p.name = bits == 1 ? "table_lookup_b1" : "table_lookup_b2";
    return p;
  }
  if (layout == KMQ_LAYOUT_TABLE) layout = KMQ_LAYOUT_TUNED;   // b = 4: the two layouts are the same
  if (linear_mma_supports(N, K, bits, M)) {
    const bool tuned = layout == KMQ_LAYOUT_TUNED;
    p.variant = tuned ? kVariantTiled : kVariantMma;
    p.launches = (int)((M + 7) / 8);
    if (tuned && linear_umma_selected(N, K, bits, M)) {
      const int64_t per = linear_umma_rows_per_launch();
      p.variant = kVariantUmma;
      p.launches = (int)((M + per - 1) / per);
      p.name = bits == 4 ? "tcgen05_table_b4" : bits == 2 ? "tcgen05_prmt_b2" : "tcgen05_select_b1";
      return p;
    }
    if (tuned && M >= linear_multi_min_rows(bits, N)) {
      const int64_t per = linear_multi_rows_per_launch(bits);
      p.variant = kVariantMulti;
      p.launches = (int)((M + per - 1) / per);
      p.name = bits == 4 ? "multi_table_b4" : bits == 2 ? "multi_prmt_b2" : "multi_select_b1";
      return p;
    }
    if (tuned) {
      const int ctas = linear_split_ctas(N, K, bits, M);
      if (ctas > 0) {
        p.variant = kVariantSplit;
        p.launches = 2;
        p.split_k = ctas;
        p.workspace = linear_split_scratch_bytes(ctas);
        p.name = bits == 4 ? "split_pairtable_b4" : bits == 2 ? "split_prmt_b2" : "split_select_b1";
        return p;
      }
    }
    if (bits == 4) p.name = tuned ? "tiled_pairtable_b4" : "staged_pairtable_b4";
    else if (bits == 2) p.name = tuned ? "tiled_prmt_b2" : "staged_prmt_b2";
    else p.name = tuned ? "tiled_select_b1" : "staged_select_b1";
  } else {
    p.variant = kVariantGeneric;
    p.launches = 1;
    p.name = "generic_warp_per_row";
  }
  return p;
}

cudaError_t launch_linear(const LinearPlan& plan, const uint32_t* packed, const uint16_t* cb, const uint16_t* x,
                          uint16_t* y, int64_t N, int64_t K, int bits, int64_t M, int layout, void* workspace,
                          cudaStream_t s) {
  if (layout == KMQ_LAYOUT_TABLE && bits == 4) layout = KMQ_LAYOUT_TUNED;
  switch (plan.variant) {
    case kVariantLut:
      return launch_linear_lut(packed, cb, x, y, N, K, bits, M, workspace, s);
    case kVariantUnsupported:
      return cudaErrorNotSupported;
    case kVariantSplit:
      return launch_linear_split(packed, cb, x, y, N, K, bits, M, workspace, plan.split_k, s);
    case kVariantUmma:
      return launch_linear_umma(packed, cb, x, y, N, K, bits, M, s);
    case kVariantMulti:
      return launch_linear_multi(packed, cb, x, y, N, K, bits, M, s);
    case kVariantTiled:
      return launch_linear_tiled(packed, cb, x, y, N, K, bits, M, s);
    case kVariantMma:
      return launch_linear_mma(packed, cb, x, y, N, K, bits, M, s);
    case kVariantGeneric:
    default:
      return launch_linear_generic(packed, cb, x, y, N, K, bits, M, layout, s);
  }
}

}  // namespace kmq
