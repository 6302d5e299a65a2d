// Kernel variants behind kmq_linear and their launchers.
#pragma once
#include "kmq_common.cuh"

namespace kmq {

enum LinearVariant : int {
  kVariantGeneric = 0,   // any legal shape and layout, CUDA-core FMAs, one warp per output row
  kVariantMma = 1,       // canonical layout, K*bits % 128 == 0: tensor-core GEMV, activations staged per warp
  kVariantTiled = 2,     // tuned (tile-major) layout: tensor-core GEMV with coalesced 1 KB steps, small batches (M <= 8)
  kVariantMulti = 3,     // tuned layout, M >= linear_multi_min_rows(): 32 or 64 rows per CTA share the staged
                         // activations, one decode feeds up to 8 MMAs
  kVariantUmma = 5,      // tuned layout, M > 32 and enough 128-row blocks to fill the SMs: tcgen05.mma, weights
                         // dequantised into tensor memory
  kVariantSplit = 4,     // tuned layout, M <= 8, more tiles than resident CTAs: equal step ranges + fix-up (scratch)
  kVariantLut = 6,       // table layout, b = 1, 2: activation tables in shared memory, one lookup per 8 weights (scratch)
  kVariantUnsupported = 7,
};

cudaError_t launch_linear_generic(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                                  int64_t K, int bits, int64_t M, int layout, cudaStream_t s);

bool linear_mma_supports(int64_t N, int64_t K, int bits, int64_t M);
cudaError_t launch_linear_mma(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                              int64_t K, int bits, int64_t M, cudaStream_t s);
cudaError_t launch_linear_tiled(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                                int64_t K, int bits, int64_t M, cudaStream_t s);

int linear_split_ctas(int64_t N, int64_t K, int bits, int64_t M);
size_t linear_split_scratch_bytes(int ctas);
cudaError_t launch_linear_split(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                                int64_t K, int bits, int64_t M, void* scratch, int ctas, cudaStream_t s);
int linear_multi_rows_per_launch(int bits);
int linear_multi_min_rows(int bits, int64_t N);   // smallest batch routed to the multi-tile kernel
cudaError_t launch_linear_multi(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                                int64_t K, int bits, int64_t M, cudaStream_t s);
bool linear_umma_selected(int64_t N, int64_t K, int bits, int64_t M);   // kmq_linear's choice of the tcgen05 kernel
int linear_umma_rows_per_launch();
int linear_umma_ksplit(int64_t N, int64_t K, int bits, int batch);   // CTAs (cluster size) per 128-row block
cudaError_t launch_linear_umma(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                               int64_t K, int bits, int64_t M, cudaStream_t s);
bool linear_lut_supports(int64_t N, int64_t K, int bits, int64_t M);
bool linear_lut_preferred(int64_t N, int64_t K, int bits, int64_t M);   // faster than the tensor-core kernels here
size_t linear_lut_scratch_bytes(int64_t N, int64_t K, int bits);
cudaError_t launch_linear_lut(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                              int64_t K, int bits, int64_t M, void* scratch, cudaStream_t s);
cudaError_t read_lut_error_flags(unsigned int* flags);   // reads and clears the table kernel's error word
cudaError_t read_device_error_flags(unsigned int* flags);   // synchronises; reads and clears the sticky error word

}  // namespace kmq
