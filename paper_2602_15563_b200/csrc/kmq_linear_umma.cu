// kmq_linear on the tuned (tile-major) layout for batches of 16 rows and more: the 5th-generation tensor core
// (tcgen05.mma) multiplies dequantised bf16 weights, held in tensor memory, with the activations in shared memory;
// the accumulator lives in tensor memory too.
//
// One CTA owns 128 output rows (8 tiles of 16) and walks K in stages of 256 (b = 4: 128) weights per row.  Its 8
// decoder warps and one MMA warp meet only through mbarriers:
//   * decoder thread (warp w, lane l) owns output row 32 (w % 4) + l of the CTA -- the tensor-memory lane a warp
//     may write is fixed by its index -- and half w / 4 of the stage's weights of that row.  In the tile-major layout
//     the 64 bytes of a row in a step are contiguous, so the thread loads its 16 or 32 bytes directly, rebuilds the
//     64 or 128 weights as bf16 pairs in registers and writes them with tcgen05.st into the A operand of the stage
//     (lane = row, 32-bit column c = weights 2c, 2c + 1 of the stage).  The decoder threads also copy the
//     activations two stages ahead (NB batch rows, zero-filled past M and past K) global -> shared with cp.async
//     into the K-major core-matrix layout of the B operand (8 rows x 16 bytes contiguous, the next 8 weights kLBO
//     bytes further, the next 8 rows kSBO bytes further).  When a warp's part of a stage is in place it arrives on
//     the stage's `full` barrier;
//   * the MMA warp waits for `full`, issues one tcgen05.mma (128 x NB x 16) per 16 weights that adds into the
//     accumulator D[128 output rows][NB batch rows], and commits them to the stage's `empty` barrier, which the
//     decoders wait for before they overwrite the A operand (ring of 2) and the B buffer (ring of 4).
// At the end the decoder warps read the accumulator with tcgen05.ld (lane = output row, column = batch row), round
// to bf16 and store.
//
// Every wait on an mbarrier is bounded; a warp whose wait runs out sets bit 0 of the device error word and goes to
// the end of the kernel (so does, after its own bounded waits, every warp that depended on it), where the tensor
// memory is freed.
#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"
#include "kmq_mma_common.cuh"

namespace kmq {

__device__ unsigned int g_device_error_flags = 0;   // sticky; read and cleared by kmq_device_error_flags()

namespace {

constexpr int kBM = 128;                                 // output rows per CTA (rows of the MMA)
constexpr int kDecodeWarps = 16;                         // 4 tensor-memory lane quarters x 4 quarters of a stage's weights
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kThreads = kDecodeThreads + 32;            // + the MMA warp
#ifndef KMQ_UMMA_ARING
#define KMQ_UMMA_ARING 6
#endif
constexpr int kARing = KMQ_UMMA_ARING;                   // A operands in tensor memory: the decoders may run this far ahead
constexpr int kBRing = kARing + 2;                       // B buffers in shared memory (activations are copied 2 stages ahead)
#ifndef KMQ_UMMA_WRING
#define KMQ_UMMA_WRING 8
#endif
constexpr int kWRing = KMQ_UMMA_WRING;                   // stages of packed words in flight per thread (cp.async ring)
constexpr int kLBO = 128;                                // bytes between core matrices that are neighbours in K
constexpr uint32_t kWaitLimit = 1u << 22;                // polls of an mbarrier before giving up (some tens of ms)

template <int BITS>
struct UGeo {
  static constexpr int kStageK = 128;                            // weights of a row per stage
  static constexpr int kStagesPerStep = (512 / BITS) / kStageK;  // 1, 2, 4 for b = 4, 2, 1
  static constexpr int kThreadBytes = kStageK * BITS / 32;       // packed bytes a thread decodes per stage: 16, 8, 4
  static constexpr int kCols = kStageK / 2;                      // 32-bit columns of the A operand of a stage
  static constexpr int kKSlices = kStageK / 16;                  // MMAs per stage
  static constexpr int kSBO = (kStageK / 8) * kLBO;              // bytes between groups of 8 batch rows in a B buffer
  static constexpr int kTmemCols = kARing * 64 + 64 <= 256 ? 256 : 512;   // kARing * kCols + up to 64 columns of D, a power of two
  static_assert(kARing * 64 + 64 <= 512, "tensor memory has 512 columns");
  static constexpr int kTableBytes = BITS == 4 ? 4 * 16 * 128 : 0;   // b = 4: [lane quarter][entry][lane]
};

template <int BITS, int NB>
struct USmem {
  static constexpr int kBStageBytes = NB * UGeo<BITS>::kStageK * 2;
  static constexpr int kB = 0;
  static constexpr int kWords = kB + kBRing * kBStageBytes;   // ring of packed words: [stage][16-byte piece][thread]
  static constexpr int kTables = kWords + kWRing * kDecodeThreads * UGeo<BITS>::kThreadBytes;
  static constexpr int kBars = kTables + UGeo<BITS>::kTableBytes;   // full[kARing], empty[kARing]
  static constexpr int kTmemSlot = kBars + 2 * kARing * 8;
  static constexpr int kTotal = kTmemSlot + 16;
};

// Shared-memory matrix descriptor: K-major, no swizzle, strides kLBO / kSBO, descriptor version of sm_100.
template <int SBO>
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(kLBO >> 4) << 16) | ((uint64_t)(SBO >> 4) << 32) |
         ((uint64_t)1 << 46);
}

// Instruction descriptor of kind::f16: D fp32, A and B bf16, both K-major, M = kBM, N = NB.
template <int NB>
__device__ __forceinline__ uint32_t instr_desc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NB >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

// D (tensor memory) (+)= A (tensor memory) x B (shared memory descriptor)
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      :
      : "r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_store8(uint32_t taddr, const uint32_t (&v)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(v[0]),
               "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void async_proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src, bool valid) {
  const int bytes = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gmem_src), "r"(bytes) : "memory");
}
// 8- and 4-byte variants (zero-filled when !valid)
__device__ __forceinline__ void cp_async8(uint32_t smem_dst, const void* gmem_src, bool valid) {
  const int bytes = valid ? 8 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(smem_dst), "l"(gmem_src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t smem_dst, const void* gmem_src, bool valid) {
  const int bytes = valid ? 4 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_dst), "l"(gmem_src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Bounded wait for the phase of parity `parity` of an mbarrier.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kWaitLimit; ++i) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

// Decode state of a thread's output row.
template <int BITS>
struct RowState;
template <>
struct RowState<2> {
  Dec2 d;
  __device__ __forceinline__ void init(const uint16_t* cb_row, const unsigned char*, int) { d.init(cb_row); }
};
template <>
struct RowState<1> {
  uint32_t base, diff;   // (c0, c0) and (c0 ^ c1, c0 ^ c1)
  __device__ __forceinline__ void init(const uint16_t* cb_row, const unsigned char*, int) {
    const uint32_t c = __ldg(reinterpret_cast<const uint32_t*>(cb_row));
    base = prmt(c, c, 0x1010u);
    diff = base ^ prmt(c, c, 0x3232u);
  }
};
template <>
struct RowState<4> {
  const unsigned char* tab;   // this lane's bank of the [entry][lane] table of its lane quarter
  __device__ __forceinline__ void init(const uint16_t*, const unsigned char* table_quarter, int lane) {
    tab = table_quarter + lane * 4;
  }
};

// One packed word of a row -> bf16 pairs in the order of k, written to consecutive columns of the row's
// tensor-memory lane starting at `taddr`.  Returns the number of columns written (weights per word / 2).
template <int BITS>
__device__ __forceinline__ void decode_word_to_tmem(uint32_t w, const RowState<BITS>& st, uint32_t taddr) {
  if constexpr (BITS == 2) {
    uint32_t a[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) st.d.pair(w, q, a[2 * q], a[2 * q + 1]);   // weights 4q .. 4q + 3
    tmem_store8(taddr, a);
  } else if constexpr (BITS == 1) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t a[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        // shift c puts weights (2c, 2c + 1) on bits 15 and 31; PRMT in sign-replicate mode turns them into
        // 16-bit masks; the masked XOR picks c0 or c1 bit-exactly
        const uint32_t sh = w * kPow2[8 * h + i];
        const uint32_t sel = prmt(sh, sh, 0xBB99u);
        asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(a[i]) : "r"(sel), "r"(st.diff), "r"(st.base));
      }
      tmem_store8(taddr + 8 * h, a);
    }
  }
}
// b = 4: two words (16 weights) per 8 columns
__device__ __forceinline__ void decode_words4_to_tmem(uint32_t w0, uint32_t w1, const RowState<4>& st, uint32_t taddr) {
  uint32_t a[8];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const uint32_t w = j ? w1 : w0;
    uint32_t e[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {   // nibble i -> byte offset nibble * 128 of the lane's table bank
      const int sh = 4 * i - 7;
      const uint32_t u = sh < 0 ? (w << -sh) : (w >> sh);
      e[i] = *reinterpret_cast<const uint32_t*>(st.tab + (u & 0x780u));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) a[4 * j + i] = prmt(e[2 * i], e[2 * i + 1], 0x7610u);
  }
  tmem_store8(taddr, a);
}

template <int BITS, int NB>
__global__ void __launch_bounds__(kThreads, 1) linear_umma_kernel(const uint32_t* __restrict__ packed,
                                                                  const uint16_t* __restrict__ cb,
                                                                  const uint16_t* __restrict__ x,
                                                                  uint16_t* __restrict__ y, int64_t N, int64_t K,
                                                                  int M) {
  using G = UGeo<BITS>;
  using SM = USmem<BITS, NB>;
  constexpr int SPS = G::kStagesPerStep;
  constexpr int NW = G::kThreadBytes / 4;   // packed words per thread and stage: 4, 2, 1
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* const tables = smem_raw + SM::kTables;
  const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
  const uint32_t b_addr = smem_base + SM::kB;
  const uint32_t full_bar = smem_base + SM::kBars, empty_bar = full_bar + 8 * kARing;
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + SM::kTmemSlot);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t block_row0 = (int64_t)blockIdx.x * kBM;
  const int chunks = (int)(K / (128 / BITS));   // 16-byte chunks per row
  const int steps = (chunks + 3) >> 2;          // the layout pads every row to whole steps of 64 bytes
  const int total = steps * SPS;                // stages

  // ---- set-up: mbarriers, tensor memory, tables ----
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 0; i < kARing; ++i) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full_bar + 8 * i), "r"(kDecodeWarps) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(empty_bar + 8 * i) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kDecodeWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_base + SM::kTmemSlot),
                 "r"((uint32_t)G::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if constexpr (BITS == 4) {
    // word [lane quarter q][entry e][lane] = (C_row[e], C_row[e]), row = block_row0 + 32 q + lane
    for (int i = threadIdx.x; i < 4 * 16 * 32; i += kThreads) {
      const int ln = i & 31, e = (i >> 5) & 15, q = i >> 9;
      const int64_t row = min(block_row0 + 32 * q + ln, N - 1);
      const uint32_t c = __ldg(cb + row * 16 + e);
      reinterpret_cast<uint32_t*>(tables)[i] = c | (c << 16);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_d = tmem_base + kARing * G::kCols;   // the accumulator follows the A operands
  bool ok = true;

  if (warp < kDecodeWarps) {
    // ================= decoder warps =================
    const int q = warp & 3, kh = warp >> 2;   // tensor-memory lane quarter; which quarter of a stage's weights
    const int rho = 32 * q + lane;            // output row inside the CTA = tensor-memory lane
    const int64_t tiles = (N + kTileRows - 1) / kTileRows;
    const int64_t tile_id = (int64_t)blockIdx.x * (kBM / 16) + (rho >> 4);
    const bool has_tile = tile_id < tiles;    // rows of a missing tile decode zeros; they are never stored
    // row rho % 16 of a tile owns bytes [64 (rho % 16), +64) of each 1 KB step
    const unsigned char* __restrict__ row_bytes = reinterpret_cast<const unsigned char*>(packed) +
                                                  (has_tile ? tile_id : 0) * (int64_t)steps * 1024 + (rho & 15) * 64;
    RowState<BITS> st;
    st.init(cb + min(block_row0 + rho, N - 1) * (1 << BITS), tables + q * 2048, lane);
    // packed words of stage i: global -> this thread's slot of ring stage i % kWRing (read back by the same thread)
    unsigned char* const w_slot = smem_raw + SM::kWords + threadIdx.x * G::kThreadBytes;
    const uint32_t w_slot_addr = smem_base + SM::kWords + threadIdx.x * G::kThreadBytes;
    constexpr int kWStage = kDecodeThreads * G::kThreadBytes;
    auto copy_words = [&](int i) {
      const int s = i / SPS, u = i % SPS;
      // the stage's bytes of the row: [u * 64 / SPS, +64 / SPS) of its 64 bytes in the step; this thread's quarter
      const unsigned char* src = row_bytes + (int64_t)s * 1024 + u * (64 / SPS) + kh * G::kThreadBytes;
      if constexpr (G::kThreadBytes == 16) cp_async16(w_slot_addr + (i % kWRing) * kWStage, src, has_tile);
      else if constexpr (G::kThreadBytes == 8) cp_async8(w_slot_addr + (i % kWRing) * kWStage, src, has_tile);
      else cp_async4(w_slot_addr + (i % kWRing) * kWStage, src, has_tile);
    };
    // activations of stage i -> B buffer i % kBRing; piece p = (batch row m, core matrix kg), bits of p:
    // kg0 | m0..2 | kg1.. | m3..  (8 consecutive threads: 4 rows x 32 contiguous bytes)
    auto stage_x = [&](int i) {
      constexpr int KGS = G::kStageK / 8;
      const uint32_t dst = b_addr + (i % kBRing) * SM::kBStageBytes;
#pragma unroll
      for (int j = 0; j < (NB * KGS + kDecodeThreads - 1) / kDecodeThreads; ++j) {
        const int p = threadIdx.x + kDecodeThreads * j;
        if (NB * KGS % kDecodeThreads != 0 && p >= NB * KGS) break;
        const int kg = (p & 1) | (((p >> 4) & (KGS / 2 - 1)) << 1);
        const int m = ((p >> 1) & 7) | ((p / (8 * KGS)) << 3);
        const int64_t k = (int64_t)i * G::kStageK + kg * 8;
        const bool valid = m < M && k < K;
        cp_async16(dst + (m >> 3) * G::kSBO + kg * kLBO + (m & 7) * 16, x + (valid ? (int64_t)m * K + k : 0), valid);
      }
      cp_async_commit();
    };

    // prologue: kWRing groups; group d holds the words of stage d and, for d < 2, the activations of stage d
#pragma unroll 1
    for (int d = 0; d < kWRing; ++d) {
      if (d < total) copy_words(d);
      if (d < 2 && d < total) stage_x(d);
      else cp_async_commit();
    }
    for (int i = 0; i < total; ++i) {
      const int abuf = i % kARing;
      cp_async_wait<kWRing - 1>();   // the group of the words of stage i has landed
      uint32_t wv[NW];
      if constexpr (NW == 4) {
        const uint4 t4 = *reinterpret_cast<const uint4*>(w_slot + (i % kWRing) * kWStage);
        wv[0] = t4.x; wv[1] = t4.y; wv[2] = t4.z; wv[3] = t4.w;
      } else if constexpr (NW == 2) {
        const uint2 t2 = *reinterpret_cast<const uint2*>(w_slot + (i % kWRing) * kWStage);
        wv[0] = t2.x; wv[1] = t2.y;
      } else {
        wv[0] = *reinterpret_cast<const uint32_t*>(w_slot + (i % kWRing) * kWStage);
      }
      if (i >= kARing) {
        // the MMAs of stage i - kARing are done: A operand i % kARing and B buffer (i + 2) % kBRing may be overwritten
        ok = mbar_wait(empty_bar + 8 * abuf, ((i / kARing) - 1) & 1);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        tc_fence_after_sync();
      }
      // this thread's quarter of the stage's weights of its row -> columns kh * kCols / 4 ... of the A operand
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + abuf * G::kCols + kh * (G::kCols / 4);
      if constexpr (BITS == 4) {
        decode_words4_to_tmem(wv[0], wv[1], st, taddr);
        decode_words4_to_tmem(wv[2], wv[3], st, taddr + 8);
      } else {
        constexpr int kColsPerWord = 16 / BITS;   // 8 or 16
#pragma unroll
        for (int jj = 0; jj < NW; ++jj) decode_word_to_tmem<BITS>(wv[jj], st, taddr + jj * kColsPerWord);
      }
      // one group per iteration: the activations of stage i + 2 and the words of stage i + kWRing (its ring slot
      // was read above, and the decode has consumed what was read)
      if (i + kWRing < total) copy_words(i + kWRing);
      if (i + 2 < total) stage_x(i + 2);
      else cp_async_commit();
      cp_async_wait<2>();   // the group with the activations of stage i has landed
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      async_proxy_fence();   // the copies into shared memory become visible to the tensor core's reads
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar + 8 * abuf);
    }
    // ---- all MMAs done -> read the accumulator, round, store ----
    if (ok && total > 0) {
      const int last = total - 1;
      ok = mbar_wait(empty_bar + 8 * (last % kARing), (last / kARing) & 1);
      ok = __all_sync(0xFFFFFFFFu, ok);
    }
    if (ok && kh < 2) {   // two warps per lane quarter split the columns
      tc_fence_after_sync();
      const int64_t n = block_row0 + rho;
#pragma unroll
      for (int c0 = 0; c0 < NB / 2; c0 += 8) {
        const int col = kh * (NB / 2) + c0;   // the two warps of a lane quarter split the columns
        uint32_t w[8];
        if (total > 0) {
          asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                       : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                       : "r"(tmem_d + ((uint32_t)(q * 32) << 16) + col));
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) w[j] = 0;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (col + j < M && n < N) y[(int64_t)(col + j) * N + n] = (uint16_t)float_to_bf16_bits(__uint_as_float(w[j]));
      }
    } else if (!ok && lane == 0) {
      atomicOr(&g_device_error_flags, 1u);
    }
  } else if (lane == 0) {
    // ================= MMA warp (one thread) =================
    const uint32_t idesc = instr_desc<NB>();
    for (int i = 0; i < total; ++i) {
      const int abuf = i % kARing;
      if (!mbar_wait(full_bar + 8 * abuf, (i / kARing) & 1)) {
        ok = false;
        break;
      }
      tc_fence_after_sync();
      const uint32_t b_stage = b_addr + (i % kBRing) * SM::kBStageBytes;
#pragma unroll
      for (int ks = 0; ks < G::kKSlices; ++ks)
        umma_bf16(tmem_d, tmem_base + abuf * G::kCols + ks * 8, smem_desc<G::kSBO>(b_stage + ks * 2 * kLBO), idesc,
                  (i | ks) != 0);
      umma_commit(empty_bar + 8 * abuf);
    }
    if (!ok) atomicOr(&g_device_error_flags, 1u);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kDecodeWarps)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)G::kTmemCols)
                 : "memory");
}

}  // namespace

namespace {

template <int BITS, int NB>
cudaError_t launch_nb(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N, int64_t K,
                      int M, cudaStream_t s) {
  constexpr int smem = USmem<BITS, NB>::kTotal;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(linear_umma_kernel<BITS, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  const unsigned grid = (unsigned)((N + kBM - 1) / kBM);
  linear_umma_kernel<BITS, NB><<<grid, kThreads, smem, s>>>(packed, cb, x, y, N, K, M);
  return cudaGetLastError();
}

template <int BITS>
cudaError_t launch_bits(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                        int64_t K, int M, cudaStream_t s) {
  if (M <= 16) return launch_nb<BITS, 16>(packed, cb, x, y, N, K, M, s);
  if (M <= 32) return launch_nb<BITS, 32>(packed, cb, x, y, N, K, M, s);
  if (M <= 48) return launch_nb<BITS, 48>(packed, cb, x, y, N, K, M, s);
  return launch_nb<BITS, 64>(packed, cb, x, y, N, K, M, s);
}

}  // namespace

int linear_umma_rows_per_launch() { return 64; }

cudaError_t launch_linear_umma(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                               int64_t K, int bits, int64_t M, cudaStream_t s) {
  const int64_t per = linear_umma_rows_per_launch();
  for (int64_t m0 = 0; m0 < M; m0 += per) {
    const int mc = (int)(M - m0 < per ? M - m0 : per);
    const uint16_t* xp = x + m0 * K;
    uint16_t* yp = y + m0 * N;
    cudaError_t e;
    if (bits == 1) e = launch_bits<1>(packed, cb, xp, yp, N, K, mc, s);
    else if (bits == 2) e = launch_bits<2>(packed, cb, xp, yp, N, K, mc, s);
    else e = launch_bits<4>(packed, cb, xp, yp, N, K, mc, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Reads and clears the device error word (synchronises the device).
cudaError_t read_device_error_flags(unsigned int* flags) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbol(flags, g_device_error_flags, sizeof(unsigned int));
  if (e != cudaSuccess) return e;
  const unsigned int zero = 0;
  return cudaMemcpyToSymbol(g_device_error_flags, &zero, sizeof(unsigned int));
}


}  // namespace kmq
