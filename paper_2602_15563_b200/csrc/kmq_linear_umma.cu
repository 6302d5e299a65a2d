// kmq_linear on the tuned (tile-major) layout for large batches: the 5th-generation tensor core (tcgen05.mma)
// multiplies dequantised bf16 weights, held in tensor memory, with the activations in shared memory; the accumulator
// lives in tensor memory too.
//
// One CTA owns 128 output rows (8 tiles of 16) and walks its share of K in stages of 128 weights per row.  Its 16
// decoder warps, one MMA warp and one TMA producer warp meet only through mbarriers:
//   * the decoder threads copy the packed words of the CTA's 8 tiles, one 1 KB step per tile at a time, global ->
//     shared with coalesced cp.async (ring of kWRing steps, rows padded to 80 bytes; one named barrier per step).
//     Decoder thread (warp w, lane l) owns output row 32 (w % 4) + l of the CTA -- the tensor-memory lane a warp may
//     write is fixed by its index -- and quarter w / 4 of each stage's weights of that row: it reads its 4..16 bytes
//     from the ring, rebuilds the 32 weights as bf16 pairs in registers and writes them with tcgen05.st into the A
//     operand of the stage (lane = row, 32-bit column c = weights 2c, 2c + 1 of the stage; ring of kARing stages).
//     When a warp's part of a stage is in place it arrives on the stage's `full` barrier;
//   * the producer thread copies the activations under a stage (NB batch rows x 128, zero-filled past M and past K)
//     with two TMA tile loads (cp.async.bulk.tensor, 64 columns = 128 bytes wide, 128-byte swizzle) into the B
//     buffer of the stage, up to a whole ring ahead; their bytes complete the same `full` barrier;
//   * the MMA thread waits for `full`, issues 8 tcgen05.mma (128 x NB x 16 each) that add into the accumulator
//     D[128 output rows][NB batch rows], and commits them to the stage's `empty` barrier, which the decoders and the
//     producer wait for before they overwrite the A operand and the B buffer.
// When the 128-row blocks alone would leave half of the SMs idle, K is split over a cluster of 2 CTAs: each
// accumulates its half, CTA 1 writes its accumulator into CTA 0's shared memory (st.shared::cluster between two
// cluster barriers), CTA 0 adds the two in a fixed order.  At the end the decoder warps read the accumulator with
// tcgen05.ld (lane = output row, column = batch row), round to bf16 and store.
//
// Every wait on an mbarrier is bounded; a warp whose wait runs out sets bit 0 of the device error word and goes to
// the end of the kernel (so does, after its own bounded waits, every warp that depended on it); every thread still
// takes part in the cluster barriers and the final CTA barrier, after which the tensor memory is freed.
#include <cuda.h>

#include "kmq_common.cuh"
#include "kmq_linear_variants.cuh"
#include "kmq_mma_common.cuh"

namespace kmq {

__device__ unsigned int g_device_error_flags = 0;   // sticky; read and cleared by kmq_device_error_flags()

namespace {

constexpr int kBM = 128;                                 // output rows per CTA (rows of the MMA)
constexpr int kDecodeWarps = 16;                         // 4 tensor-memory lane quarters x 4 quarters of a stage's weights
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kThreads = kDecodeThreads + 64;            // + the MMA warp + the TMA producer warp
// Stages in flight: A operands in tensor memory (the decoders may run this far ahead of the MMAs) and, one per A
// operand, B buffers in shared memory.  6, or 4 for more than 64 batch rows (128 columns of accumulator, 32 KB per B
// buffer).
template <int NB>
constexpr int ring_depth() {
  return NB > 64 ? 4 : 6;
}
constexpr int kWRing = 6;                   // ring of 1 KB steps of packed words per tile (cp.async), kWRing - 1 in flight
constexpr int kWRowStride = 80;                          // a row's 64 bytes of a step, padded: lanes read consecutive rows
constexpr int kWStepBytes = kBM * kWRowStride;
constexpr uint32_t kWaitHintNs = 20000;                  // one try_wait on an mbarrier may park the thread this long
constexpr uint64_t kWaitLimitNs = 100ull * 1000 * 1000;  // a wait gives up after this much time on the global timer

template <int BITS>
struct UGeo {
  static constexpr int kStageK = 128;                            // weights of a row per stage
  static constexpr int kStagesPerStep = (512 / BITS) / kStageK;  // 1, 2, 4 for b = 4, 2, 1
  static constexpr int kThreadBytes = kStageK * BITS / 32;       // packed bytes a thread decodes per stage: 16, 8, 4
  static constexpr int kCols = kStageK / 2;                      // 32-bit columns of the A operand of a stage
  static constexpr int kKSlices = kStageK / 16;                  // MMAs per stage
  static constexpr int kTableBytes = BITS == 4 ? 4 * 16 * 128 : 0;   // b = 4: [lane quarter][entry][lane]
};

template <int BITS, int NB>
struct USmem {
  static constexpr int kARing = ring_depth<NB>();
  static constexpr int kBRing = kARing;
  static constexpr int kTmemCols = 512;                             // kARing * 64 columns of A + NB columns of D <= 512
  static_assert(kARing * 64 + NB <= 512, "tensor memory has 512 columns");
  static constexpr int kBHalfBytes = NB * 128;                      // NB rows x 64 activations (one TMA box)
  static constexpr int kBStageBytes = 2 * kBHalfBytes;
  static constexpr int kB = 0;
  static constexpr int kWords = kB + kBRing * kBStageBytes;   // ring of packed words: [step][row][80]
  static constexpr int kTables = kWords + kWRing * kWStepBytes;
  static constexpr int kBars = kTables + UGeo<BITS>::kTableBytes;   // full[kARing], empty[kARing]
  static constexpr int kTmemSlot = kBars + 2 * kARing * 8;   // then a word that a failed wait sets
  static constexpr int kTotal = kTmemSlot + 16 + 1024;   // + room to align the base to 1024 bytes (swizzled B buffers)
};

// Shared-memory matrix descriptor of a K-major operand in the 128-byte-swizzle layout TMA writes: rows of 128 bytes,
// 8-row groups 1024 bytes apart (stride byte offset), descriptor version of sm_100, layout type 2 = 128-byte swizzle.
// The buffer is 1024-byte aligned; 16 weights further along K = 32 bytes further in the start address.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// TMA tile load of the box at (c0, c1) of a 2-D tensor map into shared memory; its bytes complete on `bar`.
__device__ __forceinline__ void tma_load_2d(uint32_t smem_dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
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
// the same with the accumulate flag fixed to true
__device__ __forceinline__ void umma_bf16_acc(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 0, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      :
      : "r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc)
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

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src, bool valid) {
  const int bytes = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gmem_src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// All threads of all CTAs of the cluster.
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The shared::cluster address of CTA 0's copy of this CTA's shared-memory address `saddr`.
__device__ __forceinline__ uint32_t map_to_rank0(uint32_t saddr) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(r) : "r"(saddr));
  return r;
}
// This thread's lane of the accumulator, columns [col0, col0 + NC): all loads are issued before the one wait
// (zeros when nothing was accumulated).
template <int NC>
__device__ __forceinline__ void load_acc(uint32_t (&w)[NC], uint32_t taddr, bool valid) {
  static_assert(NC % 8 == 0, "whole groups of 8 columns");
  if (valid) {
#pragma unroll
    for (int c = 0; c < NC; c += 8)
      asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=r"(w[c + 0]), "=r"(w[c + 1]), "=r"(w[c + 2]), "=r"(w[c + 3]), "=r"(w[c + 4]), "=r"(w[c + 5]),
                     "=r"(w[c + 6]), "=r"(w[c + 7])
                   : "r"(taddr + c));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  } else {
#pragma unroll
    for (int j = 0; j < NC; ++j) w[j] = 0;
  }
}

// Bounded wait for the phase of parity `parity` of an mbarrier.  try_wait parks the thread in hardware for up to the
// hinted time instead of spinning, so waiting warps do not take issue slots from the ones that decode.  The hint is
// only a hint (a try may come back early), so the bound is taken on the global timer, not on the number of tries.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  uint64_t t0 = 0;
  for (;;) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"(kWaitHintNs)
        : "memory");
    if (done) return true;
    uint64_t now;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
    if (t0 == 0) t0 = now;
    else if (now - t0 > kWaitLimitNs) return false;
  }
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
// tensor-memory lane starting at `taddr` (8 columns at b = 2, 16 at b = 1).
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
                                                                  const __grid_constant__ CUtensorMap xmap,
                                                                  uint16_t* __restrict__ y, int64_t N, int64_t K,
                                                                  int M) {
  using G = UGeo<BITS>;
  using SM = USmem<BITS, NB>;
  constexpr int SPS = G::kStagesPerStep;
  constexpr int NW = G::kThreadBytes / 4;   // packed words per thread and stage: 4, 2, 1
  constexpr int kARing = SM::kARing;
  constexpr int kReaders = NB % 32 == 0 ? 4 : 2;   // warps per lane quarter that read the accumulator
  constexpr int kReadCols = NB / kReaders;         // columns each of them reads (a multiple of 8)
  extern __shared__ __align__(1024) unsigned char smem_unaligned[];
  unsigned char* const smem_raw =
      smem_unaligned + ((1024u - ((uint32_t)__cvta_generic_to_shared(smem_unaligned) & 1023u)) & 1023u);
  unsigned char* const tables = smem_raw + SM::kTables;
  const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem_raw);
  const uint32_t b_addr = smem_base + SM::kB;
  const uint32_t full_bar = smem_base + SM::kBars, empty_bar = full_bar + 8 * kARing;
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_raw + SM::kTmemSlot);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t block_row0 = (int64_t)blockIdx.x * kBM;
  const int chunks = (int)(K / (128 / BITS));   // 16-byte chunks per row
  const int steps = (chunks + 3) >> 2;          // the layout pads every row to whole steps of 64 bytes
  // K is split over the gridDim.y CTAs of a cluster (same output rows): rank r takes steps [s_begin, s_end)
  const int ksplit = gridDim.y, rank = blockIdx.y;
  const int s_begin = (int)((int64_t)steps * rank / ksplit), s_end = (int)((int64_t)steps * (rank + 1) / ksplit);
  const int my_steps = s_end - s_begin;
  const int total = my_steps * SPS;             // stages of this CTA

  // ---- set-up: mbarriers, tensor memory, tables ----
  if (threadIdx.x == 0) {
    *reinterpret_cast<volatile uint32_t*>(smem_raw + SM::kTmemSlot + 4) = 0;
#pragma unroll
    for (int i = 0; i < kARing; ++i) {
      // decoder warps + the producer's arrive-and-expect; the TMA bytes complete the same phase
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full_bar + 8 * i), "r"(kDecodeWarps + 1) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(empty_bar + 8 * i) : "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kDecodeWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_base + SM::kTmemSlot),
                 "r"((uint32_t)SM::kTmemCols)
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
    // row rho % 16 of a tile owns bytes [64 (rho % 16), +64) of each 1 KB step; rows of a tile past N decode zeros
    // and are never stored
    RowState<BITS> st;
    st.init(cb + min(block_row0 + rho, N - 1) * (1 << BITS), tables + q * 2048, lane);
    // packed words: whole 1 KB steps of the CTA's 8 tiles, global -> shared, coalesced (thread j copies 16-byte piece
    // j % 64 of tile j / 64 = piece j % 4 of row j / 4), one cp.async group per step, kWRing - 1 steps in flight
    const unsigned char* const w_row = smem_raw + SM::kWords + rho * kWRowStride + kh * G::kThreadBytes;
    const int cj = threadIdx.x;
    const int64_t c_tile = (int64_t)blockIdx.x * (kBM / 16) + (cj >> 6);
    const unsigned char* const c_src =
        reinterpret_cast<const unsigned char*>(packed) + ((c_tile < tiles ? c_tile : 0) * (int64_t)steps + s_begin) * 1024 +
        (cj & 63) * 16;
    const uint32_t c_dst = smem_base + SM::kWords + (cj >> 2) * kWRowStride + (cj & 3) * 16;
    auto copy_step = [&](int s) {
      if (s < my_steps) cp_async16(c_dst + (s % kWRing) * kWStepBytes, c_src + (int64_t)s * 1024, c_tile < tiles);
      cp_async_commit();
    };
    volatile uint32_t* const fail_word = reinterpret_cast<volatile uint32_t*>(smem_raw + SM::kTmemSlot + 4);
#pragma unroll 1
    for (int d = 0; d < kWRing - 1; ++d) copy_step(d);
    int i = 0;   // stage
    for (int s = 0; s < my_steps; ++s) {
      cp_async_wait<kWRing - 2>();   // this thread's piece of step s has landed
      // every decoder thread's piece of step s has landed, and every one is done with step s - 1
      asm volatile("bar.sync 1, %0;" ::"n"(kDecodeThreads) : "memory");
      if (*fail_word) {   // some warp's wait ran out: all decoders leave together
        ok = false;
        break;
      }
      copy_step(s + kWRing - 1);     // into the slot of step s - 1
      const unsigned char* const w_step = w_row + (s % kWRing) * kWStepBytes;
#pragma unroll
      for (int u = 0; u < SPS; ++u, ++i) {
        const int abuf = i % kARing;
        // the stage's bytes of the row: [u * 64 / SPS, +64 / SPS) of its 64 bytes in the step; this thread's quarter
        uint32_t wv[NW];
        if constexpr (NW == 4) {
          const uint4 t4 = *reinterpret_cast<const uint4*>(w_step + u * (64 / SPS));
          wv[0] = t4.x; wv[1] = t4.y; wv[2] = t4.z; wv[3] = t4.w;
        } else if constexpr (NW == 2) {
          const uint2 t2 = *reinterpret_cast<const uint2*>(w_step + u * (64 / SPS));
          wv[0] = t2.x; wv[1] = t2.y;
        } else {
          wv[0] = *reinterpret_cast<const uint32_t*>(w_step + u * (64 / SPS));
        }
        if (ok && i >= kARing) {
          // the MMAs of stage i - kARing are done: A operand i % kARing may be overwritten
          ok = mbar_wait(empty_bar + 8 * abuf, ((i / kARing) - 1) & 1);
          ok = __all_sync(0xFFFFFFFFu, ok);
          if (!ok) *fail_word = 1;
          tc_fence_after_sync();
        }
        if (!ok) continue;   // up to the next barrier, where all decoders leave
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
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(full_bar + 8 * abuf);
      }
    }
    // ---- wait until all MMAs of this CTA are done ----
    if (ok && total > 0) {
      const int last = total - 1;
      ok = mbar_wait(empty_bar + 8 * (last % kARing), (last / kARing) & 1);
      ok = __all_sync(0xFFFFFFFFu, ok);
    }
    if (!ok && lane == 0) atomicOr(&g_device_error_flags, 1u);
  } else if (warp == kDecodeWarps && lane == 0) {
    // ================= MMA warp (one thread) =================
    // The issuing thread is blocked for about 70 clocks per tcgen05.mma and runs everything in between serially, so
    // the per-instruction work is kept to one add: descriptors differ only in their low word.
    const uint32_t idesc = instr_desc<NB>();
    const uint64_t desc0 = smem_desc_sw128(b_addr);
    const uint32_t desc_hi = (uint32_t)(desc0 >> 32);
    uint32_t desc_lo = (uint32_t)desc0, a_tmem = tmem_base, bar_off = 0;   // of the current stage's buffer
    int abuf = 0;
    uint32_t parity = 0;
    for (int i = 0; i < total; ++i) {
      if (!mbar_wait(full_bar + bar_off, parity)) {
        ok = false;
        break;
      }
      tc_fence_after_sync();
#pragma unroll
      for (int ks = 0; ks < G::kKSlices; ++ks) {   // 16 activations = 32 bytes further inside a 128-byte row
        const uint32_t lo = desc_lo + (ks >> 2) * (SM::kBHalfBytes >> 4) + (ks & 3) * 2;
        const uint64_t b_desc = ((uint64_t)desc_hi << 32) | lo;
        if (ks == 0) umma_bf16(tmem_d, a_tmem, b_desc, idesc, i != 0);
        else umma_bf16_acc(tmem_d, a_tmem + ks * 8, b_desc, idesc);
      }
      umma_commit(empty_bar + bar_off);
      if (++abuf == kARing) {
        abuf = 0;
        parity ^= 1;
        desc_lo = (uint32_t)desc0;
        a_tmem = tmem_base;
        bar_off = 0;
      } else {
        desc_lo += SM::kBStageBytes >> 4;
        a_tmem += G::kCols;
        bar_off += 8;
      }
    }
    if (!ok) atomicOr(&g_device_error_flags, 1u);
  } else if (warp == kDecodeWarps + 1 && lane == 0) {
    // ================= TMA producer (one thread) =================
    for (int j = 0; j < total; ++j) {
      const int buf = j % kARing;
      if (j >= kARing && !mbar_wait(empty_bar + 8 * buf, ((j / kARing) - 1) & 1)) {   // the MMAs that read the buffer
        ok = false;
        break;
      }
      mbar_expect_tx(full_bar + 8 * buf, SM::kBStageBytes);
      const int k0 = (s_begin * SPS + j) * G::kStageK;
      tma_load_2d(b_addr + buf * SM::kBStageBytes, &xmap, k0, 0, full_bar + 8 * buf);
      tma_load_2d(b_addr + buf * SM::kBStageBytes + SM::kBHalfBytes, &xmap, k0 + 64, 0, full_bar + 8 * buf);
    }
    if (!ok) atomicOr(&g_device_error_flags, 1u);
  }
  // ---- accumulators of the cluster -> rank 0 -> bf16 ----
  // Rank r > 0 hands its accumulator to rank 0 through rank 0's shared memory (the B buffers, free once every CTA of
  // the cluster has seen its last MMA complete): [r - 1][batch row][output row] floats.
  __syncwarp();
  if (ksplit > 1) cluster_sync();
  const bool reader = warp < kDecodeWarps && (warp >> 2) < kReaders && ok;   // the warps of a lane quarter split the columns
  if (reader) {
    const int q = warp & 3, kh = warp >> 2, rho = 32 * q + lane;
    tc_fence_after_sync();
    if (rank != 0) {
      const uint32_t remote = map_to_rank0(smem_base + SM::kB) + (uint32_t)(rank - 1) * (NB * kBM * 4);
      const int col0 = kh * kReadCols;
      uint32_t w[kReadCols];
      load_acc<kReadCols>(w, tmem_d + ((uint32_t)(q * 32) << 16) + col0, total > 0);
#pragma unroll
      for (int j = 0; j < kReadCols; ++j)
        asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(remote + ((col0 + j) * kBM + rho) * 4), "r"(w[j]) : "memory");
    }
  }
  __syncwarp();
  if (ksplit > 1) cluster_sync();
  if (reader && rank == 0) {
    const int q = warp & 3, kh = warp >> 2, rho = 32 * q + lane;
    const int64_t n = block_row0 + rho;
    const float* const partial = reinterpret_cast<const float*>(smem_raw + SM::kB);
    const int col0 = kh * kReadCols;
    uint32_t w[kReadCols];
    load_acc<kReadCols>(w, tmem_d + ((uint32_t)(q * 32) << 16) + col0, total > 0);
#pragma unroll
    for (int j = 0; j < kReadCols; ++j) {
      float v = __uint_as_float(w[j]);
      for (int r = 1; r < ksplit; ++r) v += partial[((r - 1) * NB + col0 + j) * kBM + rho];   // fixed order
      if (col0 + j < M && n < N) y[(int64_t)(col0 + j) * N + n] = (uint16_t)float_to_bf16_bits(v);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  // The tensor memory is given back on every path, also after a wait ran out: a CTA that left without freeing its
  // columns would block every later CTA on this SM in tcgen05.alloc for good.  A wait only runs out after 100 ms,
  // five orders of magnitude beyond the life of any instruction this kernel issues, so nothing of this CTA can
  // still be using the columns then.
  if (warp == kDecodeWarps)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)SM::kTmemCols)
                 : "memory");
}

}  // namespace

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up once through the runtime (no link against the driver library).
EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// x as a 2-D tensor [M rows][K] of bf16; boxes of NB rows x 64 columns (128 bytes) land in shared memory with the
// 128-byte swizzle; rows past M and columns past K read as zero.
template <int NB>
bool make_x_map(CUtensorMap* map, const uint16_t* x, int64_t K, int M) {
  EncodeTiledFn enc = encode_tiled();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
  const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)NB};
  const cuuint32_t elem[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<uint16_t*>(x), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Dynamic shared memory to launch with: what the kernel uses, but more than half of what an SM offers (the opt-in
// maximum per CTA is the SM's shared memory minus the 1 KB the system keeps per CTA).
inline int umma_launch_smem(int kernel_bytes, int max_smem_optin) {
  const int more_than_half = max_smem_optin / 2 + 1024;
  return kernel_bytes > more_than_half ? kernel_bytes : more_than_half;
}

template <int BITS, int NB>
cudaError_t launch_nb(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N, int64_t K,
                      int M, cudaStream_t s) {
  // Every CTA takes all 512 tensor-memory columns with a blocking tcgen05.alloc and frees them only at its end, after
  // cluster barriers: two such CTAs on one SM (of one cluster or of two) could wait for each other for ever.  The
  // launch therefore asks for more than half of the SM's shared memory whatever the kernel needs, so that a second
  // CTA can never become resident on the same SM.
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const int smem = umma_launch_smem(USmem<BITS, NB>::kTotal, di->max_smem_optin);
  if (smem > di->max_smem_optin || 2 * (smem + 1024) <= di->max_smem_optin + 1024) return cudaErrorInvalidConfiguration;
  static bool configured[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    cudaError_t e = cudaFuncSetAttribute(linear_umma_kernel<BITS, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    configured[dev] = true;
  }
  CUtensorMap xmap;
  if (!make_x_map<NB>(&xmap, x, K, M)) return cudaErrorInvalidValue;
  const unsigned blocks = (unsigned)((N + kBM - 1) / kBM);
  const int ksplit = linear_umma_ksplit(N, K, BITS, NB);
  if ((ksplit - 1) * NB * kBM * 4 > USmem<BITS, NB>::kBRing * USmem<BITS, NB>::kBStageBytes)
    return cudaErrorInvalidValue;   // the partial accumulators of the other CTAs must fit the B buffers
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks, (unsigned)ksplit);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = (unsigned)ksplit;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = ksplit > 1 ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, linear_umma_kernel<BITS, NB>, packed, cb, xmap, y, N, K, M);
}

template <int BITS>
cudaError_t launch_bits(const uint32_t* packed, const uint16_t* cb, const uint16_t* x, uint16_t* y, int64_t N,
                        int64_t K, int M, cudaStream_t s) {
  if (M <= 16) return launch_nb<BITS, 16>(packed, cb, x, y, N, K, M, s);
  if (M <= 32) return launch_nb<BITS, 32>(packed, cb, x, y, N, K, M, s);
  if (M <= 48) return launch_nb<BITS, 48>(packed, cb, x, y, N, K, M, s);
  if (M <= 64) return launch_nb<BITS, 64>(packed, cb, x, y, N, K, M, s);
  if (M <= 96) return launch_nb<BITS, 96>(packed, cb, x, y, N, K, M, s);
  return launch_nb<BITS, 128>(packed, cb, x, y, N, K, M, s);
}

}  // namespace

int linear_umma_rows_per_launch() { return 128; }   // one tcgen05.mma costs the same for every N <= 128

// CTAs per 128-row block: K is split over a cluster of 2 or 4 (partial sums meet in CTA 0's shared memory) while the
// blocks alone would leave at least half (three quarters) of the SMs idle and each part still has a few steps.
// `batch` = rows of one launch; 4 CTAs only up to 64 rows (three partial accumulators must fit the B buffers).
int linear_umma_ksplit(int64_t N, int64_t K, int bits, int batch) {
  const DeviceInfo* di = device_info();
  if (!di) return 1;
  const int64_t blocks = (N + kBM - 1) / kBM, steps = (K * bits / 128 + 3) / 4;
  if (blocks * 4 <= di->sm_count && steps >= 32 && batch <= 64) return 4;   // measured: no gain with fewer than 8 steps per CTA
  return (blocks * 2 <= di->sm_count && steps >= 8) ? 2 : 1;
}

// The tensor core issues one tcgen05.mma (2048 weights) per 70-100 clocks whatever the batch, so the kernel's time
// does not depend on M up to 128 rows, but a CTA covers 128 output rows: it pays when the batch is large and there
// are enough 128-row blocks to occupy most SMs.  Measured: 16384 x 3072, b = 2: 18.5 us for any M <= 64 against
// 18.5 / 28.5 / 31.6 us of the multi-tile kernel at M = 32 / 40 / 64; 12288 x 4096, M = 64: 22.7 against 38.9 us;
// 8192 x 8192 (64 blocks), M = 64: 38.9 against 36.0 us.
bool linear_umma_selected(int64_t N, int64_t K, int bits, int64_t M) {
  const DeviceInfo* di = device_info();
  // b = 1: the multi-tile kernel has no 16-warp form beyond 16 rows (its x buffers are twice as large) and takes
  // 80 us at 8192 x 28672 for M = 17..32 against 60 us here
  if (!di || M <= (bits == 1 ? 16 : 32) || (K * bits) % 128 != 0) return false;
  if (!encode_tiled()) return false;   // no tensor-map encoder in this driver: stay on the mma.sync kernels
  const int batch = (int)(M < linear_umma_rows_per_launch() ? M : linear_umma_rows_per_launch());
  const int64_t ctas = (N + kBM - 1) / kBM * linear_umma_ksplit(N, K, bits, batch);
  // with fewer CTAs it still wins where the multi-tile kernel is weakest: more than 48 rows, or b = 1 (which that
  // kernel serves 32 rows at a time): 4096 x 4096, 64 CTAs, M = 64: b = 2 18.4 against 20.7 us, b = 1 17.6 against 32.8 us
  const int64_t need = (M > 48 || bits == 1) ? (int64_t)di->sm_count * 3 / 8 : (int64_t)di->sm_count * 5 / 8;
  return ctas >= need;
}

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
  if (*flags) {
    const unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_device_error_flags, &zero, sizeof(unsigned int));
    if (e != cudaSuccess) return e;
  }
  unsigned int lut = 0;
  e = read_lut_error_flags(&lut);
  *flags |= lut;
  return e;
}


}  // namespace kmq
