// Quantiser side of libkmq: 1-D Lloyd fit of a codebook per row (or of one codebook on a sample), nearest-centroid
// assignment fused with the bit packing, block scales of the paper's block format.  Paper: Section 2.1 "Rounding to
// nearest centroids" (Eq. "centroid quantizer"), "Block formats"; Section 2.2 (the two scale functions, "Nonlinear
// k-means quantization").  Everything that decides an index or a stored value is done in float64 with explicit
// round-to-nearest operations, so that a result does not depend on how the compiler contracts expressions.
#include "kmq_common.cuh"
#include "kmq_table_layout.cuh"

namespace kmq {
namespace {

constexpr int kMaxFitLen = 32768;      // values of one fit (one row, or the sample of a tensor): they live in shared memory
constexpr int kMaxCentroids = 256;

// float <-> key whose unsigned order is the order of the floats (-0 below +0, NaNs at the two ends)
__device__ __forceinline__ uint32_t key_of(float f) {
  const uint32_t u = __float_as_uint(f);
  return u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ double value_of(uint32_t k) {
  return (double)__uint_as_float(k ^ ((k >> 31) ? 0x80000000u : 0xFFFFFFFFu));
}

// ---------------------------------------------------------------------------------------------------------------
// Fit.  One CTA per row: the row is sorted once (bitonic network on the keys); a fixed two-level float64 prefix sum
// over chunks of 32 sorted values then gives the sum of any run of sorted values, so that an iteration is one binary
// search and one partial chunk per cluster boundary.  The clusters of 1-D Lloyd are runs of the sorted row: cluster i
// holds the values in (mid_{i-1}, mid_i], mid_i = (c_i + c_{i+1}) / 2 in float64.
//
// The sort keeps 32 keys per thread in registers: key number i of the (padded) row sits in register i % 32 of lane
// (i / 32) % 32 of warp i / 1024.  A compare-exchange at distance below 32 is then a register pair of one thread, at
// distance 32 .. 512 a warp shuffle, and only at distance 1024 and above an exchange through shared memory.  The
// direction of a merge phase is the same for all keys of a thread once the runs are 32 or longer; a thread whose
// runs go downwards complements its keys for the phase and merges upwards like everybody else.
// Shared memory holds key i at word i + i / 32: a thread's 32 keys and the same register of 32 lanes both fall on 32
// different banks.
// ---------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ int phys(int i) { return i + (i >> 5); }

// compare-exchange of registers at distance 2^B; ascending where bit M of the register number is clear (M > 4: always)
template <int B, int M>
__device__ __forceinline__ void local_stage(uint32_t (&k)[32]) {
#pragma unroll
  for (int r = 0; r < 32; ++r) {
    if ((r >> B) & 1) continue;
    const uint32_t a = k[r], b = k[r | (1 << B)];
    const bool up = M > 4 || ((r >> M) & 1) == 0;
    k[r] = up ? min(a, b) : max(a, b);
    k[r | (1 << B)] = up ? max(a, b) : min(a, b);
  }
}

// the five stages at distances 16 .. 1, all ascending
__device__ __forceinline__ void local_merge(uint32_t (&k)[32]) {
  local_stage<4, 5>(k);
  local_stage<3, 5>(k);
  local_stage<2, 5>(k);
  local_stage<1, 5>(k);
  local_stage<0, 5>(k);
}

__global__ void __launch_bounds__(1024) lloyd_rows_kernel(const float* __restrict__ W, int64_t N, int64_t K, int Q,
                                                          int iters, int P, uint16_t* __restrict__ codebooks,
                                                          double* __restrict__ centroids) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // sized by the launch: P / 32 chunks, Q centroids (fit_smem_bytes)
  double* cpre = reinterpret_cast<double*>(smem_raw);            // [P / 32 + 1] exclusive prefix of the chunk sums
  double* c = cpre + (P >> 5) + 1;                               // [Q] centroids
  double* pre = c + Q;                                           // [Q + 1] prefix sum at each cluster boundary
  double* wtot = pre + Q + 1;                                    // [32] warp totals of the scan
  int* edge = reinterpret_cast<int*>(wtot + 32);                 // [Q + 2] cluster boundaries (sorted positions)
  uint32_t* keys = reinterpret_cast<uint32_t*>(edge + Q + 2);    // [P + P / 32], key i at phys(i)
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
  const int Kc = (int)K, chunks = (Kc + 31) >> 5;
  int logP = 10;
  while ((1 << logP) < P) ++logP;                                // P = 32 * nthr = 2^logP >= 1024

  for (int64_t row = blockIdx.x; row < N; row += gridDim.x) {
    const float* w = W + row * K;
    for (int i = tid; i < P; i += nthr) keys[phys(i)] = i < Kc ? key_of(w[i]) : 0xFFFFFFFFu;   // coalesced reads
    __syncthreads();
    uint32_t k[32];
#pragma unroll
    for (int r = 0; r < 32; ++r) k[r] = keys[phys((tid << 5) + r)];
    // runs of 2, 4, 8, 16 inside the thread, directions by the register number
    local_stage<0, 1>(k);
    local_stage<1, 2>(k);
    local_stage<0, 2>(k);
    local_stage<2, 3>(k);
    local_stage<1, 3>(k);
    local_stage<0, 3>(k);
    local_stage<3, 4>(k);
    local_stage<2, 4>(k);
    local_stage<1, 4>(k);
    local_stage<0, 4>(k);
    // phases m = 5 .. logP: runs of 2^m, direction by bit m of the key number (clear in the last phase)
    for (int m = 5; m <= logP; ++m) {
      const uint32_t flip = (((tid << 5) >> m) & 1) ? 0xFFFFFFFFu : 0u;
#pragma unroll
      for (int r = 0; r < 32; ++r) k[r] ^= flip;
      for (int b = m - 1; b >= 10; --b) {          // partner in another warp: through shared memory
        __syncthreads();                            // the previous readers of `keys` are done
#pragma unroll
        for (int r = 0; r < 32; ++r) keys[phys((tid << 5) + r)] = k[r];
        __syncthreads();
        const int partner = (tid ^ (1 << (b - 5))) << 5;
        const bool lower = ((tid >> (b - 5)) & 1) == 0;
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          const uint32_t o = keys[phys(partner + r)];
          k[r] = lower ? min(k[r], o) : max(k[r], o);
        }
      }
      for (int b = (m - 1 < 9 ? m - 1 : 9); b >= 5; --b) {   // partner in another lane: shuffle
        const int d = 1 << (b - 5);
        const bool lower = (lane & d) == 0;
#pragma unroll
        for (int r = 0; r < 32; ++r) {
          const uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, k[r], d);
          k[r] = lower ? min(k[r], o) : max(k[r], o);
        }
      }
      local_merge(k);
#pragma unroll
      for (int r = 0; r < 32; ++r) k[r] ^= flip;
    }
    // the sorted row goes back to shared memory; chunk t = the 32 keys of thread t: its float64 sum, then the scan
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 32; ++r) keys[phys((tid << 5) + r)] = k[r];
    double v = 0.0;
#pragma unroll
    for (int r = 0; r < 32; ++r)
      if ((tid << 5) + r < Kc) v = __dadd_rn(v, value_of(k[r]));
    double incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const double o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl = __dadd_rn(incl, o);
    }
    if (lane == 31) wtot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      double ti = lane < nwarps ? wtot[lane] : 0.0;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const double o = __shfl_up_sync(0xFFFFFFFFu, ti, d);
        if (lane >= d) ti = __dadd_rn(ti, o);
      }
      const double before = __shfl_up_sync(0xFFFFFFFFu, ti, 1);
      wtot[lane] = lane == 0 ? 0.0 : before;      // sum of the warps before this one
    }
    __syncthreads();
    {
      double excl = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
      if (lane == 0) excl = 0.0;
      excl = __dadd_rn(excl, wtot[warp]);
      if (tid < chunks) cpre[tid] = excl;
      if (tid == chunks - 1) cpre[chunks] = __dadd_rn(excl, v);
    }
    // start: linearly interpolated order statistics at (i + 1/2) / Q
    for (int j = tid; j < Q; j += nthr) {
      const double pos = __dmul_rn(__ddiv_rn((double)j + 0.5, (double)Q), (double)(Kc - 1));
      const int lo = (int)floor(pos), hi = min(lo + 1, Kc - 1);
      const double t = __dadd_rn(pos, -(double)lo);
      c[j] = __dadd_rn(__dmul_rn(value_of(keys[phys(lo)]), __dadd_rn(1.0, -t)), __dmul_rn(value_of(keys[phys(hi)]), t));
    }
    __syncthreads();
    for (int it = 0; it < iters; ++it) {
      if (Q - 1 > nwarps) {
        // more cluster boundaries than warps: a thread per boundary (the partial chunk added in index order)
        for (int i = tid; i < Q - 1; i += nthr) {
          const double mid = __dmul_rn(0.5, __dadd_rn(c[i], c[i + 1]));
          int lo = 0, hi = Kc;                      // first sorted position whose value is above mid
          while (lo < hi) {
            const int m = (lo + hi) >> 1;
            if (value_of(keys[phys(m)]) <= mid) lo = m + 1;
            else hi = m;
          }
          double part = 0.0;
          for (int j = lo & ~31; j < lo; ++j) part = __dadd_rn(part, value_of(keys[phys(j)]));
          edge[i + 1] = lo;
          pre[i + 1] = __dadd_rn(cpre[lo >> 5], part);
        }
      } else {
        for (int i = warp; i < Q - 1; i += nwarps) {   // a warp per boundary
          const double mid = __dmul_rn(0.5, __dadd_rn(c[i], c[i + 1]));
          int lo = 0, hi = Kc;                      // first sorted position whose value is above mid
          while (lo < hi) {
            const int m = (lo + hi) >> 1;
            if (value_of(keys[phys(m)]) <= mid) lo = m + 1;
            else hi = m;
          }
          const int base = lo & ~31;
          double part = (base + lane < lo) ? value_of(keys[phys(base + lane)]) : 0.0;
#pragma unroll
          for (int d = 16; d > 0; d >>= 1) part = __dadd_rn(part, __shfl_xor_sync(0xFFFFFFFFu, part, d));
          if (lane == 0) {
            edge[i + 1] = lo;
            pre[i + 1] = __dadd_rn(cpre[lo >> 5], part);
          }
        }
      }
      __syncthreads();
      for (int j = tid; j < Q; j += nthr) {
        const int e0 = j == 0 ? 0 : edge[j], e1 = j == Q - 1 ? Kc : edge[j + 1];
        const double p0 = j == 0 ? 0.0 : pre[j], p1 = j == Q - 1 ? cpre[chunks] : pre[j + 1];
        if (e1 > e0) c[j] = __ddiv_rn(__dadd_rn(p1, -p0), (double)(e1 - e0));
      }
      __syncthreads();
    }
    for (int j = tid; j < Q; j += nthr) {
      if (centroids) centroids[row * Q + j] = c[j];
      const uint32_t stored = float_to_bf16_bits(__double2float_rn(c[j]));
      codebooks[row * Q + j] = (uint16_t)((stored & 0x7FFFu) ? stored : 0u);   // a zero centroid is stored as +0
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------------------------
// Assignment.  For sorted stored centroids the nearest one (ties to the lower, equal centroids to the lowest index)
// is found by counting the midpoints strictly below the value.  The comparison is exact: with s + e = c_i + c_{i+1}
// (s the float64 sum, e its rounding error from the error-free transformation), x lies above the midpoint iff
// 2x > s, or 2x = s and e < 0.
// ---------------------------------------------------------------------------------------------------------------
struct Mid {
  double s, e;
};

__device__ __forceinline__ Mid exact_mid(uint32_t a_bits, uint32_t b_bits) {
  const double a = (double)bf16_bits_to_float(a_bits), b = (double)bf16_bits_to_float(b_bits);
  Mid m;
  m.s = __dadd_rn(a, b);
  const double bb = __dadd_rn(m.s, -a);
  m.e = __dadd_rn(__dadd_rn(a, -__dadd_rn(m.s, -bb)), __dadd_rn(b, -bb));
  return m;
}

__device__ __forceinline__ bool above(double two_x, const Mid& m) {
  return two_x > m.s || (two_x == m.s && m.e < 0.0);
}

// number of midpoints below the value; predicate monotone in i because the centroids are sorted
template <int BITS>
__device__ __forceinline__ int count_below(double two_x, const Mid* mids) {
  if constexpr (BITS <= 2) {
    int n = 0;
#pragma unroll
    for (int i = 0; i < (1 << BITS) - 1; ++i) n += above(two_x, mids[i]) ? 1 : 0;
    return n;
  } else {
    int n = 0;
#pragma unroll
    for (int step = 1 << (BITS - 1); step > 0; step >>= 1)
      if (above(two_x, mids[n + step - 1])) n += step;
    return n;
  }
}

constexpr int kLayoutCanonical = 0, kLayoutTuned = 1, kLayoutPlanes = 2;

// CTA (x, y) takes share y of the output words of tile x (16 rows); the tile's midpoints and its lowest-equal-index
// maps sit in shared memory; a thread builds one 32-bit word of the packed output from the float32 weights that word
// covers.
template <int BITS, int LAYOUT>
__global__ void __launch_bounds__(256) assign_pack_kernel(const float* __restrict__ W,
                                                          const uint16_t* __restrict__ codebooks,
                                                          uint32_t* __restrict__ packed, int64_t N, int64_t K) {
  constexpr int Q = 1 << BITS, PER = 32 / BITS;
  __shared__ Mid mids[16][Q - 1];
  __shared__ uint8_t first[16][Q];
  const int64_t tile = blockIdx.x, wpr = K / PER;
  for (int i = threadIdx.x; i < 16 * (Q - 1); i += blockDim.x) {
    const int r = i / (Q - 1), m = i % (Q - 1);
    const int64_t n = tile * 16 + r;
    if (n < N) mids[r][m] = exact_mid(codebooks[n * Q + m], codebooks[n * Q + m + 1]);
  }
  if (threadIdx.x < 16 && tile * 16 + threadIdx.x < N) {
    const uint16_t* cb = codebooks + (tile * 16 + threadIdx.x) * Q;
    int f = 0;
    first[threadIdx.x][0] = 0;
    for (int i = 1; i < Q; ++i) {
      if (bf16_bits_to_float(cb[i]) != bf16_bits_to_float(cb[i - 1])) f = i;
      first[threadIdx.x][i] = (uint8_t)f;
    }
  }
  __syncthreads();

  // indices of the 8 weights W[n, k0 .. k0 + 8), one per byte
  auto assign8 = [&](int r, int64_t n, int64_t k0, uint32_t& lo, uint32_t& hi) {
    const float4 a = *reinterpret_cast<const float4*>(W + n * K + k0);
    const float4 b = *reinterpret_cast<const float4*>(W + n * K + k0 + 4);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    lo = hi = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      const uint32_t q = first[r][count_below<BITS>(__dmul_rn(2.0, (double)v[t]), mids[r])];
      if (t < 4) lo |= q << (8 * t);
      else hi |= q << (8 * (t - 4));
    }
  };

  if constexpr (LAYOUT == kLayoutPlanes) {
    const int64_t chunks = table_chunks(K);
    const int64_t words = chunks * BITS * 128;
    uint32_t* out = packed + tile * words;
    for (int64_t l = words * blockIdx.y / gridDim.y + threadIdx.x; l < words * (blockIdx.y + 1) / gridDim.y;
         l += blockDim.x) {
      const int64_t unit = l >> 7;
      const int lane = (int)(l & 127) >> 2, q = (int)(l & 3);
      const int plane = (int)(unit % BITS);
      const int64_t chunk = unit / BITS;
      uint32_t word = 0;
#pragma unroll
      for (int bi = 0; bi < 4; ++bi) {
        int r, gl;
        table_unit_coords(lane, 4 * q + bi, r, gl);
        const int64_t n = tile * 16 + r, k0 = (chunk * 32 + gl) * 8;
        if (n < N && k0 < K) {
          uint32_t e[2];
          assign8(r, n, k0, e[0], e[1]);
          uint32_t byte = 0;
#pragma unroll
          for (int t = 0; t < 8; ++t) byte |= ((e[t >> 2] >> ((t & 3) * 8 + plane)) & 1u) << t;
          word |= byte << (8 * bi);
        }
      }
      out[l] = word;
    }
  } else {
    constexpr bool TUNED = LAYOUT == kLayoutTuned;
    const int64_t steps = tuned_steps(wpr);
    const int64_t words = TUNED ? steps * 256 : 16 * wpr;
    for (int64_t l = words * blockIdx.y / gridDim.y + threadIdx.x; l < words * (blockIdx.y + 1) / gridDim.y;
         l += blockDim.x) {
      int r;
      int64_t j;
      if constexpr (TUNED) {
        r = (int)(l >> 4) & 15;
        j = (l >> 8) * 16 + (l & 15);
      } else {
        r = (int)(l / wpr);
        j = l % wpr;
      }
      const int64_t n = tile * 16 + r;
      uint32_t word = 0;
      const bool real = n < N && j < wpr;
      if (real) {
#pragma unroll
        for (int g = 0; g < PER / 8; ++g) {
          uint32_t e[2];
          assign8(r, n, j * PER + g * 8, e[0], e[1]);
#pragma unroll
          for (int t = 0; t < 8; ++t)
            word |= ((e[t >> 2] >> ((t & 3) * 8)) & (uint32_t)(Q - 1)) << field_pos<BITS>(g * 8 + t, TUNED);
        }
      }
      if constexpr (TUNED) packed[tile * words + l] = word;
      else if (real) packed[n * wpr + j] = word;
    }
  }
}

// ---------------------------------------------------------------------------------------------------------------
// Block format: scales, normalised sample, assignment against the shared codebook.
// ---------------------------------------------------------------------------------------------------------------
// One thread per block of 64 weights.  absmean adds the 64 magnitudes in float64 in index order.
template <int MODE>
__global__ void __launch_bounds__(256) block_scales_kernel(const float* __restrict__ W, uint16_t* __restrict__ scales,
                                                           int64_t blocks) {
  int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; b < blocks; b += stride) {
    const float4* p = reinterpret_cast<const float4*>(W + b * 64);
    double acc = 0.0;
    float mx = 0.0f;
#pragma unroll 4
    for (int i = 0; i < 16; ++i) {
      const float4 v = p[i];
      if (MODE == KMQ_LAMBDA_ABSMAX) {
        mx = fmaxf(mx, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
      } else {
        acc = __dadd_rn(acc, (double)fabsf(v.x));
        acc = __dadd_rn(acc, (double)fabsf(v.y));
        acc = __dadd_rn(acc, (double)fabsf(v.z));
        acc = __dadd_rn(acc, (double)fabsf(v.w));
      }
    }
    const float lam = MODE == KMQ_LAMBDA_ABSMAX ? mx : __double2float_rn(__dmul_rn(acc, 1.0 / 64.0));
    uint32_t bits = float_to_bf16_bits(lam);
    if (!(bf16_bits_to_float(bits) > 0.0f)) bits = 0x3F80u;      // a zero scale is stored as 1
    scales[b] = (uint16_t)bits;
  }
}

__device__ __forceinline__ double normalised(float w, uint32_t scale_bits) {
  return __ddiv_rn((double)w, (double)bf16_bits_to_float(scale_bits));
}

__global__ void __launch_bounds__(256) block_sample_kernel(const float* __restrict__ W,
                                                           const uint16_t* __restrict__ scales, int64_t K,
                                                           int64_t stride, int64_t count, float* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  const int64_t f = i * stride, n = f / K, k = f % K;
  out[i] = __double2float_rn(normalised(W[f], scales[n * (K >> 6) + (k >> 6)]));
}

// One thread per 8 consecutive weights (they share a block): BITS output bytes.
template <int BITS>
__global__ void __launch_bounds__(256) block_assign_kernel(const float* __restrict__ W,
                                                           const uint16_t* __restrict__ scales,
                                                           const uint16_t* __restrict__ codebook,
                                                           uint8_t* __restrict__ wq, int64_t groups) {
  constexpr int Q = 1 << BITS;
  __shared__ Mid mids[Q > 1 ? Q - 1 : 1];
  __shared__ uint8_t first[Q];
  for (int i = threadIdx.x; i < Q - 1; i += blockDim.x) mids[i] = exact_mid(codebook[i], codebook[i + 1]);
  if (threadIdx.x == 0) {
    int f = 0;
    first[0] = 0;
    for (int i = 1; i < Q; ++i) {
      if (bf16_bits_to_float(codebook[i]) != bf16_bits_to_float(codebook[i - 1])) f = i;
      first[i] = (uint8_t)f;
    }
  }
  __syncthreads();
  int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; g < groups; g += stride) {
    const float4 a = *reinterpret_cast<const float4*>(W + g * 8);
    const float4 b = *reinterpret_cast<const float4*>(W + g * 8 + 4);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    const uint32_t sb = scales[g >> 3];
    uint64_t bits = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      const double two_x = __dmul_rn(2.0, normalised(v[t], sb));
      int n;
      if constexpr (BITS == 8) {
        n = 0;
#pragma unroll
        for (int step = 128; step > 0; step >>= 1)
          if (above(two_x, mids[n + step - 1])) n += step;
      } else {
        n = count_below<BITS>(two_x, mids);
      }
      bits |= (uint64_t)first[n] << (t * BITS);
    }
    uint8_t* dst = wq + g * BITS;
    if constexpr (BITS == 8) *reinterpret_cast<uint2*>(dst) = make_uint2((uint32_t)bits, (uint32_t)(bits >> 32));
    else if constexpr (BITS == 4) *reinterpret_cast<uint32_t*>(dst) = (uint32_t)bits;
    else if constexpr (BITS == 2) *reinterpret_cast<uint16_t*>(dst) = (uint16_t)bits;
    else *dst = (uint8_t)bits;
  }
}

inline int capped_grid(int64_t items, int threads, int sm_count, int per_sm) {
  int64_t blocks = (items + threads - 1) / threads;
  const int64_t cap = (int64_t)sm_count * per_sm;
  if (blocks > cap) blocks = cap;
  return (int)(blocks < 1 ? 1 : blocks);
}

template <int BITS>
cudaError_t launch_assign_bits(const float* W, const uint16_t* cb, int64_t N, int64_t K, int layout, uint32_t* packed,
                               cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const int64_t tiles = (N + 15) / 16;
  // enough CTAs to fill the machine several times over, each with at least a few words per thread
  int64_t shares = ((int64_t)di->sm_count * 16 + tiles - 1) / tiles;
  const int64_t max_shares = 16 * (K / (32 / BITS)) / 1024;
  if (shares > max_shares) shares = max_shares;
  if (shares < 1) shares = 1;
  if (shares > 65535) shares = 65535;
  const dim3 grid((unsigned)tiles, (unsigned)shares);
  if (layout == KMQ_LAYOUT_CANONICAL) assign_pack_kernel<BITS, kLayoutCanonical><<<grid, 256, 0, s>>>(W, cb, packed, N, K);
  else if (layout == KMQ_LAYOUT_TABLE && BITS != 4)
    assign_pack_kernel<BITS == 4 ? 1 : BITS, kLayoutPlanes><<<grid, 256, 0, s>>>(W, cb, packed, N, K);
  else assign_pack_kernel<BITS, kLayoutTuned><<<grid, 256, 0, s>>>(W, cb, packed, N, K);
  return cudaGetLastError();
}

}  // namespace

size_t fit_smem_bytes(int P, int Q) {
  return (size_t)((P >> 5) + 1 + Q + Q + 1 + 32) * 8 + (size_t)(Q + 2) * 4 + (size_t)(P + P / 32) * 4;
}

bool fit_supports(int64_t K, int bits) { return K >= (int64_t(1) << bits) && K >= 2 && K <= kMaxFitLen; }

cudaError_t launch_kmeans_rows(const float* W, int64_t N, int64_t K, int bits, int iters, uint16_t* codebooks,
                               double* centroids, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  int P = 1024;                      // keys sorted, padded: a power of two, 32 per thread
  while (P < K) P <<= 1;
  const int threads = P / 32;
  const size_t smem = fit_smem_bytes(P, 1 << bits);
  if (cudaError_t e = cudaFuncSetAttribute(lloyd_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)fit_smem_bytes(kMaxFitLen, kMaxCentroids)))
    return e;
  int per_sm = 1;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, lloyd_rows_kernel, threads, smem) != cudaSuccess || per_sm < 1)
    per_sm = 1;
  const int64_t cap = (int64_t)di->sm_count * per_sm;
  const int grid = (int)(N < cap ? N : cap);
  lloyd_rows_kernel<<<grid, threads, smem, s>>>(W, N, K, 1 << bits, iters, P, codebooks, centroids);
  return cudaGetLastError();
}

cudaError_t launch_assign_pack(const float* W, const uint16_t* cb, int64_t N, int64_t K, int bits, int layout,
                               uint32_t* packed, cudaStream_t s) {
  if (bits == 1) return launch_assign_bits<1>(W, cb, N, K, layout, packed, s);
  if (bits == 2) return launch_assign_bits<2>(W, cb, N, K, layout, packed, s);
  return launch_assign_bits<4>(W, cb, N, K, layout, packed, s);
}

cudaError_t launch_block_scales(const float* W, int64_t N, int64_t K, int mode, uint16_t* scales, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const int64_t blocks = N * (K >> 6);
  const int grid = capped_grid(blocks, 256, di->sm_count, 16);
  if (mode == KMQ_LAMBDA_ABSMAX) block_scales_kernel<KMQ_LAMBDA_ABSMAX><<<grid, 256, 0, s>>>(W, scales, blocks);
  else block_scales_kernel<KMQ_LAMBDA_ABSMEAN><<<grid, 256, 0, s>>>(W, scales, blocks);
  return cudaGetLastError();
}

cudaError_t launch_block_sample(const float* W, const uint16_t* scales, int64_t N, int64_t K, int64_t samples,
                                float* out, cudaStream_t s) {
  const int64_t total = N * K, stride = total / samples > 1 ? total / samples : 1;
  int64_t count = (total + stride - 1) / stride;
  if (count > samples) count = samples;
  block_sample_kernel<<<(unsigned)((count + 255) / 256), 256, 0, s>>>(W, scales, K, stride, count, out);
  return cudaGetLastError();
}

cudaError_t launch_block_assign(const float* W, const uint16_t* scales, const uint16_t* codebook, int64_t N, int64_t K,
                                int bits, uint8_t* wq, cudaStream_t s) {
  const DeviceInfo* di = device_info();
  if (!di) return cudaErrorInvalidDevice;
  const int64_t groups = N * (K >> 3);
  const int grid = capped_grid(groups, 256, di->sm_count, 32);
  if (bits == 1) block_assign_kernel<1><<<grid, 256, 0, s>>>(W, scales, codebook, wq, groups);
  else if (bits == 2) block_assign_kernel<2><<<grid, 256, 0, s>>>(W, scales, codebook, wq, groups);
  else if (bits == 4) block_assign_kernel<4><<<grid, 256, 0, s>>>(W, scales, codebook, wq, groups);
  else block_assign_kernel<8><<<grid, 256, 0, s>>>(W, scales, codebook, wq, groups);
  return cudaGetLastError();
}

}  // namespace kmq

using namespace kmq;

namespace {

inline bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline kmq_status st(cudaError_t e) { return e == cudaSuccess ? KMQ_OK : KMQ_ERR_CUDA; }

kmq_status check_fit(int64_t N, int64_t K, int bits, int iters) {
  if (bits != 1 && bits != 2 && bits != 4 && bits != 8) return KMQ_ERR_BITS;
  if (N < 1 || N > (int64_t(1) << 31) || iters < 0 || !fit_supports(K, bits)) return KMQ_ERR_SHAPE;
  return KMQ_OK;
}

kmq_status check_rows(int64_t N, int64_t K, int bits, int layout) {
  if (bits != 1 && bits != 2 && bits != 4) return KMQ_ERR_BITS;
  const int64_t per = 32 / bits;
  if (N < 1 || K < per || (K % per) != 0 || N > (int64_t(1) << 31) || K > (int64_t(1) << 31)) return KMQ_ERR_SHAPE;
  if (layout != KMQ_LAYOUT_CANONICAL && layout != KMQ_LAYOUT_TUNED && layout != KMQ_LAYOUT_TABLE) return KMQ_ERR_LAYOUT;
  return KMQ_OK;
}

kmq_status check_block(int64_t N, int64_t K, int bits) {
  if (bits != 1 && bits != 2 && bits != 4 && bits != 8) return KMQ_ERR_BITS;
  if (N < 1 || K < 64 || (K % 64) != 0 || N > (int64_t(1) << 31) || K > (int64_t(1) << 31)) return KMQ_ERR_SHAPE;
  return KMQ_OK;
}

}  // namespace

extern "C" {

kmq_status kmq_kmeans_rows(const float* W, int64_t N, int64_t K, int bits, int iters, uint16_t* codebooks,
                           double* centroids, void* stream) {
  if (!W || !codebooks) return KMQ_ERR_NULL;
  if (kmq_status s = check_fit(N, K, bits, iters)) return s;
  if (!al16(W) || !al16(codebooks) || !al16(centroids)) return KMQ_ERR_ALIGN;
  return st(launch_kmeans_rows(W, N, K, bits, iters, codebooks, centroids, (cudaStream_t)stream));
}

kmq_status kmq_assign_pack(const float* W, const uint16_t* codebooks, int64_t N, int64_t K, int bits, int layout,
                           uint32_t* packed, void* stream) {
  if (!W || !codebooks || !packed) return KMQ_ERR_NULL;
  if (kmq_status s = check_rows(N, K, bits, layout)) return s;
  if (!al16(W) || !al16(codebooks) || !al16(packed)) return KMQ_ERR_ALIGN;
  return st(launch_assign_pack(W, codebooks, N, K, bits, layout, packed, (cudaStream_t)stream));
}

kmq_status kmq_quantize_rows(const float* W, int64_t N, int64_t K, int bits, int iters, int layout,
                             uint16_t* codebooks, uint32_t* packed, void* stream) {
  if (!W || !codebooks || !packed) return KMQ_ERR_NULL;
  if (kmq_status s = check_rows(N, K, bits, layout)) return s;
  if (kmq_status s = check_fit(N, K, bits, iters)) return s;
  if (!al16(W) || !al16(codebooks) || !al16(packed)) return KMQ_ERR_ALIGN;
  if (launch_kmeans_rows(W, N, K, bits, iters, codebooks, nullptr, (cudaStream_t)stream) != cudaSuccess)
    return KMQ_ERR_CUDA;
  return st(launch_assign_pack(W, codebooks, N, K, bits, layout, packed, (cudaStream_t)stream));
}

kmq_status kmq_block_scales(const float* W, int64_t N, int64_t K, int lambda, uint16_t* scales, void* stream) {
  if (!W || !scales) return KMQ_ERR_NULL;
  if (kmq_status s = check_block(N, K, 1)) return s;
  if (lambda != KMQ_LAMBDA_ABSMAX && lambda != KMQ_LAMBDA_ABSMEAN) return KMQ_ERR_LAYOUT;
  if (!al16(W) || !al16(scales)) return KMQ_ERR_ALIGN;
  return st(launch_block_scales(W, N, K, lambda, scales, (cudaStream_t)stream));
}

int64_t kmq_block_sample_count(int64_t N, int64_t K, int64_t samples) {
  if (check_block(N, K, 1) != KMQ_OK || samples < 1) return 0;
  const int64_t total = N * K, stride = total / samples > 1 ? total / samples : 1;
  const int64_t count = (total + stride - 1) / stride;
  return count < samples ? count : samples;
}

kmq_status kmq_block_sample(const float* W, const uint16_t* scales, int64_t N, int64_t K, int64_t samples, float* out,
                            void* stream) {
  if (!W || !scales || !out) return KMQ_ERR_NULL;
  if (kmq_status s = check_block(N, K, 1)) return s;
  if (samples < 1) return KMQ_ERR_SHAPE;
  if (!al16(W) || !al16(scales) || !al16(out)) return KMQ_ERR_ALIGN;
  return st(launch_block_sample(W, scales, N, K, samples, out, (cudaStream_t)stream));
}

kmq_status kmq_block_assign_pack(const float* W, const uint16_t* scales, const uint16_t* codebook, int64_t N,
                                 int64_t K, int bits, uint8_t* wq, void* stream) {
  if (!W || !scales || !codebook || !wq) return KMQ_ERR_NULL;
  if (kmq_status s = check_block(N, K, bits)) return s;
  if (!al16(W) || !al16(scales) || !al16(codebook) || !al16(wq)) return KMQ_ERR_ALIGN;
  return st(launch_block_assign(W, scales, codebook, N, K, bits, wq, (cudaStream_t)stream));
}

kmq_status kmq_block_quantize(const float* W, int64_t N, int64_t K, int bits, int lambda, int iters, int64_t samples,
                              uint16_t* scales, uint16_t* codebook, uint8_t* wq, float* sample_workspace,
                              void* stream) {
  if (!W || !scales || !codebook || !wq || !sample_workspace) return KMQ_ERR_NULL;
  if (kmq_status s = check_block(N, K, bits)) return s;
  if (lambda != KMQ_LAMBDA_ABSMAX && lambda != KMQ_LAMBDA_ABSMEAN) return KMQ_ERR_LAYOUT;
  const int64_t count = kmq_block_sample_count(N, K, samples);
  if (kmq_status s = check_fit(1, count, bits, iters)) return s;
  if (!al16(W) || !al16(scales) || !al16(codebook) || !al16(wq) || !al16(sample_workspace)) return KMQ_ERR_ALIGN;
  cudaStream_t cs = (cudaStream_t)stream;
  if (launch_block_scales(W, N, K, lambda, scales, cs) != cudaSuccess) return KMQ_ERR_CUDA;
  if (launch_block_sample(W, scales, N, K, samples, sample_workspace, cs) != cudaSuccess) return KMQ_ERR_CUDA;
  if (launch_kmeans_rows(sample_workspace, 1, count, bits, iters, codebook, nullptr, cs) != cudaSuccess)
    return KMQ_ERR_CUDA;
  return st(launch_block_assign(W, scales, codebook, N, K, bits, wq, cs));
}

}  // extern "C"
