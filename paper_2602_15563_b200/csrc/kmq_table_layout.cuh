// KMQ_LAYOUT_TABLE: the packed layout read by the activation-table kernel (b = 1, 2; b = 4 is stored as in the
// tuned layout).
//
// The index bits are stored as bit planes, one byte per group of 8 consecutive weights of a row: bit t of the byte
// of plane p, row n, group g is bit p of idx[n, 8g + t].  Rows are grouped in tiles of 16 and a row's groups in
// chunks of 32 (256 weights); plane p of chunk c of tile T is one contiguous 512-byte unit at byte offset
//   ((T * chunks + c) * bits + p) * 512,          chunks = ceil(K / 256),
// so a tile's whole K range is contiguous.  Inside a unit, lane L = 2 * (n % 16) + (g % 2) of a warp owns the 16
// bytes [16 L, 16 L + 16): byte i of lane (a, r) = (L & 1, L >> 1) holds group  a + 2 * ((r + i) % 16)  of the
// chunk.  The rotation by the row makes the 32 lanes of a warp address 32 different groups at every step i, which is
// what keeps the kernel's table lookups free of shared-memory bank conflicts.  Rows beyond N and groups beyond K are
// zero padding.
#pragma once
#include <stdint.h>

namespace kmq {

constexpr int kTableChunkK = 256;     // weights of one row per chunk
constexpr int kTableUnitBytes = 512;  // one plane of one chunk of one 16-row tile

__host__ __device__ inline int64_t table_chunks(int64_t K) { return (K + kTableChunkK - 1) / kTableChunkK; }
__host__ __device__ inline int64_t table_tiles(int64_t N) { return (N + 15) >> 4; }
__host__ __device__ inline int64_t table_total_bytes(int64_t N, int64_t K, int bits) {
  return table_tiles(N) * table_chunks(K) * bits * kTableUnitBytes;
}

// Byte offset of the byte that holds plane `plane` of weights 8g .. 8g+7 of row n (g = k / 8).
__host__ __device__ inline int64_t table_byte_offset(int64_t n, int64_t g, int plane, int64_t chunks, int bits) {
  const int64_t tile = n >> 4, chunk = g >> 5;
  const int r = (int)(n & 15), gl = (int)(g & 31);
  const int a = gl & 1, t = gl >> 1;
  const int lane = 2 * r + a, i = (t - r) & 15;
  return ((tile * chunks + chunk) * bits + plane) * kTableUnitBytes + lane * 16 + i;
}

// Inverse, inside a unit: byte `i` of lane `lane` -> row within the tile and group within the chunk.
__host__ __device__ inline void table_unit_coords(int lane, int i, int& row_in_tile, int& group_in_chunk) {
  const int a = lane & 1, r = lane >> 1;
  row_in_tile = r;
  group_in_chunk = a + 2 * ((r + i) & 15);
}

}  // namespace kmq
