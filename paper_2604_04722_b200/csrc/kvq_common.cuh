// Shared device/host definitions of the mixed-precision KV store (sm_100a).
//
// Store geometry.  Precision class c in {0,1,2,3} <-> {2,4,8,16} bits.  A row
// (one token, one KV head, one of K or V) holds 64 elements = 16*W(c) bytes of
// codes with W = {1,2,4,8}.  Rows are grouped in TILES of 32 consecutive slots.
// The record of a tile is, in bytes:
//
//   [K codes : W chunks x 32 lanes x 16 B]   chunk j of slot s at j*512 + (s%32)*16
//   [V codes : same                      ]
//   [K meta  : 32 lanes x 4 B  {scale fp16, zero-point fp16}]   (classes 0..2 only)
//   [V meta  : 32 lanes x 4 B                               ]   (classes 0..2 only)
//
// so a warp reads a tile with fully coalesced 16-byte loads, one lane per
// token, and a tile is one contiguous block (1280 / 2304 / 4352 / 8192 bytes)
// that a single bulk copy can stage.  Inside a row the codes are packed
// little-endian: element i in bits [(i*b)%8, +b) of byte floor(i*b/8), and
// chunk j holds bytes [16j, 16j+16) of the row.
//
// The tiles of one (layer, sequence, KV head, class) are contiguous, in slot
// order, cap_tiles = ceil(max_ctx/32) of them.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace kvq {

constexpr int kHeadDim = 64;
constexpr int kTileTokens = 32;
constexpr int kNumPools = 4;
constexpr int kMaxSplits = 64;
constexpr int kMaxHidden = 128;   // controller block (W2 is H x H) must fit in shared memory

__host__ __device__ constexpr int pool_bits(int c) { return 2 << c; }            // 2,4,8,16
__host__ __device__ constexpr int pool_chunks(int c) { return 1 << c; }          // W: 16-byte chunks per row
__host__ __device__ constexpr int pool_has_meta(int c) { return c < 3; }
__host__ __device__ constexpr int pool_codes_bytes(int c) { return 512 * pool_chunks(c); }   // per tile, per tensor
__host__ __device__ constexpr int pool_rec_bytes(int c) {
    return 2 * pool_codes_bytes(c) + (pool_has_meta(c) ? 256 : 0);
}
__host__ __device__ constexpr int pool_row_bytes(int c) {                        // K+V bytes per (token, KV head)
    return pool_rec_bytes(c) / kTileTokens;                                      // 40, 72, 136, 256
}

// Everything a kernel needs to find a row.
struct StoreView {
    uint8_t* pool[kNumPools];     // base of each class's region
    uint32_t* index;              // [layers][batch][max_ctx]   pool<<30 | slot
    uint32_t* flags;              // device flag word
    int layers, batch, kv_heads, q_heads, max_ctx, cap_tiles;
};

__host__ __device__ inline size_t tile_offset(const StoreView& s, int c, int layer, int b, int h, int tile) {
    size_t seq = ((size_t)layer * s.batch + b) * s.kv_heads + h;
    return (seq * (size_t)s.cap_tiles + (size_t)tile) * (size_t)pool_rec_bytes(c);
}

__device__ __forceinline__ int bits_to_class(int bits) {
    return bits == 2 ? 0 : bits == 4 ? 1 : bits == 8 ? 2 : bits == 16 ? 3 : -1;
}

}  // namespace kvq
