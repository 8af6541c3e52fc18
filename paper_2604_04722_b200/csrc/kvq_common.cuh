// Shared device/host definitions of the mixed-precision KV store (sm_100a).
//
// Store geometry.  Precision class c in {0,1,2,3} <-> {2,4,8,16} bits.  A row
// (one token, one KV head, one of K or V) holds 64 elements; its two HALF-ROWS
// (elements 0..31 and 32..63) are 8 << c bytes each and are cut into UNITS of
// 8 bytes (class 0) or 16 bytes (classes 1..3: 1, 2, 4 units per half-row).
// Rows are grouped in TILES of 16 consecutive slots.  The record of a tile is,
// in bytes:
//
//   [K codes : 2 halves x units x 16 slots x unit bytes]
//              unit u of half h of slot t at ((h*units + u)*16 + t) * unit bytes
//   [V codes : same                                    ]
//   [K meta  : 16 slots x 4 B  {scale fp16, zero-point fp16}]   (classes 0..2 only)
//   [V meta  : 16 slots x 4 B                               ]   (classes 0..2 only)
//
// A warp reads a tile with one lane per (slot, half): lanes 0..15 take half 0
// of slots 0..15, lanes 16..31 half 1, so every shared-memory load of a unit
// covers contiguous bytes (no bank conflicts), and a tile is one contiguous
// block (640 / 1152 / 2176 / 4096 bytes, all multiples of 128) that a single
// bulk copy can stage.  Inside a half-row the codes are packed little-endian
// in element order, exactly as in the canonical row (element i in bits
// [(i*b)%8, +b) of byte floor(i*b/8)); half h is bytes [h*8<<c, (h+1)*8<<c) of
// the canonical row.
//
// The tiles of one (layer, sequence, KV head, class) are contiguous, in slot
// order, cap_tiles = ceil(max_ctx/16) of them.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace kvq {

constexpr int kHeadDim = 64;
constexpr int kTileTokens = 16;
constexpr int kNumPools = 4;
constexpr int kMaxSplits = 64;
constexpr int kMaxHidden = 128;   // controller block (W2 is H x H) must fit in shared memory

__host__ __device__ constexpr int pool_bits(int c) { return 2 << c; }            // 2,4,8,16
__host__ __device__ constexpr int pool_chunks(int c) { return 1 << c; }          // 16-byte chunks per canonical row
__host__ __device__ constexpr int pool_has_meta(int c) { return c < 3; }
__host__ __device__ constexpr int pool_half_bytes(int c) { return 8 << c; }      // 8, 16, 32, 64
__host__ __device__ constexpr int pool_unit_bytes(int c) { return c == 0 ? 8 : 16; }
__host__ __device__ constexpr int pool_units(int c) { return pool_half_bytes(c) / pool_unit_bytes(c); }   // 1,1,2,4
__host__ __device__ constexpr int pool_codes_bytes(int c) { return 2 * pool_half_bytes(c) * kTileTokens; }  // per tile, per tensor
__host__ __device__ constexpr int pool_meta_bytes(int c) { return pool_has_meta(c) ? 4 * kTileTokens : 0; }  // per tile, per tensor
__host__ __device__ constexpr int pool_rec_bytes(int c) { return 2 * pool_codes_bytes(c) + 2 * pool_meta_bytes(c); }
__host__ __device__ constexpr int pool_row_bytes(int c) {                        // K+V bytes per (token, KV head)
    return pool_rec_bytes(c) / kTileTokens;                                      // 40, 72, 136, 256
}
// Byte offset, inside one tensor's code block of a tile, of unit u of half h of slot t.
__host__ __device__ constexpr int unit_offset(int c, int h, int u, int t) {
    return ((h * pool_units(c) + u) * kTileTokens + t) * pool_unit_bytes(c);
}
// Byte offset, inside the record, of the {scale, zero-point} pair of slot t (tensor 0 = K, 1 = V).
__host__ __device__ constexpr int meta_offset(int c, int tensor, int t) {
    return 2 * pool_codes_bytes(c) + tensor * pool_meta_bytes(c) + 4 * t;
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
