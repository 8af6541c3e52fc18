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
// Placement.  All tile records live in one ARENA of 64 KB blocks.  A block belongs to one
// STREAM = (layer, sequence, KV head, class) and holds 100 / 55 / 30 / 16 consecutive tiles of it
// (1600 / 880 / 480 / 256 tokens; the tail of a block that no whole tile fits is unused).  A block
// table per stream lists its blocks in slot order; blocks are handed out by a device-side counter
// when an append first reaches them, so the memory in use follows what was actually stored: the
// sum of the row bytes plus at most one partly filled block per stream.  Block 0 is never handed
// out: writes that find the arena exhausted land there and set KVQ_FLAG_ARENA_FULL.
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
// Layout id g of a cache.  1 = one {scale, zero-point} pair per row (the default); 2 = one pair per half-row (32
// channels), stored as two planes of 16 words per tensor: [K half 0][K half 1][V half 0][V half 1]; 3 = keys
// quantized per CHANNEL over the 16 slots of a tile: [K: 64 channels x {scale, zero-point}][V: 16 slots x {..}].
constexpr int kLayoutPerChannelK = 3;
__host__ __device__ constexpr int pool_kmeta_bytes(int c, int g = 1) {
    return !pool_has_meta(c) ? 0 : g == kLayoutPerChannelK ? 4 * kHeadDim : 4 * kTileTokens * g;
}
__host__ __device__ constexpr int pool_vmeta_bytes(int c, int g = 1) {
    return !pool_has_meta(c) ? 0 : g == kLayoutPerChannelK ? 4 * kTileTokens : 4 * kTileTokens * g;
}
__host__ __device__ constexpr int pool_meta_bytes(int c, int g = 1) { return pool_vmeta_bytes(c, g); }   // per tile, V tensor (and K, layouts 1 and 2)
__host__ __device__ constexpr int pool_rec_bytes(int c, int g = 1) {
    return 2 * pool_codes_bytes(c) + pool_kmeta_bytes(c, g) + pool_vmeta_bytes(c, g);
}
__host__ __device__ constexpr int pool_row_bytes(int c, int g = 1) {             // K+V bytes per (token, KV head)
    return pool_rec_bytes(c, g) / kTileTokens;                                   // 40, 72, 136, 256 (g = 2: 48, 80, 144, 256; g = 3: 52, 84, 148, 256)
}
// Byte offset, inside one tensor's code block of a tile, of unit u of half h of slot t.
__host__ __device__ constexpr int unit_offset(int c, int h, int u, int t) {
    return ((h * pool_units(c) + u) * kTileTokens + t) * pool_unit_bytes(c);
}
// Byte offset, inside the record, of the {scale, zero-point} pair of slot t (tensor 0 = K, 1 = V).
// With two scale groups `half` picks the plane of the half-row.
__host__ __device__ constexpr int meta_offset(int c, int tensor, int t, int half = 0, int g = 1) {
    return 2 * pool_codes_bytes(c) + tensor * pool_kmeta_bytes(c, g) + (g == 2 ? half * 4 * kTileTokens : 0) + 4 * t;
}
// Per-channel keys: the {scale, zero-point} pair of channel i of the tile.
__host__ __device__ constexpr int chan_meta_offset(int c, int i) { return 2 * pool_codes_bytes(c) + 4 * i; }

// ---- Fragment layout of the quantized classes (caches with one scale group per row).
//
// The decode kernel feeds the codes of a 16-slot tile straight into 8-bit integer matrix instructions
// (16 rows x 8 columns per warp; a lane L = 4 g + q holds, of an operand with rows = slots, the four bytes
// 4q .. 4q+3 of row g and of row g + 8).  Both code blocks of a tile record are therefore stored in the
// order in which the lanes of the reading warp load them, so that one 8- or 16-byte load per lane yields
// operand registers without any shuffling:
//
//   K codes  rows = slots, bytes = the row's canonical bytes.  Lane (g, q) holds, for slot g (i = 0) and slot
//            g + 8 (i = 1), the canonical 32-bit words q, q + 4, q + 8, ... of the row (word wq = q + 4 wsel).
//   V codes  rows = channel groups, bytes = SLOTS (the product sums over the tokens of the tile).  Row rho of
//            an operand holds canonical byte(s) of index rho << c .. of the token rows, i.e. channels 4 rho ..
//            4 rho + 3 in every class; lane (g, q) holds, for rho = g (i = 0) and rho = g + 8 (i = 1), the words
//            whose byte j is that canonical byte of slot 4 q + j.
//
// Offsets below are relative to the start of the tensor's code block; the {scale, zero-point} words keep
// their place behind the code blocks.  Caches with two scale groups per row keep the unit layout above.
__host__ __device__ constexpr int frag_lane(int g, int q) { return 4 * g + q; }
// canonical 32-bit word wq of the K row of slot t
__host__ __device__ constexpr int kfrag_word_offset(int c, int t, int wq) {
    const int lane = frag_lane(t & 7, wq & 3), i = t >> 3, wsel = wq >> 2;
    return c == 0   ? lane * 8 + i * 4
           : c == 1 ? lane * 16 + (wsel * 2 + i) * 4
                    : ((wsel >> 1) * 32 + lane) * 16 + ((wsel & 1) * 2 + i) * 4;
}
// canonical byte cb of the V row of slot t
__host__ __device__ constexpr int vfrag_byte_offset(int c, int t, int cb) {
    const int rho = cb >> c, m = cb & ((1 << c) - 1);
    const int lane = frag_lane(rho & 7, t >> 2), i = rho >> 3, j = t & 3;
    return c == 0   ? lane * 8 + i * 4 + j
           : c == 1 ? lane * 16 + (m * 2 + i) * 4 + j
                    : ((m >> 1) * 32 + lane) * 16 + ((m & 1) * 2 + i) * 4 + j;
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may be scheduled
// while the kernel before it in the stream is still running, once every CTA of that kernel has called
// pdl_launch_dependents (or exited); it must call pdl_wait before it touches memory the earlier kernel reads
// or writes.  pdl_wait returns when the earlier kernel has completed and its writes are visible; without the
// attribute both are no-ops.  Only the decode-step kernels use this, to hide each other's launch latency.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

constexpr uint32_t kBlockBytes = 65536;
// Tiles per block: a whole number of ring stages of the decode kernel (10 / 5 / 3 / 1 tiles).
// (with two scale groups the records are 768 / 1280 / 2304 / 4096 bytes: 80 / 50 / 28 / 16 tiles)
// (per-channel keys: 832 / 1344 / 2368 / 4096 bytes: 78 / 48 / 27 / 16 tiles)
__host__ __device__ constexpr uint32_t block_tiles(int c, int g = 1) {
    return g == 2   ? (c == 0 ? 80u : c == 1 ? 50u : c == 2 ? 28u : 16u)
           : g == 3 ? (c == 0 ? 78u : c == 1 ? 48u : c == 2 ? 27u : 16u)
                    : (c == 0 ? 100u : c == 1 ? 55u : c == 2 ? 30u : 16u);
}
// Per-channel keys: the fp16 key rows of the open (incomplete) window of every quantized stream wait here until the
// window fills: [stream][class 0..2][slot 0..15][64].
constexpr size_t kResidualStreamHalves = 3 * kTileTokens * kHeadDim;
constexpr uint32_t kFlagArenaFull = 4u;

// Everything a kernel needs to find a row.
struct StoreView {
    uint8_t* arena;               // blocks of kBlockBytes
    uint32_t* table;              // [streams][table_stride] block ids, class c at table_off[c]
    uint32_t* arena_used;         // blocks handed out so far (block ids are 1 + the old value)
    uint32_t arena_blocks;        // capacity in blocks, block 0 included
    uint32_t table_stride, table_off[kNumPools];
    int groups;                   // layout id: 1 or 2 scale groups per row, or kLayoutPerChannelK
    __half* kres;                 // per-channel keys: residual rows (nullptr otherwise)
    __half* kres_old;             // ... and a copy of the current layer's, taken before a multi-token append
    uint32_t* index;              // [layers][batch][max_ctx]   pool<<30 | slot
    uint32_t* flags;              // device flag word
    int layers, batch, kv_heads, q_heads, max_ctx, cap_tiles;
};

// The block-table row of class c of stream (layer, b, h).
__host__ __device__ inline uint32_t* stream_table(const StoreView& s, int c, int layer, int b, int h) {
    const size_t stream = ((size_t)layer * s.batch + b) * s.kv_heads + h;
    return s.table + stream * s.table_stride + s.table_off[c];
}
// Address of tile `tile` of a stream whose table row is `tab`.
__device__ __forceinline__ uint8_t* tile_ptr(const StoreView& s, int c, const uint32_t* tab, uint32_t tile, int g = 1) {
    const uint32_t bt = block_tiles(c, g);
    const uint32_t blk = tile / bt;
    return s.arena + (size_t)tab[blk] * kBlockBytes + (size_t)(tile - blk * bt) * (uint32_t)pool_rec_bytes(c, g);
}
// Hand out `n` consecutive blocks; returns the id of the first (0 = the arena is exhausted: flagged).
__device__ __forceinline__ uint32_t arena_take(const StoreView& s, uint32_t n) {
    const uint32_t first = 1u + atomicAdd(s.arena_used, n);
    if (first + n > s.arena_blocks) {
        atomicOr(s.flags, kFlagArenaFull);
        return 0u;
    }
    return first;
}
// Residual rows of class c of stream (layer, b, h).
__host__ __device__ inline __half* residual_rows(const StoreView& s, int c, int layer, int b, int h) {
    const size_t stream = ((size_t)layer * s.batch + b) * s.kv_heads + h;
    return s.kres + stream * kResidualStreamHalves + (size_t)c * kTileTokens * kHeadDim;
}
// The copy of the residual rows of class c of stream (b, h) of the layer being appended to (see kres_old).
__host__ __device__ inline const __half* residual_rows_before(const StoreView& s, int c, int b, int h) {
    return s.kres_old + ((size_t)b * s.kv_heads + h) * kResidualStreamHalves + (size_t)c * kTileTokens * kHeadDim;
}
// Blocks a stream of class c needs for n tokens.
__host__ __device__ constexpr uint32_t blocks_for(int c, uint32_t n, int g = 1) {
    return ((n + kTileTokens - 1) / kTileTokens + block_tiles(c, g) - 1) / block_tiles(c, g);
}

__device__ __forceinline__ int bits_to_class(int bits) {
    return bits == 2 ? 0 : bits == 4 ? 1 : bits == 8 ? 2 : bits == 16 ? 3 : -1;
}

}  // namespace kvq
