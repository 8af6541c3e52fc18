// Canonical copy of cached tokens, position by position: looks every token up
// through the per-token index word (pool << 30 | slot) and gathers the units (or,
// in the fragment layout, the words and bytes) of
// its rows from the tile records into plain 128-byte rows (packed codes first,
// zero tail) plus {scale, zero-point} pairs.  Used to compare the store with
// other implementations of the quantizer named in Eq. 24.
#pragma once
#include "kvq_common.cuh"

namespace kvq {

struct ExportParams {
    StoreView store;
    int layer, b0, nb, pos0, n;
    uint8_t* bits;          // [nb][n]
    uint32_t* pool_slot;    // [nb][n]
    uint4* k_codes;         // [nb][n][kv_heads][8] (16-byte units)
    uint4* v_codes;
    uint16_t* k_meta;       // [nb][n][kv_heads][2 * scale groups]
    uint16_t* v_meta;
    const uint32_t* counts; // [batch][4] pool fills of the layer (per-channel keys: which windows are complete)
};

// grid = (n, nb), block = 128.
__global__ void __launch_bounds__(128)
k_export(ExportParams p) {
    const int i = blockIdx.x, bi = blockIdx.y, b = p.b0 + bi;
    const StoreView& s = p.store;
    const uint32_t word = s.index[((size_t)p.layer * s.batch + b) * s.max_ctx + p.pos0 + i];
    const int cls = (int)(word >> 30);
    const uint32_t slot = word & 0x3fffffffu;
    const int W = pool_chunks(cls);
    const size_t tok = (size_t)bi * p.n + i;
    if (threadIdx.x == 0) {
        if (p.bits) p.bits[tok] = (uint8_t)pool_bits(cls);
        if (p.pool_slot) p.pool_slot[tok] = word;
    }
    const int t = (int)(slot & (kTileTokens - 1)), tile = (int)(slot / kTileTokens);
    const int items = s.kv_heads * 2 * 8;              // (head, tensor, 16-byte chunk of the canonical row)
    for (int it = threadIdx.x; it < items; it += blockDim.x) {
        const int j = it & 7, tensor = (it >> 3) & 1, h = it >> 4;
        uint4* dst = tensor ? p.v_codes : p.k_codes;
        if (!dst) continue;
        const uint8_t* codes = tile_ptr(s, cls, stream_table(s, cls, p.layer, b, h), (uint32_t)tile, s.groups) +
                               (size_t)tensor * pool_codes_bytes(cls);
        uint4 v = make_uint4(0, 0, 0, 0);
        const bool frag = s.groups == 1 || s.groups == kLayoutPerChannelK;
        // per-channel keys: a key row is packed only once its window of 16 slots is complete; until then it is an fp16 row
        const bool open_window = s.groups == kLayoutPerChannelK && cls < 3 && tensor == 0 &&
                                 (slot | (uint32_t)(kTileTokens - 1)) >= p.counts[(size_t)b * 4 + cls];
        if (open_window) {
            v = reinterpret_cast<const uint4*>(residual_rows(s, cls, p.layer, b, h) + t * kHeadDim)[j];
        } else if (j < W && cls < 3 && frag) {         // fragment layout: K rows word by word, V rows byte by byte
            uint32_t w[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (tensor == 0) {
                    w[k] = *reinterpret_cast<const uint32_t*>(codes + kfrag_word_offset(cls, t, 4 * j + k));
                } else {
                    w[k] = 0;
#pragma unroll
                    for (int b = 0; b < 4; ++b)
                        w[k] |= (uint32_t)codes[vfrag_byte_offset(cls, t, 16 * j + 4 * k + b)] << (8 * b);
                }
            }
            v = make_uint4(w[0], w[1], w[2], w[3]);
        } else if (j < W) {
            if (cls == 0) {                            // the 16-byte row is two 8-byte half-rows
                const uint2 lo = *reinterpret_cast<const uint2*>(codes + unit_offset(0, 0, 0, t));
                const uint2 hi = *reinterpret_cast<const uint2*>(codes + unit_offset(0, 1, 0, t));
                v = make_uint4(lo.x, lo.y, hi.x, hi.y);
            } else {                                   // chunk j = unit j % units of half j / units
                const int units = pool_units(cls);
                v = *reinterpret_cast<const uint4*>(codes + unit_offset(cls, j / units, j % units, t));
            }
        }
        dst[(tok * s.kv_heads + h) * 8 + j] = v;
    }
    const int G = s.groups == 2 ? 2 : 1;               // {scale, zero-point} pairs per row in the export format
    for (int it = threadIdx.x; it < s.kv_heads * 2 * G; it += blockDim.x) {
        const int g = it % G, tensor = (it / G) & 1, h = it / (2 * G);
        uint16_t* dst = tensor ? p.v_meta : p.k_meta;
        if (!dst) continue;
        uint32_t m = 0;
        if (cls < 3 && !(s.groups == kLayoutPerChannelK && tensor == 0)) {      // (per-channel keys have no per-row pair)
            const uint8_t* rec = tile_ptr(s, cls, stream_table(s, cls, p.layer, b, h), (uint32_t)tile, s.groups);
            m = *reinterpret_cast<const uint32_t*>(rec + meta_offset(cls, tensor, t, g, s.groups));
        }
        dst[((tok * s.kv_heads + h) * G + g) * 2 + 0] = (uint16_t)(m & 0xffffu);
        dst[((tok * s.kv_heads + h) * G + g) * 2 + 1] = (uint16_t)(m >> 16);
    }
}

}  // namespace kvq
