// Quantize-append: Q_b of Eq. 24 applied to the new K and V rows, which are then
// appended to the cache (Eq. 4) -- here: written into the pool of their class.
//
// Slot assignment is deterministic: tokens of a sequence are taken in position
// order, slot = fill of the token's pool before the call + number of earlier
// new tokens of the same class.  For more than one 256-token chunk per
// sequence a first launch (k_classify) writes each token's class and a class
// histogram per chunk; the quantize launch sums the histograms of the chunks
// before its own and ranks its own tokens with warp ballots.  Pool fills are
// double-buffered (read `counts_in`, write `counts_out`) so no CTA reads a
// counter another CTA of the same launch writes.
//
// Row quantizer: eight lanes per row, 16 bytes (8 fp16) per lane; min/max by
// three xor-shuffles; fp32 scale with IEEE divide, fp16 round, IEEE reciprocal,
// codes by round-to-nearest-even -- all with explicit _rn intrinsics so the
// result is the same bit pattern on every build.
#pragma once
#include "kvq_common.cuh"
#include "k_controller.cuh"

namespace kvq {

constexpr int kChunkTokens = 256;      // tokens per slot-assignment chunk == threads per CTA

struct AppendParams {
    StoreView store;
    const __half* K;                   // [batch][n_new][kv_heads][64]
    const __half* V;
    const uint8_t* bits;               // [batch][n_new]            (modes 1 and classify<false>)
    const float* feats;                // [batch][n_new][4]         (fused modes)
    const float* ctrl;                 // controller parameter block (fused modes)
    int hidden;
    uint8_t* bits_out;                 // optional [batch][n_new]   (fused modes)
    uint8_t* cls;                      // scratch [batch][n_new] class per token (multi-chunk)
    uint4* hist;                       // scratch [batch][nchunks] class histogram per chunk
    const uint32_t* counts_in;         // [batch][4] of this layer
    uint32_t* counts_out;              // [batch][4] of this layer
    int layer, n_new, pos0, nchunks, heads_per_group;
};

// Class of one token from its bit-width; anything outside {2,4,8,16} is kept as fp16 and flagged.
__device__ __forceinline__ int class_of_bits(int bits, uint32_t* flags) {
    int c = bits_to_class(bits);
    if (c < 0) {
        atomicOr(flags, 1u);
        c = 3;
    }
    return c;
}

// Launch 1 (only when a sequence's new tokens span several chunks).
template <bool FUSED>
__global__ void __launch_bounds__(kChunkTokens)
k_classify(AppendParams p) {
    extern __shared__ float sW[];
    __shared__ uint32_t wtot[kChunkTokens / 32][4];
    const int chunk = blockIdx.x, b = blockIdx.y;
    const int t = chunk * kChunkTokens + threadIdx.x;
    const bool live = t < p.n_new;
    int c = -1;
    if (FUSED) {
        controller_stage(sW, p.ctrl, p.hidden);
        __syncthreads();
        if (live) {
            float4 f = reinterpret_cast<const float4*>(p.feats)[(size_t)b * p.n_new + t];
            float lg[4];
            c = controller_decide_any(sW, p.hidden, f.x, f.y, f.z, f.w, lg);
            if (p.bits_out) p.bits_out[(size_t)b * p.n_new + t] = (uint8_t)pool_bits(c);
        }
    } else if (live) {
        c = class_of_bits(p.bits[(size_t)b * p.n_new + t], p.store.flags);
    }
    if (live) p.cls[(size_t)b * p.n_new + t] = (uint8_t)c;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        uint32_t m = __ballot_sync(0xffffffffu, c == k);
        if (lane == 0) wtot[warp][k] = __popc(m);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint4 h = make_uint4(0, 0, 0, 0);
        for (int w = 0; w < kChunkTokens / 32; ++w) {
            h.x += wtot[w][0]; h.y += wtot[w][1]; h.z += wtot[w][2]; h.w += wtot[w][3];
        }
        p.hist[(size_t)b * p.nchunks + chunk] = h;
    }
}

// Quantize one row held by an 8-lane group (x = this lane's 8 elements) and store it.
// cls: class of the token; slot: its slot in that class's pool; tensor 0 = K, 1 = V.
__device__ __forceinline__ void quantize_store_row(const StoreView& s, uint4 raw, bool valid, int cls, int layer,
                                                   int b, int h, uint32_t slot, int tensor, int sub) {
    const __half2* hp = reinterpret_cast<const __half2*>(&raw);
    float x[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 f = __half22float2(hp[i]);
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
    }
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) {
        mn = fminf(mn, x[i]);
        mx = fmaxf(mx, x[i]);
    }
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, d));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    }
    if (mn == 0.0f) mn = 0.0f;                         // -0 is stored as +0
    if (mx == 0.0f) mx = 0.0f;
    const int bits = cls < 3 ? pool_bits(cls) : 8;     // fp16 rows skip the codes; keep the shifts in range
    const int levels = (1 << bits) - 1;
    const float s32 = __fdiv_rn(__fsub_rn(mx, mn), (float)levels);
    const __half s16 = __float2half_rn(s32);
    const float sf = __half2float(s16);
    const float inv = sf == 0.0f ? 0.0f : __frcp_rn(sf);
    uint32_t lo = 0, hi = 0;                           // this lane's packed codes (up to 64 bits)
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        int c = __float2int_rn(__fmul_rn(__fsub_rn(x[i], mn), inv));
        c = min(max(c, 0), levels);
        int pos = i * bits;                            // < 64 for bits <= 8
        if (pos < 32) lo |= (uint32_t)c << pos;
        else hi |= (uint32_t)c << (pos - 32);
    }
    // pair up 16-bit halves for the 2-bit class (executed by every lane, used by one branch)
    const uint32_t lo_next = __shfl_down_sync(0xffffffffu, lo, 1);
    if (!valid) return;

    const int t = (int)(slot & (kTileTokens - 1));
    uint8_t* rec = s.pool[cls] + tile_offset(s, cls, layer, b, h, (int)(slot / kTileTokens));
    uint8_t* codes = rec + (size_t)tensor * pool_codes_bytes(cls);
    const int half = sub >> 2, q = sub & 3;            // this lane's 8 elements: quarter q of half-row `half`
    switch (cls) {
    case 0:                                            // 2 bytes per lane -> 4-byte words from even lanes
        if ((sub & 1) == 0)
            *reinterpret_cast<uint32_t*>(codes + unit_offset(0, half, 0, t) + (q >> 1) * 4) = (lo & 0xffffu) | (lo_next << 16);
        break;
    case 1:                                            // 4 bytes per lane
        *reinterpret_cast<uint32_t*>(codes + unit_offset(1, half, 0, t) + q * 4) = lo;
        break;
    case 2:                                            // 8 bytes per lane
        *reinterpret_cast<uint2*>(codes + unit_offset(2, half, q >> 1, t) + (q & 1) * 8) = make_uint2(lo, hi);
        break;
    default:                                           // fp16: the lane's 16 input bytes are one unit
        *reinterpret_cast<uint4*>(codes + unit_offset(3, half, q, t)) = raw;
        break;
    }
    if (cls < 3 && sub == 0) {
        uint32_t meta = (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(__float2half_rn(mn)) << 16);
        *reinterpret_cast<uint32_t*>(rec + meta_offset(cls, tensor, t)) = meta;
    }
}

// Launch 2.  MODE 0: classes come from k_classify (several chunks per sequence);
// MODE 1: one chunk, classes from `bits`; MODE 2: one chunk, classes from the controller.
// grid = (nchunks, head_groups, batch), block = 256.
template <int MODE>
__global__ void __launch_bounds__(kChunkTokens)
k_quant_pack(AppendParams p) {
    extern __shared__ float sW[];
    __shared__ uint32_t wtot[kChunkTokens / 32][4];
    __shared__ uint32_t base[4];
    __shared__ uint32_t tok_slot[kChunkTokens];
    const int chunk = blockIdx.x, hg = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = chunk * kChunkTokens + threadIdx.x;
    const bool live = t < p.n_new;
    const size_t tok = (size_t)b * p.n_new + t;

    // ---- class of this thread's token
    int c = -1;
    if (MODE == 2) {
        controller_stage(sW, p.ctrl, p.hidden);
        __syncthreads();
        if (live) {
            float4 f = reinterpret_cast<const float4*>(p.feats)[tok];
            float lg[4];
            c = controller_decide_any(sW, p.hidden, f.x, f.y, f.z, f.w, lg);
            if (p.bits_out && hg == 0) p.bits_out[tok] = (uint8_t)pool_bits(c);
        }
    } else if (MODE == 1) {
        if (live) c = class_of_bits(p.bits[tok], p.store.flags);
    } else {
        if (live) c = p.cls[tok];
    }

    // ---- fill of each pool before this chunk
    if (warp == 0) {
        uint4 h = make_uint4(0, 0, 0, 0);
        if (MODE == 0) {
            for (int cc = lane; cc < chunk; cc += 32) {
                uint4 v = p.hist[(size_t)b * p.nchunks + cc];
                h.x += v.x; h.y += v.y; h.z += v.z; h.w += v.w;
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                h.x += __shfl_xor_sync(0xffffffffu, h.x, d);
                h.y += __shfl_xor_sync(0xffffffffu, h.y, d);
                h.z += __shfl_xor_sync(0xffffffffu, h.z, d);
                h.w += __shfl_xor_sync(0xffffffffu, h.w, d);
            }
        }
        if (lane == 0) {
            const uint32_t* ci = p.counts_in + (size_t)b * 4;
            base[0] = ci[0] + h.x; base[1] = ci[1] + h.y; base[2] = ci[2] + h.z; base[3] = ci[3] + h.w;
        }
    }
    // ---- rank inside the chunk
    uint32_t rank = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        uint32_t m = __ballot_sync(0xffffffffu, c == k);
        if (c == k) rank = __popc(m & ((1u << lane) - 1u));
        if (lane == 0) wtot[warp][k] = __popc(m);
    }
    __syncthreads();
    if (live) {
        uint32_t slot = base[c] + rank;
        for (int w = 0; w < warp; ++w) slot += wtot[w][c];
        uint32_t word = ((uint32_t)c << 30) | slot;
        tok_slot[threadIdx.x] = word;
        if (hg == 0) p.store.index[((size_t)p.layer * p.store.batch + b) * p.store.max_ctx + p.pos0 + t] = word;
    }
    if (hg == 0 && chunk == p.nchunks - 1 && threadIdx.x < 4) {
        uint32_t tot = base[threadIdx.x];
        for (int w = 0; w < kChunkTokens / 32; ++w) tot += wtot[w][threadIdx.x];
        p.counts_out[(size_t)b * 4 + threadIdx.x] = tot;
    }
    __syncthreads();

    // ---- rows: 8 lanes per row, K and V of (token i, head h) together
    const int ntok = min(kChunkTokens, p.n_new - chunk * kChunkTokens);
    const int h0 = hg * p.heads_per_group;
    const int nh = min(p.heads_per_group, p.store.kv_heads - h0);
    const int items = ntok * nh;
    const int group = threadIdx.x >> 3, sub = threadIdx.x & 7;
    const size_t row_stride = kHeadDim;                                  // halves
    for (int r0 = 0; r0 < items; r0 += kChunkTokens / 8) {
        const int r = r0 + group;
        const bool valid = r < items;
        const int i = valid ? r / nh : 0;
        const int h = h0 + (valid ? r % nh : 0);
        const size_t src = (((size_t)b * p.n_new + (size_t)chunk * kChunkTokens + i) * p.store.kv_heads + h) * row_stride;
        uint4 kraw = make_uint4(0, 0, 0, 0), vraw = kraw;
        if (valid) {
            kraw = __ldg(reinterpret_cast<const uint4*>(p.K + src) + sub);
            vraw = __ldg(reinterpret_cast<const uint4*>(p.V + src) + sub);
        }
        const uint32_t word = tok_slot[i];
        const int cls = (int)(word >> 30);
        const uint32_t slot = word & 0x3fffffffu;
        quantize_store_row(p.store, kraw, valid, cls, p.layer, b, h, slot, 0, sub);
        quantize_store_row(p.store, vraw, valid, cls, p.layer, b, h, slot, 1, sub);
    }
}

}  // namespace kvq
