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
// Row quantizer: a warp quantizes one 16-slot tile of one (class, KV head) at a time, with the
// lane mapping of the store (lane l: half-row l/16 of slot l%16), so the tokens of a chunk are
// first grouped by class (a list per class in slot order) and every store of the warp is one
// contiguous run of the tile record.  Min/max in packed fp16 (exact), one xor-16 shuffle, fp32
// scale with IEEE divide, fp16 round, IEEE reciprocal, codes by round-to-nearest-even (adding
// 1.5 * 2^23 rounds a float in [0, 2^22) to an integer exactly as rint does) -- all with explicit
// _rn intrinsics so the result is the same bit pattern on every build.  Codes are packed in the
// float domain (sums of code * 2^(b*i) below 2^16 are exact) or, for bytes, by byte permutes.
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

constexpr float kRoundMagic = 12582912.0f;             // 1.5 * 2^23

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Quantize the half-row this lane holds (raw = its 32 fp16 values = 64 bytes of the input row) with
// class CLS < 3 and store it: the lane's units of the tile's code block `codes`, and (half 0 only)
// the {scale, zero-point} word at `meta`.  Both lanes of a slot (l, l ^ 16) must call together.
template <int CLS>
__device__ __forceinline__ void quantize_store_half_row(const uint4 (&raw)[4], bool active, int half, int t,
                                                        uint8_t* codes, uint8_t* meta) {
    constexpr int BITS = pool_bits(CLS);
    constexpr float LEVELS = (float)((1 << BITS) - 1);
    const __half2* hp = reinterpret_cast<const __half2*>(raw);
    __half2 mn2 = hp[0], mx2 = hp[0];
#pragma unroll
    for (int i = 1; i < 16; ++i) {
        mn2 = __hmin2(mn2, hp[i]);
        mx2 = __hmax2(mx2, hp[i]);
    }
    float mn = fminf(__low2float(mn2), __high2float(mn2));
    float mx = fmaxf(__low2float(mx2), __high2float(mx2));
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 16));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
    if (mn == 0.0f) mn = 0.0f;                         // -0 is stored as +0
    if (mx == 0.0f) mx = 0.0f;
    const float s32 = __fdiv_rn(__fsub_rn(mx, mn), LEVELS);
    const __half s16 = __float2half_rn(s32);
    const float sf = __half2float(s16);
    const float inv = sf == 0.0f ? 0.0f : __frcp_rn(sf);

    // r[i] = clamp(rint((x_i - mn) * inv), 0, LEVELS) as a float; the product is never negative
    float r[32];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float2 f = __half22float2(hp[i]);
        const float v0 = fminf(__fmul_rn(__fsub_rn(f.x, mn), inv), LEVELS);
        const float v1 = fminf(__fmul_rn(__fsub_rn(f.y, mn), inv), LEVELS);
        r[2 * i] = __fadd_rn(v0, kRoundMagic);
        r[2 * i + 1] = __fadd_rn(v1, kRoundMagic);
    }
    if (!active) return;
    if (CLS == 2) {                                    // the code is the low byte of r's bit pattern
        uint32_t w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t lo = prmt(__float_as_uint(r[4 * k]), __float_as_uint(r[4 * k + 1]), 0x0040u);
            const uint32_t hi = prmt(__float_as_uint(r[4 * k + 2]), __float_as_uint(r[4 * k + 3]), 0x0040u);
            w[k] = prmt(lo, hi, 0x5410u);
        }
        *reinterpret_cast<uint4*>(codes + unit_offset(2, half, 0, t)) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(codes + unit_offset(2, half, 1, t)) = make_uint4(w[4], w[5], w[6], w[7]);
    } else {                                           // 16-bit groups summed exactly in fp32
        constexpr int PER = 16 / BITS;                 // elements per 16-bit group: 8 or 4
        constexpr int GROUPS = 32 / PER;               // 4 or 8
        uint32_t g16[GROUPS];
#pragma unroll
        for (int g = 0; g < GROUPS; ++g) {
            float a = 0.f;
#pragma unroll
            for (int e = 0; e < PER; ++e) a = fmaf(__fsub_rn(r[g * PER + e], kRoundMagic), (float)(1 << (BITS * e)), a);
            g16[g] = __float2uint_rn(a);
        }
        if (CLS == 0) {
            *reinterpret_cast<uint2*>(codes + unit_offset(0, half, 0, t)) =
                make_uint2(g16[0] | (g16[1] << 16), g16[2] | (g16[3] << 16));
        } else {
            *reinterpret_cast<uint4*>(codes + unit_offset(1, half, 0, t)) =
                make_uint4(g16[0] | (g16[1] << 16), g16[2] | (g16[3] << 16), g16[4] | (g16[5] << 16),
                           g16[6] | (g16[7] << 16));
        }
    }
    if (half == 0)
        *reinterpret_cast<uint32_t*>(meta) =
            (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(__float2half_rn(mn)) << 16);
}

// Launch 2.  MODE 0: classes come from k_classify (several chunks per sequence);
// MODE 1: one chunk, classes from `bits`; MODE 2: one chunk, classes from the controller.
// grid = (nchunks, head_groups, batch), block = 256.
template <int MODE>
__global__ void __launch_bounds__(kChunkTokens, 2)
k_quant_pack(AppendParams p) {
    extern __shared__ float sW[];
    __shared__ uint32_t wtot[kChunkTokens / 32][4];
    __shared__ uint32_t base[4];
    __shared__ uint8_t list[4][kChunkTokens];         // tokens of the chunk by class, in slot order
    const int chunk = blockIdx.x, hg = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tok_i = chunk * kChunkTokens + threadIdx.x;
    const bool live = tok_i < p.n_new;
    const size_t tok = (size_t)b * p.n_new + tok_i;

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
        for (int w = 0; w < warp; ++w) rank += wtot[w][c];
        list[c][rank] = (uint8_t)threadIdx.x;
        if (hg == 0)
            p.store.index[((size_t)p.layer * p.store.batch + b) * p.store.max_ctx + p.pos0 + tok_i] =
                ((uint32_t)c << 30) | (base[c] + rank);
    }
    uint32_t ncls[4];                                  // tokens of each class in this chunk
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        ncls[k] = 0;
        for (int w = 0; w < kChunkTokens / 32; ++w) ncls[k] += wtot[w][k];
    }
    if (hg == 0 && chunk == p.nchunks - 1 && threadIdx.x < 4)
        p.counts_out[(size_t)b * 4 + threadIdx.x] = base[threadIdx.x] + ncls[threadIdx.x];
    __syncthreads();

    // ---- tiles: class k touches tiles [first[k], first[k] + nt[k]) of its pool
    uint32_t first[4], pre[5];
    pre[0] = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        first[k] = base[k] / kTileTokens;
        const uint32_t nt = ncls[k] ? (base[k] + ncls[k] - 1) / kTileTokens - first[k] + 1 : 0;
        pre[k + 1] = pre[k] + nt;
    }
    const int h0 = hg * p.heads_per_group;
    const int nh = min(p.heads_per_group, p.store.kv_heads - h0);
    const int half = lane >> 4, t = lane & 15;
    // work items (tile tau, head hh), heads fastest, dealt round-robin to the warps
    uint32_t tau = 0;
    int hh = warp;
    while (hh >= nh) {
        hh -= nh;
        ++tau;
    }
    while (tau < pre[4]) {
        const int k = (tau >= pre[1]) + (tau >= pre[2]) + (tau >= pre[3]);
        const uint32_t basek = k == 0 ? base[0] : k == 1 ? base[1] : k == 2 ? base[2] : base[3];
        const uint32_t nk = k == 0 ? ncls[0] : k == 1 ? ncls[1] : k == 2 ? ncls[2] : ncls[3];
        const uint32_t tile = (k == 0 ? first[0] : k == 1 ? first[1] : k == 2 ? first[2] : first[3]) +
                              (tau - (k == 0 ? pre[0] : k == 1 ? pre[1] : k == 2 ? pre[2] : pre[3]));
        const uint32_t r = tile * kTileTokens + t - basek;       // rank of this lane's slot in the chunk (wraps if before)
        const bool active = r < nk;
        const int h = h0 + hh;
        uint4 kraw[4], vraw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) kraw[i] = vraw[i] = make_uint4(0, 0, 0, 0);
        if (active) {
            const int i_tok = list[k][r];
            const size_t src = (((size_t)b * p.n_new + (size_t)chunk * kChunkTokens + i_tok) * p.store.kv_heads + h) * kHeadDim +
                               half * (kHeadDim / 2);
            const uint4* ks = reinterpret_cast<const uint4*>(p.K + src);
            const uint4* vs = reinterpret_cast<const uint4*>(p.V + src);
#pragma unroll
            for (int i = 0; i < 4; ++i) kraw[i] = __ldg(ks + i);
#pragma unroll
            for (int i = 0; i < 4; ++i) vraw[i] = __ldg(vs + i);
        }
        uint8_t* rec = p.store.pool[k] + tile_offset(p.store, k, p.layer, b, h, (int)tile);
        switch (k) {
        case 0:
            quantize_store_half_row<0>(kraw, active, half, t, rec, rec + meta_offset(0, 0, t));
            quantize_store_half_row<0>(vraw, active, half, t, rec + pool_codes_bytes(0), rec + meta_offset(0, 1, t));
            break;
        case 1:
            quantize_store_half_row<1>(kraw, active, half, t, rec, rec + meta_offset(1, 0, t));
            quantize_store_half_row<1>(vraw, active, half, t, rec + pool_codes_bytes(1), rec + meta_offset(1, 1, t));
            break;
        case 2:
            quantize_store_half_row<2>(kraw, active, half, t, rec, rec + meta_offset(2, 0, t));
            quantize_store_half_row<2>(vraw, active, half, t, rec + pool_codes_bytes(2), rec + meta_offset(2, 1, t));
            break;
        default:                                       // fp16: the lane's 64 input bytes are its four units
            if (active) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    *reinterpret_cast<uint4*>(rec + unit_offset(3, half, u, t)) = kraw[u];
                    *reinterpret_cast<uint4*>(rec + pool_codes_bytes(3) + unit_offset(3, half, u, t)) = vraw[u];
                }
            }
            break;
        }
        hh += kChunkTokens / 32;
        while (hh >= nh) {
            hh -= nh;
            ++tau;
        }
    }
}

}  // namespace kvq
