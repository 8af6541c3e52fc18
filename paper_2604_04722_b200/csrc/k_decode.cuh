// Decode-step attention over the mixed-precision cache (Eq. 5):
//   a = Softmax(q K^T / sqrt(d_k)) V,   K, V dequantized on the fly.
//
// Softmax attention does not depend on the order of the cached tokens, so the
// kernel never touches the per-token index: it walks each precision pool of a
// (sequence, KV head) front to back.  The sequence is cut into `splits` parts
// (every part takes the same fraction of every pool, hence the same bytes);
// each CTA keeps an online softmax in fp32 and emits (m, l, o[64]); a second
// kernel merges the parts.
//
// Work layout inside a CTA: one lane per token (a warp reads one 32-token tile
// with coalesced 16-byte loads), so the q.k dot product needs no shuffles and
// the output accumulators are per-lane partial sums reduced once at the end.
//
// Dequantization is hoisted out of the inner loops:
//   q.khat = s_k * sum_i q_i c_i + z_k * sum_i q_i
//   sum_t p_t vhat_t = sum_t (p_t s_t) c_t + sum_t p_t z_t
// and the integer codes enter the fp32 FMAs without any int->float conversion:
// a bit field of a packed word that lies inside bits [0,24) of a 32-bit word,
// read as an fp32 bit pattern, IS the number code * 2^(k-149) (subnormal /
// first-binade encoding is linear), so one AND per element isolates it and the
// power of two is folded into a pre-scaled copy of q (for K) or into the
// accumulator's exponent (for V).  Products stay in the normal range, so the
// arithmetic is exact fp32 FMA work: ~2 issue slots per cached element.
#pragma once
#include "kvq_common.cuh"

namespace kvq {

constexpr int kDecodeThreads = 128;
constexpr int kDecodeWarps = kDecodeThreads / 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleSlack = 8.0f;            // the running maximum may lag by 2^8 before a rescale
constexpr float kNegBig = -1.0e30f;

struct DecodeParams {
    StoreView store;
    const uint32_t* counts;        // [batch][4] pool fills of this layer
    const __half* Q;               // [batch][q_heads][64]
    __half* O;                     // [batch][q_heads][64]
    float* part_o;                 // [batch][q_heads][splits][64]  unnormalised
    float2* part_ml;               // [batch][q_heads][splits]      (m in log2 units, l)
    int layer, splits, group;      // group = q_heads / kv_heads
};

__device__ __forceinline__ float pow2f(int e) { return __int_as_float((127 + e) << 23); }

// Exponent offset of element e (0-based inside its 32-bit word) for BITS-wide codes:
// the field sits at bit k = e*BITS of the word, or of (word >> 8) when it would cross bit 24.
template <int BITS>
__device__ __forceinline__ constexpr int field_pos(int e) {
    return (e * BITS + BITS <= 24) ? e * BITS : (BITS == 8 ? 0 : e * BITS - 8);
}

// The code of element e of word w as an fp32 number scaled by 2^(field_pos - 149).
template <int BITS>
__device__ __forceinline__ float field_as_float(uint32_t w, uint32_t w_shr8, int e) {
    constexpr uint32_t mask = (1u << BITS) - 1u;
    const int k = e * BITS;
    if (k + BITS <= 24) return __uint_as_float(w & (mask << k));
    if (BITS == 8) return __uint_as_float(w >> 24);
    return __uint_as_float(w_shr8 & (mask << (k - 8)));
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, d));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

struct Softmax {
    float m, l, bsum;              // running max (log2 units), sum of p, sum of p * zero-point
};

// Fold a tile's logits into the running state and return this lane's p.
__device__ __forceinline__ float softmax_step(Softmax& st, float (&acc)[kHeadDim], float y) {
    const float tmax = warp_max(y);
    if (tmax > st.m + kRescaleSlack) {                 // warp-uniform
        const float f = exp2f(st.m - tmax);
        st.m = tmax;
        st.l *= f;
        st.bsum *= f;
#pragma unroll
        for (int j = 0; j < kHeadDim; ++j) acc[j] *= f;
    }
    const float p = exp2f(y - st.m);
    st.l += p;
    return p;
}

// Walk the tiles [lo, hi) of one quantized pool that belong to this warp.
template <int CLS>
__device__ __forceinline__ void walk_quantized(const uint8_t* __restrict__ base, int first, int hi, uint32_t cnt,
                                               int lane, const float* q_s, float sumq, Softmax& st,
                                               float (&acc)[kHeadDim]) {
    constexpr int BITS = pool_bits(CLS), W = pool_chunks(CLS), REC = pool_rec_bytes(CLS);
    constexpr int EPW = 32 / BITS;                     // elements per 32-bit word
    constexpr int EPC = 4 * EPW;                       // elements per 16-byte chunk
    float qk[kHeadDim];
#pragma unroll
    for (int i = 0; i < kHeadDim; ++i) {
        qk[i] = q_s[i] * pow2f(100 - field_pos<BITS>(i % EPW));
        acc[i] *= pow2f(field_pos<BITS>(i % EPW) - 49);           // into this pool's exponent domain
    }
    for (int t = first; t < hi; t += kDecodeWarps) {
        const uint8_t* rec = base + (size_t)t * REC;
        const bool valid = (uint32_t)(t * kTileTokens + lane) < cnt;
        // ---- K: sum_i q_i c_i
        float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < W; ++j) {
            const uint4 w4 = __ldg(reinterpret_cast<const uint4*>(rec + j * 512) + lane);
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                const uint32_t hi8 = w[wi] >> 8;
#pragma unroll
                for (int e = 0; e < EPW; ++e)
                    d[wi] = fmaf(field_as_float<BITS>(w[wi], hi8, e), qk[j * EPC + wi * EPW + e], d[wi]);
            }
        }
        const uint32_t kmeta = __ldg(reinterpret_cast<const uint32_t*>(rec + 2 * W * 512) + lane);
        const uint32_t vmeta = __ldg(reinterpret_cast<const uint32_t*>(rec + 2 * W * 512 + 128) + lane);
        const float sk = __half2float(__ushort_as_half((unsigned short)(kmeta & 0xffffu)));
        const float zk = __half2float(__ushort_as_half((unsigned short)(kmeta >> 16)));
        const float dot = (d[0] + d[1]) + (d[2] + d[3]);
        float y = fmaf(sk * pow2f(49), dot, zk * sumq) * (0.125f * kLog2e);
        y = valid ? y : -INFINITY;
        const float p = softmax_step(st, acc, y);
        // ---- V: acc_j += (p s_v) c_j, and sum p z_v on the side
        const float sv = __half2float(__ushort_as_half((unsigned short)(vmeta & 0xffffu)));
        const float zv = __half2float(__ushort_as_half((unsigned short)(vmeta >> 16)));
        const float wv = (p * sv) * pow2f(100);
        st.bsum = fmaf(p, zv, st.bsum);
#pragma unroll
        for (int j = 0; j < W; ++j) {
            const uint4 w4 = __ldg(reinterpret_cast<const uint4*>(rec + W * 512 + j * 512) + lane);
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                const uint32_t hi8 = w[wi] >> 8;
#pragma unroll
                for (int e = 0; e < EPW; ++e) {
                    const int i = j * EPC + wi * EPW + e;
                    acc[i] = fmaf(field_as_float<BITS>(w[wi], hi8, e), wv, acc[i]);
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kHeadDim; ++i) acc[i] *= pow2f(49 - field_pos<BITS>(i % EPW));   // back to plain values
}

// The fp16 pool: rows are stored unchanged.
__device__ __forceinline__ void walk_fp16(const uint8_t* __restrict__ base, int first, int hi, uint32_t cnt, int lane,
                                          const float* q_s, Softmax& st, float (&acc)[kHeadDim]) {
    constexpr int W = pool_chunks(3), REC = pool_rec_bytes(3);
    for (int t = first; t < hi; t += kDecodeWarps) {
        const uint8_t* rec = base + (size_t)t * REC;
        const bool valid = (uint32_t)(t * kTileTokens + lane) < cnt;
        float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < W; ++j) {
            const uint4 w4 = __ldg(reinterpret_cast<const uint4*>(rec + j * 512) + lane);
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[wi]));
                d[wi] = fmaf(f.x, q_s[j * 8 + wi * 2], d[wi]);
                d[wi] = fmaf(f.y, q_s[j * 8 + wi * 2 + 1], d[wi]);
            }
        }
        float y = ((d[0] + d[1]) + (d[2] + d[3])) * (0.125f * kLog2e);
        y = valid ? y : -INFINITY;
        const float p = softmax_step(st, acc, y);
#pragma unroll
        for (int j = 0; j < W; ++j) {
            uint4 w4 = __ldg(reinterpret_cast<const uint4*>(rec + W * 512 + j * 512) + lane);
            if (!valid) w4 = make_uint4(0, 0, 0, 0);               // stale bytes may hold anything
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[wi]));
                acc[j * 8 + wi * 2] = fmaf(p, f.x, acc[j * 8 + wi * 2]);
                acc[j * 8 + wi * 2 + 1] = fmaf(p, f.y, acc[j * 8 + wi * 2 + 1]);
            }
        }
    }
}

// grid = (splits, q_heads, batch), block = 128.
__global__ void __launch_bounds__(kDecodeThreads)
k_decode_split(DecodeParams P) {
    __shared__ float q_s[kHeadDim];
    __shared__ float red_o[kDecodeWarps][kHeadDim];
    __shared__ float2 red_ml[kDecodeWarps];
    const int split = blockIdx.x, qh = blockIdx.y, b = blockIdx.z;
    const int kvh = qh / P.group;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x < kHeadDim)
        q_s[threadIdx.x] = __half2float(P.Q[((size_t)b * P.store.q_heads + qh) * kHeadDim + threadIdx.x]);
    __syncthreads();
    float sumq = 0.f;
#pragma unroll
    for (int i = 0; i < kHeadDim; ++i) sumq += q_s[i];

    Softmax st = {kNegBig, 0.f, 0.f};
    float acc[kHeadDim];
#pragma unroll
    for (int i = 0; i < kHeadDim; ++i) acc[i] = 0.f;

    const uint32_t* cnt = P.counts + (size_t)b * 4;
    int rr = 0;                                        // tiles handed out so far (mod warps): round robin
#pragma unroll
    for (int c = 0; c < kNumPools; ++c) {
        const uint32_t n = cnt[c];
        const int ntiles = (int)((n + kTileTokens - 1) / kTileTokens);
        const int lo = (int)((long long)ntiles * split / P.splits);
        const int hi = (int)((long long)ntiles * (split + 1) / P.splits);
        const int first = lo + ((warp - rr) & (kDecodeWarps - 1));
        rr = (rr + (hi - lo)) & (kDecodeWarps - 1);
        if (first >= hi) continue;                     // warp-uniform
        const uint8_t* base = P.store.pool[c] + tile_offset(P.store, c, P.layer, b, kvh, 0);
        if (c == 0) walk_quantized<0>(base, first, hi, n, lane, q_s, sumq, st, acc);
        else if (c == 1) walk_quantized<1>(base, first, hi, n, lane, q_s, sumq, st, acc);
        else if (c == 2) walk_quantized<2>(base, first, hi, n, lane, q_s, sumq, st, acc);
        else walk_fp16(base, first, hi, n, lane, q_s, st, acc);
    }

    // ---- reduce the per-lane partial sums: after five halving steps lane L holds elements 2L, 2L+1
    float r32[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const bool up = lane & 16;
        const float keep = up ? acc[j + 32] : acc[j], send = up ? acc[j] : acc[j + 32];
        r32[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
    float r16[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const bool up = lane & 8;
        const float keep = up ? r32[j + 16] : r32[j], send = up ? r32[j] : r32[j + 16];
        r16[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
    float r8[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const bool up = lane & 4;
        const float keep = up ? r16[j + 8] : r16[j], send = up ? r16[j] : r16[j + 8];
        r8[j] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    float r4[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const bool up = lane & 2;
        const float keep = up ? r8[j + 4] : r8[j], send = up ? r8[j] : r8[j + 4];
        r4[j] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    }
    float r2[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const bool up = lane & 1;
        const float keep = up ? r4[j + 2] : r4[j], send = up ? r4[j] : r4[j + 2];
        r2[j] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
    }
    const float l_w = warp_sum(st.l);
    const float b_w = warp_sum(st.bsum);
    red_o[warp][2 * lane] = r2[0] + b_w;
    red_o[warp][2 * lane + 1] = r2[1] + b_w;
    if (lane == 0) red_ml[warp] = make_float2(st.m, l_w);
    __syncthreads();

    // ---- combine the warps and emit this split's partial
    if (threadIdx.x < kHeadDim) {
        float M = red_ml[0].x;
#pragma unroll
        for (int w = 1; w < kDecodeWarps; ++w) M = fmaxf(M, red_ml[w].x);
        float L = 0.f, o = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            const float f = exp2f(red_ml[w].x - M);
            L = fmaf(red_ml[w].y, f, L);
            o = fmaf(red_o[w][threadIdx.x], f, o);
        }
        const size_t unit = ((size_t)b * P.store.q_heads + qh) * P.splits + split;
        P.part_o[unit * kHeadDim + threadIdx.x] = o;
        if (threadIdx.x == 0) P.part_ml[unit] = make_float2(M, L);
    }
}

// Merge the splits: M = max m_j, l = sum l_j 2^(m_j-M), O = sum o_j 2^(m_j-M) / l.
// grid = batch*q_heads, block = 64.
__global__ void __launch_bounds__(kHeadDim)
k_decode_merge(DecodeParams P) {
    const size_t unit0 = (size_t)blockIdx.x * P.splits;
    float M = kNegBig;
    for (int s = 0; s < P.splits; ++s) M = fmaxf(M, P.part_ml[unit0 + s].x);
    float L = 0.f, o = 0.f;
    for (int s = 0; s < P.splits; ++s) {
        const float2 ml = P.part_ml[unit0 + s];
        const float f = exp2f(ml.x - M);
        L = fmaf(ml.y, f, L);
        o = fmaf(P.part_o[(unit0 + s) * kHeadDim + threadIdx.x], f, o);
    }
    P.O[(size_t)blockIdx.x * kHeadDim + threadIdx.x] = __float2half_rn(o / L);
}

}  // namespace kvq
