// Quantize-append (Q_b of Eq. 24, append of Eq. 4) for caches with one {scale, zero-point} pair per row, whose
// code blocks are stored in the operand order of the decode kernel (the fragment layout of kvq_common.cuh).
//
// Ownership.  A warp quantizes one whole 16-slot tile of one (class, KV head) at a time and writes the record
// with contiguous 8/16-byte stores straight from registers.  For that every tile must belong to exactly one
// CTA although the tokens of a class do not stop at chunk borders: the CTA of a chunk owns the tiles of class k
// whose FIRST slot one of the chunk's own tokens takes, and fetches the up to 15 tokens that complete its last
// tile from the chunks that follow (a forward scan over the class bytes that the classify launch left behind).
// Tokens at the start of a chunk that fall into a tile begun by an earlier chunk are left to that chunk.  Only
// the tile that an EARLIER APPEND CALL left partly filled is special: the first chunk owns it and blends its
// new slots into the words already stored (it is the only writer of the stream during the call).
//
// Lane mapping (lane L = 4 g + q, the reading warp's):
//   K: lane (g, q) quantizes, of the rows of slots g and g + 8, the elements of the canonical words q, q + 4, ...
//      that it will store (2-bit: one word of 16 elements, 4-bit: two words of 8, 8-bit: four words of 4);
//      the row's minimum and maximum meet through two xor-shuffles inside the quad.
//   V: lane (g, q) quantizes elements 4g .. 4g+3 and 32+4g .. 32+4g+3 of the rows of slots 4q .. 4q+3 (the
//      bytes of its words); a row's minimum and maximum meet through three xor-shuffles over g.
// The arithmetic per element is the row quantizer's (k_append.cuh): fl(fl(fl(x - mn) * inv) + 1.5 * 2^23), the
// codes packed by adding shifted bit patterns.
#pragma once
#include "k_append.cuh"

#ifndef KVQ_APPEND_FRAG_MIN_CTAS
#define KVQ_APPEND_FRAG_MIN_CTAS 2
#endif
#ifndef KVQ_APPEND_FRAG_DEPTH
#define KVQ_APPEND_FRAG_DEPTH 2
#endif

namespace kvq {

constexpr int kFragDepth = KVQ_APPEND_FRAG_DEPTH;      // items whose input rows are in flight per warp

// Input stage of a work item in shared memory: [tensor][slot 0..15][piece 0..7] 16-byte pieces, the piece index
// xor-ed with a function of the slot so that every read pattern below (and the fp16 copy) is free of bank
// conflicts: f(s) = 5 s0 ^ 2 s1 ^ 3 s2 ^ 4 s3 over the bits of s.
__host__ __device__ constexpr int stage_swizzle(int s) {
    return ((s & 1) ? 5 : 0) ^ ((s & 2) ? 2 : 0) ^ ((s & 4) ? 3 : 0) ^ ((s & 8) ? 4 : 0);
}
__device__ __forceinline__ int stage_piece_offset(int s, int p) { return ((s << 3) + (p ^ stage_swizzle(s))) << 4; }
constexpr int kStageTensorBytes = kTileTokens * kHeadDim * 2;            // 2 KB: 16 rows of one tensor
constexpr int kFragStageBytes = 2 * kStageTensorBytes;                   // K rows, then V rows
constexpr size_t kFragRingBytes = (size_t)(kChunkTokens / 32) * kFragDepth * kFragStageBytes;

// 16-byte async copy that writes zeros when `live` is false (the source is not read then).
__device__ __forceinline__ void cp_async16_or_zero(void* smem_dst, const void* gmem_src, bool live) {
    const int n = live ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
                 "l"(gmem_src), "r"(n)
                 : "memory");
}

// {scale fp16, reciprocal, minimum} of a row from its minimum and maximum (the row quantizer's set-up).
struct RowScale {
    uint32_t meta;                 // {scale, zero-point} fp16 bit patterns
    float inv, mn;
    bool tiny;                     // subnormal scale: the quotient may exceed the top code and is clamped
};
template <int CLS>
__device__ __forceinline__ RowScale row_scale(float mn, float mx) {
    constexpr float LEVELS = (float)((1 << pool_bits(CLS)) - 1);
    if (mn == 0.0f) mn = 0.0f;                         // -0 is stored as +0
    if (mx == 0.0f) mx = 0.0f;
    const float s32 = __fdiv_rn(__fsub_rn(mx, mn), LEVELS);
    const __half s16 = __float2half_rn(s32);
    const float sf = __half2float(s16);
    RowScale r;
    r.inv = sf == 0.0f ? 0.0f : __frcp_rn(sf);
    r.mn = mn;
    r.meta = (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(__float2half_rn(mn)) << 16);
    r.tiny = sf != 0.0f && sf < 6.103515625e-05f;
    return r;
}

// (min, -max) of the 2 n fp16 values in h[0..n), as one half2: both halves then reduce with the same min.
template <int N>
__device__ __forceinline__ __half2 min_negmax(const __half2 (&h)[N]) {
    __half2 mn2 = h[0], mx2 = h[0];
#pragma unroll
    for (int i = 1; i < N; ++i) {
        mn2 = __hmin2(mn2, h[i]);
        mx2 = __hmax2(mx2, h[i]);
    }
    const __half mn = __hmin(__low2half(mn2), __high2half(mn2)), mx = __hmax(__low2half(mx2), __high2half(mx2));
    return __halves2half2(mn, __hneg(mx));
}
__device__ __forceinline__ __half2 shfl_min2(__half2 v, int lane_xor) {
    uint32_t u = *reinterpret_cast<uint32_t*>(&v);
    u = __shfl_xor_sync(0xffffffffu, u, lane_xor);
    return __hmin2(v, *reinterpret_cast<__half2*>(&u));
}

// Code bit patterns of two values: 0x4B400000 + code each (see pack_codes in k_append.cuh).
template <int CLS, bool CLAMP>
__device__ __forceinline__ void code_pair(__half2 h, float mn, float inv, uint32_t& b0, uint32_t& b1) {
    constexpr float LEVELS = (float)((1 << pool_bits(CLS)) - 1);
    const float2 f = __half22float2(h);
    float r0, r1;
    if (CLAMP) {
        r0 = __fadd_rn(fminf(__fmul_rn(__fsub_rn(f.x, mn), inv), LEVELS), kRoundMagic);
        r1 = __fadd_rn(fminf(__fmul_rn(__fsub_rn(f.y, mn), inv), LEVELS), kRoundMagic);
    } else {
        quantize_pair(f.x, f.y, mn, inv, kRoundMagic, r0, r1);
    }
    b0 = __float_as_uint(r0);
    b1 = __float_as_uint(r1);
}

// ---- K side of one tile.  stage: the 16 K rows (2 KB, swizzled).  Returns the lane's words of the K code block in
// store order (see kfrag_word_offset) and, in lanes q < 2, the {scale, zero-point} word of slot g + 8 q.
template <int CLS>
struct FragK {
    static constexpr int BITS = pool_bits(CLS), EPW = 32 / BITS, WT = 16 / EPW, NW = 2 * WT;     // words per token / per lane
    // position of token i's word wsel in the lane's store vector
    __device__ static constexpr int pos(int i, int wsel) { return CLS == 0 ? i : CLS == 1 ? wsel * 2 + i : 4 * (wsel >> 1) + (wsel & 1) * 2 + i; }

    __device__ static __forceinline__ void load_token(const uint8_t* stage, int s, int q, __half2 (&h)[8]) {
        if (CLS == 0) {                                // elements 16q .. 16q+15: pieces 2q, 2q+1
            *reinterpret_cast<uint4*>(&h[0]) = *reinterpret_cast<const uint4*>(stage + stage_piece_offset(s, 2 * q));
            *reinterpret_cast<uint4*>(&h[4]) = *reinterpret_cast<const uint4*>(stage + stage_piece_offset(s, 2 * q + 1));
        } else if (CLS == 1) {                         // elements 8q .. 8q+7 and 32+8q ..: pieces q, 4+q
            *reinterpret_cast<uint4*>(&h[0]) = *reinterpret_cast<const uint4*>(stage + stage_piece_offset(s, q));
            *reinterpret_cast<uint4*>(&h[4]) = *reinterpret_cast<const uint4*>(stage + stage_piece_offset(s, 4 + q));
        } else {                                       // elements 4q + 16 w .. +3: half q % 2 of piece 2w + q / 2
#pragma unroll
            for (int w = 0; w < 4; ++w)
                *reinterpret_cast<uint2*>(&h[2 * w]) =
                    *reinterpret_cast<const uint2*>(stage + stage_piece_offset(s, 2 * w + (q >> 1)) + 8 * (q & 1));
        }
    }
    __device__ static __forceinline__ void codes(const __half2 (&h)[8], float mn, float inv, int i, uint32_t (&kw)[NW]) {
        uint32_t bias = 0;
#pragma unroll
        for (int e = 0; e < EPW; ++e) bias += 0x4B400000u << (BITS * e);
#pragma unroll
        for (int w = 0; w < WT; ++w) {
            uint32_t acc = 0u - bias;
#pragma unroll
            for (int e = 0; e < EPW; e += 2) {
                uint32_t b0, b1;
                code_pair<CLS, false>(h[(w * EPW + e) / 2], mn, inv, b0, b1);
                acc += b0 << (BITS * e);
                acc += b1 << (BITS * (e + 1));
            }
            kw[pos(i, w)] = acc;
        }
    }
    // false: some row of the tile has a subnormal scale (its quotients need the clamp): the caller takes the
    // compact general routine for the whole item instead.
    __device__ static __forceinline__ bool tile(const uint8_t* stage, int g, int q, uint32_t (&kw)[NW], uint32_t& meta) {
        __half2 h0[8], h1[8];
        load_token(stage, g, q, h0);
        load_token(stage, g + 8, q, h1);
        __half2 m0 = min_negmax(h0), m1 = min_negmax(h1);
        m0 = shfl_min2(shfl_min2(m0, 1), 2);
        m1 = shfl_min2(shfl_min2(m1, 1), 2);
        // even lanes set up slot g, odd lanes slot g + 8; the neighbour's result comes back through one exchange
        const __half2 mine = (q & 1) ? m1 : m0;
        const RowScale rs = row_scale<CLS>(__low2float(mine), -__high2float(mine));
        if (__any_sync(0xffffffffu, rs.tiny)) return false;
        meta = rs.meta;
        const float inv_o = __shfl_xor_sync(0xffffffffu, rs.inv, 1), mn_o = __shfl_xor_sync(0xffffffffu, rs.mn, 1);
        codes(h0, (q & 1) ? mn_o : rs.mn, (q & 1) ? inv_o : rs.inv, 0, kw);
        codes(h1, (q & 1) ? rs.mn : mn_o, (q & 1) ? rs.inv : inv_o, 1, kw);
        return true;
    }
};

// ---- V side of one tile.  stage: the 16 V rows.  scratch: 16 float2 of shared memory owned by the warp.  Returns the
// lane's words of the V code block in store order (see vfrag_byte_offset) and, in lanes g < 4, the {scale,
// zero-point} word of slot 4 q + g.
template <int CLS>
struct FragV {
    static constexpr int BITS = pool_bits(CLS), NW = 2 << CLS;
    // word (in the lane's store vector) and bit position of the code of element e (0..3) of slot j, channel group i
    __device__ static constexpr int pos(int i, int e) { return CLS == 0 ? i : CLS == 1 ? (e >> 1) * 2 + i : 4 * (e >> 1) + (e & 1) * 2 + i; }
    __device__ static constexpr int shift(int j, int e) { return 8 * j + (CLS == 0 ? 2 * e : CLS == 1 ? 4 * (e & 1) : 0); }

    template <bool CLAMP>
    __device__ static __forceinline__ void codes(const __half2 (&h)[4][4], const float4 (&sc)[2], uint32_t (&vw)[NW]) {
        uint32_t bias[NW];
#pragma unroll
        for (int w = 0; w < NW; ++w) bias[w] = 0;
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) bias[pos(i, e)] += 0x4B400000u << shift(j, e);
#pragma unroll
        for (int w = 0; w < NW; ++w) vw[w] = 0u - bias[w];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float inv = j == 0 ? sc[0].x : j == 1 ? sc[0].z : j == 2 ? sc[1].x : sc[1].z;
            const float mn = j == 0 ? sc[0].y : j == 1 ? sc[0].w : j == 2 ? sc[1].y : sc[1].w;
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int e = 0; e < 4; e += 2) {
                    uint32_t b0, b1;
                    code_pair<CLS, CLAMP>(h[j][2 * i + (e >> 1)], mn, inv, b0, b1);
                    vw[pos(i, e)] += b0 << shift(j, e);
                    vw[pos(i, e + 1)] += b1 << shift(j, e + 1);
                }
        }
    }
    // voff[j]: byte offset, inside the stage, of elements 4g .. 4g+3 of slot 4q + j (elements 32+4g .. sit 64 bytes
    // further, xor-wise).  false: a subnormal scale in the tile (see FragK::tile); with CLAMP every quotient is
    // clamped and the answer is always true.
    template <bool CLAMP = false>
    __device__ static __forceinline__ bool tile(const uint8_t* stage, const int (&voff)[4], float2* scratch, int g, int q,
                                                uint32_t (&vw)[NW], uint32_t& meta) {
        __half2 h[4][4];                               // [slot 4q + j][elements 4g..4g+3, then 32+4g..32+4g+3]
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            *reinterpret_cast<uint2*>(&h[j][0]) = *reinterpret_cast<const uint2*>(stage + voff[j]);
            *reinterpret_cast<uint2*>(&h[j][2]) = *reinterpret_cast<const uint2*>(stage + (voff[j] ^ 64));
        }
        __half2 mm[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) mm[j] = shfl_min2(shfl_min2(shfl_min2(min_negmax(h[j]), 4), 8), 16);
        // lanes g and g + 4 set up slot 4q + (g & 3); the results reach every lane through shared memory
        const __half2 mine = (g & 3) == 0 ? mm[0] : (g & 3) == 1 ? mm[1] : (g & 3) == 2 ? mm[2] : mm[3];
        const RowScale rs = row_scale<CLS>(__low2float(mine), -__high2float(mine));
        if (!CLAMP && __any_sync(0xffffffffu, rs.tiny)) return false;
        meta = rs.meta;
        __syncwarp();                                  // the scratch may still be read for the previous tile
        if (g < 4) scratch[4 * q + g] = make_float2(rs.inv, rs.mn);
        __syncwarp();
        float4 sc[2];
        sc[0] = *reinterpret_cast<const float4*>(scratch + 4 * q);
        sc[1] = *reinterpret_cast<const float4*>(scratch + 4 * q + 2);
        codes<CLAMP>(h, sc, vw);
        return true;
    }
};

// ---- K side of one COMPLETE tile of a cache with per-channel keys: every channel's 16 values (one per slot) are a
// row for the row quantizer.  Lane (g, q) holds the same elements as in FragK (16 per slot, slots g and g + 8);
// a channel's minimum and maximum meet through three xor-shuffles over g; the lane with g = k sets up the two
// channels of its element pair k and all lanes fetch the pairs' {reciprocal, minimum} through shared memory
// (chan: 4 x 16 float2 owned by the warp).  The quotient is always clamped (no separate routine for subnormal scales).
template <int CLS>
struct FragKPC {
    static constexpr int BITS = pool_bits(CLS), EPW = 32 / BITS, WT = 16 / EPW, NW = 2 * WT;
    // canonical element index of element 2k (and 2k + 1) of the lane's 16 elements
    __device__ static constexpr int element(int q, int k) {
        return CLS == 0 ? 16 * q + 2 * k : CLS == 1 ? 8 * q + 32 * (k >> 2) + 2 * (k & 3) : 4 * q + 16 * (k >> 1) + 2 * (k & 1);
    }
    __device__ static __forceinline__ void codes(const __half2 (&h)[8], const float4 (&sc)[8], int i, uint32_t (&kw)[NW]) {
        constexpr float LEVELS = (float)((1 << BITS) - 1);
        uint32_t bias = 0;
#pragma unroll
        for (int e = 0; e < EPW; ++e) bias += 0x4B400000u << (BITS * e);
#pragma unroll
        for (int w = 0; w < WT; ++w) {
            uint32_t acc = 0u - bias;
#pragma unroll
            for (int e = 0; e < EPW; e += 2) {
                const int k = (w * EPW + e) / 2;       // sc[k] = {inv, mn} of element 2k, {inv, mn} of element 2k + 1
                const float2 f = __half22float2(h[k]);
                const float r0 = __fadd_rn(fminf(__fmul_rn(__fsub_rn(f.x, sc[k].y), sc[k].x), LEVELS), kRoundMagic);
                const float r1 = __fadd_rn(fminf(__fmul_rn(__fsub_rn(f.y, sc[k].w), sc[k].z), LEVELS), kRoundMagic);
                acc += __float_as_uint(r0) << (BITS * e);
                acc += __float_as_uint(r1) << (BITS * (e + 1));
            }
            kw[FragK<CLS>::pos(i, w)] = acc;
        }
    }
    // chan_meta: the tile's 64 {scale, zero-point} words in the record.
    __device__ static __forceinline__ void tile(const uint8_t* stage, float4* chan, uint32_t* chan_meta, int g, int q,
                                                uint32_t (&kw)[NW]) {
        __half2 h0[8], h1[8];
        FragK<CLS>::load_token(stage, g, q, h0);
        FragK<CLS>::load_token(stage, g + 8, q, h1);
        float4 sc[8];
        {
            __half2 mn[8], mx[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                mn[k] = __hmin2(h0[k], h1[k]);
                mx[k] = __hmax2(h0[k], h1[k]);
#pragma unroll
                for (int d = 4; d <= 16; d <<= 1) {
                    uint32_t a = *reinterpret_cast<uint32_t*>(&mn[k]), b = *reinterpret_cast<uint32_t*>(&mx[k]);
                    a = __shfl_xor_sync(0xffffffffu, a, d);
                    b = __shfl_xor_sync(0xffffffffu, b, d);
                    mn[k] = __hmin2(mn[k], *reinterpret_cast<__half2*>(&a));
                    mx[k] = __hmax2(mx[k], *reinterpret_cast<__half2*>(&b));
                }
            }
            __half2 my_mn = mn[0], my_mx = mx[0];      // the pair this lane sets up: k = g
#pragma unroll
            for (int k = 1; k < 8; ++k) {
                my_mn = g == k ? mn[k] : my_mn;
                my_mx = g == k ? mx[k] : my_mx;
            }
            const RowScale lo = row_scale<CLS>(__low2float(my_mn), __low2float(my_mx));
            const RowScale hi = row_scale<CLS>(__high2float(my_mn), __high2float(my_mx));
            int e0 = element(q, 0);
#pragma unroll
            for (int k = 1; k < 8; ++k) e0 = g == k ? element(q, k) : e0;
            chan_meta[e0] = lo.meta;
            chan_meta[e0 + 1] = hi.meta;
            __syncwarp();                              // the scratch may still be read for the previous tile
            chan[q * 8 + g] = make_float4(lo.inv, lo.mn, hi.inv, hi.mn);
            __syncwarp();
#pragma unroll
            for (int k = 0; k < 8; ++k) sc[k] = chan[q * 8 + k];
        }
        codes(h0, sc, 0, kw);
        codes(h1, sc, 1, kw);
    }
};

// Store (or, for a tile that an earlier append call began, blend and store) a lane's words of one code block.
// keep_k[i]: K block: the word of token i stays as it is.  keep_bytes: V block: mask of the bytes that stay.
template <int NW>
__device__ __forceinline__ void store_block(uint8_t* codes, int lane, const uint32_t (&w)[NW]) {
    if (NW == 2) {
        *reinterpret_cast<uint2*>(codes + lane * 8) = make_uint2(w[0], w[1]);
    } else {
#pragma unroll
        for (int u = 0; u < NW / 4; ++u)
            *reinterpret_cast<uint4*>(codes + (u * 32 + lane) * 16) = make_uint4(w[4 * u], w[4 * u + 1], w[4 * u + 2], w[4 * u + 3]);
    }
}
template <int NW>
__device__ __forceinline__ void load_block(const uint8_t* codes, int lane, uint32_t (&w)[NW]) {
    if (NW == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(codes + lane * 8);
        w[0] = v.x; w[1] = v.y;
    } else {
#pragma unroll
        for (int u = 0; u < NW / 4; ++u) {
            const uint4 v = *reinterpret_cast<const uint4*>(codes + (u * 32 + lane) * 16);
            w[4 * u] = v.x; w[4 * u + 1] = v.y; w[4 * u + 2] = v.z; w[4 * u + 3] = v.w;
        }
    }
}

// Work of a warp on one (tile, head) item whose rows sit in `stage`: quantize both tensors and store the record.
// first_new: slots below it hold tokens of an earlier append call and stay as they are (0 for every other tile).
// Returns false if a row of the tile needs the clamp (subnormal scale): the caller then runs general_item, which
// rewrites whatever this routine has stored already with the same values.
template <int CLS>
__device__ __forceinline__ bool frag_item(const uint8_t* stage, const int (&voff)[4], float2* scratch, uint8_t* rec, int lane,
                                          int first_new) {
    const int g = lane >> 2, q = lane & 3;
    constexpr int NW = FragK<CLS>::NW;
    uint8_t* vcodes = rec + pool_codes_bytes(CLS);
    {
        uint32_t kw[NW], kmeta;
        if (!FragK<CLS>::tile(stage, g, q, kw, kmeta)) return false;
        if (first_new > 0) {                           // warp-uniform, once per class and call at most
            uint32_t ko[NW];
            load_block<NW>(rec, lane, ko);
#pragma unroll
            for (int w = 0; w < NW; ++w)
                if (g + 8 * (w & 1) < first_new) kw[w] = ko[w];       // K word w belongs to slot g (even w) or g + 8
        }
        store_block<NW>(rec, lane, kw);
        if (q < 2 && g + 8 * q >= first_new) *reinterpret_cast<uint32_t*>(rec + meta_offset(CLS, 0, g + 8 * q)) = kmeta;
    }
    {
        uint32_t vw[NW], vmeta;
        if (!FragV<CLS>::tile(stage + kStageTensorBytes, voff, scratch, g, q, vw, vmeta)) return false;
        if (first_new > 0) {
            uint32_t vo[NW];
            load_block<NW>(vcodes, lane, vo);
            const int nb = min(max(first_new - 4 * q, 0), 4);          // bytes (slots 4q ..) of a V word that stay
            const uint32_t keep = nb == 4 ? 0xffffffffu : ((1u << (8 * nb)) - 1u);
#pragma unroll
            for (int w = 0; w < NW; ++w) vw[w] = (vw[w] & ~keep) | (vo[w] & keep);
        }
        store_block<NW>(vcodes, lane, vw);
        if (g < 4 && 4 * q + g >= first_new) *reinterpret_cast<uint32_t*>(rec + meta_offset(CLS, 1, 4 * q + g)) = vmeta;
    }
    return true;
}

// The same for a cache with per-channel keys.  live: slots that receive a token of this call; the tile's keys are
// packed only when it is complete (slots below first_new came from earlier calls: their rows were fetched from the
// residual buffer into the stage), otherwise the new rows join the residual rows `kres` [16][64] of the stream.
template <int CLS>
__device__ __forceinline__ void frag_item_pc(const uint8_t* stage, const int (&voff)[4], float2* scratch, float4* chan,
                                             uint8_t* rec, __half* kres, int lane, int first_new, uint32_t live) {
    const int g = lane >> 2, q = lane & 3;
    constexpr int NW = FragK<CLS>::NW;
    const bool complete = (live | ((1u << first_new) - 1u)) == 0xffffu;
    if (complete) {
        uint32_t kw[NW];
        FragKPC<CLS>::tile(stage, chan, reinterpret_cast<uint32_t*>(rec + chan_meta_offset(CLS, 0)), g, q, kw);
        store_block<NW>(rec, lane, kw);
    } else {
        const int half = lane >> 4, t = lane & 15;
        if ((live >> t) & 1u) {
#pragma unroll
            for (int u = 0; u < 4; ++u)
                *reinterpret_cast<uint4*>(kres + t * kHeadDim + 32 * half + 8 * u) =
                    *reinterpret_cast<const uint4*>(stage + stage_piece_offset(t, 4 * half + u));
        }
    }
    uint8_t* vcodes = rec + pool_codes_bytes(CLS);
    uint32_t vw[NW], vmeta;
    FragV<CLS>::template tile<true>(stage + kStageTensorBytes, voff, scratch, g, q, vw, vmeta);
    if (first_new > 0) {
        uint32_t vo[NW];
        load_block<NW>(vcodes, lane, vo);
        const int nb = min(max(first_new - 4 * q, 0), 4);
        const uint32_t keep = nb == 4 ? 0xffffffffu : ((1u << (8 * nb)) - 1u);
#pragma unroll
        for (int w = 0; w < NW; ++w) vw[w] = (vw[w] & ~keep) | (vo[w] & keep);
    }
    store_block<NW>(vcodes, lane, vw);
    if (g < 4 && 4 * q + g >= first_new)
        *reinterpret_cast<uint32_t*>(rec + meta_offset(CLS, 1, 4 * q + g, 0, kLayoutPerChannelK)) = vmeta;
}

// The general routine for one item: any class < 3, clamp included, every slot >= first_new written code word by
// code word (K) and byte by byte (V).  Compact on purpose (loops are not unrolled): it runs only for tiles that
// hold a row whose scale is a subnormal fp16.  Lane (half h, slot t) takes the half-row of 32 elements.
__device__ __noinline__ void general_item(const uint8_t* stage, uint8_t* rec, int cls, int lane, int first_new) {
    const int half = lane >> 4, t = lane & 15;
    const int bits = pool_bits(cls), epw = 32 / bits;
    const float levels = (float)((1 << bits) - 1);
#pragma unroll 1
    for (int tensor = 0; tensor < 2; ++tensor) {
        const uint8_t* rows = stage + tensor * kStageTensorBytes;
        uint8_t* codes = rec + tensor * pool_codes_bytes(cls);
        float mn = INFINITY, mx = -INFINITY;
#pragma unroll 1
        for (int i = 0; i < 32; ++i) {
            const int e = 32 * half + i;
            const float x = __half2float(*reinterpret_cast<const __half*>(rows + stage_piece_offset(t, e >> 3) + 2 * (e & 7)));
            mn = fminf(mn, x);
            mx = fmaxf(mx, x);
        }
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 16));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        if (mn == 0.0f) mn = 0.0f;
        if (mx == 0.0f) mx = 0.0f;
        const float s32 = __fdiv_rn(__fsub_rn(mx, mn), levels);
        const __half s16 = __float2half_rn(s32);
        const float sf = __half2float(s16);
        const float inv = sf == 0.0f ? 0.0f : __frcp_rn(sf);
        if (t < first_new) continue;                   // (after the shuffles: every lane takes part in them)
        uint32_t word = 0;
#pragma unroll 1
        for (int i = 0; i < 32; ++i) {
            const int e = 32 * half + i;
            const float x = __half2float(*reinterpret_cast<const __half*>(rows + stage_piece_offset(t, e >> 3) + 2 * (e & 7)));
            const float v = fminf(__fmul_rn(__fsub_rn(x, mn), inv), levels);
            const uint32_t code = __float_as_uint(__fadd_rn(v, kRoundMagic)) - 0x4B400000u;
            word |= code << (bits * (e % epw));
            if ((e + 1) % epw == 0) {                  // a canonical 32-bit word is complete
                const int wq = e / epw;
                if (tensor == 0) {
                    *reinterpret_cast<uint32_t*>(codes + kfrag_word_offset(cls, t, wq)) = word;
                } else {
                    for (int b = 0; b < 4; ++b) codes[vfrag_byte_offset(cls, t, 4 * wq + b)] = (uint8_t)(word >> (8 * b));
                }
                word = 0;
            }
        }
        if (half == 0)
            *reinterpret_cast<uint32_t*>(rec + meta_offset(cls, tensor, t)) =
                (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(__float2half_rn(mn)) << 16);
    }
}

// fp16 tile: the lane (half h, slot t) copies its 64 bytes of both rows (the unit layout of the fp16 pool).
__device__ __forceinline__ void frag_item_fp16(const uint8_t* stage, uint8_t* rec, int lane, int first_new, uint32_t live_mask) {
    const int half = lane >> 4, t = lane & 15;
    if (t < first_new || !((live_mask >> t) & 1u)) return;
    uint8_t* vcodes = rec + pool_codes_bytes(3);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        *reinterpret_cast<uint4*>(rec + unit_offset(3, half, u, t)) =
            *reinterpret_cast<const uint4*>(stage + stage_piece_offset(t, 4 * half + u));
        *reinterpret_cast<uint4*>(vcodes + unit_offset(3, half, u, t)) =
            *reinterpret_cast<const uint4*>(stage + kStageTensorBytes + stage_piece_offset(t, 4 * half + u));
    }
}

// The quantize-and-pack launch for caches with one scale group.  MODE as in k_quant_pack: 0 = classes from the
// classify launch (several chunks per sequence), 1 = one chunk, classes from `bits`, 2 = one chunk, classes from
// the controller.  grid = (nchunks, head_groups, batch), block = 256, dynamic smem = kFragRingBytes (+ controller).
// PC: the cache keeps per-channel keys (layout kLayoutPerChannelK).
template <int MODE, int R = 1, bool PC = false>
__global__ void __launch_bounds__(kChunkTokens, KVQ_APPEND_FRAG_MIN_CTAS)
k_quant_pack_frag(AppendParams p) {
    constexpr int LAYOUT = PC ? kLayoutPerChannelK : 1;
    static_assert(MODE == 0 || R == 1, "single-chunk appends hold at most 256 tokens per sequence");
    constexpr int CT = kChunkTokens * R;               // tokens per chunk
    constexpr int NWARPS = kChunkTokens / 32;
    extern __shared__ __align__(16) uint8_t dyn_smem[];   // [ring: warps x depth x 4 KB][controller block (MODE 2)]
    float* sW = reinterpret_cast<float*>(dyn_smem + kFragRingBytes);
    __shared__ uint32_t wtot[R][NWARPS][4];
    __shared__ uint32_t base[4];
    __shared__ uint16_t list[4][CT];                   // the chunk's tokens by class, in slot order
    __shared__ uint32_t ext[4][kTileTokens];           // tokens of later chunks that complete the last owned tile (index in the call)
    __shared__ uint32_t ext_n[4];
    __shared__ float2 vscratch[NWARPS][kTileTokens];
    __shared__ float4 kchan[PC ? NWARPS : 1][32];      // per-channel keys: {reciprocal, minimum} of a tile's channels
    const int chunk = blockIdx.x, hg = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_b = new_tokens_of(p, b);

    // ---- classes of this thread's tokens (pass r: token r * 256 + thread of the chunk)
    int c[R];
    if (MODE == 2) {
        controller_stage(sW, p.ctrl, p.hidden);
        __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int tok_i = chunk * CT + r * kChunkTokens + threadIdx.x;
        const bool live = tok_i < n_b;
        const size_t tok = (size_t)b * p.n_new + tok_i;
        c[r] = -1;
        if (MODE == 2) {
            if (live) {
                float4 f = reinterpret_cast<const float4*>(p.feats)[tok];
                float lg[4];
                c[r] = controller_decide_any(sW, p.hidden, f.x, f.y, f.z, f.w, lg);
                if (p.bits_out && hg == 0) p.bits_out[tok] = (uint8_t)pool_bits(c[r]);
            }
        } else if (MODE == 1) {
            if (live) c[r] = class_of_bits(p.bits[tok], p.store.flags);
        } else {
            if (live) c[r] = p.cls[tok];
        }
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
    // ---- rank inside the chunk: tokens of earlier passes, of earlier warps of the pass, of earlier lanes
    uint32_t rank[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        rank[r] = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t m = __ballot_sync(0xffffffffu, c[r] == k);
            if (c[r] == k) rank[r] = __popc(m & ((1u << lane) - 1u));
            if (lane == 0) wtot[r][warp][k] = __popc(m);
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (c[r] < 0) continue;
        uint32_t before = rank[r];
        for (int rr = 0; rr < r; ++rr)
            for (int w = 0; w < NWARPS; ++w) before += wtot[rr][w][c[r]];
        for (int w = 0; w < warp; ++w) before += wtot[r][w][c[r]];
        const int in_chunk = r * kChunkTokens + threadIdx.x;
        list[c[r]][before] = (uint16_t)in_chunk;
        if (hg == 0)
            p.store.index[((size_t)p.layer * p.store.batch + b) * p.store.max_ctx + first_pos_of(p, b) + chunk * CT + in_chunk] =
                ((uint32_t)c[r] << 30) | (base[c[r]] + before);
    }
    uint32_t ncls[4];                                  // tokens of each class in this chunk
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        ncls[k] = 0;
        for (int r = 0; r < R; ++r)
            for (int w = 0; w < NWARPS; ++w) ncls[k] += wtot[r][w][k];
    }
    if (hg == 0 && chunk == p.nchunks - 1 && threadIdx.x < 4)
        p.counts_out[(size_t)b * 4 + threadIdx.x] = base[threadIdx.x] + ncls[threadIdx.x];
    const int h0 = hg * p.heads_per_group;
    const int nh = min(p.heads_per_group, p.store.kv_heads - h0);
    if (MODE != 0) {
        // One chunk per sequence: this CTA is the only one that writes the streams of its heads, so it
        // reserves the blocks they grow into itself (with several chunks the classify launch did it before).
        if (warp < kNumPools) reserve_blocks(p.store, warp, p.layer, b, h0, nh, base[warp], base[warp] + ncls[warp], lane);
    }

    // ---- owned tiles of class k: first slot in [own0, base + n); the first chunk also owns the tile that an
    //      earlier call left partly filled.  need[k]: tokens of later chunks that complete the last owned tile.
    uint32_t first[4], pre[5], need[4];
    pre[0] = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t own0 = chunk == 0 ? (base[k] & ~(uint32_t)(kTileTokens - 1)) : base[k];
        const uint32_t t_first = (own0 + kTileTokens - 1) / kTileTokens, t_end = (base[k] + ncls[k] + kTileTokens - 1) / kTileTokens;
        first[k] = t_first;
        const uint32_t nt = t_end > t_first ? t_end - t_first : 0;
        pre[k + 1] = pre[k] + nt;
        need[k] = nt ? t_end * kTileTokens - (base[k] + ncls[k]) : 0;
    }
    if (MODE == 0 && warp < kNumPools) {               // warp k looks ahead for the class-k tokens that follow the chunk
        const int k = warp;
        const uint32_t want = need[k];
        uint32_t found = 0;
        for (int pos = (chunk + 1) * CT; found < want && pos < n_b; pos += 32) {
            const int v = pos + lane < n_b ? (int)p.cls[(size_t)b * p.n_new + pos + lane] : -1;
            const uint32_t m = __ballot_sync(0xffffffffu, v == k);
            const uint32_t at = found + __popc(m & ((1u << lane) - 1u));
            if (v == k && at < want) ext[k][at] = (uint32_t)(pos + lane);
            found += __popc(m);
        }
        if (lane == 0) ext_n[k] = found < want ? found : want;
    } else if (warp < kNumPools && lane == 0) {
        ext_n[warp] = 0;
    }
    __syncthreads();

    // ---- work items (owned tile tau, head hh), heads fastest, dealt round-robin to the warps.  The input rows of
    // the next kFragDepth items are kept in flight with 16-byte async copies into a per-warp ring: eight
    // neighbouring lanes fetch one whole 128-byte row, slots without a token are filled with zeros.
    struct Item {
        int k;                                         // class, -1 = no more items
        int first_new;                                 // slots below it belong to an earlier call
        uint32_t live;                                 // bit s: slot s receives a token of this call
        uint8_t* rec;
        int h;                                         // KV head
    };
    // Tiles are dealt round-robin to the warps; a warp takes a tile through all heads of the CTA's group, so what
    // depends on the tile alone (class, ranks of its slots, the source rows of the four slots this lane fetches,
    // the place of the record inside its arena block) is worked out once per tile.
    uint32_t tau = (uint32_t)warp;
    int hh = 0;
    struct TileInfo {
        int k, first_new;
        uint32_t live, blk, rec_off;
        size_t src[4];                                 // element offset of the row of slot (lane >> 3) + 4 i, head 0 (live slots)
        uint32_t fetch;                                // bit i: that slot receives a token of this call; bit 4 + i: it is older
    } ti;
    ti.k = -1;
    uint8_t* my_ring = dyn_smem + (size_t)warp * kFragDepth * kFragStageBytes;
    int voff[4];                                       // where this lane's V elements of slots 4q .. 4q+3 sit in a stage
#pragma unroll
    for (int j = 0; j < 4; ++j) voff[j] = stage_piece_offset(4 * (lane & 3) + j, lane >> 3) + 8 * ((lane >> 2) & 1);
    const int piece = lane & 7;
    int soff[4];                                       // where the piece this lane fetches of slot (lane >> 3) + 4 i goes
#pragma unroll
    for (int i = 0; i < 4; ++i) soff[i] = stage_piece_offset((lane >> 3) + 4 * i, piece);
    const size_t row_stride = (size_t)p.store.kv_heads * kHeadDim;
    const uint32_t* tab_b = p.store.table + ((size_t)p.layer * p.store.batch + b) * p.store.kv_heads * p.store.table_stride;
    auto load_tile = [&]() {
        const int k = (tau >= pre[1]) + (tau >= pre[2]) + (tau >= pre[3]);
        const uint32_t basek = k == 0 ? base[0] : k == 1 ? base[1] : k == 2 ? base[2] : base[3];
        const uint32_t nk = (k == 0 ? ncls[0] : k == 1 ? ncls[1] : k == 2 ? ncls[2] : ncls[3]);
        const uint32_t nke = nk + ext_n[k];
        const uint32_t tile = (k == 0 ? first[0] : k == 1 ? first[1] : k == 2 ? first[2] : first[3]) +
                              (tau - (k == 0 ? pre[0] : k == 1 ? pre[1] : k == 2 ? pre[2] : pre[3]));
        const int r0 = (int)(tile * kTileTokens) - (int)basek;           // rank of the tile's slot 0 (negative: older slots)
        ti.k = k;
        ti.first_new = r0 < 0 ? -r0 : 0;
        switch (k) {                                   // (constant divisors)
        case 0: ti.blk = tile / block_tiles(0, LAYOUT); ti.rec_off = (tile - ti.blk * block_tiles(0, LAYOUT)) * pool_rec_bytes(0, LAYOUT); break;
        case 1: ti.blk = tile / block_tiles(1, LAYOUT); ti.rec_off = (tile - ti.blk * block_tiles(1, LAYOUT)) * pool_rec_bytes(1, LAYOUT); break;
        case 2: ti.blk = tile / block_tiles(2, LAYOUT); ti.rec_off = (tile - ti.blk * block_tiles(2, LAYOUT)) * pool_rec_bytes(2, LAYOUT); break;
        default: ti.blk = tile / block_tiles(3, LAYOUT); ti.rec_off = (tile - ti.blk * block_tiles(3, LAYOUT)) * pool_rec_bytes(3, LAYOUT); break;
        }
        ti.blk += p.store.table_off[k];
        ti.fetch = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = r0 + (lane >> 3) + 4 * i;
            const bool live = r >= 0 && (uint32_t)r < nke;
            size_t tok_i = 0;
            if (live) tok_i = (uint32_t)r < nk ? (size_t)chunk * CT + list[k][r] : (size_t)ext[k][(uint32_t)r - nk];
            ti.src[i] = ((size_t)b * p.n_new + tok_i) * row_stride;
            ti.fetch |= (live ? 1u : 0u) << i | (r < 0 ? 16u : 0u) << i;
        }
        // slots that receive a token: ranks 0 .. nke-1 that fall into this tile
        const int lo = r0 < 0 ? -r0 : 0, hi_ = min((int)kTileTokens, (int)nke - r0);
        ti.live = hi_ > lo ? (((1u << hi_) - 1u) & ~((1u << lo) - 1u)) : 0u;
    };
    auto next_item = [&](int stage) {
        Item it;
        it.k = -1;
        it.first_new = 0;
        it.live = 0;
        it.rec = nullptr;
        it.h = 0;
        if (tau < pre[4]) {
            if (hh == 0) load_tile();
            const int k = ti.k, h = h0 + hh;
            it.k = k;
            it.first_new = ti.first_new;
            it.live = ti.live;
            it.h = h;
            it.rec = p.store.arena + (size_t)tab_b[(size_t)h * p.store.table_stride + ti.blk] * kBlockBytes + ti.rec_off;
            uint8_t* dst = my_ring + (size_t)stage * kFragStageBytes;
            const size_t head_off = (size_t)h * kHeadDim;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const bool live = (ti.fetch >> i) & 1u;
                const size_t src = ti.src[i] + head_off;
                // a slot of an earlier call: its key row waits in the residual buffer -- read from the copy taken before this
                // launch, because the rows of the stream's NEXT open window go to the same places during the launch
                if (PC && ((ti.fetch >> (4 + i)) & 1u) && k < 3)
                    cp_async16_or_zero(dst + soff[i], reinterpret_cast<const uint4*>(residual_rows_before(p.store, k, b, h) + ((lane >> 3) + 4 * i) * kHeadDim) + piece, true);
                else
                    cp_async16_or_zero(dst + soff[i], reinterpret_cast<const uint4*>(p.K + src) + piece, live);
                cp_async16_or_zero(dst + kStageTensorBytes + soff[i], reinterpret_cast<const uint4*>(p.V + src) + piece, live);
            }
            if (++hh == nh) {
                hh = 0;
                tau += NWARPS;
            }
        }
        cp_async_commit();                             // one group per call, possibly empty
        return it;
    };
    Item items[kFragDepth];
#pragma unroll
    for (int d = 0; d < kFragDepth; ++d) items[d] = next_item(d);
    int stage = 0;
    while (items[0].k >= 0) {
        cp_async_wait<kFragDepth - 1>();             // this lane's copies of the oldest group have landed
        __syncwarp();                                  // ... and so have the other lanes'
        const Item cur = items[0];
        const uint8_t* st = my_ring + (size_t)stage * kFragStageBytes;
        if (cur.live != 0u) {                          // (a tile of an earlier call that this call adds nothing to)
            bool done = true;
            if (PC) {
                __half* kres = cur.k < 3 ? residual_rows(p.store, cur.k, p.layer, b, cur.h) : nullptr;
                switch (cur.k) {
                case 0: frag_item_pc<0>(st, voff, vscratch[warp], kchan[PC ? warp : 0], cur.rec, kres, lane, cur.first_new, cur.live); break;
                case 1: frag_item_pc<1>(st, voff, vscratch[warp], kchan[PC ? warp : 0], cur.rec, kres, lane, cur.first_new, cur.live); break;
                case 2: frag_item_pc<2>(st, voff, vscratch[warp], kchan[PC ? warp : 0], cur.rec, kres, lane, cur.first_new, cur.live); break;
                default: frag_item_fp16(st, cur.rec, lane, cur.first_new, cur.live); break;
                }
            } else
            switch (cur.k) {
            case 0: done = frag_item<0>(st, voff, vscratch[warp], cur.rec, lane, cur.first_new); break;
            case 1: done = frag_item<1>(st, voff, vscratch[warp], cur.rec, lane, cur.first_new); break;
            case 2: done = frag_item<2>(st, voff, vscratch[warp], cur.rec, lane, cur.first_new); break;
            default: frag_item_fp16(st, cur.rec, lane, cur.first_new, cur.live); break;
            }
            if (!done) general_item(st, cur.rec, cur.k, lane, cur.first_new);
        }
        __syncwarp();                                  // every lane has read the stage before it is refilled
#pragma unroll
        for (int d = 0; d + 1 < kFragDepth; ++d) items[d] = items[d + 1];
        items[kFragDepth - 1] = next_item(stage);
        if (++stage == kFragDepth) stage = 0;
    }
    cp_async_wait<0>();
}

// Per-channel keys, after a one-token append: the token that took the last slot of a window completes it, and one
// warp per (KV head, sequence) packs the window's 16 residual rows.  grid = (kv_heads, batch), block = 32.
__global__ void __launch_bounds__(32)
k_pack_window(AppendParams p) {
    __shared__ __align__(16) uint8_t stage[kStageTensorBytes];
    __shared__ float4 chan[32];
    const int h = blockIdx.x, b = blockIdx.y, lane = threadIdx.x;
    const StoreView& s = p.store;
    const uint32_t word = s.index[((size_t)p.layer * s.batch + b) * s.max_ctx + first_pos_of(p, b)];
    const int c = (int)(word >> 30);
    const uint32_t slot = word & 0x3fffffffu;
    if (c == 3 || (slot & (kTileTokens - 1)) != kTileTokens - 1) return;
    const __half* rows = residual_rows(s, c, p.layer, b, h);
#pragma unroll
    for (int i = 0; i < 4; ++i) {                      // eight neighbouring lanes copy one 128-byte row
        const int t = (lane >> 3) + 4 * i, piece = lane & 7;
        *reinterpret_cast<uint4*>(stage + stage_piece_offset(t, piece)) = reinterpret_cast<const uint4*>(rows + t * kHeadDim)[piece];
    }
    __syncwarp();
    uint8_t* rec = tile_ptr(s, c, stream_table(s, c, p.layer, b, h), slot / kTileTokens, kLayoutPerChannelK);
    const int g = lane >> 2, q = lane & 3;
    switch (c) {
    case 0: {
        uint32_t kw[FragK<0>::NW];
        FragKPC<0>::tile(stage, chan, reinterpret_cast<uint32_t*>(rec + chan_meta_offset(0, 0)), g, q, kw);
        store_block<FragK<0>::NW>(rec, lane, kw);
        break;
    }
    case 1: {
        uint32_t kw[FragK<1>::NW];
        FragKPC<1>::tile(stage, chan, reinterpret_cast<uint32_t*>(rec + chan_meta_offset(1, 0)), g, q, kw);
        store_block<FragK<1>::NW>(rec, lane, kw);
        break;
    }
    default: {
        uint32_t kw[FragK<2>::NW];
        FragKPC<2>::tile(stage, chan, reinterpret_cast<uint32_t*>(rec + chan_meta_offset(2, 0)), g, q, kw);
        store_block<FragK<2>::NW>(rec, lane, kw);
        break;
    }
    }
}

}  // namespace kvq
