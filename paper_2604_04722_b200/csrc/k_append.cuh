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
// _rn intrinsics so the result is the same bit pattern on every build.  Codes are packed by adding
// the shifted bit patterns of the rounded sums in wrapping 32-bit arithmetic.
#pragma once
#include "kvq_common.cuh"
#include "k_controller.cuh"

namespace kvq {

constexpr int kChunkTokens = 256;      // threads per CTA of the chunked kernels; a chunk holds 256 * tpt tokens
constexpr int kMaxTokensPerThread = 4; // (a thread takes tokens x, x + 256, ... of its chunk, so position order = pass order)
#ifndef KVQ_APPEND_DEPTH
#define KVQ_APPEND_DEPTH 2
#endif
#ifndef KVQ_APPEND_MIN_CTAS
#define KVQ_APPEND_MIN_CTAS 3
#endif

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
    int tpt;                           // tokens per thread: a slot-assignment chunk is kChunkTokens * tpt tokens
    // Ragged batches: tokens each sequence adds in this call (nullptr: n_new for all; the input tensors keep
    // n_new rows per sequence) and position of each sequence's first new token (nullptr: pos0 for all).
    const int* lens;
    const int* pos;
    uint32_t* chunk_arrivals;          // [batch] classify CTAs of a sequence that have finished; zero between launches
    // One-launch decode step with a controller wider than 32: the storing CTAs publish each sequence's class here as
    // (step_serial << 2) | class for the attending warps of the same launch (nullptr: nobody asks).
    uint32_t* step_cls;                // [batch]
    uint32_t step_serial;
};

__device__ __forceinline__ int new_tokens_of(const AppendParams& p, int b) { return p.lens ? p.lens[b] : p.n_new; }
__device__ __forceinline__ int first_pos_of(const AppendParams& p, int b) { return p.pos ? p.pos[b] : p.pos0; }

// Class of one token from its bit-width; anything outside {2,4,8,16} is kept as fp16 and flagged.
__device__ __forceinline__ int class_of_bits(int bits, uint32_t* flags) {
    int c = bits_to_class(bits);
    if (c < 0) {
        atomicOr(flags, 1u);
        c = 3;
    }
    return c;
}

__device__ __forceinline__ void reserve_blocks(const StoreView& s, int c, int layer, int b, int h0, int nh,
                                               uint32_t n_old, uint32_t n_new, int lane);

// Launch 1 (only when a sequence's new tokens span several chunks): class of every new token, a class histogram per
// chunk, and -- by the CTA that finishes last for its sequence (an arrival counter, nobody waits) -- the arena blocks
// that the sequence's streams grow into.
template <bool FUSED>
__global__ void __launch_bounds__(kChunkTokens)
k_classify(AppendParams p) {
    extern __shared__ float sW[];
    __shared__ uint32_t wtot[kChunkTokens / 32][4];
    const int chunk = blockIdx.x, b = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (FUSED) {
        controller_stage(sW, p.ctrl, p.hidden);
        __syncthreads();
    }
    uint32_t mine[4] = {0, 0, 0, 0};                   // lane 0: this warp's tokens per class over all passes
    if (FUSED && p.hidden == 32 && p.tpt == 2) {       // the usual prefill shape: both tokens of the thread at once
        const int t0 = chunk * 2 * kChunkTokens + threadIdx.x, t1 = t0 + kChunkTokens;
        const int n_b = new_tokens_of(p, b);
        const bool live0 = t0 < n_b, live1 = t1 < n_b;
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 f0 = live0 ? reinterpret_cast<const float4*>(p.feats)[(size_t)b * p.n_new + t0] : z;
        const float4 f1 = live1 ? reinterpret_cast<const float4*>(p.feats)[(size_t)b * p.n_new + t1] : z;
        int c0 = -1, c1 = -1;
        if (__any_sync(0xffffffffu, live0 || live1)) controller_decide_two32(sW, f0, f1, c0, c1);
        c0 = live0 ? c0 : -1;
        c1 = live1 ? c1 : -1;
        if (live0) {
            p.cls[(size_t)b * p.n_new + t0] = (uint8_t)c0;
            if (p.bits_out) p.bits_out[(size_t)b * p.n_new + t0] = (uint8_t)pool_bits(c0);
        }
        if (live1) {
            p.cls[(size_t)b * p.n_new + t1] = (uint8_t)c1;
            if (p.bits_out) p.bits_out[(size_t)b * p.n_new + t1] = (uint8_t)pool_bits(c1);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) mine[k] += __popc(__ballot_sync(0xffffffffu, c0 == k)) + __popc(__ballot_sync(0xffffffffu, c1 == k));
    } else
    for (int r = 0; r < p.tpt; ++r) {
        const int t = (chunk * p.tpt + r) * kChunkTokens + threadIdx.x;
        const bool live = t < new_tokens_of(p, b);
        int c = -1;
        if (FUSED) {
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
#pragma unroll
        for (int k = 0; k < 4; ++k) mine[k] += __popc(__ballot_sync(0xffffffffu, c == k));
    }
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) wtot[warp][k] = mine[k];
    }
    __syncthreads();
    __shared__ uint32_t is_last;
    if (threadIdx.x == 0) {
        uint4 h = make_uint4(0, 0, 0, 0);
        for (int w = 0; w < kChunkTokens / 32; ++w) {
            h.x += wtot[w][0]; h.y += wtot[w][1]; h.z += wtot[w][2]; h.w += wtot[w][3];
        }
        p.hist[(size_t)b * p.nchunks + chunk] = h;
        __threadfence();                               // the histogram is visible before this CTA is counted
        is_last = atomicAdd(p.chunk_arrivals + b, 1u) + 1u == (uint32_t)p.nchunks;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();                                   // the other chunks' histograms, counted before ours
    if (warp < kNumPools) {                            // warp k reserves for class k
        uint32_t add = 0;
        for (int cc = lane; cc < p.nchunks; cc += 32) {
            const uint4 v = __ldcg(p.hist + (size_t)b * p.nchunks + cc);
            add += warp == 0 ? v.x : warp == 1 ? v.y : warp == 2 ? v.z : v.w;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) add += __shfl_xor_sync(0xffffffffu, add, d);
        const uint32_t n_old = p.counts_in[(size_t)b * 4 + warp];
        reserve_blocks(p.store, warp, p.layer, b, 0, p.store.kv_heads, n_old, n_old + add, lane);
    }
    if (threadIdx.x == 0) p.chunk_arrivals[b] = 0;
}

constexpr float kRoundMagic = 12582912.0f;             // 1.5 * 2^23
constexpr int kAppendDepth = KVQ_APPEND_DEPTH;         // items whose input rows are in flight per warp
constexpr size_t kAppendRingBytes = (size_t)(kChunkTokens / 32) * kAppendDepth * 8 * 32 * sizeof(uint4);

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
                 "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

#ifndef KVQ_APPEND_F32X2
#define KVQ_APPEND_F32X2 1         // the quantizer's subtract and multiply as packed two-lane fp32 operations
#endif
// v0 = fl(fl(fl(x0 - mn) * inv) + magic), v1 likewise: three correctly rounded operations per lane.  The
// subtraction and the product are packed two-lane instructions (same results as the scalar ones); the
// rounding add stays scalar, because a packed product followed by a packed sum is contracted into one
// fused operation by the assembler even with explicit rounding modifiers, and a fused product-sum
// rounds differently where the product is within half an ulp of a tie.
__device__ __forceinline__ void quantize_pair(float x0, float x1, float mn, float inv, float magic, float& v0, float& v1) {
#if KVQ_APPEND_F32X2
    float p0, p1;
    asm("{ .reg .b64 x, m, s;\n mov.b64 x, {%2, %3};\n mov.b64 m, {%4, %4};\n mov.b64 s, {%5, %5};\n"
        " sub.rn.f32x2 x, x, m;\n mul.rn.f32x2 x, x, s;\n mov.b64 {%0, %1}, x; }"
        : "=f"(p0), "=f"(p1)
        : "f"(x0), "f"(x1), "f"(mn), "f"(inv));
    v0 = __fadd_rn(p0, magic);
    v1 = __fadd_rn(p1, magic);
#else
    v0 = __fadd_rn(__fmul_rn(__fsub_rn(x0, mn), inv), magic);
    v1 = __fadd_rn(__fmul_rn(__fsub_rn(x1, mn), inv), magic);
#endif
}

// Codes of the 32 values hp[0..15] packed little-endian into words.  rint is done by adding
// 1.5 * 2^23 (the sum's bit pattern is 0x4B400000 + code); the words are sums of shifted bit patterns
// in wrapping 32-bit arithmetic, minus the constant the 0x4B400000 terms add up to.
template <int CLS, bool CLAMP>
__device__ __forceinline__ void pack_codes(const __half2* hp, float mn, float inv, uint32_t (&w)[pool_half_bytes(CLS) / 4]) {
    constexpr int BITS = pool_bits(CLS), EPW = 32 / BITS, WORDS = pool_half_bytes(CLS) / 4;
    constexpr float LEVELS = (float)((1 << BITS) - 1);
    uint32_t bias = 0;
#pragma unroll
    for (int e = 0; e < EPW; ++e) bias += 0x4B400000u << (BITS * e);
#pragma unroll
    for (int wi = 0; wi < WORDS; ++wi) {
        uint32_t acc = 0u - bias;
#pragma unroll
        for (int e = 0; e < EPW; e += 2) {
            const float2 f = __half22float2(hp[(wi * EPW + e) / 2]);
            float r0, r1;
            if (CLAMP) {
                const float v0 = fminf(__fmul_rn(__fsub_rn(f.x, mn), inv), LEVELS);
                const float v1 = fminf(__fmul_rn(__fsub_rn(f.y, mn), inv), LEVELS);
                r0 = __fadd_rn(v0, kRoundMagic);
                r1 = __fadd_rn(v1, kRoundMagic);
            } else {
                quantize_pair(f.x, f.y, mn, inv, kRoundMagic, r0, r1);
            }
            acc += __float_as_uint(r0) << (BITS * e);
            acc += __float_as_uint(r1) << (BITS * (e + 1));
        }
        w[wi] = acc;
    }
}

// Quantize the half-row this lane holds (raw = its 32 fp16 values = 64 bytes of the input row) with
// class CLS < 3 and store it: the lane's units of the tile's code block `codes`, and (half 0 only)
// the {scale, zero-point} word at `meta`.  Both lanes of a slot (l, l ^ 16) must call together.
// PARTNER: lane distance (xor) to the lane that holds the other half of the same row.
// `tail`: the lane's slot lies beyond the stream's fill (it will be written by a later append); its
// {scale, zero-point} word is cleared so that a reader, which gives such a slot weight zero, never
// multiplies that zero with whatever a recycled block held before.
// G: scale groups per row.  With G == 2 the half-row is a group of its own: no exchange with the partner lane,
// and every lane stores (or clears) the {scale, zero-point} word of its own group at `meta`.
// TENSOR: 0 = K, 1 = V.  With one scale group per row (G == 1: only the one-token append gets here, tiles go
// through k_append_frag.cuh) the codes go into the fragment layout of the decode kernel (kvq_common.cuh): a K
// row's canonical words as 32-bit words, a V row's canonical bytes one by one (they sit slot-minor).
template <int CLS, int PARTNER = 16, int G = 1, int TENSOR = 0>
__device__ __forceinline__ void quantize_store_half_row(const uint4 (&raw)[4], bool active, bool tail, int half, int t,
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
    if (G == 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, PARTNER));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, PARTNER));
    }
    if (mn == 0.0f) mn = 0.0f;                         // -0 is stored as +0
    if (mx == 0.0f) mx = 0.0f;
    const float s32 = __fdiv_rn(__fsub_rn(mx, mn), LEVELS);
    const __half s16 = __float2half_rn(s32);
    const float sf = __half2float(s16);
    const float inv = sf == 0.0f ? 0.0f : __frcp_rn(sf);

    // code_i = min(rint((x_i - mn) * inv), LEVELS); the product is never negative.  With a normal fp16
    // scale the quotient exceeds LEVELS by less than 2^-10 LEVELS, so the clamp only matters for
    // subnormal scales (warp-uniform rare path).
    constexpr int WORDS = pool_half_bytes(CLS) / 4;
    uint32_t w[WORDS];
    const bool tiny = sf != 0.0f && sf < 6.103515625e-05f;
    if (__any_sync(0xffffffffu, tiny)) pack_codes<CLS, true>(hp, mn, inv, w);
    else pack_codes<CLS, false>(hp, mn, inv, w);
    if (!active) {
        if (tail && (G == 2 || half == 0)) *reinterpret_cast<uint32_t*>(meta) = 0u;
        return;
    }
    if (G == 1 && TENSOR == 0) {
#pragma unroll
        for (int wi = 0; wi < WORDS; ++wi)
            *reinterpret_cast<uint32_t*>(codes + kfrag_word_offset(CLS, t, half * WORDS + wi)) = w[wi];
    } else if (G == 1) {                               // a single token: its V bytes one by one
#pragma unroll
        for (int wi = 0; wi < WORDS; ++wi)
#pragma unroll
            for (int b = 0; b < 4; ++b)
                codes[vfrag_byte_offset(CLS, t, 4 * (half * WORDS + wi) + b)] = (uint8_t)(w[wi] >> (8 * b));
    } else if (CLS == 0) {
        *reinterpret_cast<uint2*>(codes + unit_offset(0, half, 0, t)) = make_uint2(w[0], w[1]);
    } else {
#pragma unroll
        for (int u = 0; u < WORDS / 4; ++u)
            *reinterpret_cast<uint4*>(codes + unit_offset(CLS, half, u, t)) =
                make_uint4(w[4 * u], w[4 * u + 1], w[4 * u + 2], w[4 * u + 3]);
    }
    if (G == 2 || half == 0)
        *reinterpret_cast<uint32_t*>(meta) =
            (uint32_t)__half_as_ushort(s16) | ((uint32_t)__half_as_ushort(__float2half_rn(mn)) << 16);
}

// Reserve the blocks that class c of the streams (layer, b, heads h0 .. h0+nh) grows into when its fill
// goes from n_old to n_new tokens.  Called by one warp; the new table entries are visible to the
// CTA after its next barrier and to later launches.
__device__ __forceinline__ void reserve_blocks(const StoreView& s, int c, int layer, int b, int h0, int nh,
                                               uint32_t n_old, uint32_t n_new, int lane) {
    const uint32_t have = blocks_for(c, n_old, s.groups), want = blocks_for(c, n_new, s.groups);
    if (want == have) return;
    const uint32_t per = want - have;
    uint32_t first = 0;
    if (lane == 0) first = arena_take(s, per * (uint32_t)nh);
    first = __shfl_sync(0xffffffffu, first, 0);
    for (uint32_t i = lane; i < per * (uint32_t)nh; i += 32) {
        const uint32_t hh = i / per, j = i - hh * per;
        stream_table(s, c, layer, b, h0 + (int)hh)[have + j] = first ? first + i : 0u;
    }
}

// Launch 2.  MODE 0: classes come from k_classify (several chunks per sequence);
// MODE 1: one chunk, classes from `bits`; MODE 2: one chunk, classes from the controller.
// R: tokens per thread (= p.tpt): a chunk is 256 R tokens.  A 16-slot tile that a chunk only partly fills
// costs as much as a full one, and every class has one at each end of a chunk, so long prefills take R = 4
// (about 94 % of the slots a warp works on hold a token, against 81 % with R = 1).
// grid = (nchunks, head_groups, batch), block = 256.
template <int MODE, int G, int R = 1>
__global__ void __launch_bounds__(kChunkTokens, KVQ_APPEND_MIN_CTAS)
k_quant_pack(AppendParams p) {
    static_assert(MODE == 0 || R == 1, "single-chunk appends hold at most 256 tokens per sequence");
    constexpr int CT = kChunkTokens * R;               // tokens per chunk
    extern __shared__ __align__(16) uint8_t dyn_smem[];   // [ring: warps x depth x 4 KB][controller block (MODE 2)]
    uint8_t* ring_raw = dyn_smem;
    float* sW = reinterpret_cast<float*>(dyn_smem + kAppendRingBytes);
    __shared__ uint32_t wtot[R][kChunkTokens / 32][4];
    __shared__ uint32_t base[4];
    __shared__ uint16_t list[4][CT];                   // tokens of the chunk by class, in slot order
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
            for (int w = 0; w < kChunkTokens / 32; ++w) before += wtot[rr][w][c[r]];
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
            for (int w = 0; w < kChunkTokens / 32; ++w) ncls[k] += wtot[r][w][k];
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
    __syncthreads();

    // ---- tiles: class k touches tiles [first[k], first[k] + nt[k]) of its pool
    uint32_t first[4], pre[5];
    pre[0] = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        first[k] = base[k] / kTileTokens;
        uint32_t nt = ncls[k] ? (base[k] + ncls[k] - 1) / kTileTokens - first[k] + 1 : 0;
        // The append's last chunk also visits the partly filled last tile of a class that got no token in
        // this chunk, only to clear the {scale, zero-point} words of its unused slots (see `tail`).
        if (ncls[k] == 0 && chunk == p.nchunks - 1 && base[k] % kTileTokens != 0) nt = 1;
        pre[k + 1] = pre[k] + nt;
    }
    const int half = lane >> 4, t = lane & 15;
    // Work items (tile tau, head hh), heads fastest, dealt round-robin to the warps.  The input rows of
    // the next kAppendDepth items are kept in flight with per-lane 16-byte async copies into a per-warp
    // ring in shared memory.  For copying, lanes 2j and 2j+1 take adjacent 16-byte pieces (2i, 2i+1) of
    // the row of slot j, so neighbouring lanes complete a 32-byte sector; each lane then reads the
    // contiguous half-row it quantizes (pieces 4*half + i of slot lane%16) back from the ring.  A stage
    // holds [tensor][piece 0..7][slot 0..15] 16-byte pieces, odd pieces rotated by four slots so that
    // neither access pattern has bank conflicts.
    struct Item {
        int k;                                         // class, -1 = no more items
        bool active, tail;                             // the lane's slot gets a token / lies beyond the fill
        uint8_t* rec;                                  // the tile record (found through the stream's block table)
    };
    uint32_t tau = 0;
    int hh = warp;
    auto settle = [&]() {
        while (hh >= nh) {
            hh -= nh;
            ++tau;
        }
    };
    settle();
    uint4* my_ring = reinterpret_cast<uint4*>(ring_raw) + (size_t)warp * kAppendDepth * 8 * 32;
    // describe the next item and start the copies of its rows into ring stage `stage`
    auto next_item = [&](int stage) {
        Item it;
        it.k = -1;
        it.active = it.tail = false;
        it.rec = nullptr;
        if (tau < pre[4]) {
            const int k = (tau >= pre[1]) + (tau >= pre[2]) + (tau >= pre[3]);
            const uint32_t basek = k == 0 ? base[0] : k == 1 ? base[1] : k == 2 ? base[2] : base[3];
            const uint32_t nk = k == 0 ? ncls[0] : k == 1 ? ncls[1] : k == 2 ? ncls[2] : ncls[3];
            it.k = k;
            const uint32_t tile = (k == 0 ? first[0] : k == 1 ? first[1] : k == 2 ? first[2] : first[3]) +
                                  (tau - (k == 0 ? pre[0] : k == 1 ? pre[1] : k == 2 ? pre[2] : pre[3]));
            const uint32_t r0 = tile * kTileTokens - basek;        // rank of the tile's slot 0 in the chunk (may wrap)
            it.active = r0 + t < nk;                               // the slot this lane quantizes
            // beyond the fill only in the append's last chunk (otherwise the next chunk's tokens go there)
            it.tail = !it.active && (int32_t)(r0 + t) >= 0 && chunk == p.nchunks - 1;
            const int h = h0 + hh;
            it.rec = tile_ptr(p.store, k, stream_table(p.store, k, p.layer, b, h), tile, G);
            const uint32_t r_ld = r0 + (lane >> 1);                // the slot this lane copies a piece of
            if (r_ld < nk) {
                const int i_tok = list[k][r_ld];
                const size_t src = (((size_t)b * p.n_new + (size_t)chunk * CT + i_tok) * p.store.kv_heads + h) *
                                   kHeadDim;
                const int odd = lane & 1;
                const uint4* ks = reinterpret_cast<const uint4*>(p.K + src) + odd;
                const uint4* vs = reinterpret_cast<const uint4*>(p.V + src) + odd;
                uint4* dst = my_ring + (size_t)stage * 8 * 32 + odd * 16 + (((lane >> 1) + 4 * odd) & 15);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    cp_async16(dst + (2 * i) * 16, ks + 2 * i);            // piece 2i + odd of K
                    cp_async16(dst + (8 + 2 * i) * 16, vs + 2 * i);        // piece 2i + odd of V
                }
            }
            hh += kChunkTokens / 32;
            settle();
        }
        cp_async_commit();                             // one group per call, possibly empty
        return it;
    };
    Item items[kAppendDepth];
#pragma unroll
    for (int d = 0; d < kAppendDepth; ++d) items[d] = next_item(d);
    int stage = 0;
    while (items[0].k >= 0) {
        cp_async_wait<kAppendDepth - 1>();             // this lane's copies of the oldest group have landed
        __syncwarp();                                  // ... and so have its partner's
        const Item cur = items[0];
        uint4 kraw[4], vraw[4];
        const uint4* src = my_ring + (size_t)stage * 8 * 32 + (4 * half) * 16;
#pragma unroll
        for (int i = 0; i < 4; ++i) {                  // piece 4*half + i sits at slot (t + 4*(i&1)) % 16
            const int at = i * 16 + ((t + 4 * (i & 1)) & 15);
            kraw[i] = cur.active ? src[at] : make_uint4(0, 0, 0, 0);
            vraw[i] = cur.active ? src[8 * 16 + at] : make_uint4(0, 0, 0, 0);
        }
        __syncwarp();                                  // every lane has read the stage before it is refilled
#pragma unroll
        for (int d = 0; d + 1 < kAppendDepth; ++d) items[d] = items[d + 1];
        items[kAppendDepth - 1] = next_item(stage);
        if (++stage == kAppendDepth) stage = 0;

        uint8_t* rec = cur.rec;
        uint8_t* vcodes = rec + pool_codes_bytes(cur.k);
        const bool active = cur.active;
        switch (cur.k) {
        case 0:
            quantize_store_half_row<0, 16, G>(kraw, active, cur.tail, half, t, rec, rec + meta_offset(0, 0, t, half, G));
            quantize_store_half_row<0, 16, G, 1>(vraw, active, cur.tail, half, t, vcodes, rec + meta_offset(0, 1, t, half, G));
            break;
        case 1:
            quantize_store_half_row<1, 16, G>(kraw, active, cur.tail, half, t, rec, rec + meta_offset(1, 0, t, half, G));
            quantize_store_half_row<1, 16, G, 1>(vraw, active, cur.tail, half, t, vcodes, rec + meta_offset(1, 1, t, half, G));
            break;
        case 2:
            quantize_store_half_row<2, 16, G>(kraw, active, cur.tail, half, t, rec, rec + meta_offset(2, 0, t, half, G));
            quantize_store_half_row<2, 16, G, 1>(vraw, active, cur.tail, half, t, vcodes, rec + meta_offset(2, 1, t, half, G));
            break;
        default:                                       // fp16: the lane's 64 input bytes are its four units
            if (active) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    *reinterpret_cast<uint4*>(rec + unit_offset(3, half, u, t)) = kraw[u];
                    *reinterpret_cast<uint4*>(vcodes + unit_offset(3, half, u, t)) = vraw[u];
                }
            }
            break;
        }
    }
    cp_async_wait<0>();
}

// The stores of k_append_token: both tensors of the lane's half-row into the tile record `rec`.
template <int G>
__device__ __forceinline__ void token_store(int c, const uint4 (&kraw)[4], const uint4 (&vraw)[4], bool active, int half,
                                            int t, uint8_t* rec) {
    uint8_t* vcodes = rec + pool_codes_bytes(c);
    if (t == 0 && c < 3 && active) {                   // the token opens a tile: clear the tile's {scale, zero-point} words
        if (G == 1) {
            uint4* m = reinterpret_cast<uint4*>(rec + meta_offset(c, half, 0));    // half 0: K words, half 1: V words
#pragma unroll
            for (int i = 0; i < 4; ++i) m[i] = make_uint4(0, 0, 0, 0);
        } else {                                       // the planes of this lane's group, for K and for V
#pragma unroll
            for (int tensor = 0; tensor < 2; ++tensor) {
                uint4* m = reinterpret_cast<uint4*>(rec + meta_offset(c, tensor, 0, half, 2));
#pragma unroll
                for (int i = 0; i < 4; ++i) m[i] = make_uint4(0, 0, 0, 0);
            }
        }
    }
    __syncwarp();                                      // slot 0's own word is written after the clearing
    switch (c) {
    case 0:
        quantize_store_half_row<0, 1, G>(kraw, active, false, half, t, rec, rec + meta_offset(0, 0, t, half, G));
        quantize_store_half_row<0, 1, G, 1>(vraw, active, false, half, t, vcodes, rec + meta_offset(0, 1, t, half, G));
        break;
    case 1:
        quantize_store_half_row<1, 1, G>(kraw, active, false, half, t, rec, rec + meta_offset(1, 0, t, half, G));
        quantize_store_half_row<1, 1, G, 1>(vraw, active, false, half, t, vcodes, rec + meta_offset(1, 1, t, half, G));
        break;
    case 2:
        quantize_store_half_row<2, 1, G>(kraw, active, false, half, t, rec, rec + meta_offset(2, 0, t, half, G));
        quantize_store_half_row<2, 1, G, 1>(vraw, active, false, half, t, vcodes, rec + meta_offset(2, 1, t, half, G));
        break;
    default:
        if (active) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                *reinterpret_cast<uint4*>(rec + unit_offset(3, half, u, t)) = kraw[u];
                *reinterpret_cast<uint4*>(vcodes + unit_offset(3, half, u, t)) = vraw[u];
            }
        }
        break;
    }
}

// The stores of k_append_token for a cache with per-channel keys: the key half-row joins the fp16 residual rows of
// its stream (it is packed when its window of 16 slots is complete, by k_pack_window); the value half-row is
// quantized per token as in the other layouts.  kres: the stream's residual rows of class c, [16][64].
__device__ __forceinline__ void token_store_pc(int c, const uint4 (&kraw)[4], const uint4 (&vraw)[4], bool active, int half,
                                               int t, uint8_t* rec, __half* kres) {
    uint8_t* vcodes = rec + pool_codes_bytes(c);
    if (t == 0 && c < 3 && active && half == 0) {      // the token opens a tile: clear the tile's value {scale, zero-point} words
        uint4* m = reinterpret_cast<uint4*>(rec + meta_offset(c, 1, 0, 0, kLayoutPerChannelK));
#pragma unroll
        for (int i = 0; i < 4; ++i) m[i] = make_uint4(0, 0, 0, 0);
    }
    __syncwarp();
    if (c < 3 && active) {
#pragma unroll
        for (int u = 0; u < 4; ++u) *reinterpret_cast<uint4*>(kres + t * kHeadDim + 32 * half + 8 * u) = kraw[u];
    }
    uint8_t* vmeta = rec + meta_offset(c < 3 ? c : 0, 1, t, 0, kLayoutPerChannelK);
    switch (c) {
    case 0: quantize_store_half_row<0, 1, 1, 1>(vraw, active, false, half, t, vcodes, vmeta); break;
    case 1: quantize_store_half_row<1, 1, 1, 1>(vraw, active, false, half, t, vcodes, vmeta); break;
    case 2: quantize_store_half_row<2, 1, 1, 1>(vraw, active, false, half, t, vcodes, vmeta); break;
    default:
        if (active) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                *reinterpret_cast<uint4*>(rec + unit_offset(3, half, u, t)) = kraw[u];
                *reinterpret_cast<uint4*>(vcodes + unit_offset(3, half, u, t)) = vraw[u];
            }
        }
        break;
    }
}

// One new token per sequence (a decode step), the work of one warp: the token of sequence b, KV heads
// 16 bx .. 16 bx + 15; lane l handles half-row l % 2 of KV head 16 bx + l / 2.  Everything the warp needs (the K and
// V rows, the pool fills, the features) is requested up front so the loads overlap the controller; the decision is
// taken by the warp (FUSED) or read from `bits`.  ctl says who evaluates the controller: kCtlWarp32 the warp alone
// (hidden width 32); kCtlCtaStaged / kCtlCtaDirect: the warp is the first of four (threads 0..127 of the CTA) that
// evaluate a controller of any width together -- the other three call this too and return after the decision --
// with W2 staged in shared memory (controller_fetch_cta128 has been called by all four; ctrl_sh holds
// kControllerCtaSmemFloats floats) or read straight from global memory (kControllerDirectSmemFloats floats).
constexpr int kCtlWarp32 = 0, kCtlCtaStaged = 1, kCtlCtaDirect = 2;
template <bool FUSED, int G>
__device__ __forceinline__ void append_token_warp(const AppendParams& p, int bx, int b, int ctl, float* ctrl_sh) {
    const int lane = threadIdx.x & 31;
    const int h = bx * 16 + (lane >> 1), half = lane & 1;
    const bool active = h < p.store.kv_heads;
    uint4 kraw[4], vraw[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) kraw[i] = vraw[i] = make_uint4(0, 0, 0, 0);
    if (active) {
        const size_t src = ((size_t)b * p.store.kv_heads + h) * kHeadDim + half * (kHeadDim / 2);
        const uint4* ks = reinterpret_cast<const uint4*>(p.K + src);
        const uint4* vs = reinterpret_cast<const uint4*>(p.V + src);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            kraw[i] = __ldg(ks + i);
            vraw[i] = __ldg(vs + i);
        }
    }
    const uint4 fill = *reinterpret_cast<const uint4*>(p.counts_in + (size_t)b * 4);
    // The block-table entry is needed once the class is known; the four candidates (one per class) are
    // requested now, so that they travel while the controller runs.  An entry of a block that is not
    // reserved yet may hold anything and is not used.
    const int hs = active ? h : 0;
    const uint32_t id0 = stream_table(p.store, 0, p.layer, b, hs)[fill.x / (kTileTokens * block_tiles(0, G))];
    const uint32_t id1 = stream_table(p.store, 1, p.layer, b, hs)[fill.y / (kTileTokens * block_tiles(1, G))];
    const uint32_t id2 = stream_table(p.store, 2, p.layer, b, hs)[fill.z / (kTileTokens * block_tiles(2, G))];
    const uint32_t id3 = stream_table(p.store, 3, p.layer, b, hs)[fill.w / (kTileTokens * block_tiles(3, G))];
    int c;
    if (FUSED) {
        const float4 f = reinterpret_cast<const float4*>(p.feats)[b];
        c = ctl == kCtlWarp32    ? controller_decide_warp32(p.ctrl, f.x, f.y, f.z, f.w, lane)
            : ctl == kCtlCtaStaged ? controller_decide_cta128(p.ctrl, p.hidden, f.x, f.y, f.z, f.w, ctrl_sh)
                                   : controller_decide_cta_direct(p.ctrl, p.hidden, f.x, f.y, f.z, f.w, ctrl_sh);
        if (p.step_cls && bx == 0 && threadIdx.x == 0) {       // for the attending warps of this launch
            const uint32_t word = (p.step_serial << 2) | (uint32_t)c;
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.step_cls + b), "r"(word) : "memory");
        }
        if (ctl != kCtlWarp32 && threadIdx.x >= 32) return;    // the helpers are done
    } else {
        c = class_of_bits(p.bits[b], p.store.flags);
    }
    const uint32_t slot = c == 0 ? fill.x : c == 1 ? fill.y : c == 2 ? fill.z : fill.w;
    if (bx == 0 && lane == 0) {
        p.store.index[((size_t)p.layer * p.store.batch + b) * p.store.max_ctx + first_pos_of(p, b)] = ((uint32_t)c << 30) | slot;
        *reinterpret_cast<uint4*>(p.counts_out + (size_t)b * 4) =
            make_uint4(fill.x + (c == 0), fill.y + (c == 1), fill.z + (c == 2), fill.w + (c == 3));
        if (FUSED && p.bits_out) p.bits_out[b] = (uint8_t)pool_bits(c);
    }
    const int t = (int)(slot & (kTileTokens - 1));
    const uint32_t tile = slot / kTileTokens;
    uint32_t* tab = stream_table(p.store, c, p.layer, b, active ? h : 0);
    if (slot % (kTileTokens * block_tiles(c, G)) == 0) {              // the token opens a new block of its stream
        uint32_t id = 0;
        if (active && half == 0) {
            id = arena_take(p.store, 1);
            tab[tile / block_tiles(c, G)] = id;
        }
        id = __shfl_sync(0xffffffffu, id, lane & ~1);
        // the partner lane must not read the table before the entry is written: hand it the address instead
        uint8_t* rec_new = p.store.arena + (size_t)id * kBlockBytes;
        if constexpr (G == kLayoutPerChannelK)
            token_store_pc(c, kraw, vraw, active, half, t, rec_new, c < 3 ? residual_rows(p.store, c, p.layer, b, active ? h : 0) : nullptr);
        else
            token_store<G>(c, kraw, vraw, active, half, t, rec_new);
        return;
    }
    const uint32_t id = c == 0 ? id0 : c == 1 ? id1 : c == 2 ? id2 : id3;
    uint8_t* rec = p.store.arena + (size_t)id * kBlockBytes + (size_t)(tile % block_tiles(c, G)) * (uint32_t)pool_rec_bytes(c, G);
    if constexpr (G == kLayoutPerChannelK)
        token_store_pc(c, kraw, vraw, active, half, t, rec, c < 3 ? residual_rows(p.store, c, p.layer, b, active ? h : 0) : nullptr);
    else
        token_store<G>(c, kraw, vraw, active, half, t, rec);
}

// grid = (ceil(kv_heads / 16), batch), block = 32 -- or 128 when the controller is wider than 32 hidden units.
template <bool FUSED, int G>
__global__ void __launch_bounds__(128)
k_append_token(AppendParams p) {
    extern __shared__ __align__(16) float ctrl_sh[];    // kControllerCtaSmemFloats floats when four warps evaluate the controller
    pdl_launch_dependents();
    const bool wide = blockDim.x != 32;
    if (FUSED && wide) controller_fetch_cta128(p.ctrl, p.hidden, ctrl_sh);   // no kernel writes the weights
    pdl_wait();                                        // the attention of the previous step still reads the store
    append_token_warp<FUSED, G>(p, (int)blockIdx.x, (int)blockIdx.y, wide ? kCtlCtaStaged : kCtlWarp32, ctrl_sh);
}

}  // namespace kvq
