// Decode-step attention over the mixed-precision cache (Eq. 5):
//   a = Softmax(q K^T / sqrt(d_k)) V,   K, V dequantized on the fly.
//
// Softmax attention does not depend on the order of the cached tokens, so the
// kernel never touches the per-token index: it walks each precision pool of a
// (sequence, KV head) front to back.
//
// Work split.  The (sequence, query head) units are laid end to end on an axis
// x, every unit gw ticks long; working warp j of gw owns ticks
// [j*units, (j+1)*units), i.e. an equal share of the whole launch, cut into
// SEGMENTS where it crosses unit borders.  A segment [a0, a1) of a unit takes
// tiles [nt*a0/gw, nt*a1/gw) of EVERY pool of that unit (the same fraction of
// every pool, hence the same byte and instruction mix for every warp).  Warps
// are independent: each has its own ring, softmax state and accumulators, and
// writes one partial (m, l, o[64]) per segment into the slot of its unit.  A
// counter per unit tells a warp whether it delivered the unit's last partial;
// that warp merges the slots (M = max m_j, l = sum l_j 2^(m_j-M),
// O = sum o_j 2^(m_j-M) / l), writes the fp16 output row and puts the counter
// back to zero.  The launch is persistent when gw is the number of warps
// resident on the device; nothing in the kernel waits for another warp.
//
// Data movement: the tiles of a segment are cut into chunks of up to one stage of
// contiguous bytes; every warp runs its own ring of a few stages (see DecodeGeom) of
// shared-memory buffers filled by 1-D bulk async copies (cp.async.bulk,
// completion on an mbarrier), issued kStages chunks ahead by lane 0.  Every
// mbarrier wait is bounded: on expiry the warp records KVQ_FLAG_WAIT_TIMEOUT
// and stops.
//
// Arithmetic.  Dequantization is hoisted out of the inner loops:
//   q.khat = s_k * sum_i q_i c_i + z_k * sum_i q_i
//   sum_t p_t vhat_t = sum_t (p_t s_t) c_t + sum_t p_t z_t
// so both sides are sums of products of small unsigned codes with a weight.
//
// Caches with one {scale, zero-point} pair per row, and caches with per-channel keys, run both sums on the 8-bit
// integer matrix instructions (FragRows below): the packed codes are the row operand as they are stored
// (kvq_common.cuh stores them in operand order), byte planes cut out with one mask each, and the weights -- the
// query for K, the softmax weights times the value scales for V -- are the column operand as balanced / unsigned
// base-256 digits of a fixed-point number, one digit per column, int32 accumulation.  Two 16-slot tiles per
// iteration, every lane owning one slot's logit and weight.
//
// The fp16 pool, and the quantized pools of caches with two scale groups per row (Quantized below), use the older
// lane mapping: two lanes per token, lane l handles half l/16 (elements 32*(l/16) .. +32) of slot l%16 of a tile,
// with 32 pre-scaled query values and 32 output accumulators in registers; the two half dot products meet through
// one xor-16 shuffle; the output accumulators are per-lane partial sums reduced once per segment.  There the K
// side is an integer dot product over a 24-bit fixed-point query (a signed 16-bit limb through dp2a, a signed
// 8-bit limb through dp4a, codes masked in place into byte planes, the planes' weights undone by a Horner step),
// and the V side feeds masked bit fields to fp32 FMAs as they are: a bit field inside bits [0,24) of a 32-bit
// word, read as an fp32 bit pattern, IS the number code * 2^(k-149) (the subnormal / first-binade encoding is
// linear), so one AND per element isolates it and the power of two is folded into the accumulator's exponent.
#pragma once
#include "kvq_common.cuh"
#include "k_append.cuh"

#ifndef KVQ_SMALL_WARPS
#define KVQ_SMALL_WARPS 16
#endif
#ifndef KVQ_SMALL_STAGES
#define KVQ_SMALL_STAGES 3
#endif
#ifndef KVQ_SMALL_END_TO_END
#define KVQ_SMALL_END_TO_END 1
#endif
#ifndef KVQ_DECODE_FMA2
#define KVQ_DECODE_FMA2 1          // fp16 pool: V-side accumulation with packed two-lane fp32 FMAs
#endif

namespace kvq {

// Launch geometry.  The kernel is instantiated twice:
//   Large: 4 warps per CTA, 4 CTAs per SM, per-warp rings of two 6.5 KB stages -- the bandwidth configuration
//          (16 resident warps per SM, 209 KB of rings);
//   Small: 16 warps per CTA, 1 CTA per SM, per-warp rings of three 4.25 KB stages -- for launches of few warps,
//          where a warp's whole share is in flight at once and the parts of a (sequence, query head) unit sit in
//          one CTA, which merges them through shared memory (no partial records, no global counter).
template <int WARPS, int STAGES, int STAGE_BYTES, int MIN_CTAS>
struct DecodeGeom {
    static constexpr int kWarps = WARPS, kThreads = WARPS * 32, kStages = STAGES, kStageBytes = STAGE_BYTES, kCtasPerSm = MIN_CTAS;
    static constexpr size_t kSmemBytes = (size_t)WARPS * STAGES * STAGE_BYTES;
    static constexpr bool kCtaMerge = true;            // units cut into a divisor of WARPS parts are merged inside their CTA
    // One CTA per SM is the geometry of short caches, where a launch is a chain of latencies and a tile costs a warp
    // the same time whatever its class: there a warp's share is a stretch of the unit's pools laid end to end.  In
    // the bandwidth geometry every warp takes the same fraction of every pool, so that all warps move the same bytes.
    static constexpr bool kPoolsEndToEnd = KVQ_SMALL_END_TO_END && MIN_CTAS == 1;
    // tiles of class c that fit one stage
    __host__ __device__ static constexpr int tps(int c, int g = 1) { return STAGE_BYTES / pool_rec_bytes(c, g); }
    static_assert(STAGE_BYTES % 16 == 0 && STAGE_BYTES >= pool_rec_bytes(3), "a stage must hold one fp16 tile");
};
using GeomLarge = DecodeGeom<4, 2, 6528, 4>;          // 10 / 5 / 3 / 1 tiles of the four classes per stage
using GeomSmall = DecodeGeom<KVQ_SMALL_WARPS, KVQ_SMALL_STAGES, 4352, 1>;    //  6 / 3 / 2 / 1

constexpr int kHalfDim = kHeadDim / 2;           // elements per lane
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLogitScale = 0.125f * kLog2e;   // 1/sqrt(64), in log2 units
constexpr float kRescaleSlack = 8.0f;            // the running maximum may lag by 2^8 before a rescale
constexpr float kNegBig = -1.0e30f;
constexpr uint32_t kWaitLimit = 1u << 20;        // mbarrier polls before a wait is abandoned
constexpr uint32_t kFlagWaitTimeout = 2u;

struct DecodeParams {
    StoreView store;
    const uint32_t* counts;        // [batch][4] pool fills of this layer
    const __half* Q;               // [batch][t_total][q_heads][64]
    __half* O;                     // [batch][t_total][q_heads][64]
    float* part_o;                 // [units][pslots][64]  unnormalised
    float2* part_ml;               // [units][pslots]      (m in log2 units, l)
    uint32_t* part_cnt;            // [units] partials delivered so far; zero between launches
    float* part_s2;                // [units][pslots] sum of p^2 (statistics variant only)
    float* unit_var;               // [units] variance of the unit's attention weights (statistics variant only)
    int layer, group;              // group = q_heads / kv_heads
    // Query rows per sequence.  A decode step has one (tq = t_total = 1, t0 = 0).  With several (the last
    // t_total cached tokens each ask, causally), a launch serves rows t0 .. t0+tq of every sequence and
    // `counts` has one row of visible pool fills per (sequence, query row of the launch).
    uint32_t tq, t_total, t0;
    uint32_t units;                // batch * tq * q_heads
    uint32_t gw;                   // working warps = parts the x axis is cut into
    uint32_t pslots;               // partial slots per unit = decode_pslots(units, gw)
    uint32_t cta_parts;            // > 0: gw = units * cta_parts and the parts of a unit share a CTA, which merges them itself
    // One-launch decode step with a controller wider than 32 (k_decode_step<.., true>): the attending CTAs start at
    // block cta0 (the storing CTAs come first) and read each sequence's class from step_cls, where a storing CTA of
    // the same launch publishes it as (step_serial << 2) | class.
    uint32_t cta0;
    const uint32_t* step_cls;
    uint32_t step_serial;
};

// Warps that can overlap one unit: ceil(gw/units) + 1.
__host__ __device__ inline uint32_t decode_pslots(uint32_t units, uint32_t gw) { return (gw + units - 1) / units + 1; }
// First warp whose share overlaps unit u, and the number of warps that do.
__host__ __device__ inline uint32_t decode_first_warp(uint32_t u, uint32_t units, uint32_t gw) {
    return (uint32_t)((uint64_t)u * gw / units);
}
__host__ __device__ inline uint32_t decode_warps_of_unit(uint32_t u, uint32_t units, uint32_t gw) {
    return (uint32_t)(((uint64_t)(u + 1) * gw - 1) / units) - decode_first_warp(u, units, gw) + 1;
}

// ---------------------------------------------------------------- PTX helpers

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
// Bounded wait; false if the phase did not complete within kWaitLimit polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < kWaitLimit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// 1-D bulk async copy global -> shared, completion counted in bytes on `bar`.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// d = c + a.h0 * b.b0 + a.h1 * b.b1 (lo) or a.h0 * b.b2 + a.h1 * b.b3 (hi); a signed 16-bit, b unsigned 8-bit.
__device__ __forceinline__ int dp2a_lo(uint32_t a, uint32_t b, int c) {
    int d;
    asm("dp2a.lo.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ int dp2a_hi(uint32_t a, uint32_t b, int c) {
    int d;
    asm("dp2a.hi.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// d = c + sum_j a.b_j * b.b_j; a signed 8-bit, b unsigned 8-bit.
__device__ __forceinline__ int dp4a_su(uint32_t a, uint32_t b, int c) {
    int d;
    asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

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

// c0 += a0 * b, c1 += a1 * b as one packed instruction (two fp32 lanes in a 64-bit register pair).
__device__ __forceinline__ void fma2(float& c0, float& c1, float a0, float a1, float b) {
#if KVQ_DECODE_FMA2
    asm("{ .reg .b64 a, b, c;\n mov.b64 a, {%2, %3};\n mov.b64 b, {%4, %4};\n mov.b64 c, {%0, %1};\n"
        " fma.rn.f32x2 c, a, b, c;\n mov.b64 {%0, %1}, c; }"
        : "+f"(c0), "+f"(c1)
        : "f"(a0), "f"(a1), "f"(b));
#else
    c0 = fmaf(a0, b, c0);
    c1 = fmaf(a1, b, c1);
#endif
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

// What the store will hold for two elements of a 64-element row that the warp quantizes at class c (Eq. 24, the row
// quantizer of k_append.cuh followed by x^ = code * scale + zero-point): every lane passes two of the row's elements,
// all lanes the same c.  Class 3 keeps the fp16 values.
// G = 2: the row has two scale groups of 32 elements, each quantized on its own; the lanes of a half-warp hold one.
template <int G>
__device__ __forceinline__ float2 row_values_as_stored(float2 x, int c) {
    if (c == 3) return x;
    float mn = -fminf(x.x, x.y), mx = fmaxf(x.x, x.y);
#pragma unroll
    for (int d = G == 2 ? 8 : 16; d > 0; d >>= 1) {
        mn = fmaxf(mn, __shfl_xor_sync(0xffffffffu, mn, d));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    }
    mn = -mn;
    if (mn == 0.0f) mn = 0.0f;                         // -0 is stored as +0
    if (mx == 0.0f) mx = 0.0f;
    const float levels = c == 0 ? 3.0f : c == 1 ? 15.0f : 255.0f;
    const float sf = __half2float(__float2half_rn(__fdiv_rn(__fsub_rn(mx, mn), levels)));
    const float inv = sf == 0.0f ? 0.0f : __frcp_rn(sf);
    const float c0 = rintf(fminf(__fmul_rn(__fsub_rn(x.x, mn), inv), levels));
    const float c1 = rintf(fminf(__fmul_rn(__fsub_rn(x.y, mn), inv), levels));
    return make_float2(__fadd_rn(__fmul_rn(c0, sf), mn), __fadd_rn(__fmul_rn(c1, sf), mn));
}

__device__ __forceinline__ float half_sum(float v) {    // over the 16 lanes of a half-warp
#pragma unroll
    for (int d = 8; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

// STATS: also keep the sum of squared weights (for the attention-variance feature of Eq. 16).
template <bool STATS>
struct SoftmaxT {
    float m, l, bsum;              // running max (log2 units), sum of p, sum of p * zero-point
    float thr;                     // m + kRescaleSlack: a logit above it forces a rescale
    static constexpr bool kStats = STATS;
    float s2;                      // sum of p^2 (STATS only)
    float of[4];                   // fragment path: this lane's four output channels, sum of (p s) c so far
};

// Fold a tile's logits into the running state and return this lane's p.  The running maximum
// is only raised when some logit exceeds it by more than kRescaleSlack (one vote per tile).
// COUNT: whether this lane adds its p to the running sum (with two lanes per token only one of them may,
// unless the sum is halved afterwards).
template <bool STATS>
__device__ __forceinline__ float softmax_step(SoftmaxT<STATS>& st, float (&acc)[kHalfDim], float y, bool COUNT = true) {
    if (__any_sync(0xffffffffu, y > st.thr)) {                     // warp-uniform
        const float tmax = warp_max(y);
        const float f = fast_exp2(st.m - tmax);
        st.m = tmax;
        st.thr = tmax + kRescaleSlack;
        st.l *= f;
        st.bsum *= f;
        if (STATS) st.s2 *= f * f;
#pragma unroll
        for (int j = 0; j < 4; ++j) st.of[j] *= f;
#pragma unroll
        for (int j = 0; j < kHalfDim; ++j) acc[j] *= f;
    }
    const float p = fast_exp2(y - st.m);
    st.l += COUNT ? p : 0.f;
    if (STATS) st.s2 = COUNT ? fmaf(p, p, st.s2) : st.s2;
    return p;
}

__device__ __forceinline__ float2 meta_to_float2(uint32_t m) {     // {scale, zero-point}
    return __half22float2(*reinterpret_cast<const __half2*>(&m));
}

// ---------------------------------------------------------------- tile consumers (data in shared memory)
// Every consumer sees one 16-token tile record `rec`; the lane handles half `half` of slot `t`.

// What a consumer needs to know about the query of the current segment.
struct QueryInfo {
    const float* q_half;           // this lane's 32 query values (shared memory)
    float fix_scale;               // 256 R: rint(q * 256 R) is the 24-bit fixed-point query
    float inv_fix;                 // kLogitScale / (256 R)
    float sumq;                    // kLogitScale * sum_i q_i over the row (over this lane's half with two scale groups)
};
constexpr int kQRegs = kHalfDim;   // registers a consumer may use for its copy of the query

// G: scale groups per row (1: one {scale, zero-point} per row; 2: one per half-row).
template <int CLS, int G = 1>
struct Quantized {
    static constexpr int BITS = pool_bits(CLS), REC = pool_rec_bytes(CLS, G);
    static constexpr int EPW = 32 / BITS;              // elements per 32-bit word
    static constexpr int WORDS = pool_half_bytes(CLS) / 4;         // words per half-row: 2, 4, 8
    static constexpr int UNITS = pool_units(CLS), UWORDS = pool_unit_bytes(CLS) / 4;
    static constexpr int PLANES = 8 / BITS;            // codes per byte: 4, 2, 1
    static constexpr uint32_t PLANE0 = 0x01010101u * ((1u << BITS) - 1u);   // mask of plane 0

    // Element (inside the half-row) that sits in byte j of plane k of word wi.
    __device__ static constexpr int element(int wi, int k, int j) { return wi * EPW + j * PLANES + k; }

    // The fixed-point query T = 256 * hi + lo.  qreg[0..15]: hi as 16-bit pairs, pair (wi, k, hh) = bytes
    // 2hh, 2hh+1 of plane k of word wi; qreg[16..23]: lo as 8-bit quads, quad (wi, k) = bytes 0..3 of that
    // plane.  The accumulators move to this class's exponent domain (for the V side).
    __device__ static __forceinline__ void enter(const QueryInfo& qi, uint32_t (&qreg)[kQRegs], float (&acc)[kHalfDim]) {
#pragma unroll
        for (int wi = 0; wi < WORDS; ++wi)
#pragma unroll
            for (int k = 0; k < PLANES; ++k) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int T = __float2int_rn(qi.q_half[element(wi, k, j)] * qi.fix_scale);
                    const int h = (T + 128) >> 8;                  // T = 256 h + l, -128 <= l <= 127
                    hi[j] = (uint32_t)h & 0xffffu;
                    lo[j] = (uint32_t)(T - (h << 8)) & 0xffu;
                }
                qreg[(wi * PLANES + k) * 2] = hi[0] | (hi[1] << 16);
                qreg[(wi * PLANES + k) * 2 + 1] = hi[2] | (hi[3] << 16);
                qreg[16 + wi * PLANES + k] = lo[0] | (lo[1] << 8) | (lo[2] << 16) | (lo[3] << 24);
            }
#pragma unroll
        for (int i = 0; i < kHalfDim; ++i) acc[i] *= pow2f(field_pos<BITS>(i % EPW) - 49);
    }
    __device__ static __forceinline__ void leave(float (&acc)[kHalfDim]) {
#pragma unroll
        for (int i = 0; i < kHalfDim; ++i) acc[i] *= pow2f(49 - field_pos<BITS>(i % EPW));
    }
    __device__ static __forceinline__ void load_half_row(const uint8_t* codes, int half, int t, uint32_t (&w)[WORDS]) {
#pragma unroll
        for (int u = 0; u < UNITS; ++u) {
            if (UWORDS == 2) {
                const uint2 v = *reinterpret_cast<const uint2*>(codes + unit_offset(CLS, half, u, t));
                w[0] = v.x; w[1] = v.y;
            } else {
                const uint4 v = *reinterpret_cast<const uint4*>(codes + unit_offset(CLS, half, u, t));
                w[4 * u] = v.x; w[4 * u + 1] = v.y; w[4 * u + 2] = v.z; w[4 * u + 3] = v.w;
            }
        }
    }
    // The K half-row and K meta word of a tile, fetched from shared memory one tile ahead of their use.
    struct KIn {
        uint32_t w[WORDS];
        uint32_t meta;
    };
    __device__ static __forceinline__ KIn load_k(const uint8_t* rec, int half, int t) {
        KIn k;
        load_half_row(rec, half, t, k.w);
        k.meta = *reinterpret_cast<const uint32_t*>(rec + meta_offset(CLS, 0, t, half, G));
        return k;
    }
    template <class SM>
    __device__ static __forceinline__ void tile(const uint8_t* rec, const KIn& kin, bool valid, int half, int t,
                                                const uint32_t (&qreg)[kQRegs], const QueryInfo& qi, SM& st,
                                                float (&acc)[kHalfDim]) {
        uint32_t w[WORDS];
#pragma unroll
        for (int i = 0; i < WORDS; ++i) w[i] = kin.w[i];
        const float2 km = meta_to_float2(kin.meta);
        uint32_t wv_codes[WORDS];                      // the V side's inputs are requested before the K arithmetic
        load_half_row(rec + pool_codes_bytes(CLS), half, t, wv_codes);
        const uint32_t vmeta = *reinterpret_cast<const uint32_t*>(rec + meta_offset(CLS, 1, t, half, G));
        int dh[PLANES], dl[PLANES];
#pragma unroll
        for (int k = 0; k < PLANES; ++k) dh[k] = dl[k] = 0;
#pragma unroll
        for (int wi = 0; wi < WORDS; ++wi)
#pragma unroll
            for (int k = 0; k < PLANES; ++k) {
                const uint32_t plane = PLANES == 1 ? w[wi] : (w[wi] & (PLANE0 << (k * BITS)));   // bytes = code << k*BITS
                dh[k] = dp2a_lo(qreg[(wi * PLANES + k) * 2], plane, dh[k]);
                dh[k] = dp2a_hi(qreg[(wi * PLANES + k) * 2 + 1], plane, dh[k]);
                dl[k] = dp4a_su(qreg[16 + wi * PLANES + k], plane, dl[k]);
            }
        int hsum = dh[0], lsum = dl[0];                // Horner: sum_k d[k] * 2^(BITS*(PLANES-1-k))
#pragma unroll
        for (int k = 1; k < PLANES; ++k) {
            hsum = (hsum << BITS) + dh[k];
            lsum = (lsum << BITS) + dl[k];
        }
        float dot = fmaf((float)hsum, 256.0f, (float)lsum);
        if (G == 1) dot += __shfl_xor_sync(0xffffffffu, dot, 16);  // the other half of the row
        float y = fmaf(km.x * (qi.inv_fix * (1.0f / (float)(1 << (BITS * (PLANES - 1))))), dot, km.y * qi.sumq);
        if (G == 2) y += __shfl_xor_sync(0xffffffffu, y, 16);      // each half carries its own scale and zero-point
        y = valid ? y : -INFINITY;
        const float p = softmax_step(st, acc, y);

#pragma unroll
        for (int i = 0; i < WORDS; ++i) w[i] = wv_codes[i];
        const float2 vm = meta_to_float2(vmeta);
        const float wv = (p * vm.x) * pow2f(100);
        st.bsum = fmaf(p, vm.y, st.bsum);
#pragma unroll
        for (int wi = 0; wi < WORDS; ++wi) {
            const uint32_t hi8 = w[wi] >> 8;
#pragma unroll
            for (int e = 0; e < EPW; e += 2) {
                const int i = wi * EPW + e;
                fma2(acc[i], acc[i + 1], field_as_float<BITS>(w[wi], hi8, e), field_as_float<BITS>(w[wi], hi8, e + 1), wv);
            }
        }
    }
};

// The fp16 pool: rows are stored unchanged; qk holds the plain query.
// BOTH: both lanes of a token add its p to the running sum (which is then halved at the end of the segment).
template <bool BOTH>
struct Fp16Rows {
    static constexpr int REC = pool_rec_bytes(3), UNITS = pool_units(3), WORDS = pool_half_bytes(3) / 4;
    __device__ static __forceinline__ void enter(const QueryInfo& qi, uint32_t (&qreg)[kQRegs], float (&)[kHalfDim]) {
#pragma unroll
        for (int i = 0; i < kHalfDim; ++i) qreg[i] = __float_as_uint(qi.q_half[i] * kLogitScale);
    }
    __device__ static __forceinline__ void leave(float (&)[kHalfDim]) {}
    struct KIn {};                                     // fp16 rows are read where they are used
    __device__ static __forceinline__ KIn load_k(const uint8_t*, int, int) { return KIn{}; }
    template <class SM>
    __device__ static __forceinline__ void tile(const uint8_t* rec, const KIn&, bool valid, int half, int t,
                                                const uint32_t (&qreg)[kQRegs], const QueryInfo&, SM& st,
                                                float (&acc)[kHalfDim]) {
        float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int u = 0; u < UNITS; ++u) {
            const uint4 w4 = *reinterpret_cast<const uint4*>(rec + unit_offset(3, half, u, t));
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[wi]));
                d[wi] = fmaf(f.x, __uint_as_float(qreg[u * 8 + wi * 2]), d[wi]);
                d[wi] = fmaf(f.y, __uint_as_float(qreg[u * 8 + wi * 2 + 1]), d[wi]);
            }
        }
        float y = (d[0] + d[1]) + (d[2] + d[3]);
        y += __shfl_xor_sync(0xffffffffu, y, 16);
        y = valid ? y : -INFINITY;
        const float p = softmax_step(st, acc, y, BOTH || half == 0);
#pragma unroll
        for (int u = 0; u < UNITS; ++u) {
            uint4 w4 = *reinterpret_cast<const uint4*>(rec + pool_codes_bytes(3) + unit_offset(3, half, u, t));
            if (!valid) w4 = make_uint4(0, 0, 0, 0);               // stale bytes may hold anything
            const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
            for (int wi = 0; wi < 4; ++wi) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[wi]));
                fma2(acc[u * 8 + wi * 2], acc[u * 8 + wi * 2 + 1], f.x, f.y, p);
            }
        }
    }
};


// ---------------------------------------------------------------- fragment path (one scale group per row)
//
// The quantized pools of a cache with one {scale, zero-point} pair per row are read with 8-bit integer matrix
// instructions (mma.sync m16n8k32 / m16n8k16, int32 accumulation: exact), two 16-slot tiles (A, B) per loop
// iteration.  Lane L = 4 g + q.
//
// K side: D[slot][column] = sum over the row's code bytes of code * digit, with the codes of a tile's 16 slots
// as the row operand and the query as the column operand.  The byte planes of the packed words are masked IN
// PLACE (code << 2p for plane p of a 2-bit byte, code << 4p of a 4-bit byte); the weight 4^p or 16^p that a
// plane carries is undone on the query's side: q is put on a fixed-point grid once per segment,
// T_i = rint(q_i * F * 4^(3-p)) for a channel that sits in plane p (16^(1-p) for 4-bit codes), so that every
// product comes out as 64 F q c (16 F q c, F q c).  |q_i F| < 2^22, hence |T_i| < 2^28 = four balanced base-256
// digits, T = d0 + 256 d1 + 65536 d2 + 2^24 d3, -128 <= d < 128.  Tile A's products use columns 0..3 = digits
// 0..3 (columns 4..7 zero), tile B's columns 4..7, and both accumulate into the same registers: lane (g, q) then
// holds, for q = 0: digits 0, 1 of A's slots g and g + 8, q = 1: digits 2, 3 of the same, q = 2, 3: the same of
// tile B.  One exchange between lanes q and q ^ 1 gives every lane the dot product of ONE slot, which it OWNS:
// slot g + 8 (q & 1) of tile A (q < 2) or B (q >= 2).  The owner evaluates the slot's logit, its softmax weight
// p and its value weight w = p * scale_v.
//
// V side: D[channel group][column] += sum over a tile's 16 slots of code * digit of w, with the V codes stored
// slot-minor (see kvq_common.cuh) as the row operand and the weights as the column operand: the owners put w
// on a 24-bit unsigned grid X = rint(w * 2^(24-E)) shared by all tiles of an epoch, the 32 X of the two tiles
// travel through shared memory, column n < 3 = digit n.  Four products per tile (one per byte plane of the
// 2-bit and 4-bit codes, one per channel group of the 8-bit codes) accumulate in four int32 accumulators per
// lane ACROSS tiles; they are turned into fp32 and added to the lane's four output channels only when the grid
// changes: the running maximum moves, a weight would exceed the grid, or about a thousand tiles have been added
// (int32 headroom).  Rounding w to the grid loses less than 2^-23 of the largest weight of the epoch per token,
// the same order as fp32 accumulation.  The V products of a pair run one iteration after its K side: they do
// not depend on the next pair's K side, and the weights have time to cross shared memory.
__device__ __forceinline__ void mma_k32_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_k16_u8u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm("mma.sync.aligned.m16n8k16.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ uint32_t byte_perm(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// The four balanced base-256 digits of T (|T| < 2^31 - 2^23), one per byte, in two's complement: adding 128 to
// each of the three low digits makes them unsigned without a borrow, so they are the bytes of the sum; flipping
// bit 7 of each takes the 128 off again.  The top byte is the top digit as it stands.
__device__ __forceinline__ uint32_t balanced_digits(int T) { return ((uint32_t)T + 0x00808080u) ^ 0x00808080u; }
// Selector that picks byte n of both source words of a prmt into the two low bytes of its result.
__device__ __forceinline__ uint32_t digit_selector(int n) { return (uint32_t)n | ((uint32_t)(4 + n) << 4); }
// Byte n (through sel = digit_selector(n)) of u0, u1, u2, u3 as bytes 0..3 of one word.
__device__ __forceinline__ uint32_t pick_bytes(uint32_t u0, uint32_t u1, uint32_t u2, uint32_t u3, uint32_t sel) {
    return byte_perm(byte_perm(u0, u1, sel), byte_perm(u2, u3, sel), 0x5410u);
}

constexpr float kGridLimit = 16777215.0f;          // weights on the grid stay below 2^24
constexpr int kFlushTiles = 1000;                  // int32 headroom: 16 slots * 255 * 255 per tile and accumulator

// The int32 accumulators of the V products and the grid they are on.
struct ValueAcc {
    int d[4][4];
    float fix;                     // 2^(24-E): w * fix is the weight on the grid; +inf = no grid chosen yet
    float ifix;                    // 2^(E-24)
};

// LAYOUT: 1 = one {scale, zero-point} pair per key row, kLayoutPerChannelK = one pair per channel and tile.
template <int CLS, int LAYOUT = 1>
struct FragRows {
    static constexpr int BITS = pool_bits(CLS), REC = pool_rec_bytes(CLS, LAYOUT);
    static constexpr int NW = 2 << CLS;            // 32-bit words per lane of one tensor's codes: 2, 4, 8
    static constexpr int PLANES = 8 / BITS;        // codes per byte: 4, 2, 1
    static constexpr uint32_t MASK = CLS == 0 ? 0x03030303u : CLS == 1 ? 0x0f0f0f0fu : 0xffffffffu;
    static constexpr float kDotScale = 1.0f / (float)(1 << (BITS * (PLANES - 1)));    // 1/64, 1/16, 1

    // Channel in byte j of operand register r (0: bytes 4q.., 1: bytes 16+4q..) of K product u, and its byte plane.
    __device__ static constexpr int k_plane(int u, int r) { return CLS == 0 ? 2 * u + r : CLS == 1 ? u : 0; }
    __device__ static constexpr int k_element(int u, int r, int q, int j) {
        return CLS == 0 ? 16 * q + 4 * j + (2 * u + r) : CLS == 1 ? 8 * (q + 4 * r) + 2 * j + u : 4 * (q + 8 * u + 4 * r) + j;
    }
    // Column operand of the K products: digit g & 3 of the fixed-point query (the same words serve tile A from
    // the lanes with g < 4 and tile B from the lanes with g >= 4; see the walk).
    __device__ static __forceinline__ void make_kb(const float* qrow, float fix_scale, int g, int q, uint32_t (&bk)[4]) {
        const uint32_t sel = digit_selector(g & 3);
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const float plane_scale = (float)(1 << (BITS * (PLANES - 1 - k_plane(u, r))));
                uint32_t dgt[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int e = k_element(u, r, q, j);
                    dgt[j] = balanced_digits(__float2int_rn(qrow[(e >> 5) * (kHalfDim + 4) + (e & 31)] * (fix_scale * plane_scale)));
                }
                bk[2 * u + r] = pick_bytes(dgt[0], dgt[1], dgt[2], dgt[3], sel);
            }
    }
    __device__ static __forceinline__ void load_words(const uint8_t* codes, int lane, uint32_t (&w)[NW]) {
        if (CLS == 0) {
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
    // The two K products of one tile, added to d.
    __device__ static __forceinline__ void k_products(int (&d)[4], const uint32_t (&kw)[NW], const uint32_t (&bk)[4]) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (CLS == 0)
                mma_k32_u8s8(d, kw[0] & (MASK << (4 * u)), kw[1] & (MASK << (4 * u)), kw[0] & (MASK << (4 * u + 2)),
                             kw[1] & (MASK << (4 * u + 2)), bk[2 * u], bk[2 * u + 1]);
            else if (CLS == 1)
                mma_k32_u8s8(d, kw[0] & (MASK << (4 * u)), kw[1] & (MASK << (4 * u)), kw[2] & (MASK << (4 * u)),
                             kw[3] & (MASK << (4 * u)), bk[2 * u], bk[2 * u + 1]);
            else
                mma_k32_u8s8(d, kw[4 * u], kw[4 * u + 1], kw[4 * u + 2], kw[4 * u + 3], bk[2 * u], bk[2 * u + 1]);
        }
    }
    // Weight of V product m in the lane's output channels (the planes stay where they are in the byte).
    __device__ static constexpr float plane_weight(int m) {
        return CLS == 0 ? 1.0f / (float)(1 << (2 * m)) : CLS == 1 ? ((m & 1) ? 1.0f / 16.0f : 1.0f) : 1.0f;
    }
    // Move the int32 accumulators into fp32 and clear them.  Lane (g, 0) holds digits 0, 1 of channel groups g
    // and g + 8, lane (g, 1) digit 2 (the other columns are zero): after one exchange per product lane (g, 0)
    // has the four channels 4 g .. 4 g + 3 and lane (g, 1) the channels 4 (g + 8) .. + 3, in st.of.
    template <class SM>
    __device__ static __forceinline__ void flush(ValueAcc& va, SM& st, int q) {
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const float c0 = (float)va.d[m][0], c1 = (float)va.d[m][1], c2 = (float)va.d[m][2], c3 = (float)va.d[m][3];
            const float send = q == 0 ? fmaf(c3, 256.0f, c2) : c0 * 65536.0f;
            const float mine = q == 0 ? fmaf(c1, 256.0f, c0) : c2 * 65536.0f;
            const float tot = mine + __shfl_xor_sync(0xffffffffu, send, 1);
            st.of[m] = fmaf(tot, va.ifix * plane_weight(m), st.of[m]);
            va.d[m][0] = va.d[m][1] = va.d[m][2] = va.d[m][3] = 0;
        }
    }
    // k_part: logits, softmax weights and value weights of a pair of tiles (recA, recB).  `valid`: the slot this
    // lane owns holds a token.  The value weights go to xbuf (32 words of shared memory: tile A's 16 slots, then
    // tile B's; two buffers alternate), the pair's V code words are returned for the v_part one iteration later.
    template <class SM>
    __device__ static __forceinline__ void k_part(const uint8_t* recA, const uint8_t* recB, bool valid, int lane, int g, int q,
                                                  const uint32_t (&bkA)[4], const uint32_t (&bkB)[4], const QueryInfo& qi,
                                                  SM& st, ValueAcc& va, uint32_t* xbuf, uint32_t (&vwA)[NW],
                                                  uint32_t (&vwB)[NW]) {
        uint32_t kwA[NW], kwB[NW];
        load_words(recA, lane, kwA);
        load_words(recB, lane, kwB);
        const int slot = g + 8 * (q & 1);
        const uint8_t* rec_own = q < 2 ? recA : recB;
        const float2 km = meta_to_float2(*reinterpret_cast<const uint32_t*>(rec_own + meta_offset(CLS, 0, slot)));
        const float2 vm = meta_to_float2(*reinterpret_cast<const uint32_t*>(rec_own + meta_offset(CLS, 1, slot)));
        load_words(recA + pool_codes_bytes(CLS), lane, vwA);
        load_words(recB + pool_codes_bytes(CLS), lane, vwB);

        int d[4] = {0, 0, 0, 0};
        k_products(d, kwA, bkA);
        k_products(d, kwB, bkB);
        // columns 2q, 2q+1 of slots g (d[0], d[1]) and g + 8 (d[2], d[3]): even q digits 0 and 1, odd q digits 2 and 3
        const float w0 = (q & 1) ? 65536.0f : 1.0f, w1 = (q & 1) ? 16777216.0f : 256.0f;
        const float lo = fmaf((float)d[1], w1, (float)d[0] * w0), hi = fmaf((float)d[3], w1, (float)d[2] * w0);
        const float dot = ((q & 1) ? hi : lo) + __shfl_xor_sync(0xffffffffu, (q & 1) ? lo : hi, 1);
        float y = fmaf(km.x * (qi.inv_fix * kDotScale), dot, km.y * qi.sumq);
        y = valid ? y : -INFINITY;

        finish_k_part(y, vm, q, slot, st, va, xbuf);
    }
    // The part of k_part that follows the logit: softmax weight, value weight on the grid, the rare grid changes.
    template <class SM>
    __device__ static __forceinline__ void finish_k_part(float y, float2 vm, int q, int slot, SM& st, ValueAcc& va, uint32_t* xbuf) {
        float e = fast_exp2(y - st.m);                 // the weight under the current maximum
        float x = (e * vm.x) * va.fix;                 // ... and its place on the current grid
        if (__builtin_expect(__any_sync(0xffffffffu, y > st.thr || !(x < kGridLimit)), 0)) {   // warp-uniform, rare
            flush(va, st, q);
            if (__any_sync(0xffffffffu, y > st.thr)) {
                const float tmax = warp_max(y);
                const float f = fast_exp2(st.m - tmax);
                st.m = tmax;
                st.thr = tmax + kRescaleSlack;
                st.l *= f;
                st.bsum *= f;
                if (SM::kStats) st.s2 *= f * f;
#pragma unroll
                for (int j = 0; j < 4; ++j) st.of[j] *= f;
                e = fast_exp2(y - st.m);
            }
            // a new grid: two bits of headroom above the largest weight of this pair of tiles
            const float wmax = warp_max(e * vm.x);
            uint32_t ew = __float_as_uint(wmax) >> 23;
            ew = ew < 30u ? 30u : ew;
            va.fix = wmax > 0.f ? __uint_as_float((275u - ew) << 23) : INFINITY;
            va.ifix = __uint_as_float((ew - 21u) << 23);
            x = (e * vm.x) * va.fix;
            x = x < kGridLimit ? x : 0.f;              // no grid yet (every weight of the pair is zero)
        }
        st.l += e;
        st.bsum = fmaf(e, vm.y, st.bsum);
        if (SM::kStats) st.s2 = fmaf(e, e, st.s2);
        xbuf[(q >> 1) * kTileTokens + slot] = __float2uint_rn(x);
    }
    // ---- per-channel keys.  khat_ti = c_ti s_i + z_i with one {s_i, z_i} per channel and TILE, so the scale moves to
    // the query's side: q . khat_t = sum_i (q_i s_i) c_ti + sum_i q_i z_i, and the column operand of a tile's K products
    // is the fixed-point form of q_i s_i, rebuilt for every tile (its own grid F: |q_i s_i F| < 2^22).  The lanes with
    // g < 4 do that for tile A, the others for tile B (each lane the 16 channels of its operand registers).
    // Position, among the lane's 16 channels, of the channel in byte j of operand register r of K product u; the
    // channels are runs of 16 / 8 / 4 consecutive ones starting at pc_run(q, idx / run length).
    __device__ static constexpr int pc_index(int u, int r, int j) {
        return CLS == 0 ? 4 * j + 2 * u + r : CLS == 1 ? 8 * r + 2 * j + u : 4 * (2 * u + r) + j;
    }
    __device__ static constexpr int pc_channel(int q, int idx) {
        return CLS == 0 ? 16 * q + idx : CLS == 1 ? 8 * q + 32 * (idx >> 3) + (idx & 7) : 4 * q + 16 * (idx >> 2) + (idx & 3);
    }
    __device__ static __forceinline__ void pc_load_query(const float* qrow, int q, float (&qe)[16]) {
#pragma unroll
        for (int idx = 0; idx < 16; ++idx) {
            const int e = pc_channel(q, idx);
            qe[idx] = qrow[(e >> 5) * (kHalfDim + 4) + (e & 31)];
        }
    }
    // res_a / res_b: the tile's keys are still fp16 rows in kres (the open window of the stream): their logits are
    // plain dot products, the tile's K products are ignored.
    template <class SM>
    __device__ static __forceinline__ void k_part_pc(const uint8_t* recA, const uint8_t* recB, bool valid, bool res_a, bool res_b,
                                                     const __half* kres, const float* qrow, int lane, int g, int q,
                                                     const float (&qe)[16], SM& st, ValueAcc& va, uint32_t* xbuf,
                                                     uint32_t (&vwA)[NW], uint32_t (&vwB)[NW]) {
        uint32_t kwA[NW], kwB[NW];
        load_words(recA, lane, kwA);
        load_words(recB, lane, kwB);
        const int slot = g + 8 * (q & 1);
        const uint8_t* rec_own = q < 2 ? recA : recB;
        const float2 vm = meta_to_float2(*reinterpret_cast<const uint32_t*>(rec_own + meta_offset(CLS, 1, slot, 0, LAYOUT)));
        load_words(recA + pool_codes_bytes(CLS), lane, vwA);
        load_words(recB + pool_codes_bytes(CLS), lane, vwB);

        // column operand of this lane's tile (A for g < 4, B otherwise)
        const uint8_t* rec_x = g < 4 ? recA : recB;
        float qs[16], zsum = 0.f, amax = 0.f;
        constexpr int RUN = CLS == 0 ? 16 : CLS == 1 ? 8 : 4;
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {               // four {scale, zero-point} words per 16-byte load
            const int e0 = pc_channel(q, 4 * v4);
            const uint4 m4 = *reinterpret_cast<const uint4*>(rec_x + chan_meta_offset(CLS, e0));
            const uint32_t m[4] = {m4.x, m4.y, m4.z, m4.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 sz = meta_to_float2(m[k]);
                qs[4 * v4 + k] = qe[4 * v4 + k] * sz.x;
                zsum = fmaf(qe[4 * v4 + k], sz.y, zsum);
                amax = fmaxf(amax, fabsf(qs[4 * v4 + k]));
            }
        }
        static_assert(RUN % 4 == 0, "a 16-byte load stays inside a run of consecutive channels");
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
        zsum += __shfl_xor_sync(0xffffffffu, zsum, 1);
        zsum += __shfl_xor_sync(0xffffffffu, zsum, 2);
        uint32_t ex = __float_as_uint(fmaxf(amax, 1.0e-30f)) >> 23;
        ex = ex > 254u ? 254u : ex;                    // (garbage of a tile whose keys are residual rows)
        const float fix = __uint_as_float((275u - ex) << 23), inv_fix = __uint_as_float((ex - 21u) << 23);
        uint32_t bk[4];
        const uint32_t sel = digit_selector(g & 3);
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const float plane_scale = (float)(1 << (BITS * (PLANES - 1 - k_plane(u, r))));
                uint32_t dgt[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    dgt[j] = balanced_digits(__float2int_rn(qs[pc_index(u, r, j)] * (fix * plane_scale)));
                bk[2 * u + r] = pick_bytes(dgt[0], dgt[1], dgt[2], dgt[3], sel);
            }
        uint32_t bkA[4], bkB[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            bkA[i] = g < 4 ? bk[i] : 0u;
            bkB[i] = g < 4 ? 0u : bk[i];
        }
        int d[4] = {0, 0, 0, 0};
        k_products(d, kwA, bkA);
        k_products(d, kwB, bkB);
        const float w0 = (q & 1) ? 65536.0f : 1.0f, w1 = (q & 1) ? 16777216.0f : 256.0f;
        const float lo = fmaf((float)d[1], w1, (float)d[0] * w0), hi = fmaf((float)d[3], w1, (float)d[2] * w0);
        const float dot = ((q & 1) ? hi : lo) + __shfl_xor_sync(0xffffffffu, (q & 1) ? lo : hi, 1);
        // the owner's tile: its grid and its zero-point term sit with the lanes that built its operand
        const int src = q < 2 ? 0 : 16;
        const float inv_own = __shfl_sync(0xffffffffu, inv_fix, src), z_own = __shfl_sync(0xffffffffu, zsum, src);
        float y = fmaf(inv_own * (kDotScale * kLogitScale), dot, z_own * kLogitScale);
        if (res_a || res_b) {                          // warp-uniform: at most once per pool and segment
            if (valid && (q < 2 ? res_a : res_b)) {
                const __half2* row = reinterpret_cast<const __half2*>(kres + slot * kHeadDim);
                float a = 0.f;
#pragma unroll 8
                for (int i = 0; i < kHeadDim / 2; ++i) {
                    const float2 k2 = __half22float2(row[i]);
                    const int e = 2 * i;
                    a = fmaf(k2.x, qrow[(e >> 5) * (kHalfDim + 4) + (e & 31)], a);
                    a = fmaf(k2.y, qrow[(e >> 5) * (kHalfDim + 4) + (e & 31) + 1], a);
                }
                y = a * kLogitScale;
            }
        }
        y = valid ? y : -INFINITY;
        finish_k_part(y, vm, q, slot, st, va, xbuf);
    }

    // The four V products of one tile with the weights xs of its slots 4q .. 4q+3.
    __device__ static __forceinline__ void v_products(ValueAcc& va, const uint32_t (&vw)[NW], const uint4 xs, uint32_t sel) {
        const uint32_t bv = byte_perm(byte_perm(xs.x, xs.y, sel), byte_perm(xs.z, xs.w, sel), 0x5410u);
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            if (CLS == 0)
                mma_k16_u8u8(va.d[m], vw[0] & (MASK << (2 * m)), vw[1] & (MASK << (2 * m)), bv);
            else if (CLS == 1)
                mma_k16_u8u8(va.d[m], vw[2 * (m >> 1)] & (MASK << (4 * (m & 1))), vw[2 * (m >> 1) + 1] & (MASK << (4 * (m & 1))), bv);
            else
                mma_k16_u8u8(va.d[m], vw[4 * (m >> 1) + 2 * (m & 1)], vw[4 * (m >> 1) + 2 * (m & 1) + 1], bv);
        }
    }
    // v_part: the V products of a pair whose weights were written to xbuf before the warp last synchronised.
    __device__ static __forceinline__ void v_part(const uint32_t (&vwA)[NW], const uint32_t (&vwB)[NW], const uint32_t* xbuf,
                                                  int q, uint32_t sel, ValueAcc& va) {
        v_products(va, vwA, *reinterpret_cast<const uint4*>(xbuf + 4 * q), sel);
        v_products(va, vwB, *reinterpret_cast<const uint4*>(xbuf + kTileTokens + 4 * q), sel);
    }
};

// ---------------------------------------------------------------- the split kernel

// Per-warp scratch in shared memory: the segment being worked on.
template <int STAGES>
struct alignas(16) WarpScratch {
    uint64_t bars[STAGES];
    const uint32_t* tab[kNumPools];    // block table of this (layer, sequence, KV head) in each pool
    int lo[kNumPools], hi[kNumPools];  // tile range of the segment in each pool
    uint32_t cnt[kNumPools];           // tokens in each pool
    uint32_t id[kNumPools];            // arena block that holds tile lo of each pool
    alignas(16) float q[kHeadDim + 4]; // query row; half 1 starts at q[36] so the two halves sit in different banks
    alignas(16) uint32_t x[2][2 * kTileTokens];    // (read 16 bytes at a time) fragment path: the value weights of a pair of tiles on the integer grid (two pairs alternate)
    alignas(16) float o[kHeadDim];     // the segment's output row (fragment path: gathered from the lanes that own channels;
                                       // CTA merge: this warp's partial)
    float2 ml;                         // CTA merge: this warp's (m, l)
    float s2;                          //            and its sum of squared weights
    uint32_t arrived;                  // CTA merge: partials delivered to the unit whose first warp this is
};
constexpr int kQHalfStride = kHalfDim + 4;

// Relative cost of a tile of each class to a warp of the short-cache geometry: a constant for the walk plus the
// tile's share of a stage refill (6 / 3 / 2 / 1 tiles of the four classes fit a stage); the best of four sets
// tried on the three short workloads, all within 4 % of one another.
#ifndef KVQ_TILE_COST_2BIT
#define KVQ_TILE_COST_2BIT 4u
#define KVQ_TILE_COST_4BIT 5u
#define KVQ_TILE_COST_8BIT 7u
#define KVQ_TILE_COST_FP16 12u
#endif
__device__ constexpr uint32_t kTileCost[kNumPools] = {KVQ_TILE_COST_2BIT, KVQ_TILE_COST_4BIT, KVQ_TILE_COST_8BIT, KVQ_TILE_COST_FP16};

// floor(n * a / g) for a <= g < 65536 in 32-bit arithmetic: n = q*g + r gives q*a + floor(r*a/g).
__device__ __forceinline__ uint32_t scale_by_fraction(uint32_t n, uint32_t a, uint32_t g) {
    const uint32_t q = n / g, r = n - q * g;
    return q * a + r * a / g;
}
// Chunks of a stream end where a stage is full (counted from the start of the arena block, tps tiles per stage),
// where the block ends, or where the segment's tiles of the pool end -- so a chunk is one contiguous run of bytes,
// and the copying and the reading side cut the same chunks.  A cursor carries the tiles left up to the next stage
// boundary and up to the end of the block.
struct ChunkCursor {
    int to_stage, to_block;
    __device__ __forceinline__ void start(int in_block_index, int tps, int bt) {
        to_stage = tps - in_block_index % tps;
        to_block = bt - in_block_index;
    }
    __device__ __forceinline__ int next(int left) const { return min(min(to_stage, to_block), left); }
    // true if the chunk of n tiles ended the block
    __device__ __forceinline__ bool advance(int n, int tps, int bt) {
        to_block -= n;
        to_stage = to_stage == n ? tps : to_stage - n;
        if (to_block != 0) return false;
        to_block = bt;
        to_stage = tps;
        return true;
    }
};

// Merge n_u partials (M = max m_j, l = sum l_j 2^(m_j - M), O = sum o_j 2^(m_j - M) / l) and write the fp16 row.
// ml(s), o(s) [this lane's float2 of partial s], s2(s) read partial s, from global records or from shared memory.
template <bool STATS, class LoadMl, class LoadO, class LoadS2>
__device__ __forceinline__ void merge_partials(const DecodeParams& P, uint32_t u, uint32_t row, size_t qo, uint32_t n_u, int lane,
                                               LoadMl ml_of, LoadO o_of, LoadS2 s2_of) {
    float M = kNegBig, L = 0.f, o0 = 0.f, o1 = 0.f;
    if (n_u <= 32) {                                   // the usual case: lane s weighs partial s; loads go out eight at a time
        const float2 ml = lane < n_u ? ml_of(lane) : make_float2(kNegBig, 0.f);
        float2 o[8];
#pragma unroll
        for (uint32_t k = 0; k < 8; ++k) o[k] = k < n_u ? o_of(k) : make_float2(0.f, 0.f);
        M = warp_max(ml.x);
        const float f = fast_exp2(ml.x - M);
        L = warp_sum(ml.y * f);
#pragma unroll
        for (uint32_t k = 0; k < 8; ++k) {
            const float fk = __shfl_sync(0xffffffffu, f, k);
            o0 = fmaf(o[k].x, fk, o0);
            o1 = fmaf(o[k].y, fk, o1);
        }
        for (uint32_t k0 = 8; k0 < n_u; k0 += 8) {
#pragma unroll
            for (uint32_t k = 0; k < 8; ++k) o[k] = k0 + k < n_u ? o_of(k0 + k) : make_float2(0.f, 0.f);
#pragma unroll
            for (uint32_t k = 0; k < 8; ++k) {
                const float fk = __shfl_sync(0xffffffffu, f, (k0 + k) & 31);
                o0 = fmaf(o[k].x, fk, o0);
                o1 = fmaf(o[k].y, fk, o1);
            }
        }
    } else {
        for (uint32_t s0 = 0; s0 < n_u; s0 += 32) {    // the maximum, 32 partials at a time
            const uint32_t s = s0 + lane;
            M = fmaxf(M, s < n_u ? ml_of(s).x : kNegBig);
        }
        M = warp_max(M);
        for (uint32_t s0 = 0; s0 < n_u; s0 += 32) {
            const uint32_t s = s0 + lane;
            const float2 ml = s < n_u ? ml_of(s) : make_float2(kNegBig, 0.f);
            const float f = fast_exp2(ml.x - M);
            L += warp_sum(ml.y * f);
            const uint32_t cnt = min(32u, n_u - s0);
            for (uint32_t k0 = 0; k0 < cnt; k0 += 8) {
                float2 o[8];
#pragma unroll
                for (uint32_t k = 0; k < 8; ++k) o[k] = k0 + k < cnt ? o_of(s0 + k0 + k) : make_float2(0.f, 0.f);
#pragma unroll
                for (uint32_t k = 0; k < 8; ++k) {
                    const float fk = __shfl_sync(0xffffffffu, f, (k0 + k) & 31);
                    o0 = fmaf(o[k].x, fk, o0);
                    o1 = fmaf(o[k].y, fk, o1);
                }
            }
        }
    }
    const float inv = L > 0.f ? 1.0f / L : 0.f;        // a sequence that holds no token yet gets zeros
    reinterpret_cast<__half2*>(P.O + qo)[lane] = __floats2half2_rn(o0 * inv, o1 * inv);
    if (STATS) {
        // weights a_t = p_t / L sum to one over the n cached tokens: Var = sum a_t^2 / n - 1 / n^2
        float S2 = 0.f;
        for (uint32_t s0 = 0; s0 < n_u; s0 += 32) {
            const uint32_t s = s0 + lane;
            if (s < n_u) {
                const float f = fast_exp2(ml_of(s).x - M);
                S2 = fmaf(s2_of(s), f * f, S2);
            }
        }
        S2 = warp_sum(S2);
        if (lane == 0) {
            const uint4 cnt = *reinterpret_cast<const uint4*>(P.counts + (size_t)row * 4);
            const float n = (float)(cnt.x + cnt.y + cnt.z + cnt.w);
            P.unit_var[u] = n > 0.f ? (S2 * inv * inv) / n - 1.0f / (n * n) : 0.f;
        }
    }
}

// grid = ceil(gw / Geo::kWarps), block = Geo::kThreads, dynamic smem = Geo::kSmemBytes.
// STATS: also emit, per unit, the variance of its attention weights over the cached tokens.
// P.cta_parts > 0: every unit is cut into that many parts (a divisor of Geo::kWarps), so all parts of a unit run in
// one CTA, which merges them through shared memory.
//
// STEP (not for per-channel keys): the launch is a whole decode step.  `P.counts` are the pool fills BEFORE the
// step's token, whose fp16 rows, features and controller come in A; other CTAs of the same launch store it (see
// k_decode_step) and nobody waits for them: the warp that works on the last part of a unit evaluates the controller
// itself and quantizes the token's K and V rows in registers the way the store does (row_values_as_stored) while its
// first copies travel, and adds the token to its partial at the end.  The slot the token is being written to lies beyond the fills this launch reads.
// STEP = 1: the controller has hidden width 32 and the warp evaluates it itself, early.  STEP = 2: any other width;
// the storing CTAs of the launch (which come first in the grid, so that they are resident before any attending
// CTA) evaluate it with 128 threads and publish the class; the attending warp picks it up at the END of its walk,
// by when it has long been written: a bounded wait that has never been seen to spin, with the usual flag if it
// should run out.
template <bool STATS, int G, class Geo, int STEP>
__device__ __forceinline__ void decode_attn_body(const DecodeParams& P, const AppendParams* A) {
    static_assert(!STEP || (G != kLayoutPerChannelK && !STATS), "the one-launch step exists for the plain decode with one pair per row or group");
    constexpr int kStages = Geo::kStages, kStageBytes = Geo::kStageBytes;
    extern __shared__ __align__(128) uint8_t ring[];   // [warps][stages][kStageBytes]
    __shared__ WarpScratch<kStages> scratch[Geo::kWarps];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int half = lane >> 4, t = lane & 15;
    const uint32_t j = (STEP == 2 ? blockIdx.x - P.cta0 : blockIdx.x) * Geo::kWarps + warp;
    if (Geo::kCtaMerge && P.cta_parts) {               // the arrival counters of this CTA's units start at zero:
        if (lane == 0) scratch[warp].arrived = 0u;     // the only barrier of the kernel, before any warp can wait
        __syncthreads();
    }
    if (j >= P.gw) return;                             // warps never wait for one another
    WarpScratch<kStages>& ws = scratch[warp];
    uint8_t* my_ring = ring + (size_t)warp * kStages * kStageBytes;
    if (lane == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&ws.bars[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    pdl_launch_dependents();                           // the next step's append may be scheduled behind this launch
    pdl_wait();                                        // the append before this launch has stored its token

    int pslot = 0, cslot = 0;                          // ring slot the next copy goes to / the next chunk is read from
    uint32_t par_bits = 0;                             // phase parity of every ring slot (bit s: slot s)
    bool failed = false;
    uint64_t x = (uint64_t)j * P.units;
    const uint64_t xend = x + P.units;

    while (x < xend) {
        // After an expired wait the warp starts no further copy and walks no further tile, but it still
        // delivers a (then empty) partial for every remaining segment of its share: the arrival counters of
        // those units reach their totals and go back to zero, so the handle stays usable after the flag.
        // ---- this segment: ticks [a0, a1) of unit u
        const uint32_t u = (x >> 32) ? (uint32_t)(x / P.gw) : (uint32_t)x / P.gw;
        const uint32_t a0 = (uint32_t)(x - (uint64_t)u * P.gw);
        const uint64_t room = xend - x;
        const uint32_t a1 = room < (uint64_t)(P.gw - a0) ? a0 + (uint32_t)room : P.gw;
        x += a1 - a0;
        const uint32_t row = u / (uint32_t)P.store.q_heads, qh = u - row * (uint32_t)P.store.q_heads;
        const uint32_t b = row / P.tq;                 // row = b * tq + (query row - t0)
        const size_t qo = (((size_t)b * P.t_total + P.t0 + (row - b * P.tq)) * P.store.q_heads + qh) * kHeadDim;
        const int kvh = (int)qh / P.group;
        const bool adds_token = STEP && a1 == P.gw;    // this warp works on the unit's last part
        __half2 k_new = __half2(), v_new = __half2();  // elements 2 lane, 2 lane + 1 of the step's token
        if constexpr (STEP) {
            if (adds_token) {
                const size_t src = ((size_t)b * P.store.kv_heads + kvh) * kHeadDim;
                k_new = reinterpret_cast<const __half2*>(A->K + src)[lane];
                v_new = reinterpret_cast<const __half2*>(A->V + src)[lane];
            }
        }
        if (lane < kNumPools) {                        // lane c plans pool c
            const int c = lane;
            const uint32_t* tab = stream_table(P.store, c, P.layer, (int)b, kvh);
            // The id of the stream's first block is requested together with the pool fill: a short cache starts in
            // it, and then the block table costs no memory round trip of its own.
            const uint32_t id_first = tab[0];
            const uint32_t n = P.counts[(size_t)row * 4 + c];
            const uint32_t nt = (n + kTileTokens - 1) / kTileTokens;
            ws.cnt[c] = n;
            int lo, hi;
            if constexpr (Geo::kPoolsEndToEnd) {
                // The four pools of the unit laid end to end and THAT axis cut into the warps' shares: a warp then
                // walks one pool, or two where its share crosses a border, instead of a sliver of each of the four
                // (every pool a warp enters costs it an operand set-up and a drained pipeline).
                // A tile counts with what it costs a warp here (kTileCost: its walk plus its part of a stage refill).
                const uint32_t cost = kTileCost[c];
                uint32_t before = 0, total = 0;
#pragma unroll
                for (int k = 0; k < kNumPools; ++k) {
                    const uint32_t wk = __shfl_sync(0xfu, nt * cost, k);
                    before += k < c ? wk : 0u;
                    total += wk;
                }
                const int r0 = (int)scale_by_fraction(total, a0, P.gw) - (int)before;
                const int r1 = (int)scale_by_fraction(total, a1, P.gw) - (int)before;
                lo = min(max(r0, 0) / (int)cost, (int)nt);       // the same rounding for a share's end and the next one's start
                hi = a1 == P.gw ? (int)nt : min(max(r1, 0) / (int)cost, (int)nt);
            } else if (P.gw < 65536u) {
                lo = (int)scale_by_fraction(nt, a0, P.gw);
                hi = (int)scale_by_fraction(nt, a1, P.gw);
            } else {
                lo = (int)((uint64_t)nt * a0 / P.gw);
                hi = (int)((uint64_t)nt * a1 / P.gw);
            }
            ws.lo[c] = lo;
            ws.hi[c] = hi;
            ws.tab[c] = tab;
            const uint32_t blk = (uint32_t)lo / block_tiles(c, G);
            ws.id[c] = (blk == 0 || lo >= hi) ? id_first : tab[blk];
        }
        {
            const float2 q2 = __half22float2(reinterpret_cast<const __half2*>(P.Q + qo)[lane]);
            const int i = 2 * lane;                    // elements i, i+1 (same half)
            float* dst = ws.q + (i >> 5) * kQHalfStride + (i & 31);
            dst[0] = q2.x;
            dst[1] = q2.y;
        }
        __syncwarp();
        QueryInfo qi;
        {
            const float qa = ws.q[lane], qb = ws.q[kQHalfStride + lane];
            if (G != 2) {
                qi.sumq = warp_sum(qa + qb) * kLogitScale;         // sum_i q_i, in logit units
            } else {                                   // the sum over this lane's half: 32 elements over its 16 lanes
                const float* qh_ = ws.q + half * kQHalfStride;
                qi.sumq = half_sum(qh_[t] + qh_[16 + t]) * kLogitScale;
            }
            // 256 R = 2^(22 - floor(log2 max|q|)), max|q| taken as at least the smallest normal fp16
            const float qmax = fmaxf(warp_max(fmaxf(fabsf(qa), fabsf(qb))), 6.103515625e-05f);
            const uint32_t e = __float_as_uint(qmax) >> 23;        // biased exponent, 113..142
            // (the fragment path keeps one bit less: |q F| < 2^22, see FragRows)
            qi.fix_scale = __uint_as_float(((G != 2 ? 275u : 276u) - e) << 23);
            qi.inv_fix = __uint_as_float((e - (G != 2 ? 21u : 22u)) << 23) * kLogitScale;
            qi.q_half = ws.q + half * kQHalfStride;
        }

        // ---- producer cursor (warp-uniform; lane 0 issues): next tile to fetch, tiles left in its pool.
        // A chunk never crosses a 64 KB block of the arena (see chunk_tiles); the id of the block after the current
        // one is fetched from the stream's table a whole block ahead of its first use.
        int p_c = -1, p_left = 0, p_tps = 0, p_bt = 0;
        ChunkCursor p_cur = {0, 0};
        uint32_t p_rec = 0, p_next_id = 0;
        const uint8_t* p_ptr = nullptr;
        const uint32_t* p_tab = nullptr;               // entry of the block after the current one
        auto next_pool = [&]() {                       // move to the next pool that has tiles in this segment
            while (p_left == 0 && ++p_c < kNumPools) {
                const int lo = ws.lo[p_c];
                p_left = ws.hi[p_c] - lo;
                if (p_left == 0) continue;
                p_tps = p_c == 0 ? Geo::tps(0, G) : p_c == 1 ? Geo::tps(1, G) : p_c == 2 ? Geo::tps(2, G) : Geo::tps(3, G);
                p_rec = (uint32_t)pool_rec_bytes(p_c, G);
                p_bt = (int)block_tiles(p_c, G);
                const int blk = lo / p_bt, ib = lo - blk * p_bt;
                p_cur.start(ib, p_tps, p_bt);
                p_tab = ws.tab[p_c] + blk + 1;
                p_ptr = P.store.arena + (size_t)ws.id[p_c] * kBlockBytes + (size_t)ib * p_rec;
                // (only a segment that goes on into the stream's next block asks for its id: a request that nobody
                // waits for would still hold up the next request for the same register)
                if (p_left > p_cur.to_block) p_next_id = p_tab[0];
            }
        };
        if (!failed) next_pool();
        auto issue_next = [&]() {
            const int n = p_cur.next(p_left);
            const uint32_t bytes = (uint32_t)n * p_rec;
            if (lane == 0) {
                mbar_arrive_expect_tx(&ws.bars[pslot], bytes);
                bulk_load(my_ring + (size_t)pslot * kStageBytes, p_ptr, bytes, &ws.bars[pslot]);
            }
            if (++pslot == kStages) pslot = 0;
            p_ptr += bytes;
            p_left -= n;
            const bool block_end = p_cur.advance(n, p_tps, p_bt);
            if (p_left == 0) {
                next_pool();
            } else if (block_end) {                    // on to the stream's next block
                p_ptr = P.store.arena + (size_t)p_next_id * kBlockBytes;
                ++p_tab;
                if (p_left > p_bt) p_next_id = p_tab[0];
            }
        };
        int in_flight = 0;
        for (; in_flight < kStages && p_left > 0; ++in_flight) issue_next();

        // The step's token, worked out while the first copies travel: its logit and its two value elements as stored.
        float y_new = 0.f;
        float2 v_tok = make_float2(0.f, 0.f);
        if constexpr (STEP == 1) {
            if (adds_token) {                          // warp-uniform
                const float4 f = reinterpret_cast<const float4*>(A->feats)[b];
                const int c = controller_decide_warp32(A->ctrl, f.x, f.y, f.z, f.w, lane);
                const float2 kh = row_values_as_stored<G>(__half22float2(k_new), c);
                v_tok = row_values_as_stored<G>(__half22float2(v_new), c);
                const int i = 2 * lane;
                const float* qp = ws.q + (i >> 5) * kQHalfStride + (i & 31);
                y_new = warp_sum(fmaf(kh.y, qp[1], kh.x * qp[0])) * kLogitScale;
            }
        }

        SoftmaxT<STATS> st = {kNegBig, 0.f, 0.f, kNegBig, 0.f, {0.f, 0.f, 0.f, 0.f}};
        float acc[kHalfDim];
#pragma unroll
        for (int i = 0; i < kHalfDim; ++i) acc[i] = 0.f;

        // The reading side of the ring: wait for the chunk in slot cslot / hand the slot back and start the next copy.
        auto chunk_wait = [&]() {
            if (!mbar_wait(&ws.bars[cslot], (par_bits >> cslot) & 1u)) failed = true;
            return !failed;
        };
        auto chunk_done = [&]() {
            --in_flight;
            __syncwarp();                              // every lane is done with the slot before it is refilled
            if (p_left > 0) {
                issue_next();
                ++in_flight;
            }
            par_bits ^= 1u << cslot;
            if (++cslot == kStages) cslot = 0;
        };

        auto walk = [&](auto cls_tag, auto consumer) {
            constexpr int CLS = decltype(cls_tag)::value;
            using C = decltype(consumer);
            constexpr int TPS = Geo::tps(CLS, G), BT = (int)block_tiles(CLS, G);
            int tile0 = ws.lo[CLS];
            const int hi = ws.hi[CLS];
            if (tile0 >= hi || failed) return;
            const uint32_t cnt = ws.cnt[CLS];
            ChunkCursor cur;
            cur.start(tile0 % BT, TPS, BT);
            uint32_t qreg[kQRegs];
            C::enter(qi, qreg, acc);
            while (tile0 < hi) {
                if (!chunk_wait()) break;
                const int ntiles = cur.next(hi - tile0);
                cur.advance(ntiles, TPS, BT);
                const uint8_t* buf = my_ring + (size_t)cslot * kStageBytes;
                typename C::KIn kin = C::load_k(buf, half, t);
                for (int i = 0; i < ntiles; ++i) {
                    const bool valid = (uint32_t)((tile0 + i) * kTileTokens + t) < cnt;
                    // the next tile's K side (the last tile fetches itself again)
                    const typename C::KIn knext = C::load_k(buf + (size_t)min(i + 1, ntiles - 1) * C::REC, half, t);
                    C::tile(buf + (size_t)i * C::REC, kin, valid, half, t, qreg, qi, st, acc);
                    kin = knext;
                }
                tile0 += ntiles;
                chunk_done();
            }
            C::leave(acc);
        };
        // The same walk for the fragment path, two tiles (A, B) per iteration: lane L = 4 g + q owns slot
        // g + 8 (q & 1) of tile A (q < 2) or of tile B (q >= 2).  A chunk with an odd number of tiles ends with
        // a pair whose B is absent: it points at A's record again and every one of its slots counts as empty.
        auto walk_frag = [&](auto cls_tag) {
            constexpr int CLS = decltype(cls_tag)::value;
            constexpr bool PC = G == kLayoutPerChannelK;
            using C = FragRows<CLS, PC ? kLayoutPerChannelK : 1>;
            constexpr int TPS = Geo::tps(CLS, G), BT = (int)block_tiles(CLS, G);
            int tile0 = ws.lo[CLS];
            const int hi = ws.hi[CLS];
            if (tile0 >= hi || failed) return;
            const uint32_t cnt = ws.cnt[CLS];
            const int g = lane >> 2, q = lane & 3;
            const uint32_t my_slot = (uint32_t)((q >> 1) * kTileTokens + g + 8 * (q & 1));     // 0..15 in A, 16..31 in B
            const uint32_t dg = g < 3 ? (uint32_t)g : 3u;                            // byte 3 of a weight on the grid is zero
            const uint32_t sel = dg | ((4u + dg) << 4) | (dg << 8) | ((4u + dg) << 12);
            ChunkCursor cur;
            cur.start(tile0 % BT, TPS, BT);
            uint32_t bkA[4], bkB[4];
            float qe[PC ? 16 : 1];                     // per-channel keys: the query channels of this lane's operand registers
            if constexpr (PC) {
                C::pc_load_query(ws.q, q, qe);
            } else {
                C::make_kb(ws.q, qi.fix_scale, g, q, bkA);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    bkB[i] = g >= 4 ? bkA[i] : 0u;
                    bkA[i] = g < 4 ? bkA[i] : 0u;
                }
            }
            // per-channel keys: the tile whose keys still wait as fp16 rows (the stream's open window), if any
            const int res_tile = PC && (cnt & (kTileTokens - 1)) ? (int)(cnt / kTileTokens) : -1;
            const __half* kres = PC ? residual_rows(P.store, CLS, P.layer, (int)b, kvh) : nullptr;
            ValueAcc va;
#pragma unroll
            for (int m = 0; m < 4; ++m) va.d[m][0] = va.d[m][1] = va.d[m][2] = va.d[m][3] = 0;
            va.fix = INFINITY;
            va.ifix = 0.f;
            int since_flush = 0;
            // The V products of a pair run one iteration late: before the first pair there is a pair of zero
            // weights, after the last one the pending products are drained.
            uint32_t vpA[C::NW], vpB[C::NW];
#pragma unroll
            for (int i = 0; i < C::NW; ++i) vpA[i] = vpB[i] = 0u;
            uint32_t pp = 0;                           // buffer the current pair writes its weights to
            ws.x[1][lane] = 0u;
            __syncwarp();
            while (tile0 < hi) {
                if (!chunk_wait()) break;
                const int ntiles = cur.next(hi - tile0);
                cur.advance(ntiles, TPS, BT);
                const uint8_t* buf = my_ring + (size_t)cslot * kStageBytes;
                for (int i = 0; i < ntiles; i += 2) {
                    const bool has_b = i + 1 < ntiles;
                    const uint8_t* recA = buf + (size_t)i * C::REC;
                    const uint8_t* recB = has_b ? recA + C::REC : recA;
                    const bool valid = (uint32_t)((tile0 + i) * kTileTokens) + my_slot < cnt && (q < 2 || has_b);
                    uint32_t vwA[C::NW], vwB[C::NW];
                    C::v_part(vpA, vpB, ws.x[pp ^ 1u], q, sel, va);
                    if constexpr (PC)
                        C::k_part_pc(recA, recB, valid, tile0 + i == res_tile, has_b && tile0 + i + 1 == res_tile, kres, ws.q, lane, g,
                                     q, qe, st, va, ws.x[pp], vwA, vwB);
                    else
                        C::k_part(recA, recB, valid, lane, g, q, bkA, bkB, qi, st, va, ws.x[pp], vwA, vwB);
                    __syncwarp();                      // the pair's weights are in shared memory
                    pp ^= 1u;
#pragma unroll
                    for (int k = 0; k < C::NW; ++k) {
                        vpA[k] = vwA[k];
                        vpB[k] = vwB[k];
                    }
                }
                tile0 += ntiles;
                since_flush += ntiles;
                if (since_flush >= kFlushTiles) {
                    C::flush(va, st, q);
                    since_flush = 0;
                }
                chunk_done();
            }
            C::v_part(vpA, vpB, ws.x[pp ^ 1u], q, sel, va);     // the last pair's products
            C::flush(va, st, q);
        };
        if constexpr (G != 2) {
            walk_frag(std::integral_constant<int, 0>{});
            walk_frag(std::integral_constant<int, 1>{});
            walk_frag(std::integral_constant<int, 2>{});
            walk(std::integral_constant<int, 3>{}, Fp16Rows<false>{});
        } else {
            walk(std::integral_constant<int, 0>{}, Quantized<0, G>{});
            walk(std::integral_constant<int, 1>{}, Quantized<1, G>{});
            walk(std::integral_constant<int, 2>{}, Quantized<2, G>{});
            walk(std::integral_constant<int, 3>{}, Fp16Rows<true>{});
        }

        if (failed && in_flight > 0) {
            // Copies that were started but not consumed may still land in this warp's ring: give
            // each a bounded wait before the warp can retire, then report.
            for (int i = 1; i < in_flight; ++i) {
                par_bits ^= 1u << cslot;
                if (++cslot == kStages) cslot = 0;
                mbar_wait(&ws.bars[cslot], (par_bits >> cslot) & 1u);
            }
            in_flight = 0;
            if (lane == 0) atomicOr(P.store.flags, kFlagWaitTimeout);
        }

        // ---- reduce the per-lane partial sums over the 16 slots of a half: after four halving
        //      steps lane L holds elements 2L, 2L+1 of the row
        float r16[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const bool up = lane & 8;
            const float keep = up ? acc[k + 16] : acc[k], send = up ? acc[k] : acc[k + 16];
            r16[k] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
        float r8[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const bool up = lane & 4;
            const float keep = up ? r16[k + 8] : r16[k], send = up ? r16[k] : r16[k + 8];
            r8[k] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
        }
        float r4[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool up = lane & 2;
            const float keep = up ? r8[k + 4] : r8[k], send = up ? r8[k] : r8[k + 4];
            r4[k] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
        }
        float r2[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const bool up = lane & 1;
            const float keep = up ? r4[k + 2] : r4[k], send = up ? r4[k] : r4[k + 2];
            r2[k] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
        }
        // Two scale groups: both lanes of a token added its p and p * zero-point, so the warp sums are halved
        // (each half has its own zero-points: that sum stays inside the half).  One scale group: every token was
        // counted by exactly one lane; the quantized pools' part of the row sits with the lanes that own channels
        // and is gathered through shared memory.
        const float l_w = (G != 2 ? 1.0f : 0.5f) * warp_sum(st.l);
        const float b_w = G != 2 ? warp_sum(st.bsum) : half_sum(st.bsum);
        if (G != 2) {
            if ((lane & 3) < 2)
                *reinterpret_cast<float4*>(ws.o + 4 * ((lane >> 2) + 8 * (lane & 3))) =
                    make_float4(st.of[0] + b_w, st.of[1] + b_w, st.of[2] + b_w, st.of[3] + b_w);
            __syncwarp();
            const float2 o2 = *reinterpret_cast<const float2*>(ws.o + 2 * lane);
            r2[0] += o2.x;
            r2[1] += o2.y;
            __syncwarp();                              // ws.o is written again below or in the warp's next segment
        } else {
            r2[0] += b_w;
            r2[1] += b_w;
        }
        const float s2_w = STATS ? (G != 2 ? 1.0f : 0.5f) * warp_sum(st.s2) : 0.f;
        float l_tot = l_w;
        if constexpr (STEP == 2) {
            if (adds_token) {                          // warp-uniform: the class comes from a storing CTA of this launch
                uint32_t word = 0;
                if (lane == 0) {
                    bool found = false;
                    for (uint32_t spin = 0; spin < kWaitLimit && !found; ++spin) {
                        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(word) : "l"(P.step_cls + b) : "memory");
                        found = (word >> 2) == P.step_serial;
                        if (!found) __nanosleep(64);
                    }
                    if (!found) {
                        atomicOr(P.store.flags, kFlagWaitTimeout);
                        word = 3u;                     // keep the row as it is; the call's output is flagged invalid
                    }
                }
                const int c = (int)(__shfl_sync(0xffffffffu, word, 0) & 3u);
                const float2 kh = row_values_as_stored<G>(__half22float2(k_new), c);
                v_tok = row_values_as_stored<G>(__half22float2(v_new), c);
                const int i = 2 * lane;
                const float* qp = ws.q + (i >> 5) * kQHalfStride + (i & 31);
                y_new = warp_sum(fmaf(kh.y, qp[1], kh.x * qp[0])) * kLogitScale;
            }
        }
        if constexpr (STEP != 0) {
            if (adds_token) {                          // warp-uniform: one more online-softmax update
                const float m_new = fmaxf(st.m, y_new);
                const float keep = fast_exp2(st.m - m_new), e = fast_exp2(y_new - m_new);
                r2[0] = fmaf(r2[0], keep, e * v_tok.x);
                r2[1] = fmaf(r2[1], keep, e * v_tok.y);
                l_tot = fmaf(l_w, keep, e);
                st.m = m_new;
            }
        }

        if (Geo::kCtaMerge && P.cta_parts) {
            // ---- all parts of the unit run in this CTA: partials and the arrival counter stay in shared memory
            const uint32_t parts = P.cta_parts;
            const int wf = warp - (int)(j % parts);    // the unit's first warp in this CTA holds its counter
            reinterpret_cast<float2*>(ws.o)[lane] = make_float2(r2[0], r2[1]);
            if (lane == 0) {
                ws.ml = make_float2(st.m, l_tot);
                ws.s2 = s2_w;
            }
            __syncwarp();
            uint32_t seen = 0;
            if (lane == 0) {
                __threadfence_block();                 // this warp's partial is visible to the CTA before it is counted
                seen = atomicAdd(&scratch[wf].arrived, 1u);
            }
            seen = __shfl_sync(0xffffffffu, seen, 0);
            if (seen + 1 == parts) {
                __threadfence_block();
                merge_partials<STATS>(
                    P, u, row, qo, parts, lane,
                    [&](uint32_t s) {
                        const volatile float* pm = reinterpret_cast<const volatile float*>(&scratch[wf + s].ml);
                        return make_float2(pm[0], pm[1]);
                    },
                    [&](uint32_t s) {
                        const volatile float* po = scratch[wf + s].o + 2 * lane;
                        return make_float2(po[0], po[1]);
                    },
                    [&](uint32_t s) { return *const_cast<const volatile float*>(&scratch[wf + s].s2); });
            }
            continue;                                  // (one segment per warp in this mode)
        }
        const uint32_t jf = decode_first_warp(u, P.units, P.gw);
        const size_t rec0 = (size_t)u * P.pslots;
        reinterpret_cast<float2*>(P.part_o + (rec0 + (j - jf)) * kHeadDim)[lane] = make_float2(r2[0], r2[1]);
        if (lane == 0) P.part_ml[rec0 + (j - jf)] = make_float2(st.m, l_tot);
        if (STATS) {
            if (lane == 0) P.part_s2[rec0 + (j - jf)] = s2_w;
        }

        // ---- the warp that delivers the last partial of the unit merges them
        const uint32_t n_u = decode_warps_of_unit(u, P.units, P.gw);
        __threadfence();                               // this warp's partial is visible device-wide ...
        __syncwarp();
        uint32_t seen = 0;
        if (lane == 0) seen = atomicAdd(P.part_cnt + u, 1u);       // ... before it is counted
        seen = __shfl_sync(0xffffffffu, seen, 0);
        if (seen + 1 == n_u) {
            __threadfence();                           // the other warps' partials, counted before ours
            merge_partials<STATS>(
                P, u, row, qo, n_u, lane, [&](uint32_t s) { return __ldcg(&P.part_ml[rec0 + s]); },
                [&](uint32_t s) { return __ldcg(reinterpret_cast<const float2*>(P.part_o + (rec0 + s) * kHeadDim) + lane); },
                [&](uint32_t s) { return __ldcg(&P.part_s2[rec0 + s]); });
            if (lane == 0) P.part_cnt[u] = 0;
        }
    }
}

template <bool STATS, int G, class Geo>
__global__ void __launch_bounds__(Geo::kThreads, Geo::kCtasPerSm)
k_decode_attn(DecodeParams P) {
    decode_attn_body<STATS, G, Geo, 0>(P, nullptr);
}

// One decode step (Eq. 4, then Eq. 5) in one launch: the first ceil(gw / Geo::kWarps) CTAs attend over the cache
// as it was plus the step's token (decode_attn_body with STEP), the others store the token: every warp of theirs
// is one warp of k_append_token.  Neither side reads what the other writes.
// grid = ceil(gw / Geo::kWarps) + ceil(batch * ceil(kv_heads / 16) / Geo::kWarps).
// WIDE (a controller of another hidden width than 32): the storing CTAs come FIRST in the grid, one per (sequence,
// group of 16 KV heads); their first 128 threads evaluate the controller together and publish the class for the
// attending warps (see decode_attn_body).  grid = batch * ceil(kv_heads / 16) + ceil(gw / Geo::kWarps).
template <class Geo, int G, bool WIDE>
__global__ void __launch_bounds__(Geo::kThreads, Geo::kCtasPerSm)
k_decode_step(DecodeParams P, AppendParams A) {
    static_assert(sizeof(float) * kControllerDirectSmemFloats <= Geo::kSmemBytes, "the storing CTAs' controller scratch lies in the ring");
    const int head_groups = (A.store.kv_heads + 15) / 16;
    if constexpr (WIDE) {
        if (blockIdx.x >= P.cta0) {
            decode_attn_body<false, G, Geo, 2>(P, &A);
            return;
        }
        extern __shared__ __align__(128) uint8_t ring[];       // the storing CTAs use its start for the controller
        pdl_launch_dependents();
        pdl_wait();                                    // the attention of the previous step still reads the store
        if (threadIdx.x < 128)
            append_token_warp<true, G>(A, (int)blockIdx.x % head_groups, (int)blockIdx.x / head_groups, kCtlCtaDirect,
                                       reinterpret_cast<float*>(ring));
    } else {
        const uint32_t attn_ctas = (P.gw + Geo::kWarps - 1) / Geo::kWarps;
        if (blockIdx.x < attn_ctas) {
            decode_attn_body<false, G, Geo, 1>(P, &A);
            return;
        }
        pdl_launch_dependents();
        pdl_wait();                                    // the attention of the previous step still reads the store
        const int item = (int)(blockIdx.x - attn_ctas) * Geo::kWarps + (int)(threadIdx.x >> 5);
        if (item < head_groups * A.store.batch) append_token_warp<true, G>(A, item % head_groups, item / head_groups, kCtlWarp32, nullptr);
    }
}

// Pool fills each of the last t_total cached tokens may see when it asks as a query (causal
// attention over the mixed cache).  Slots of a pool are handed out in position order, so query row i
// (position len - t_total + i) sees every slot of pool c except those of the later rows of that class:
// vis[b][i - t0][c] = fill[b][c] - #{ j > i : class(position of row j) == c }, for rows t0 .. t0+tq.
// grid = batch, block = tq threads.
// lens: cached tokens per sequence (nullptr: `len` for all).
__global__ void k_visible_counts(StoreView s, const uint32_t* __restrict__ fill, int layer, int len,
                                 const int* __restrict__ lens, uint32_t t_total, uint32_t t0, uint32_t tq,
                                 uint32_t* __restrict__ vis) {
    const uint32_t b = blockIdx.x, il = threadIdx.x;
    if (il >= tq) return;
    if (lens) len = lens[b];
    const uint32_t i = t0 + il;
    uint32_t l0 = 0, l1 = 0, l2 = 0, l3 = 0;
    const uint32_t* idx = s.index + ((size_t)layer * s.batch + b) * s.max_ctx + (len - (int)t_total);
    for (uint32_t j = i + 1; j < t_total; ++j) {
        const uint32_t c = idx[j] >> 30;
        l0 += c == 0; l1 += c == 1; l2 += c == 2; l3 += c == 3;
    }
    const uint4 f = *reinterpret_cast<const uint4*>(fill + (size_t)b * 4);
    *reinterpret_cast<uint4*>(vis + ((size_t)b * tq + il) * 4) = make_uint4(f.x - l0, f.y - l1, f.z - l2, f.w - l3);
}

// Eq. 16: V = (1/h) sum over the query heads of the variance of the head's attention weights.
// unit_var [batch][q_heads] -> var_out [batch].  grid = batch, block = 32.
__global__ void k_head_mean(const float* __restrict__ unit_var, int q_heads, float* __restrict__ var_out) {
    float s = 0.f;
    for (int h = threadIdx.x; h < q_heads; h += 32) s += unit_var[(size_t)blockIdx.x * q_heads + h];
    s = warp_sum(s);
    if (threadIdx.x == 0) var_out[blockIdx.x] = s / (float)q_heads;
}

}  // namespace kvq
