// Token-level saliency features (Section 3.2): the controller's input vector of Eq. 17,
//   s_t = [H_t, R_t, V_t, C_t],
// computed on the device from what a forward pass leaves behind:
//   H_t  entropy of the next-token distribution, -sum_v p log p with p = Softmax(z_t)        (Eq. 14)
//   R_t  rarity, -log((c(x_t) + 1) / (N + |V_obs| + 1)) from running token counts             (Eq. 15)
//   V_t  attention variance of the last layer, passed in (k_decode_attn<true> produces it)    (Eq. 16)
//   C_t  confidence; the paper names it without defining it: taken as max_v p_t(v)
//
// One CTA per token streams the token's logits once (16-byte loads), every thread keeping an online
// triple (m, s, w) = (running maximum, sum e^(z-m), sum (z-m) e^(z-m)); triples merge exactly:
// for a new maximum m' the old sums become s r and (w + (m - m') s) r with r = e^(m - m').
// Then H = log s - w / s and C = 1 / s.  The kernel is bound by HBM: |V| logits per token.
#pragma once
#include "kvq_common.cuh"
#include <type_traits>

namespace kvq {

constexpr int kFeatureThreads = 256;       // many tokens: several CTAs per SM
constexpr int kFeatureThreadsFew = 1024;   // a decode step's handful of tokens: more loads in flight per row
#ifndef KVQ_FEATURE_LOADS
#define KVQ_FEATURE_LOADS 2
#endif
constexpr int kFeatureLoads = KVQ_FEATURE_LOADS;   // vector loads a thread has in flight

struct OnlineEntropy {
    float m, s, w;
    __device__ __forceinline__ void raise_to(float m2) {       // m2 >= m
        if (s > 0.f) {                                         // (an empty triple has m = -inf)
            const float r = __expf(m - m2);
            w = (w + (m - m2) * s) * r;
            s *= r;
        }
        m = m2;
    }
    // A term whose weight underflows to zero (a masked logit, z = -inf, in particular) adds nothing:
    // p log p -> 0 as p -> 0 (Eq. 14), whereas d * e would be -inf * 0.
    __device__ __forceinline__ void add(float z) {             // z <= m
        const float d = z - m, e = __expf(d);
        if (e > 0.f) {
            s += e;
            w = fmaf(d, e, w);
        }
    }
    __device__ __forceinline__ void merge(const OnlineEntropy& o) {
        if (o.m > m) {
            OnlineEntropy t = o;
            if (s > 0.f) {                                     // fold this into the other's frame
                const float r = __expf(m - o.m);
                t.w += (w + (m - o.m) * s) * r;
                t.s += s * r;
            }
            *this = t;
        } else if (o.s > 0.f) {
            const float r = __expf(o.m - m);
            w += (o.w + (o.m - m) * o.s) * r;
            s += o.s * r;
        }
    }
};

// Two OnlineEntropy sums side by side under one running maximum m, for the vector path: the four fp32 operations
// per element run as packed two-lane instructions (sub, mul, add, fma .f32x2: same results as the scalar ones),
// which halves the issue slots they take; the exponentials stay one per element.  Elements must be finite or
// clamped (see clamp_masked): a weight of zero then adds 0 * (finite) = 0.
struct OnlineEntropyPair {
    float m, s0, s1, w0, w1;
    __device__ __forceinline__ void raise_to(float m2) {       // m2 >= m
        const float dm = m - m2, r = __expf(dm);
        w0 = fmaf(dm, s0, w0) * r;
        w1 = fmaf(dm, s1, w1) * r;
        s0 *= r;
        s1 *= r;
        m = m2;
    }
    __device__ __forceinline__ void add2(float z0, float z1) {  // z0, z1 <= m
        float d0, d1;
        asm("{ .reg .b64 z, mm, d;\n mov.b64 z, {%2, %3};\n mov.b64 mm, {%4, %4};\n"
            " sub.rn.f32x2 d, z, mm;\n mov.b64 {%0, %1}, d; }"
            : "=f"(d0), "=f"(d1)
            : "f"(z0), "f"(z1), "f"(m));
        add_differences(d0, d1);
    }
    // The same for two fp16 logits: the mixed-precision subtract widens and subtracts in one instruction
    // (fl(float(z) - m), what the conversion followed by an fp32 subtract gives).
    __device__ __forceinline__ void add2(__half2 z) {          // both halves <= m
        float d0, d1;
        asm("{ .reg .b16 lo, hi;\n mov.b32 {lo, hi}, %2;\n sub.rn.f32.f16 %0, lo, %3;\n sub.rn.f32.f16 %1, hi, %3; }"
            : "=f"(d0), "=f"(d1)
            : "r"(*reinterpret_cast<const uint32_t*>(&z)), "f"(m));
        add_differences(d0, d1);
    }
    __device__ __forceinline__ void add_differences(float d0, float d1) {     // d = z - m <= 0
        float t0, t1;
        asm("{ .reg .b64 d, l, t;\n mov.b64 d, {%2, %3};\n mov.b64 l, {%4, %4};\n"
            " mul.rn.f32x2 t, d, l;\n mov.b64 {%0, %1}, t; }"
            : "=f"(t0), "=f"(t1)
            : "f"(d0), "f"(d1), "f"(1.4426950408889634f));
        float e0, e1;
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(t0));
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(t1));
        asm("{ .reg .b64 s, e, d, w;\n mov.b64 s, {%0, %1};\n mov.b64 w, {%2, %3};\n mov.b64 e, {%4, %5};\n mov.b64 d, {%6, %7};\n"
            " add.rn.f32x2 s, s, e;\n fma.rn.f32x2 w, d, e, w;\n mov.b64 {%0, %1}, s;\n mov.b64 {%2, %3}, w; }"
            : "+f"(s0), "+f"(s1), "+f"(w0), "+f"(w1)
            : "f"(e0), "f"(e1), "f"(d0), "f"(d1));
    }
};

// Masked logits (-inf) are taken down to a large finite value before the sums: their weight e^(z - m) is still
// exactly zero, and (z - m) e stays 0 instead of -inf * 0.  fp16 rows: the most negative fp16; fp32 rows: -1e28
// (times any number of terms it stays finite).
constexpr float kMaskedFloor = -1.0e28f;

// Eight consecutive logits of a row, clamped from below (see kMaskedFloor).
template <typename T>
struct Chunk8;
template <>
struct Chunk8<__half> {
    __half2 h[4];
    __device__ __forceinline__ void load(const __half* p) {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const __half2* q = reinterpret_cast<const __half2*>(&v);
        const __half2 floor2 = __float2half2_rn(-65504.0f);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __hmax2(q[i], floor2);
    }
};
template <>
struct Chunk8<float> {
    float z[8];
    __device__ __forceinline__ void load(const float* p) {
        const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
        z[0] = fmaxf(a.x, kMaskedFloor); z[1] = fmaxf(a.y, kMaskedFloor); z[2] = fmaxf(a.z, kMaskedFloor); z[3] = fmaxf(a.w, kMaskedFloor);
        z[4] = fmaxf(b.x, kMaskedFloor); z[5] = fmaxf(b.y, kMaskedFloor); z[6] = fmaxf(b.z, kMaskedFloor); z[7] = fmaxf(b.w, kMaskedFloor);
    }
};

// grid = n tokens, block = kFeatureThreads or kFeatureThreadsFew.  logits [n][vocab] of T; vocab % 8 == 0 and a 32-byte
// aligned base are needed for the vector path (`vec`), otherwise elements are read one by one.
template <typename T>
__global__ void __launch_bounds__(kFeatureThreadsFew)
k_token_features(const T* __restrict__ logits, int vocab, bool vec, const int32_t* __restrict__ token_ids,
                 const uint32_t* __restrict__ counts, float rarity_denominator, const float* __restrict__ attn_var,
                 float* __restrict__ feats) {
    const size_t tok = blockIdx.x;
    const T* row = logits + tok * (size_t)vocab;
    OnlineEntropy acc = {-INFINITY, 0.f, 0.f};
    if (vec) {
        OnlineEntropyPair pr = {-INFINITY, 0.f, 0.f, 0.f, 0.f};
        auto new_maximum = [&](float mm) {
            if (mm > pr.m) {
                if (pr.m == -INFINITY) pr.m = mm;      // nothing summed yet
                else pr.raise_to(mm);
            }
        };
        auto take8 = [&](const Chunk8<T>& c) {
            if constexpr (std::is_same<T, __half>::value) {    // maximum and clamp on fp16 pairs, widened by the subtract
                const __half2 mx = __hmax2(__hmax2(c.h[0], c.h[1]), __hmax2(c.h[2], c.h[3]));
                new_maximum(__half2float(__hmax(__low2half(mx), __high2half(mx))));
#pragma unroll
                for (int i = 0; i < 4; ++i) pr.add2(c.h[i]);
            } else {
                const float* z = c.z;
                new_maximum(fmaxf(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), fmaxf(fmaxf(z[4], z[5]), fmaxf(z[6], z[7]))));
#pragma unroll
                for (int i = 0; i < 8; i += 2) pr.add2(z[i], z[i + 1]);
            }
        };
        // kFeatureLoads 16/32-byte loads of a thread are in flight at once: a row is streamed once, so what keeps
        // the memory system busy is the number of bytes requested ahead, not the arithmetic.
        const int stride = (int)blockDim.x * 8;
        int v0 = threadIdx.x * 8;
        for (; v0 + (kFeatureLoads - 1) * stride < vocab; v0 += kFeatureLoads * stride) {
            Chunk8<T> c[kFeatureLoads];
#pragma unroll
            for (int k = 0; k < kFeatureLoads; ++k) c[k].load(row + v0 + k * stride);
#pragma unroll
            for (int k = 0; k < kFeatureLoads; ++k) take8(c[k]);
        }
        for (; v0 < vocab; v0 += stride) {
            Chunk8<T> c;
            c.load(row + v0);
            take8(c);
        }
        acc.m = pr.m;
        acc.s = pr.s0 + pr.s1;
        acc.w = pr.w0 + pr.w1;
    } else {
        for (int v = threadIdx.x; v < vocab; v += (int)blockDim.x) {
            const float z = (float)row[v];
            if (z > acc.m) acc.raise_to(z);
            acc.add(z);
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        OnlineEntropy o;
        o.m = __shfl_xor_sync(0xffffffffu, acc.m, d);
        o.s = __shfl_xor_sync(0xffffffffu, acc.s, d);
        o.w = __shfl_xor_sync(0xffffffffu, acc.w, d);
        acc.merge(o);
    }
    __shared__ OnlineEntropy part[kFeatureThreadsFew / 32];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x < 32) {                            // warp 0 merges the warps' triples
        const int nwarps = (int)blockDim.x / 32;
        OnlineEntropy tot = {-INFINITY, 0.f, 0.f};
        if ((int)threadIdx.x < nwarps) tot = part[threadIdx.x];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            OnlineEntropy o;
            o.m = __shfl_xor_sync(0xffffffffu, tot.m, d);
            o.s = __shfl_xor_sync(0xffffffffu, tot.s, d);
            o.w = __shfl_xor_sync(0xffffffffu, tot.w, d);
            tot.merge(o);
        }
        if (threadIdx.x != 0) return;
        const float H = logf(tot.s) - tot.w / tot.s;
        const float C = 1.0f / tot.s;
        const int32_t id = token_ids[tok];             // an id outside the table counts as never seen
        const float cnt = ((uint32_t)id < (uint32_t)vocab ? (float)counts[id] : 0.0f) + 1.0f;
        const float R = -logf(cnt / rarity_denominator);
        reinterpret_cast<float4*>(feats)[tok] = make_float4(H, R, attn_var ? attn_var[tok] : 0.f, C);
    }
}

}  // namespace kvq
