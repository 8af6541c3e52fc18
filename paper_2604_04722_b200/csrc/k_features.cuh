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

namespace kvq {

constexpr int kFeatureThreads = 256;       // many tokens: several CTAs per SM
constexpr int kFeatureThreadsFew = 1024;   // a decode step's handful of tokens: more loads in flight per row

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

template <typename T>
__device__ __forceinline__ void load8(const T* p, float (&z)[8]);
template <>
__device__ __forceinline__ void load8<__half>(const __half* p, float (&z)[8]) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h[i]);
        z[2 * i] = f.x;
        z[2 * i + 1] = f.y;
    }
}
template <>
__device__ __forceinline__ void load8<float>(const float* p, float (&z)[8]) {
    const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
    z[0] = a.x; z[1] = a.y; z[2] = a.z; z[3] = a.w;
    z[4] = b.x; z[5] = b.y; z[6] = b.z; z[7] = b.w;
}

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
        for (int v0 = threadIdx.x * 8; v0 < vocab; v0 += (int)blockDim.x * 8) {
            float z[8];
            load8<T>(row + v0, z);
            float mm = z[0];
#pragma unroll
            for (int i = 1; i < 8; ++i) mm = fmaxf(mm, z[i]);
            if (mm > acc.m) acc.raise_to(mm);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc.add(z[i]);
        }
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
