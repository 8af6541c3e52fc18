// Controller MLP of Eq. 19-23: 4 -> H -> H -> 4, ReLU after the first two
// layers, argmax over the four logits, class index -> bit-width (Algorithm 1's
// label map {2,4,8,16} <-> {0,1,2,3}).
//
// One thread per token.  The decision must be reproducible bit for bit, so the
// arithmetic is pinned: fp32, every product rounded (__fmul_rn), then every sum
// rounded (__fadd_rn), inputs in ascending order starting from the bias -- the
// intrinsics also keep the compiler from contracting them into FMAs.  Softmax
// (Eq. 22) is monotone, so the argmax of Eq. 23 is taken on the logits; ties go
// to the lowest class and a NaN logit selects the fp16 class.
//
// Weights live in shared memory in the order W1[H][4] b1[H] W2[H][H] b2[H]
// W3[4][H] b3[4]; every lane reads the same word at the same time (broadcast).
#pragma once
#include "kvq_common.cuh"

namespace kvq {

__host__ __device__ inline int controller_floats(int H) { return 4 * H + H + H * H + H + 4 * H + 4; }

// Copy the parameter block to shared memory (all threads of the CTA take part).
__device__ __forceinline__ void controller_stage(float* sW, const float* __restrict__ gW, int H) {
    int n = controller_floats(H);
    for (int i = threadIdx.x; i < n; i += blockDim.x) sW[i] = gW[i];
}

// HC > 0: hidden width known at compile time (fully unrolled, h1 in registers);
// HC == 0: runtime width H <= kMaxHidden (h1 in local memory).
template <int HC>
__device__ __forceinline__ int controller_decide(const float* sW, int Hrt, float x0, float x1, float x2,
                                                 float x3, float logits[4]) {
    const int H = HC > 0 ? HC : Hrt;
    const float* W1 = sW;
    const float* b1 = W1 + 4 * H;
    const float* W2 = b1 + H;
    const float* b2 = W2 + H * H;
    const float* W3 = b2 + H;
    const float* b3 = W3 + 4 * H;
    float h1[HC > 0 ? HC : kMaxHidden];
#pragma unroll
    for (int j = 0; j < H; ++j) {
        float acc = b1[j];
        acc = __fadd_rn(acc, __fmul_rn(W1[4 * j + 0], x0));
        acc = __fadd_rn(acc, __fmul_rn(W1[4 * j + 1], x1));
        acc = __fadd_rn(acc, __fmul_rn(W1[4 * j + 2], x2));
        acc = __fadd_rn(acc, __fmul_rn(W1[4 * j + 3], x3));
        h1[j] = acc > 0.0f ? acc : 0.0f;
    }
    float o0 = b3[0], o1 = b3[1], o2 = b3[2], o3 = b3[3];
#pragma unroll 4
    for (int j = 0; j < H; ++j) {
        float acc = b2[j];
#pragma unroll
        for (int i = 0; i < H; ++i) acc = __fadd_rn(acc, __fmul_rn(W2[j * H + i], h1[i]));
        float h2 = acc > 0.0f ? acc : 0.0f;
        o0 = __fadd_rn(o0, __fmul_rn(W3[0 * H + j], h2));
        o1 = __fadd_rn(o1, __fmul_rn(W3[1 * H + j], h2));
        o2 = __fadd_rn(o2, __fmul_rn(W3[2 * H + j], h2));
        o3 = __fadd_rn(o3, __fmul_rn(W3[3 * H + j], h2));
    }
    logits[0] = o0; logits[1] = o1; logits[2] = o2; logits[3] = o3;
    if (o0 != o0 || o1 != o1 || o2 != o2 || o3 != o3) return 3;
    int cls = 0;
    float best = o0;
    if (o1 > best) { best = o1; cls = 1; }
    if (o2 > best) { best = o2; cls = 2; }
    if (o3 > best) { best = o3; cls = 3; }
    return cls;
}

// Two tokens at once, hidden width 32: every weight is read from shared memory once for both and the two chains of
// rounded products and sums are independent, so they overlap.  Same arithmetic and order per token as above.
__device__ __forceinline__ void controller_decide_two32(const float* sW, const float4& xa, const float4& xb, int& cls_a,
                                                        int& cls_b) {
    constexpr int H = 32;
    const float* W1 = sW;
    const float* b1 = W1 + 4 * H;
    const float* W2 = b1 + H;
    const float* b2 = W2 + H * H;
    const float* W3 = b2 + H;
    const float* b3 = W3 + 4 * H;
    float ha[H], hb[H];
#pragma unroll
    for (int j = 0; j < H; ++j) {
        const float4 w = *reinterpret_cast<const float4*>(W1 + 4 * j);
        float a = b1[j], b = a;
        a = __fadd_rn(a, __fmul_rn(w.x, xa.x)); b = __fadd_rn(b, __fmul_rn(w.x, xb.x));
        a = __fadd_rn(a, __fmul_rn(w.y, xa.y)); b = __fadd_rn(b, __fmul_rn(w.y, xb.y));
        a = __fadd_rn(a, __fmul_rn(w.z, xa.z)); b = __fadd_rn(b, __fmul_rn(w.z, xb.z));
        a = __fadd_rn(a, __fmul_rn(w.w, xa.w)); b = __fadd_rn(b, __fmul_rn(w.w, xb.w));
        ha[j] = a > 0.0f ? a : 0.0f;
        hb[j] = b > 0.0f ? b : 0.0f;
    }
    float oa[4], ob[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) oa[c] = ob[c] = b3[c];
#pragma unroll 4
    for (int j = 0; j < H; ++j) {
        float a = b2[j], b = a;
#pragma unroll
        for (int i = 0; i < H; i += 4) {
            const float4 w = *reinterpret_cast<const float4*>(W2 + j * H + i);
            a = __fadd_rn(a, __fmul_rn(w.x, ha[i + 0])); b = __fadd_rn(b, __fmul_rn(w.x, hb[i + 0]));
            a = __fadd_rn(a, __fmul_rn(w.y, ha[i + 1])); b = __fadd_rn(b, __fmul_rn(w.y, hb[i + 1]));
            a = __fadd_rn(a, __fmul_rn(w.z, ha[i + 2])); b = __fadd_rn(b, __fmul_rn(w.z, hb[i + 2]));
            a = __fadd_rn(a, __fmul_rn(w.w, ha[i + 3])); b = __fadd_rn(b, __fmul_rn(w.w, hb[i + 3]));
        }
        const float h2a = a > 0.0f ? a : 0.0f, h2b = b > 0.0f ? b : 0.0f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float w = W3[c * H + j];
            oa[c] = __fadd_rn(oa[c], __fmul_rn(w, h2a));
            ob[c] = __fadd_rn(ob[c], __fmul_rn(w, h2b));
        }
    }
    auto pick = [](const float (&o)[4]) {
        if (o[0] != o[0] || o[1] != o[1] || o[2] != o[2] || o[3] != o[3]) return 3;
        int cls = 0;
        float best = o[0];
        if (o[1] > best) { best = o[1]; cls = 1; }
        if (o[2] > best) { best = o[2]; cls = 2; }
        if (o[3] > best) { best = o[3]; cls = 3; }
        return cls;
    };
    cls_a = pick(oa);
    cls_b = pick(ob);
}

__device__ __forceinline__ int controller_decide_any(const float* sW, int H, float x0, float x1, float x2,
                                                     float x3, float logits[4]) {
    if (H == 32) return controller_decide<32>(sW, H, x0, x1, x2, x3, logits);
    return controller_decide<0>(sW, H, x0, x1, x2, x3, logits);
}

// The same decision taken by a whole warp for ONE token, hidden width 32: lane j owns hidden unit j.
// Every sum still runs in ascending input order with separately rounded products and sums, so the
// result is bit-identical to controller_decide; the warp only removes the serial walk over the 32 x 32
// second layer from the critical path of a decode step (one token per sequence).  gW is the
// parameter block in global memory (row j of W2 and of W3 is read straight into registers).
// Returns the class in every lane.
__device__ __forceinline__ int controller_decide_warp32(const float* __restrict__ gW, float x0, float x1, float x2,
                                                        float x3, int lane) {
    constexpr int H = 32;
    const float* W1 = gW;
    const float* b1 = W1 + 4 * H;
    const float* W2 = b1 + H;
    const float* b2 = W2 + H * H;
    const float* W3 = b2 + H;
    const float* b3 = W3 + 4 * H;
    float w2row[H], w3row[H];
#pragma unroll
    for (int i = 0; i < H / 4; ++i) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(W2 + lane * H) + i);
        w2row[4 * i] = v.x; w2row[4 * i + 1] = v.y; w2row[4 * i + 2] = v.z; w2row[4 * i + 3] = v.w;
        const float4 u = __ldg(reinterpret_cast<const float4*>(W3 + (lane & 3) * H) + i);
        w3row[4 * i] = u.x; w3row[4 * i + 1] = u.y; w3row[4 * i + 2] = u.z; w3row[4 * i + 3] = u.w;
    }
    const float4 w1 = __ldg(reinterpret_cast<const float4*>(W1) + lane);
    float acc = __ldg(b1 + lane);
    acc = __fadd_rn(acc, __fmul_rn(w1.x, x0));
    acc = __fadd_rn(acc, __fmul_rn(w1.y, x1));
    acc = __fadd_rn(acc, __fmul_rn(w1.z, x2));
    acc = __fadd_rn(acc, __fmul_rn(w1.w, x3));
    const float h1 = acc > 0.0f ? acc : 0.0f;
    acc = __ldg(b2 + lane);
#pragma unroll
    for (int i = 0; i < H; ++i) acc = __fadd_rn(acc, __fmul_rn(w2row[i], __shfl_sync(0xffffffffu, h1, i)));
    const float h2 = acc > 0.0f ? acc : 0.0f;
    float o = __ldg(b3 + (lane & 3));                  // lanes 0..3 hold the four logits (the others mirror them)
#pragma unroll
    for (int j = 0; j < H; ++j) o = __fadd_rn(o, __fmul_rn(w3row[j], __shfl_sync(0xffffffffu, h2, j)));
    const float o0 = __shfl_sync(0xffffffffu, o, 0), o1 = __shfl_sync(0xffffffffu, o, 1);
    const float o2 = __shfl_sync(0xffffffffu, o, 2), o3 = __shfl_sync(0xffffffffu, o, 3);
    if (o0 != o0 || o1 != o1 || o2 != o2 || o3 != o3) return 3;
    int cls = 0;
    float best = o0;
    if (o1 > best) { best = o1; cls = 1; }
    if (o2 > best) { best = o2; cls = 2; }
    if (o3 > best) { best = o3; cls = 3; }
    return cls;
}

// The same decision taken by a CTA of 128 threads for ONE token, any hidden width H <= 128: thread j owns hidden
// unit j.  W2 and W3 come into shared memory with 16-byte async copies in which neighbouring threads take
// neighbouring pieces of the matrices (whole 128-byte lines per request); their rows are padded by four floats
// there, so that the 16-byte reads of the sums below (thread j reads row j of W2, lane l row l % 4 of W3) fall into
// different banks.  First- and second-layer outputs cross shared memory; all sums in ascending input order with
// separately rounded products and sums, so the result is bit-identical to controller_decide.  Every thread of
// the CTA must call both parts; part 2 returns the class in every thread.  sh: kControllerCtaSmemFloats floats,
// 16-byte aligned.
constexpr int kW2RowStride = kMaxHidden + 4;
constexpr int kControllerCtaSmemFloats = 2 * kMaxHidden + 4 * kW2RowStride + kMaxHidden * kW2RowStride;
// Whether W2 and W3 of the parameter block at gW can be moved and read in 16-byte pieces.
__device__ __forceinline__ bool controller_rows_vectorized(const float* gW, int H) {
    return (H & 3) == 0 && (reinterpret_cast<uintptr_t>(gW + 5 * H) & 15u) == 0 && (reinterpret_cast<uintptr_t>(gW + 6 * H + H * H) & 15u) == 0;
}
__device__ __forceinline__ void cp_async16_ca(float* smem_dst, const float* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
// acc + sum over i of w[i] * h[i], i ascending, every product and every sum rounded (w, h: 16-byte aligned when VEC).
template <bool VEC>
__device__ __forceinline__ float ordered_dot(float acc, const float* w, const float* h, int H) {
    if (VEC) {
#pragma unroll 4
        for (int i = 0; i < H; i += 4) {
            const float4 w4 = *reinterpret_cast<const float4*>(w + i), h4 = *reinterpret_cast<const float4*>(h + i);
            acc = __fadd_rn(acc, __fmul_rn(w4.x, h4.x));
            acc = __fadd_rn(acc, __fmul_rn(w4.y, h4.y));
            acc = __fadd_rn(acc, __fmul_rn(w4.z, h4.z));
            acc = __fadd_rn(acc, __fmul_rn(w4.w, h4.w));
        }
    } else {
#pragma unroll 8
        for (int i = 0; i < H; ++i) acc = __fadd_rn(acc, __fmul_rn(w[i], h[i]));
    }
    return acc;
}
// Part 1: request W2 and W3 (they are written by kvq_set_controller only, never by a kernel).
__device__ __forceinline__ void controller_fetch_cta128(const float* __restrict__ gW, int H, float* sh) {
    const int j = threadIdx.x;
    const float* W2 = gW + 5 * H;
    const float* W3 = W2 + H * H + H;
    float* w3s = sh + 2 * kMaxHidden;                  // the four rows of W3, kW2RowStride apart
    float* w2s = w3s + 4 * kW2RowStride;               // the H rows of W2, kW2RowStride apart
    if (controller_rows_vectorized(gW, H)) {
        const int per_row = H >> 2;                    // 16-byte pieces per row
        for (int piece = j; piece < H * per_row; piece += 128) {
            const int r = piece / per_row, c = (piece - r * per_row) << 2;
            cp_async16_ca(w2s + r * kW2RowStride + c, W2 + (size_t)r * H + c);
        }
        for (int piece = j; piece < 4 * per_row; piece += 128) {
            const int r = piece / per_row, c = (piece - r * per_row) << 2;
            cp_async16_ca(w3s + r * kW2RowStride + c, W3 + (size_t)r * H + c);
        }
    } else {
        for (int i = j; i < H * H; i += 128) w2s[(i / H) * kW2RowStride + i % H] = __ldg(W2 + i);
        for (int i = j; i < 4 * H; i += 128) w3s[(i / H) * kW2RowStride + i % H] = __ldg(W3 + i);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}
// Part 2: the decision, once controller_fetch_cta128 has been called with the same arguments.
__device__ __forceinline__ int controller_decide_cta128(const float* __restrict__ gW, int H, float x0, float x1, float x2,
                                                        float x3, float* sh) {
    const int j = threadIdx.x;
    const float* W1 = gW;
    const float* b1 = W1 + 4 * H;
    const float* b2 = b1 + H + H * H;
    const float* b3 = b2 + H + 4 * H;
    float* h1s = sh;
    float* h2s = sh + kMaxHidden;
    float* w3s = sh + 2 * kMaxHidden;
    float* w2s = w3s + 4 * kW2RowStride;
    const bool mine = j < H;
    const bool vec = controller_rows_vectorized(gW, H);
    float acc = 0.f;
    if (mine) {
        float a = __ldg(b1 + j);
        a = __fadd_rn(a, __fmul_rn(__ldg(W1 + 4 * j + 0), x0));
        a = __fadd_rn(a, __fmul_rn(__ldg(W1 + 4 * j + 1), x1));
        a = __fadd_rn(a, __fmul_rn(__ldg(W1 + 4 * j + 2), x2));
        a = __fadd_rn(a, __fmul_rn(__ldg(W1 + 4 * j + 3), x3));
        h1s[j] = a > 0.0f ? a : 0.0f;
        acc = __ldg(b2 + j);
    }
    const int lane = threadIdx.x & 31;
    float o = __ldg(b3 + (lane & 3));                  // lanes 0..3 of every warp hold the four logits
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    if (mine) {
        acc = vec ? ordered_dot<true>(acc, w2s + j * kW2RowStride, h1s, H) : ordered_dot<false>(acc, w2s + j * kW2RowStride, h1s, H);
        h2s[j] = acc > 0.0f ? acc : 0.0f;
    }
    __syncthreads();
    const float* w3 = w3s + (lane & 3) * kW2RowStride;
    o = vec ? ordered_dot<true>(o, w3, h2s, H) : ordered_dot<false>(o, w3, h2s, H);
    const float o0 = __shfl_sync(0xffffffffu, o, 0), o1 = __shfl_sync(0xffffffffu, o, 1);
    const float o2 = __shfl_sync(0xffffffffu, o, 2), o3 = __shfl_sync(0xffffffffu, o, 3);
    if (o0 != o0 || o1 != o1 || o2 != o2 || o3 != o3) return 3;
    int cls = 0;
    float best = o0;
    if (o1 > best) { best = o1; cls = 1; }
    if (o2 > best) { best = o2; cls = 2; }
    if (o3 > best) { best = o3; cls = 3; }
    return cls;
}

// The same decision taken by the first 128 threads of a CTA (any CTA size) with a few KB of shared memory: thread j
// owns hidden unit j and reads its row of W2 straight from global memory, 32 weights at a time (they are read by
// every CTA of a launch and stay in L2).  The 128 threads meet at the named barrier 1, so the other threads of the
// CTA need not take part.  Sums in ascending input order with separately rounded products and sums: bit-identical
// to controller_decide.  Every one of the 128 threads must call it; returns the class in all of them.
// sh: kControllerDirectSmemFloats floats, 16-byte aligned.
constexpr int kControllerDirectSmemFloats = 2 * kMaxHidden + 4 * kW2RowStride;
__device__ __forceinline__ void barrier_first_128() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ int controller_decide_cta_direct(const float* __restrict__ gW, int H, float x0, float x1, float x2,
                                                            float x3, float* sh) {
    const int j = threadIdx.x;
    const float* W1 = gW;
    const float* b1 = W1 + 4 * H;
    const float* W2 = b1 + H;
    const float* b2 = W2 + H * H;
    const float* W3 = b2 + H;
    const float* b3 = W3 + 4 * H;
    float* h1s = sh;
    float* h2s = sh + kMaxHidden;
    float* w3s = sh + 2 * kMaxHidden;                  // the four rows of W3, kW2RowStride apart
    const bool mine = j < H;
    const bool vec = controller_rows_vectorized(gW, H);
    for (int i = j; i < 4 * H; i += 128) w3s[(i / H) * kW2RowStride + i % H] = __ldg(W3 + i);
    float acc = 0.f;
    if (mine) {
        float a = __ldg(b1 + j);
        a = __fadd_rn(a, __fmul_rn(__ldg(W1 + 4 * j + 0), x0));
        a = __fadd_rn(a, __fmul_rn(__ldg(W1 + 4 * j + 1), x1));
        a = __fadd_rn(a, __fmul_rn(__ldg(W1 + 4 * j + 2), x2));
        a = __fadd_rn(a, __fmul_rn(__ldg(W1 + 4 * j + 3), x3));
        h1s[j] = a > 0.0f ? a : 0.0f;
        acc = __ldg(b2 + j);
    }
    barrier_first_128();
    if (mine) {
        const float* row = W2 + (size_t)j * H;
        if (vec) {
            for (int i0 = 0; i0 < H; i0 += 32) {       // 32 weights in flight, then their 32 ordered terms
                float4 w[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) w[k] = i0 + 4 * k < H ? __ldg(reinterpret_cast<const float4*>(row + i0) + k) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (i0 + 4 * k < H) {
                        const float4 h4 = *reinterpret_cast<const float4*>(h1s + i0 + 4 * k);
                        acc = __fadd_rn(acc, __fmul_rn(w[k].x, h4.x));
                        acc = __fadd_rn(acc, __fmul_rn(w[k].y, h4.y));
                        acc = __fadd_rn(acc, __fmul_rn(w[k].z, h4.z));
                        acc = __fadd_rn(acc, __fmul_rn(w[k].w, h4.w));
                    }
                }
            }
        } else {
#pragma unroll 4
            for (int i = 0; i < H; ++i) acc = __fadd_rn(acc, __fmul_rn(__ldg(row + i), h1s[i]));
        }
        h2s[j] = acc > 0.0f ? acc : 0.0f;
    }
    barrier_first_128();
    const int lane = threadIdx.x & 31;
    float o = __ldg(b3 + (lane & 3));                  // lanes 0..3 of every warp hold the four logits
    const float* w3 = w3s + (lane & 3) * kW2RowStride;
    o = (H & 3) == 0 ? ordered_dot<true>(o, w3, h2s, H) : ordered_dot<false>(o, w3, h2s, H);
    const float o0 = __shfl_sync(0xffffffffu, o, 0), o1 = __shfl_sync(0xffffffffu, o, 1);
    const float o2 = __shfl_sync(0xffffffffu, o, 2), o3 = __shfl_sync(0xffffffffu, o, 3);
    if (o0 != o0 || o1 != o1 || o2 != o2 || o3 != o3) return 3;
    int cls = 0;
    float best = o0;
    if (o1 > best) { best = o1; cls = 1; }
    if (o2 > best) { best = o2; cls = 2; }
    if (o3 > best) { best = o3; cls = 3; }
    return cls;
}

// kvq_select_bits: one thread per token.
__global__ void __launch_bounds__(128)
k_select_bits(const float* __restrict__ feats, int n, const float* __restrict__ gW, int H,
              uint8_t* __restrict__ bits, float* __restrict__ logits_opt) {
    extern __shared__ float sW[];
    controller_stage(sW, gW, H);
    __syncthreads();
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n) return;
    float4 f = reinterpret_cast<const float4*>(feats)[t];
    float lg[4];
    int cls = controller_decide_any(sW, H, f.x, f.y, f.z, f.w, lg);
    bits[t] = (uint8_t)pool_bits(cls);
    if (logits_opt) reinterpret_cast<float4*>(logits_opt)[t] = make_float4(lg[0], lg[1], lg[2], lg[3]);
}

}  // namespace kvq
