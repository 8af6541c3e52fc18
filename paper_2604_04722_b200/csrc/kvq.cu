// Host side of the C ABI declared in include/kvq.h: handle, argument checks,
// launch planning.  All arithmetic of the method runs in the kernels included
// below; nothing here computes on the CPU.
#include "../../include/kvq.h"

#include <cstdio>
#include <cstdlib>
#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>
#include <vector>

#include "kvq_common.cuh"
#include "k_controller.cuh"
#include "k_append.cuh"
#include "k_append_frag.cuh"
#include "k_decode.cuh"
#include "k_export.cuh"
#include "k_features.cuh"

#ifndef KVQ_NVTX
#define KVQ_NVTX 1                       // NVTX ranges around the entry points that launch the hot kernels
#endif
#if KVQ_NVTX
#include <nvtx3/nvToolsExt.h>
#endif

using namespace kvq;

struct kvq_ctx {
    int device = 0, sm_count = 0;
    int layers = 0, q_heads = 0, kv_heads = 0, max_ctx = 0, batch = 0;
    int groups = 1;                      // {scale, zero-point} pairs per quantized row: 1 or 2
    StoreView store{};
    uint8_t* arena = nullptr;            // the tile records: blocks of kBlockBytes
    uint32_t* table = nullptr;           // block tables of all streams
    uint32_t* arena_used = nullptr;      // device counter of blocks handed out
    uint32_t* counts = nullptr;          // [2][layers][batch][4], double-buffered pool fills
    __half* kres = nullptr;              // per-channel keys: fp16 rows of the open windows (nullptr in the other layouts)
    size_t kres_bytes = 0;
    __half* kres_old = nullptr;          // copy of one layer's residual rows, taken before a multi-token append
    std::vector<int> len;                // host mirror: tokens of the longest sequence, per layer
    std::vector<int> lens;               // host mirror: tokens per (layer, sequence)
    std::vector<char> ragged;            // per layer: sequences differ in length
    // Per-sequence lengths of ragged calls travel through a small ring of page-locked host slots and matching
    // device slots: one asynchronous copy per call, no synchronisation of the caller's stream.  A slot is reused
    // only after the event recorded behind its last copy has completed (checked on the host).
    static constexpr int kLenSlots = 8;
    int* d_lens = nullptr;               // device [kLenSlots][3][batch]: a call's new tokens, first positions, lengths
    int* h_lens = nullptr;               // page-locked host mirror of the same shape
    cudaEvent_t len_ev[kLenSlots] = {};
    int len_slot = 0;
    std::vector<int> cur;                // which counts buffer is current, per layer
    uint8_t* cls = nullptr;              // append scratch [batch][max_ctx]
    uint4* hist = nullptr;               // append scratch [batch][max chunks]
    uint32_t* chunk_arrivals = nullptr;  // append scratch [batch], zero between launches
    float* ctrl = nullptr;               // controller parameter block
    uint32_t* step_cls = nullptr;        // [batch] class of the step's token, published inside a one-launch step (wide controllers)
    uint32_t step_serial = 0;            // tag of the last such launch
    int hidden = 0;
    float* part_o = nullptr;             // decode scratch [units][partial slots][64]
    float2* part_ml = nullptr;           //                [units][partial slots]
    uint32_t* part_cnt = nullptr;        //                [units] arrival counters, zero between launches
    float* part_s2 = nullptr;            //                [units][partial slots] sum of squared weights (kvq_decode_attn_var)
    float* unit_var = nullptr;           //                [units] variance of a unit's attention weights
    uint32_t* vis = nullptr;             // kvq_attend_last: visible pool fills [batch][query rows of a launch][4]
    int splits_override = 0;
    int chunk_override = 0;              // kvq_set_append_chunk: 0 = automatic, else tokens per thread of a prefill chunk
    uint32_t* flags = nullptr;
    // device staging for the host-buffer entry points
    float* st_feats = nullptr;
    __half *st_K = nullptr, *st_V = nullptr, *st_Q = nullptr, *st_O = nullptr;
    uint8_t* st_bits = nullptr;
    uint8_t* st_export = nullptr;
    bool profiling = false;              // decode timing hooks
    std::vector<cudaEvent_t> prof_ev;    // 2 events per recorded call
    int prof_calls = 0;
    uint64_t device_bytes = 0, launches = 0;
    // Where the device buffers come from: 0 = one cudaMalloc each; 1 = none, only their sizes are added up
    // (kvq_workspace_bytes); 2 = carved out of the caller's workspace (kvq_create_in).
    int mem_mode = 0;
    uint8_t* slab = nullptr;
    size_t slab_size = 0, slab_used = 0;
    bool slab_short = false;             // the caller's workspace was too small
    size_t table_bytes = 0;              // size of `table`
    cudaError_t last_err = cudaSuccess;
};

namespace {

struct TraceRange {                      // a named range for timeline tools; costs nothing when none is attached
#if KVQ_NVTX
    explicit TraceRange(const char* name) { nvtxRangePushA(name); }
    ~TraceRange() { nvtxRangePop(); }
#else
    explicit TraceRange(const char*) {}
#endif
};

struct DeviceGuard {                     // make the handle's device current for the duration of a call
    int prev = -1;
    explicit DeviceGuard(int dev) {
        cudaGetDevice(&prev);
        if (prev != dev) cudaSetDevice(dev);
        else prev = -1;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

#define KVQ_CUDA(ctx, call)                         \
    do {                                            \
        cudaError_t e__ = (call);                   \
        if (e__ != cudaSuccess) {                   \
            (ctx)->last_err = e__;                  \
            return KVQ_ERR_CUDA;                    \
        }                                           \
    } while (0)

template <typename T>
cudaError_t dev_alloc(kvq_ctx* c, T** p, size_t bytes) {
    if (c->mem_mode != 0) {                          // 256-byte aligned pieces of one workspace
        const size_t need = ((bytes ? bytes : 1) + 255) & ~(size_t)255;
        if (c->mem_mode == 2 && c->slab_used + need > c->slab_size) {
            c->slab_short = true;
            return cudaErrorMemoryAllocation;
        }
        *p = c->mem_mode == 2 ? reinterpret_cast<T*>(c->slab + c->slab_used) : nullptr;
        c->slab_used += need;
        c->device_bytes += bytes;
        return cudaSuccess;
    }
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), bytes ? bytes : 1);
    if (e == cudaSuccess) c->device_bytes += bytes;
    return e;
}

constexpr int kProfMaxCalls = 1024;

#ifndef KVQ_APPEND_WAVES_SMALL
#define KVQ_APPEND_WAVES_SMALL 2
#endif
#ifndef KVQ_APPEND_WAVES
#define KVQ_APPEND_WAVES 16
#endif
#ifndef KVQ_APPEND_TOKENS_PER_THREAD
#define KVQ_APPEND_TOKENS_PER_THREAD 2
#endif
static_assert(KVQ_APPEND_TOKENS_PER_THREAD >= 1 && KVQ_APPEND_TOKENS_PER_THREAD <= kMaxTokensPerThread, "chunk size");
#ifndef KVQ_OVERLAP_LAUNCHES
#define KVQ_OVERLAP_LAUNCHES 1
#endif
// Launch with programmatic stream serialization (see pdl_wait): the kernel may be scheduled before the
// kernel ahead of it in the stream has finished, if that kernel allows it; it waits inside for its end.
template <class... Params>
void launch_overlapped(void (*kernel)(Params...), dim3 grid, unsigned block, size_t smem, cudaStream_t st, const Params&... p) {
#if KVQ_OVERLAP_LAUNCHES
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, p...);
#else
    kernel<<<grid, block, smem, st>>>(p...);
#endif
}

void free_all(kvq_ctx* c) {
    for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
    c->prof_ev.clear();
    for (cudaEvent_t& e : c->len_ev) {
        if (e) cudaEventDestroy(e);
        e = nullptr;
    }
    if (c->h_lens) cudaFreeHost(c->h_lens);
    c->h_lens = nullptr;
    if (c->mem_mode != 0) return;                      // the buffers belong to the caller's workspace (or do not exist)
    cudaFree(c->arena);
    cudaFree(c->table);
    cudaFree(c->arena_used);
    cudaFree(c->store.index);
    cudaFree(c->counts);
    cudaFree(c->kres);
    cudaFree(c->kres_old);
    cudaFree(c->cls);
    cudaFree(c->hist);
    cudaFree(c->chunk_arrivals);
    cudaFree(c->ctrl);
    cudaFree(c->step_cls);
    cudaFree(c->part_o);
    cudaFree(c->part_ml);
    cudaFree(c->part_cnt);
    cudaFree(c->vis);
    cudaFree(c->part_s2);
    cudaFree(c->unit_var);
    cudaFree(c->d_lens);
    cudaFree(c->flags);
    cudaFree(c->st_feats);
    cudaFree(c->st_K);
    cudaFree(c->st_V);
    cudaFree(c->st_Q);
    cudaFree(c->st_O);
    cudaFree(c->st_bits);
    cudaFree(c->st_export);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The device's address for a page-locked host buffer, or nullptr if `p` is not one (pageable memory, or an
// address the kernels' 16-byte accesses could not use).
const void* device_view(const void* p) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer || !aligned16(a.devicePointer)) return nullptr;
    return a.devicePointer;
}

// The next slot of the lengths ring: host and device addresses.  Waits (on the host, for an event) only if the slot's
// previous copy, kLenSlots ragged calls ago, has not run yet.
int claim_len_slot(kvq_ctx* c, int** host, int** dev) {
    const int s = c->len_slot;
    c->len_slot = (s + 1) % kvq_ctx::kLenSlots;
    if (cudaEventQuery(c->len_ev[s]) == cudaErrorNotReady) KVQ_CUDA(c, cudaEventSynchronize(c->len_ev[s]));
    cudaGetLastError();
    *host = c->h_lens + (size_t)s * 3 * c->batch;
    *dev = c->d_lens + (size_t)s * 3 * c->batch;
    return s;
}

inline uint32_t* counts_of(kvq_ctx* c, int which, int layer) {
    return c->counts + ((size_t)which * c->layers + layer) * c->batch * 4;
}

int check_layer(kvq_ctx* c, int layer) { return (c && layer >= 0 && layer < c->layers) ? KVQ_OK : KVQ_ERR_ARG; }

size_t controller_smem(int hidden) { return sizeof(float) * (size_t)controller_floats(hidden); }

// Shared by kvq_append, kvq_append_fused and kvq_append_ragged.  host_lens: tokens each sequence adds (host
// int [batch], each 0..n_new) or nullptr for n_new everywhere.
int append_impl(kvq_ctx* c, int layer, const void* K, const void* V, const uint8_t* bits, const float* feats,
                uint8_t* bits_out, int n_new, const int* host_lens, cudaStream_t st) {
    TraceRange trace(feats ? "kvq_append (controller inside)" : "kvq_append");
    if (check_layer(c, layer) != KVQ_OK || n_new < 0) return KVQ_ERR_ARG;
    if (n_new == 0) return KVQ_OK;
    int* cur_lens = &c->lens[(size_t)layer * c->batch];
    bool call_ragged = false;
    if (host_lens) {
        for (int b = 0; b < c->batch; ++b) {
            if (host_lens[b] < 0 || host_lens[b] > n_new) return KVQ_ERR_ARG;
            call_ragged = call_ragged || host_lens[b] != n_new;
        }
    }
    if (!K || !V || !aligned16(K) || !aligned16(V)) return KVQ_ERR_ARG;
    const bool fused = feats != nullptr;
    if (fused) {
        if (!aligned16(feats)) return KVQ_ERR_ARG;
        if (c->hidden == 0) return KVQ_ERR_NO_CONTROLLER;
    } else if (!bits) {
        return KVQ_ERR_ARG;
    }
    for (int b = 0; b < c->batch; ++b)
        if (cur_lens[b] + (host_lens ? host_lens[b] : n_new) > c->max_ctx) return KVQ_ERR_CAPACITY;
    DeviceGuard guard(c->device);

    AppendParams p{};
    p.store = c->store;
    p.K = static_cast<const __half*>(K);
    p.V = static_cast<const __half*>(V);
    p.bits = bits;
    p.feats = feats;
    p.ctrl = c->ctrl;
    p.hidden = c->hidden;
    p.bits_out = bits_out;
    p.cls = c->cls;
    p.hist = c->hist;
    p.chunk_arrivals = c->chunk_arrivals;
    p.counts_in = counts_of(c, c->cur[layer], layer);
    p.counts_out = counts_of(c, c->cur[layer] ^ 1, layer);
    p.layer = layer;
    p.n_new = n_new;
    p.pos0 = c->len[layer];
    if (call_ragged || c->ragged[layer]) {             // per-sequence counts and positions travel with the call
        int *h_slot = nullptr, *d_slot = nullptr;
        const int slot = claim_len_slot(c, &h_slot, &d_slot);
        if (slot < 0) return slot;
        for (int b = 0; b < c->batch; ++b) {
            h_slot[b] = host_lens ? host_lens[b] : n_new;
            h_slot[c->batch + b] = cur_lens[b];
        }
        KVQ_CUDA(c, cudaMemcpyAsync(d_slot, h_slot, sizeof(int) * 2 * c->batch, cudaMemcpyHostToDevice, st));
        KVQ_CUDA(c, cudaEventRecord(c->len_ev[slot], st));
        p.lens = d_slot;
        p.pos = d_slot + c->batch;
    }
    // Long prefills use chunks of 1024 tokens (fewer partly filled tiles at chunk ends), as long as that still
    // leaves several waves of CTAs once the KV heads are split into groups; everything else 256.
    p.tpt = 1;
    if (c->chunk_override) {
        p.tpt = c->chunk_override;
    } else if (KVQ_APPEND_TOKENS_PER_THREAD > 1) {
        const long long big_chunks = (n_new + kChunkTokens * KVQ_APPEND_TOKENS_PER_THREAD - 1) / (kChunkTokens * KVQ_APPEND_TOKENS_PER_THREAD);
        if (big_chunks * c->batch * c->kv_heads >= 12LL * c->sm_count * 2) p.tpt = KVQ_APPEND_TOKENS_PER_THREAD;
    }
    if (n_new <= kChunkTokens) p.tpt = 1;              // one CTA per (head group, sequence) does everything
    const int chunk_tokens = kChunkTokens * p.tpt;
    p.nchunks = (n_new + chunk_tokens - 1) / chunk_tokens;
    // enough CTAs to fill the device: split the KV heads into groups when chunks x batch is small
    const int waves = p.tpt > 1 ? KVQ_APPEND_WAVES : KVQ_APPEND_WAVES_SMALL;
    int want_groups = (waves * c->sm_count + p.nchunks * c->batch - 1) / (p.nchunks * c->batch);
    int groups = want_groups < 1 ? 1 : (want_groups > c->kv_heads ? c->kv_heads : want_groups);
    p.heads_per_group = (c->kv_heads + groups - 1) / groups;
    groups = (c->kv_heads + p.heads_per_group - 1) / p.heads_per_group;

    const size_t smem = fused ? controller_smem(c->hidden) : 0;
    dim3 grid_q(p.nchunks, groups, c->batch);
    if (c->groups == kLayoutPerChannelK && !(n_new == 1 && !call_ragged) && c->len[layer] > 0) {
        // Per-channel keys: the multi-token kernels read the rows of the windows left open by earlier calls from a
        // copy, because the rows of each stream's next open window go to the same places during the launch.
        const size_t slice = c->kres_bytes / c->layers;
        KVQ_CUDA(c, cudaMemcpyAsync(c->kres_old, reinterpret_cast<const uint8_t*>(c->kres) + (size_t)layer * slice, slice,
                                    cudaMemcpyDeviceToDevice, st));
    }
    if (n_new == 1 && !call_ragged) {                  // a decode step: one warp per 16 heads
        dim3 grid_t((c->kv_heads + 15) / 16, c->batch);
        const unsigned bt = fused && c->hidden != 32 ? 128 : 32;   // a controller of another width is evaluated by four warps
        const size_t ts = bt == 128 ? sizeof(float) * kControllerCtaSmemFloats : 0;
        if (c->groups == kLayoutPerChannelK) {         // keys wait as fp16 rows; a second small launch packs completed windows
            if (fused) launch_overlapped(k_append_token<true, kLayoutPerChannelK>, grid_t, bt, ts, st, p);
            else launch_overlapped(k_append_token<false, kLayoutPerChannelK>, grid_t, bt, ts, st, p);
            k_pack_window<<<dim3(c->kv_heads, c->batch), 32, 0, st>>>(p);
            c->launches += 1;
        } else if (c->groups == 1) {
            if (fused) launch_overlapped(k_append_token<true, 1>, grid_t, bt, ts, st, p);
            else launch_overlapped(k_append_token<false, 1>, grid_t, bt, ts, st, p);
        } else {
            if (fused) launch_overlapped(k_append_token<true, 2>, grid_t, bt, ts, st, p);
            else launch_overlapped(k_append_token<false, 2>, grid_t, bt, ts, st, p);
        }
        c->launches += 1;
    } else if (n_new <= kChunkTokens) {
        if (c->groups == kLayoutPerChannelK) {
            if (fused) k_quant_pack_frag<2, 1, true><<<grid_q, kChunkTokens, kFragRingBytes + smem, st>>>(p);
            else k_quant_pack_frag<1, 1, true><<<grid_q, kChunkTokens, kFragRingBytes, st>>>(p);
        } else if (c->groups == 1) {
            if (fused) k_quant_pack_frag<2><<<grid_q, kChunkTokens, kFragRingBytes + smem, st>>>(p);
            else k_quant_pack_frag<1><<<grid_q, kChunkTokens, kFragRingBytes, st>>>(p);
        } else {
            if (fused) k_quant_pack<2, 2><<<grid_q, kChunkTokens, kAppendRingBytes + smem, st>>>(p);
            else k_quant_pack<1, 2><<<grid_q, kChunkTokens, kAppendRingBytes, st>>>(p);
        }
        c->launches += 1;
    } else {
        dim3 grid_c(p.nchunks, c->batch);
        if (fused) k_classify<true><<<grid_c, kChunkTokens, smem, st>>>(p);
        else k_classify<false><<<grid_c, kChunkTokens, 0, st>>>(p);
        if (p.tpt == 1) {
            if (c->groups == kLayoutPerChannelK) k_quant_pack_frag<0, 1, true><<<grid_q, kChunkTokens, kFragRingBytes, st>>>(p);
            else if (c->groups == 1) k_quant_pack_frag<0, 1><<<grid_q, kChunkTokens, kFragRingBytes, st>>>(p);
            else k_quant_pack<0, 2, 1><<<grid_q, kChunkTokens, kAppendRingBytes, st>>>(p);
        } else {
            if (c->groups == kLayoutPerChannelK) k_quant_pack_frag<0, KVQ_APPEND_TOKENS_PER_THREAD, true><<<grid_q, kChunkTokens, kFragRingBytes, st>>>(p);
            else if (c->groups == 1) k_quant_pack_frag<0, KVQ_APPEND_TOKENS_PER_THREAD><<<grid_q, kChunkTokens, kFragRingBytes, st>>>(p);
            else k_quant_pack<0, 2, KVQ_APPEND_TOKENS_PER_THREAD><<<grid_q, kChunkTokens, kAppendRingBytes, st>>>(p);
        }
        c->launches += 2;
    }
    KVQ_CUDA(c, cudaGetLastError());
    c->cur[layer] ^= 1;
    int longest = 0;
    for (int b = 0; b < c->batch; ++b) {
        cur_lens[b] += host_lens ? host_lens[b] : n_new;
        longest = cur_lens[b] > longest ? cur_lens[b] : longest;
    }
    c->len[layer] = longest;
    c->ragged[layer] = c->ragged[layer] || call_ragged;
    return KVQ_OK;
}

// Shortest sequence of a layer.
int min_len(const kvq_ctx* c, int layer) {
    int m = c->lens[(size_t)layer * c->batch];
    for (int b = 1; b < c->batch; ++b) m = c->lens[(size_t)layer * c->batch + b] < m ? c->lens[(size_t)layer * c->batch + b] : m;
    return m;
}

// Number of working warps of a decode launch (the x axis is cut into that many equal parts).
// With an explicit split count every (sequence, query head) unit is cut into exactly that many
// parts.  Otherwise the count is taken from a small cost model.  A warp should own about eight
// tiles to pay for its set-up, which bounds the count for small problems.  For large ones the
// candidates are a persistent launch (as many warps as stay resident; warps whose share crosses a
// unit border work on two units and finish last, measured at about 0.9 of the ideal) and whole
// numbers of parts per unit (every warp does the same single piece of work; what counts is how
// full the last wave of CTAs is and how much of a warp's time goes into set-up).
constexpr int kMaxQueryRows = 8;       // query rows per sequence that one launch of kvq_attend_last serves

size_t max_partial_records(const kvq_ctx* c);

#ifndef KVQ_SMALL_MAX_TILES_PER_WARP
#define KVQ_SMALL_MAX_TILES_PER_WARP 40
#endif
// A launch plan: working warps, geometry, and (small geometry) parts per unit merged inside the CTA.
struct DecodePlan {
    uint32_t gw = 0;
    bool small = false;
    uint32_t cta_parts = 0;
};
// room: partial records the caller has scratch for (0: the handle's own).  gw == 0 if not even one part per unit
// fits.  Launches of few warps take the small geometry (8 warps per CTA, one CTA per SM, deep rings): with 1, 2, 4
// or 8 parts per unit the parts of a unit share a CTA and need no partial records at all.
DecodePlan choose_plan(kvq_ctx* c, int len, uint64_t units, uint64_t room = 0) {
    DecodePlan plan;
    if (room == 0) room = max_partial_records(c);
    auto fits = [&](uint64_t gw) { return units * (uint64_t)decode_pslots((uint32_t)units, (uint32_t)gw) <= room; };
    const uint64_t small_resident = (uint64_t)GeomSmall::kWarps * GeomSmall::kCtasPerSm * c->sm_count;
    auto cta_mergeable = [&](uint64_t parts) { return parts >= 1 && parts <= (uint64_t)GeomSmall::kWarps && GeomSmall::kWarps % parts == 0; };
    if (c->splits_override > 0) {
        const uint64_t parts = (uint64_t)c->splits_override, gw = units * parts;
        if (gw <= small_resident && cta_mergeable(parts)) {
            plan.gw = (uint32_t)gw;
            plan.small = true;
            plan.cta_parts = (uint32_t)parts;
            return plan;
        }
        if (GeomLarge::kWarps % parts == 0) {          // whole CTAs of the bandwidth geometry: no partial records either
            plan.gw = (uint32_t)gw;
            plan.cta_parts = (uint32_t)parts;
            return plan;
        }
        if (units * (parts + 1) <= room) {
            plan.gw = (uint32_t)gw;
            plan.small = gw <= small_resident;
            return plan;
        }
    }
    const uint64_t tiles_per_unit = (uint64_t)((len + kTileTokens - 1) / kTileTokens + (kNumPools - 1));
    const uint64_t tiles = units * tiles_per_unit;
    const uint64_t resident = (uint64_t)GeomLarge::kWarps * GeomLarge::kCtasPerSm * c->sm_count;
    if (!fits(units) && units > small_resident) return plan;
    if (tiles / 4 <= resident) {
        // A short cache is a chain of latencies, not a stream: a warp walks a tile in about kTileUs, parts merged
        // inside their CTA cost about kCtaMergeUs, parts merged through global partial records about kGlobalMergeUs
        // (measured on warps' own timestamps).  Take the cheaper of: 16 / 8 / 4 / 2 / 1 parts per unit in the small
        // geometry, or as many parts as leave a warp four tiles, merged globally.
        const double kTileUs = 0.3, kCtaMergeUs = 0.5, kGlobalMergeUs = 3.0;
        double best_cost = 1e30;
        for (uint64_t parts = GeomSmall::kWarps; parts >= 1; parts /= 2) {
            if (units * parts > small_resident) continue;
            const double cost = kTileUs * (double)((tiles_per_unit + parts - 1) / parts) + kCtaMergeUs;
            if (cost < best_cost) {
                best_cost = cost;
                plan.gw = (uint32_t)(units * parts);
                plan.small = true;
                plan.cta_parts = (uint32_t)parts;
            }
        }
        uint64_t cap = tiles / 4 < 1 ? 1 : tiles / 4;
        uint64_t gw = cap >= units ? cap / units * units : cap;
        if (gw > 0 && !fits(gw)) gw = fits(units) ? (room / units - 1) * units : 0;
        if (gw > 0) {
            const double cost = kTileUs * (double)((tiles + gw - 1) / gw) + kGlobalMergeUs;
            if (cost < best_cost) {
                plan.gw = (uint32_t)gw;
                plan.small = gw <= small_resident;
                plan.cta_parts = 0;
            }
        }
        return plan;
    }
    {
        const uint64_t parts = GeomSmall::kWarps;
        if (units * parts <= small_resident && tiles_per_unit / parts <= KVQ_SMALL_MAX_TILES_PER_WARP) {
            plan.gw = (uint32_t)(units * parts);       // a medium cache of few units: one CTA per unit, merged in shared memory
            plan.small = true;
            plan.cta_parts = (uint32_t)parts;
            return plan;
        }
    }
    if (!fits(units)) return plan;
    uint64_t cap = tiles / 8;
    if (cap <= resident) {
        uint64_t gw = cap >= units ? cap / units * units : cap;
        if (!fits(gw)) gw = (room / units - 1) * units;            // the most whole parts per unit that fit
        plan.gw = (uint32_t)gw;
        return plan;
    }
    // set-up, ring fill and the final reduction cost a warp about as much as fifteen tiles per part
    // (constants fitted to measured sweeps over the split count on four workload shapes)
    const double tiles_d = (double)tiles;
    uint64_t best = units;
    double best_score = 0.0;
    if (fits(resident)) {
        const double tpw_p = tiles_d / (double)resident;
        best = resident;
        best_score = 0.90 * tpw_p / (tpw_p + 25.0);               // some warps work on two parts
    }
    for (uint64_t s = 1; s <= (uint64_t)kMaxSplits && units * s <= cap && units * (s + 1) <= room; ++s) {
        const double fill = (double)(units * s) / (double)resident;
        const double waves = (double)(uint64_t)(fill + 0.999999);
        if (waves > 8.0) break;
        const double tpw = tiles_d / (double)(units * s);
        const double score = fill / waves * tpw / (tpw + 15.0);
        if (score > best_score + 1e-9) {
            best_score = score;
            best = units * s;
        }
    }
    plan.gw = (uint32_t)best;
    if (best % units == 0 && GeomLarge::kWarps % (best / units) == 0) plan.cta_parts = (uint32_t)(best / units);
    return plan;
}

// Partial records a handle may need: explicit splits up to kMaxSplits, or a persistent launch.
size_t max_partial_records(const kvq_ctx* c) {
    const size_t units = (size_t)c->batch * c->q_heads;
    const size_t resident = (size_t)GeomLarge::kWarps * GeomLarge::kCtasPerSm * c->sm_count;
    const size_t by_splits = units * (kMaxSplits + 1);
    const size_t by_residency = resident + 2 * units * kMaxQueryRows;
    return by_splits > by_residency ? by_splits : by_residency;
}

// Fill the launch parameters of a decode call and queue split + merge on `st`.
void fill_decode_params(kvq_ctx* c, int layer, const void* Q, void* O, float* part_o, float2* part_ml,
                        uint32_t* part_cnt, const DecodePlan& plan, DecodeParams& p) {
    p.store = c->store;
    p.counts = counts_of(c, c->cur[layer], layer);
    p.Q = static_cast<const __half*>(Q);
    p.O = static_cast<__half*>(O);
    p.part_o = part_o;
    p.part_ml = part_ml;
    p.part_cnt = part_cnt;
    p.part_s2 = c->part_s2;
    p.unit_var = c->unit_var;
    p.layer = layer;
    p.group = c->q_heads / c->kv_heads;
    p.tq = p.t_total = 1;
    p.t0 = 0;
    p.units = (uint32_t)c->batch * (uint32_t)c->q_heads;
    p.gw = plan.gw;
    p.pslots = decode_pslots(p.units, plan.gw);
    p.cta_parts = plan.cta_parts;
}

template <bool STATS, class Geo>
void launch_decode_geo(const kvq_ctx* c, const DecodeParams& p, cudaStream_t st) {
    const dim3 grid((p.gw + Geo::kWarps - 1) / Geo::kWarps);
    if (c->groups == 1) launch_overlapped(k_decode_attn<STATS, 1, Geo>, grid, Geo::kThreads, Geo::kSmemBytes, st, p);
    else if (c->groups == 2) launch_overlapped(k_decode_attn<STATS, 2, Geo>, grid, Geo::kThreads, Geo::kSmemBytes, st, p);
    else launch_overlapped(k_decode_attn<STATS, kLayoutPerChannelK, Geo>, grid, Geo::kThreads, Geo::kSmemBytes, st, p);
}
template <bool STATS>
void launch_decode(const kvq_ctx* c, const DecodePlan& plan, const DecodeParams& p, cudaStream_t st) {
    if (plan.small) launch_decode_geo<STATS, GeomSmall>(c, p, st);
    else launch_decode_geo<STATS, GeomLarge>(c, p, st);
}

int export_impl(kvq_ctx* c, int layer, int b0, int nb, int pos0, int n, uint8_t* bits, uint32_t* pool_slot,
                void* k_codes, void* v_codes, uint16_t* k_meta, uint16_t* v_meta, cudaStream_t st) {
    ExportParams p{};
    p.store = c->store;
    p.layer = layer;
    p.b0 = b0;
    p.nb = nb;
    p.pos0 = pos0;
    p.n = n;
    p.bits = bits;
    p.pool_slot = pool_slot;
    p.k_codes = static_cast<uint4*>(k_codes);
    p.v_codes = static_cast<uint4*>(v_codes);
    p.k_meta = k_meta;
    p.v_meta = v_meta;
    p.counts = counts_of(c, c->cur[layer], layer);
    k_export<<<dim3(n, nb), 128, 0, st>>>(p);
    c->launches += 1;
    KVQ_CUDA(c, cudaGetLastError());
    return KVQ_OK;
}

int create_impl(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch,
                uint64_t arena_bytes, int scale_groups, int mem_mode, void* workspace, uint64_t workspace_bytes,
                uint64_t* bytes_out);

}  // namespace

extern "C" {

int kvq_create(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch) {
    return kvq_create_arena(out, layers, q_heads, kv_heads, head_dim, max_ctx, batch, 0);
}

int kvq_create_arena(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch,
                     uint64_t arena_bytes) {
    return kvq_create_grouped(out, layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes, 1);
}

int kvq_create_grouped(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch,
                       uint64_t arena_bytes, int scale_groups) {
    if (scale_groups != 1 && scale_groups != 2) return KVQ_ERR_ARG;
    return create_impl(out, layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes, scale_groups, 0, nullptr, 0, nullptr);
}

int kvq_create_perchannel(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch,
                          uint64_t arena_bytes) {
    return create_impl(out, layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes, kLayoutPerChannelK, 0, nullptr, 0, nullptr);
}

int kvq_workspace_bytes(int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch, uint64_t arena_bytes,
                        int scale_groups, uint64_t* bytes_out) {
    if (!bytes_out || (scale_groups != 1 && scale_groups != 2)) return KVQ_ERR_ARG;
    kvq_ctx* none = nullptr;
    return create_impl(&none, layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes, scale_groups, 1, nullptr, 0,
                       bytes_out);
}

int kvq_create_in(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch,
                  uint64_t arena_bytes, int scale_groups, void* workspace, uint64_t workspace_bytes) {
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || (scale_groups != 1 && scale_groups != 2)) return KVQ_ERR_ARG;
    cudaPointerAttributes attr;                        // it has to be memory of a device, not of the host
    if (cudaPointerGetAttributes(&attr, workspace) != cudaSuccess) {
        cudaGetLastError();
        return KVQ_ERR_ARG;
    }
    if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged) return KVQ_ERR_ARG;
    return create_impl(out, layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes, scale_groups, 2, workspace,
                       workspace_bytes, nullptr);
}

}  // extern "C"

namespace {

int create_impl(kvq_ctx** out, int layers, int q_heads, int kv_heads, int head_dim, int max_ctx, int batch,
                uint64_t arena_bytes, int scale_groups, int mem_mode, void* workspace, uint64_t workspace_bytes,
                uint64_t* bytes_out) {
    if (!out) return KVQ_ERR_ARG;
    *out = nullptr;
    if (scale_groups != 1 && scale_groups != 2 && scale_groups != kLayoutPerChannelK) return KVQ_ERR_ARG;
    if (layers < 1 || q_heads < 1 || kv_heads < 1 || batch < 1 || max_ctx < 1) return KVQ_ERR_ARG;
    if (head_dim != kHeadDim || q_heads % kv_heads != 0) return KVQ_ERR_ARG;
    if (max_ctx > (1 << 30) - 1 || batch > 65535 || q_heads > 65535) return KVQ_ERR_ARG;
    kvq_ctx* c = new (std::nothrow) kvq_ctx();
    if (!c) return KVQ_ERR_NOMEM;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (e != cudaSuccess) {
        delete c;
        return KVQ_ERR_CUDA;
    }
    c->layers = layers;
    c->q_heads = q_heads;
    c->kv_heads = kv_heads;
    c->max_ctx = max_ctx;
    c->batch = batch;
    c->groups = scale_groups;
    c->mem_mode = mem_mode;
    c->slab = static_cast<uint8_t*>(workspace);
    c->slab_size = (size_t)workspace_bytes;
    c->len.assign(layers, 0);
    c->lens.assign((size_t)layers * batch, 0);
    c->ragged.assign(layers, 0);
    c->cur.assign(layers, 0);
    StoreView& s = c->store;
    s.layers = layers;
    s.batch = batch;
    s.kv_heads = kv_heads;
    s.q_heads = q_heads;
    s.max_ctx = max_ctx;
    s.groups = scale_groups;
    s.cap_tiles = (max_ctx + kTileTokens - 1) / kTileTokens;

    // block tables: one row per stream, class k at table_off[k]; one spare entry at the very end because
    // the decode kernel reads the entry after the block it is working on
    const size_t streams = (size_t)layers * batch * kv_heads;
    uint32_t row = 0;
    for (int k = 0; k < kNumPools; ++k) {
        s.table_off[k] = row;
        row += blocks_for(k, (uint32_t)max_ctx, scale_groups);
    }
    s.table_stride = row;
    const uint64_t worst_blocks = (uint64_t)streams * row + 1;           // every token in every class, plus block 0
    uint64_t blocks = arena_bytes ? arena_bytes / kBlockBytes : worst_blocks;
    if (blocks > worst_blocks) blocks = worst_blocks;
    if (blocks < 2 || blocks > 0xffffffffull) {
        delete c;
        return KVQ_ERR_ARG;
    }
    s.arena_blocks = (uint32_t)blocks;
    const size_t total = (size_t)blocks * kBlockBytes;
    const size_t table_bytes = sizeof(uint32_t) * (streams * row + 1);
    c->table_bytes = table_bytes;
    const size_t max_chunks = (size_t)(max_ctx + kChunkTokens - 1) / kChunkTokens;
    const size_t units = (size_t)batch * q_heads;
    bool ok = dev_alloc(c, &c->arena, total) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->table, table_bytes) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->arena_used, sizeof(uint32_t)) == cudaSuccess;
    ok = ok && dev_alloc(c, &s.index, sizeof(uint32_t) * (size_t)layers * batch * max_ctx) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->counts, sizeof(uint32_t) * 2 * (size_t)layers * batch * 4) == cudaSuccess;
    c->kres_bytes = scale_groups == kLayoutPerChannelK ? sizeof(__half) * kResidualStreamHalves * streams : 0;
    if (c->kres_bytes) ok = ok && dev_alloc(c, &c->kres, c->kres_bytes) == cudaSuccess;
    if (c->kres_bytes) ok = ok && dev_alloc(c, &c->kres_old, c->kres_bytes / layers) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->cls, (size_t)batch * max_ctx) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->hist, sizeof(uint4) * batch * max_chunks) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->chunk_arrivals, sizeof(uint32_t) * batch) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->ctrl, controller_smem(kMaxHidden)) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->step_cls, sizeof(uint32_t) * batch) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->part_o, sizeof(float) * max_partial_records(c) * kHeadDim) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->part_ml, sizeof(float2) * max_partial_records(c)) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->part_cnt, sizeof(uint32_t) * units * kMaxQueryRows) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->part_s2, sizeof(float) * max_partial_records(c)) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->unit_var, sizeof(float) * units) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->vis, sizeof(uint32_t) * 4 * (size_t)batch * kMaxQueryRows) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->d_lens, sizeof(int) * 3 * (size_t)batch * kvq_ctx::kLenSlots) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->flags, sizeof(uint32_t)) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->st_feats, sizeof(float) * 4 * batch) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->st_K, sizeof(__half) * (size_t)batch * kv_heads * kHeadDim) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->st_V, sizeof(__half) * (size_t)batch * kv_heads * kHeadDim) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->st_Q, sizeof(__half) * units * kHeadDim) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->st_O, sizeof(__half) * units * kHeadDim) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->st_bits, (size_t)batch) == cudaSuccess;
    ok = ok && dev_alloc(c, &c->st_export, (size_t)kv_heads * (2 * KVQ_EXPORT_ROW_BYTES + 8 * (scale_groups == 2 ? 2 : 1)) + 16) == cudaSuccess;
    if (ok && mem_mode == 1) {                         // only the size was asked for
        *bytes_out = c->slab_used;
        delete c;
        return KVQ_OK;
    }
    if (ok) {
        ok = cudaMallocHost(reinterpret_cast<void**>(&c->h_lens), sizeof(int) * 3 * (size_t)batch * kvq_ctx::kLenSlots) == cudaSuccess;
        for (int i = 0; ok && i < kvq_ctx::kLenSlots; ++i)
            ok = cudaEventCreateWithFlags(&c->len_ev[i], cudaEventDisableTiming) == cudaSuccess;
    }
    if (ok) {
        s.arena = c->arena;
        s.kres = c->kres;
        s.kres_old = c->kres_old;
        if (c->kres_bytes) ok = ok && cudaMemset(c->kres, 0, c->kres_bytes) == cudaSuccess;
        s.table = c->table;
        s.arena_used = c->arena_used;
        s.flags = c->flags;
        ok = cudaMemset(c->arena, 0, total) == cudaSuccess;
        ok = ok && cudaMemset(c->table, 0, table_bytes) == cudaSuccess;
        ok = ok && cudaMemset(c->arena_used, 0, sizeof(uint32_t)) == cudaSuccess;
        ok = ok && cudaMemset(s.index, 0, sizeof(uint32_t) * (size_t)layers * batch * max_ctx) == cudaSuccess;
        ok = ok && cudaMemset(c->counts, 0, sizeof(uint32_t) * 2 * (size_t)layers * batch * 4) == cudaSuccess;
        ok = ok && cudaMemset(c->flags, 0, sizeof(uint32_t)) == cudaSuccess;
        ok = ok && cudaMemset(c->chunk_arrivals, 0, sizeof(uint32_t) * batch) == cudaSuccess;
        ok = ok && cudaMemset(c->step_cls, 0, sizeof(uint32_t) * batch) == cudaSuccess;
        ok = ok && cudaMemset(c->part_cnt, 0, sizeof(uint32_t) * units * kMaxQueryRows) == cudaSuccess;
        // the controller block may exceed the default 48 KB of dynamic shared memory
        const int smem_max = (int)controller_smem(kMaxHidden);
        ok = ok && cudaFuncSetAttribute(k_select_bits, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(k_classify<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) == cudaSuccess;
        const int ring = (int)kAppendRingBytes;
        auto dyn_smem = [](auto kernel, int bytes) {
            return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
        };
        const int tsm = (int)(sizeof(float) * kControllerCtaSmemFloats);
        ok = ok && dyn_smem(k_append_token<true, 1>, tsm) && dyn_smem(k_append_token<true, 2>, tsm) && dyn_smem(k_append_token<true, kLayoutPerChannelK>, tsm);
        // The kernels of a decode step alternate; the attention kernel needs almost all of an SM's shared memory, so the
        // small ones ask for the same split of the L1 / shared-memory array and the SMs need not be reconfigured between them.
        auto max_shared = [](auto kernel) {
            return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared) == cudaSuccess;
        };
        ok = ok && max_shared(k_append_token<true, 1>) && max_shared(k_append_token<false, 1>) && max_shared(k_append_token<true, 2>) &&
             max_shared(k_append_token<false, 2>) && max_shared(k_append_token<true, kLayoutPerChannelK>) &&
             max_shared(k_append_token<false, kLayoutPerChannelK>) && max_shared(k_pack_window);
        const int fring = (int)kFragRingBytes;
        ok = ok && dyn_smem(k_quant_pack_frag<0, 1>, fring) && dyn_smem(k_quant_pack<0, 2>, ring);
        ok = ok && dyn_smem(k_quant_pack_frag<0, KVQ_APPEND_TOKENS_PER_THREAD>, fring) &&
             dyn_smem(k_quant_pack<0, 2, KVQ_APPEND_TOKENS_PER_THREAD>, ring);
        ok = ok && dyn_smem(k_quant_pack_frag<1>, fring) && dyn_smem(k_quant_pack<1, 2>, ring);
        ok = ok && dyn_smem(k_quant_pack_frag<2>, fring + smem_max) && dyn_smem(k_quant_pack<2, 2>, ring + smem_max);
        ok = ok && dyn_smem(k_quant_pack_frag<0, 1, true>, fring) && dyn_smem(k_quant_pack_frag<0, KVQ_APPEND_TOKENS_PER_THREAD, true>, fring) &&
             dyn_smem(k_quant_pack_frag<1, 1, true>, fring) && dyn_smem(k_quant_pack_frag<2, 1, true>, fring + smem_max);
        ok = ok && dyn_smem(k_decode_attn<false, 1, GeomLarge>, (int)GeomLarge::kSmemBytes) &&
             dyn_smem(k_decode_attn<false, 2, GeomLarge>, (int)GeomLarge::kSmemBytes);
        ok = ok && dyn_smem(k_decode_attn<true, 1, GeomLarge>, (int)GeomLarge::kSmemBytes) &&
             dyn_smem(k_decode_attn<true, 2, GeomLarge>, (int)GeomLarge::kSmemBytes);
        ok = ok && dyn_smem(k_decode_attn<false, 3, GeomLarge>, (int)GeomLarge::kSmemBytes) &&
             dyn_smem(k_decode_attn<true, 3, GeomLarge>, (int)GeomLarge::kSmemBytes) &&
             dyn_smem(k_decode_attn<false, 3, GeomSmall>, (int)GeomSmall::kSmemBytes) &&
             dyn_smem(k_decode_attn<true, 3, GeomSmall>, (int)GeomSmall::kSmemBytes);
        ok = ok && dyn_smem(k_decode_attn<false, 1, GeomSmall>, (int)GeomSmall::kSmemBytes) &&
             dyn_smem(k_decode_attn<false, 2, GeomSmall>, (int)GeomSmall::kSmemBytes);
        ok = ok && dyn_smem(k_decode_attn<true, 1, GeomSmall>, (int)GeomSmall::kSmemBytes) &&
             dyn_smem(k_decode_attn<true, 2, GeomSmall>, (int)GeomSmall::kSmemBytes);
        ok = ok && dyn_smem(k_decode_step<GeomSmall, 1, false>, (int)GeomSmall::kSmemBytes) && dyn_smem(k_decode_step<GeomLarge, 1, false>, (int)GeomLarge::kSmemBytes) &&
             dyn_smem(k_decode_step<GeomSmall, 2, false>, (int)GeomSmall::kSmemBytes) && dyn_smem(k_decode_step<GeomLarge, 2, false>, (int)GeomLarge::kSmemBytes);
        ok = ok && dyn_smem(k_decode_step<GeomSmall, 1, true>, (int)GeomSmall::kSmemBytes) && dyn_smem(k_decode_step<GeomLarge, 1, true>, (int)GeomLarge::kSmemBytes) &&
             dyn_smem(k_decode_step<GeomSmall, 2, true>, (int)GeomSmall::kSmemBytes) && dyn_smem(k_decode_step<GeomLarge, 2, true>, (int)GeomLarge::kSmemBytes);
        ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    }
    if (!ok) {
        cudaError_t err = cudaGetLastError();
        const bool too_small = c->slab_short;
        free_all(c);
        delete c;
        return err == cudaErrorMemoryAllocation || too_small ? KVQ_ERR_NOMEM : KVQ_ERR_CUDA;
    }
    *out = c;
    return KVQ_OK;
}

}  // namespace

extern "C" {

int kvq_destroy(kvq_ctx* c) {
    if (!c) return KVQ_OK;
    DeviceGuard guard(c->device);
    cudaDeviceSynchronize();
    free_all(c);
    delete c;
    return KVQ_OK;
}

int kvq_set_controller(kvq_ctx* c, int hidden, const float* W1, const float* b1, const float* W2, const float* b2,
                       const float* W3, const float* b3) {
    if (!c || hidden < 1 || hidden > kMaxHidden || !W1 || !b1 || !W2 || !b2 || !W3 || !b3) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    std::vector<float> blk;
    blk.reserve(controller_floats(hidden));
    blk.insert(blk.end(), W1, W1 + 4 * hidden);
    blk.insert(blk.end(), b1, b1 + hidden);
    blk.insert(blk.end(), W2, W2 + (size_t)hidden * hidden);
    blk.insert(blk.end(), b2, b2 + hidden);
    blk.insert(blk.end(), W3, W3 + 4 * hidden);
    blk.insert(blk.end(), b3, b3 + 4);
    KVQ_CUDA(c, cudaDeviceSynchronize());                          // earlier launches may still read the old block
    KVQ_CUDA(c, cudaMemcpy(c->ctrl, blk.data(), sizeof(float) * blk.size(), cudaMemcpyHostToDevice));
    c->hidden = hidden;
    return KVQ_OK;
}

int kvq_select_bits(kvq_ctx* c, const float* feats, int n, uint8_t* bits, float* logits_opt, void* stream) {
    if (!c || n < 0) return KVQ_ERR_ARG;
    if (n == 0) return KVQ_OK;
    if (!feats || !bits || !aligned16(feats) || (logits_opt && !aligned16(logits_opt))) return KVQ_ERR_ARG;
    if (c->hidden == 0) return KVQ_ERR_NO_CONTROLLER;
    DeviceGuard guard(c->device);
    k_select_bits<<<(n + 127) / 128, 128, controller_smem(c->hidden), static_cast<cudaStream_t>(stream)>>>(
        feats, n, c->ctrl, c->hidden, bits, logits_opt);
    c->launches += 1;
    KVQ_CUDA(c, cudaGetLastError());
    return KVQ_OK;
}

int kvq_append(kvq_ctx* c, int layer, const void* K, const void* V, const uint8_t* bits, int n_new, void* stream) {
    if (!c) return KVQ_ERR_ARG;
    return append_impl(c, layer, K, V, bits, nullptr, nullptr, n_new, nullptr, static_cast<cudaStream_t>(stream));
}

int kvq_append_fused(kvq_ctx* c, int layer, const void* K, const void* V, const float* feats, int n_new,
                     uint8_t* bits_out_opt, void* stream) {
    if (!c || (n_new > 0 && !feats)) return KVQ_ERR_ARG;
    return append_impl(c, layer, K, V, nullptr, feats, bits_out_opt, n_new, nullptr, static_cast<cudaStream_t>(stream));
}

int kvq_append_ragged(kvq_ctx* c, int layer, const void* K, const void* V, const uint8_t* bits, const float* feats,
                      int n_max, const int* host_lens, uint8_t* bits_out_opt, void* stream) {
    if (!c || !host_lens || (!bits && !feats) || (bits && feats)) return KVQ_ERR_ARG;
    return append_impl(c, layer, K, V, bits, feats, feats ? bits_out_opt : nullptr, n_max, host_lens,
                       static_cast<cudaStream_t>(stream));
}

int kvq_seq_lens(kvq_ctx* c, int layer, int* host_lens_out) {
    if (check_layer(c, layer) != KVQ_OK || !host_lens_out) return KVQ_ERR_ARG;
    for (int b = 0; b < c->batch; ++b) host_lens_out[b] = c->lens[(size_t)layer * c->batch + b];
    return KVQ_OK;
}

int kvq_decode_attn(kvq_ctx* c, int layer, const void* Q, void* O, void* stream) {
    TraceRange trace("kvq_decode_attn");
    if (check_layer(c, layer) != KVQ_OK || !Q || !O) return KVQ_ERR_ARG;
    if (c->len[layer] == 0) return KVQ_ERR_EMPTY;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DecodeParams p{};
    const DecodePlan plan = choose_plan(c, c->len[layer], (uint64_t)c->batch * c->q_heads);
    fill_decode_params(c, layer, Q, O, c->part_o, c->part_ml, c->part_cnt, plan, p);
    const bool rec = c->profiling && c->prof_calls < kProfMaxCalls;
    cudaEvent_t* ev = rec ? &c->prof_ev[(size_t)c->prof_calls * 2] : nullptr;
    if (rec) cudaEventRecord(ev[0], st);
    launch_decode<false>(c, plan, p, st);
    if (rec) {
        cudaEventRecord(ev[1], st);
        c->prof_calls += 1;
    }
    c->launches += 1;
    KVQ_CUDA(c, cudaGetLastError());
    return KVQ_OK;
}

int kvq_decode_step(kvq_ctx* c, int layer, const float* feats, const void* K, const void* V, const void* Q, void* O,
                    uint8_t* bits_out_opt, void* stream) {
    TraceRange trace("kvq_decode_step");
    if (check_layer(c, layer) != KVQ_OK || !feats || !K || !V || !Q || !O) return KVQ_ERR_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(feats)) return KVQ_ERR_ARG;
    if (c->hidden == 0) return KVQ_ERR_NO_CONTROLLER;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // One launch when keys have their scales per token (per-channel keys pack windows in a launch of their own);
    // otherwise the two calls, whose kernels overlap their launches.  With hidden width 32 the warp that adds the
    // token evaluates the controller itself; a wider one is evaluated by the storing CTAs, which then come first in
    // the grid and publish the class (tagged with a serial number that no earlier launch used).
    const uint64_t units = (uint64_t)c->batch * c->q_heads;
    DecodePlan plan;
    bool one_launch = c->groups != kLayoutPerChannelK;
    if (one_launch) {
        plan = choose_plan(c, c->len[layer], units);
        one_launch = plan.gw > 0;
    }
    if (!one_launch) {
        const int rc = append_impl(c, layer, K, V, nullptr, feats, bits_out_opt, 1, nullptr, st);
        return rc != KVQ_OK ? rc : kvq_decode_attn(c, layer, Q, O, stream);
    }
    int* cur_lens = &c->lens[(size_t)layer * c->batch];
    for (int b = 0; b < c->batch; ++b)
        if (cur_lens[b] + 1 > c->max_ctx) return KVQ_ERR_CAPACITY;
    DeviceGuard guard(c->device);
    AppendParams a{};
    a.store = c->store;
    a.K = static_cast<const __half*>(K);
    a.V = static_cast<const __half*>(V);
    a.feats = feats;
    a.ctrl = c->ctrl;
    a.hidden = c->hidden;
    a.bits_out = bits_out_opt;
    a.counts_in = counts_of(c, c->cur[layer], layer);
    a.counts_out = counts_of(c, c->cur[layer] ^ 1, layer);
    a.layer = layer;
    a.n_new = 1;
    a.pos0 = c->len[layer];
    a.tpt = 1;
    a.nchunks = 1;
    if (c->ragged[layer]) {                            // every sequence's own position travels with the call
        int *h_slot = nullptr, *d_slot = nullptr;
        const int slot = claim_len_slot(c, &h_slot, &d_slot);
        if (slot < 0) return slot;
        for (int b = 0; b < c->batch; ++b) {
            h_slot[b] = 1;
            h_slot[c->batch + b] = cur_lens[b];
        }
        KVQ_CUDA(c, cudaMemcpyAsync(d_slot, h_slot, sizeof(int) * 2 * c->batch, cudaMemcpyHostToDevice, st));
        KVQ_CUDA(c, cudaEventRecord(c->len_ev[slot], st));
        a.lens = d_slot;
        a.pos = d_slot + c->batch;
    }
    DecodeParams p{};
    fill_decode_params(c, layer, Q, O, c->part_o, c->part_ml, c->part_cnt, plan, p);      // the fills before the step
    const unsigned cta_warps = plan.small ? GeomSmall::kWarps : GeomLarge::kWarps;
    const unsigned attn_ctas = (p.gw + cta_warps - 1) / cta_warps;
    const unsigned items = (unsigned)c->batch * (unsigned)((c->kv_heads + 15) / 16);
    const bool w32 = c->hidden == 32;
    if (!w32) {
        if (c->step_serial >= 0x3fffffffu) {           // the tag is about to repeat: forget the old ones first
            KVQ_CUDA(c, cudaMemsetAsync(c->step_cls, 0, sizeof(uint32_t) * c->batch, st));
            c->step_serial = 0;
        }
        a.step_cls = c->step_cls;
        a.step_serial = ++c->step_serial;
        p.cta0 = items;                                // one storing CTA per (sequence, group of 16 KV heads), first in the grid
        p.step_cls = c->step_cls;
        p.step_serial = a.step_serial;
    }
    const dim3 grid(w32 ? attn_ctas + (items + cta_warps - 1) / cta_warps : items + attn_ctas);
    const bool rec = c->profiling && c->prof_calls < kProfMaxCalls;
    cudaEvent_t* ev = rec ? &c->prof_ev[(size_t)c->prof_calls * 2] : nullptr;
    if (rec) cudaEventRecord(ev[0], st);
    auto launch = [&](auto small_kernel, auto large_kernel) {
        if (plan.small) launch_overlapped(small_kernel, grid, GeomSmall::kThreads, GeomSmall::kSmemBytes, st, p, a);
        else launch_overlapped(large_kernel, grid, GeomLarge::kThreads, GeomLarge::kSmemBytes, st, p, a);
    };
    if (c->groups == 1 && w32) launch(k_decode_step<GeomSmall, 1, false>, k_decode_step<GeomLarge, 1, false>);
    else if (c->groups == 1) launch(k_decode_step<GeomSmall, 1, true>, k_decode_step<GeomLarge, 1, true>);
    else if (w32) launch(k_decode_step<GeomSmall, 2, false>, k_decode_step<GeomLarge, 2, false>);
    else launch(k_decode_step<GeomSmall, 2, true>, k_decode_step<GeomLarge, 2, true>);
    if (rec) {
        cudaEventRecord(ev[1], st);
        c->prof_calls += 1;
    }
    c->launches += 1;
    KVQ_CUDA(c, cudaGetLastError());
    c->cur[layer] ^= 1;
    for (int b = 0; b < c->batch; ++b) cur_lens[b] += 1;
    c->len[layer] += 1;
    return KVQ_OK;
}

int kvq_decode_attn_var(kvq_ctx* c, int layer, const void* Q, void* O, float* var_out, void* stream) {
    if (check_layer(c, layer) != KVQ_OK || !Q || !O || !var_out) return KVQ_ERR_ARG;
    if (c->len[layer] == 0) return KVQ_ERR_EMPTY;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DecodeParams p{};
    const DecodePlan plan = choose_plan(c, c->len[layer], (uint64_t)c->batch * c->q_heads);
    fill_decode_params(c, layer, Q, O, c->part_o, c->part_ml, c->part_cnt, plan, p);
    launch_decode<true>(c, plan, p, st);
    k_head_mean<<<c->batch, 32, 0, st>>>(c->unit_var, c->q_heads, var_out);
    c->launches += 2;
    KVQ_CUDA(c, cudaGetLastError());
    return KVQ_OK;
}

int kvq_token_features(const void* logits, int logits_are_fp32, int n, int vocab, const int32_t* token_ids,
                       const uint32_t* counts, uint64_t total_count, uint32_t observed_tokens,
                       const float* attn_var_opt, float* feats, void* stream) {
    if (n < 0 || vocab < 1) return KVQ_ERR_ARG;
    if (n == 0) return KVQ_OK;
    if (!logits || !token_ids || !counts || !feats || !aligned16(feats)) return KVQ_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float denom = (float)((double)total_count + (double)observed_tokens + 1.0);
    const bool vec = vocab % 8 == 0 && (reinterpret_cast<uintptr_t>(logits) & 31u) == 0;
    const int threads = n <= 1024 ? kFeatureThreadsFew : kFeatureThreads;
    if (logits_are_fp32)
        k_token_features<float><<<n, threads, 0, st>>>(static_cast<const float*>(logits), vocab, vec, token_ids,
                                                               counts, denom, attn_var_opt, feats);
    else
        k_token_features<__half><<<n, threads, 0, st>>>(static_cast<const __half*>(logits), vocab, vec, token_ids,
                                                                counts, denom, attn_var_opt, feats);
    return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA;
}

int kvq_attend_last(kvq_ctx* c, int layer, const void* Q, void* O, int n_queries, void* stream) {
    if (check_layer(c, layer) != KVQ_OK || !Q || !O || n_queries < 1) return KVQ_ERR_ARG;
    if (c->groups == kLayoutPerChannelK && n_queries > 1) return KVQ_ERR_ARG;   // an earlier row would see windows packed later
    if (c->len[layer] == 0) return KVQ_ERR_EMPTY;
    if (n_queries > min_len(c, layer)) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int* d_len = nullptr;
    if (c->ragged[layer]) {
        int *h_slot = nullptr, *d_slot = nullptr;
        const int slot = claim_len_slot(c, &h_slot, &d_slot);
        if (slot < 0) return slot;
        for (int b = 0; b < c->batch; ++b) h_slot[2 * c->batch + b] = c->lens[(size_t)layer * c->batch + b];
        KVQ_CUDA(c, cudaMemcpyAsync(d_slot + 2 * c->batch, h_slot + 2 * c->batch, sizeof(int) * c->batch, cudaMemcpyHostToDevice, st));
        KVQ_CUDA(c, cudaEventRecord(c->len_ev[slot], st));
        d_len = d_slot + 2 * c->batch;
    }
    for (int t0 = 0; t0 < n_queries; t0 += kMaxQueryRows) {
        const int tq = n_queries - t0 < kMaxQueryRows ? n_queries - t0 : kMaxQueryRows;
        k_visible_counts<<<c->batch, tq, 0, st>>>(c->store, counts_of(c, c->cur[layer], layer), layer, c->len[layer],
                                                  d_len, (uint32_t)n_queries, (uint32_t)t0, (uint32_t)tq, c->vis);
        const uint64_t units = (uint64_t)c->batch * tq * c->q_heads;
        DecodeParams p{};
        const DecodePlan plan = choose_plan(c, c->len[layer], units);
        fill_decode_params(c, layer, Q, O, c->part_o, c->part_ml, c->part_cnt, plan, p);
        p.counts = c->vis;
        p.tq = (uint32_t)tq;
        p.t_total = (uint32_t)n_queries;
        p.t0 = (uint32_t)t0;
        p.units = (uint32_t)units;
        p.pslots = decode_pslots(p.units, p.gw);
        launch_decode<false>(c, plan, p, st);
        c->launches += 2;
    }
    KVQ_CUDA(c, cudaGetLastError());
    return KVQ_OK;
}

// ---- decode attention with its partials in the library image (no allocation at all)
//
// The array below is a device symbol.  Its NAME in host code is only a host-side stand-in, not
// a device address; the address is fetched with cudaGetSymbolAddress once per device (that
// device current) and passed to the kernels like any other pointer.
#define KVQ_STATIC_MAX_DEVICES 64
// Layout: [records][64] partial rows, [records] (m, l) pairs, [records / 2] arrival counters (a unit
// has at least two partial slots).  The counters are zero when the library is loaded and every launch
// leaves them at zero again.
static __device__ __align__(256) float g_static_partials[(size_t)KVQ_STATIC_MAX_PARTIALS * (kHeadDim + 2) +
                                                         KVQ_STATIC_MAX_PARTIALS / 2];
static float* g_static_partials_addr[KVQ_STATIC_MAX_DEVICES];   // per device, nullptr until looked up
static std::mutex g_static_partials_lock;

int kvq_decode_attn_static(kvq_ctx* c, int layer, const void* Q, void* O, void* stream) {
    if (check_layer(c, layer) != KVQ_OK || !Q || !O) return KVQ_ERR_ARG;
    if (c->len[layer] == 0) return KVQ_ERR_EMPTY;
    if (c->device < 0 || c->device >= KVQ_STATIC_MAX_DEVICES) return KVQ_ERR_ARG;
    const uint64_t units = (uint64_t)c->batch * c->q_heads;
    // an explicit split count is taken as given; the automatic plan is the best one that fits the array
    if (c->splits_override > 0 && units * (uint64_t)(c->splits_override + 1) > (uint64_t)KVQ_STATIC_MAX_PARTIALS) return KVQ_ERR_TOO_LARGE;
    const DecodePlan plan = choose_plan(c, c->len[layer], units, KVQ_STATIC_MAX_PARTIALS);
    if (plan.gw == 0) return KVQ_ERR_TOO_LARGE;
    DeviceGuard guard(c->device);
    float* base = nullptr;
    {
        std::lock_guard<std::mutex> hold(g_static_partials_lock);
        if (!g_static_partials_addr[c->device]) {
            void* p = nullptr;
            KVQ_CUDA(c, cudaGetSymbolAddress(&p, g_static_partials));
            g_static_partials_addr[c->device] = static_cast<float*>(p);
        }
        base = g_static_partials_addr[c->device];
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DecodeParams p{};
    fill_decode_params(c, layer, Q, O, base, reinterpret_cast<float2*>(base + (size_t)KVQ_STATIC_MAX_PARTIALS * kHeadDim),
                       reinterpret_cast<uint32_t*>(base + (size_t)KVQ_STATIC_MAX_PARTIALS * (kHeadDim + 2)), plan, p);
    launch_decode<false>(c, plan, p, st);
    c->launches += 1;
    KVQ_CUDA(c, cudaGetLastError());
    return KVQ_OK;
}

int kvq_decode_step_host(kvq_ctx* c, int layer, const float* feats, const void* K, const void* V, const void* Q,
                         void* O, uint8_t* bits_out_opt, void* stream) {
    TraceRange trace("kvq_decode_step_host");
    if (check_layer(c, layer) != KVQ_OK || !feats || !K || !V || !Q || !O) return KVQ_ERR_ARG;
    if (c->hidden == 0) return KVQ_ERR_NO_CONTROLLER;
    if (c->len[layer] + 1 > c->max_ctx) return KVQ_ERR_CAPACITY;
    DeviceGuard guard(c->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t kv_bytes = sizeof(__half) * (size_t)c->batch * c->kv_heads * kHeadDim;
    const size_t q_bytes = sizeof(__half) * (size_t)c->batch * c->q_heads * kHeadDim;
    // Page-locked host buffers are reachable from the device under unified addressing: the kernels then read
    // the step's inputs and write its result across the bus themselves, which saves five copy launches.  Any
    // buffer that is pageable (or misaligned for the kernels' 16-byte loads) sends the call through the
    // staging buffers instead.
    const void *d_feats = device_view(feats), *d_K = device_view(K), *d_V = device_view(V), *d_Q = device_view(Q);
    void* d_O = const_cast<void*>(device_view(O));
    const bool direct = d_feats && d_K && d_V && d_Q && d_O;
    if (!direct) {
        KVQ_CUDA(c, cudaMemcpyAsync(c->st_feats, feats, sizeof(float) * 4 * c->batch, cudaMemcpyHostToDevice, st));
        KVQ_CUDA(c, cudaMemcpyAsync(c->st_K, K, kv_bytes, cudaMemcpyHostToDevice, st));
        KVQ_CUDA(c, cudaMemcpyAsync(c->st_V, V, kv_bytes, cudaMemcpyHostToDevice, st));
        KVQ_CUDA(c, cudaMemcpyAsync(c->st_Q, Q, q_bytes, cudaMemcpyHostToDevice, st));
        d_feats = c->st_feats;
        d_K = c->st_K;
        d_V = c->st_V;
        d_Q = c->st_Q;
        d_O = c->st_O;
    }
    const int rc = kvq_decode_step(c, layer, static_cast<const float*>(d_feats), d_K, d_V, d_Q, d_O, c->st_bits, stream);
    if (rc != KVQ_OK) return rc;
    if (!direct) KVQ_CUDA(c, cudaMemcpyAsync(O, c->st_O, q_bytes, cudaMemcpyDeviceToHost, st));
    if (bits_out_opt) KVQ_CUDA(c, cudaMemcpyAsync(bits_out_opt, c->st_bits, c->batch, cudaMemcpyDeviceToHost, st));
    KVQ_CUDA(c, cudaStreamSynchronize(st));
    return KVQ_OK;
}

int kvq_reset(kvq_ctx* c, void* stream) {
    if (!c) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    KVQ_CUDA(c, cudaMemsetAsync(c->counts, 0, sizeof(uint32_t) * 2 * (size_t)c->layers * c->batch * 4,
                                static_cast<cudaStream_t>(stream)));
    KVQ_CUDA(c, cudaMemsetAsync(c->arena_used, 0, sizeof(uint32_t), static_cast<cudaStream_t>(stream)));
    std::fill(c->lens.begin(), c->lens.end(), 0);
    for (int l = 0; l < c->layers; ++l) {
        c->len[l] = 0;
        c->cur[l] = 0;
        c->ragged[l] = 0;
    }
    return KVQ_OK;
}

int kvq_seq_len(kvq_ctx* c, int layer, int* host_len_out) {
    if (check_layer(c, layer) != KVQ_OK || !host_len_out) return KVQ_ERR_ARG;
    *host_len_out = c->len[layer];
    return KVQ_OK;
}

int kvq_set_append_chunk(kvq_ctx* c, int chunk_tokens) {
    if (!c) return KVQ_ERR_ARG;
    if (chunk_tokens != 0 && chunk_tokens != kChunkTokens && chunk_tokens != kChunkTokens * KVQ_APPEND_TOKENS_PER_THREAD)
        return KVQ_ERR_ARG;
    c->chunk_override = chunk_tokens / kChunkTokens;
    return KVQ_OK;
}

int kvq_set_splits(kvq_ctx* c, int splits) {
    if (!c || splits < 0 || splits > kMaxSplits) return KVQ_ERR_ARG;
    c->splits_override = splits;
    return KVQ_OK;
}

int kvq_export_range(kvq_ctx* c, int layer, int pos0, int n, uint8_t* bits, uint32_t* pool_slot, void* k_codes,
                     void* v_codes, uint16_t* k_meta, uint16_t* v_meta, void* stream) {
    if (check_layer(c, layer) != KVQ_OK || pos0 < 0 || n < 0 || pos0 + n > min_len(c, layer)) return KVQ_ERR_ARG;
    if (n == 0) return KVQ_OK;
    if ((k_codes && !aligned16(k_codes)) || (v_codes && !aligned16(v_codes))) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    return export_impl(c, layer, 0, c->batch, pos0, n, bits, pool_slot, k_codes, v_codes, k_meta, v_meta,
                       static_cast<cudaStream_t>(stream));
}

int kvq_export_token(kvq_ctx* c, int layer, int b, int pos, uint8_t* bits, uint32_t* pool_slot, void* k_codes,
                     void* v_codes, uint16_t* k_meta, uint16_t* v_meta) {
    if (check_layer(c, layer) != KVQ_OK || b < 0 || b >= c->batch || pos < 0 ||
        pos >= c->lens[(size_t)layer * c->batch + (b < 0 || b >= c->batch ? 0 : b)])
        return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    const size_t row = (size_t)c->kv_heads * KVQ_EXPORT_ROW_BYTES, meta = (size_t)c->kv_heads * 4 * (c->groups == 2 ? 2 : 1);
    uint8_t* d_k = c->st_export;
    uint8_t* d_v = d_k + row;
    uint8_t* d_km = d_v + row;
    uint8_t* d_vm = d_km + meta;
    uint8_t* d_ps = d_vm + meta;           // 4 bytes pool_slot, then 1 byte bits
    KVQ_CUDA(c, cudaDeviceSynchronize());
    int rc = export_impl(c, layer, b, 1, pos, 1, d_ps + 4, reinterpret_cast<uint32_t*>(d_ps), d_k, d_v,
                         reinterpret_cast<uint16_t*>(d_km), reinterpret_cast<uint16_t*>(d_vm), nullptr);
    if (rc != KVQ_OK) return rc;
    if (k_codes) KVQ_CUDA(c, cudaMemcpy(k_codes, d_k, row, cudaMemcpyDeviceToHost));
    if (v_codes) KVQ_CUDA(c, cudaMemcpy(v_codes, d_v, row, cudaMemcpyDeviceToHost));
    if (k_meta) KVQ_CUDA(c, cudaMemcpy(k_meta, d_km, meta, cudaMemcpyDeviceToHost));
    if (v_meta) KVQ_CUDA(c, cudaMemcpy(v_meta, d_vm, meta, cudaMemcpyDeviceToHost));
    if (pool_slot) KVQ_CUDA(c, cudaMemcpy(pool_slot, d_ps, 4, cudaMemcpyDeviceToHost));
    if (bits) KVQ_CUDA(c, cudaMemcpy(bits, d_ps + 4, 1, cudaMemcpyDeviceToHost));
    KVQ_CUDA(c, cudaDeviceSynchronize());
    return KVQ_OK;
}

int kvq_export_k_channels(kvq_ctx* c, int layer, int b, int kv_head, int bits, int window, uint16_t* host_meta) {
    if (check_layer(c, layer) != KVQ_OK || !host_meta || c->groups != kLayoutPerChannelK) return KVQ_ERR_ARG;
    const int cls = bits == 2 ? 0 : bits == 4 ? 1 : bits == 8 ? 2 : -1;
    if (cls < 0 || b < 0 || b >= c->batch || kv_head < 0 || kv_head >= c->kv_heads || window < 0) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    KVQ_CUDA(c, cudaDeviceSynchronize());
    uint32_t fill[4];
    KVQ_CUDA(c, cudaMemcpy(fill, counts_of(c, c->cur[layer], layer) + (size_t)b * 4, sizeof(fill), cudaMemcpyDeviceToHost));
    if ((uint64_t)(window + 1) * kTileTokens > fill[cls]) return KVQ_ERR_ARG;           // the window is not complete
    const uint32_t bt = block_tiles(cls, kLayoutPerChannelK);
    uint32_t id = 0;
    KVQ_CUDA(c, cudaMemcpy(&id, stream_table(c->store, cls, layer, b, kv_head) + (uint32_t)window / bt, sizeof(id), cudaMemcpyDeviceToHost));
    const uint8_t* rec = c->arena + (size_t)id * kBlockBytes + (size_t)((uint32_t)window % bt) * pool_rec_bytes(cls, kLayoutPerChannelK);
    KVQ_CUDA(c, cudaMemcpy(host_meta, rec + chan_meta_offset(cls, 0), 4 * kHeadDim, cudaMemcpyDeviceToHost));
    return KVQ_OK;
}

int kvq_stats(kvq_ctx* c, int layer, uint32_t* host_counts, uint64_t* resident_bytes, double* expected_bits) {
    if (check_layer(c, layer) != KVQ_OK) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    std::vector<uint32_t> cnt((size_t)c->batch * 4);
    KVQ_CUDA(c, cudaDeviceSynchronize());
    KVQ_CUDA(c, cudaMemcpy(cnt.data(), counts_of(c, c->cur[layer], layer), sizeof(uint32_t) * cnt.size(),
                           cudaMemcpyDeviceToHost));
    uint64_t bytes = 0, tokens = 0, bit_sum = 0;
    for (int b = 0; b < c->batch; ++b)
        for (int k = 0; k < kNumPools; ++k) {
            const uint64_t n = cnt[(size_t)b * 4 + k];
            bytes += n * (uint64_t)c->kv_heads * pool_row_bytes(k, c->groups);
            tokens += n;
            bit_sum += n * (uint64_t)pool_bits(k);
        }
    if (host_counts) memcpy(host_counts, cnt.data(), sizeof(uint32_t) * cnt.size());
    if (resident_bytes) *resident_bytes = bytes;
    if (expected_bits) *expected_bits = tokens ? (double)bit_sum / (double)tokens : 0.0;
    return KVQ_OK;
}

int kvq_arena_usage(kvq_ctx* c, uint64_t* blocks_in_use, uint64_t* blocks_total, uint64_t* block_bytes) {
    if (!c) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    uint32_t used = 0;
    KVQ_CUDA(c, cudaDeviceSynchronize());
    KVQ_CUDA(c, cudaMemcpy(&used, c->arena_used, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    const uint64_t total = c->store.arena_blocks - 1;                     // block 0 is never handed out
    if (blocks_in_use) *blocks_in_use = used < total ? used : total;
    if (blocks_total) *blocks_total = total;
    if (block_bytes) *block_bytes = kBlockBytes;
    return KVQ_OK;
}

// ---- snapshots: [StateHeader][len][lens][ragged][cur][arena blocks 0 .. used][table][index][counts]
namespace {
struct StateHeader {
    uint32_t magic, version;
    int32_t layers, q_heads, kv_heads, max_ctx, batch, groups;
    uint32_t arena_blocks, blocks_used;
    uint64_t table_bytes, index_bytes, counts_bytes, total_bytes;
};
constexpr uint32_t kStateMagic = 0x5156564bu, kStateVersion = 1;   // "KVVQ"

int state_header(kvq_ctx* c, StateHeader& h) {
    uint32_t used = 0;
    KVQ_CUDA(c, cudaDeviceSynchronize());
    KVQ_CUDA(c, cudaMemcpy(&used, c->arena_used, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    if (used > c->store.arena_blocks - 1) used = c->store.arena_blocks - 1;       // an exhausted arena counts past its end
    h = StateHeader{};
    h.magic = kStateMagic;
    h.version = kStateVersion;
    h.layers = c->layers;
    h.q_heads = c->q_heads;
    h.kv_heads = c->kv_heads;
    h.max_ctx = c->max_ctx;
    h.batch = c->batch;
    h.groups = c->groups;
    h.arena_blocks = c->store.arena_blocks;
    h.blocks_used = used;
    h.table_bytes = c->table_bytes;
    h.index_bytes = sizeof(uint32_t) * (uint64_t)c->layers * c->batch * c->max_ctx;
    h.counts_bytes = sizeof(uint32_t) * 2 * (uint64_t)c->layers * c->batch * 4;
    const uint64_t host_ints = (uint64_t)c->layers * 3 + (uint64_t)c->layers * c->batch;
    h.total_bytes = sizeof(StateHeader) + sizeof(int32_t) * host_ints + (uint64_t)(used + 1) * kBlockBytes + h.table_bytes +
                    h.index_bytes + h.counts_bytes + c->kres_bytes;
    return KVQ_OK;
}
}  // namespace

int kvq_state_bytes(kvq_ctx* c, uint64_t* bytes_out) {
    if (!c || !bytes_out) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    StateHeader h;
    const int rc = state_header(c, h);
    if (rc == KVQ_OK) *bytes_out = h.total_bytes;
    return rc;
}

int kvq_save_state(kvq_ctx* c, void* host_buf, uint64_t host_bytes) {
    if (!c || !host_buf) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    StateHeader h;
    int rc = state_header(c, h);
    if (rc != KVQ_OK) return rc;
    if (host_bytes < h.total_bytes) return KVQ_ERR_ARG;
    uint8_t* out = static_cast<uint8_t*>(host_buf);
    std::memcpy(out, &h, sizeof(h));
    out += sizeof(h);
    auto put_ints = [&](auto&& get, size_t n) {
        for (size_t i = 0; i < n; ++i) {
            const int32_t v = (int32_t)get(i);
            std::memcpy(out, &v, sizeof(v));
            out += sizeof(v);
        }
    };
    put_ints([&](size_t i) { return c->len[i]; }, c->len.size());
    put_ints([&](size_t i) { return c->lens[i]; }, c->lens.size());
    put_ints([&](size_t i) { return (int)c->ragged[i]; }, c->ragged.size());
    put_ints([&](size_t i) { return c->cur[i]; }, c->cur.size());
    const size_t arena_bytes = (size_t)(h.blocks_used + 1) * kBlockBytes;
    KVQ_CUDA(c, cudaMemcpy(out, c->arena, arena_bytes, cudaMemcpyDeviceToHost));
    out += arena_bytes;
    KVQ_CUDA(c, cudaMemcpy(out, c->table, h.table_bytes, cudaMemcpyDeviceToHost));
    out += h.table_bytes;
    KVQ_CUDA(c, cudaMemcpy(out, c->store.index, h.index_bytes, cudaMemcpyDeviceToHost));
    out += h.index_bytes;
    KVQ_CUDA(c, cudaMemcpy(out, c->counts, h.counts_bytes, cudaMemcpyDeviceToHost));
    out += h.counts_bytes;
    if (c->kres_bytes) KVQ_CUDA(c, cudaMemcpy(out, c->kres, c->kres_bytes, cudaMemcpyDeviceToHost));
    return KVQ_OK;
}

int kvq_load_state(kvq_ctx* c, const void* host_buf, uint64_t host_bytes) {
    if (!c || !host_buf || host_bytes < sizeof(StateHeader)) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    StateHeader h;
    std::memcpy(&h, host_buf, sizeof(h));
    if (h.magic != kStateMagic || h.version != kStateVersion || host_bytes < h.total_bytes) return KVQ_ERR_ARG;
    if (h.layers != c->layers || h.q_heads != c->q_heads || h.kv_heads != c->kv_heads || h.max_ctx != c->max_ctx ||
        h.batch != c->batch || h.groups != c->groups)
        return KVQ_ERR_ARG;
    // the arena may differ in size as long as the snapshot's blocks fit (block ids are positions in the arena);
    // every other size in the header has to be this handle's own, whatever the blob claims
    if ((uint64_t)h.blocks_used + 1 > (uint64_t)c->store.arena_blocks || h.table_bytes != c->table_bytes) return KVQ_ERR_ARG;
    if (h.index_bytes != sizeof(uint32_t) * (uint64_t)c->layers * c->batch * c->max_ctx ||
        h.counts_bytes != sizeof(uint32_t) * 2 * (uint64_t)c->layers * c->batch * 4)
        return KVQ_ERR_ARG;
    const uint64_t host_ints = (uint64_t)c->layers * 3 + (uint64_t)c->layers * c->batch;
    if (h.total_bytes != sizeof(StateHeader) + sizeof(int32_t) * host_ints + ((uint64_t)h.blocks_used + 1) * kBlockBytes +
                             h.table_bytes + h.index_bytes + h.counts_bytes + c->kres_bytes)
        return KVQ_ERR_ARG;
    const uint8_t* in = static_cast<const uint8_t*>(host_buf) + sizeof(h);
    auto get_int = [&]() {
        int32_t v;
        std::memcpy(&v, in, sizeof(v));
        in += sizeof(v);
        return v;
    };
    // Nothing the kernels use as an address may point outside the handle's buffers: check lengths, fills,
    // block ids and index words on the host before anything is replaced.
    std::vector<uint32_t> clean_table;
    {
        const uint8_t* q = in;
        auto peek = [&]() {
            int32_t v;
            std::memcpy(&v, q, sizeof(v));
            q += sizeof(v);
            return v;
        };
        std::vector<int32_t> len(c->layers), lens((size_t)c->layers * c->batch), cur(c->layers);
        for (auto& v : len) v = peek();
        for (auto& v : lens) v = peek();
        for (int l = 0; l < c->layers; ++l) peek();    // ragged flags
        for (auto& v : cur) v = peek() & 1;
        for (int l = 0; l < c->layers; ++l) {
            int longest = 0;
            for (int b = 0; b < c->batch; ++b) {
                const int n = lens[(size_t)l * c->batch + b];
                if (n < 0 || n > c->max_ctx) return KVQ_ERR_ARG;
                longest = n > longest ? n : longest;
            }
            if (len[l] != longest) return KVQ_ERR_ARG;
        }
        const uint8_t* arena_blob = q;
        const uint8_t* table = arena_blob + (size_t)(h.blocks_used + 1) * kBlockBytes;
        const uint8_t* index = table + h.table_bytes;
        for (size_t i = 0; i < h.index_bytes / sizeof(uint32_t); ++i) {
            uint32_t w;
            std::memcpy(&w, index + i * sizeof(uint32_t), sizeof(w));
            if ((w & 0x3fffffffu) >= (uint32_t)c->max_ctx) return KVQ_ERR_ARG;
        }
        const uint8_t* counts = index + h.index_bytes;
        for (int which = 0; which < 2; ++which)
            for (int l = 0; l < c->layers; ++l)
                for (int b = 0; b < c->batch; ++b) {
                    uint32_t f[4];
                    std::memcpy(f, counts + sizeof(uint32_t) * 4 * (((size_t)which * c->layers + l) * c->batch + b), sizeof(f));
                    const uint64_t sum = (uint64_t)f[0] + f[1] + f[2] + f[3];
                    if (which == cur[l] ? sum != (uint64_t)lens[(size_t)l * c->batch + b] : sum > (uint64_t)c->max_ctx) return KVQ_ERR_ARG;
                }
        // Block tables: the entries that the current fills reach must name blocks of the snapshot; the rest
        // (left over from before a reset) are not used and are cleared.
        clean_table.assign(h.table_bytes / sizeof(uint32_t), 0u);
        for (int l = 0; l < c->layers; ++l)
            for (int b = 0; b < c->batch; ++b) {
                uint32_t f[4];
                std::memcpy(f, counts + sizeof(uint32_t) * 4 * (((size_t)cur[l] * c->layers + l) * c->batch + b), sizeof(f));
                for (int hh = 0; hh < c->kv_heads; ++hh)
                    for (int k = 0; k < kNumPools; ++k) {
                        const size_t row = (((size_t)l * c->batch + b) * c->kv_heads + hh) * c->store.table_stride + c->store.table_off[k];
                        const uint32_t reached = blocks_for(k, f[k], c->groups);
                        for (uint32_t e = 0; e < reached; ++e) {
                            uint32_t id;
                            std::memcpy(&id, table + sizeof(uint32_t) * (row + e), sizeof(id));
                            if (id > h.blocks_used) return KVQ_ERR_ARG;
                            clean_table[row + e] = id;
                        }
                    }
            }
    }
    KVQ_CUDA(c, cudaDeviceSynchronize());
    for (auto& v : c->len) v = get_int();
    for (auto& v : c->lens) v = get_int();
    for (auto& v : c->ragged) v = (char)get_int();
    for (auto& v : c->cur) v = get_int() & 1;
    const size_t arena_bytes = (size_t)(h.blocks_used + 1) * kBlockBytes;
    KVQ_CUDA(c, cudaMemcpy(c->arena, in, arena_bytes, cudaMemcpyHostToDevice));
    in += arena_bytes;
    KVQ_CUDA(c, cudaMemcpy(c->table, clean_table.data(), h.table_bytes, cudaMemcpyHostToDevice));
    in += h.table_bytes;
    KVQ_CUDA(c, cudaMemcpy(c->store.index, in, h.index_bytes, cudaMemcpyHostToDevice));
    in += h.index_bytes;
    KVQ_CUDA(c, cudaMemcpy(c->counts, in, h.counts_bytes, cudaMemcpyHostToDevice));
    in += h.counts_bytes;
    if (c->kres_bytes) KVQ_CUDA(c, cudaMemcpy(c->kres, in, c->kres_bytes, cudaMemcpyHostToDevice));
    KVQ_CUDA(c, cudaMemcpy(c->arena_used, &h.blocks_used, sizeof(uint32_t), cudaMemcpyHostToDevice));
    KVQ_CUDA(c, cudaMemset(c->flags, 0, sizeof(uint32_t)));
    return KVQ_OK;
}

int kvq_set_profiling(kvq_ctx* c, int on) {
    if (!c) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    if (on && c->prof_ev.empty()) {
        c->prof_ev.resize((size_t)kProfMaxCalls * 2);
        for (size_t i = 0; i < c->prof_ev.size(); ++i) {
            cudaError_t e = cudaEventCreate(&c->prof_ev[i]);
            if (e != cudaSuccess) {
                for (size_t j = 0; j < i; ++j) cudaEventDestroy(c->prof_ev[j]);
                c->prof_ev.clear();
                c->last_err = e;
                return KVQ_ERR_CUDA;
            }
        }
    }
    c->profiling = on != 0;
    return KVQ_OK;
}

int kvq_profile_read(kvq_ctx* c, double* attn_ms_total, int* calls) {
    if (!c) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    KVQ_CUDA(c, cudaDeviceSynchronize());
    double ms = 0.0;
    for (int i = 0; i < c->prof_calls; ++i) {
        float a = 0.f;
        KVQ_CUDA(c, cudaEventElapsedTime(&a, c->prof_ev[(size_t)i * 2], c->prof_ev[(size_t)i * 2 + 1]));
        ms += a;
    }
    if (attn_ms_total) *attn_ms_total = ms;
    if (calls) *calls = c->prof_calls;
    c->prof_calls = 0;
    return KVQ_OK;
}

int kvq_device_status(kvq_ctx* c, uint32_t* host_flags_out) {
    if (!c || !host_flags_out) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    KVQ_CUDA(c, cudaDeviceSynchronize());
    KVQ_CUDA(c, cudaMemcpy(host_flags_out, c->flags, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    KVQ_CUDA(c, cudaMemset(c->flags, 0, sizeof(uint32_t)));
    if (*host_flags_out & KVQ_FLAG_WAIT_TIMEOUT) {     // belt and braces: the kernel already left them at zero
        const int rc = kvq_recover(c);
        if (rc != KVQ_OK) return rc;
    }
    return *host_flags_out ? KVQ_ERR_DEVICE_FLAG : KVQ_OK;
}

int kvq_recover(kvq_ctx* c) {
    if (!c) return KVQ_ERR_ARG;
    DeviceGuard guard(c->device);
    KVQ_CUDA(c, cudaDeviceSynchronize());
    KVQ_CUDA(c, cudaMemset(c->part_cnt, 0, sizeof(uint32_t) * (size_t)c->batch * c->q_heads * kMaxQueryRows));
    KVQ_CUDA(c, cudaMemset(c->flags, 0, sizeof(uint32_t)));
    float* base = nullptr;
    if (c->device >= 0 && c->device < KVQ_STATIC_MAX_DEVICES) {
        std::lock_guard<std::mutex> hold(g_static_partials_lock);
        base = g_static_partials_addr[c->device];      // only if kvq_decode_attn_static ever ran on this device
    }
    if (base)
        KVQ_CUDA(c, cudaMemset(base + (size_t)KVQ_STATIC_MAX_PARTIALS * (kHeadDim + 2), 0,
                               sizeof(uint32_t) * (KVQ_STATIC_MAX_PARTIALS / 2)));
    return KVQ_OK;
}

int kvq_device_bytes(kvq_ctx* c, uint64_t* host_bytes_out) {
    if (!c || !host_bytes_out) return KVQ_ERR_ARG;
    *host_bytes_out = c->device_bytes;
    return KVQ_OK;
}

int kvq_launch_count(kvq_ctx* c, uint64_t* host_count_out) {
    if (!c || !host_count_out) return KVQ_ERR_ARG;
    *host_count_out = c->launches;
    return KVQ_OK;
}

int kvq_last_cuda_error(kvq_ctx* c) { return c ? (int)c->last_err : 0; }

const char* kvq_strerror(int code) {
    switch (code) {
    case KVQ_OK: return "ok";
    case KVQ_ERR_ARG: return "invalid argument";
    case KVQ_ERR_CAPACITY: return "append would exceed max_ctx";
    case KVQ_ERR_NO_CONTROLLER: return "controller weights not set";
    case KVQ_ERR_CUDA: return "CUDA call failed";
    case KVQ_ERR_EMPTY: return "layer holds no token";
    case KVQ_ERR_DEVICE_FLAG: return "a kernel recorded a problem";
    case KVQ_ERR_NOMEM: return "out of memory";
    case KVQ_ERR_TOO_LARGE: return "batch * q_heads * (parts + 1) exceeds the static scratch of kvq_decode_attn_static";
    default: return "unknown error";
    }
}

}  // extern "C"
