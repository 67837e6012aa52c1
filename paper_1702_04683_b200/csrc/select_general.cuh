// SELECT_GRAD (Algorithm 1), general route: exact radix select on magnitude keys followed by an
// index-ordered compaction.  Works for any data (any number of ties, any tensor size) and is the
// route every (worker, tensor) selection can always fall back to.
//
// Per selected (worker, tensor) "instance":
//   pass 0..2  histogram of key bits [30:20], [19:10], [9:0] over the entries that match the
//              bits decided so far; the block that finishes an instance last walks the histogram
//              from the top and fixes the next digit of the threshold key T;
//   pass 3     per chunk, count entries with key > T and key == T; the last block turns the
//              counts into exclusive prefixes over the chunks of the instance;
//   pass 4     per chunk, write the kept entries in index order: every key > T, and the r
//              lowest-index entries with key == T (r = k - #{key > T}).
// Work items are (instance, chunk) pairs taken from a device-built list, so the same kernels
// serve "all instances" and "only the instances another route gave up on".
#pragma once

#include <cstddef>

#include "common.cuh"

namespace adacomp {

constexpr int kThreads = 256;
constexpr uint32_t kElemsPerIter = kThreads * 4;             // one float4 per thread
constexpr uint32_t kItersPerChunk = 128;
constexpr uint32_t kChunkElems = kElemsPerIter * kItersPerChunk;   // 131072 entries per work item
constexpr int kBins = 2048;

struct Layer {            // one tensor V_l / beta_l of the layout
    uint64_t offset;      // first entry inside a worker's gradient vector
    uint64_t out_offset;  // first pair inside a worker's output (sum of k of earlier tensors)
    uint32_t n, k;
    uint32_t n_slots;     // chunk slots reserved for it (covers any 16-byte misalignment)
    uint32_t slot_base;   // first slot inside a worker's slot range
    // bracketed route (select_bracket.cuh); all zero when the tensor is not on it
    uint32_t bracket;     // 1: eligible for the bracketed single-pass route
    uint32_t sample;      // sample size m (multiple of 32)
    uint32_t n_spans;     // spans of kSpanElems entries (covers any misalignment)
    uint32_t span_base;   // first span inside a worker's span range
    uint32_t cand_cap;    // room in the candidate list
    uint32_t win_cap;     // room in the window list
    uint64_t cand_base;   // first candidate slot inside a worker's candidate range
    uint64_t win_base;    // first window slot inside a worker's window range
    uint32_t cluster;     // 1: large enough, and small enough, for the cluster route (select_cluster.cuh) on this device
    uint32_t pad;
};

struct Inst {             // selection state of one (worker, tensor)
    uint32_t prefix;      // threshold key bits decided so far; after pass 2 the threshold key T
    uint32_t k_rem;       // rank still to be found inside the current bucket; after pass 2: r
    uint32_t n_gt;        // entries whose key is above the current bucket; after pass 2: #{key > T}
    uint32_t flags;       // route bookkeeping (kInstGeneral ...)
    uint32_t done[5];     // finished chunks per pass
    // bracketed route
    uint32_t t_lo;        // the threshold key lies in [t_lo, t_hi]
    uint32_t cand_count;  // entries with key >= t_lo appended so far   } one 8-byte word, advanced
    uint32_t win_count;   // of those, entries with key <= t_hi         } by a single 64-bit atomic
    uint32_t t_hi;
    uint32_t spare;
    uint32_t T, cut;      // exact threshold: keep key > T, and key == T with shifted index < cut
};
static_assert(sizeof(Inst) == 64, "Inst is one 64-byte record");
static_assert(offsetof(Inst, cand_count) % 8 == 0 && offsetof(Inst, win_count) == offsetof(Inst, cand_count) + 4,
              "cand_count / win_count form one aligned 64-bit word");
constexpr uint32_t kInstGeneral = 1u;   // instance is (to be) handled by the general route

struct SelectParams {
    const float* grads;
    uint64_t stride;
    uint32_t n_workers, n_layers;
    const Layer* layers;
    Inst* inst;
    uint32_t* hist;             // [list position][kBins]
    uint32_t* list;             // instances on the general route
    uint32_t* list_slot_start;  // exclusive prefix of their chunk slots
    uint32_t* list_len;         // [0] = instances listed, [1] = total chunk slots
    uint2* chunk_cnt;           // [worker][slot]: (#key>T, #key==T), then their exclusive prefixes
    uint32_t slots_per_worker;
    uint32_t* idx_out;
    float* val_out;
    uint64_t K;
    int* status;
    // bracketed route
    const uint2* items;         // scan / emit work items: (tensor, first span)
    uint32_t* cand_idx;         // [worker][cand_stride] shifted index of each candidate
    float* cand_val;            //                        its value
    uint32_t* win_key;          // [worker][win_stride] key of each window entry
    uint32_t* win_idx;          //                       its shifted index
    uint2* sub_tab;             // [worker][span_stride * 8] per 1024-entry piece: (first candidate slot, count | above-window count << 16)
    uint32_t* span_off;         // [worker][span_stride] kept entries before the span
    uint64_t cand_stride, win_stride, span_stride;
};

// ---------------------------------------------------------------------------------------------
// Block-wide exclusive prefix sum of one value per thread (kThreads threads). Returns the
// exclusive prefix; *total receives the block total.  Two barriers.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* total, uint32_t* s_warp /*[9]*/) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += y;
    }
    __syncthreads();            // protects s_warp against a previous use
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    uint32_t base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
        uint32_t t = s_warp[w];
        if (w < warp) base += t;
        tot += t;
    }
    *total = tot;
    return base + inc - v;
}

// The same for any block size that is a multiple of 32 (up to 1024): warp scans, then a scan of
// the warp totals by the first warp.  s_warp needs 33 entries.
template <int THREADS>
__device__ __forceinline__ uint32_t block_exclusive_scan_t(uint32_t v, uint32_t* total, uint32_t* s_warp /*[33]*/) {
    constexpr int WARPS = THREADS / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += y;
    }
    __syncthreads();
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const uint32_t t = lane < WARPS ? s_warp[lane] : 0u;
        uint32_t winc = t;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t y = __shfl_up_sync(0xFFFFFFFFu, winc, d);
            if (lane >= d) winc += y;
        }
        if (lane < WARPS) s_warp[lane] = winc - t;       // exclusive prefix of the warp totals
        if (lane == 31) s_warp[32] = winc;               // block total
    }
    __syncthreads();
    *total = s_warp[32];
    return s_warp[warp] + inc - v;
}

// Geometry of one work item: a chunk of an instance, in "shifted" coordinates that start at the
// 16-byte boundary at or below the tensor's first entry, so that every load is an aligned float4.
struct ChunkView {
    const float4* vec;     // aligned base
    uint64_t nvec;         // float4 count covering the tensor
    uint32_t mis;          // entries between the aligned base and the tensor's first entry (0..3)
    uint64_t n_shift;      // mis + n
    uint64_t vec_begin;    // first float4 of this chunk
    uint32_t iters;        // block iterations in this chunk (0 for an empty slot)
};

__device__ __forceinline__ ChunkView chunk_view(const SelectParams& p, uint32_t w, const Layer& L, uint32_t c) {
    ChunkView v;
    const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
    v.mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
    v.vec = reinterpret_cast<const float4*>(first - v.mis);
    v.n_shift = static_cast<uint64_t>(L.n) + v.mis;
    v.nvec = (v.n_shift + 3) >> 2;
    v.vec_begin = static_cast<uint64_t>(c) * (kChunkElems / 4);
    uint64_t left = v.nvec > v.vec_begin ? v.nvec - v.vec_begin : 0;
    uint64_t its = (left + kThreads - 1) / kThreads;
    v.iters = static_cast<uint32_t>(its < kItersPerChunk ? its : kItersPerChunk);
    return v;
}

struct WorkItem {
    uint32_t f, inst, w, l, c;
};

__device__ __forceinline__ WorkItem decode_item(const SelectParams& p, uint32_t g, uint32_t n_list) {
    // largest f with list_slot_start[f] <= g
    uint32_t lo = 0, hi = n_list;
    while (hi - lo > 1) {
        uint32_t mid = (lo + hi) >> 1;
        if (__ldcg(&p.list_slot_start[mid]) <= g) lo = mid; else hi = mid;
    }
    WorkItem it;
    it.f = lo;
    it.inst = __ldcg(&p.list[lo]);
    it.c = g - __ldcg(&p.list_slot_start[lo]);
    it.w = it.inst / p.n_layers;
    it.l = it.inst - it.w * p.n_layers;
    return it;
}

// ---------------------------------------------------------------------------------------------
// Builds the work list: the instances flagged for the general route (their state was reset at
// the start of the call).  One block.
__global__ void __launch_bounds__(kThreads) k_general_plan(SelectParams p) {
    __shared__ uint32_t s_warp[9];
    __shared__ uint32_t s_carry[2];
    if (threadIdx.x == 0) { s_carry[0] = 0; s_carry[1] = 0; }
    __syncthreads();
    const uint32_t n_inst = p.n_workers * p.n_layers;
    for (uint32_t base = 0; base < n_inst; base += kThreads) {
        const uint32_t i = base + threadIdx.x;
        uint32_t take = 0, slots = 0;
        if (i < n_inst) {
            const Layer& L = p.layers[i % p.n_layers];
            take = (__ldcg(&p.inst[i].flags) & kInstGeneral) ? 1u : 0u;
            slots = take ? L.n_slots : 0u;
        }
        uint32_t tot_take, tot_slots;
        uint32_t pos = block_exclusive_scan(take, &tot_take, s_warp);
        uint32_t spos = block_exclusive_scan(slots, &tot_slots, s_warp);
        const uint32_t c0 = s_carry[0], c1 = s_carry[1];
        if (take) {
            p.list[c0 + pos] = i;
            p.list_slot_start[c0 + pos] = c1 + spos;
        }
        __syncthreads();
        if (threadIdx.x == 0) { s_carry[0] = c0 + tot_take; s_carry[1] = c1 + tot_slots; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { p.list_len[0] = s_carry[0]; p.list_len[1] = s_carry[1]; }
}

// ---------------------------------------------------------------------------------------------
template <int PASS> struct Digit;
template <> struct Digit<0> {
    static constexpr int bins = 2048, shift = 20;
    __device__ static bool match(uint32_t, uint32_t) { return true; }
    __device__ static uint32_t of(uint32_t key) { return key >> 20; }
};
template <> struct Digit<1> {
    static constexpr int bins = 1024, shift = 10;
    __device__ static bool match(uint32_t key, uint32_t prefix) { return (key >> 20) == (prefix >> 20); }
    __device__ static uint32_t of(uint32_t key) { return (key >> 10) & 1023u; }
};
template <> struct Digit<2> {
    static constexpr int bins = 1024, shift = 0;
    __device__ static bool match(uint32_t key, uint32_t prefix) { return (key >> 10) == (prefix >> 10); }
    __device__ static uint32_t of(uint32_t key) { return key & 1023u; }
};

// The last block of an instance: walk the digit histogram from the largest digit down and pick
// the bucket that holds the k_rem-th largest matching key.
template <int PASS>
__device__ void fix_next_digit(uint32_t* hist, Inst* st, uint32_t* s_warp) {
    constexpr int NB = Digit<PASS>::bins, M = NB / kThreads;
    const uint32_t k_rem = st->k_rem;
    uint32_t h[M], sum = 0;
    const int top = NB - 1 - static_cast<int>(threadIdx.x) * M;   // thread 0 owns the largest digits
#pragma unroll
    for (int q = 0; q < M; ++q) { h[q] = __ldcg(&hist[top - q]); sum += h[q]; }
    uint32_t total;
    uint32_t above = block_exclusive_scan(sum, &total, s_warp);
#pragma unroll
    for (int q = 0; q < M; ++q) {
        if (above < k_rem && k_rem <= above + h[q]) {
            st->prefix |= static_cast<uint32_t>(top - q) << Digit<PASS>::shift;
            st->k_rem = k_rem - above;
            st->n_gt += above;
        }
        above += h[q];
        hist[top - q] = 0;          // ready for the next pass
    }
}

template <int PASS>
__global__ void __launch_bounds__(kThreads) k_general_hist(SelectParams p) {
    __shared__ uint32_t sh[kBins];
    __shared__ uint32_t s_warp[9];
    __shared__ uint32_t s_last;
    constexpr int NB = Digit<PASS>::bins;
    const uint32_t n_list = __ldcg(&p.list_len[0]), total = __ldcg(&p.list_len[1]);
    for (uint32_t g = blockIdx.x; g < total; g += gridDim.x) {
        const WorkItem it = decode_item(p, g, n_list);
        const Layer L = p.layers[it.l];
        Inst* st = &p.inst[it.inst];
        const uint32_t prefix = PASS ? __ldcg(&st->prefix) : 0u;
        const ChunkView cv = chunk_view(p, it.w, L, it.c);
        for (int b = threadIdx.x; b < NB; b += kThreads) sh[b] = 0;
        __syncthreads();
        for (uint32_t i = 0; i < cv.iters; ++i) {
            const uint64_t v = cv.vec_begin + static_cast<uint64_t>(i) * kThreads + threadIdx.x;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (v < cv.nvec) x = __ldg(&cv.vec[v]);
            const float xs[4] = {x.x, x.y, x.z, x.w};
            const uint64_t e0 = v * 4;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint64_t e = e0 + q;
                const uint32_t key = magnitude_key(xs[q]);
                const bool on = v < cv.nvec && e >= cv.mis && e < cv.n_shift && Digit<PASS>::match(key, prefix);
                // plain shared-memory atomics: on this GPU they take the crowding of magnitudes into a few exponent values in
                // their stride (the pass runs at 4.5 TB/s on Gaussian data); finding equal digits across the warp first with
                // a match and adding once per distinct digit was measured seven times slower
                if (on) atomicAdd(&sh[Digit<PASS>::of(key)], 1u);
            }
        }
        __syncthreads();
        uint32_t* hist = p.hist + static_cast<size_t>(it.f) * kBins;
        for (int b = threadIdx.x; b < NB; b += kThreads)
            if (sh[b]) atomicAdd(&hist[b], sh[b]);
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) s_last = (atomicAdd(&st->done[PASS], 1u) == L.n_slots - 1) ? 1u : 0u;
        __syncthreads();
        if (s_last) {
            __threadfence();
            fix_next_digit<PASS>(hist, st, s_warp);
        }
        __syncthreads();
    }
}

// pass 3: per-chunk counts of key > T and key == T, then exclusive prefixes over the chunks.
__global__ void __launch_bounds__(kThreads) k_general_count(SelectParams p) {
    __shared__ uint32_t s_warp[9];
    __shared__ uint32_t s_last;
    __shared__ uint32_t s_carry[2];
    const uint32_t n_list = __ldcg(&p.list_len[0]), total = __ldcg(&p.list_len[1]);
    for (uint32_t g = blockIdx.x; g < total; g += gridDim.x) {
        const WorkItem it = decode_item(p, g, n_list);
        const Layer L = p.layers[it.l];
        Inst* st = &p.inst[it.inst];
        const uint32_t T = __ldcg(&st->prefix);
        const ChunkView cv = chunk_view(p, it.w, L, it.c);
        uint32_t gt = 0, eq = 0;
        for (uint32_t i = 0; i < cv.iters; ++i) {
            const uint64_t v = cv.vec_begin + static_cast<uint64_t>(i) * kThreads + threadIdx.x;
            if (v < cv.nvec) {
                const float4 x = __ldg(&cv.vec[v]);
                const float xs[4] = {x.x, x.y, x.z, x.w};
                const uint64_t e0 = v * 4;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint64_t e = e0 + q;
                    const uint32_t key = magnitude_key(xs[q]);
                    const bool ok = e >= cv.mis && e < cv.n_shift;
                    gt += (ok && key > T) ? 1u : 0u;
                    eq += (ok && key == T) ? 1u : 0u;
                }
            }
        }
        uint32_t tg, te;
        block_exclusive_scan(gt, &tg, s_warp);
        block_exclusive_scan(eq, &te, s_warp);
        uint2* cnt = p.chunk_cnt + static_cast<size_t>(it.w) * p.slots_per_worker + L.slot_base;
        if (threadIdx.x == 0) {
            cnt[it.c] = make_uint2(tg, te);
            __threadfence();
            s_last = (atomicAdd(&st->done[3], 1u) == L.n_slots - 1) ? 1u : 0u;
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            if (threadIdx.x == 0) { s_carry[0] = 0; s_carry[1] = 0; }
            __syncthreads();
            for (uint32_t base = 0; base < L.n_slots; base += kThreads) {
                const uint32_t c = base + threadIdx.x;
                uint2 v = make_uint2(0, 0);
                if (c < L.n_slots) v = __ldcg(&cnt[c]);
                uint32_t t0, t1;
                uint32_t e0 = block_exclusive_scan(v.x, &t0, s_warp);
                uint32_t e1 = block_exclusive_scan(v.y, &t1, s_warp);
                const uint32_t c0 = s_carry[0], c1 = s_carry[1];
                if (c < L.n_slots) cnt[c] = make_uint2(c0 + e0, c1 + e1);
                __syncthreads();
                if (threadIdx.x == 0) { s_carry[0] = c0 + t0; s_carry[1] = c1 + t1; }
                __syncthreads();
            }
        }
        __syncthreads();
    }
}

// pass 4: ordered write.
__global__ void __launch_bounds__(kThreads) k_general_write(SelectParams p) {
    __shared__ uint32_t s_warp[9];
    const uint32_t n_list = __ldcg(&p.list_len[0]), total = __ldcg(&p.list_len[1]);
    for (uint32_t g = blockIdx.x; g < total; g += gridDim.x) {
        const WorkItem it = decode_item(p, g, n_list);
        const Layer L = p.layers[it.l];
        const Inst* st = &p.inst[it.inst];
        const uint32_t T = __ldcg(&st->prefix), r = __ldcg(&st->k_rem);
        const ChunkView cv = chunk_view(p, it.w, L, it.c);
        const uint2 before = __ldcg(&p.chunk_cnt[static_cast<size_t>(it.w) * p.slots_per_worker + L.slot_base + it.c]);
        uint32_t gt_base = before.x, eq_base = before.y;
        uint32_t* idx_out = p.idx_out + static_cast<uint64_t>(it.w) * p.K + L.out_offset;
        float* val_out = p.val_out + static_cast<uint64_t>(it.w) * p.K + L.out_offset;
        for (uint32_t i = 0; i < cv.iters; ++i) {
            const uint64_t v = cv.vec_begin + static_cast<uint64_t>(i) * kThreads + threadIdx.x;
            float xs[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t gtm = 0, eqm = 0;
            const uint64_t e0 = v * 4;
            if (v < cv.nvec) {
                const float4 x = __ldg(&cv.vec[v]);
                xs[0] = x.x; xs[1] = x.y; xs[2] = x.z; xs[3] = x.w;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint64_t e = e0 + q;
                    const uint32_t key = magnitude_key(xs[q]);
                    const bool ok = e >= cv.mis && e < cv.n_shift;
                    gtm |= (ok && key > T) ? (1u << q) : 0u;
                    eqm |= (ok && key == T) ? (1u << q) : 0u;
                }
            }
            uint32_t tot;
            const uint32_t ex = block_exclusive_scan(__popc(gtm) | (__popc(eqm) << 16), &tot, s_warp);
            uint32_t gt_before = gt_base + (ex & 0xFFFFu), eq_before = eq_base + (ex >> 16);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bool is_gt = (gtm >> q) & 1u, is_eq = (eqm >> q) & 1u;
                if (is_gt || (is_eq && eq_before < r)) {
                    const uint32_t pos = gt_before + (eq_before < r ? eq_before : r);
                    idx_out[pos] = static_cast<uint32_t>(L.offset + (e0 + q - cv.mis));
                    val_out[pos] = xs[q];
                }
                gt_before += is_gt ? 1u : 0u;
                eq_before += is_eq ? 1u : 0u;
            }
            gt_base += tot & 0xFFFFu;
            eq_base += tot >> 16;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Values of entries chosen elsewhere (e.g. a random selection, as one of the Comp-ASGD variants
// makes): val[w][e] = g[w][idx[w][e]].  An index outside the layout is reported and reads as 0.
__global__ void __launch_bounds__(kThreads)
k_gather(const float* __restrict__ grads, uint64_t stride, uint64_t extent, const uint32_t* __restrict__ idx,
         float* __restrict__ val_out, uint64_t pairs_per_worker, uint64_t total, int* status) {
    for (uint64_t t = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x; t < total;
         t += static_cast<uint64_t>(gridDim.x) * kThreads) {
        const uint64_t w = t / pairs_per_worker;
        const uint32_t k = idx[t];
        float v = 0.f;
        if (k < extent) v = __ldg(grads + w * stride + k);
        else record_error(status, ADACOMP_ERR_INVALID);
        val_out[t] = v;
    }
}

}  // namespace adacomp
