// SELECT_GRAD (Algorithm 1), bracketed route: the dense gradient crosses HBM once.
//
// The k-th largest magnitude of a tensor is first bracketed from a small sample, then one
// streaming pass keeps only what can still matter:
//   k_bracket_sample   per (worker, tensor): read a stratified sample, take two of its order
//                      statistics t_lo <= t_hi chosen so that, with overwhelming probability,
//                      #{key > t_hi} <= k <= #{key >= t_lo};
//   k_bracket_scan     the single pass over the gradient: every entry with key >= t_lo (a
//                      "candidate", about 1.1-2.5 k of them) is appended, in index order span by
//                      span, to the instance's candidate list; candidates with key <= t_hi (the
//                      "window", where the threshold must lie) are also appended to a small
//                      unordered list; per span the pass records where its candidates went and
//                      how many entries are above the window;
//   k_bracket_resolve  per instance: verify the bracket with the exact counts, find the exact
//                      threshold inside the window (radix select on (key, index) composites,
//                      finished by brute force once few entries remain), count the kept window
//                      entries per span and turn the per-span kept counts into output offsets;
//   k_bracket_emit     per span: read its candidates, keep those at or above the exact threshold,
//                      write them to the output in index order.
// The result is exact whatever the sample looked like: if the exact counts contradict the
// bracket, or a list overflows its capacity, the instance is handed to the general route.
// No kernel waits on another block; all cross-block traffic is atomics plus kernel boundaries.
#pragma once

#include "select_general.cuh"

namespace adacomp {

constexpr uint32_t kSpanElems = 8192;                 // entries per span (one block iteration)
constexpr uint32_t kSpanVecs = kSpanElems / 4;
constexpr uint32_t kSpansPerBlock = 8;                // scan: consecutive spans per block; emit: one per warp
constexpr uint32_t kMaxSpans = 4096;                  // per tensor on this route (n <= 33.5 M)
constexpr uint32_t kBracketMinN = 32768;
constexpr uint32_t kSampleMax = 16384;
constexpr uint32_t kSampleMin = 2048;
constexpr float kBracketZ = 5.0f;                     // half-width of the bracket in sample standard deviations
constexpr uint32_t kGatherMax = 512;

constexpr uint32_t kInstBracket = 2u;                 // bracket valid, scan/emit act on the instance
constexpr uint32_t kInstOverflow = 4u;                // a candidate or window list ran out of room

// Sample ranks (1 = largest) whose keys bracket the k-th largest of n entries, from a sample of m.
__host__ __device__ inline void bracket_ranks(uint32_t n, uint32_t k, uint32_t m, uint32_t* r_hi, uint32_t* r_lo) {
    const float p = static_cast<float>(k) / static_cast<float>(n);
    const float mp = p * static_cast<float>(m);
    const float sd = sqrtf(mp * (1.0f - p));
    const float hi = floorf(mp - kBracketZ * sd) - 1.0f;
    const float lo = ceilf(mp + kBracketZ * sd) + 1.0f;
    *r_hi = hi >= 1.0f ? static_cast<uint32_t>(hi) : 0u;            // 0: no upper bound from the sample
    *r_lo = static_cast<uint32_t>(lo);                              // may exceed m: no lower bound
}

__device__ __forceinline__ uint32_t hash32(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
    return x;
}

// Descending walk over a histogram in shared memory: the bucket holding the rem-th largest.
// All kThreads threads call; results are returned to all.  NB must be a multiple of kThreads.
template <int NB>
__device__ __forceinline__ void block_pick_bucket(const uint32_t* hist, uint32_t rem, uint32_t* bucket,
                                                  uint32_t* above_out, uint32_t* count_out,
                                                  uint32_t* s_warp, uint32_t* s_bc /*[3]*/) {
    constexpr int M = NB / kThreads;
    const int top = NB - 1 - static_cast<int>(threadIdx.x) * M;
    uint32_t h[M], sum = 0;
#pragma unroll
    for (int q = 0; q < M; ++q) { h[q] = hist[top - q]; sum += h[q]; }
    uint32_t total;
    uint32_t above = block_exclusive_scan(sum, &total, s_warp);
#pragma unroll
    for (int q = 0; q < M; ++q) {
        if (above < rem && rem <= above + h[q]) { s_bc[0] = top - q; s_bc[1] = above; s_bc[2] = h[q]; }
        above += h[q];
    }
    __syncthreads();
    *bucket = s_bc[0]; *above_out = s_bc[1]; *count_out = s_bc[2];
    __syncthreads();
}

// rank-th largest (1 = largest) of m keys in shared memory; three digit passes.
__device__ uint32_t smem_kth_largest(const uint32_t* keys, uint32_t m, uint32_t rank, uint32_t* hist,
                                     uint32_t* s_warp, uint32_t* s_bc) {
    uint32_t prefix = 0, rem = rank;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 20 : (pass == 1 ? 10 : 0);
        const int nb = pass == 0 ? 2048 : 1024;
        for (int b = threadIdx.x; b < 2048; b += kThreads) hist[b] = 0;
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < m; i += kThreads) {
            const uint32_t key = keys[i];
            const bool match = pass == 0 || (key >> (shift + 10)) == (prefix >> (shift + 10));
            if (match) atomicAdd(&hist[(key >> shift) & (nb - 1)], 1u);
        }
        __syncthreads();
        uint32_t b, above, cnt;
        block_pick_bucket<2048>(hist, rem, &b, &above, &cnt, s_warp, s_bc);   // unused upper bins are zero
        prefix |= b << shift;
        rem -= above;
    }
    return prefix;
}

// ---------------------------------------------------------------------------------------------
// One block per (worker, tensor): reset the instance, and bracket its threshold if it is on
// this route.  Dynamic shared memory: the sample keys.
__global__ void __launch_bounds__(kThreads) k_bracket_sample(SelectParams p, int general_only) {
    extern __shared__ uint32_t s_keys[];
    __shared__ uint32_t s_hist[2048];
    __shared__ uint32_t s_warp[9];
    __shared__ uint32_t s_bc[3];
    const uint32_t inst = blockIdx.x;
    const uint32_t w = inst / p.n_layers, l = inst - w * p.n_layers;
    const Layer L = p.layers[l];
    Inst* st = &p.inst[inst];
    const bool bracket = L.bracket && !general_only;
    if (threadIdx.x == 0) {
        st->prefix = 0; st->k_rem = L.k; st->n_gt = 0;
        st->flags = bracket ? 0u : (L.k > 0 ? kInstGeneral : 0u);
#pragma unroll
        for (int q = 0; q < 5; ++q) st->done[q] = 0;
        st->cand_count = 0; st->win_count = 0; st->n_def = 0; st->T = 0; st->cut = 0;
    }
    if (!bracket) return;

    const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
    const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
    const float4* vec = reinterpret_cast<const float4*>(first - mis);
    const uint32_t m = L.sample, n_chunks = m / 32, stratum = L.n / n_chunks;   // stratum >= 128
    // chunk j: 32 consecutive entries starting at a hashed position inside stratum j, moved up to
    // the next 32-byte boundary; always inside the tensor
    for (uint32_t t = threadIdx.x; t < n_chunks * 8; t += kThreads) {
        const uint32_t j = t >> 3, part = t & 7;
        const uint32_t e = j * stratum + hash32(j * 2654435761u + l * 40503u + 977u) % (stratum - 40);
        const uint32_t s = (e + mis + 7) & ~7u;                  // shifted coordinate, multiple of 8
        const float4 x = __ldg(&vec[(s >> 2) + part]);
        uint32_t* dst = &s_keys[j * 32 + part * 4];
        dst[0] = magnitude_key(x.x); dst[1] = magnitude_key(x.y);
        dst[2] = magnitude_key(x.z); dst[3] = magnitude_key(x.w);
    }
    __syncthreads();
    uint32_t r_hi, r_lo;
    bracket_ranks(L.n, L.k, m, &r_hi, &r_lo);
    if (r_lo > m) {                                   // cannot bound from below: general route
        if (threadIdx.x == 0) st->flags = kInstGeneral;
        return;
    }
    const uint32_t t_lo = smem_kth_largest(s_keys, m, r_lo, s_hist, s_warp, s_bc);
    const uint32_t t_hi = r_hi ? smem_kth_largest(s_keys, m, r_hi, s_hist, s_warp, s_bc) : 0x7FFFFFFFu;
    if (threadIdx.x == 0) { st->t_lo = t_lo; st->t_hi = t_hi; st->flags = kInstBracket; }
}

// ---------------------------------------------------------------------------------------------
// The single pass over the gradient.  grid = (scan items, workers); an item is up to
// kSpansPerBlock consecutive spans of one tensor.  Each warp holds 1024 consecutive entries of a
// span in registers (8 coalesced float4 loads), so candidates come out in index order.
__global__ void __launch_bounds__(kThreads) k_bracket_scan(SelectParams p) {
    __shared__ uint32_t s_tot[kThreads / 32];
    __shared__ uint32_t s_base[2];
    __shared__ uint32_t s_over;
    const uint2 item = p.items[blockIdx.x];
    const uint32_t l = item.x, w = blockIdx.y;
    const Layer L = p.layers[l];
    Inst* st = &p.inst[w * p.n_layers + l];
    if (!(__ldcg(&st->flags) & kInstBracket)) return;
    const uint32_t t_lo = __ldcg(&st->t_lo), t_hi = __ldcg(&st->t_hi);
    const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
    const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
    const float4* vec = reinterpret_cast<const float4*>(first - mis);
    const uint32_t n_shift = L.n + mis;                        // n <= 2^31 on this route
    const uint32_t nvec = (n_shift + 3) >> 2;
    uint32_t* cand_idx = p.cand_idx + static_cast<uint64_t>(w) * p.cand_stride + L.cand_base;
    float* cand_val = p.cand_val + static_cast<uint64_t>(w) * p.cand_stride + L.cand_base;
    uint32_t* win_key = p.win_key + static_cast<uint64_t>(w) * p.win_stride + L.win_base;
    uint32_t* win_idx = p.win_idx + static_cast<uint64_t>(w) * p.win_stride + L.win_base;
    uint2* span_tab = p.span_tab + static_cast<uint64_t>(w) * p.span_stride + L.span_base;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t s_end = min(item.y + kSpansPerBlock, L.n_spans);

    for (uint32_t s = item.y; s < s_end; ++s) {
        const uint32_t vec0 = s * kSpanVecs + warp * 256;
        const bool full = (s * kSpanElems >= mis) && ((s + 1) * kSpanElems <= n_shift);
        float4 x[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t v = vec0 + i * 32 + lane;
            x[i] = (v < nvec) ? __ldcs(&vec[v]) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        // pass A: classify; one bit per held entry
        uint32_t mask_c = 0, mask_w = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float xs[4] = {x[i].x, x[i].y, x[i].z, x[i].w};
            const uint32_t e0 = (vec0 + i * 32 + lane) * 4;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t key = magnitude_key(xs[q]);
                const bool ok = full || (e0 + q >= mis && e0 + q < n_shift);
                const bool c = ok && key >= t_lo;
                mask_c |= (c ? 1u : 0u) << (i * 4 + q);
                mask_w |= ((c && key <= t_hi) ? 1u : 0u) << (i * 4 + q);
            }
        }
        const uint32_t cw = __popc(mask_w);
        const uint32_t tc = __reduce_add_sync(0xFFFFFFFFu, __popc(mask_c));
        const uint32_t tw = __reduce_add_sync(0xFFFFFFFFu, cw);
        if (lane == 0) s_tot[warp] = tc | (tw << 16);
        __syncthreads();
        uint32_t pc = 0, pw = 0, totc = 0, totw = 0;
#pragma unroll
        for (int ww = 0; ww < kThreads / 32; ++ww) {
            const uint32_t t = s_tot[ww];
            if (ww < warp) { pc += t & 0xFFFFu; pw += t >> 16; }
            totc += t & 0xFFFFu; totw += t >> 16;
        }
        if (threadIdx.x == 0) {
            const uint32_t cb = totc ? atomicAdd(&st->cand_count, totc) : 0u;
            const uint32_t wb = totw ? atomicAdd(&st->win_count, totw) : 0u;
            const uint32_t ndef = totc - totw;
            if (ndef) atomicAdd(&st->n_def, ndef);
            const bool over = (static_cast<uint64_t>(cb) + totc > L.cand_cap) || (static_cast<uint64_t>(wb) + totw > L.win_cap);
            if (over) atomicOr(&st->flags, kInstOverflow);
            s_base[0] = cb; s_base[1] = wb; s_over = over ? 1u : 0u;
            span_tab[s] = make_uint2(cb, totc | (ndef << 16));
        }
        __syncthreads();
        const uint32_t cb = s_base[0], wb = s_base[1];
        const bool over = s_over != 0;
        if (!over && tc > 0) {
            // pass B: positions.  Candidates in index order = (load i, lane, component q).
            uint32_t wpos = 0;
            if (tw > 0) {                                  // window: any order, lane-major
                uint32_t inc = cw;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                    if (lane >= d) inc += y;
                }
                wpos = wb + pw + inc - cw;
            }
            uint32_t running = cb + pc;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t m4 = (mask_c >> (i * 4)) & 15u;
                if (!__any_sync(0xFFFFFFFFu, m4 != 0)) continue;
                const uint32_t c4 = __popc(m4);
                const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, c4 & 1u);
                const uint32_t b1 = __ballot_sync(0xFFFFFFFFu, c4 & 2u);
                const uint32_t b2 = __ballot_sync(0xFFFFFFFFu, c4 & 4u);
                uint32_t pos = running + __popc(b0 & lt) + 2 * __popc(b1 & lt) + 4 * __popc(b2 & lt);
                running += __popc(b0) + 2 * __popc(b1) + 4 * __popc(b2);
                if (m4) {
                    const float xs[4] = {x[i].x, x[i].y, x[i].z, x[i].w};
                    const uint32_t e0 = (vec0 + i * 32 + lane) * 4;
                    const uint32_t w4 = (mask_w >> (i * 4)) & 15u;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if ((m4 >> q) & 1u) {
                            cand_idx[pos] = e0 + q;            // shifted coordinate inside the tensor
                            cand_val[pos] = xs[q];
                            ++pos;
                            if ((w4 >> q) & 1u) {
                                win_key[wpos] = magnitude_key(xs[q]);
                                win_idx[wpos] = e0 + q;
                                ++wpos;
                            }
                        }
                    }
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// One block per instance: exact threshold inside the window, per-span output offsets.
__global__ void __launch_bounds__(kThreads) k_bracket_resolve(SelectParams p) {
    __shared__ uint32_t s_hist[2048];
    __shared__ uint32_t s_sel[kMaxSpans];
    __shared__ unsigned long long s_g[kGatherMax];
    __shared__ uint32_t s_warp[9];
    __shared__ uint32_t s_bc[3];
    __shared__ uint32_t s_cnt;
    __shared__ unsigned long long s_cstar;
    __shared__ uint32_t s_carry;
    const uint32_t inst = blockIdx.x;
    const uint32_t w = inst / p.n_layers, l = inst - w * p.n_layers;
    const Layer L = p.layers[l];
    Inst* st = &p.inst[inst];
    const uint32_t flags = __ldcg(&st->flags);
    if (!(flags & kInstBracket)) return;
    const uint32_t n_cand = __ldcg(&st->cand_count), n_win = __ldcg(&st->win_count), n_def = __ldcg(&st->n_def);
    const uint32_t t_lo = __ldcg(&st->t_lo), t_hi = __ldcg(&st->t_hi);
    const bool bad = (flags & kInstOverflow) || n_cand > L.cand_cap || n_win > L.win_cap || n_def > L.k ||
                     L.k - n_def > n_win;
    if (bad) {                                        // the bracket missed: hand over, state is still pristine
        if (threadIdx.x == 0) st->flags = kInstGeneral;
        return;
    }
    const uint32_t* win_key = p.win_key + static_cast<uint64_t>(w) * p.win_stride + L.win_base;
    const uint32_t* win_idx = p.win_idx + static_cast<uint64_t>(w) * p.win_stride + L.win_base;
    uint2* span_tab = p.span_tab + static_cast<uint64_t>(w) * p.span_stride + L.span_base;
    uint32_t* span_off = p.span_off + static_cast<uint64_t>(w) * p.span_stride + L.span_base;
    const uint32_t need = L.k - n_def;

    // composite of a window entry: larger = kept first (larger key, then lower index)
    auto composite = [&](uint32_t i) -> unsigned long long {
        return (static_cast<unsigned long long>(__ldcg(&win_key[i]) - t_lo) << 32) |
               static_cast<unsigned long long>(0xFFFFFFFFu - __ldcg(&win_idx[i]));
    };

    unsigned long long cstar = ~0ull;                 // keep window entries with composite >= cstar
    if (need > 0) {
        const uint32_t range = t_hi - t_lo;
        int hi_shift = (range ? 32 - __clz(range) : 0) + 32;   // undecided low bits of the composite
        unsigned long long prefix = 0;
        uint32_t rem = need, count = n_win;
        while (true) {
            if (count <= kGatherMax) {                // few left: gather them and rank by brute force
                if (threadIdx.x == 0) s_cnt = 0;
                __syncthreads();
                for (uint32_t i = threadIdx.x; i < n_win; i += kThreads) {
                    const unsigned long long c = composite(i);
                    if (hi_shift >= 64 || (c >> hi_shift) == prefix) s_g[atomicAdd(&s_cnt, 1u)] = c;
                }
                __syncthreads();
                for (uint32_t t = threadIdx.x; t < count; t += kThreads) {
                    const unsigned long long mine = s_g[t];
                    uint32_t larger = 0;
                    for (uint32_t u = 0; u < count; ++u) larger += s_g[u] > mine ? 1u : 0u;
                    if (larger == rem - 1) s_cstar = mine;
                }
                __syncthreads();
                cstar = s_cstar;
                break;
            }
            if (hi_shift == 0) { cstar = prefix; break; }     // cannot happen: composites are distinct
            const int bits = hi_shift < 11 ? hi_shift : 11;
            const int new_shift = hi_shift - bits;
            for (int b = threadIdx.x; b < 2048; b += kThreads) s_hist[b] = 0;
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < n_win; i += kThreads) {
                const unsigned long long c = composite(i);
                if (hi_shift >= 64 || (c >> hi_shift) == prefix)
                    atomicAdd(&s_hist[static_cast<uint32_t>(c >> new_shift) & ((1u << bits) - 1u)], 1u);
            }
            __syncthreads();
            uint32_t b, above, cnt;
            block_pick_bucket<2048>(s_hist, rem, &b, &above, &cnt, s_warp, s_bc);
            prefix = (prefix << bits) | b;
            rem -= above;
            count = cnt;
            hi_shift = new_shift;
        }
    }
    // kept window entries per span
    for (uint32_t s = threadIdx.x; s < L.n_spans; s += kThreads) s_sel[s] = 0;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    if (need > 0) {
        for (uint32_t i = threadIdx.x; i < n_win; i += kThreads)
            if (composite(i) >= cstar) atomicAdd(&s_sel[__ldcg(&win_idx[i]) / kSpanElems], 1u);
    }
    __syncthreads();
    // exclusive prefix of kept entries over the spans
    for (uint32_t base = 0; base < L.n_spans; base += kThreads) {
        const uint32_t s = base + threadIdx.x;
        uint32_t kept = 0;
        if (s < L.n_spans) kept = (__ldcg(&span_tab[s]).y >> 16) + s_sel[s];
        uint32_t tot;
        const uint32_t ex = block_exclusive_scan(kept, &tot, s_warp);
        const uint32_t carry = s_carry;
        if (s < L.n_spans) span_off[s] = carry + ex;
        __syncthreads();
        if (threadIdx.x == 0) s_carry = carry + tot;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (s_carry != L.k) {
            st->flags = kInstGeneral;                 // defensive: counts must add up to k
        } else if (need > 0) {
            st->T = t_lo + static_cast<uint32_t>(cstar >> 32);
            st->cut = 0u - static_cast<uint32_t>(cstar);     // keep key == T iff shifted index < cut
        } else {
            st->T = t_hi;                             // everything above the window, nothing inside it
            st->cut = 0;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// grid = (scan items, workers); one warp per span: filter its candidates, write in order.
__global__ void __launch_bounds__(kThreads) k_bracket_emit(SelectParams p) {
    const uint2 item = p.items[blockIdx.x];
    const uint32_t l = item.x, w = blockIdx.y;
    const Layer L = p.layers[l];
    const Inst* st = &p.inst[w * p.n_layers + l];
    if (!(__ldcg(&st->flags) & kInstBracket)) return;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t s = item.y + warp;
    if (s >= L.n_spans) return;
    const uint32_t T = __ldcg(&st->T), cut = __ldcg(&st->cut);
    const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
    const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
    const uint32_t* cand_idx = p.cand_idx + static_cast<uint64_t>(w) * p.cand_stride + L.cand_base;
    const float* cand_val = p.cand_val + static_cast<uint64_t>(w) * p.cand_stride + L.cand_base;
    const uint2 tab = __ldcg(&p.span_tab[static_cast<uint64_t>(w) * p.span_stride + L.span_base + s]);
    const uint32_t cnt = tab.y & 0xFFFFu;
    uint32_t off = __ldcg(&p.span_off[static_cast<uint64_t>(w) * p.span_stride + L.span_base + s]);
    uint32_t* idx_out = p.idx_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
    float* val_out = p.val_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t glob = static_cast<uint32_t>(L.offset) - mis;        // shifted coordinate -> vector index
    for (uint32_t c = lane; c < ((cnt + 31) & ~31u); c += 32) {
        bool keep = false;
        uint32_t e = 0;
        float v = 0.f;
        if (c < cnt) {
            e = __ldcs(&cand_idx[tab.x + c]);
            v = __ldcs(&cand_val[tab.x + c]);
            const uint32_t key = magnitude_key(v);
            keep = key > T || (key == T && e < cut);
        }
        const uint32_t b = __ballot_sync(0xFFFFFFFFu, keep);
        if (keep) {
            const uint32_t pos = off + __popc(b & lt);
            idx_out[pos] = glob + e;
            val_out[pos] = v;
        }
        off += __popc(b);
    }
}

}  // namespace adacomp
