// SELECT_GRAD (Algorithm 1), bracketed route: the dense gradient crosses HBM once.
//
// The k-th largest magnitude of a tensor is first bracketed from a small sample, then one
// streaming pass keeps only what can still matter:
//   k_bracket_sample   per (worker, tensor): read a stratified sample, take two of its order
//                      statistics t_lo <= t_hi chosen so that, with overwhelming probability,
//                      #{key > t_hi} <= k <= #{key >= t_lo};
//   k_bracket_scan     the single pass over the gradient.  Every warp works on its own: its pieces of
//                      1024 entries arrive in shared memory by bulk asynchronous copies, every lane masks
//                      its 32 consecutive entries, and the entries with key >= t_lo ("candidates", about
//                      1.1-2.5 k of them per tensor) are appended, in index order, to the instance's
//                      candidate list; candidates with key <= t_hi (the "window", where the threshold
//                      must lie) also go to a small unordered list; a table records where each piece put
//                      its candidates and how many of them are above the window;
//   k_bracket_resolve  per instance: verify the bracket with the exact counts, find the exact
//                      threshold inside the window (radix select on (key, index) composites,
//                      finished by brute force once few entries remain), count the kept window
//                      entries per span and turn the per-span kept counts into output offsets;
//   k_bracket_emit     per span (8 pieces), one warp: read its candidates, keep those at or above
//                      the exact threshold, write them to the output in index order.
// The result is exact whatever the sample looked like: if the exact counts contradict the
// bracket, a list overflows its capacity or a NaN is seen, the instance is flagged and redone
// exactly: by k_fallback_solo (one block per flagged instance) when all tensors of the handle are on
// this route or small enough to be selected whole in shared memory, else by the general route.
// No kernel waits on another block; all cross-block traffic is atomics plus kernel boundaries.
#pragma once

#include "select_general.cuh"

namespace adacomp {

constexpr uint32_t kSubElems = 1024;                  // entries one warp classifies at a time
constexpr uint32_t kSubsPerSpan = 8;
constexpr uint32_t kSpanElems = kSubElems * kSubsPerSpan;   // 8192: unit of the output-offset prefix
constexpr uint32_t kSpansPerBlock = 8;                // scan: consecutive spans per block; emit: one per warp
constexpr uint32_t kMaxSpans = 4096;                  // spans whose counters the resolve kernel keeps in shared memory
constexpr uint32_t kBracketMaxN = 0xFFFF0000u;        // shifted 32-bit coordinates must not wrap
constexpr uint32_t kBracketMinN = 32768;
constexpr uint32_t kSampleMax = 16384;
constexpr uint32_t kSmallMax = kBracketMinN - 1;         // longest tensor whose keys are selected whole in shared memory
constexpr uint32_t kSampleMin = 2048;
constexpr float kBracketZ = 5.0f;                     // half-width of the bracket in sample standard deviations
constexpr uint32_t kGatherMax = 1024;
// Threads of the per-instance kernels (sample, resolve): a template parameter, chosen per call by the number of
// instances.  Measured: with thousands of instances (the ResNet-50-shaped call has 5152) 512 threads are 9 % faster
// over the whole call than 1024, with 400 instances 1 % faster, with 16 instances (one segment over a whole model of
// 10^8 parameters) 10 % slower.
constexpr int kBigFew = 1024;                         // calls with few instances
constexpr int kBigMany = 512;                         // calls with many
constexpr int kSoloThreads = 512;                     // the fallback kernel

constexpr uint32_t kRouteSmall = 3u;                  // Layer::bracket of a tensor that is selected whole in shared memory
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

// Descending walk over a 2048-bin histogram in shared memory: the bucket holding the rem-th
// largest.  All kT threads of the block call; results are returned to all.
template <int kT>
__device__ __forceinline__ void block_pick_bucket(const uint32_t* hist, uint32_t rem, uint32_t* bucket,
                                                  uint32_t* above_out, uint32_t* count_out,
                                                  uint32_t* s_warp /*[33]*/, uint32_t* s_bc /*[3]*/) {
    constexpr int M = 2048 / kT;
    const int top = 2047 - static_cast<int>(threadIdx.x) * M;
    uint32_t h[M], sum = 0;
#pragma unroll
    for (int q = 0; q < M; ++q) { h[q] = hist[top - q]; sum += h[q]; }
    uint32_t total;
    uint32_t above = block_exclusive_scan_t<kT>(sum, &total, s_warp);
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
template <int kT>
__device__ uint32_t smem_kth_largest(const uint32_t* keys, uint32_t m, uint32_t rank, uint32_t* hist,
                                     uint32_t* s_warp, uint32_t* s_bc) {
    uint32_t prefix = 0, rem = rank;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 20 : (pass == 1 ? 10 : 0);
        const int nb = pass == 0 ? 2048 : 1024;
        for (int b = threadIdx.x; b < 2048; b += kT) hist[b] = 0;
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < m; i += kT) {
            const uint32_t key = keys[i];
            const bool match = pass == 0 || (key >> (shift + 10)) == (prefix >> (shift + 10));
            if (match) atomicAdd(&hist[(key >> shift) & (nb - 1)], 1u);
        }
        __syncthreads();
        uint32_t b, above, cnt;
        block_pick_bucket<kT>(hist, rem, &b, &above, &cnt, s_warp, s_bc);   // unused upper bins are zero
        prefix |= b << shift;
        rem -= above;
    }
    return prefix;
}

// ---------------------------------------------------------------------------------------------
// One block per (worker, tensor): reset the instance, and bracket its threshold if it is on
// this route.  Dynamic shared memory: the sample keys.
template <int kT>
__global__ void __launch_bounds__(kT) k_bracket_sample(SelectParams p, int general_only) {
    extern __shared__ uint32_t s_keys[];
    __shared__ uint32_t s_hist[2048];
    __shared__ uint32_t s_warp[33];
    __shared__ uint32_t s_bc[3];
    const uint32_t inst = blockIdx.x;
    const uint32_t w = inst / p.n_layers, l = inst - w * p.n_layers;
    const Layer L = p.layers[l];
    Inst* st = &p.inst[inst];
    const bool bracket = L.bracket && general_only != 1;
    if (inst == 0 && threadIdx.x == 0) p.list_len[0] = 0;        // selections that took the general route: none so far
    if (threadIdx.x == 0) {
        st->prefix = 0; st->k_rem = L.k; st->n_gt = 0;
        st->flags = bracket ? 0u : (L.k > 0 ? kInstGeneral : 0u);
#pragma unroll
        for (int q = 0; q < 5; ++q) st->done[q] = 0;
        st->cand_count = 0; st->win_count = 0; st->T = 0; st->cut = 0;
    }
    if (!bracket) return;
    if (L.bracket == kRouteSmall) {
        // ---- a tensor that fits into shared memory whole is selected right here: the exact threshold by
        // digit passes over the keys on chip, then an ordered write (a warp per stretch of the tensor)
        const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
        const uint32_t n = L.n, k = L.k;
        for (uint32_t i = threadIdx.x; i < n; i += kT) s_keys[i] = magnitude_key(first[i]);
        __syncthreads();
        // k-th largest key; with k = n every entry is kept (T = 0: all keys are above or equal)
        const uint32_t T = k < n ? smem_kth_largest<kT>(s_keys, n, k, s_hist, s_warp, s_bc) : 0u;
        const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, lt = (1u << lane) - 1u;
        constexpr uint32_t kWarps = kT / 32;
        const uint32_t seg = (((n + kWarps - 1) / kWarps) + 31) & ~31u;    // entries per warp, a multiple of 32
        const uint32_t e0 = warp * seg < n ? warp * seg : n, e1 = e0 + seg < n ? e0 + seg : n;
        uint32_t gt = 0, eq = 0;
        for (uint32_t e = e0 + lane; e < e1; e += 32) {
            const uint32_t key = s_keys[e];
            gt += key > T ? 1u : 0u;
            eq += key == T ? 1u : 0u;
        }
#pragma unroll
        for (int d = 16; d; d >>= 1) {
            gt += __shfl_xor_sync(0xFFFFFFFFu, gt, d);
            eq += __shfl_xor_sync(0xFFFFFFFFu, eq, d);
        }
        if (lane == 0) { s_hist[warp] = gt; s_hist[32 + warp] = eq; }
        __syncthreads();
        // every warp works out where all stretches begin: lane j stands for warp j's stretch
        const uint32_t gt_j = lane < kWarps ? s_hist[lane] : 0u, eq_j = lane < kWarps ? s_hist[32 + lane] : 0u;
        uint32_t n_gt = gt_j, eq_inc = eq_j;
#pragma unroll
        for (int d = 16; d; d >>= 1) n_gt += __shfl_xor_sync(0xFFFFFFFFu, n_gt, d);
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, eq_inc, d);
            if (lane >= static_cast<uint32_t>(d)) eq_inc += y;
        }
        const uint32_t r = k - n_gt;                            // entries equal to T to keep: the lowest indices
        const uint32_t eq_before_j = eq_inc - eq_j;
        const uint32_t eq_kept_j = r > eq_before_j ? (r - eq_before_j < eq_j ? r - eq_before_j : eq_j) : 0u;
        uint32_t out_inc = gt_j + eq_kept_j;
        const uint32_t kept_j = out_inc;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, out_inc, d);
            if (lane >= static_cast<uint32_t>(d)) out_inc += y;
        }
        uint32_t run_eq = __shfl_sync(0xFFFFFFFFu, eq_before_j, warp);
        uint32_t run_out = __shfl_sync(0xFFFFFFFFu, out_inc - kept_j, warp);
        uint32_t* idx_out = p.idx_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
        float* val_out = p.val_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
        const uint32_t glob = static_cast<uint32_t>(L.offset);
        for (uint32_t base = e0; base < e1; base += 32) {
            const uint32_t e = base + lane;
            const bool valid = e < e1;
            const uint32_t key = valid ? s_keys[e] : 0u;
            const bool is_eq = valid && key == T;
            const uint32_t b_eq = __ballot_sync(0xFFFFFFFFu, is_eq);
            const bool keep = valid && (key > T || (is_eq && run_eq + __popc(b_eq & lt) < r));
            const uint32_t b_keep = __ballot_sync(0xFFFFFFFFu, keep);
            if (keep) {
                const uint32_t pos = run_out + __popc(b_keep & lt);
                idx_out[pos] = glob + e;
                val_out[pos] = first[e];
            }
            run_eq += __popc(b_eq);
            run_out += __popc(b_keep);
        }
        return;
    }
    {   // the scan only writes the table entries of pieces that hold candidates
        uint2* sub_tab = p.sub_tab + (static_cast<uint64_t>(w) * p.span_stride + L.span_base) * kSubsPerSpan;
        for (uint32_t t = threadIdx.x; t < L.n_spans * kSubsPerSpan; t += kT) sub_tab[t] = make_uint2(0u, 0u);
    }

    const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
    const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
    const float4* vec = reinterpret_cast<const float4*>(first - mis);
    const uint32_t m = L.sample, n_chunks = m / 32, stratum = L.n / n_chunks;   // stratum >= 128
    // chunk j: 32 consecutive entries starting at a hashed position inside stratum j, moved up to
    // the next 32-byte boundary; always inside the tensor
    for (uint32_t t = threadIdx.x; t < n_chunks * 8; t += kT) {
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
    const uint32_t t_lo = smem_kth_largest<kT>(s_keys, m, r_lo, s_hist, s_warp, s_bc);
    uint32_t t_hi = r_hi ? smem_kth_largest<kT>(s_keys, m, r_hi, s_hist, s_warp, s_bc) : 0x7FFFFFFFu;
    if (t_hi > 0x7F800000u) t_hi = 0x7FFFFFFFu;       // "no upper bound" (as a float: unordered)
    // the scan compares magnitudes as floats and blanks padding with zeros: it needs a positive,
    // non-NaN lower bound
    const bool usable = t_lo != 0 && t_lo <= 0x7F800000u;
    // with the cluster route switched on (general_only == 2) the tensors that fit it are marked for the cluster kernel
    // (flag 8), the others, as always, for scan / resolve / emit
    if (threadIdx.x == 0) {
        st->t_lo = t_lo;
        st->t_hi = t_hi;
        st->flags = usable ? (general_only == 2 && L.cluster ? 8u : kInstBracket) : kInstGeneral;
    }
}

// ---------------------------------------------------------------------------------------------
// The single pass over the gradient.  A work item is up to kSpansPerBlock consecutive spans of one
// tensor = 64 pieces of 1024 entries, and each of the 8 warps of a block takes 8 of them (round robin),
// entirely on its own: no block-level barrier.  The pieces do not travel through registers: a bulk
// asynchronous copy (cp.async.bulk, completion on an mbarrier of the warp's own) brings a piece into the
// warp's 4 KB buffer in shared memory while the piece after it is prefetched into L2, so loading costs the
// warp two instructions per piece.  One buffer, not a ring: what the kernel needs to keep the memory
// system and the issue slots busy is warps (7 KB of shared memory per warp leave room for four blocks,
// 32 warps, per SM), and the other warps' work covers the wait for a copy that comes from L2.  Per piece:
//   mask     lane L reads ITS 32 consecutive entries of the piece (eight 16-byte reads, the order of
//            the eight rotated by the lane so that the banks are spread) and builds a 32-bit mask of
//            its candidates (key >= t_lo; for non-NaN data |x| >= t as floats is the integer test on
//            the key, and a NaN counts as a candidate): a compare and a predicated OR per entry;
//            entries outside the tensor (the first and the last piece) are cleared from the mask, so
//            no piece needs a path of its own;
//   rank     population counts and one warp scan give every lane the place of its first candidate
//            in index order (lane after lane: a lane's entries are consecutive);
//   place    each lane walks the set bits of its mask and moves value and position, one 8-byte
//            entry per candidate, from the piece's buffer to its place on a shared-memory stage
//            behind the candidates staged before: work in proportion to the candidates, not to
//            the entries.
// Flush, when the stage cannot take the piece just counted and after the last one, while the next
// piece is on its way to L2: a first pass with one lane per staged candidate counts the window
// entries (those not above t_hi; also per piece, for the table) and looks for NaN; two atomics
// reserve room in the candidate and the window list; a second pass writes both lists with
// coalesced stores, window entries ranked by ballot.  A piece with more candidates than the stage
// holds (a stretch of large entries) goes to the lists directly, each lane writing its own.
// Candidates stay in index order inside a piece; the table records, per piece, where its candidates
// are in the list, how many, and how many of them lie above the window.  A NaN hands the instance to
// the general route, which works on bit patterns only.
constexpr uint32_t kDenseStage = 352;                          // candidates the stage holds; a piece that brings more is written directly
constexpr uint32_t kDenseRing = 1;                             // piece buffers per warp
constexpr uint32_t kPieceBytes = kSubElems * 4;
constexpr size_t kDenseSmemPerWarp = kDenseRing * kPieceBytes + kDenseStage * 8 + 64 + 16;
static_assert(kDenseSmemPerWarp % 16 == 0, "the warps' slices stay 16-byte aligned");
constexpr uint32_t kWaitSpins = 1u << 20;                      // bounded wait for a bulk copy (each try suspends for a while)

__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t mbar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
    return ok != 0;
}
// bytes: a multiple of 16; both addresses 16-byte aligned.  The copy lands in this block only (a plain bulk copy).
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* gmem_src, uint32_t bytes, uint32_t mbar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(gmem_src), "r"(bytes), "r"(mbar) : "memory");
}

// mask |= kBit << c for each of the four components c with |x| >= t or unordered
template <uint32_t kBit>
__device__ __forceinline__ void mask_or(const float4& x, float t, uint32_t& mask) {
    asm("{\n\t"
        ".reg .pred p;\n\t"
        ".reg .f32 a;\n\t"
        "abs.f32 a, %1;\n\t"
        "setp.geu.f32 p, a, %5;\n\t"
        "@p or.b32 %0, %0, %6;\n\t"
        "abs.f32 a, %2;\n\t"
        "setp.geu.f32 p, a, %5;\n\t"
        "@p or.b32 %0, %0, %7;\n\t"
        "abs.f32 a, %3;\n\t"
        "setp.geu.f32 p, a, %5;\n\t"
        "@p or.b32 %0, %0, %8;\n\t"
        "abs.f32 a, %4;\n\t"
        "setp.geu.f32 p, a, %5;\n\t"
        "@p or.b32 %0, %0, %9;\n\t"
        "}"
        : "+r"(mask)
        : "f"(x.x), "f"(x.y), "f"(x.z), "f"(x.w), "f"(t), "n"(kBit), "n"(kBit << 1), "n"(kBit << 2), "n"(kBit << 3));
}

__global__ void __launch_bounds__(kThreads, 4) k_bracket_scan(SelectParams p) {
    extern __shared__ __align__(16) unsigned char s_scan[];
    const uint2 item = p.items[blockIdx.x];
    const uint32_t l = item.x, w = blockIdx.y;
    const Layer L = p.layers[l];
    Inst* st = &p.inst[w * p.n_layers + l];
    if (!(__ldcg(&st->flags) & kInstBracket)) return;
    const float tlo_f = __uint_as_float(__ldcg(&st->t_lo)), thi_f = __uint_as_float(__ldcg(&st->t_hi));
    const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
    const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
    const float4* vec = reinterpret_cast<const float4*>(first - mis);
    const uint32_t n_shift = L.n + mis;                        // n <= kBracketMaxN on this route
    const uint32_t nvec = (n_shift + 3) >> 2;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    constexpr uint32_t kStep = kThreads / 32;
    constexpr uint32_t kBatch = kSpansPerBlock * kSubsPerSpan / kStep;
    static_assert(kStep == 8, "the piece of a staged position is found with a shift");
    const uint32_t ss_end = min(item.y + kSpansPerBlock, L.n_spans) * kSubsPerSpan;
    const uint32_t ss0 = item.y * kSubsPerSpan + warp;
    if (ss0 >= ss_end) return;
    unsigned char* mine = s_scan + warp * kDenseSmemPerWarp;
    uint2* stage = reinterpret_cast<uint2*>(mine + kDenseRing * kPieceBytes);                   // [kDenseStage] (value bits, shifted position)
    uint32_t* s_tc = reinterpret_cast<uint32_t*>(mine + kDenseRing * kPieceBytes + kDenseStage * 8);   // [8] candidates per piece
    uint32_t* s_tw = s_tc + kBatch;                                                           // [8] window entries per piece
    const uint32_t ring_base = static_cast<uint32_t>(__cvta_generic_to_shared(mine));
    const uint32_t stage_base = static_cast<uint32_t>(__cvta_generic_to_shared(stage));
    const uint32_t mbar_base = stage_base + kDenseStage * 8 + 64;                             // [kDenseRing] one mbarrier per buffer
    uint32_t* cand_idx = p.cand_idx + static_cast<uint64_t>(w) * p.cand_stride + L.cand_base;
    float* cand_val = p.cand_val + static_cast<uint64_t>(w) * p.cand_stride + L.cand_base;
    uint32_t* win_key = p.win_key + static_cast<uint64_t>(w) * p.win_stride + L.win_base;
    uint32_t* win_idx = p.win_idx + static_cast<uint64_t>(w) * p.win_stride + L.win_base;
    uint2* sub_tab = p.sub_tab + (static_cast<uint64_t>(w) * p.span_stride + L.span_base) * kSubsPerSpan;

    // this warp's pieces: ss0 + kStep * j, j < n_mine; every one of them overlaps the tensor
    uint32_t n_mine = 0;
    while (n_mine < kBatch && ss0 + kStep * n_mine < ss_end && (ss0 + kStep * n_mine) * (kSubElems / 4) < nvec) ++n_mine;
    if (n_mine == 0) return;
    // the copy of piece j into buffer j % kDenseRing: the 16-byte groups of the piece that overlap the tensor
    auto fetch = [&](uint32_t j) {
        const uint32_t vec0 = (ss0 + kStep * j) * (kSubElems / 4);
        const uint32_t groups = nvec - vec0 < kSubElems / 4 ? nvec - vec0 : kSubElems / 4;
        const uint32_t mbar = mbar_base + 8u * (j % kDenseRing);
        mbar_expect_tx(mbar, groups * 16u);
        bulk_load(ring_base + (j % kDenseRing) * kPieceBytes, vec + vec0, groups * 16u, mbar);
        if (j + 1 < n_mine) {                                  // the piece after it: on its way to L2 meanwhile
            const uint32_t v1 = (ss0 + kStep * (j + 1)) * (kSubElems / 4);
            const uint32_t g1 = nvec - v1 < kSubElems / 4 ? nvec - v1 : kSubElems / 4;
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(vec + v1), "r"(g1 * 16u) : "memory");
        }
    };
    if (lane == 0) {
#pragma unroll
        for (uint32_t r = 0; r < kDenseRing; ++r) mbar_init(mbar_base + 8u * r, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (uint32_t j = 0; j < kDenseRing && j < n_mine; ++j) fetch(j);
    }
    __syncwarp();

    bool saw_nan = false, lost = false;                        // lost: something did not fit, or a copy never arrived
    uint32_t staged = 0, j_first = 0;                          // candidates on the stage; first piece they belong to
    // everything staged since the last flush (pieces j_first .. j_end - 1) goes to the lists
    auto flush = [&](uint32_t j_end) {
        if (staged) {
            if (lane < kBatch) s_tw[lane] = 0;
            __syncwarp();
            uint32_t tw = 0;
#pragma unroll 1
            for (uint32_t r0 = 0; r0 < staged; r0 += 32) {         // window entries: how many, and per piece
                const uint32_t r = r0 + lane;
                bool isw = false;
                if (r < staged) {
                    const uint2 c = stage[r];
                    const float a = fabsf(__uint_as_float(c.x));
                    saw_nan |= a != a;
                    isw = !(a > thi_f);
                    if (isw) atomicAdd(&s_tw[((c.y >> 10) - ss0) >> 3], 1u);
                }
                tw += __popc(__ballot_sync(0xFFFFFFFFu, isw));
            }
            uint32_t old_c = 0, old_w = 0;
            if (lane == 0) {
                old_c = atomicAdd(&st->cand_count, staged);    // room in the candidate list
                if (tw) old_w = atomicAdd(&st->win_count, tw); // room in the window list
            }
            __syncwarp();
            // where each piece's candidates begin
            const bool mine_in = lane >= j_first && lane < j_end;
            const uint32_t tcj = mine_in ? s_tc[lane] : 0u, twj = mine_in ? s_tw[lane] : 0u;
            uint32_t inc = tcj;
#pragma unroll
            for (int d = 1; d < static_cast<int>(kBatch); d <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= static_cast<uint32_t>(d)) inc += y;
            }
            const uint32_t cb = __shfl_sync(0xFFFFFFFFu, old_c, 0), wb = __shfl_sync(0xFFFFFFFFu, old_w, 0);
            if (tcj) sub_tab[ss0 + kStep * lane] = make_uint2(cb + inc - tcj, tcj | ((tcj - twj) << 16));
            if (static_cast<uint64_t>(cb) + staged > L.cand_cap || static_cast<uint64_t>(wb) + tw > L.win_cap) {
                lost = true;
            } else {
                uint32_t wr = wb;
#pragma unroll 1
                for (uint32_t r0 = 0; r0 < staged; r0 += 32) {
                    const uint32_t r = r0 + lane;
                    bool isw = false;
                    uint2 c = make_uint2(0u, 0u);
                    if (r < staged) {
                        c = stage[r];
                        cand_idx[cb + r] = c.y;
                        cand_val[cb + r] = __uint_as_float(c.x);
                        isw = !(fabsf(__uint_as_float(c.x)) > thi_f);
                    }
                    const uint32_t bw = __ballot_sync(0xFFFFFFFFu, isw);
                    if (isw) {
                        const uint32_t o = wr + __popc(bw & lt);
                        win_idx[o] = c.y;
                        win_key[o] = c.x & 0x7FFFFFFFu;          // the magnitude key
                    }
                    wr += __popc(bw);
                }
            }
            __syncwarp();                                     // the stage is reused
        }
        staged = 0;
        j_first = j_end;
    };

    const uint32_t lane_base = lane * 128u, rot = (lane & 7u) << 4;   // the lane's 128 bytes of a buffer; its rotation of the 16-byte groups
#pragma unroll 1
    for (uint32_t j = 0; j < n_mine; ++j) {
        const uint32_t ss = ss0 + kStep * j;
        const uint32_t buf = ring_base + (j % kDenseRing) * kPieceBytes;
        {   // the copy of this piece has landed (bounded wait: a copy that never arrives must not hang the GPU)
            const uint32_t mbar = mbar_base + 8u * (j % kDenseRing), parity = (j / kDenseRing) & 1u;
            uint32_t spins = 0;
            while (!mbar_try_wait(mbar, parity) && ++spins <= kWaitSpins) {}
            if (__any_sync(0xFFFFFFFFu, spins > kWaitSpins)) {
                // give up on the instance (the general route redoes it), but not before the copies still
                // under way have had a second, equally bounded, chance to land: the block must not end under them
                lost = true;
                record_error(p.status, ADACOMP_ERR_TIMEOUT);
                for (uint32_t jj = j; jj < n_mine && jj < j + kDenseRing; ++jj) {
                    spins = 0;
                    while (!mbar_try_wait(mbar_base + 8u * (jj % kDenseRing), (jj / kDenseRing) & 1u) && ++spins <= kWaitSpins) {}
                }
                break;
            }
        }
        // ---- mask of the lane's candidates among its 32 consecutive entries
        const uint32_t e_lane = ss * kSubElems + lane * 32u;   // shifted position of the lane's first entry
        uint32_t mask = 0;
        {
            float4 q[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)                        // group i ^ (lane & 7) first: the eight lanes of a quarter warp hit distinct banks
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(q[i].x), "=f"(q[i].y), "=f"(q[i].z), "=f"(q[i].w)
                             : "r"(buf + lane_base + ((static_cast<uint32_t>(i) << 4) ^ rot)));
            // q[i] holds group i ^ (lane & 7), i.e. entries 4 * (i ^ (lane & 7)) ..: the bits are put where they belong below
            uint32_t raw = 0;                                  // bit 4 i + c: component c of q[i]
            mask_or<1u << 0>(q[0], tlo_f, raw);  mask_or<1u << 4>(q[1], tlo_f, raw);
            mask_or<1u << 8>(q[2], tlo_f, raw);  mask_or<1u << 12>(q[3], tlo_f, raw);
            mask_or<1u << 16>(q[4], tlo_f, raw); mask_or<1u << 20>(q[5], tlo_f, raw);
            mask_or<1u << 24>(q[6], tlo_f, raw); mask_or<1u << 28>(q[7], tlo_f, raw);
            // nibble i of raw is group i ^ r of the lane (r = lane & 7): nibble g of mask = nibble g ^ r of raw.
            // XOR with r permutes the nibbles in three steps, one per bit of r: swap neighbours, pairs, halves.
            const uint32_t r = lane & 7u;
            uint32_t m = raw;
            if (r & 1u) m = ((m & 0x0F0F0F0Fu) << 4) | ((m >> 4) & 0x0F0F0F0Fu);
            if (r & 2u) m = ((m & 0x00FF00FFu) << 8) | ((m >> 8) & 0x00FF00FFu);
            if (r & 4u) m = (m << 16) | (m >> 16);
            mask = m;
        }
        {   // entries before the tensor's first or at / after its end do not count
            const uint32_t lo_cut = mis > e_lane ? mis - e_lane : 0u;                       // <= 3
            const uint32_t hi_cut = n_shift > e_lane ? (n_shift - e_lane < 32u ? n_shift - e_lane : 32u) : 0u;
            const uint32_t keep = (hi_cut == 32u ? 0xFFFFFFFFu : (1u << hi_cut) - 1u) & ~((1u << lo_cut) - 1u);
            mask &= keep;
        }
        // ---- rank: where the lane's first candidate goes
        const uint32_t cnt = __popc(mask);
        uint32_t inc = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= static_cast<uint32_t>(d)) inc += y;
        }
        uint32_t tc = __shfl_sync(0xFFFFFFFFu, inc, 31);
        if (staged + tc > kDenseStage) flush(j);               // make room first (pieces before this one)
        if (tc > kDenseStage) {
            // ---- a crowded piece does not fit the stage: its candidates go to the lists directly, every lane
            // its own run (rare: a stretch in which most entries are large)
            uint32_t wcnt = 0;
            for (uint32_t m = mask; m; m &= m - 1u) {
                const float a = fabsf(*reinterpret_cast<const float*>(mine + (j % kDenseRing) * kPieceBytes + lane_base + ((__ffs(m) - 1u) << 2)));
                saw_nan |= a != a;
                wcnt += !(a > thi_f) ? 1u : 0u;
            }
            uint32_t winc = wcnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, winc, d);
                if (lane >= static_cast<uint32_t>(d)) winc += y;
            }
            const uint32_t tw = __shfl_sync(0xFFFFFFFFu, winc, 31);
            uint32_t old_c = 0, old_w = 0;
            if (lane == 0) {
                old_c = atomicAdd(&st->cand_count, tc);
                if (tw) old_w = atomicAdd(&st->win_count, tw);
            }
            const uint32_t cb = __shfl_sync(0xFFFFFFFFu, old_c, 0), wb = __shfl_sync(0xFFFFFFFFu, old_w, 0);
            if (lane == 0) sub_tab[ss] = make_uint2(cb, tc | ((tc - tw) << 16));
            if (static_cast<uint64_t>(cb) + tc > L.cand_cap || static_cast<uint64_t>(wb) + tw > L.win_cap) {
                lost = true;
            } else {
                uint32_t o = cb + inc - cnt, wo = wb + winc - wcnt;
                for (uint32_t m = mask; m; m &= m - 1u) {
                    const uint32_t b = __ffs(m) - 1u;
                    const float v = *reinterpret_cast<const float*>(mine + (j % kDenseRing) * kPieceBytes + lane_base + (b << 2));
                    cand_idx[o] = e_lane + b;
                    cand_val[o] = v;
                    ++o;
                    if (!(fabsf(v) > thi_f)) {
                        win_idx[wo] = e_lane + b;
                        win_key[wo] = magnitude_key(v);
                        ++wo;
                    }
                }
            }
            tc = 0;                                            // nothing of this piece is on the stage or in a later flush
        }
        if (tc) {
            // ---- place: walk the set bits, value and position from the piece's buffer to the stage
            uint32_t o = stage_base + 8u * (staged + inc - cnt);
            uint32_t m = mask;
            const uint32_t turns = __reduce_max_sync(0xFFFFFFFFu, cnt);
#pragma unroll 1
            for (uint32_t t = 0; t < turns; ++t) {
                if (m) {
                    const uint32_t b = __ffs(m) - 1u;
                    m &= m - 1u;
                    uint32_t v;
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(buf + lane_base + (b << 2)));   // the buffer holds the piece as it is in memory
                    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(o), "r"(v), "r"(e_lane + b) : "memory");
                    o += 8u;
                }
            }
        }
        if (lane == 0) s_tc[j] = tc;
        staged += tc;
        __syncwarp();                                          // the buffer has been read by every lane, the stage written
        if (lane == 0 && j + kDenseRing < n_mine) fetch(j + kDenseRing);
    }
    flush(n_mine);
    if (saw_nan || lost) atomicOr(&st->flags, kInstOverflow);
}

// ---------------------------------------------------------------------------------------------
// One block per instance: exact threshold inside the window, per-span output offsets.
template <int kT>
__global__ void __launch_bounds__(kT) k_bracket_resolve(SelectParams p) {
    __shared__ uint32_t s_hist[2048];
    __shared__ uint32_t s_sel[kMaxSpans];
    __shared__ unsigned long long s_g[kGatherMax];
    __shared__ uint32_t s_warp[33];
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
    const uint32_t n_cand = __ldcg(&st->cand_count), n_win = __ldcg(&st->win_count);
    const uint32_t n_def = n_cand - n_win;            // entries above the window
    const uint32_t t_lo = __ldcg(&st->t_lo), t_hi = __ldcg(&st->t_hi);
    const bool bad = (flags & kInstOverflow) || n_cand > L.cand_cap || n_win > L.win_cap || n_def > L.k ||
                     L.k - n_def > n_win;
    if (bad) {                                        // the bracket missed: hand over, state is still pristine
        if (threadIdx.x == 0) st->flags = kInstGeneral;
        return;
    }
    const uint32_t* win_key = p.win_key + static_cast<uint64_t>(w) * p.win_stride + L.win_base;
    const uint32_t* win_idx = p.win_idx + static_cast<uint64_t>(w) * p.win_stride + L.win_base;
    const uint2* sub_tab = p.sub_tab + (static_cast<uint64_t>(w) * p.span_stride + L.span_base) * kSubsPerSpan;
    uint32_t* span_off = p.span_off + static_cast<uint64_t>(w) * p.span_stride + L.span_base;
    const uint32_t need = L.k - n_def;

    // composite of a window entry = (key - t_lo) << 32 | ~index: larger = kept first (larger key,
    // then lower index)
    // calls fn(composite, shifted index) for every window entry; eight entries per thread are
    // fetched before any is used, so their loads overlap (a pass over the list is bound by their latency)
    auto for_each_window = [&](auto fn) {
        constexpr int kAhead = 8;
        for (uint32_t i0 = threadIdx.x; i0 < n_win; i0 += kT * kAhead) {
            uint32_t key[kAhead], idx[kAhead];
#pragma unroll
            for (int u = 0; u < kAhead; ++u) {
                const uint32_t i = i0 + u * kT;
                key[u] = i < n_win ? __ldcg(&win_key[i]) : 0u;
                idx[u] = i < n_win ? __ldcg(&win_idx[i]) : 0u;
            }
#pragma unroll
            for (int u = 0; u < kAhead; ++u)
                if (i0 + u * kT < n_win)
                    fn((static_cast<unsigned long long>(key[u] - t_lo) << 32) |
                           static_cast<unsigned long long>(0xFFFFFFFFu - idx[u]),
                       idx[u]);
        }
    };
    // kept window entries per span: counted in shared memory, or for very long tensors in the table
    // that receives the spans' output offsets anyway.  The pass that collects the last undecided entries
    // also counts the entries it sees above them, so the list is not read again once the threshold is known.
    uint32_t* sel = L.n_spans <= kMaxSpans ? s_sel : span_off;
    for (uint32_t s = threadIdx.x; s < L.n_spans; s += kT) sel[s] = 0;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    bool failed = false;

    unsigned long long cstar = ~0ull;                 // keep window entries with composite >= cstar
    if (need > 0) {
        const uint32_t range = t_hi - t_lo;
        int hi_shift = (range ? 32 - __clz(range) : 0) + 32;   // undecided low bits of the composite (<= 63)
        unsigned long long prefix = 0;
        uint32_t rem = need, count = n_win;
        while (true) {
            if (count <= kGatherMax) {                // few left: gather them and rank by brute force
                if (threadIdx.x == 0) s_cnt = 0;
                __syncthreads();
                for_each_window([&](unsigned long long c, uint32_t idx) {
                    const unsigned long long top = c >> hi_shift;
                    if (top == prefix) s_g[atomicAdd(&s_cnt, 1u)] = c;
                    else if (top > prefix) atomicAdd(&sel[idx / kSpanElems], 1u);   // above the undecided ones: kept
                });
                __syncthreads();
                for (uint32_t t = threadIdx.x; t < count; t += kT) {
                    const unsigned long long mine = s_g[t];
                    uint32_t larger = 0;
                    for (uint32_t u = 0; u < count; ++u) larger += s_g[u] > mine ? 1u : 0u;
                    if (larger == rem - 1) s_cstar = mine;
                }
                __syncthreads();
                cstar = s_cstar;
                for (uint32_t t = threadIdx.x; t < count; t += kT)      // the kept ones among the collected entries
                    if (s_g[t] >= cstar) atomicAdd(&sel[(0xFFFFFFFFu - static_cast<uint32_t>(s_g[t])) / kSpanElems], 1u);
                break;
            }
            if (hi_shift == 0) { failed = true; break; }      // cannot happen: composites are distinct
            const int bits = hi_shift < 11 ? hi_shift : 11;
            const int new_shift = hi_shift - bits;
            for (int b = threadIdx.x; b < 2048; b += kT) s_hist[b] = 0;
            __syncthreads();
            for_each_window([&](unsigned long long c, uint32_t) {
                if ((c >> hi_shift) == prefix)
                    atomicAdd(&s_hist[static_cast<uint32_t>(c >> new_shift) & ((1u << bits) - 1u)], 1u);
            });
            __syncthreads();
            uint32_t b, above, cnt;
            block_pick_bucket<kT>(s_hist, rem, &b, &above, &cnt, s_warp, s_bc);
            prefix = (prefix << bits) | b;
            rem -= above;
            count = cnt;
            hi_shift = new_shift;
        }
    }
    __syncthreads();
    // exclusive prefix of kept entries over the spans
    for (uint32_t base = 0; base < L.n_spans; base += kT) {
        const uint32_t s = base + threadIdx.x;
        uint32_t kept = 0;
        if (s < L.n_spans) {
            kept = sel == s_sel ? s_sel[s] : __ldcg(&sel[s]);
#pragma unroll
            for (uint32_t j = 0; j < kSubsPerSpan; ++j) kept += __ldcg(&sub_tab[s * kSubsPerSpan + j]).y >> 16;
        }
        uint32_t tot;
        const uint32_t ex = block_exclusive_scan_t<kT>(kept, &tot, s_warp);
        const uint32_t carry = s_carry;
        if (s < L.n_spans) span_off[s] = carry + ex;
        __syncthreads();
        if (threadIdx.x == 0) s_carry = carry + tot;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (failed || s_carry != L.k) {
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
// grid = (scan items, workers); one warp per span: walk the candidates of its 8 pieces in index
// order, keep those at or above the exact threshold, write them out contiguously.
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
    const uint64_t span_at = static_cast<uint64_t>(w) * p.span_stride + L.span_base + s;
    uint2 tab = make_uint2(0, 0);
    if (lane < kSubsPerSpan) tab = __ldcg(&p.sub_tab[span_at * kSubsPerSpan + lane]);
    const uint32_t cnt = tab.y & 0xFFFFu;
    uint32_t inc = cnt;                                        // inclusive prefix over the 8 pieces
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += y;
    }
    const uint32_t pre = inc - cnt;
    const uint32_t total = __shfl_sync(0xFFFFFFFFu, inc, kSubsPerSpan - 1);
    uint32_t off = __ldcg(&p.span_off[span_at]);
    uint32_t* idx_out = p.idx_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
    float* val_out = p.val_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t glob = static_cast<uint32_t>(L.offset) - mis;        // shifted coordinate -> vector index
    // where each piece's candidates start in the span's flattened order (warp-uniform registers):
    // flattened position f of piece j lives at slot f + delta[j]
    uint32_t start[kSubsPerSpan], delta[kSubsPerSpan];
#pragma unroll
    for (int j = 0; j < static_cast<int>(kSubsPerSpan); ++j) {
        start[j] = __shfl_sync(0xFFFFFFFFu, pre, j);
        delta[j] = __shfl_sync(0xFFFFFFFFu, tab.x, j) - start[j];
    }
    constexpr int kUnroll = 4;                                 // 128 candidates in flight per warp
    for (uint32_t f0 = 0; f0 < total; f0 += 32 * kUnroll) {
        uint32_t e[kUnroll];
        float v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t f = f0 + u * 32 + lane;
            uint32_t d = delta[0];
#pragma unroll
            for (int j = 1; j < static_cast<int>(kSubsPerSpan); ++j)
                if (f >= start[j]) d = delta[j];               // starts never decrease: the last match wins
            e[u] = 0;
            v[u] = 0.f;
            if (f < total) {
                e[u] = __ldcs(&cand_idx[f + d]);
                v[u] = __ldcs(&cand_val[f + d]);
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t key = magnitude_key(v[u]);
            const bool keep = (f0 + u * 32 + lane < total) && (key > T || (key == T && e[u] < cut));
            const uint32_t b = __ballot_sync(0xFFFFFFFFu, keep);
            if (keep) {
                const uint32_t pos = off + __popc(b & lt);
                __stcs(&idx_out[pos], glob + e[u]);              // written once, read by another kernel much later
                __stcs(&val_out[pos], v[u]);
            }
            off += __popc(b);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// The same ordered write for calls whose tensors have a handful of candidates per piece (low keep fractions): there
// the kernel above spends a warp, and its whole set-up, on a span with a dozen candidates, and is bound by instruction
// issue.  Here a LANE takes a piece and a warp four spans: the lane reads its piece's table entry, walks the piece's
// candidates once to count the kept ones (remembering which of the first 32), a scan over the eight lanes of a span
// gives it its place behind the span's output offset, and it walks them again to write.  grid = (scan items,
// workers), two warps per block.  Any data is handled, only not fast when pieces hold many candidates.
constexpr int kEmitThinThreads = 64;
__global__ void __launch_bounds__(kEmitThinThreads) k_bracket_emit_thin(SelectParams p) {
    const uint2 item = p.items[blockIdx.x];
    const uint32_t l = item.x, w = blockIdx.y;
    const Layer L = p.layers[l];
    const Inst* st = &p.inst[w * p.n_layers + l];
    if (!(__ldcg(&st->flags) & kInstBracket)) return;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t sub = lane & 7u;
    const uint32_t s = item.y + warp * 4 + (lane >> 3);        // kSpansPerBlock = 8 spans per item: two warps, four spans each
    static_assert(kSpansPerBlock == 8 && kSubsPerSpan == 8, "a lane per piece, eight lanes per span, two warps per item");
    const bool valid = s < L.n_spans;
    const uint32_t T = __ldcg(&st->T), cut = __ldcg(&st->cut);
    const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
    const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
    const uint32_t* cand_idx = p.cand_idx + static_cast<uint64_t>(w) * p.cand_stride + L.cand_base;
    const float* cand_val = p.cand_val + static_cast<uint64_t>(w) * p.cand_stride + L.cand_base;
    const uint64_t span_at = static_cast<uint64_t>(w) * p.span_stride + L.span_base + s;
    uint2 tab = make_uint2(0, 0);
    uint32_t off = 0;
    if (valid) {
        tab = __ldcg(&p.sub_tab[span_at * kSubsPerSpan + sub]);
        off = __ldcg(&p.span_off[span_at]);
    }
    const uint32_t cnt = tab.y & 0xFFFFu, at = tab.x;
    uint32_t kept = 0, keep_mask = 0;
    for (uint32_t i = 0; i < cnt; ++i) {
        const uint32_t e = __ldg(&cand_idx[at + i]);
        const uint32_t key = magnitude_key(__ldg(&cand_val[at + i]));
        const uint32_t k = (key > T || (key == T && e < cut)) ? 1u : 0u;
        kept += k;
        if (i < 32) keep_mask |= k << i;
    }
    uint32_t inc = kept;                                       // inclusive prefix over the 8 pieces of the span
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (sub >= static_cast<uint32_t>(d)) inc += y;
    }
    if (!kept) return;
    uint32_t pos = off + inc - kept;
    uint32_t* idx_out = p.idx_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
    float* val_out = p.val_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
    const uint32_t glob = static_cast<uint32_t>(L.offset) - mis;        // shifted coordinate -> vector index
    for (uint32_t i = 0; i < cnt; ++i) {
        const uint32_t e = __ldg(&cand_idx[at + i]);
        const float v = __ldg(&cand_val[at + i]);
        bool keep;
        if (i < 32) {
            keep = (keep_mask >> i) & 1u;
        } else {
            const uint32_t key = magnitude_key(v);
            keep = key > T || (key == T && e < cut);
        }
        if (keep) {
            __stcs(&idx_out[pos], glob + e);
            __stcs(&val_out[pos], v);
            ++pos;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// The general route done by ONE block per instance, for layouts whose tensors are all on a single-pass
// route: only instances whose bracket missed (or that hold a NaN) are flagged then, which is rare, so
// one launch that usually finds nothing replaces the general route's six.  A block takes the flagged
// instances blockIdx.x, blockIdx.x + gridDim.x, ... and does for each what the general route does:
// three digit passes over bits [30:20], [19:10], [9:0] of the keys give the exact k-th largest key T,
// then one more pass writes, in index order, every entry with key > T and the r lowest-index entries
// with key == T (a block walks its tensor front to back, so the running counts are simply carried
// along: no count pass).  Four reads of the tensor, the later ones mostly from L2.
__global__ void __launch_bounds__(kSoloThreads) k_fallback_solo(SelectParams p) {
    __shared__ uint32_t s_hist[2048];
    __shared__ uint32_t s_warp[33];
    __shared__ uint32_t s_bc[3];
    const uint32_t n_inst = p.n_workers * p.n_layers;
    for (uint32_t inst = blockIdx.x; inst < n_inst; inst += gridDim.x) {
        Inst* st = &p.inst[inst];
        if (!(__ldcg(&st->flags) & kInstGeneral)) continue;      // the same for every thread of the block
        const uint32_t w = inst / p.n_layers, l = inst - w * p.n_layers;
        const Layer L = p.layers[l];
        if (L.k == 0) continue;
        const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
        const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
        const float4* vec = reinterpret_cast<const float4*>(first - mis);
        const uint64_t n_shift = static_cast<uint64_t>(L.n) + mis, nvec = (n_shift + 3) >> 2;
        uint32_t prefix = 0, rem = L.k;
        if (L.k < L.n) {
#pragma unroll 1
            for (int pass = 0; pass < 3; ++pass) {
                const int shift = pass == 0 ? 20 : (pass == 1 ? 10 : 0);
                const uint32_t nb = pass == 0 ? 2048u : 1024u;
                for (int b = threadIdx.x; b < 2048; b += kSoloThreads) s_hist[b] = 0;
                __syncthreads();
                for (uint64_t base = 0; base < nvec; base += kSoloThreads) {
                    const uint64_t v = base + threadIdx.x;
                    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (v < nvec) x = __ldg(&vec[v]);
                    const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint64_t e = v * 4 + q;
                        const uint32_t key = magnitude_key(xs[q]);
                        const bool on = e >= mis && e < n_shift &&
                                        (pass == 0 || (key >> (shift + 10)) == (prefix >> (shift + 10)));
                        const uint32_t bin = (key >> shift) & (nb - 1u);
                        if (on) atomicAdd(&s_hist[bin], 1u);
                    }
                }
                __syncthreads();
                uint32_t b, above, cnt;
                block_pick_bucket<kSoloThreads>(s_hist, rem, &b, &above, &cnt, s_warp, s_bc);   // unused upper bins are zero
                prefix |= b << shift;
                rem -= above;
            }
        }
        // k = n: prefix = 0 and rem = n keep every entry (all keys are >= 0)
        const uint32_t T = prefix, r = rem;
        uint32_t gt_base = 0, eq_base = 0;
        uint32_t* idx_out = p.idx_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
        float* val_out = p.val_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
        for (uint64_t base = 0; base < nvec; base += kSoloThreads) {
            const uint64_t v = base + threadIdx.x;
            float xs[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t gtm = 0, eqm = 0;
            if (v < nvec) {
                const float4 x = __ldg(&vec[v]);
                xs[0] = x.x; xs[1] = x.y; xs[2] = x.z; xs[3] = x.w;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint64_t e = v * 4 + q;
                    const uint32_t key = magnitude_key(xs[q]);
                    const bool ok = e >= mis && e < n_shift;
                    gtm |= (ok && key > T) ? (1u << q) : 0u;
                    eqm |= (ok && key == T) ? (1u << q) : 0u;
                }
            }
            // a tile holds 4096 entries: both counts fit 16 bits only up to 4095, so they are scanned apart
            uint32_t tot_gt, tot_eq;
            uint32_t gt_before = gt_base + block_exclusive_scan_t<kSoloThreads>(__popc(gtm), &tot_gt, s_warp);
            uint32_t eq_before = eq_base + block_exclusive_scan_t<kSoloThreads>(__popc(eqm), &tot_eq, s_warp);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bool is_gt = (gtm >> q) & 1u, is_eq = (eqm >> q) & 1u;
                if (is_gt || (is_eq && eq_before < r)) {
                    const uint32_t pos = gt_before + (eq_before < r ? eq_before : r);
                    idx_out[pos] = static_cast<uint32_t>(L.offset + (v * 4 + q - mis));
                    val_out[pos] = xs[q];
                }
                gt_before += is_gt ? 1u : 0u;
                eq_before += is_eq ? 1u : 0u;
            }
            gt_base += tot_gt;
            eq_base += tot_eq;
        }
        if (threadIdx.x == 0) atomicAdd(&p.list_len[0], 1u);       // reported as "took the general route"
        __syncthreads();
    }
}

}  // namespace adacomp
