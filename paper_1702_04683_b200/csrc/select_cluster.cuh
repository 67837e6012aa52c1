// SELECT_GRAD (Algorithm 1), cluster route: a large tensor is selected by ONE thread-block cluster that
// keeps everything between the single pass over the gradient and the ordered write ON CHIP, in the
// distributed shared memory of its blocks.  DRAM sees the gradient once (4 bytes per entry) and the
// output once (8 bytes per kept entry): the algorithmic traffic of SELECT_GRAD, nothing else.
//
// A cluster of C blocks (8, or 16 where the device allows) takes one (worker, tensor) instance at a time;
// block r owns a contiguous run of the tensor's 1024-entry pieces.  Per instance:
//   pass     every warp streams its pieces through a ring of 4 KB shared-memory buffers filled by bulk
//            asynchronous copies (cp.async.bulk + an mbarrier per buffer, the warp's own), exactly as the
//            list route's scan kernel does.  A lane reads its 32 consecutive entries, builds the mask of
//            its candidates (key >= t_lo, the lower bracket bound from the sample kernel) and copies the
//            candidates' VALUES, in index order, into the block's value store; the piece's 1024-bit mask
//            and where its values start are kept too.  Positions are never stored: mask + order give
//            them back.
//   select   the k-th largest candidate key, exactly: digit passes over the keys in the value stores
//            (bins of the undecided key range, shared-memory histograms, summed over the cluster
//            through distributed shared memory so that every block picks the same bin), two or three
//            passes until the range is one key T; r = how many entries equal to T are kept.
//   count    per piece (one thread each) the candidates above T and equal to T; prefix sums over the
//            pieces of a block and, through one exchange, over the blocks give every piece its place in
//            the output and the rank of its first tie (the r lowest-index ties are the ones kept).
//   write    per piece (one thread each) a walk over the mask's set bits writes the kept (index, value)
//            pairs.
// Between the steps stands the cluster's hardware barrier; no block waits on a flag, and none leaves
// while its shared memory may still be read.  If a store overflows, a NaN turns up, or fewer than k
// candidates were seen (the bracket missed), the instance is handed to the general route untouched.
#pragma once

#include <cooperative_groups.h>

#include "select_bracket.cuh"

namespace adacomp {

constexpr int kClMaxThreads = 512;                    // blocks run 8, 12 or 16 warps: more warps where the value store can be smaller
constexpr uint32_t kClPiece = kSubElems;              // entries per piece: 32 per lane
constexpr uint32_t kClPieceBytes = kClPiece * 4;
constexpr uint32_t kClMaxCtas = 16;
constexpr uint32_t kInstCluster = 8u;                 // bracket valid, the cluster kernel acts on the instance
constexpr uint32_t kClMinN = 1u << 20;                // shorter tensors stay on the list route: the barriers would cost more than they save

// Shared memory of one block, in bytes from its start.  The ring is idle after the pass, so the select / count /
// write steps keep their tables in it.
struct ClusterLayout {
    uint32_t ring, mbar, bitmap, pinfo, misc, vals, vals_cap;      // vals_cap: values the store holds
    uint32_t hist, pcount, ppost;                                   // inside the ring
};
__host__ __device__ inline ClusterLayout cluster_layout(uint32_t n_warps, uint32_t ring_slots, uint32_t q_max, uint32_t total_bytes) {
    ClusterLayout y;
    y.ring = 0;
    const uint32_t ring_bytes = n_warps * ring_slots * kClPieceBytes;
    y.hist = 0;                                       // 2048 bins
    y.pcount = 8192;                                  // [q_max] (above T, equal to T)
    y.ppost = 8192 + q_max * 8;                       // [q_max] (above T before the piece, equal to T before it)
    y.mbar = ring_bytes;                              // [warps][ring_slots] mbarriers
    y.bitmap = y.mbar + ((n_warps * ring_slots * 8 + 15) & ~15u);   // [q_max][32] 32-bit masks
    y.pinfo = y.bitmap + q_max * 128;                 // [q_max] first value | count << 21
    y.misc = (y.pinfo + q_max * 4 + 15) & ~15u;       // counters, exchange slots, scan scratch
    y.vals = y.misc + 512;
    y.vals_cap = total_bytes > y.vals ? (total_bytes - y.vals) / 4 : 0;
    if (y.vals_cap > (1u << 21) - 1) y.vals_cap = (1u << 21) - 1;
    return y;
}
// the tables of the later steps must fit the ring
__host__ __device__ inline bool cluster_layout_ok(uint32_t n_warps, uint32_t ring_slots, uint32_t q_max) {
    return 8192 + q_max * 16 <= n_warps * ring_slots * kClPieceBytes;
}

// Block-wide exclusive prefix sum for a block of n_warps (<= 32) full warps.  s_warp needs 33 entries.
__device__ __forceinline__ uint32_t block_exclusive_scan_rt(uint32_t v, uint32_t* total, uint32_t* s_warp, uint32_t n_warps) {
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= static_cast<uint32_t>(d)) inc += y;
    }
    __syncthreads();
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const uint32_t t = lane < n_warps ? s_warp[lane] : 0u;
        uint32_t winc = t;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, winc, d);
            if (lane >= static_cast<uint32_t>(d)) winc += y;
        }
        if (lane < n_warps) s_warp[lane] = winc - t;
        if (lane == 31) s_warp[32] = winc;
    }
    __syncthreads();
    *total = s_warp[32];
    return s_warp[warp] + inc - v;
}

// Descending walk over a 2048-bin histogram in shared memory by the first 256 threads of a block of n_warps warps
// (8 bins each): the bin holding the rem-th largest.  out[0] = bin, out[1] = entries above it, out[2] = its count,
// out[3] = 1 if found.  All threads call.
__device__ __forceinline__ void block_pick_bin(const uint32_t* hist, uint32_t rem, uint32_t* out /*[4] shared*/, uint32_t* s_warp /*[33]*/,
                                               uint32_t n_warps) {
    constexpr int M = 8;
    const bool mine = threadIdx.x < 2048 / M;
    const int top = 2047 - static_cast<int>(threadIdx.x) * M;
    uint32_t h[M], sum = 0;
#pragma unroll
    for (int q = 0; q < M; ++q) { h[q] = mine ? hist[top - q] : 0u; sum += h[q]; }
    if (threadIdx.x == 0) out[3] = 0;
    uint32_t total;
    uint32_t above = block_exclusive_scan_rt(sum, &total, s_warp, n_warps);     // (barriers inside: out[3] = 0 is seen)
#pragma unroll
    for (int q = 0; q < M; ++q) {
        if (mine && above < rem && rem <= above + h[q]) { out[0] = top - q; out[1] = above; out[2] = h[q]; out[3] = 1; }
        above += h[q];
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kClMaxThreads, 1)
k_select_cluster(SelectParams p, const uint32_t* __restrict__ cl_layers, uint32_t n_cl, uint32_t ring_slots, uint32_t q_max,
                 uint32_t smem_bytes) {
    extern __shared__ __align__(16) unsigned char s_cl[];
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t C = cluster.num_blocks(), rank = cluster.block_rank();
    const uint32_t cluster_id = blockIdx.x / C, n_clusters = gridDim.x / C;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n_threads = blockDim.x, n_warps = n_threads >> 5;
    const ClusterLayout Y = cluster_layout(n_warps, ring_slots, q_max, smem_bytes);
    uint32_t* s_bitmap = reinterpret_cast<uint32_t*>(s_cl + Y.bitmap);
    uint32_t* s_pinfo = reinterpret_cast<uint32_t*>(s_cl + Y.pinfo);
    uint32_t* s_vals = reinterpret_cast<uint32_t*>(s_cl + Y.vals);
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(s_cl + Y.hist);
    uint2* s_pcount = reinterpret_cast<uint2*>(s_cl + Y.pcount);
    uint2* s_ppost = reinterpret_cast<uint2*>(s_cl + Y.ppost);
    uint32_t* s_misc = reinterpret_cast<uint32_t*>(s_cl + Y.misc);
    uint32_t* s_used = s_misc + 0;                    // values in the store
    uint32_t* s_over = s_misc + 1;                    // != 0: the store overflowed, or a copy never arrived
    uint32_t* s_above = s_misc + 2;                   // keys above the hinted range (first digit pass)
    uint32_t* s_nan = s_misc + 3;                     // != 0: a NaN among them
    uint32_t* s_x = s_misc + 4;                       // [4] what this block tells the others: used, over, above-T total, equal-T total
    uint32_t* s_bc = s_misc + 8;                      // [4] result of a bin pick
    uint32_t* s_carry = s_misc + 12;                  // [2]
    uint32_t* s_warp = s_misc + 16;                   // [33] scan scratch
    const uint32_t ring_base = static_cast<uint32_t>(__cvta_generic_to_shared(s_cl + Y.ring)) + warp * ring_slots * kClPieceBytes;
    const uint32_t mbar_base = static_cast<uint32_t>(__cvta_generic_to_shared(s_cl + Y.mbar)) + warp * ring_slots * 8;
    const uint32_t vals_base = static_cast<uint32_t>(__cvta_generic_to_shared(s_vals));

    if (lane == 0) {
        for (uint32_t r = 0; r < ring_slots; ++r) mbar_init(mbar_base + 8u * r, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    uint32_t fetched = 0;                             // pieces this warp has fetched since the launch: ring position and phase
    bool dead = false;                                // a copy never arrived: the warp stops fetching, its instances go to the general route

    const uint32_t n_ord = p.n_workers * n_cl;
    for (uint32_t ord = cluster_id; ord < n_ord; ord += n_clusters) {
        const uint32_t w = ord / n_cl, l = cl_layers[ord - w * n_cl];
        const Layer L = p.layers[l];
        Inst* st = &p.inst[w * p.n_layers + l];
        // nobody writes this record before the instance's last barrier: every block reads the same flags
        if (!(__ldcg(&st->flags) & kInstCluster)) continue;
        const uint32_t t_lo = __ldcg(&st->t_lo), t_hi_hint = __ldcg(&st->t_hi);
        const float tlo_f = __uint_as_float(t_lo);
        const float* first = p.grads + static_cast<uint64_t>(w) * p.stride + L.offset;
        const uint32_t mis = static_cast<uint32_t>((reinterpret_cast<uintptr_t>(first) >> 2) & 3u);
        const float4* vec = reinterpret_cast<const float4*>(first - mis);
        const uint32_t n_shift = L.n + mis;
        const uint32_t nvec = (n_shift + 3) >> 2;
        const uint32_t n_pieces = (n_shift + kClPiece - 1) / kClPiece;
        const uint32_t Q = (n_pieces + C - 1) / C;                      // pieces per block (<= q_max by the host's choice of C)
        const uint32_t q0 = rank * Q;
        const uint32_t q_count = q0 < n_pieces ? (n_pieces - q0 < Q ? n_pieces - q0 : Q) : 0u;
        if (threadIdx.x == 0) { *s_used = 0; *s_over = (Q > q_max) ? 1u : 0u; }
        __syncthreads();

        // ============================ pass: candidates' values into the block's store
        // (Q > q_max cannot happen with the host's choice of q_max; if it did the tables would not hold the pieces: nothing is read)
        const uint32_t n_mine = (q_count > warp && !dead && Q <= q_max) ? (q_count - warp + n_warps - 1) / n_warps : 0u;
        auto fetch = [&](uint32_t j) {               // lane 0: piece q0 + warp + n_warps j into ring slot (fetched + j) % ring_slots
            const uint32_t vec0 = (q0 + warp + n_warps * j) * (kClPiece / 4);
            const uint32_t groups = nvec - vec0 < kClPiece / 4 ? nvec - vec0 : kClPiece / 4;
            const uint32_t slot = (fetched + j) % ring_slots;
            mbar_expect_tx(mbar_base + 8u * slot, groups * 16u);
            bulk_load(ring_base + slot * kClPieceBytes, vec + vec0, groups * 16u, mbar_base + 8u * slot);
        };
        if (lane == 0 && n_mine) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the ring held tables written by ordinary stores
            for (uint32_t j = 0; j < ring_slots && j < n_mine; ++j) fetch(j);
        }
        if (dead && q_count > warp && lane == 0) *s_over = 1u;
        const uint32_t lane_base = lane * 128u, rot = (lane & 7u) << 4;   // the lane's 128 bytes of a buffer; its rotation of the 16-byte groups
#pragma unroll 1
        for (uint32_t j = 0; j < n_mine; ++j) {
            const uint32_t u = fetched + j, slot = u % ring_slots;
            {
                const uint32_t mbar = mbar_base + 8u * slot, parity = (u / ring_slots) & 1u;
                uint32_t spins = 0;
                while (!mbar_try_wait(mbar, parity) && ++spins <= kWaitSpins) {}
                if (__any_sync(0xFFFFFFFFu, spins > kWaitSpins)) {
                    // a copy never arrived: give the copies under way a second, equally bounded, chance to land,
                    // then stop using the ring for good (its phases are no longer known)
                    for (uint32_t jj = j; jj < n_mine && jj < j + ring_slots; ++jj) {
                        spins = 0;
                        while (!mbar_try_wait(mbar_base + 8u * ((fetched + jj) % ring_slots), ((fetched + jj) / ring_slots) & 1u) &&
                               ++spins <= kWaitSpins) {}
                    }
                    dead = true;
                    if (lane == 0) { *s_over = 1u; record_error(p.status, ADACOMP_ERR_TIMEOUT); }
                    break;
                }
            }
            const uint32_t lq = warp + n_warps * j;                       // the piece's number inside the block
            const uint32_t e_lane = (q0 + lq) * kClPiece + lane * 32u;    // shifted position of the lane's first entry
            const uint32_t buf = ring_base + slot * kClPieceBytes;
            uint32_t mask;
            {
                float4 q[8];
#pragma unroll
                for (int i = 0; i < 8; ++i)                               // group i ^ (lane & 7) first: the eight lanes of a quarter warp hit distinct banks
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                 : "=f"(q[i].x), "=f"(q[i].y), "=f"(q[i].z), "=f"(q[i].w)
                                 : "r"(buf + lane_base + ((static_cast<uint32_t>(i) << 4) ^ rot)));
                uint32_t raw = 0;                                         // nibble i: group i ^ (lane & 7)
                mask_or<1u << 0>(q[0], tlo_f, raw);  mask_or<1u << 4>(q[1], tlo_f, raw);
                mask_or<1u << 8>(q[2], tlo_f, raw);  mask_or<1u << 12>(q[3], tlo_f, raw);
                mask_or<1u << 16>(q[4], tlo_f, raw); mask_or<1u << 20>(q[5], tlo_f, raw);
                mask_or<1u << 24>(q[6], tlo_f, raw); mask_or<1u << 28>(q[7], tlo_f, raw);
                const uint32_t r7 = lane & 7u;                            // nibble g of the mask = nibble g ^ r7 of raw
                uint32_t m = raw;
                if (r7 & 1u) m = ((m & 0x0F0F0F0Fu) << 4) | ((m >> 4) & 0x0F0F0F0Fu);
                if (r7 & 2u) m = ((m & 0x00FF00FFu) << 8) | ((m >> 8) & 0x00FF00FFu);
                if (r7 & 4u) m = (m << 16) | (m >> 16);
                const uint32_t lo_cut = mis > e_lane ? mis - e_lane : 0u;                    // <= 3
                const uint32_t hi_cut = n_shift > e_lane ? (n_shift - e_lane < 32u ? n_shift - e_lane : 32u) : 0u;
                mask = m & (hi_cut == 32u ? 0xFFFFFFFFu : (1u << hi_cut) - 1u) & ~((1u << lo_cut) - 1u);
            }
            const uint32_t cnt = __popc(mask);
            uint32_t inc = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= static_cast<uint32_t>(d)) inc += y;
            }
            const uint32_t tc = __shfl_sync(0xFFFFFFFFu, inc, 31);
            uint32_t off = 0;
            if (lane == 0 && tc) off = atomicAdd(s_used, tc);            // room in the block's store
            off = __shfl_sync(0xFFFFFFFFu, off, 0);
            const bool fits = off + tc <= Y.vals_cap;
            s_bitmap[lq * 32u + lane] = fits ? mask : 0u;
            if (lane == 0) {
                s_pinfo[lq] = fits ? (off | (tc << 21)) : 0u;
                if (!fits) *s_over = 1u;
            }
            if (tc && fits) {
                uint32_t o = vals_base + 4u * (off + inc - cnt);
                uint32_t m = mask;
                const uint32_t turns = __reduce_max_sync(0xFFFFFFFFu, cnt);
#pragma unroll 1
                for (uint32_t t = 0; t < turns; ++t) {
                    if (m) {
                        const uint32_t b = __ffs(m) - 1u;
                        m &= m - 1u;
                        uint32_t v;
                        asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(buf + lane_base + (b << 2)));
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(o), "r"(v) : "memory");
                        o += 4u;
                    }
                }
            }
            __syncwarp();                                              // the buffer has been read by every lane
            if (lane == 0 && j + ring_slots < n_mine) fetch(j + ring_slots);
        }
        if (!dead) fetched += n_mine;
        __syncthreads();                                               // this block's store is complete

        // ============================ select: the k-th largest candidate key, exactly
        if (threadIdx.x == 0) { s_x[0] = *s_used; s_x[1] = *s_over; }
        cluster.sync();                                                // ---- every block's store is complete, its counts are out
        uint32_t n_cand = 0, any_over = 0;
        for (uint32_t b = 0; b < C; ++b) {
            const uint32_t* x_b = cluster.map_shared_rank(s_x, b);
            n_cand += x_b[0];
            any_over |= x_b[1];
        }
        bool bad = any_over != 0 || n_cand < L.k;                      // the same in every block
        uint32_t why = any_over ? 1u : (n_cand < L.k ? 2u : 0u);        // kept in the record: why the instance was handed over
        const uint32_t used = bad ? 0u : *s_used;
        uint32_t T = 0, r = 0;                                         // threshold key; entries equal to it that are kept
        if (!bad) {
            uint32_t lo = t_lo, hi = t_hi_hint <= 0x7F800000u && t_hi_hint >= t_lo ? t_hi_hint : 0x7F800000u;
            uint32_t rem = L.k;
            bool hinted = true;                                        // keys above hi have not been counted yet
#pragma unroll 1
            for (int pass = 0; pass < 8 && !bad; ++pass) {
                const uint32_t width = hi - lo + 1u;                   // >= 1
                const uint32_t sh = width > 2048u ? (32u - __clz(width - 1u)) - 11u : 0u;
                for (uint32_t b = threadIdx.x; b < 2048u; b += n_threads) s_hist[b] = 0;
                if (threadIdx.x == 0) { *s_above = 0; *s_nan = 0; }
                __syncthreads();
                uint32_t above = 0, nan = 0;
                for (uint32_t i = threadIdx.x; i < used; i += n_threads) {
                    const uint32_t key = s_vals[i] & 0x7FFFFFFFu;
                    if (key >= lo && key <= hi) atomicAdd(&s_hist[(key - lo) >> sh], 1u);
                    else if (key > hi) { ++above; nan |= key > 0x7F800000u ? 1u : 0u; }
                }
                if (hinted) {
                    above = __reduce_add_sync(0xFFFFFFFFu, above);
                    nan = __reduce_or_sync(0xFFFFFFFFu, nan);
                    if (lane == 0 && above) atomicAdd(s_above, above);
                    if (lane == 0 && nan) atomicOr(s_nan, 1u);
                }
                __syncthreads();
                cluster.sync();                                        // all shares counted
                // this block's bins, summed over the cluster and handed to everyone (the loads of a bin's C shares are
                // independent: they overlap); block 0 does the same for the count above
                for (uint32_t t = threadIdx.x; t < 2048u / C; t += n_threads) {
                    const uint32_t bin = rank * (2048u / C) + t;
                    uint32_t part[kClMaxCtas];
#pragma unroll
                    for (uint32_t b = 0; b < kClMaxCtas; ++b) part[b] = b < C ? cluster.map_shared_rank(s_hist, b)[bin] : 0u;
                    uint32_t sum = 0;
#pragma unroll
                    for (uint32_t b = 0; b < kClMaxCtas; ++b) sum += part[b];
#pragma unroll
                    for (uint32_t b = 0; b < kClMaxCtas; ++b) if (b < C) cluster.map_shared_rank(s_hist, b)[bin] = sum;
                }
                if (hinted && rank == 0 && threadIdx.x == 32) {
                    uint32_t sum = 0, flag = 0;
                    for (uint32_t b = 0; b < C; ++b) {
                        sum += *cluster.map_shared_rank(s_above, b);
                        flag |= *cluster.map_shared_rank(s_nan, b);
                    }
                    for (uint32_t b = 0; b < C; ++b) {
                        *cluster.map_shared_rank(s_above, b) = sum;
                        *cluster.map_shared_rank(s_nan, b) = flag;
                    }
                }
                cluster.sync();                                        // every block holds the whole histogram
                if (hinted) {
                    const uint32_t a = *s_above;
                    if (*s_nan) { bad = true; why = 3u; break; }       // a NaN among the candidates: the general route's business
                    if (a >= rem) {                                    // the threshold lies above the hinted range: look there
                        lo = hi + 1u;
                        hi = 0x7F800000u;
                        hinted = false;                                // nothing lies above +Inf (NaN was ruled out)
                        continue;
                    }
                    rem -= a;
                    hinted = false;
                }
                block_pick_bin(s_hist, rem, s_bc, s_warp, n_warps);
                if (!s_bc[3]) { bad = true; why = 4u; break; }         // cannot happen: the counts add up to >= rem
                const uint32_t bin = s_bc[0];
                rem -= s_bc[1];
                const uint32_t lo_bin = lo + (bin << sh);
                if (sh == 0) { T = lo_bin; r = rem; break; }           // the range is one key
                const uint32_t hi_bin = lo_bin + ((1u << sh) - 1u);
                lo = lo_bin;
                hi = hi_bin < hi ? hi_bin : hi;
                __syncthreads();                                       // s_bc is read by all before the next pass writes it
                if (pass == 7) { bad = true; why = 5u; }               // cannot happen: 31 bits are decided in three passes
            }
        }
        if (bad) {
            if (rank == 0 && threadIdx.x == 0) { st->flags = kInstGeneral; st->spare = why | (n_cand << 4); }   // handed over untouched
            cluster.sync();                                            // nobody re-uses shared memory that is still being read
            continue;
        }

        // ============================ count: per piece (one thread each), candidates above T and equal to T
        for (uint32_t lq = threadIdx.x; lq < q_count; lq += n_threads) {
            const uint32_t info = s_pinfo[lq], off = info & 0x1FFFFFu, cnt = info >> 21;
            uint32_t gt = 0, eq = 0;
            for (uint32_t i = 0; i < cnt; ++i) {
                const uint32_t key = s_vals[off + i] & 0x7FFFFFFFu;
                gt += key > T ? 1u : 0u;
                eq += key == T ? 1u : 0u;
            }
            s_pcount[lq] = make_uint2(gt, eq);
        }
        if (threadIdx.x == 0) { s_carry[0] = 0; s_carry[1] = 0; }
        __syncthreads();
        // exclusive prefixes over the block's pieces (kept for the write step in s_ppost: above-T before, equal-T before)
        for (uint32_t base = 0; base < q_count; base += n_threads) {
            const uint32_t lq = base + threadIdx.x;
            uint2 c = make_uint2(0u, 0u);
            if (lq < q_count) c = s_pcount[lq];
            uint32_t tg, te;
            const uint32_t eg = block_exclusive_scan_rt(c.x, &tg, s_warp, n_warps);
            const uint32_t ee = block_exclusive_scan_rt(c.y, &te, s_warp, n_warps);
            const uint32_t c0 = s_carry[0], c1 = s_carry[1];
            if (lq < q_count) s_ppost[lq] = make_uint2(c0 + eg, c1 + ee);
            __syncthreads();
            if (threadIdx.x == 0) { s_carry[0] = c0 + tg; s_carry[1] = c1 + te; }
            __syncthreads();
        }
        if (threadIdx.x == 0) { s_x[2] = s_carry[0]; s_x[3] = s_carry[1]; }
        cluster.sync();                                                // ---- every block's totals are out
        // this block's place: what the blocks before it keep, and how many ties they hold
        uint32_t out_base = 0, eq_base = 0, kept_all = 0;
        {
            uint32_t eq_run = 0;
            for (uint32_t b = 0; b < C; ++b) {
                const uint32_t* x_b = cluster.map_shared_rank(s_x, b);
                const uint32_t g_b = x_b[2], e_b = x_b[3];
                const uint32_t ties_kept = r > eq_run ? (r - eq_run < e_b ? r - eq_run : e_b) : 0u;
                if (b < rank) { out_base += g_b + ties_kept; eq_base += e_b; }
                kept_all += g_b + ties_kept;
                eq_run += e_b;
            }
        }
        if (kept_all != L.k) {                                         // defensive: the counts must add up to k (same verdict in every block)
            if (rank == 0 && threadIdx.x == 0) { st->flags = kInstGeneral; st->spare = 6u | (kept_all << 4); }
            cluster.sync();
            continue;
        }

        // ============================ write: the kept pairs, in index order; one thread walks one piece
        uint32_t* idx_out = p.idx_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
        float* val_out = p.val_out + static_cast<uint64_t>(w) * p.K + L.out_offset;
        const uint32_t glob = static_cast<uint32_t>(L.offset) - mis;    // shifted position -> index in the gradient vector
        for (uint32_t lq = threadIdx.x; lq < q_count; lq += n_threads) {
            const uint32_t info = s_pinfo[lq];
            if ((info >> 21) == 0) continue;
            uint32_t at = info & 0x1FFFFFu;                             // the piece's next value in the store
            const uint2 post = s_ppost[lq];
            uint32_t tie_rank = eq_base + post.y;                       // global rank of the piece's first tie
            const uint32_t ties_before = r > eq_base ? (r - eq_base < post.y ? r - eq_base : post.y) : 0u;   // kept ties before the piece, inside this block
            uint32_t o = out_base + post.x + ties_before;               // the piece's first place in the output
            const uint32_t e_piece = glob + (q0 + lq) * kClPiece;
            const uint4* words = reinterpret_cast<const uint4*>(s_bitmap + lq * 32u);
#pragma unroll 1
            for (uint32_t g4 = 0; g4 < 8; ++g4) {                       // 4 lanes' masks at a time
                const uint4 wv = words[g4];
                const uint32_t wd[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                for (uint32_t c4 = 0; c4 < 4; ++c4) {
                    const uint32_t e_word = e_piece + (g4 * 4u + c4) * 32u;
                    for (uint32_t m = wd[c4]; m; m &= m - 1u, ++at) {
                        const uint32_t bits = s_vals[at], key = bits & 0x7FFFFFFFu;
                        bool keep = key > T;
                        if (key == T) { keep = tie_rank < r; ++tie_rank; }
                        if (keep) {
                            __stcs(&idx_out[o], e_word + (__ffs(m) - 1u));
                            __stcs(&val_out[o], __uint_as_float(bits));
                            ++o;
                        }
                    }
                }
            }
        }
        cluster.sync();                                                // ---- the instance is done; shared memory may be re-used
    }
}

}  // namespace adacomp
