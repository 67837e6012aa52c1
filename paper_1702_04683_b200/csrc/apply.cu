// Server side of libadacomp: Algorithm 2 (Eq. 3, 4, 5) with the update history kept as
// per-parameter chains through a ring of the most recent pairs.
//
// History layout.  Every pair the server ever applies gets a position: pairs are numbered in
// application order, so update u occupies positions [start(u), start(u) + pairs(u)).  The device
// holds, relative to a host-side 64-bit base, 32-bit positions:
//   head[k]           position of the latest pair that changed parameter k (kNone if none),
//   prev[slot(pos)]   position of the pair that changed the same parameter before `pos`,
// with slot(pos) = pos mod ring size (a power of two).  For an update that pulled at timestamp
// j, sigma_k (Eq. 3) is the number of chain entries of k with position >= start(j): the chain is
// walked from head[k] until it leaves the window, i.e. O(1 + sigma_k) instead of the one search
// per remembered update of the paper's "Complexity" paragraph.  The host refuses updates whose
// window start has been overwritten in the ring.
#include <algorithm>
#include <cmath>
#include <map>
#include <new>
#include <utility>
#include <vector>

#include "common.cuh"

using namespace adacomp;

#ifndef ADACOMP_THIN_PAIRS
#define ADACOMP_THIN_PAIRS 3.0      // updates that bring at most this many pairs per 256 parameters count as thin (build-time tunable;
                                    // measured: 5 loses 7 % at four pairs per 256, 2 makes stale updates of 2.6 per 256 twice as slow)
#endif

namespace {

constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr uint64_t kRebaseAt = 0xFFFFFFF0ull;     // positions stay below this
constexpr int kApplyThreads = 256;

struct ServerParams {
    float* theta;
    uint32_t* head;
    uint32_t* prev;
    int* status;
    const uint32_t* gate;    // see BatchDesc::gate_hi
    uint64_t n_params;
    uint32_t ring_mask;
    uint32_t ring_shift;     // (position base) mod ring size: slot = (pos32 + ring_shift) & ring_mask
    uint32_t max_window;
    int validate;
};

struct UpdateDesc {
    uint64_t pair_begin;     // first pair in d_idx / d_val
    uint32_t n_pairs;
    uint32_t pos_start;      // 32-bit position of its first pair
    uint32_t win_start;      // 32-bit position of the first pair of update j (window start)
    uint32_t pad;
};

// One pair of one update: Eq. 3 (chain walk), Eq. 5, Eq. 4, then link the pair into the chain.
__device__ __forceinline__ void apply_pair(const ServerParams& sp, uint32_t k, float v, uint32_t pos,
                                           uint32_t win_start, float lr, uint32_t* sigma_slot) {
    const uint32_t latest = sp.head[k];
    uint32_t q = latest, sigma = 0;
    while (q != kNone && q >= win_start) {
        if (++sigma > sp.max_window) { record_error(sp.status, ADACOMP_ERR_WINDOW); break; }
        q = sp.prev[(q + sp.ring_shift) & sp.ring_mask];
    }
    if (sigma_slot) *sigma_slot = sigma;
    if (v != 0.0f) {                       // Eq. 3 counts changes: a zero entry is not one
        const float alpha_k = sigma ? __fdiv_rn(lr, static_cast<float>(sigma)) : lr;   // Eq. 5
        const float step = __fmul_rn(alpha_k, v);
        sp.theta[k] = __fsub_rn(sp.theta[k], step);                                       // Eq. 4
        sp.prev[(pos + sp.ring_shift) & sp.ring_mask] = latest;
        sp.head[k] = pos;
    }
}

// One update per launch, one thread per pair.  Indices inside an update are distinct, so threads
// never touch the same parameter; the stream orders successive updates.
__global__ void __launch_bounds__(kApplyThreads)
k_apply_update(ServerParams sp, UpdateDesc u, const uint32_t* __restrict__ idx, const float* __restrict__ val,
               float lr, uint32_t* sigma_out) {
    const uint32_t e = blockIdx.x * kApplyThreads + threadIdx.x;
    if (e >= u.n_pairs) return;
    const uint64_t at = u.pair_begin + e;
    const uint32_t k = idx[at];
    if (k >= sp.n_params) { record_error(sp.status, ADACOMP_ERR_UNSORTED); return; }
    if (sp.validate && e > 0 && idx[at - 1] >= k) { record_error(sp.status, ADACOMP_ERR_UNSORTED); return; }
    apply_pair(sp, k, val[at], u.pos_start + e, u.win_start, lr, sigma_out ? sigma_out + at : nullptr);
}

// ---------------------------------------------------------------------------------------------
// Several updates per launch: what the kernels below are told about them.
constexpr int kMaxBatch = 32;                  // updates per launch: one bit each in a parameter's mask

struct BatchDesc {
    uint64_t pair_begin[kMaxBatch];
    uint32_t n_pairs[kMaxBatch];
    uint32_t pos_start[kMaxBatch];
    uint32_t win_start[kMaxBatch];
    uint32_t win_bits[kMaxBatch];              // updates of this launch inside update b's window (bits below b)
    uint32_t pre_mask;                         // bit b: update b's window starts before the launch
    uint32_t n_updates;
    uint32_t gate_lo, gate_hi;                 // gate_hi != 0: the launch does its work only if gate_lo <= *gate < gate_hi
};

// Two kernels may be enqueued for the same updates, of which a count taken on the device picks one.
__device__ __forceinline__ bool gate_open(const ServerParams& sp, const BatchDesc& d) {
    if (d.gate_hi == 0) return true;
    const uint32_t v = *sp.gate;
    return v >= d.gate_lo && v < d.gate_hi;
}

// How crowded the updates' index lists are where they crowd: 256 stretches of 32 consecutive pairs are looked at per
// update (one block each), and the stretches that would put 16 pairs or more into 256 parameters are counted into
// *gate.  Evenly spread thin updates have next to none of these; updates whose pairs sit in a small part of the
// parameters have little else.
constexpr uint32_t kProbeThreads = 256;
__global__ void __launch_bounds__(kProbeThreads)
k_apply_probe(const BatchDesc d, const uint32_t* __restrict__ idx, uint32_t* gate) {
    const uint32_t n = d.n_pairs[blockIdx.x];
    if (n < 64) return;
    const uint32_t* list = idx + d.pair_begin[blockIdx.x];
    const uint32_t e = static_cast<uint32_t>(static_cast<uint64_t>(n - 32) * threadIdx.x / kProbeThreads);
    const uint32_t span = __ldg(list + e + 31) - __ldg(list + e);          // 31 gaps
    const int crowded = __syncthreads_count(span < 31u * 256u / 16u);
    if (threadIdx.x == 0 && crowded) atomicAdd(gate, static_cast<uint32_t>(crowded));
}

constexpr uint32_t kAlphaTable = 33;             // alpha / sigma kept ready for sigma < 33

// First position of an ascending index list whose entry is >= target.  The lists of an update are spread
// over [0, n_params) more or less evenly, so a few interpolation steps narrow the search before the
// bisection that finishes it: far fewer dependent loads than bisection alone on a long list.
__device__ __forceinline__ uint32_t first_at_or_above(const uint32_t* __restrict__ list, uint32_t n, uint64_t target,
                                                      uint64_t n_params) {
    uint32_t lo = 0, hi = n;                                    // answer in [lo, hi]
    uint64_t v_lo = 0, v_hi = n_params;                         // list[lo - 1] < target <= list[hi], bounds on those values
#pragma unroll 1
    for (int step = 0; step < 4 && hi - lo > 64; ++step) {
        if (target <= v_lo || target >= v_hi) break;
        const uint64_t span = hi - lo;
        uint64_t guess = lo + (target - v_lo) * span / (v_hi - v_lo);
        // two probes a little either side of the guess: both outcomes shrink the range a lot
        const uint64_t slack = 8 + (span >> 7);
        const uint32_t p0 = static_cast<uint32_t>(guess > lo + slack ? guess - slack : lo);
        const uint32_t p1 = static_cast<uint32_t>(guess + slack < hi - 1 ? guess + slack : hi - 1);
        const uint32_t x0 = list[p0], x1 = list[p1];
        if (x0 >= target) { hi = p0; v_hi = x0; }
        else if (x1 < target) { lo = p1 + 1; v_lo = x1; }
        else { lo = p0 + 1; v_lo = x0; hi = p1; v_hi = x1; }
    }
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo) >> 1);
        if (list[mid] < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// ---------------------------------------------------------------------------------------------
// Several updates per launch, one WARP per range of parameters, no block barrier in the loop.  A
// warp owns a run of ranges of R consecutive parameters and a slice of shared memory: Theta and
// the heads of the range (two buffers: the next range's arrive by asynchronous copies while this
// one is worked on) and a mask per parameter (bit b: update b of the launch changed it).  The
// updates' pairs never pass through shared memory: every lane keeps, IN REGISTERS, one pair of
// each update (lane t: the pair at the update's cursor + t), i.e. the warp holds the next 32 pairs
// of all updates at once.  The loop over the updates is unrolled, so that "update b" is a fixed
// set of registers and its descriptor (first pair, pair count, position, window bits) constant
// operands of the instructions; a stage is refilled by plain loads right after it was used, a
// whole range before it is needed again, so their latency is hidden by program order alone.
// Per range the warp takes the updates ONE AFTER THE OTHER in arrival order.  The lanes whose
// pair lies below the range's end hold the update's pairs of this range (its index list is
// ascending), and each applies its pair against shared memory exactly as Algorithm 2 states it:
// Eq. 3 inside the launch is a population count of the parameter's mask under the update's window
// bits, the part of a window before the launch a chain walk from the head the parameter had when
// the launch began; Eq. 5; Eq. 4; the pair is linked behind the head (one coalesced store to the
// ring per update) and becomes the head.  When all 32 pairs lay in the range the update may have
// more there: they are loaded and applied before the next update is looked at (the host sizes R so
// that this is rare).  At the end of the range Theta and heads go back, 16 bytes per lane, where a
// parameter changed.  Updates are applied in order per range, which is all Algorithm 2 needs:
// same results, bit for bit, as one launch per update.  NB: updates the unrolled loop covers (16 or
// 32).  kExtra: staleness counts are written, or the lists are validated.
constexpr int kWpThreads = 128;
constexpr uint32_t kWpWarps = kWpThreads / 32;

// Buffers for Theta and the records of a range: two (the next range arrives while this one is worked on), or one for
// ranges of 512, where shared memory, not registers, decides how many warps an SM holds.
__host__ __device__ constexpr uint32_t wp_bufs(uint32_t range) { return range >= 512 ? 1u : 2u; }
__host__ __device__ inline size_t wp_warp_words(uint32_t range, bool pre) {
    return (3 * wp_bufs(range) + (pre ? 1 : 0)) * static_cast<size_t>(range);   // Theta, (mask, head) records, (heads at the launch's start)
}
__host__ __device__ inline size_t wp_smem_bytes(uint32_t range, bool pre) {
    return 64 * 4 + kWpWarps * wp_warp_words(range, pre) * 4;
}

__device__ __forceinline__ uint32_t smem_address(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void copy_async_16(uint32_t smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem), "l"(gmem) : "memory");
}
__device__ __forceinline__ void copy_async_4(uint32_t smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem), "l"(gmem) : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void* gmem) { asm volatile("prefetch.global.L2 [%0];" ::"l"(gmem)); }
__device__ __forceinline__ void copy_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void copy_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory"); }

template <uint32_t R, uint32_t NB, bool kPre, bool kExtra>
__global__ void __launch_bounds__(kWpThreads)
k_apply_warps(const ServerParams sp, const BatchDesc d, const uint32_t* __restrict__ idx, const float* __restrict__ val,
              float lr, uint32_t* sigma_out, uint32_t n_ranges) {
    extern __shared__ __align__(16) unsigned char s_wp[];
    static_assert(R % 64 == 0 && R >= 128, "16-byte pieces, whole warps");
    static_assert(NB <= kMaxBatch, "one mask bit per update");
    if (!gate_open(sp, d)) return;
    float* s_alpha = reinterpret_cast<float*>(s_wp);                            // [64] alpha / sigma for the small counts
    const uint32_t B = d.n_updates;                                             // <= NB
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* s_theta = reinterpret_cast<float*>(s_wp) + 64 + warp * wp_warp_words(R, kPre);   // [2][R] Theta of the range
    // [2][R] per parameter ONE 8-byte record: .x = updates of this launch that changed it (mask), .y = its latest change
    // (head).  A pair reads and writes both with one access each: the shared-memory pipe is what bounds this kernel, and
    // lanes that fall on the same bank cost a pass each.
    constexpr uint32_t kBufs = wp_bufs(R);
    uint2* s_rec = reinterpret_cast<uint2*>(s_theta + kBufs * R);
    uint32_t* s_head0 = reinterpret_cast<uint32_t*>(s_rec + kBufs * R);         // [R] head when the launch began (kPre)

    if (tid < kAlphaTable) s_alpha[tid] = tid ? __fdiv_rn(lr, static_cast<float>(tid)) : lr;   // Eq. 5 for the small counts, once
    __syncthreads();                                            // the only block barrier
    const uint32_t gw = blockIdx.x * kWpWarps + warp, n_gw = gridDim.x * kWpWarps;
    const uint32_t r_lo = static_cast<uint32_t>(static_cast<uint64_t>(n_ranges) * gw / n_gw);
    const uint32_t r_hi = static_cast<uint32_t>(static_cast<uint64_t>(n_ranges) * (gw + 1) / n_gw);
    if (r_lo == r_hi) return;

    auto range_end = [&](uint32_t r) -> uint32_t {
        const uint64_t e = (static_cast<uint64_t>(r) + 1) * R;
        return e <= sp.n_params ? static_cast<uint32_t>(e) : static_cast<uint32_t>(sp.n_params);
    };
    // Theta and heads of range r into buffer p
    auto sweep_in = [&](uint32_t r, uint32_t p) {
        const uint32_t lo = r * R, hi = range_end(r);
        if (hi - lo == R) {
#pragma unroll
            for (uint32_t o = lane * 4; o < R; o += 128) copy_async_16(smem_address(s_theta + p * R + o), sp.theta + lo + o);
#pragma unroll
            for (uint32_t o = lane; o < R; o += 32) copy_async_4(smem_address(&s_rec[p * R + o].y), sp.head + lo + o);
        } else {                                                // the last range may be short: plain loads
            for (uint32_t o = lane; o < R; o += 32) {
                s_theta[p * R + o] = lo + o < hi ? sp.theta[lo + o] : 0.f;
                s_rec[p * R + o].y = lo + o < hi ? sp.head[lo + o] : kNone;
            }
        }
    };

    // ---- the registers that stand for the updates: cursor, and this lane's pair of the 32 at the cursor
    uint32_t cur[NB], k[NB];
    float v[NB];
    {
        uint32_t mine = 0;                                      // lane b: first pair of update b at or above the first owned parameter
        if (lane < B) mine = first_at_or_above(idx + d.pair_begin[lane], d.n_pairs[lane], static_cast<uint64_t>(r_lo) * R, sp.n_params);
#pragma unroll
        for (uint32_t b = 0; b < NB; ++b) cur[b] = __shfl_sync(0xFFFFFFFFu, mine, b & 31u);
    }
    // the lane's pair of update b at its cursor (kNone beyond the end of the list, and for updates the launch does not have)
#define ADACOMP_WP_LOAD(b)                                                                    \
    do {                                                                                      \
        const uint32_t t_ = cur[b] + lane;                                                    \
        k[b] = kNone;                                                                         \
        v[b] = 0.f;                                                                           \
        if ((b) < B && t_ < d.n_pairs[b]) {                                                   \
            k[b] = __ldg(idx + d.pair_begin[b] + t_);                                         \
            v[b] = __ldg(val + d.pair_begin[b] + t_);                                         \
        }                                                                                     \
    } while (0)
#pragma unroll
    for (uint32_t b = 0; b < NB; ++b) ADACOMP_WP_LOAD(b);
    sweep_in(r_lo, 0);
    copy_async_commit();

    for (uint32_t r = r_lo; r < r_hi; ++r) {
        const uint32_t p = kBufs == 2 ? (r - r_lo) & 1u : 0u;
        const uint32_t lo = r * R, hi = range_end(r);
        float* th = s_theta + p * R;
        uint2* rec = s_rec + p * R;
        if (kBufs == 2) {
            if (r + 1 < r_hi) sweep_in(r + 1, p ^ 1u);          // lands while this range is worked on
        } else if (r != r_lo) {
            sweep_in(r, 0);                                     // one buffer: free since the last range went back
        }
        copy_async_commit();
#pragma unroll
        for (uint32_t o = lane; o < R; o += 32) rec[o].x = 0u;  // (the heads are copied into other bytes of the records)
        if (kBufs == 2) copy_async_wait<1>();                   // this range's Theta and heads have landed
        else copy_async_wait<0>();
        __syncwarp();
        if (kPre) {
#pragma unroll
            for (uint32_t o = lane; o < R; o += 32) s_head0[o] = rec[o].y;
            __syncwarp();
        }
        // ---- the updates in arrival order
#pragma unroll
        for (uint32_t b = 0; b < NB; ++b) {
            if (b >= B) break;                                  // the same for every lane
            uint32_t bal = __ballot_sync(0xFFFFFFFFu, k[b] < hi);
            if (bal == 0) continue;                             // no pair of this update in the range
            const uint32_t bits_b = d.win_bits[b], bit_b = 1u << b;
            for (;;) {
                const uint32_t kk = k[b];
                if (kExtra && sp.validate) {
                    uint32_t before = __shfl_up_sync(0xFFFFFFFFu, kk, 1);
                    if (lane == 0) before = cur[b] > 0 ? idx[d.pair_begin[b] + cur[b] - 1] : 0u;
                    if (kk < hi && cur[b] + lane > 0 && before >= kk) record_error(sp.status, ADACOMP_ERR_UNSORTED);
                }
                if (kk < hi) {
                    if (kk >= lo) {
                        const uint32_t kl = kk - lo;
                        const float vv = v[b];
                        const bool change = vv != 0.0f;         // Eq. 3 counts changes: a zero entry is not one
                        const uint2 mh = rec[kl];                // lanes of one update hold distinct parameters: no atomics
                        uint32_t sigma = __popc(mh.x & bits_b);                                        // Eq. 3, inside the launch
                        if (kPre && (d.pre_mask & bit_b)) {                                            // Eq. 3, before the launch
                            const uint32_t ws = d.win_start[b];
                            uint32_t q = s_head0[kl], hops = 0;
                            while (q != kNone && q >= ws) {
                                if (++hops > sp.max_window) { record_error(sp.status, ADACOMP_ERR_WINDOW); break; }
                                q = sp.prev[(q + sp.ring_shift) & sp.ring_mask];
                            }
                            sigma += hops;
                        }
                        if (kExtra && sigma_out) sigma_out[d.pair_begin[b] + cur[b] + lane] = sigma;
                        if (change) {
                            const float alpha_k = sigma < kAlphaTable ? s_alpha[sigma] : __fdiv_rn(lr, static_cast<float>(sigma));   // Eq. 5
                            th[kl] = __fsub_rn(th[kl], __fmul_rn(alpha_k, vv));                        // Eq. 4
                            const uint32_t pos = d.pos_start[b] + cur[b] + lane;
                            sp.prev[(pos + sp.ring_shift) & sp.ring_mask] = mh.y;
                            rec[kl] = make_uint2(mh.x | bit_b, pos);
                        }
                    } else {                                    // an index before the range: the list was not ascending
                        record_error(sp.status, ADACOMP_ERR_UNSORTED);
                    }
                }
                __syncwarp();                                   // the next update sees this one's changes
                const uint32_t cnt = __popc(bal);
                cur[b] += cnt;
                ADACOMP_WP_LOAD(b);                             // the next 32 pairs from the new cursor: wanted a range from now
                if (cnt < 32) break;
                bal = __ballot_sync(0xFFFFFFFFu, k[b] < hi);    // all 32 lay in the range: the update may have more there
                if (bal == 0) break;
            }
        }
        // ---- Theta and heads go back where a parameter changed
        if (hi - lo == R) {
#pragma unroll
            for (uint32_t o = lane * 4; o < R; o += 128) {
                const uint4 a = *reinterpret_cast<const uint4*>(rec + o), c = *reinterpret_cast<const uint4*>(rec + o + 2);   // records o .. o + 3
                if (a.x | a.z | c.x | c.z) {
                    *reinterpret_cast<float4*>(sp.theta + lo + o) = *reinterpret_cast<const float4*>(th + o);
                    *reinterpret_cast<uint4*>(sp.head + lo + o) = make_uint4(a.y, a.w, c.y, c.w);
                }
            }
        } else {
            for (uint32_t o = lane; o < R; o += 32)
                if (lo + o < hi && rec[o].x) { sp.theta[lo + o] = th[o]; sp.head[lo + o] = rec[o].y; }
        }
        __syncwarp();
    }
    copy_async_wait<0>();
    // whoever owns the last range sees what no range claimed: indices >= n_params
    if (r_hi == n_ranges) {
#pragma unroll
        for (uint32_t b = 0; b < NB; ++b)
            if (b < B && cur[b] < d.n_pairs[b] && lane == 0) record_error(sp.status, ADACOMP_ERR_UNSORTED);
    }
#undef ADACOMP_WP_LOAD
}

// ---------------------------------------------------------------------------------------------
// Several thin updates per launch, one WARP per range of parameters, no block barrier in the loop.
// A warp owns a run of ranges and keeps, per update, a stage with the update's next 32 pairs from
// its cursor (lane b looks after update b).  Per range: lane b counts the staged pairs of update b
// below the range's end (a bisection: the list is ascending); a warp scan lines all of them up in
// arrival order (update after update); then they are applied 32 at a time, one pair per lane,
// exactly as Algorithm 2 states it.  Pairs of one update name distinct parameters; two lanes that
// hold the same parameter (different updates) are found with a match and take turns in arrival
// order, a warp-level barrier between turns.  A stage that runs low is refilled from the update's
// new cursor while the pairs are worked on; one that ran dry inside the range is refilled at once
// and the range is looked at again (later updates wait until that update is through with it).
// Same results, bit for bit, as one launch per update.  Two forms:
//   R = 0   nothing is swept, only the parameters that are named are touched, straight on global
//           memory: Eq. 3 is the walk along the parameter's chain while it stays inside the window
//           (pairs of this launch applied earlier are on the chain already), Eq. 5, Eq. 4, and the
//           pair becomes the head.  Loads of Theta, heads and links go to L2 (no L1 line survives
//           a change by another lane).  The host sizes the ranges to about 48 pairs.
//   R > 0   ranges of R parameters whose Theta, heads and change masks live in the warp's shared
//           memory, as in k_apply_warps (asynchronous copies a range ahead, Eq. 3 inside the launch
//           from the mask, written back where changed): for launches that touch most 32-byte
//           sectors of Theta anyway with updates too thin to fill a warp one at a time.
constexpr int kMgThreads = 128;
constexpr uint32_t kMgWarps = kMgThreads / 32;
constexpr uint32_t kMgPitch = 33;              // words per staged update: lanes that probe, and lanes that fill, hit distinct banks
constexpr uint32_t kMgLow = 10;                // refill a stage with fewer pairs left

// Buffers for Theta and heads of a range: two (the next range arrives while this one is worked on) for ranges of 256,
// one for ranges of 512, where two leave room for three blocks per SM only and more resident warps pay more than the
// overlap (measured, 16 updates of 625 000 pairs on 10^8 parameters: 0.39 -> 0.36 ms; ranges of 256 lose 3 % with one).
__host__ __device__ constexpr uint32_t mg_bufs(uint32_t range) { return range >= 512 ? 1u : 2u; }
__host__ __device__ inline size_t mg_warp_words(uint32_t range, uint32_t n_updates, bool pre) {
    return (range ? (2 * mg_bufs(range) + (pre ? 2 : 1)) * static_cast<size_t>(range) : 0) + ((static_cast<size_t>(n_updates) * kMgPitch * 2 + 3) & ~static_cast<size_t>(3));
}
__host__ __device__ inline size_t mg_smem_bytes(uint32_t range, uint32_t n_updates, bool pre) {
    return (range ? 256 : 0) + kMgWarps * mg_warp_words(range, n_updates, pre) * 4;
}

template <uint32_t R, bool kPre, bool kExtra>
__global__ void __launch_bounds__(kMgThreads)
k_apply_merged(const ServerParams sp, const BatchDesc d, uint32_t range, const uint32_t* __restrict__ idx,
               const float* __restrict__ val, float lr, uint32_t* sigma_out, uint32_t n_ranges) {
    extern __shared__ __align__(16) unsigned char s_mg[];
    static_assert(R % 128 == 0, "16-byte pieces, whole warps");
    constexpr bool kSlices = R != 0;                            // Theta, heads and masks of the range in shared memory
    if (!gate_open(sp, d)) return;
    if constexpr (kSlices) range = R;
    const uint32_t B = d.n_updates;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    float* s_alpha = reinterpret_cast<float*>(s_mg);                            // [64] alpha / sigma for the small counts (slices only)
    uint32_t* mine = reinterpret_cast<uint32_t*>(s_mg) + (kSlices ? 64 : 0) + warp * mg_warp_words(R, B, kPre);
    constexpr uint32_t kMgBufs = mg_bufs(R);
    float* s_theta = reinterpret_cast<float*>(mine);                            // [kMgBufs][R] Theta of the range
    uint32_t* s_head = mine + kMgBufs * R;                                      // [kMgBufs][R] latest change of the parameter
    uint32_t* s_mask = s_head + kMgBufs * R;                                    // [R] updates of this launch that changed it
    uint32_t* s_head0 = s_mask + R;                                             // [R] head when the launch began (kPre)
    uint32_t* s_k = mine + (2 * kMgBufs + (kPre ? 2 : 1)) * R;                  // [B][33] staged indices
    float* s_v = reinterpret_cast<float*>(s_k + B * kMgPitch);                  // [B][33] staged values
    if constexpr (kSlices) {
        if (threadIdx.x < kAlphaTable) s_alpha[threadIdx.x] = threadIdx.x ? __fdiv_rn(lr, static_cast<float>(threadIdx.x)) : lr;   // Eq. 5, once
        __syncthreads();                                        // the only block barrier
    }
    const uint32_t gw = blockIdx.x * kMgWarps + warp, n_gw = gridDim.x * kMgWarps;
    const uint32_t r_lo = static_cast<uint32_t>(static_cast<uint64_t>(n_ranges) * gw / n_gw);
    const uint32_t r_hi = static_cast<uint32_t>(static_cast<uint64_t>(n_ranges) * (gw + 1) / n_gw);
    if (r_lo == r_hi) return;

    // lane b's view of update b
    const bool has = lane < B;
    const uint32_t n_b = has ? d.n_pairs[lane] : 0u, pos0_b = has ? d.pos_start[lane] : 0u, ws_b = has ? d.win_start[lane] : 0u;
    const uint32_t bits_b = has ? d.win_bits[lane] : 0u;
    const uint64_t begin_b = has ? d.pair_begin[lane] : 0ull;
    uint32_t cur = 0, sb = 0;                                   // cursor; cursor of the stage's slot 0
    if (has) cur = first_at_or_above(idx + begin_b, n_b, static_cast<uint64_t>(r_lo) * range, sp.n_params);
    // the stage of update b takes its next 32 pairs from cursor c (kNone beyond the end of the list); all lanes;
    // the copies are asynchronous: copy_async_wait<0>() and a warp barrier before the stage is read
    const uint32_t a_k = smem_address(s_k + lane), a_v = smem_address(s_v + lane);
    auto fill = [&](uint32_t b, uint32_t c) {
        const uint32_t t = c + lane;
        if (t < d.n_pairs[b]) {
            copy_async_4(a_k + b * (kMgPitch * 4), idx + d.pair_begin[b] + t);
            copy_async_4(a_v + b * (kMgPitch * 4), val + d.pair_begin[b] + t);
        } else {
            s_k[b * kMgPitch + lane] = kNone;
        }
    };
    auto range_end = [&](uint32_t r) -> uint32_t {
        const uint64_t e = (static_cast<uint64_t>(r) + 1) * range;
        return e <= sp.n_params ? static_cast<uint32_t>(e) : static_cast<uint32_t>(sp.n_params);
    };
    // Theta and heads of range r into buffer p (slices only)
    auto sweep_in = [&](uint32_t r, uint32_t p) {
        if constexpr (kSlices) {
            const uint32_t lo = r * R, hi = range_end(r);
            if (hi - lo == R) {
#pragma unroll
                for (uint32_t o = lane * 4; o < R; o += 128) {
                    copy_async_16(smem_address(s_theta + p * R + o), sp.theta + lo + o);
                    copy_async_16(smem_address(s_head + p * R + o), sp.head + lo + o);
                }
            } else {                                            // the last range may be short: plain loads
                for (uint32_t o = lane; o < R; o += 32) {
                    s_theta[p * R + o] = lo + o < hi ? sp.theta[lo + o] : 0.f;
                    s_head[p * R + o] = lo + o < hi ? sp.head[lo + o] : kNone;
                }
            }
        }
    };
    for (uint32_t b = 0; b < B; ++b) fill(b, __shfl_sync(0xFFFFFFFFu, cur, b));
    sb = cur;
    if constexpr (kSlices) sweep_in(r_lo, 0);
    copy_async_commit();
    copy_async_wait<0>();
    __syncwarp();

    for (uint32_t r = r_lo; r < r_hi; ++r) {
        const uint32_t hi = range_end(r);
        const uint32_t lo = r * range;
        const uint32_t p = kMgBufs == 2 ? (r - r_lo) & 1u : 0u;
        float* th = s_theta + p * R;
        uint32_t* hd = s_head + p * R;
        if constexpr (kSlices) {
            if (kMgBufs == 2 && r + 1 < r_hi) sweep_in(r + 1, p ^ 1u);   // lands while this range is worked on
#pragma unroll
            for (uint32_t o = lane * 4; o < R; o += 128) {
                *reinterpret_cast<uint4*>(s_mask + o) = make_uint4(0, 0, 0, 0);
                if (kPre) *reinterpret_cast<uint4*>(s_head0 + o) = *reinterpret_cast<const uint4*>(hd + o);
            }
            __syncwarp();
        }
        for (;;) {
            // ---- how many staged pairs of update b lie below the range's end
            const uint32_t c0 = cur - sb;                       // first staged slot not yet applied, 0..32
            uint32_t cnt = 0;
            bool dry = false;
            if (has) {
                uint32_t a = c0, z = 32;                        // first slot in [c0, 32) whose index is >= hi
                while (a < z) {
                    const uint32_t mid = (a + z) >> 1;
                    if (s_k[lane * kMgPitch + mid] < hi) a = mid + 1; else z = mid;
                }
                cnt = a - c0;
                dry = a == 32 && sb + 32 < n_b;                 // every staged pair lies in the range: more may follow
            }
            // a stage that ran dry: its update may have more pairs in the range, and they come before those of
            // every later update, so the later updates wait for the next turn
            const uint32_t dry_mask = __ballot_sync(0xFFFFFFFFu, dry);
            if (dry_mask) {
                const uint32_t first_dry = __ffs(dry_mask) - 1;
                if (lane > first_dry) cnt = 0;
                dry = lane == first_dry;
            }
            uint32_t incl = cnt;
#pragma unroll
            for (int s = 1; s < 32; s <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, s);
                if (lane >= static_cast<uint32_t>(s)) incl += y;
            }
            const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31), off = incl - cnt;
            // stages that run low are refilled from the cursor the update will have after this turn
            const uint32_t cur_next = cur + cnt;
            const bool low = has && sb + 32 < n_b && (dry || sb + 32 - cur_next < kMgLow);
            const uint32_t low_mask = __ballot_sync(0xFFFFFFFFu, low);
            auto refill = [&]() {
                __syncwarp();                                   // every lane has what it wanted from the stages
                uint32_t m = low_mask;
                while (m) {
                    const uint32_t b = __ffs(m) - 1;
                    m &= m - 1;
                    fill(b, __shfl_sync(0xFFFFFFFFu, cur_next, b));
                }
                copy_async_commit();
            };
            // ---- up to 128 pairs at a time, four per lane, in arrival order
            const bool early = total <= 128;                    // one turn of the loop below: refill while it works
            bool refilled = false;
#pragma unroll 1
            for (uint32_t c = 0; c < total; c += 128) {
                uint32_t kq[4], posq[4], wsq[4], bq[4], bitsq[4];
                uint64_t sq[4];                                 // kExtra: where the pair's staleness count goes
                float vq[4];
#pragma unroll
                for (uint32_t u = 0; u < 4; ++u) {
                    const uint32_t e = c + 32 * u + lane;
                    const bool valid = e < total;
                    uint32_t b = 0;                             // the update of pair e: how many updates end at or before e
#pragma unroll
                    for (uint32_t s = 16; s; s >>= 1) {
                        const uint32_t t = __shfl_sync(0xFFFFFFFFu, incl, (b + s - 1) & 31u);
                        if (t <= e) b += s;
                    }
                    b &= 31u;
                    const uint32_t jj = e - __shfl_sync(0xFFFFFFFFu, off, b);    // its place among the update's pairs of this turn
                    const uint32_t slot = __shfl_sync(0xFFFFFFFFu, c0, b) + jj;
                    const uint32_t at = __shfl_sync(0xFFFFFFFFu, cur, b) + jj;  // its place in the update's list
                    posq[u] = __shfl_sync(0xFFFFFFFFu, pos0_b, b) + at;
                    wsq[u] = __shfl_sync(0xFFFFFFFFu, ws_b, b);
                    bitsq[u] = kSlices ? __shfl_sync(0xFFFFFFFFu, bits_b, b) : 0u;
                    bq[u] = b;
                    sq[u] = 0;
                    if (kExtra) {
                        const uint32_t blo = __shfl_sync(0xFFFFFFFFu, static_cast<uint32_t>(begin_b), b);
                        const uint32_t bhi = __shfl_sync(0xFFFFFFFFu, static_cast<uint32_t>(begin_b >> 32), b);
                        sq[u] = ((static_cast<uint64_t>(bhi) << 32) | blo) + at;
                    }
                    kq[u] = kNone;
                    vq[u] = 0.f;
                    if (valid) {
                        kq[u] = s_k[b * kMgPitch + slot];
                        vq[u] = s_v[b * kMgPitch + slot];
                        if (!kSlices) {
                            prefetch_l2(sp.head + kq[u]);       // wanted in a moment, by a load that must see the latest value
                            prefetch_l2(sp.theta + kq[u]);
                        }
                        if (kExtra && sp.validate && at > 0) {
                            const uint32_t before = slot > 0 ? s_k[b * kMgPitch + slot - 1] : idx[sq[u] - 1];
                            if (before >= kq[u]) record_error(sp.status, ADACOMP_ERR_UNSORTED);
                        }
                        if (kq[u] < lo) {                       // the list was not ascending: consumed, not applied
                            record_error(sp.status, ADACOMP_ERR_UNSORTED);
                            kq[u] = kNone;
                        }
                    }
                }
                // Eq. 3 before the launch: the walk from the head the parameter had when the launch began does not
                // depend on the order inside the launch, so the walks of a lane's four pairs run side by side here
                uint32_t hops[4] = {0u, 0u, 0u, 0u};
                if (kSlices && kPre) {
                    uint32_t q[4];
#pragma unroll
                    for (uint32_t u = 0; u < 4; ++u)
                        q[u] = (kq[u] != kNone && ((d.pre_mask >> bq[u]) & 1u)) ? s_head0[kq[u] - lo] : kNone;
                    bool walking = true;
                    while (walking) {
                        walking = false;
#pragma unroll
                        for (uint32_t u = 0; u < 4; ++u) {
                            if (q[u] != kNone && q[u] >= wsq[u]) {
                                if (++hops[u] > sp.max_window) { record_error(sp.status, ADACOMP_ERR_WINDOW); q[u] = kNone; }
                                else q[u] = sp.prev[(q[u] + sp.ring_shift) & sp.ring_mask];
                                walking = true;
                            }
                        }
                    }
                }
                if (early && low_mask) { refill(); refilled = true; }
#pragma unroll
                for (uint32_t u = 0; u < 4; ++u) {
                    if (c + 32 * u >= total) break;
                    const uint32_t k = kq[u], ws = wsq[u], pos = posq[u];
                    const float v = vq[u];
                    // lanes that hold the same parameter take turns, lower lane (earlier update) first
                    const uint32_t vmask = __ballot_sync(0xFFFFFFFFu, k != kNone);
                    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, k) & vmask;
                    uint32_t pending = vmask;
                    bool waiting = k != kNone;
                    while (pending) {
                        const bool go = waiting && (peers & pending & lt) == 0;
                        if (go && kSlices) {
                            const uint32_t kl = k - lo, bit = 1u << bq[u];
                            const bool change = v != 0.0f;      // Eq. 3 counts changes: a zero entry is not one
                            const uint32_t m = change ? atomicOr(&s_mask[kl], bit) : s_mask[kl];
                            uint32_t sigma = __popc(m & bitsq[u]);                                     // Eq. 3, inside the launch
                            if (kPre) sigma += hops[u];                                                // Eq. 3, before the launch
                            if (kExtra && sigma_out) sigma_out[sq[u]] = sigma;
                            if (change) {
                                const float alpha_k = sigma < kAlphaTable ? s_alpha[sigma] : __fdiv_rn(lr, static_cast<float>(sigma));   // Eq. 5
                                th[kl] = __fsub_rn(th[kl], __fmul_rn(alpha_k, v));                     // Eq. 4
                                sp.prev[(pos + sp.ring_shift) & sp.ring_mask] = atomicExch(&hd[kl], pos);
                            }
                            waiting = false;
                        }
                        if (go && !kSlices) {
                            const uint32_t latest = __ldcg(sp.head + k);
                            const float theta = __ldcg(sp.theta + k);
                            uint32_t q = latest, sigma = 0;                                            // Eq. 3
                            while (q != kNone && q >= ws) {
                                if (++sigma > sp.max_window) { record_error(sp.status, ADACOMP_ERR_WINDOW); break; }
                                q = __ldcg(sp.prev + ((q + sp.ring_shift) & sp.ring_mask));
                            }
                            if (kExtra && sigma_out) sigma_out[sq[u]] = sigma;
                            if (v != 0.0f) {                    // Eq. 3 counts changes: a zero entry is not one
                                const float alpha_k = sigma ? __fdiv_rn(lr, static_cast<float>(sigma)) : lr;   // Eq. 5
                                __stcg(sp.theta + k, __fsub_rn(theta, __fmul_rn(alpha_k, v)));         // Eq. 4
                                __stcg(sp.prev + ((pos + sp.ring_shift) & sp.ring_mask), latest);
                                __stcg(sp.head + k, pos);
                            }
                            waiting = false;
                        }
                        __syncwarp();                           // what this turn wrote is seen by the next
                        pending &= ~__ballot_sync(0xFFFFFFFFu, go);
                    }
                }
            }
            if (low_mask && !refilled) refill();
            // ---- cursors move on
            cur = cur_next;
            if (low) sb = cur;
            if (low_mask) {
                copy_async_wait<0>();
                __syncwarp();
            }
            const bool again = dry_mask != 0;
            if (!again) break;
        }
        if constexpr (kSlices) {                                // ---- Theta and heads go back where a parameter changed
            if (hi - lo == R) {
#pragma unroll
                for (uint32_t o = lane * 4; o < R; o += 128) {
                    const uint4 m4 = *reinterpret_cast<const uint4*>(s_mask + o);
                    if (m4.x | m4.y | m4.z | m4.w) {
                        *reinterpret_cast<float4*>(sp.theta + lo + o) = *reinterpret_cast<const float4*>(th + o);
                        *reinterpret_cast<uint4*>(sp.head + lo + o) = *reinterpret_cast<const uint4*>(hd + o);
                    }
                }
            } else {
                for (uint32_t o = lane; o < R; o += 32)
                    if (lo + o < hi && s_mask[o]) { sp.theta[lo + o] = th[o]; sp.head[lo + o] = hd[o]; }
            }
            if (kMgBufs == 1) {                                 // one buffer: it is free only now
                __syncwarp();
                if (r + 1 < r_hi) sweep_in(r + 1, 0);
            }
            copy_async_commit();                                // the next range's Theta and heads
            copy_async_wait<0>();
            __syncwarp();
        }
    }
    // whoever owns the last range sees what no range claimed: indices >= n_params
    if (r_hi == n_ranges && has && cur < n_b) record_error(sp.status, ADACOMP_ERR_UNSORTED);
}

// ---------------------------------------------------------------------------------------------
// The competitors' rule ("Experimental setup": ASGD and Comp-ASGD use one learning rate per update,
// the base rate over the update's staleness): every entry of an update gets the same learning
// rate alpha / (i - j), which the host has already computed (one fp32 division); Eq. 4 is applied
// to every entry as written.  No history is read or kept.  One launch per update, the stream
// orders updates.
__global__ void __launch_bounds__(kApplyThreads)
k_apply_global(ServerParams sp, UpdateDesc u, const uint32_t* __restrict__ idx, const float* __restrict__ val,
               float alpha_u, uint32_t sigma_u, uint32_t* sigma_out) {
    const uint32_t e = blockIdx.x * kApplyThreads + threadIdx.x;
    if (e >= u.n_pairs) return;
    const uint64_t at = u.pair_begin + e;
    const uint32_t k = idx[at];
    if (k >= sp.n_params) { record_error(sp.status, ADACOMP_ERR_UNSORTED); return; }
    if (sp.validate && e > 0 && idx[at - 1] >= k) { record_error(sp.status, ADACOMP_ERR_UNSORTED); return; }
    if (sigma_out) sigma_out[at] = sigma_u;
    sp.theta[k] = __fsub_rn(sp.theta[k], __fmul_rn(alpha_u, val[at]));                             // Eq. 4
}

// A dense update (ASGD pushes the whole gradient): Theta <- Theta - alpha_u * delta, 16 bytes per
// thread and step where both arrays allow it (`vec` = number of leading float4 groups).
__global__ void __launch_bounds__(kApplyThreads)
k_apply_dense(float* __restrict__ theta, const float* __restrict__ delta, uint64_t n, uint64_t vec, float alpha_u) {
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kApplyThreads;
    const uint64_t t0 = static_cast<uint64_t>(blockIdx.x) * kApplyThreads + threadIdx.x;
    for (uint64_t v = t0; v < vec; v += stride) {
        float4 th = reinterpret_cast<float4*>(theta)[v];
        const float4 d = __ldg(reinterpret_cast<const float4*>(delta) + v);
        th.x = __fsub_rn(th.x, __fmul_rn(alpha_u, d.x));
        th.y = __fsub_rn(th.y, __fmul_rn(alpha_u, d.y));
        th.z = __fsub_rn(th.z, __fmul_rn(alpha_u, d.z));
        th.w = __fsub_rn(th.w, __fmul_rn(alpha_u, d.w));
        reinterpret_cast<float4*>(theta)[v] = th;
    }
    for (uint64_t k = vec * 4 + t0; k < n; k += stride) theta[k] = __fsub_rn(theta[k], __fmul_rn(alpha_u, delta[k]));
}

// ---------------------------------------------------------------------------------------------
// The paper's own history structure ("Complexity" paragraph): the server keeps the sorted index
// lists of the last d updates and finds sigma_k of Eq. 3 with one dichotomous search per list of
// the window.  Here the ring that otherwise holds the chains holds copies of the lists (positions
// are the same: update u owns ring slots start(u) .. start(u) + pairs(u) - 1), one byte per slot
// says whether the entry was a change (non-zero), and the window's lists come as a table in the
// kernel's arguments, which bounds d to kListWindow.  One launch per update, one thread per pair:
// O((i - j) log K) probes per pair, against O(1 + sigma_k) for the chains.
constexpr uint32_t kListWindow = 448;          // most updates a window may span with this structure

struct ListWindow {
    uint32_t slot[kListWindow];                // ring slot of the first pair of update j + t
    uint32_t count[kListWindow];               // its number of pairs
    uint32_t n;                                // i - j
};

__global__ void __launch_bounds__(kApplyThreads)
k_apply_lists(ServerParams sp, UpdateDesc u, ListWindow win, uint8_t* __restrict__ changed,
              const uint32_t* __restrict__ idx, const float* __restrict__ val, float lr, uint32_t* sigma_out) {
    const uint32_t e = blockIdx.x * kApplyThreads + threadIdx.x;
    if (e >= u.n_pairs) return;
    const uint64_t at = u.pair_begin + e;
    const uint32_t k = idx[at];
    const float v = val[at];
    const uint32_t own = (u.pos_start + e) & sp.ring_mask;      // this pair's slot (pos_start: slot of the first pair)
    if (k >= sp.n_params) {                                     // skipped and reported; its slot must not match anything
        record_error(sp.status, ADACOMP_ERR_UNSORTED);
        sp.prev[own] = kNone;
        changed[own] = 0;
        return;
    }
    if (sp.validate && e > 0 && idx[at - 1] >= k) record_error(sp.status, ADACOMP_ERR_UNSORTED);
    uint32_t sigma = 0;
    for (uint32_t t = 0; t < win.n; ++t) {                      // Eq. 3: one search per update of the window
        uint32_t lo = 0, hi = win.count[t];
        const uint32_t first = win.slot[t];
        while (lo < hi) {
            const uint32_t mid = lo + ((hi - lo) >> 1);
            if (sp.prev[(first + mid) & sp.ring_mask] < k) lo = mid + 1; else hi = mid;
        }
        if (lo < win.count[t]) {
            const uint32_t slot = (first + lo) & sp.ring_mask;
            sigma += (sp.prev[slot] == k && changed[slot]) ? 1u : 0u;
        }
    }
    if (sigma_out) sigma_out[at] = sigma;
    sp.prev[own] = k;
    changed[own] = v != 0.0f ? 1 : 0;                           // Eq. 3 counts changes: a zero entry is not one
    if (v != 0.0f) {
        const float alpha_k = sigma ? __fdiv_rn(lr, static_cast<float>(sigma)) : lr;    // Eq. 5
        sp.theta[k] = __fsub_rn(sp.theta[k], __fmul_rn(alpha_k, v));                     // Eq. 4
    }
}

// Moves every stored position down by `delta` (entries older than that become kNone).
__global__ void k_rebase(uint32_t* a, uint64_t n, uint32_t delta) {
    for (uint64_t i = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x; i < n;
         i += static_cast<uint64_t>(gridDim.x) * blockDim.x) {
        const uint32_t q = a[i];
        if (q != kNone) a[i] = (q >= delta) ? q - delta : kNone;
    }
}

uint64_t pow2_at_least(uint64_t x) {
    uint64_t p = 1;
    while (p < x) p <<= 1;
    return p;
}

}  // namespace

struct adacomp_server {
    int device = 0;
    int n_sms = 0;
    uint64_t n_params = 0;
    uint64_t history_pairs = 0;   // as requested
    uint64_t ring = 0;            // power of two >= history_pairs
    uint32_t max_window = 0;
    float* d_theta = nullptr;     // borrowed
    uint32_t* d_head = nullptr;
    uint32_t* d_prev = nullptr;
    uint8_t* d_changed = nullptr; // one byte per ring slot, used by the list structure only
    int* d_status = nullptr;
    // host-side bookkeeping
    uint64_t timestamp = 0;       // i
    uint64_t pos_next = 0;        // absolute position of the next pair
    uint64_t pos_base = 0;        // absolute position that 32-bit position 0 stands for
    std::vector<uint64_t> start_of;   // start_of[u % size] = absolute start position of update u
    int validate = 0;
    int mode = 0;
    int rule = 0;                 // 0: per-parameter staleness (Eq. 3); 1: the update's staleness i - j for every entry
    bool poisoned = false;        // a launch failed after earlier launches of the same call were enqueued: reset needed
    // resident blocks per SM of every (kernel, shared memory size) launched so far: asked once, not per launch
    mutable std::map<std::pair<const void*, size_t>, int> blocks_per_sm;
};

namespace {

size_t carve_server(adacomp_server_t* s, void* base, uint64_t n_params, uint64_t ring) {
    Carver c(base);
    s->d_head = c.take<uint32_t>(n_params);
    s->d_prev = c.take<uint32_t>(ring);
    s->d_changed = c.take<uint8_t>(ring);
    s->d_status = c.take<int>(2);        // [0] the error word, [1] the count that picks between two enqueued kernels
    return c.used;
}

// How many blocks of `kernel` with `smem` bytes of dynamic shared memory stay resident per SM; the first time a
// (kernel, size) pair is seen the kernel is also allowed `max_smem` bytes.
template <typename Kernel>
int resident_blocks(const adacomp_server_t* s, Kernel kernel, int threads, size_t smem, size_t max_smem, int* per_sm) {
    const auto key = std::make_pair(reinterpret_cast<const void*>(kernel), smem);
    const auto it = s->blocks_per_sm.find(key);
    if (it != s->blocks_per_sm.end()) { *per_sm = it->second; return ADACOMP_OK; }
    ADACOMP_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(max_smem)));
    int n = 1;
    ADACOMP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem));
    if (n < 1) n = 1;
    try { s->blocks_per_sm[key] = n; } catch (...) { return ADACOMP_ERR_ALLOC; }
    *per_sm = n;
    return ADACOMP_OK;
}

// Launches k_apply_warps<R, NB, kPre, kExtra> over all ranges of R parameters with as many blocks as stay resident.
template <uint32_t R, uint32_t NB, bool kPre, bool kExtra>
int launch_apply_warps_as(const adacomp_server_t* s, const ServerParams& sp, const BatchDesc& d, const uint32_t* d_idx,
                          const float* d_val, float lr, uint32_t* d_sigma_out, cudaStream_t st) {
    const size_t smem = wp_smem_bytes(R, kPre);
    const uint32_t n_ranges = static_cast<uint32_t>((s->n_params + R - 1) / R);
    int per_sm = 1;
    const int rc = resident_blocks(s, k_apply_warps<R, NB, kPre, kExtra>, kWpThreads, smem, smem, &per_sm);
    if (rc != ADACOMP_OK) return rc;
    unsigned grid = static_cast<unsigned>(s->n_sms) * static_cast<unsigned>(per_sm > 0 ? per_sm : 1);
    const unsigned most_blocks = (n_ranges + kWpWarps - 1) / kWpWarps;
    if (grid > most_blocks) grid = most_blocks;
    k_apply_warps<R, NB, kPre, kExtra><<<grid, kWpThreads, smem, st>>>(sp, d, d_idx, d_val, lr, d_sigma_out, n_ranges);
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

template <uint32_t R, uint32_t NB>
int launch_apply_warps_with(const adacomp_server_t* s, const ServerParams& sp, const BatchDesc& d, const uint32_t* d_idx,
                            const float* d_val, float lr, uint32_t* d_sigma_out, cudaStream_t st) {
    const bool pre = d.pre_mask != 0, extra = d_sigma_out != nullptr || sp.validate != 0;
    if (pre) return extra ? launch_apply_warps_as<R, NB, true, true>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st)
                          : launch_apply_warps_as<R, NB, true, false>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
    return extra ? launch_apply_warps_as<R, NB, false, true>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st)
                 : launch_apply_warps_as<R, NB, false, false>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
}

// The unrolled loop over the updates comes in two lengths: launches of up to 16 updates keep 16 pairs per lane in
// registers, longer ones 32.
template <uint32_t R>
int launch_apply_warps(const adacomp_server_t* s, const ServerParams& sp, const BatchDesc& d, const uint32_t* d_idx,
                       const float* d_val, float lr, uint32_t* d_sigma_out, cudaStream_t st) {
    if (d.n_updates <= 16) return launch_apply_warps_with<R, 16>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
    return launch_apply_warps_with<R, 32>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
}

// Launches k_apply_merged<R, kPre, kExtra>.  R = 0: only the named parameters are touched, ranges sized so that
// one holds about 48 pairs of the launch; R > 0: ranges of R parameters, swept through shared memory.
template <uint32_t R, bool kPre, bool kExtra>
int launch_apply_merged_as(const adacomp_server_t* s, const ServerParams& sp, const BatchDesc& d, uint64_t pairs,
                           const uint32_t* d_idx, const float* d_val, float lr, uint32_t* d_sigma_out, cudaStream_t st) {
    const size_t smem = mg_smem_bytes(R, d.n_updates, kPre);
    int per_sm = 1;
    const int rc = resident_blocks(s, k_apply_merged<R, kPre, kExtra>, kMgThreads, smem, mg_smem_bytes(R, kMaxBatch, kPre), &per_sm);
    if (rc != ADACOMP_OK) return rc;
    const uint64_t warps = static_cast<uint64_t>(s->n_sms) * static_cast<uint64_t>(per_sm > 0 ? per_sm : 1) * kMgWarps;
    uint64_t range = R;
    if (R == 0) {
        // a range should hold about 48 pairs (a few per update, so that a stage of 32 lasts several ranges; measured:
        // 32 to 64 do equally well, 128 and more are slower), and every warp should get at least two ranges
        double want = 48.0 * static_cast<double>(s->n_params) / static_cast<double>(pairs);
        const double balance = static_cast<double>(s->n_params) / (2.0 * static_cast<double>(warps));
        if (want > balance) want = balance;
        range = want < 32.0 ? 32 : static_cast<uint64_t>(want) / 32 * 32;
        if (range > (1u << 30)) range = 1u << 30;
    }
    const uint64_t n_ranges = (s->n_params + range - 1) / range;
    uint64_t grid = warps / kMgWarps;
    const uint64_t most_blocks = (n_ranges + kMgWarps - 1) / kMgWarps;
    if (grid > most_blocks) grid = most_blocks;
    k_apply_merged<R, kPre, kExtra><<<static_cast<unsigned>(grid), kMgThreads, smem, st>>>(
        sp, d, static_cast<uint32_t>(range), d_idx, d_val, lr, d_sigma_out, static_cast<uint32_t>(n_ranges));
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

template <uint32_t R>
int launch_apply_merged(const adacomp_server_t* s, const ServerParams& sp, const BatchDesc& d, uint64_t pairs,
                        const uint32_t* d_idx, const float* d_val, float lr, uint32_t* d_sigma_out, cudaStream_t st) {
    const bool pre = R != 0 && d.pre_mask != 0, extra = d_sigma_out != nullptr || sp.validate != 0;
    if (pre) return extra ? launch_apply_merged_as<R, R != 0, true>(s, sp, d, pairs, d_idx, d_val, lr, d_sigma_out, st)
                          : launch_apply_merged_as<R, R != 0, false>(s, sp, d, pairs, d_idx, d_val, lr, d_sigma_out, st);
    return extra ? launch_apply_merged_as<R, false, true>(s, sp, d, pairs, d_idx, d_val, lr, d_sigma_out, st)
                 : launch_apply_merged_as<R, false, false>(s, sp, d, pairs, d_idx, d_val, lr, d_sigma_out, st);
}

bool sizes_ok(uint64_t n_params, uint64_t history_pairs) {
    return n_params >= 1 && n_params <= 0xFFFFFFFEull && history_pairs >= 1 && history_pairs < (1ull << 31);
}

}  // namespace

extern "C" {

int adacomp_server_workspace_bytes(uint64_t n_params, uint64_t history_pairs, size_t* bytes_out) {
    if (!bytes_out || !sizes_ok(n_params, history_pairs)) return ADACOMP_ERR_INVALID;
    adacomp_server_t tmp;
    *bytes_out = carve_server(&tmp, nullptr, n_params, pow2_at_least(history_pairs));
    return ADACOMP_OK;
}

int adacomp_server_create(adacomp_server_t** out, uint64_t n_params, uint64_t history_pairs,
                          uint32_t max_window_updates, void* d_workspace, size_t workspace_bytes,
                          int device) {
    if (!out) return ADACOMP_ERR_INVALID;
    *out = nullptr;
    if (!sizes_ok(n_params, history_pairs) || max_window_updates == 0 || max_window_updates >= (1u << 24))
        return ADACOMP_ERR_INVALID;
    if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) % kAlign) != 0) return ADACOMP_ERR_INVALID;
    adacomp_server_t* s = new (std::nothrow) adacomp_server_t;
    if (!s) return ADACOMP_ERR_ALLOC;
    s->ring = pow2_at_least(history_pairs);
    const size_t need = carve_server(s, d_workspace, n_params, s->ring);
    if (need > workspace_bytes) { delete s; return ADACOMP_ERR_ALLOC; }
    s->device = device;
    s->n_params = n_params;
    s->history_pairs = history_pairs;
    s->max_window = max_window_updates;
    try {
        s->start_of.assign(static_cast<size_t>(max_window_updates) + 1, 0);
    } catch (...) { delete s; return ADACOMP_ERR_ALLOC; }
    DeviceGuard guard(device);
    cudaError_t e = guard.err;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&s->n_sms, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaMemset(s->d_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { delete s; return cuda_fail(e); }
    *out = s;
    return ADACOMP_OK;
}

int adacomp_server_reset(adacomp_server_t* s, float* d_theta, void* cuda_stream) {
    if (!s || !d_theta) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(s->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ADACOMP_CUDA(cudaMemsetAsync(s->d_head, 0xFF, s->n_params * sizeof(uint32_t), st));
    ADACOMP_CUDA(cudaMemsetAsync(s->d_status, 0, sizeof(int), st));
    s->d_theta = d_theta;
    s->poisoned = false;
    s->timestamp = 0;
    s->pos_next = 0;
    s->pos_base = 0;
    std::fill(s->start_of.begin(), s->start_of.end(), 0);
    return ADACOMP_OK;
}

int adacomp_server_pull(adacomp_server_t* s, float* d_theta_copy, uint64_t* h_timestamp_out,
                        void* cuda_stream) {
    if (!s || !h_timestamp_out || !s->d_theta) return ADACOMP_ERR_INVALID;
    *h_timestamp_out = s->timestamp;
    if (d_theta_copy) {
        DeviceGuard guard(s->device);
        if (guard.err != cudaSuccess) return cuda_fail(guard.err);
        ADACOMP_CUDA(cudaMemcpyAsync(d_theta_copy, s->d_theta, s->n_params * sizeof(float),
                                     cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)));
    }
    return ADACOMP_OK;
}

// The body of adacomp_apply; may throw std::bad_alloc from its host-side tables (caught by the caller).
// `*enqueued` is set once the first kernel of the call has been launched: an error after that leaves device
// and host bookkeeping out of step.
static int apply_body(adacomp_server_t* s, const uint32_t* d_idx, const float* d_val,
                      const uint64_t* h_pair_begin, const uint32_t* h_pair_count, const uint64_t* h_pull_ts,
                      uint32_t n_updates, float lr, uint32_t* d_sigma_out, void* cuda_stream, bool* enqueued) {
    if (!s || !s->d_theta) return ADACOMP_ERR_INVALID;
    if (s->poisoned) return ADACOMP_ERR_CUDA;
    if (n_updates == 0) return ADACOMP_OK;
    if (!h_pair_begin || !h_pair_count || !h_pull_ts) return ADACOMP_ERR_INVALID;
    uint64_t call_pairs = 0;
    for (uint32_t b = 0; b < n_updates; ++b) call_pairs += h_pair_count[b];
    if (call_pairs && (!d_idx || !d_val)) return ADACOMP_ERR_INVALID;
    if (s->rule == 0 && (n_updates > s->max_window || call_pairs > s->history_pairs)) return ADACOMP_ERR_CAPACITY;

    if (s->rule == 1) {
        // ---- the competitors' rule: one learning rate per update, no history
        const uint64_t i0 = s->timestamp;
        for (uint32_t b = 0; b < n_updates; ++b) {
            const uint64_t i = i0 + b, j = h_pull_ts[b];
            if (j > i || i - j >= (1ull << 24)) return ADACOMP_ERR_WINDOW;     // the staleness must be exact as a float
        }
        DeviceGuard guard(s->device);
        if (guard.err != cudaSuccess) return cuda_fail(guard.err);
        cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
        *enqueued = true;
        ServerParams sp;
        sp.theta = s->d_theta;
        sp.head = nullptr;
        sp.prev = nullptr;
        sp.status = s->d_status;
        sp.n_params = s->n_params;
        sp.ring_mask = sp.ring_shift = 0;
        sp.max_window = s->max_window;
        sp.validate = s->validate;
        sp.gate = nullptr;
        for (uint32_t b = 0; b < n_updates; ++b) {
            UpdateDesc u;
            u.pair_begin = h_pair_begin[b];
            u.n_pairs = h_pair_count[b];
            u.pos_start = u.win_start = u.pad = 0;
            const uint32_t sigma_u = static_cast<uint32_t>(i0 + b - h_pull_ts[b]);
            const float alpha_u = sigma_u ? lr / static_cast<float>(sigma_u) : lr;   // Eq. 5 with the update's staleness
            if (u.n_pairs) {
                const unsigned grid = (u.n_pairs + kApplyThreads - 1) / kApplyThreads;
                k_apply_global<<<grid, kApplyThreads, 0, st>>>(sp, u, d_idx, d_val, alpha_u, sigma_u, d_sigma_out);
                ADACOMP_LAUNCH_CHECK();
            }
        }
        s->timestamp = i0 + n_updates;
        return ADACOMP_OK;
    }

    // ---- host-side window checks; nothing is enqueued and nothing changes until all pass
    const uint64_t i0 = s->timestamp;
    const size_t cap = s->start_of.size();
    std::vector<uint64_t> start_abs(n_updates + 1), win_abs(n_updates);
    start_abs[0] = s->pos_next;
    for (uint32_t b = 0; b < n_updates; ++b) start_abs[b + 1] = start_abs[b] + h_pair_count[b];
    for (uint32_t b = 0; b < n_updates; ++b) {
        const uint64_t i = i0 + b, j = h_pull_ts[b];
        if (j > i || i - j > s->max_window) return ADACOMP_ERR_WINDOW;
        const uint64_t ws = (j >= i0) ? start_abs[j - i0] : s->start_of[j % cap];
        if (start_abs[b + 1] - ws > s->ring) return ADACOMP_ERR_WINDOW;   // update j's pairs would be overwritten
        win_abs[b] = ws;
    }

    // ---- which updates share a launch (modes 0, 2, 3): up to kMaxBatch consecutive ones, and no more than the
    // ring allows.  Warps of one launch work on different parameter ranges at their own pace, so a pair of a late
    // update may be linked into the ring while an early update of the same launch still walks its window: the
    // slot written must not be one the window can reach, i.e. the launch must end within `ring` positions of
    // the oldest window start among its updates.  A launch is cut before the update that would break this (one
    // update alone never does: that is the check above).
    std::vector<uint32_t> launch_first;               // first update of every launch, plus n_updates at the end
    launch_first.reserve(n_updates / kMaxBatch + 2);
    for (uint32_t b0 = 0; b0 < n_updates;) {
        launch_first.push_back(b0);
        uint64_t oldest = win_abs[b0];
        uint32_t b1 = b0 + 1;
        while (b1 < n_updates && b1 - b0 < kMaxBatch) {
            const uint64_t o = win_abs[b1] < oldest ? win_abs[b1] : oldest;
            if (start_abs[b1 + 1] - o > s->ring) break;
            oldest = o;
            ++b1;
        }
        b0 = b1;
    }
    launch_first.push_back(n_updates);
    bool shared_slots = false;                 // two updates write their counts to the same slots: order matters
    if (d_sigma_out && n_updates > 1 && s->mode != 1) {
        std::vector<std::pair<uint64_t, uint64_t>> slices;
        for (uint32_t b = 0; b < n_updates; ++b)
            if (h_pair_count[b]) slices.emplace_back(h_pair_begin[b], h_pair_begin[b] + h_pair_count[b]);
        std::sort(slices.begin(), slices.end());
        for (size_t a = 1; a < slices.size(); ++a)
            if (slices[a].first < slices[a - 1].second) { shared_slots = true; break; }
    }

    DeviceGuard guard(s->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    *enqueued = true;

    if (s->mode == 4) {
        // ---- the paper's list structure: windows are bounded, positions are only ring slots (no re-basing)
        for (uint32_t b = 0; b < n_updates; ++b)
            if (i0 + b - h_pull_ts[b] > kListWindow) return ADACOMP_ERR_WINDOW;
        ServerParams sp;
        sp.theta = s->d_theta;
        sp.head = s->d_head;
        sp.prev = s->d_prev;
        sp.status = s->d_status;
        sp.n_params = s->n_params;
        sp.ring_mask = static_cast<uint32_t>(s->ring - 1);
        sp.ring_shift = 0;
        sp.max_window = s->max_window;
        sp.validate = s->validate;
        sp.gate = nullptr;
        const uint64_t mask = s->ring - 1;
        for (uint32_t b = 0; b < n_updates; ++b) {
            const uint64_t i = i0 + b, j = h_pull_ts[b];
            ListWindow win;
            win.n = static_cast<uint32_t>(i - j);
            for (uint64_t t = j; t < i; ++t) {                  // start and size of update t, from this call or before
                const uint64_t st_t = t >= i0 ? start_abs[t - i0] : s->start_of[t % cap];
                const uint64_t en_t = t + 1 >= i0 ? start_abs[t + 1 - i0] : s->start_of[(t + 1) % cap];
                win.slot[t - j] = static_cast<uint32_t>(st_t & mask);
                win.count[t - j] = static_cast<uint32_t>(en_t - st_t);
            }
            UpdateDesc u;
            u.pair_begin = h_pair_begin[b];
            u.n_pairs = h_pair_count[b];
            u.pos_start = static_cast<uint32_t>(start_abs[b] & mask);
            u.win_start = u.pad = 0;
            if (u.n_pairs) {
                const unsigned grid = (u.n_pairs + kApplyThreads - 1) / kApplyThreads;
                k_apply_lists<<<grid, kApplyThreads, 0, st>>>(sp, u, win, s->d_changed, d_idx, d_val, lr, d_sigma_out);
                ADACOMP_LAUNCH_CHECK();
            }
        }
        for (uint32_t b = 0; b < n_updates; ++b) s->start_of[(i0 + b) % cap] = start_abs[b];
        s->pos_next = start_abs[n_updates];
        s->timestamp = i0 + n_updates;
        return ADACOMP_OK;
    }

    // ---- keep 32-bit positions in range
    if (s->pos_next + call_pairs - s->pos_base >= kRebaseAt) {
        uint64_t oldest = s->pos_next > s->ring ? s->pos_next - s->ring : 0;   // oldest position still in the ring
        if (oldest < s->pos_base) oldest = s->pos_base;
        const uint64_t delta = oldest - s->pos_base;
        if (delta == 0 || s->pos_next + call_pairs - oldest >= kRebaseAt) return ADACOMP_ERR_CAPACITY;
        const unsigned grid = static_cast<unsigned>(s->n_sms * 8);
        k_rebase<<<grid, 256, 0, st>>>(s->d_head, s->n_params, static_cast<uint32_t>(delta));
        ADACOMP_LAUNCH_CHECK();
        k_rebase<<<grid, 256, 0, st>>>(s->d_prev, s->ring, static_cast<uint32_t>(delta));
        ADACOMP_LAUNCH_CHECK();
        s->pos_base = oldest;
    }

    ServerParams sp;
    sp.theta = s->d_theta;
    sp.head = s->d_head;
    sp.prev = s->d_prev;
    sp.status = s->d_status;
    sp.n_params = s->n_params;
    sp.ring_mask = static_cast<uint32_t>(s->ring - 1);
    sp.ring_shift = static_cast<uint32_t>(s->pos_base & (s->ring - 1));
    sp.max_window = s->max_window;
    sp.validate = s->validate;
    sp.gate = reinterpret_cast<const uint32_t*>(s->d_status + 1);

    // ---- launches.  One launch per update, or launches of up to kMaxBatch updates each: same results.
    // Automatic choice per launch: a dense sweep of Theta through shared memory when the launch's pairs number
    // 8 % of the parameters or more (most 32-byte sectors of Theta are touched anyway), else the kernel that
    // touches only the named parameters; a single update, and updates whose staleness slots overlap in memory, go
    // one per launch.
    const bool one_by_one = s->mode == 1 || shared_slots || (s->mode == 0 && n_updates == 1);
    const bool theta_aligned = reinterpret_cast<uintptr_t>(s->d_theta) % 16 == 0;
    for (size_t g = 0; g + 1 < launch_first.size() && !one_by_one; ++g) {
        const uint32_t b0 = launch_first[g];
        BatchDesc d;
        d.n_updates = launch_first[g + 1] - b0;
        d.pre_mask = 0;
        d.gate_lo = d.gate_hi = 0;
        uint64_t pairs = 0;
        uint32_t most = 0;
        const uint64_t ts0 = i0 + b0;
        for (uint32_t b = 0; b < kMaxBatch; ++b) {
            const bool live = b < d.n_updates;
            d.pair_begin[b] = live ? h_pair_begin[b0 + b] : 0;
            d.n_pairs[b] = live ? h_pair_count[b0 + b] : 0;
            d.pos_start[b] = live ? static_cast<uint32_t>(start_abs[b0 + b] - s->pos_base) : 0;
            d.win_start[b] = live ? static_cast<uint32_t>(win_abs[b0 + b] - s->pos_base) : 0;
            d.win_bits[b] = 0;
            if (!live) continue;
            pairs += d.n_pairs[b];
            most = d.n_pairs[b] > most ? d.n_pairs[b] : most;
            const uint64_t j = h_pull_ts[b0 + b];           // which updates of this launch lie in the window [j, i - 1]
            const uint32_t first_in = j > ts0 ? static_cast<uint32_t>(j - ts0) : 0u;     // <= b
            d.win_bits[b] = ((1u << b) - 1u) & ~((1u << first_in) - 1u);
            if (j < ts0) d.pre_mask |= 1u << b;
        }
        if (!pairs) continue;
        const double dens = static_cast<double>(most) / static_cast<double>(s->n_params);   // of the densest update
        const bool sweep = theta_aligned &&
                           (s->mode == 3 || (s->mode == 0 && static_cast<double>(pairs) >= 0.08 * static_cast<double>(s->n_params)));
        int rc;
        if (sweep && dens * 256.0 <= ADACOMP_THIN_PAIRS) {
            // thin updates (a handful of pairs per update and range): all updates' pairs of a range lined up and
            // applied 32 at a time against the range's slices in shared memory
            // ... unless the pairs crowd into a small part of the parameters, where the ranges they fall into are
            // as busy as a dense update's: a count taken on the device picks between the two kernels, both enqueued
            uint32_t probed = 0;
            for (uint32_t b = 0; b < d.n_updates; ++b) probed += d.n_pairs[b] >= 64 ? kProbeThreads : 0;
            const uint32_t crowded_from = probed / 4;
            if (crowded_from) {
                uint32_t* gate = reinterpret_cast<uint32_t*>(s->d_status + 1);
                ADACOMP_CUDA(cudaMemsetAsync(gate, 0, sizeof(uint32_t), st));
                k_apply_probe<<<d.n_updates, kProbeThreads, 0, st>>>(d, d_idx, gate);
                ADACOMP_LAUNCH_CHECK();
                d.gate_lo = crowded_from;
                d.gate_hi = 0xFFFFFFFFu;
                rc = launch_apply_warps<128>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
                if (rc != ADACOMP_OK) return rc;
                d.gate_lo = 0;
                d.gate_hi = crowded_from;
            }
            // (thin = at most six pairs of the densest update per 512 parameters: ranges of 512 throughout)
            rc = launch_apply_merged<512>(s, sp, d, pairs, d_idx, d_val, lr, d_sigma_out, st);
        } else if (sweep) {
            // range size: the densest update should bring about 26 pairs per range (mean of a uniformly spread
            // update), so that one load of 32 pairs per update and range is usually all of them
            const double want = 26.0 / dens;
            if (want >= 512.0) rc = launch_apply_warps<512>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
            else if (want >= 384.0) rc = launch_apply_warps<384>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
            else if (want >= 256.0) rc = launch_apply_warps<256>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
            else if (want >= 192.0) rc = launch_apply_warps<192>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
            else rc = launch_apply_warps<128>(s, sp, d, d_idx, d_val, lr, d_sigma_out, st);
        } else {
            rc = launch_apply_merged<0>(s, sp, d, pairs, d_idx, d_val, lr, d_sigma_out, st);
        }
        if (rc != ADACOMP_OK) return rc;
    }
    for (uint32_t b = 0; b < n_updates && one_by_one; ++b) {
        UpdateDesc u;
        u.pair_begin = h_pair_begin[b];
        u.n_pairs = h_pair_count[b];
        u.pos_start = static_cast<uint32_t>(start_abs[b] - s->pos_base);
        u.win_start = static_cast<uint32_t>(win_abs[b] - s->pos_base);
        u.pad = 0;
        if (u.n_pairs) {
            const unsigned grid = (u.n_pairs + kApplyThreads - 1) / kApplyThreads;
            k_apply_update<<<grid, kApplyThreads, 0, st>>>(sp, u, d_idx, d_val, lr, d_sigma_out);
            ADACOMP_LAUNCH_CHECK();
        }
    }
    for (uint32_t b = 0; b < n_updates; ++b) s->start_of[(i0 + b) % cap] = start_abs[b];
    s->pos_next = start_abs[n_updates];
    s->timestamp = i0 + n_updates;        // the timestamp advances once per update (Algorithm 2)
    return ADACOMP_OK;
}

int adacomp_apply(adacomp_server_t* s, const uint32_t* d_idx, const float* d_val,
                  const uint64_t* h_pair_begin, const uint32_t* h_pair_count, const uint64_t* h_pull_ts,
                  uint32_t n_updates, float lr, uint32_t* d_sigma_out, void* cuda_stream) {
    bool enqueued = false;
    int rc;
    try {
        rc = apply_body(s, d_idx, d_val, h_pair_begin, h_pair_count, h_pull_ts, n_updates, lr, d_sigma_out, cuda_stream,
                        &enqueued);
    } catch (...) {                                     // a host-side table could not be allocated
        rc = ADACOMP_ERR_ALLOC;
    }
    // an error after the first launch leaves the device's history ahead of the host's bookkeeping: the server
    // refuses further updates until it is reset
    if (rc != ADACOMP_OK && enqueued && s) s->poisoned = true;
    return rc;
}

int adacomp_apply_host(adacomp_server_t* s, const uint32_t* h_idx, const float* h_val,
                       const uint64_t* h_pair_begin, const uint32_t* h_pair_count, const uint64_t* h_pull_ts,
                       uint32_t n_updates, float lr, uint32_t* d_idx_staging, float* d_val_staging,
                       uint32_t* d_sigma_staging, uint32_t* h_sigma_out, void* cuda_stream) {
    if (!s) return ADACOMP_ERR_INVALID;
    if (n_updates == 0) return ADACOMP_OK;
    if (!h_pair_begin || !h_pair_count) return ADACOMP_ERR_INVALID;
    // one copy over the range of pairs the updates span
    uint64_t first = ~0ull, last = 0;
    for (uint32_t b = 0; b < n_updates; ++b) {
        if (!h_pair_count[b]) continue;
        first = h_pair_begin[b] < first ? h_pair_begin[b] : first;
        const uint64_t end = h_pair_begin[b] + h_pair_count[b];
        last = end > last ? end : last;
    }
    const uint64_t pairs = last > first ? last - first : 0;
    if (pairs && (!h_idx || !h_val || !d_idx_staging || !d_val_staging)) return ADACOMP_ERR_INVALID;
    if (h_sigma_out && !d_sigma_staging) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(s->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (pairs) {
        ADACOMP_CUDA(cudaMemcpyAsync(d_idx_staging + first, h_idx + first, pairs * sizeof(uint32_t), cudaMemcpyHostToDevice, st));
        ADACOMP_CUDA(cudaMemcpyAsync(d_val_staging + first, h_val + first, pairs * sizeof(float), cudaMemcpyHostToDevice, st));
    }
    int rc = adacomp_apply(s, d_idx_staging, d_val_staging, h_pair_begin, h_pair_count, h_pull_ts, n_updates, lr,
                           h_sigma_out ? d_sigma_staging : nullptr, cuda_stream);
    if (rc != ADACOMP_OK) return rc;
    if (h_sigma_out && pairs)
        ADACOMP_CUDA(cudaMemcpyAsync(h_sigma_out + first, d_sigma_staging + first, pairs * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    return ADACOMP_OK;
}

int adacomp_server_timestamp(const adacomp_server_t* s, uint64_t* h_timestamp_out) {
    if (!s || !h_timestamp_out) return ADACOMP_ERR_INVALID;
    *h_timestamp_out = s->timestamp;
    return ADACOMP_OK;
}

int adacomp_server_set_validation(adacomp_server_t* s, int on) {
    if (!s) return ADACOMP_ERR_INVALID;
    s->validate = on ? 1 : 0;
    return ADACOMP_OK;
}

int adacomp_server_set_mode(adacomp_server_t* s, int mode) {
    if (!s || mode < 0 || mode > 4) return ADACOMP_ERR_INVALID;
    // the list structure keeps another history in the same ring: no switching once updates were applied
    if ((mode == 4) != (s->mode == 4) && s->timestamp != 0) return ADACOMP_ERR_INVALID;
    s->mode = mode;
    return ADACOMP_OK;
}

int adacomp_server_set_rule(adacomp_server_t* s, int rule) {
    if (!s || rule < 0 || rule > 1) return ADACOMP_ERR_INVALID;
    if (rule != s->rule && s->timestamp != 0) return ADACOMP_ERR_INVALID;   // the history of the other rule is missing
    s->rule = rule;
    return ADACOMP_OK;
}

int adacomp_apply_dense(adacomp_server_t* s, const float* d_delta, uint64_t pull_ts, float lr, void* cuda_stream) {
    if (!s || !s->d_theta || !d_delta || s->rule != 1) return ADACOMP_ERR_INVALID;
    const uint64_t i = s->timestamp;
    if (pull_ts > i || i - pull_ts >= (1ull << 24)) return ADACOMP_ERR_WINDOW;
    DeviceGuard guard(s->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    const uint32_t sigma_u = static_cast<uint32_t>(i - pull_ts);
    const float alpha_u = sigma_u ? lr / static_cast<float>(sigma_u) : lr;       // Eq. 5 with the update's staleness
    const bool aligned = reinterpret_cast<uintptr_t>(s->d_theta) % 16 == 0 && reinterpret_cast<uintptr_t>(d_delta) % 16 == 0;
    const uint64_t vec = aligned ? s->n_params / 4 : 0;
    uint64_t want = (s->n_params / 4 + kApplyThreads - 1) / kApplyThreads;
    const uint64_t cap = static_cast<uint64_t>(s->n_sms) * 16;
    const unsigned grid = static_cast<unsigned>(want < 1 ? 1 : (want > cap ? cap : want));
    k_apply_dense<<<grid, kApplyThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(s->d_theta, d_delta, s->n_params, vec, alpha_u);
    ADACOMP_LAUNCH_CHECK();
    s->timestamp = i + 1;
    return ADACOMP_OK;
}

int adacomp_server_debug_skip_positions(adacomp_server_t* s, uint64_t count) {
    if (!s) return ADACOMP_ERR_INVALID;
    s->pos_next += count;
    return ADACOMP_OK;
}

int adacomp_server_last_error(adacomp_server_t* s, void* cuda_stream) {
    if (!s) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(s->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int status = 0;
    ADACOMP_CUDA(cudaMemcpyAsync(&status, s->d_status, sizeof status, cudaMemcpyDeviceToHost, st));
    ADACOMP_CUDA(cudaMemsetAsync(s->d_status, 0, sizeof(int), st));
    ADACOMP_CUDA(cudaStreamSynchronize(st));
    return status;
}

int adacomp_server_destroy(adacomp_server_t* s) {
    delete s;
    return ADACOMP_OK;
}

}  // extern "C"
