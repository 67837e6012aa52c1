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
#include <new>
#include <vector>

#include "common.cuh"

using namespace adacomp;

namespace {

constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr uint64_t kRebaseAt = 0xFFFFFFF0ull;     // positions stay below this
constexpr int kApplyThreads = 256;

struct ServerParams {
    float* theta;
    uint32_t* head;
    uint32_t* prev;
    int* status;
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
// Several updates per launch ("owner computes").  The parameter vector is cut into ranges of
// kRangeParams consecutive parameters; every warp owns a run of consecutive ranges and, range by
// range, walks the updates of the batch IN ARRIVAL ORDER, applying the pairs that fall into the
// range.  Every update's index list is ascending, so its pairs for a range are one contiguous
// slice; lane b of the warp keeps update b's cursor, which only ever moves forward, so nothing
// is searched except each cursor's starting point.  A parameter is only ever touched by the
// warp that owns its range and sees its updates in arrival order, so the result is bit-identical
// to one-launch-per-update application, with no synchronisation between warps.  The owner's
// range of Theta / head stays in L1 / L2 across the updates of the batch, so DRAM sees each
// touched sector once per batch instead of once per update.
constexpr int kMaxBatch = 32;                  // updates per launch: one cursor per lane
constexpr uint32_t kRangeParams = 1024;

struct BatchDesc {
    uint64_t pair_begin[kMaxBatch];
    uint32_t n_pairs[kMaxBatch];
    uint32_t pos_start[kMaxBatch];
    uint32_t win_start[kMaxBatch];
    uint32_t n_updates;
};

__global__ void __launch_bounds__(kApplyThreads)
k_apply_batch(ServerParams sp, BatchDesc d, const uint32_t* __restrict__ idx, const float* __restrict__ val,
              float lr, uint32_t* sigma_out, uint32_t n_ranges) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp_global = blockIdx.x * (kApplyThreads / 32) + (threadIdx.x >> 5);
    const uint32_t n_warps = gridDim.x * (kApplyThreads / 32);
    const uint32_t r_lo = static_cast<uint32_t>(static_cast<uint64_t>(n_ranges) * warp_global / n_warps);
    const uint32_t r_hi = static_cast<uint32_t>(static_cast<uint64_t>(n_ranges) * (warp_global + 1) / n_warps);
    if (r_lo == r_hi) return;
    const uint32_t B = d.n_updates;
    // lane b: update b's description and its cursor = first pair with index >= the first owned parameter
    const uint64_t my_begin = lane < B ? d.pair_begin[lane] : 0;
    const uint32_t my_n = lane < B ? d.n_pairs[lane] : 0;
    const uint32_t my_pos = lane < B ? d.pos_start[lane] : 0;
    const uint32_t my_win = lane < B ? d.win_start[lane] : 0;
    uint32_t cursor = 0;
    {
        const uint64_t first_param = static_cast<uint64_t>(r_lo) * kRangeParams;
        uint32_t lo = 0, hi = my_n;                       // lower bound by bisection: at most 32 steps
        while (lo < hi) {
            const uint32_t mid = lo + ((hi - lo) >> 1);
            if (idx[my_begin + mid] < first_param) lo = mid + 1; else hi = mid;
        }
        cursor = lo;
    }
    for (uint32_t r = r_lo; r < r_hi; ++r) {
        const uint64_t range_end64 = static_cast<uint64_t>(r + 1) * kRangeParams;
        const uint32_t range_end = range_end64 < sp.n_params ? static_cast<uint32_t>(range_end64)
                                                             : static_cast<uint32_t>(sp.n_params);
        for (uint32_t b = 0; b < B; ++b) {
            const uint64_t begin = __shfl_sync(0xFFFFFFFFu, my_begin, b);
            const uint32_t n_b = __shfl_sync(0xFFFFFFFFu, my_n, b);
            const uint32_t pos_b = __shfl_sync(0xFFFFFFFFu, my_pos, b);
            const uint32_t win_b = __shfl_sync(0xFFFFFFFFu, my_win, b);
            uint32_t cur = __shfl_sync(0xFFFFFFFFu, cursor, b);
            while (true) {
                const uint32_t e = cur + lane;
                uint32_t k = kNone;
                if (e < n_b) k = idx[begin + e];
                const bool mine = k < range_end;              // ascending list: the lanes that match form a prefix
                if (mine) {
                    if (sp.validate && e > 0 && idx[begin + e - 1] >= k) record_error(sp.status, ADACOMP_ERR_UNSORTED);
                    apply_pair(sp, k, val[begin + e], pos_b + e, win_b, lr, sigma_out ? sigma_out + begin + e : nullptr);
                }
                const uint32_t took = __popc(__ballot_sync(0xFFFFFFFFu, mine));
                cur += took;
                if (took < 32) break;
            }
            if (lane == b) cursor = cur;
            __syncwarp();                                     // update b's writes are visible before update b + 1 reads
        }
    }
    // whoever owns the last range sees what no range claimed: indices >= n_params
    if (r_hi == n_ranges && lane < B && cursor < my_n) record_error(sp.status, ADACOMP_ERR_UNSORTED);
}

// ---------------------------------------------------------------------------------------------
// Several updates per launch, block-level owner ("owner block"), for batches that touch a good
// part of the parameters.  A block owns a run of kOwnRange-parameter ranges.  Per range it loads
// Theta and the history heads into shared memory (coalesced), then works in rounds: all warps
// together stage, for every update of the batch at once, the next pairs of the range (so the
// global loads of all updates overlap); the updates are then applied IN ARRIVAL ORDER out of
// shared memory, one block barrier per update.  Only parameters below a limit are applied in a
// round: the smallest index some update could not stage any more, so every update's pairs below
// the limit are on chip.  Staleness inside the batch comes from a per-parameter bit mask of the
// batch's updates that changed it (Eq. 3 restricted to the batch is a population count); the
// part of a window that lies before the batch is counted by walking the chain from the head the
// parameter had when the batch began.  Theta and heads of the range are written back once.
// Same results, bit for bit, as one launch per update.
constexpr uint32_t kOwnRange = 1024;
constexpr uint32_t kOwnStage = 128;            // pairs staged per update and round
constexpr int kOwnThreads = 256;

struct OwnDesc {
    BatchDesc b;
    uint32_t win_bits[kMaxBatch];              // updates of this batch inside update b's window (bits below b)
    uint32_t pre_mask;                         // bit b: update b's window starts before the batch
};

constexpr size_t kOwnSmemBytes = kOwnRange * 16 + kMaxBatch * kOwnStage * 6 + kMaxBatch * 8 + 16;

__global__ void __launch_bounds__(kOwnThreads)
k_apply_owner(ServerParams sp, OwnDesc d, const uint32_t* __restrict__ idx, const float* __restrict__ val,
              float lr, uint32_t* sigma_out, uint32_t n_ranges) {
    extern __shared__ __align__(16) unsigned char s_own[];
    float* s_theta = reinterpret_cast<float*>(s_own);
    uint32_t* s_head = reinterpret_cast<uint32_t*>(s_own + kOwnRange * 4);       // head when the batch began
    uint32_t* s_last = reinterpret_cast<uint32_t*>(s_own + kOwnRange * 8);       // latest position set by the batch
    uint32_t* s_mask = reinterpret_cast<uint32_t*>(s_own + kOwnRange * 12);      // updates of the batch that changed it
    float* s_v = reinterpret_cast<float*>(s_own + kOwnRange * 16);                                    // [B][kOwnStage]
    uint16_t* s_k = reinterpret_cast<uint16_t*>(s_own + kOwnRange * 16 + kMaxBatch * kOwnStage * 4);   // [B][kOwnStage]
    uint32_t* s_cnt = reinterpret_cast<uint32_t*>(s_own + kOwnRange * 16 + kMaxBatch * kOwnStage * 6);
    uint32_t* s_cur = s_cnt + kMaxBatch;
    uint32_t* s_limit = s_cur + kMaxBatch;

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t B = d.b.n_updates;
    const uint32_t r_lo = static_cast<uint32_t>(static_cast<uint64_t>(n_ranges) * blockIdx.x / gridDim.x);
    const uint32_t r_hi = static_cast<uint32_t>(static_cast<uint64_t>(n_ranges) * (blockIdx.x + 1) / gridDim.x);
    if (r_lo == r_hi) return;
    if (tid < B) {                                              // cursor: first pair at or above the first owned parameter
        const uint64_t first_param = static_cast<uint64_t>(r_lo) * kOwnRange;
        const uint64_t begin = d.b.pair_begin[tid];
        uint32_t lo = 0, hi = d.b.n_pairs[tid];
        while (lo < hi) {
            const uint32_t mid = lo + ((hi - lo) >> 1);
            if (idx[begin + mid] < first_param) lo = mid + 1; else hi = mid;
        }
        s_cur[tid] = lo;
    }
    __syncthreads();

    for (uint32_t r = r_lo; r < r_hi; ++r) {
        const uint32_t lo = r * kOwnRange;
        const uint64_t hi64 = static_cast<uint64_t>(lo) + kOwnRange;
        const uint32_t hi = hi64 < sp.n_params ? static_cast<uint32_t>(hi64) : static_cast<uint32_t>(sp.n_params);
        for (uint32_t t = tid; t < kOwnRange; t += kOwnThreads) {
            const bool in = lo + t < hi;
            s_theta[t] = in ? sp.theta[lo + t] : 0.f;
            s_head[t] = in ? sp.head[lo + t] : kNone;
            s_last[t] = kNone;
            s_mask[t] = 0;
        }
        while (true) {
            if (tid == 0) *s_limit = hi;
            __syncthreads();
            // ---- stage: warp w takes updates w, w + 8, ...; 4 x 32 pairs each
            for (uint32_t b = warp; b < B; b += kOwnThreads / 32) {
                const uint64_t begin = d.b.pair_begin[b];
                const uint32_t n_b = d.b.n_pairs[b], cur = s_cur[b];
                uint32_t cnt = 0, last_k = 0;
#pragma unroll
                for (uint32_t c = 0; c < kOwnStage / 32; ++c) {
                    const uint32_t t = c * 32 + lane, e = cur + t;
                    uint32_t k = kNone;
                    float v = 0.f;
                    if (e < n_b) {                              // both loads at once: the value does not wait for the index
                        k = idx[begin + e];
                        v = val[begin + e];
                    }
                    const bool mine = k < hi;                   // ascending list: matching slots form a prefix
                    if (mine) {
                        if (sp.validate && e > 0 && idx[begin + e - 1] >= k) record_error(sp.status, ADACOMP_ERR_UNSORTED);
                        s_k[b * kOwnStage + t] = static_cast<uint16_t>(k - lo);
                        s_v[b * kOwnStage + t] = v;
                    }
                    cnt += __popc(__ballot_sync(0xFFFFFFFFu, mine));
                    if (c == kOwnStage / 32 - 1) last_k = __shfl_sync(0xFFFFFFFFu, k, 31);
                }
                if (lane == 0) {
                    s_cnt[b] = cnt;
                    if (cnt == kOwnStage) atomicMin(s_limit, last_k + 1);   // more of this update may follow in the range
                }
            }
            __syncthreads();
            const uint32_t limit = *s_limit;
            // ---- apply, update after update
            for (uint32_t b = 0; b < B; ++b) {
                const uint32_t cnt = s_cnt[b];
                if (cnt == 0) continue;                         // nothing of update b in this round (same for all threads)
                bool take = false;
                if (tid < cnt) {
                    const uint32_t kl = s_k[b * kOwnStage + tid];
                    take = lo + kl < limit;
                    if (take) {
                        const float v = s_v[b * kOwnStage + tid];
                        const uint32_t e = s_cur[b] + tid;
                        const uint32_t m = s_mask[kl], ho = s_head[kl];
                        uint32_t sigma = __popc(m & d.win_bits[b]);
                        if ((d.pre_mask >> b) & 1u) {           // the part of the window before the batch
                            uint32_t q = ho, hops = 0;
                            const uint32_t ws = d.b.win_start[b];
                            while (q != kNone && q >= ws) {
                                if (++hops > sp.max_window) { record_error(sp.status, ADACOMP_ERR_WINDOW); break; }
                                q = sp.prev[(q + sp.ring_shift) & sp.ring_mask];
                            }
                            sigma += hops;
                        }
                        if (sigma_out) sigma_out[d.b.pair_begin[b] + e] = sigma;
                        if (v != 0.0f) {                        // Eq. 3 counts changes: a zero entry is not one
                            const float alpha_k = sigma ? __fdiv_rn(lr, static_cast<float>(sigma)) : lr;      // Eq. 5
                            s_theta[kl] = __fsub_rn(s_theta[kl], __fmul_rn(alpha_k, v));                       // Eq. 4
                            const uint32_t pos = d.b.pos_start[b] + e;
                            sp.prev[(pos + sp.ring_shift) & sp.ring_mask] = m ? s_last[kl] : ho;
                            s_last[kl] = pos;
                            s_mask[kl] = m | (1u << b);
                        }
                    }
                }
                const uint32_t took = __syncthreads_count(take);   // also orders update b before update b + 1
                if (tid == 0) s_cur[b] += took;
            }
            __syncthreads();
            if (limit >= hi) break;                             // every update's pairs of the range are done
        }
        for (uint32_t t = tid; t < kOwnRange; t += kOwnThreads) {
            if (lo + t < hi && s_mask[t]) {
                sp.theta[lo + t] = s_theta[t];
                sp.head[lo + t] = s_last[t];
            }
        }
        __syncthreads();
    }
    // whoever owns the last range sees what no range claimed: indices >= n_params
    if (r_hi == n_ranges && tid < B && s_cur[tid] < d.b.n_pairs[tid]) record_error(sp.status, ADACOMP_ERR_UNSORTED);
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
    int* d_status = nullptr;
    // host-side bookkeeping
    uint64_t timestamp = 0;       // i
    uint64_t pos_next = 0;        // absolute position of the next pair
    uint64_t pos_base = 0;        // absolute position that 32-bit position 0 stands for
    std::vector<uint64_t> start_of;   // start_of[u % size] = absolute start position of update u
    int validate = 0;
    int mode = 0;
};

namespace {

size_t carve_server(adacomp_server_t* s, void* base, uint64_t n_params, uint64_t ring) {
    Carver c(base);
    s->d_head = c.take<uint32_t>(n_params);
    s->d_prev = c.take<uint32_t>(ring);
    s->d_status = c.take<int>(1);
    return c.used;
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
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_apply_owner, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kOwnSmemBytes));
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

int adacomp_apply(adacomp_server_t* s, const uint32_t* d_idx, const float* d_val,
                  const uint64_t* h_pair_begin, const uint32_t* h_pair_count, const uint64_t* h_pull_ts,
                  uint32_t n_updates, float lr, uint32_t* d_sigma_out, void* cuda_stream) {
    if (!s || !s->d_theta) return ADACOMP_ERR_INVALID;
    if (n_updates == 0) return ADACOMP_OK;
    if (!h_pair_begin || !h_pair_count || !h_pull_ts) return ADACOMP_ERR_INVALID;
    if (n_updates > s->max_window) return ADACOMP_ERR_CAPACITY;
    uint64_t call_pairs = 0;
    for (uint32_t b = 0; b < n_updates; ++b) call_pairs += h_pair_count[b];
    if (call_pairs > s->history_pairs) return ADACOMP_ERR_CAPACITY;
    if (call_pairs && (!d_idx || !d_val)) return ADACOMP_ERR_INVALID;

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

    DeviceGuard guard(s->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

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

    // one launch per update, or owner-computes launches of up to kMaxBatch updates: same results
    // (automatic: the batched kernel pays off when an update names between about 0.2 % and 6 % of
    // the parameters; sparser updates are launch-bound either way, denser ones keep DRAM busy alone)
    const double density = static_cast<double>(call_pairs) / n_updates / static_cast<double>(s->n_params);
    // (automatic: when the updates of a launch (up to 32) together name about half as many pairs as
    // there are parameters, the block owner kernel, which sweeps Theta once per launch; else the warp
    // owner kernel for updates that name 0.2 % - 6 % of the parameters; else one launch per update)
    const uint32_t per_launch = n_updates < kMaxBatch ? n_updates : kMaxBatch;
    const bool owner = s->mode == 3 || (s->mode == 0 && n_updates >= 2 && density * per_launch >= 0.4);
    const bool batched = !owner && (s->mode == 2 || (s->mode == 0 && n_updates >= 2 && density >= 0.002 && density <= 0.06));
    if (owner || batched) {
        const uint32_t n_ranges = static_cast<uint32_t>((s->n_params + kRangeParams - 1) / kRangeParams);   // kOwnRange == kRangeParams
        uint64_t want_warps = static_cast<uint64_t>(s->n_sms) * 64;            // 64 resident warps per SM
        if (want_warps > n_ranges) want_warps = n_ranges;
        const unsigned grid = static_cast<unsigned>((want_warps + kApplyThreads / 32 - 1) / (kApplyThreads / 32));
        unsigned own_grid = static_cast<unsigned>(s->n_sms) * 5;
        if (own_grid > n_ranges) own_grid = n_ranges;
        for (uint32_t b0 = 0; b0 < n_updates; b0 += kMaxBatch) {
            OwnDesc od;
            BatchDesc& d = od.b;
            d.n_updates = (n_updates - b0 < kMaxBatch) ? n_updates - b0 : kMaxBatch;
            od.pre_mask = 0;
            uint64_t pairs = 0;
            for (uint32_t b = 0; b < d.n_updates; ++b) {
                d.pair_begin[b] = h_pair_begin[b0 + b];
                d.n_pairs[b] = h_pair_count[b0 + b];
                d.pos_start[b] = static_cast<uint32_t>(start_abs[b0 + b] - s->pos_base);
                d.win_start[b] = static_cast<uint32_t>(win_abs[b0 + b] - s->pos_base);
                pairs += h_pair_count[b0 + b];
                // which updates of this launch lie in update b's window [j, i - 1]
                const uint64_t ts0 = i0 + b0, j = h_pull_ts[b0 + b];
                const uint32_t first_in = j > ts0 ? static_cast<uint32_t>(j - ts0) : 0u;     // <= b
                od.win_bits[b] = ((1u << b) - 1u) & ~((1u << first_in) - 1u);
                if (j < ts0) od.pre_mask |= 1u << b;
            }
            for (uint32_t b = d.n_updates; b < kMaxBatch; ++b) od.win_bits[b] = 0;
            if (!pairs) continue;
            if (owner) {
                k_apply_owner<<<own_grid, kOwnThreads, kOwnSmemBytes, st>>>(sp, od, d_idx, d_val, lr, d_sigma_out, n_ranges);
            } else {
                k_apply_batch<<<grid, kApplyThreads, 0, st>>>(sp, d, d_idx, d_val, lr, d_sigma_out, n_ranges);
            }
            ADACOMP_LAUNCH_CHECK();
        }
    } else {
        for (uint32_t b = 0; b < n_updates; ++b) {
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
    }
    for (uint32_t b = 0; b < n_updates; ++b) s->start_of[(i0 + b) % cap] = start_abs[b];
    s->pos_next = start_abs[n_updates];
    s->timestamp = i0 + n_updates;        // the timestamp advances once per update (Algorithm 2)
    return ADACOMP_OK;
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
    if (!s || mode < 0 || mode > 3) return ADACOMP_ERR_INVALID;
    s->mode = mode;
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
