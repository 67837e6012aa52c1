// Index coding for the (index, value) pairs an update carries.  The paper leaves the encoding open
// (footnote of "Algorithm details"); this is the lossless format the library offers for the index
// half, values travel as they are.  An update's ascending index list is cut into blocks of 256
// entries; a block is stored as
//   word 0   the first index of the block,
//   word 1   w = the number of bits of the largest gap in the block, the gap of an entry being
//            (index - previous index - 1) modulo 2^32,
//   then     the gaps of entries 1 .. n - 1, w bits each, entry e at bit (e - 1) * w of a
//            little-endian bit string held in 32-bit words (none if w = 0).
// block_off[b] is the word at which block b starts inside the worker's stream, block_off[n_blocks]
// the stream's length.  The values have a lossless packing of the same shape (blocks of 256 entries, one
// header word with the block's smallest exponent field e_min and the width w_e of the exponent range,
// then sign / exponent - e_min / mantissa in 24 + w_e bits per entry): k_values_measure, k_values_pack,
// k_values_decode, with the same prefix-sum kernel between the first two.  Three kernels encode (measure every block, prefix-sum the sizes, pack), one
// decodes; a block of the format is one warp's work, eight entries per lane.
#include "common.cuh"

using namespace adacomp;

namespace {

constexpr int kCodeBlock = 256;                 // entries per block of the format
constexpr int kRows = kCodeBlock / 32;          // a warp holds a block as 8 rows of 32 entries, entry e = row * 32 + lane
constexpr int kCodeWarps = 8;                   // blocks of the format per CUDA block, one warp each
constexpr int kCodeThreads = kCodeWarps * 32;

// Block `b` of worker `w`, held by one warp: v[r] = entry r * 32 + lane (0 past the end), gap[r] its gap (0 for the
// block's first entry and past the end).  Returns the block's width.  Every load is one coalesced row.
__device__ __forceinline__ uint32_t load_block_gaps(const uint32_t* __restrict__ list, uint64_t first, uint32_t n,
                                                    uint32_t lane, uint32_t (&v)[kRows], uint32_t (&gap)[kRows]) {
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const uint32_t e = r * 32 + lane;
        v[r] = e < n ? __ldg(list + first + e) : 0u;
    }
    uint32_t widest = 0;
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        uint32_t before = __shfl_up_sync(0xFFFFFFFFu, v[r], 1);
        if (r > 0) {
            const uint32_t last_row = __shfl_sync(0xFFFFFFFFu, v[r - 1], 31);
            if (lane == 0) before = last_row;
        }
        const uint32_t e = r * 32 + lane;
        gap[r] = (e >= 1 && e < n) ? v[r] - before - 1u : 0u;
        widest = max(widest, gap[r]);
    }
    widest = __reduce_max_sync(0xFFFFFFFFu, widest);
    return widest ? 32u - static_cast<uint32_t>(__clz(widest)) : 0u;
}

__global__ void __launch_bounds__(kCodeThreads)
k_encode_measure(const uint32_t* __restrict__ idx, uint64_t K, uint64_t n_blocks, uint64_t* __restrict__ block_off) {
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t b = static_cast<uint64_t>(blockIdx.x) * kCodeWarps + (threadIdx.x >> 5), w = blockIdx.y;
    if (b >= n_blocks) return;
    const uint64_t first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    uint32_t v[kRows], gap[kRows];
    const uint32_t width = load_block_gaps(idx + w * K, first, n, lane, v, gap);
    if (lane == 0) {
        block_off[w * (n_blocks + 1) + b + 1] = 2 + (static_cast<uint64_t>(n - 1) * width + 31) / 32;   // size, summed up next
        if (b == 0) block_off[w * (n_blocks + 1)] = 0;
    }
}

// In place: sizes in entries 1 .. n_blocks become the running totals (entry 0 stays 0).
__global__ void __launch_bounds__(1024) k_encode_offsets(uint64_t* __restrict__ block_off, uint64_t n_blocks) {
    __shared__ uint64_t s_warp[32];
    __shared__ uint64_t s_carry;
    uint64_t* a = block_off + blockIdx.x * (n_blocks + 1) + 1;
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (uint64_t base = 0; base < n_blocks; base += 1024) {
        const uint64_t i = base + threadIdx.x;
        uint64_t v = i < n_blocks ? a[i] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, v, d);
            if (lane >= static_cast<uint32_t>(d)) v += y;
        }
        if (lane == 31) s_warp[warp] = v;
        __syncthreads();
        if (warp == 0) {
            uint64_t t = s_warp[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, t, d);
                if (lane >= static_cast<uint32_t>(d)) t += y;
            }
            s_warp[lane] = t;
        }
        __syncthreads();
        const uint64_t before = s_carry + (warp ? s_warp[warp - 1] : 0);
        if (i < n_blocks) a[i] = before + v;
        __syncthreads();
        if (threadIdx.x == 1023) s_carry = before + v;
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kCodeThreads)
k_encode_pack(const uint32_t* __restrict__ idx, uint64_t K, uint64_t n_blocks, const uint64_t* __restrict__ block_off,
              uint32_t* __restrict__ words, uint64_t words_per_worker) {
    __shared__ uint32_t s_bits[kCodeWarps][kCodeBlock];          // the payload of each warp's block
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t b = static_cast<uint64_t>(blockIdx.x) * kCodeWarps + warp, w = blockIdx.y;
    if (b >= n_blocks) return;
    const uint64_t first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    uint32_t v[kRows], gap[kRows];
    const uint32_t width = load_block_gaps(idx + w * K, first, n, lane, v, gap);
    uint32_t* out = words + w * words_per_worker + block_off[w * (n_blocks + 1) + b];
    if (lane == 0) {
        out[0] = v[0];
        out[1] = width;
    }
    const uint32_t payload = ((n - 1) * width + 31) / 32;
    if (!payload) return;
    uint32_t* bits = s_bits[warp];
#pragma unroll
    for (int r = 0; r < kRows; ++r) bits[r * 32 + lane] = 0;
    __syncwarp();
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const uint32_t e = r * 32 + lane;
        if (e >= 1 && e < n) {
            const uint32_t pos = (e - 1) * width, word = pos >> 5, shift = pos & 31;
            const unsigned long long spread = static_cast<unsigned long long>(gap[r]) << shift;
            atomicOr(&bits[word], static_cast<uint32_t>(spread));
            if (shift + width > 32) atomicOr(&bits[word + 1], static_cast<uint32_t>(spread >> 32));
        }
    }
    __syncwarp();
    for (uint32_t t = lane; t < payload; t += 32) out[2 + t] = bits[t];
}

__global__ void __launch_bounds__(kCodeThreads)
k_decode(const uint32_t* __restrict__ words, uint64_t words_per_worker, const uint64_t* __restrict__ block_off,
         uint64_t K, uint64_t n_blocks, uint32_t* __restrict__ idx_out) {
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t b = static_cast<uint64_t>(blockIdx.x) * kCodeWarps + (threadIdx.x >> 5), w = blockIdx.y;
    if (b >= n_blocks) return;
    const uint64_t first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    uint32_t* out = idx_out + w * K + first;
    // the stream is untrusted (it arrives from a worker): the block must lie inside the worker's words with a
    // width of at most 32 bits, else the block decodes to 0xFFFFFFFF everywhere, an index no server accepts
    // (adacomp_apply skips and reports it), and nothing outside the stream is read
    const uint64_t off = block_off[w * (n_blocks + 1) + b];
    bool sound = off + 2 <= words_per_worker;
    const uint32_t* in = words + w * words_per_worker + (sound ? off : 0);
    const uint32_t width = sound ? __ldg(in + 1) : 0u;
    sound = sound && width <= 32 && off + 2 + (static_cast<uint64_t>(n - 1) * width + 31) / 32 <= words_per_worker;
    if (!sound) {
#pragma unroll
        for (int r = 0; r < kRows; ++r)
            if (r * 32 + lane < n) out[r * 32 + lane] = 0xFFFFFFFFu;
        return;
    }
    const uint32_t keep = width == 32 ? 0xFFFFFFFFu : ((1u << width) - 1u);
    uint32_t step[kRows];                                // what an entry adds to its predecessor
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const uint32_t e = r * 32 + lane;
        step[r] = 0;
        if (e == 0) step[r] = __ldg(in);
        else if (e < n) {
            uint32_t gap = 0;
            if (width) {
                const uint32_t pos = (e - 1) * width, word = pos >> 5, shift = pos & 31;
                unsigned long long window = __ldg(in + 2 + word);
                if (shift + width > 32) window |= static_cast<unsigned long long>(__ldg(in + 2 + word + 1)) << 32;
                gap = static_cast<uint32_t>(window >> shift) & keep;
            }
            step[r] = gap + 1u;
        }
    }
    uint32_t carry = 0;                                  // running sum modulo 2^32: the index
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        uint32_t v = step[r];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, v, d);
            if (lane >= static_cast<uint32_t>(d)) v += y;
        }
        v += carry;
        if (r * 32 + lane < n) out[r * 32 + lane] = v;
        carry = __shfl_sync(0xFFFFFFFFu, v, 31);
    }
}

// ---- values: a block of the format is again one warp's work, eight coalesced rows in registers

// Block of worker `w` held by one warp: bits[r] = the bit pattern of entry r * 32 + lane (unused past the end).
// Returns the header word e_min | w_e << 8.
__device__ __forceinline__ uint32_t load_block_values(const float* __restrict__ list, uint64_t first, uint32_t n,
                                                      uint32_t lane, uint32_t (&bits)[kRows]) {
    uint32_t e_lo = 255u, e_hi = 0u;
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const uint32_t t = r * 32 + lane;
        bits[r] = t < n ? __float_as_uint(__ldg(list + first + t)) : 0u;
        if (t < n) {
            const uint32_t e = (bits[r] >> 23) & 0xFFu;
            e_lo = min(e_lo, e);
            e_hi = max(e_hi, e);
        }
    }
    e_lo = __reduce_min_sync(0xFFFFFFFFu, e_lo);
    e_hi = __reduce_max_sync(0xFFFFFFFFu, e_hi);
    const uint32_t spread = e_hi - e_lo;                         // n >= 1: the block has an entry
    return e_lo | ((spread ? 32u - static_cast<uint32_t>(__clz(spread)) : 0u) << 8);
}

__global__ void __launch_bounds__(kCodeThreads)
k_values_measure(const float* __restrict__ val, uint64_t K, uint64_t n_blocks, uint64_t* __restrict__ block_off) {
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t b = static_cast<uint64_t>(blockIdx.x) * kCodeWarps + (threadIdx.x >> 5), w = blockIdx.y;
    if (b >= n_blocks) return;
    const uint64_t first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    uint32_t bits[kRows];
    const uint32_t header = load_block_values(val + w * K, first, n, lane, bits);
    if (lane == 0) {
        block_off[w * (n_blocks + 1) + b + 1] = 1 + (static_cast<uint64_t>(n) * (24 + (header >> 8)) + 31) / 32;   // size, summed up next
        if (b == 0) block_off[w * (n_blocks + 1)] = 0;
    }
}

__global__ void __launch_bounds__(kCodeThreads)
k_values_pack(const float* __restrict__ val, uint64_t K, uint64_t n_blocks, const uint64_t* __restrict__ block_off,
              uint32_t* __restrict__ words, uint64_t words_per_worker) {
    __shared__ uint32_t s_bits[kCodeWarps][kCodeBlock];          // the payload of each warp's block: at most 32 bits an entry
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t b = static_cast<uint64_t>(blockIdx.x) * kCodeWarps + warp, w = blockIdx.y;
    if (b >= n_blocks) return;
    const uint64_t first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    uint32_t bits[kRows];
    const uint32_t header = load_block_values(val + w * K, first, n, lane, bits);
    const uint32_t e_min = header & 0xFFu, w_e = header >> 8, width = 24 + w_e;
    uint32_t* out = words + w * words_per_worker + block_off[w * (n_blocks + 1) + b];
    if (lane == 0) out[0] = header;
    uint32_t* image = s_bits[warp];
#pragma unroll
    for (int r = 0; r < kRows; ++r) image[r * 32 + lane] = 0;
    __syncwarp();
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const uint32_t t = r * 32 + lane;
        if (t < n) {
            const uint32_t x = bits[r];
            const unsigned long long entry = (x & 0x7FFFFFu) | (static_cast<unsigned long long>(((x >> 23) & 0xFFu) - e_min) << 23) |
                                             (static_cast<unsigned long long>(x >> 31) << (23 + w_e));
            const uint32_t pos = t * width, word = pos >> 5, shift = pos & 31;
            const unsigned long long spread = entry << shift;    // width <= 32, shift <= 31: fits 64 bits
            atomicOr(&image[word], static_cast<uint32_t>(spread));
            if (shift + width > 32) atomicOr(&image[word + 1], static_cast<uint32_t>(spread >> 32));
        }
    }
    __syncwarp();
    const uint32_t payload = (n * width + 31) / 32;
    for (uint32_t t = lane; t < payload; t += 32) out[1 + t] = image[t];
}

__global__ void __launch_bounds__(kCodeThreads)
k_values_decode(const uint32_t* __restrict__ words, uint64_t words_per_worker, const uint64_t* __restrict__ block_off,
                uint64_t K, uint64_t n_blocks, float* __restrict__ val_out) {
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t b = static_cast<uint64_t>(blockIdx.x) * kCodeWarps + (threadIdx.x >> 5), w = blockIdx.y;
    if (b >= n_blocks) return;
    const uint64_t first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    float* out = val_out + w * K + first;
    // the stream is untrusted: a block that does not lie inside the worker's words, or whose header no encoder
    // writes, decodes to +0.0 everywhere (a value that changes no parameter), and nothing outside the stream is read
    const uint64_t off = block_off[w * (n_blocks + 1) + b];
    bool sound = off + 1 <= words_per_worker;
    const uint32_t* in = words + w * words_per_worker + (sound ? off : 0);
    const uint32_t header = sound ? __ldg(in) : 0u;
    const uint32_t e_min = header & 0xFFu, w_e = (header >> 8) & 0xFFu, width = 24 + w_e;
    sound = sound && w_e <= 8 && (header >> 16) == 0 && off + 1 + (static_cast<uint64_t>(n) * width + 31) / 32 <= words_per_worker;
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const uint32_t t = r * 32 + lane;
        if (t >= n) continue;
        uint32_t x = 0;
        if (sound) {
            const uint32_t pos = t * width, word = pos >> 5, shift = pos & 31;
            unsigned long long window = __ldg(in + 1 + word);
            if (shift + width > 32) window |= static_cast<unsigned long long>(__ldg(in + 1 + word + 1)) << 32;
            const unsigned long long entry = (window >> shift) & ((1ull << width) - 1ull);
            const uint32_t e = e_min + (static_cast<uint32_t>(entry >> 23) & ((1u << w_e) - 1u));
            x = (static_cast<uint32_t>(entry) & 0x7FFFFFu) | ((e & 0xFFu) << 23) | (static_cast<uint32_t>(entry >> (23 + w_e)) << 31);
            if (e > 255u) x = 0;                                 // an exponent no float has: the block's header lied
        }
        out[t] = __uint_as_float(x);
    }
}

}  // namespace

extern "C" {

uint64_t adacomp_encode_capacity_words(uint64_t pairs_per_worker) {
    return pairs_per_worker + 2 * ((pairs_per_worker + kCodeBlock - 1) / kCodeBlock);
}

int adacomp_encode_indices(const uint32_t* d_idx, uint64_t pairs_per_worker, uint32_t n_workers, uint32_t* d_words,
                           uint64_t words_per_worker, uint64_t* d_block_off, int device, void* cuda_stream) {
    if (n_workers == 0 || n_workers > 65535) return ADACOMP_ERR_INVALID;
    if (!d_block_off) return ADACOMP_ERR_INVALID;
    const uint64_t K = pairs_per_worker, n_blocks = (K + kCodeBlock - 1) / kCodeBlock;
    if (n_blocks > 0x7FFFFFFFull) return ADACOMP_ERR_CAPACITY;
    if (words_per_worker < adacomp_encode_capacity_words(K)) return ADACOMP_ERR_CAPACITY;
    if (K && (!d_idx || !d_words)) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (K == 0) {
        ADACOMP_CUDA(cudaMemsetAsync(d_block_off, 0, n_workers * sizeof(uint64_t), st));
        return ADACOMP_OK;
    }
    const dim3 grid(static_cast<unsigned>((n_blocks + kCodeWarps - 1) / kCodeWarps), n_workers);
    k_encode_measure<<<grid, kCodeThreads, 0, st>>>(d_idx, K, n_blocks, d_block_off);
    ADACOMP_LAUNCH_CHECK();
    k_encode_offsets<<<n_workers, 1024, 0, st>>>(d_block_off, n_blocks);
    ADACOMP_LAUNCH_CHECK();
    k_encode_pack<<<grid, kCodeThreads, 0, st>>>(d_idx, K, n_blocks, d_block_off, d_words, words_per_worker);
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

int adacomp_decode_indices(const uint32_t* d_words, uint64_t words_per_worker, const uint64_t* d_block_off,
                           uint64_t pairs_per_worker, uint32_t n_workers, uint32_t* d_idx_out, int device,
                           void* cuda_stream) {
    if (n_workers == 0 || n_workers > 65535 || !d_block_off) return ADACOMP_ERR_INVALID;
    const uint64_t K = pairs_per_worker, n_blocks = (K + kCodeBlock - 1) / kCodeBlock;
    if (K == 0) return ADACOMP_OK;
    if (n_blocks > 0x7FFFFFFFull) return ADACOMP_ERR_CAPACITY;
    if (!d_words || !d_idx_out) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    k_decode<<<dim3(static_cast<unsigned>((n_blocks + kCodeWarps - 1) / kCodeWarps), n_workers), kCodeThreads, 0,
               static_cast<cudaStream_t>(cuda_stream)>>>(
        d_words, words_per_worker, d_block_off, K, n_blocks, d_idx_out);
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

uint64_t adacomp_encode_values_capacity_words(uint64_t pairs_per_worker) {
    return pairs_per_worker + (pairs_per_worker + kCodeBlock - 1) / kCodeBlock;
}

int adacomp_encode_values(const float* d_val, uint64_t pairs_per_worker, uint32_t n_workers, uint32_t* d_words,
                          uint64_t words_per_worker, uint64_t* d_block_off, int device, void* cuda_stream) {
    if (n_workers == 0 || n_workers > 65535) return ADACOMP_ERR_INVALID;
    if (!d_block_off) return ADACOMP_ERR_INVALID;
    const uint64_t K = pairs_per_worker, n_blocks = (K + kCodeBlock - 1) / kCodeBlock;
    if (n_blocks > 0x7FFFFFFFull) return ADACOMP_ERR_CAPACITY;
    if (words_per_worker < adacomp_encode_values_capacity_words(K)) return ADACOMP_ERR_CAPACITY;
    if (K && (!d_val || !d_words)) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (K == 0) {
        ADACOMP_CUDA(cudaMemsetAsync(d_block_off, 0, n_workers * sizeof(uint64_t), st));
        return ADACOMP_OK;
    }
    const dim3 grid(static_cast<unsigned>((n_blocks + kCodeWarps - 1) / kCodeWarps), n_workers);
    k_values_measure<<<grid, kCodeThreads, 0, st>>>(d_val, K, n_blocks, d_block_off);
    ADACOMP_LAUNCH_CHECK();
    k_encode_offsets<<<n_workers, 1024, 0, st>>>(d_block_off, n_blocks);
    ADACOMP_LAUNCH_CHECK();
    k_values_pack<<<grid, kCodeThreads, 0, st>>>(d_val, K, n_blocks, d_block_off, d_words, words_per_worker);
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

int adacomp_decode_values(const uint32_t* d_words, uint64_t words_per_worker, const uint64_t* d_block_off,
                          uint64_t pairs_per_worker, uint32_t n_workers, float* d_val_out, int device,
                          void* cuda_stream) {
    if (n_workers == 0 || n_workers > 65535 || !d_block_off) return ADACOMP_ERR_INVALID;
    const uint64_t K = pairs_per_worker, n_blocks = (K + kCodeBlock - 1) / kCodeBlock;
    if (K == 0) return ADACOMP_OK;
    if (n_blocks > 0x7FFFFFFFull) return ADACOMP_ERR_CAPACITY;
    if (!d_words || !d_val_out) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    k_values_decode<<<dim3(static_cast<unsigned>((n_blocks + kCodeWarps - 1) / kCodeWarps), n_workers), kCodeThreads, 0,
                      static_cast<cudaStream_t>(cuda_stream)>>>(d_words, words_per_worker, d_block_off, K, n_blocks, d_val_out);
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

}  // extern "C"
