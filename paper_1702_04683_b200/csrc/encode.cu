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
// the stream's length.  Three kernels encode (measure every block, prefix-sum the sizes, pack), one
// decodes; a block is one CUDA block of 256 threads, one entry per thread.
#include "common.cuh"

using namespace adacomp;

namespace {

constexpr int kCodeBlock = 256;

__device__ __forceinline__ uint32_t block_max_256(uint32_t v, uint32_t* s_red) {
    v = __reduce_max_sync(0xFFFFFFFFu, v);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t m = s_red[0];
#pragma unroll
    for (int i = 1; i < kCodeBlock / 32; ++i) m = max(m, s_red[i]);
    __syncthreads();
    return m;
}

// the gap of entry t of the block (0 for the block's first entry and past the end) and the block's width
__device__ __forceinline__ uint32_t gap_and_width(const uint32_t* idx, uint64_t first, uint32_t n, uint32_t* s_red, uint32_t* width) {
    const uint32_t t = threadIdx.x;
    uint32_t gap = 0;
    if (t >= 1 && t < n) gap = idx[first + t] - idx[first + t - 1] - 1u;
    const uint32_t widest = block_max_256(gap, s_red);
    *width = widest ? 32u - static_cast<uint32_t>(__clz(widest)) : 0u;
    return gap;
}

__global__ void __launch_bounds__(kCodeBlock)
k_encode_measure(const uint32_t* __restrict__ idx, uint64_t K, uint64_t n_blocks, uint64_t* __restrict__ block_off) {
    __shared__ uint32_t s_red[kCodeBlock / 32];
    const uint64_t b = blockIdx.x, w = blockIdx.y, first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    uint32_t width;
    gap_and_width(idx + w * K, first, n, s_red, &width);
    if (threadIdx.x == 0) {
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

__global__ void __launch_bounds__(kCodeBlock)
k_encode_pack(const uint32_t* __restrict__ idx, uint64_t K, uint64_t n_blocks, const uint64_t* __restrict__ block_off,
              uint32_t* __restrict__ words, uint64_t words_per_worker) {
    __shared__ uint32_t s_red[kCodeBlock / 32];
    __shared__ uint32_t s_bits[kCodeBlock];
    const uint64_t b = blockIdx.x, w = blockIdx.y, first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    const uint32_t t = threadIdx.x;
    s_bits[t] = 0;
    uint32_t width;
    const uint32_t gap = gap_and_width(idx + w * K, first, n, s_red, &width);     // (its barriers also publish s_bits = 0)
    uint32_t* out = words + w * words_per_worker + block_off[w * (n_blocks + 1) + b];
    if (t == 0) {
        out[0] = idx[w * K + first];
        out[1] = width;
    }
    if (t >= 1 && t < n && width) {
        const uint32_t pos = (t - 1) * width, word = pos >> 5, shift = pos & 31;
        const unsigned long long spread = static_cast<unsigned long long>(gap) << shift;
        atomicOr(&s_bits[word], static_cast<uint32_t>(spread));
        if (shift + width > 32) atomicOr(&s_bits[word + 1], static_cast<uint32_t>(spread >> 32));
    }
    __syncthreads();
    const uint32_t payload = ((n - 1) * width + 31) / 32;
    if (t < payload) out[2 + t] = s_bits[t];
}

__global__ void __launch_bounds__(kCodeBlock)
k_decode(const uint32_t* __restrict__ words, uint64_t words_per_worker, const uint64_t* __restrict__ block_off,
         uint64_t K, uint64_t n_blocks, uint32_t* __restrict__ idx_out) {
    __shared__ uint32_t s_warp[kCodeBlock / 32];
    const uint64_t b = blockIdx.x, w = blockIdx.y, first = b * kCodeBlock;
    const uint32_t n = static_cast<uint32_t>(K - first < kCodeBlock ? K - first : kCodeBlock);
    const uint32_t t = threadIdx.x, lane = t & 31, warp = t >> 5;
    // the stream is untrusted (it arrives from a worker): the block must lie inside the worker's words with a
    // width of at most 32 bits, else the block decodes to 0xFFFFFFFF everywhere, an index no server accepts
    // (adacomp_apply skips and reports it), and nothing outside the stream is read
    const uint64_t off = block_off[w * (n_blocks + 1) + b];
    bool sound = off + 2 <= words_per_worker;
    const uint32_t* in = words + w * words_per_worker + (sound ? off : 0);
    uint32_t width = sound ? in[1] : 0u;
    sound = sound && width <= 32 && off + 2 + (static_cast<uint64_t>(n - 1) * width + 31) / 32 <= words_per_worker;
    if (!sound) {
        if (t < n) idx_out[w * K + first + t] = 0xFFFFFFFFu;
        return;
    }
    uint32_t step = 0;                                   // what entry t adds to its predecessor
    if (t == 0) step = in[0];
    else if (t < n) {
        uint32_t gap = 0;
        if (width) {
            const uint32_t pos = (t - 1) * width, word = pos >> 5, shift = pos & 31;
            unsigned long long window = in[2 + word];
            if (shift + width > 32) window |= static_cast<unsigned long long>(in[2 + word + 1]) << 32;
            gap = static_cast<uint32_t>(window >> shift) & (width == 32 ? 0xFFFFFFFFu : ((1u << width) - 1u));
        }
        step = gap + 1u;
    }
    uint32_t v = step;                                   // running sum modulo 2^32: the index
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= static_cast<uint32_t>(d)) v += y;
    }
    if (lane == 31) s_warp[warp] = v;
    __syncthreads();
    uint32_t before = 0;
    for (uint32_t i = 0; i < warp; ++i) before += s_warp[i];
    if (t < n) idx_out[w * K + first + t] = before + v;
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
    const dim3 grid(static_cast<unsigned>(n_blocks), n_workers);
    k_encode_measure<<<grid, kCodeBlock, 0, st>>>(d_idx, K, n_blocks, d_block_off);
    ADACOMP_LAUNCH_CHECK();
    k_encode_offsets<<<n_workers, 1024, 0, st>>>(d_block_off, n_blocks);
    ADACOMP_LAUNCH_CHECK();
    k_encode_pack<<<grid, kCodeBlock, 0, st>>>(d_idx, K, n_blocks, d_block_off, d_words, words_per_worker);
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
    k_decode<<<dim3(static_cast<unsigned>(n_blocks), n_workers), kCodeBlock, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        d_words, words_per_worker, d_block_off, K, n_blocks, d_idx_out);
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

}  // extern "C"
