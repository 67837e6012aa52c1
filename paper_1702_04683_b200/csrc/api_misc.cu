// Status strings, version and the keep-count rule.
#include "common.cuh"

namespace adacomp {
thread_local int g_last_cuda_error = 0;
std::atomic<uint64_t> g_kernel_launches{0};
}

extern "C" {

const char* adacomp_status_string(int status) {
    switch (status) {
        case ADACOMP_OK: return "ok";
        case ADACOMP_ERR_INVALID: return "invalid argument";
        case ADACOMP_ERR_ALLOC: return "allocation failed or workspace too small";
        case ADACOMP_ERR_CUDA: return "CUDA runtime error";
        case ADACOMP_ERR_WINDOW: return "pull timestamp outside the kept history window";
        case ADACOMP_ERR_CAPACITY: return "capacity exceeded";
        case ADACOMP_ERR_UNSORTED: return "update indices not strictly ascending or out of range";
        case ADACOMP_ERR_TIMEOUT: return "bounded device wait gave up";
        case ADACOMP_ERR_UNIMPLEMENTED: return "not implemented";
        default: return "unknown status";
    }
}

int adacomp_version(void) { return 100; }

int adacomp_last_cuda_error(void) { return adacomp::g_last_cuda_error; }

uint64_t adacomp_kernel_launches(void) { return adacomp::g_kernel_launches.load(std::memory_order_relaxed); }

// Keep count for a fraction c_num / c_den of a tensor of n entries (Algorithm 1, SELECT_GRAD keeps
// "the (100 x c)% largest"): the ceiling of n * c, clamped to [1, n].
int adacomp_keep_count(uint64_t n, uint32_t c_num, uint32_t c_den, uint32_t* k_out) {
    if (!k_out || c_den == 0 || c_num > c_den || n >= (1ull << 32)) return ADACOMP_ERR_INVALID;
    if (n == 0) {
        *k_out = 0;
        return ADACOMP_OK;
    }
    // n < 2^32 and c_num < 2^32, so the product fits 64 bits
    const uint64_t scaled = n * static_cast<uint64_t>(c_num);
    uint64_t k = scaled / c_den + (scaled % c_den != 0 ? 1 : 0);
    if (k < 1) k = 1;
    if (k > n) k = n;
    *k_out = static_cast<uint32_t>(k);
    return ADACOMP_OK;
}

}  // extern "C"
