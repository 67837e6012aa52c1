// AdaComp oracle: a plain, slow, single-threaded CPU statement of what the
// worker-side gradient selection and the parameter-server update compute.
//
// THIS IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be
// checked against something written straight from the paper.  It shares no
// code, header, table or helper with the CUDA path and must never be called
// from it.  Everything here is exact (integer work on fp32 bit patterns, and
// fp32 arithmetic with one rounding per operation), so results are unique.
//
// Parity status: every function below is pinned by tests that do not call it
// to produce their expectation (brute-force set definitions on tiny inputs,
// the paper's worked staleness example, closed forms, invariants; for the
// competitors' global-staleness rule also its agreement with the per-parameter
// rule on full updates, where the two must coincide).  The only
// thing that stays "parity unpinned" is what this file does not compute at
// all: model accuracy and traffic curves, which need the paper's dataset.
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math -shared -fPIC

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>

namespace {

// Magnitude key of a gradient entry: the fp32 bit pattern with the sign bit
// cleared.  For every non-NaN float, unsigned order of this key equals the
// order of |g| ("largest parameters, in absolute value", Algorithm 1,
// SELECT_GRAD); +0 and -0 get the same key.
inline uint32_t magnitude_key(float g) {
    uint32_t bits;
    std::memcpy(&bits, &g, sizeof bits);
    return bits & 0x7FFFFFFFu;
}

// The total order that makes the selection unique: larger magnitude first,
// and among equal magnitudes the lower index first.
struct LargerMagnitudeThenLowerIndex {
    const float* g;
    bool operator()(uint32_t a, uint32_t b) const {
        const uint32_t ka = magnitude_key(g[a]), kb = magnitude_key(g[b]);
        if (ka != kb) return ka > kb;
        return a < b;
    }
};

void emit_ascending(const float* g, std::vector<uint32_t>& chosen, uint64_t offset,
                    uint32_t* idx_out, float* val_out) {
    std::sort(chosen.begin(), chosen.end());
    for (size_t t = 0; t < chosen.size(); ++t) {
        idx_out[t] = static_cast<uint32_t>(offset + chosen[t]);
        val_out[t] = g[chosen[t]];   // the raw gradient entry, bit for bit
    }
}

}  // namespace

extern "C" {

// How many entries a fraction c = c_num / c_den keeps of a tensor of n
// entries: ceil(c * n), at least 1, at most n.  The paper only says "the
// (100 x c)% largest" (Algorithm 1, SELECT_GRAD); the ceiling keeps every
// tensor represented, which is the stated purpose of selecting per tensor
// ("Selection method" paragraph).  n = 0 keeps nothing.
uint32_t oracle_keep_count(uint64_t n, uint32_t c_num, uint32_t c_den) {
    if (n == 0 || c_den == 0) return 0;
    unsigned __int128 prod = static_cast<unsigned __int128>(n) * c_num;
    unsigned __int128 k = (prod + c_den - 1) / c_den;
    if (k < 1) k = 1;
    if (k > n) k = n;
    return static_cast<uint32_t>(k);
}

// SELECT_GRAD on one tensor, written as its definition (Algorithm 1,
// SELECT_GRAD; "Selection method" paragraph): order ALL entries by decreasing
// |g| (ties: lower index first), keep the first k, report them by ascending
// index as (offset + e, g[e]).  Returns 0, or -1 on k > n.
int oracle_select_sort(const float* g, uint32_t n, uint32_t k, uint64_t offset,
                       uint32_t* idx_out, float* val_out) {
    if (k > n) return -1;
    std::vector<uint32_t> order(n);
    std::iota(order.begin(), order.end(), 0u);
    std::sort(order.begin(), order.end(), LargerMagnitudeThenLowerIndex{g});
    std::vector<uint32_t> chosen(order.begin(), order.begin() + k);
    emit_ascending(g, chosen, offset, idx_out, val_out);
    return 0;
}

// The same selection with a partial sort (std::nth_element) under the same
// total order.  The order is strict and total, so the first k elements after
// partitioning are the same set as in oracle_select_sort.  This is the variant
// used on large inputs.
int oracle_select(const float* g, uint32_t n, uint32_t k, uint64_t offset,
                  uint32_t* idx_out, float* val_out) {
    if (k > n) return -1;
    std::vector<uint32_t> order(n);
    std::iota(order.begin(), order.end(), 0u);
    if (k > 0 && k < n)
        std::nth_element(order.begin(), order.begin() + (k - 1), order.end(),
                         LargerMagnitudeThenLowerIndex{g});
    std::vector<uint32_t> chosen(order.begin(), order.begin() + k);
    emit_ascending(g, chosen, offset, idx_out, val_out);
    return 0;
}

// SELECT_GRAD over a whole gradient vector: each tensor (V_l or beta_l) is a
// contiguous range [offset_l, offset_l + n_l) and is selected independently
// (the fraction is "per V_l or beta_l", notation table).  Output: the tensors'
// selections one after the other, sum(k_l) pairs.
int oracle_select_layers(const float* grad, const uint64_t* offsets, const uint32_t* ns,
                         const uint32_t* ks, uint32_t n_layers, int use_full_sort,
                         uint32_t* idx_out, float* val_out) {
    uint64_t out = 0;
    for (uint32_t l = 0; l < n_layers; ++l) {
        int rc = use_full_sort
            ? oracle_select_sort(grad + offsets[l], ns[l], ks[l], offsets[l], idx_out + out, val_out + out)
            : oracle_select(grad + offsets[l], ns[l], ks[l], offsets[l], idx_out + out, val_out + out);
        if (rc != 0) return rc;
        out += ks[l];
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Parameter server (Algorithm 2), two statements of the same function.
// ---------------------------------------------------------------------------

// One fp32 parameter update, Eq. 4 with the learning rate of Eq. 5:
//   alpha_k = alpha / sigma_k  if sigma_k != 0, else alpha
//   Theta_k <- Theta_k - alpha_k * dTheta_k
// Each operation is rounded to fp32 on its own (divide, multiply, subtract);
// the build forbids fusing the last two.
static inline float updated_parameter(float theta_k, float alpha, uint32_t sigma_k, float delta_k) {
    const float alpha_k = (sigma_k != 0) ? alpha / static_cast<float>(sigma_k) : alpha;
    const float step = alpha_k * delta_k;
    return theta_k - step;
}

// --- literal form -----------------------------------------------------------
// Keeps every past update as the set of parameter indices it changed with a
// non-zero value, and evaluates Eq. 3 as written: for each entry of the
// arriving update, test membership of k in every update u = j .. i-1.
struct LiteralServer {
    std::vector<float> theta;
    uint64_t timestamp = 0;                         // i: number of updates applied so far
    std::vector<std::vector<uint32_t>> nonzero_idx; // nonzero_idx[u] = sorted {k : dTheta_k(u) != 0}
};

void* oracle_literal_create(uint64_t n_params, const float* theta0) {
    auto* s = new LiteralServer;
    s->theta.assign(theta0, theta0 + n_params);
    return s;
}
void oracle_literal_destroy(void* h) { delete static_cast<LiteralServer*>(h); }
uint64_t oracle_literal_timestamp(void* h) { return static_cast<LiteralServer*>(h)->timestamp; }
void oracle_literal_theta(void* h, float* out) {
    auto* s = static_cast<LiteralServer*>(h);
    std::copy(s->theta.begin(), s->theta.end(), out);
}

// One iteration of Algorithm 2: Get (update, j), then for every entry of the
// update compute sigma_k (Eq. 3), alpha_k (Eq. 5), the new Theta_k (Eq. 4);
// then the timestamp advances.  An entry whose value is +-0 is present but is
// not a change: it is not recorded for later windows and leaves Theta_k as it
// is; its sigma is still reported.  Returns 0; -1 if j > i, idx out of range
// or idx not strictly ascending.
int oracle_literal_apply(void* h, const uint32_t* idx, const float* val, uint64_t n_pairs,
                         uint64_t j, float alpha, uint32_t* sigma_out) {
    auto* s = static_cast<LiteralServer*>(h);
    const uint64_t i = s->timestamp;
    if (j > i) return -1;
    for (uint64_t e = 0; e < n_pairs; ++e) {
        if (idx[e] >= s->theta.size()) return -1;
        if (e > 0 && idx[e] <= idx[e - 1]) return -1;
    }
    std::vector<uint32_t> changed;
    for (uint64_t e = 0; e < n_pairs; ++e) {
        const uint32_t k = idx[e];
        uint32_t sigma_k = 0;
        for (uint64_t u = j; u < i; ++u)
            if (std::binary_search(s->nonzero_idx[u].begin(), s->nonzero_idx[u].end(), k)) ++sigma_k;
        if (sigma_out) sigma_out[e] = sigma_k;
        if (val[e] != 0.0f) {
            s->theta[k] = updated_parameter(s->theta[k], alpha, sigma_k, val[e]);
            changed.push_back(k);
        }
    }
    s->nonzero_idx.push_back(std::move(changed));
    s->timestamp = i + 1;
    return 0;
}

// --- per-parameter form -----------------------------------------------------
// The text under Eq. 3 reads sigma_k as a count of the updates that changed
// parameter k since the worker's last pull: every parameter keeps the ascending list of
// timestamps at which a non-zero update touched it; sigma_k is how many of
// them are >= j.  Same function as the literal form, cost O(sigma_k) per
// entry, usable on the full-size workloads.
struct ListServer {
    std::vector<float> theta;
    uint64_t timestamp = 0;
    std::vector<std::vector<uint64_t>> touched_at;  // touched_at[k]: ascending timestamps
};

void* oracle_server_create(uint64_t n_params, const float* theta0) {
    auto* s = new ListServer;
    s->theta.assign(theta0, theta0 + n_params);
    s->touched_at.resize(n_params);
    return s;
}
void oracle_server_destroy(void* h) { delete static_cast<ListServer*>(h); }
uint64_t oracle_server_timestamp(void* h) { return static_cast<ListServer*>(h)->timestamp; }
void oracle_server_theta(void* h, float* out) {
    auto* s = static_cast<ListServer*>(h);
    std::copy(s->theta.begin(), s->theta.end(), out);
}

int oracle_server_apply(void* h, const uint32_t* idx, const float* val, uint64_t n_pairs,
                        uint64_t j, float alpha, uint32_t* sigma_out) {
    auto* s = static_cast<ListServer*>(h);
    const uint64_t i = s->timestamp;
    if (j > i) return -1;
    for (uint64_t e = 0; e < n_pairs; ++e) {
        if (idx[e] >= s->theta.size()) return -1;
        if (e > 0 && idx[e] <= idx[e - 1]) return -1;
    }
    for (uint64_t e = 0; e < n_pairs; ++e) {
        const uint32_t k = idx[e];
        const std::vector<uint64_t>& ts = s->touched_at[k];
        uint32_t sigma_k = 0;
        for (size_t t = ts.size(); t > 0 && ts[t - 1] >= j; --t) ++sigma_k;
        if (sigma_out) sigma_out[e] = sigma_k;
        if (val[e] != 0.0f) {
            s->theta[k] = updated_parameter(s->theta[k], alpha, sigma_k, val[e]);
            s->touched_at[k].push_back(i);
        }
    }
    s->timestamp = i + 1;
    return 0;
}

// --- the competitors' rule ------------------------------------------------------
// ASGD and Comp-ASGD ("Experimental setup"): one learning rate per update, the
// base rate over the update's staleness.  The staleness of an update is the
// number of times Theta has evolved between the fetch at timestamp j and the push
// at timestamp i ("The parameter server model": w2's update on Figure 2 has
// staleness 2), i.e. sigma = i - j, the same for every entry of the update.  The
// update itself is Eq. 4 with alpha / sigma (alpha when sigma = 0, as in Eq. 5),
// applied to every entry as written: no history is needed and none is kept.
struct GlobalServer {
    std::vector<float> theta;
    uint64_t timestamp = 0;
};

void* oracle_global_create(uint64_t n_params, const float* theta0) {
    auto* s = new GlobalServer;
    s->theta.assign(theta0, theta0 + n_params);
    return s;
}
void oracle_global_destroy(void* h) { delete static_cast<GlobalServer*>(h); }
uint64_t oracle_global_timestamp(void* h) { return static_cast<GlobalServer*>(h)->timestamp; }
void oracle_global_theta(void* h, float* out) {
    auto* s = static_cast<GlobalServer*>(h);
    std::copy(s->theta.begin(), s->theta.end(), out);
}

// A sparse update (Comp-ASGD: a selection of the gradient entries).
int oracle_global_apply(void* h, const uint32_t* idx, const float* val, uint64_t n_pairs,
                        uint64_t j, float alpha, uint32_t* sigma_out) {
    auto* s = static_cast<GlobalServer*>(h);
    const uint64_t i = s->timestamp;
    if (j > i || i - j > 0xFFFFFFFFull) return -1;
    for (uint64_t e = 0; e < n_pairs; ++e) {
        if (idx[e] >= s->theta.size()) return -1;
        if (e > 0 && idx[e] <= idx[e - 1]) return -1;
    }
    const uint32_t sigma = static_cast<uint32_t>(i - j);
    for (uint64_t e = 0; e < n_pairs; ++e) {
        if (sigma_out) sigma_out[e] = sigma;
        s->theta[idx[e]] = updated_parameter(s->theta[idx[e]], alpha, sigma, val[e]);
    }
    s->timestamp = i + 1;
    return 0;
}

// A dense update (ASGD: the whole gradient).
int oracle_global_apply_dense(void* h, const float* delta, uint64_t j, float alpha) {
    auto* s = static_cast<GlobalServer*>(h);
    const uint64_t i = s->timestamp;
    if (j > i || i - j > 0xFFFFFFFFull) return -1;
    const uint32_t sigma = static_cast<uint32_t>(i - j);
    for (size_t k = 0; k < s->theta.size(); ++k) s->theta[k] = updated_parameter(s->theta[k], alpha, sigma, delta[k]);
    s->timestamp = i + 1;
    return 0;
}

// Values of chosen entries: val[e] = g[idx[e]] (a selection made elsewhere, e.g. at random).
int oracle_gather(const float* g, uint64_t n, const uint32_t* idx, uint64_t n_pairs, float* val_out) {
    for (uint64_t e = 0; e < n_pairs; ++e) {
        if (idx[e] >= n) return -1;
        val_out[e] = g[idx[e]];
    }
    return 0;
}

// --- index coding -------------------------------------------------------------------
// The paper leaves the encoding of the (index, value) pairs open (footnote of
// "Algorithm details").  This is the format the library offers for the index half,
// stated entry by entry; values travel as they are.  An update's ascending index
// list is cut into blocks of 256 entries.  A block is stored as
//   word 0      the first index of the block,
//   word 1      w = the number of bits of the largest gap in the block, where the gap
//               of an entry is (index - previous index - 1), modulo 2^32,
//   then        the gaps of entries 1 .. n-1 of the block, w bits each, entry e at bit
//               (e - 1) * w of a little-endian bit string held in 32-bit words
//               (ceil((n - 1) * w / 32) words; none if w = 0).
// block_off[b] is the word at which block b starts; block_off[n_blocks] the total.
static inline uint32_t bits_needed(uint32_t x) {
    uint32_t n = 0;
    while (x) { ++n; x >>= 1; }
    return n;
}

uint64_t oracle_encode_indices(const uint32_t* idx, uint64_t n_pairs, uint32_t* words_out, uint64_t* block_off_out) {
    uint64_t at = 0, n_blocks = (n_pairs + 255) / 256;
    for (uint64_t b = 0; b < n_blocks; ++b) {
        const uint64_t first = b * 256, n = std::min<uint64_t>(256, n_pairs - first);
        block_off_out[b] = at;
        uint32_t widest = 0;
        for (uint64_t e = 1; e < n; ++e) widest = std::max(widest, bits_needed(idx[first + e] - idx[first + e - 1] - 1u));
        words_out[at++] = idx[first];
        words_out[at++] = widest;
        const uint64_t payload = ((n - 1) * widest + 31) / 32;
        for (uint64_t i = 0; i < payload; ++i) words_out[at + i] = 0;
        for (uint64_t e = 1; e < n; ++e) {
            const uint64_t gap = idx[first + e] - idx[first + e - 1] - 1u;      // 32 bits, zero-extended
            for (uint32_t bit = 0; bit < widest; ++bit) {                        // bit by bit, as the format is defined
                const uint64_t pos = (e - 1) * widest + bit;
                if ((gap >> bit) & 1u) words_out[at + pos / 32] |= 1u << (pos % 32);
            }
        }
        at += payload;
    }
    block_off_out[n_blocks] = at;
    return at;
}

int oracle_decode_indices(const uint32_t* words, const uint64_t* block_off, uint64_t n_pairs, uint32_t* idx_out) {
    const uint64_t n_blocks = (n_pairs + 255) / 256;
    for (uint64_t b = 0; b < n_blocks; ++b) {
        const uint64_t first = b * 256, n = std::min<uint64_t>(256, n_pairs - first), at = block_off[b];
        const uint32_t widest = words[at + 1];
        if (widest > 32) return -1;
        uint32_t k = words[at];
        idx_out[first] = k;
        for (uint64_t e = 1; e < n; ++e) {
            uint32_t gap = 0;
            for (uint32_t bit = 0; bit < widest; ++bit) {
                const uint64_t pos = (e - 1) * widest + bit;
                gap |= ((words[at + 2 + pos / 32] >> (pos % 32)) & 1u) << bit;
            }
            k = k + gap + 1u;
            idx_out[first + e] = k;
        }
    }
    return 0;
}

// --- value packing ----------------------------------------------------------------
// The value half of the same open point (footnote of "Algorithm details"), lossless:
// every fp32 bit pattern comes back as it went in, so Eq. 4 sees the same inputs.  The
// values of an update are cut into blocks of 256 entries, as the indices are.  With
// E(x) = the 8-bit exponent field of x (bits 30..23), a block is stored as
//   word 0      e_min | w_e << 8: e_min the smallest E in the block, w_e the number of
//               bits of the largest (E - e_min), 0..8,
//   then        the n entries, 24 + w_e bits each, entry t at bit t * (24 + w_e) of a
//               little-endian bit string held in 32-bit words; an entry is the 23 mantissa
//               bits, above them (E - e_min) in w_e bits, above that the sign bit.
// The largest magnitudes of a tensor lie within a few powers of two of each other, so
// w_e is 2 or 3 and a value costs 26 or 27 bits instead of 32.
uint64_t oracle_encode_values(const float* val, uint64_t n_pairs, uint32_t* words_out, uint64_t* block_off_out) {
    uint64_t at = 0, n_blocks = (n_pairs + 255) / 256;
    for (uint64_t b = 0; b < n_blocks; ++b) {
        const uint64_t first = b * 256, n = std::min<uint64_t>(256, n_pairs - first);
        block_off_out[b] = at;
        uint32_t e_min = 255, e_max = 0;
        for (uint64_t t = 0; t < n; ++t) {
            uint32_t bits;
            std::memcpy(&bits, &val[first + t], 4);
            const uint32_t e = (bits >> 23) & 0xFFu;
            e_min = std::min(e_min, e);
            e_max = std::max(e_max, e);
        }
        const uint32_t w_e = bits_needed(e_max - e_min), width = 24 + w_e;
        words_out[at++] = e_min | (w_e << 8);
        const uint64_t payload = (n * width + 31) / 32;
        for (uint64_t i = 0; i < payload; ++i) words_out[at + i] = 0;
        for (uint64_t t = 0; t < n; ++t) {
            uint32_t bits;
            std::memcpy(&bits, &val[first + t], 4);
            const uint64_t mantissa = bits & 0x7FFFFFu, e_rel = ((bits >> 23) & 0xFFu) - e_min, sign = bits >> 31;
            const uint64_t entry = mantissa | (e_rel << 23) | (sign << (23 + w_e));
            for (uint32_t bit = 0; bit < width; ++bit) {                          // bit by bit, as the format is defined
                const uint64_t pos = t * width + bit;
                if ((entry >> bit) & 1u) words_out[at + pos / 32] |= 1u << (pos % 32);
            }
        }
        at += payload;
    }
    block_off_out[n_blocks] = at;
    return at;
}

int oracle_decode_values(const uint32_t* words, const uint64_t* block_off, uint64_t n_pairs, float* val_out) {
    const uint64_t n_blocks = (n_pairs + 255) / 256;
    for (uint64_t b = 0; b < n_blocks; ++b) {
        const uint64_t first = b * 256, n = std::min<uint64_t>(256, n_pairs - first), at = block_off[b];
        const uint32_t e_min = words[at] & 0xFFu, w_e = (words[at] >> 8) & 0xFFu, width = 24 + w_e;
        if (w_e > 8 || (words[at] >> 16) != 0) return -1;
        for (uint64_t t = 0; t < n; ++t) {
            uint64_t entry = 0;
            for (uint32_t bit = 0; bit < width; ++bit) {
                const uint64_t pos = t * width + bit;
                entry |= static_cast<uint64_t>((words[at + 1 + pos / 32] >> (pos % 32)) & 1u) << bit;
            }
            const uint32_t mantissa = static_cast<uint32_t>(entry & 0x7FFFFFu);
            const uint32_t e = e_min + static_cast<uint32_t>((entry >> 23) & ((1u << w_e) - 1u));
            const uint32_t sign = static_cast<uint32_t>((entry >> (23 + w_e)) & 1u);
            if (e > 255) return -1;
            const uint32_t bits = mantissa | (e << 23) | (sign << 31);
            std::memcpy(&val_out[first + t], &bits, 4);
        }
    }
    return 0;
}

// --- one parameter at a time --------------------------------------------------
// The history of a single parameter k through a whole sequence of updates,
// computed the way the paper's complexity paragraph describes it: each update
// keeps its sorted index list, and Eq. 3 is a membership search per update in
// the window.  Lets a test check sampled parameters of a workload that is too
// large to replay in full.  pair_begin[u] .. pair_begin[u+1] delimit update u
// inside idx/val; pull_ts[u] is its j; update u is applied at timestamp
// first_timestamp + u, and nothing touched k before first_timestamp.
// Writes the sigma of each update that contains k to sigma_out (in order,
// at most n_updates values), their number to *n_hits, the final value to
// *theta_k.  Returns 0, or -1 if some j is out of range.
int oracle_parameter_trace(uint32_t k, float theta0_k, const uint32_t* idx, const float* val,
                           const uint64_t* pair_begin, const uint64_t* pull_ts, uint64_t n_updates,
                           uint64_t first_timestamp, float alpha,
                           uint32_t* sigma_out, uint64_t* n_hits, float* theta_k) {
    float theta = theta0_k;
    uint64_t hits = 0;
    std::vector<char> changed_k(n_updates, 0);   // did update u change k with a non-zero value
    for (uint64_t u = 0; u < n_updates; ++u) {
        const uint64_t i = first_timestamp + u, j = pull_ts[u];
        if (j > i) return -1;
        const uint32_t* lo = idx + pair_begin[u];
        const uint32_t* hi = idx + pair_begin[u + 1];
        const uint32_t* at = std::lower_bound(lo, hi, k);
        if (at == hi || *at != k) continue;
        uint32_t sigma_k = 0;
        for (uint64_t t = (j > first_timestamp ? j - first_timestamp : 0); t < u; ++t)
            sigma_k += changed_k[t];
        if (sigma_out) sigma_out[hits] = sigma_k;
        ++hits;
        const float v = val[at - idx];
        if (v != 0.0f) {
            theta = updated_parameter(theta, alpha, sigma_k, v);
            changed_k[u] = 1;
        }
    }
    *n_hits = hits;
    *theta_k = theta;
    return 0;
}

}  // extern "C"
