// Worker side of libadacomp: handle, workspace layout and launch sequence of SELECT_GRAD
// (Algorithm 1).
#include <cmath>
#include <mutex>
#include <new>
#include <vector>

#include "select_cluster.cuh"

using namespace adacomp;

namespace {
constexpr int kSelectStages = 11;
constexpr int kProfileRing = 32;
const char* const kStageNames[kSelectStages] = {
    "bracket_sample", "bracket_scan", "bracket_resolve", "bracket_emit", "general_plan",
    "general_hist0", "general_hist1", "general_hist2", "general_count", "general_write", "fallback_solo"};
}  // namespace

struct adacomp_select {
    int device = 0;
    int n_sms = 0;
    int route = 0;         // 0 = automatic, 1 = general route for everything
    bool all_bracketed = false;   // every tensor with k > 0 is eligible for the bracketed route
    bool any_small = false;       // some tensor is selected whole in shared memory by the sample kernel
    bool emit_thin = false;       // every tensor of the list route expects a handful of candidates per piece: a lane per piece writes them
    // cluster route: large tensors selected by one thread-block cluster each, everything between the pass and the write on chip
    uint32_t n_cl = 0;            // tensors on the cluster route
    uint32_t cl_ctas = 0, cl_warps = 0, cl_ring = 0, cl_qmax = 0, cl_smem = 0;   // blocks per cluster, warps per block, ring slots per warp, most pieces per block, shared memory per block
    int cl_active = 0;            // clusters the device keeps resident
    uint32_t* d_cl_layers = nullptr;
    uint32_t n_layers = 0, max_workers = 0, slots_per_worker = 0, n_items = 0, max_sample = 0;
    uint64_t extent = 0;   // one past the last entry any segment covers
    uint64_t K = 0;        // pairs per worker
    uint64_t cand_stride = 0, win_stride = 0, span_stride = 0;
    // device (inside the caller's workspace)
    Layer* d_layers = nullptr;
    Inst* d_inst = nullptr;
    uint32_t* d_hist = nullptr;
    uint32_t* d_list = nullptr;
    uint32_t* d_list_slot_start = nullptr;
    uint32_t* d_list_len = nullptr;
    uint2* d_chunk_cnt = nullptr;
    int* d_status = nullptr;
    uint2* d_items = nullptr;
    uint32_t* d_cand_idx = nullptr;
    float* d_cand_val = nullptr;
    uint32_t* d_win_key = nullptr;
    uint32_t* d_win_idx = nullptr;
    uint2* d_sub_tab = nullptr;
    uint32_t* d_span_off = nullptr;
    // optional stage timing: a ring of event lists, one per call, folded into sums when reused or read
    int profiling = 0;            // 0 off, 1 events around every kernel, 2 around the pass over the gradient only
    struct Span { int stage; cudaEvent_t a, b; };
    std::vector<Span> spans[kProfileRing];
    size_t spans_used[kProfileRing] = {};
    bool ring_used[kProfileRing] = {};
    int ring_next = 0;
    double stage_ms_sum[kSelectStages] = {};
    uint64_t profiled_calls = 0;
};

namespace {

struct Layout {
    std::vector<Layer> layers;
    std::vector<uint2> items;          // scan / emit work items: (tensor, first span)
    std::vector<double> cand_frac;     // [tensor] expected fraction of candidates (0: not on a bracketed route)
    uint64_t extent = 0, K = 0;
    uint64_t cand_stride = 0, win_stride = 0, span_stride = 0;
    uint32_t slots_per_worker = 0, max_sample = 0;
    bool any_small = false;            // some tensor is selected whole in shared memory by the sample kernel
};

// Decides whether a tensor takes the bracketed route and how much room its lists get.  The
// capacities follow the bracket's expected size plus six standard deviations of the sample
// quantiles; exceeding them is not an error, it only sends the instance to the general route.
void plan_bracket(Layer& L, Layout* out) {
    L.bracket = 0;
    L.cluster = L.pad = 0;
    L.sample = L.n_spans = L.span_base = L.cand_cap = L.win_cap = 0;
    L.cand_base = L.win_base = 0;
    if (L.n < kBracketMinN || L.n > kBracketMaxN || L.k == 0 || static_cast<uint64_t>(L.k) * 4 > L.n) {
        if (L.k > 0 && L.n <= kSmallMax) {                     // small enough for the keys to sit in shared memory whole
            L.bracket = kRouteSmall;
            if (L.n > out->max_sample) out->max_sample = L.n;
        }
        return;
    }
    const uint32_t n_spans = static_cast<uint32_t>((static_cast<uint64_t>(L.n) + 3 + kSpanElems - 1) / kSpanElems);
    uint32_t m = L.n / 8;
    if (m > kSampleMax) m = kSampleMax;
    if (m < kSampleMin) m = kSampleMin;
    m &= ~31u;
    uint32_t r_hi, r_lo;
    bracket_ranks(L.n, L.k, m, &r_hi, &r_lo);
    if (r_lo + 1 > m) return;                              // sample cannot bound the threshold from below
    const double n = L.n;
    const double lo_frac = static_cast<double>(r_lo + 1) / m;
    const double win_frac = static_cast<double>(r_lo + 1 - r_hi) / m;
    double cand = n * lo_frac * (1.0 + 6.0 / std::sqrt(static_cast<double>(r_lo))) + 2048.0;
    double win = n * win_frac * (1.0 + 6.0 / std::sqrt(static_cast<double>(r_lo + 1 - r_hi))) + 2048.0;
    if (cand > n) cand = n;
    if (win > n) win = n;
    L.bracket = 1;
    out->cand_frac.back() = lo_frac;
    L.sample = m;
    L.n_spans = n_spans;
    L.span_base = static_cast<uint32_t>(out->span_stride);
    L.cand_cap = static_cast<uint32_t>(cand);
    L.win_cap = static_cast<uint32_t>(win);
    L.cand_base = out->cand_stride;
    L.win_base = out->win_stride;
    out->span_stride += n_spans;
    out->cand_stride += (L.cand_cap + 63) & ~63ull;
    out->win_stride += (L.win_cap + 63) & ~63ull;
    if (m > out->max_sample) out->max_sample = m;
}

// Work items of the list route's scan and emit kernels: the tensors whose Layer::bracket is 1.
void build_items(Layout* out) {
    out->items.clear();
    for (uint32_t l = 0; l < out->layers.size(); ++l) {
        const Layer& L = out->layers[l];
        for (uint32_t s0 = 0; L.bracket == 1 && s0 < L.n_spans; s0 += kSpansPerBlock) out->items.push_back(make_uint2(l, s0));
    }
}

// Chooses the tensors of the cluster route on this device: bracketed tensors of at least kClMinN entries whose
// expected candidates (with a margin) fit the value stores of a cluster.  Clusters of 8 blocks if every such
// tensor fits them, else of 16 where the device takes clusters of that size; what fits neither stays on the
// list route.  Fills h->cl_* and re-labels the chosen layers; returns their indices.
std::vector<uint32_t> plan_cluster_route(adacomp_select_t* h, Layout* lay, int device) {
    std::vector<uint32_t> chosen;
    int smem_optin = 0;
    if (cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess || smem_optin < 160 * 1024)
        return chosen;
    std::vector<uint32_t> large;
    for (uint32_t l = 0; l < lay->layers.size(); ++l)
        if (lay->layers[l].bracket == 1 && lay->layers[l].n >= kClMinN) large.push_back(l);
    if (large.empty()) return chosen;
    auto pieces_of = [&](uint32_t l) { return (lay->layers[l].n + 3u + kClPiece - 1u) / kClPiece; };
    // does tensor l fit clusters of C blocks of n_warps warps with `ring` ring slots per warp when no block holds more than q_max pieces?
    auto fits = [&](uint32_t l, uint32_t C, uint32_t n_warps, uint32_t ring, uint32_t q_max) {
        const ClusterLayout y = cluster_layout(n_warps, ring, q_max, static_cast<uint32_t>(smem_optin));
        const double per_block = lay->layers[l].n * lay->cand_frac[l] / C;
        return per_block * 1.12 + 1024.0 <= static_cast<double>(y.vals_cap);
    };
    // how many clusters of C blocks stay resident (0: the device does not take them)
    auto resident = [&](uint32_t C, uint32_t n_warps) -> int {
        if (cudaFuncSetAttribute(k_select_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess) return 0;
        if (C > 8 && cudaFuncSetAttribute(k_select_cluster, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) return 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(C);
        cfg.blockDim = dim3(n_warps * 32);
        cfg.dynamicSmemBytes = static_cast<size_t>(smem_optin);
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = C;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, k_select_cluster, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
        return n;
    };
    // block shapes in order of preference: more warps and more bytes in flight first, a larger value store last
    const uint32_t shapes[4][2] = {{16, 2}, {12, 2}, {8, 3}, {8, 2}};
    uint32_t best_C = 0, best_warps = 0, best_ring = 0, best_q = 0;
    std::vector<uint32_t> best_set;
    for (uint32_t C : {8u, 16u}) {
        uint32_t q_max = 0;
        for (uint32_t l : large) q_max = std::max(q_max, (pieces_of(l) + C - 1) / C);
        for (const auto& shape : shapes) {
            if (!cluster_layout_ok(shape[0], shape[1], q_max)) continue;
            std::vector<uint32_t> set;
            for (uint32_t l : large) if (fits(l, C, shape[0], shape[1], q_max)) set.push_back(l);
            if (set.size() > best_set.size()) { best_set = set; best_C = C; best_warps = shape[0]; best_ring = shape[1]; best_q = q_max; }
        }
        if (best_set.size() == large.size()) break;        // everything fits: no need for larger clusters
    }
    if (best_set.empty()) return chosen;
    const int n_resident = resident(best_C, best_warps);
    if (n_resident < 1) return chosen;
    h->cl_ctas = best_C;
    h->cl_warps = best_warps;
    h->cl_ring = best_ring;
    h->cl_qmax = best_q;
    h->cl_smem = static_cast<uint32_t>(smem_optin);
    h->cl_active = n_resident;
    for (uint32_t l : best_set) lay->layers[l].cluster = 1;
    return best_set;
}

int build_layout(const adacomp_segment_t* segs, uint32_t n_segs, uint32_t max_workers, Layout* out) {
    if (!segs || n_segs == 0 || max_workers == 0) return ADACOMP_ERR_INVALID;
    constexpr uint64_t kMaxIndex = 0xFFFFFFFEull;
    uint64_t end_prev = 0, K = 0, slots = 0;
    out->layers.resize(n_segs);
    for (uint32_t l = 0; l < n_segs; ++l) {
        const adacomp_segment_t& s = segs[l];
        if (s.k > s.n) return ADACOMP_ERR_INVALID;
        if (s.offset < end_prev) return ADACOMP_ERR_INVALID;             // overlap or not ascending
        if (s.offset + s.n > kMaxIndex) return ADACOMP_ERR_INVALID;      // indices are uint32
        Layer& L = out->layers[l];
        L.offset = s.offset;
        L.out_offset = K;
        L.n = s.n;
        L.k = s.k;
        L.n_slots = static_cast<uint32_t>((static_cast<uint64_t>(s.n) + 3 + kChunkElems - 1) / kChunkElems);
        if (L.n_slots == 0) L.n_slots = 1;
        L.slot_base = static_cast<uint32_t>(slots);
        slots += L.n_slots;
        K += s.k;
        end_prev = s.offset + s.n;
        out->cand_frac.push_back(0.0);
        plan_bracket(L, out);
        if (L.bracket == kRouteSmall) out->any_small = true;
    }
    build_items(out);
    if (K > kMaxIndex || slots * max_workers > 0x7FFFFFFFull ||
        static_cast<uint64_t>(n_segs) * max_workers > 0x7FFFFFFFull ||
        out->span_stride * max_workers > 0x7FFFFFFFull || out->items.size() > 0x7FFFFFFFull)
        return ADACOMP_ERR_INVALID;
    out->extent = end_prev;
    out->K = K;
    out->slots_per_worker = static_cast<uint32_t>(slots);
    return ADACOMP_OK;
}

// One place that decides the workspace layout; with a null base it only measures.
size_t carve(adacomp_select_t* h, void* base, const Layout& lay, uint32_t max_workers) {
    Carver c(base);
    const size_t W = max_workers;
    const size_t n_inst = lay.layers.size() * W;
    h->d_layers = c.take<Layer>(lay.layers.size());
    h->d_inst = c.take<Inst>(n_inst);
    h->d_hist = c.take<uint32_t>(n_inst * kBins);
    h->d_list = c.take<uint32_t>(n_inst);
    h->d_list_slot_start = c.take<uint32_t>(n_inst);
    h->d_list_len = c.take<uint32_t>(2);
    h->d_chunk_cnt = c.take<uint2>(lay.slots_per_worker * W);
    h->d_status = c.take<int>(1);
    h->d_items = c.take<uint2>(lay.items.size() + 1);
    h->d_cand_idx = c.take<uint32_t>(lay.cand_stride * W);
    h->d_cand_val = c.take<float>(lay.cand_stride * W);
    h->d_win_key = c.take<uint32_t>(lay.win_stride * W);
    h->d_win_idx = c.take<uint32_t>(lay.win_stride * W);
    h->d_sub_tab = c.take<uint2>(lay.span_stride * W * kSubsPerSpan + 1);
    h->d_span_off = c.take<uint32_t>(lay.span_stride * W + 1);
    h->d_cl_layers = c.take<uint32_t>(lay.layers.size());
    return c.used;
}

// Adds the stage times of one finished (or finishing: waits for it) call to the sums.
cudaError_t fold_profile_slot(adacomp_select_t* h, int slot) {
    if (!h->ring_used[slot]) return cudaSuccess;
    for (size_t i = 0; i < h->spans_used[slot]; ++i) {
        const adacomp_select::Span& sp = h->spans[slot][i];
        cudaError_t e = cudaEventSynchronize(sp.b);
        if (e != cudaSuccess) return e;
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, sp.a, sp.b);
        if (e != cudaSuccess) return e;
        h->stage_ms_sum[sp.stage] += ms;
    }
    h->spans_used[slot] = 0;
    h->ring_used[slot] = false;
    h->profiled_calls += 1;
    return cudaSuccess;
}

}  // namespace

extern "C" {

int adacomp_select_workspace_bytes(const adacomp_segment_t* h_segs, uint32_t n_segs,
                                   uint32_t max_workers, size_t* bytes_out) {
    if (!bytes_out) return ADACOMP_ERR_INVALID;
    Layout lay;
    int rc = build_layout(h_segs, n_segs, max_workers, &lay);
    if (rc != ADACOMP_OK) return rc;
    adacomp_select_t tmp;
    *bytes_out = carve(&tmp, nullptr, lay, max_workers);
    return ADACOMP_OK;
}

int adacomp_select_create(adacomp_select_t** h, const adacomp_segment_t* h_segs, uint32_t n_segs,
                          uint32_t max_workers, void* d_workspace, size_t workspace_bytes, int device) {
    if (!h) return ADACOMP_ERR_INVALID;
    *h = nullptr;
    if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) % kAlign) != 0) return ADACOMP_ERR_INVALID;
    Layout lay;
    int rc = build_layout(h_segs, n_segs, max_workers, &lay);
    if (rc != ADACOMP_OK) return rc;
    adacomp_select_t* s = new (std::nothrow) adacomp_select_t;
    if (!s) return ADACOMP_ERR_ALLOC;
    const size_t need = carve(s, d_workspace, lay, max_workers);
    if (need > workspace_bytes) { delete s; return ADACOMP_ERR_ALLOC; }
    s->device = device;
    s->n_layers = n_segs;
    s->max_workers = max_workers;
    s->slots_per_worker = lay.slots_per_worker;
    s->extent = lay.extent;
    s->K = lay.K;
    s->n_items = static_cast<uint32_t>(lay.items.size());
    s->all_bracketed = true;
    for (const Layer& L : lay.layers)
        if (L.k > 0 && !L.bracket) s->all_bracketed = false;
    s->max_sample = lay.max_sample;
    s->any_small = lay.any_small;
    {   // at most about six candidates per 1024-entry piece everywhere: the thin form of the ordered write
        double most = 0.0;
        for (uint32_t l = 0; l < lay.layers.size(); ++l)
            if (lay.layers[l].bracket == 1 && lay.cand_frac[l] > most) most = lay.cand_frac[l];
        s->emit_thin = most > 0.0 && most * kSubElems <= 6.0;      // measured: at ten per piece the warp-per-span form is faster again
    }
    s->cand_stride = lay.cand_stride;
    s->win_stride = lay.win_stride;
    s->span_stride = lay.span_stride;
    DeviceGuard guard(device);
    cudaError_t e = guard.err;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&s->n_sms, cudaDevAttrMultiProcessorCount, device);
    std::vector<uint32_t> cl_layers;
    if (e == cudaSuccess) {
        try { cl_layers = plan_cluster_route(s, &lay, device); } catch (...) { delete s; return ADACOMP_ERR_ALLOC; }
        s->n_cl = static_cast<uint32_t>(cl_layers.size());
        s->n_items = static_cast<uint32_t>(lay.items.size());
    }
    if (e == cudaSuccess && !cl_layers.empty())
        e = cudaMemcpy(s->d_cl_layers, cl_layers.data(), cl_layers.size() * sizeof(uint32_t), cudaMemcpyHostToDevice);
    // only the bookkeeping needs clearing; the candidate / window lists are write-before-read
    if (e == cudaSuccess) {
        const size_t head = reinterpret_cast<char*>(s->d_items) - static_cast<char*>(d_workspace);
        e = cudaMemset(d_workspace, 0, head);
    }
    if (e == cudaSuccess)
        e = cudaMemcpy(s->d_layers, lay.layers.data(), lay.layers.size() * sizeof(Layer), cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !lay.items.empty())
        e = cudaMemcpy(s->d_items, lay.items.data(), lay.items.size() * sizeof(uint2), cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_bracket_sample<kBigFew>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kSmallMax * sizeof(uint32_t)));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_bracket_sample<kBigMany>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kSmallMax * sizeof(uint32_t)));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_bracket_scan, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(kDenseSmemPerWarp * (kThreads / 32)));
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { delete s; return cuda_fail(e); }
    *h = s;
    return ADACOMP_OK;
}

int adacomp_select_route_info(const adacomp_select_t* h, uint32_t* h_info_out) {
    if (!h || !h_info_out) return ADACOMP_ERR_INVALID;
    h_info_out[0] = h->n_cl;
    h_info_out[1] = h->cl_ctas;
    h_info_out[2] = h->cl_ring | (h->cl_warps << 8);
    h_info_out[3] = static_cast<uint32_t>(h->cl_active);
    return ADACOMP_OK;
}

int adacomp_select_set_route(adacomp_select_t* h, int route) {
    if (!h || route < 0 || route > 2) return ADACOMP_ERR_INVALID;
    h->route = route;
    return ADACOMP_OK;
}

int adacomp_select(adacomp_select_t* h, const float* d_grads, uint64_t worker_stride_elems,
                   uint32_t n_workers, uint32_t* d_idx_out, float* d_val_out, void* cuda_stream) {
    if (!h || !d_grads || n_workers == 0 || n_workers > h->max_workers) return ADACOMP_ERR_INVALID;
    if (h->K > 0 && (!d_idx_out || !d_val_out)) return ADACOMP_ERR_INVALID;
    if (n_workers > 1 && worker_stride_elems < h->extent) return ADACOMP_ERR_INVALID;
    if (reinterpret_cast<uintptr_t>(d_grads) % 4 != 0) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    SelectParams p;
    p.grads = d_grads;
    p.stride = worker_stride_elems;
    p.n_workers = n_workers;
    p.n_layers = h->n_layers;
    p.layers = h->d_layers;
    p.inst = h->d_inst;
    p.hist = h->d_hist;
    p.list = h->d_list;
    p.list_slot_start = h->d_list_slot_start;
    p.list_len = h->d_list_len;
    p.chunk_cnt = h->d_chunk_cnt;
    p.slots_per_worker = h->slots_per_worker;
    p.idx_out = d_idx_out;
    p.val_out = d_val_out;
    p.K = h->K;
    p.status = h->d_status;
    p.items = h->d_items;
    p.cand_idx = h->d_cand_idx;
    p.cand_val = h->d_cand_val;
    p.win_key = h->d_win_key;
    p.win_idx = h->d_win_idx;
    p.sub_tab = h->d_sub_tab;
    p.span_off = h->d_span_off;
    p.cand_stride = h->cand_stride;
    p.win_stride = h->win_stride;
    p.span_stride = h->span_stride;

    const unsigned n_inst = n_workers * h->n_layers;
    const bool bracketed = h->route != 1 && (h->n_items > 0 || h->any_small);
    const bool clusters = bracketed && h->route == 2 && h->n_cl > 0;
    int slot = 0;
    if (h->profiling) {                                   // take the next event list of the ring
        slot = h->ring_next;
        h->ring_next = (h->ring_next + 1) % kProfileRing;
        ADACOMP_CUDA(fold_profile_slot(h, slot));         // its previous user finished long ago
        h->ring_used[slot] = true;
    }
    // begin(stage) ... end(): CUDA events around one launch (only while profiling)
    bool recording = false;
    auto begin = [&](int stage) -> cudaError_t {
        recording = h->profiling == 1 || (h->profiling == 2 && stage == 1);
        if (!recording) return cudaSuccess;
        std::vector<adacomp_select::Span>& v = h->spans[slot];
        if (h->spans_used[slot] == v.size()) {
            adacomp_select::Span sp = {stage, nullptr, nullptr};
            cudaError_t e = cudaEventCreate(&sp.a);
            if (e == cudaSuccess) e = cudaEventCreate(&sp.b);
            if (e != cudaSuccess) return e;
            try { v.push_back(sp); } catch (...) { return cudaErrorMemoryAllocation; }
        }
        v[h->spans_used[slot]].stage = stage;
        return cudaEventRecord(v[h->spans_used[slot]].a, st);
    };
    auto end = [&]() -> cudaError_t {
        if (!recording) return cudaSuccess;
        return cudaEventRecord(h->spans[slot][h->spans_used[slot]++].b, st);
    };

    // single-pass routes: sample (and the tensors that are selected on chip), the one pass over the gradient,
    // the exact threshold, the ordered write
    ADACOMP_CUDA(begin(0));
    // per-instance kernels: smaller blocks when the instances are many (more of them resident, finer rounds)
    const bool many = n_inst > 2u * static_cast<uint32_t>(h->n_sms);
    const size_t sample_smem = bracketed ? h->max_sample * sizeof(uint32_t) : 0;
    const int sample_mode = bracketed ? (clusters ? 2 : 0) : 1;
    if (many) k_bracket_sample<kBigMany><<<n_inst, kBigMany, sample_smem, st>>>(p, sample_mode);
    else k_bracket_sample<kBigFew><<<n_inst, kBigFew, sample_smem, st>>>(p, sample_mode);
    ADACOMP_LAUNCH_CHECK();
    ADACOMP_CUDA(end());
    if (bracketed && h->n_items > 0) {
        const dim3 grid(h->n_items, n_workers);
        ADACOMP_CUDA(begin(1));
        k_bracket_scan<<<grid, kThreads, kDenseSmemPerWarp * (kThreads / 32), st>>>(p);
        ADACOMP_LAUNCH_CHECK();
        ADACOMP_CUDA(end());
        ADACOMP_CUDA(begin(2));
        if (many) k_bracket_resolve<kBigMany><<<n_inst, kBigMany, 0, st>>>(p);
        else k_bracket_resolve<kBigFew><<<n_inst, kBigFew, 0, st>>>(p);
        ADACOMP_LAUNCH_CHECK();
        ADACOMP_CUDA(end());
        ADACOMP_CUDA(begin(3));
        if (h->emit_thin) k_bracket_emit_thin<<<grid, kEmitThinThreads, 0, st>>>(p);
        else k_bracket_emit<<<grid, kThreads, 0, st>>>(p);
        ADACOMP_LAUNCH_CHECK();
        ADACOMP_CUDA(end());
    }

    if (clusters) {
        // cluster route: persistent clusters, one (worker, tensor) instance at a time
        const uint64_t n_ord = static_cast<uint64_t>(n_workers) * h->n_cl;
        const uint32_t n_clusters = static_cast<uint32_t>(n_ord < static_cast<uint64_t>(h->cl_active) ? n_ord : h->cl_active);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(n_clusters * h->cl_ctas);
        cfg.blockDim = dim3(h->cl_warps * 32);
        cfg.dynamicSmemBytes = h->cl_smem;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = h->cl_ctas;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        ADACOMP_CUDA(begin(1));
        ADACOMP_CUDA(cudaLaunchKernelEx(&cfg, k_select_cluster, p, static_cast<const uint32_t*>(h->d_cl_layers), h->n_cl, h->cl_ring,
                                        h->cl_qmax, h->cl_smem));
        ADACOMP_LAUNCH_CHECK();
        ADACOMP_CUDA(end());
    }

    if (bracketed && h->all_bracketed) {
        // every tensor is on a single-pass route: only instances whose bracket missed are left, which is
        // rare, so one launch in which a block works such an instance off alone replaces the six below
        unsigned solo = static_cast<unsigned>(h->n_sms) * 2;
        if (solo > n_inst) solo = n_inst;
        ADACOMP_CUDA(begin(10));
        k_fallback_solo<<<solo, kSoloThreads, 0, st>>>(p);
        ADACOMP_LAUNCH_CHECK();
        ADACOMP_CUDA(end());
        return ADACOMP_OK;
    }

    // general route for whatever is flagged for it (tensors not on a single-pass route, and
    // instances whose bracket missed)
    const uint64_t total_slots = static_cast<uint64_t>(h->slots_per_worker) * n_workers;
    uint64_t grid64 = static_cast<uint64_t>(h->n_sms) * 8;
    if (grid64 > total_slots) grid64 = total_slots;
    if (grid64 == 0) grid64 = 1;
    const unsigned grid = static_cast<unsigned>(grid64);
    ADACOMP_CUDA(begin(4));
    k_general_plan<<<1, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    ADACOMP_CUDA(end());
    ADACOMP_CUDA(begin(5));
    k_general_hist<0><<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    ADACOMP_CUDA(end());
    ADACOMP_CUDA(begin(6));
    k_general_hist<1><<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    ADACOMP_CUDA(end());
    ADACOMP_CUDA(begin(7));
    k_general_hist<2><<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    ADACOMP_CUDA(end());
    ADACOMP_CUDA(begin(8));
    k_general_count<<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    ADACOMP_CUDA(end());
    ADACOMP_CUDA(begin(9));
    k_general_write<<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    ADACOMP_CUDA(end());
    return ADACOMP_OK;
}

int adacomp_select_set_profiling(adacomp_select_t* h, int on) {
    if (!h) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    for (int r = 0; r < kProfileRing; ++r) ADACOMP_CUDA(fold_profile_slot(h, r));
    for (int i = 0; i < kSelectStages; ++i) h->stage_ms_sum[i] = 0.0;      // a fresh measurement starts here
    h->profiled_calls = 0;
    h->profiling = on == 2 ? 2 : (on != 0 ? 1 : 0);
    return ADACOMP_OK;
}

int adacomp_select_profile(adacomp_select_t* h, float* h_ms_out, uint32_t n_stages, uint64_t* h_calls_out) {
    if (!h || !h_ms_out || n_stages != kSelectStages) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    for (int r = 0; r < kProfileRing; ++r) ADACOMP_CUDA(fold_profile_slot(h, r));
    for (int i = 0; i < kSelectStages; ++i)
        h_ms_out[i] = h->profiled_calls ? static_cast<float>(h->stage_ms_sum[i] / static_cast<double>(h->profiled_calls)) : 0.0f;
    if (h_calls_out) *h_calls_out = h->profiled_calls;
    return ADACOMP_OK;
}

const char* adacomp_select_stage_name(uint32_t stage) {
    return stage < kSelectStages ? kStageNames[stage] : "";
}

int adacomp_select_host(adacomp_select_t* h, const float* h_grads, uint64_t worker_stride_elems,
                        uint32_t n_workers, float* d_grads_staging, uint32_t* d_idx_staging,
                        float* d_val_staging, uint32_t* h_idx_out, float* h_val_out,
                        void* cuda_stream) {
    if (!h || !h_grads || !d_grads_staging || n_workers == 0 || n_workers > h->max_workers)
        return ADACOMP_ERR_INVALID;
    if (h->K > 0 && (!d_idx_staging || !d_val_staging || !h_idx_out || !h_val_out)) return ADACOMP_ERR_INVALID;
    if (n_workers > 1 && worker_stride_elems < h->extent) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const uint64_t elems = (n_workers - 1) * worker_stride_elems + h->extent;
    ADACOMP_CUDA(cudaMemcpyAsync(d_grads_staging, h_grads, elems * sizeof(float), cudaMemcpyHostToDevice, st));
    int rc = adacomp_select(h, d_grads_staging, worker_stride_elems, n_workers, d_idx_staging, d_val_staging, cuda_stream);
    if (rc != ADACOMP_OK) return rc;
    const uint64_t pairs = h->K * n_workers;
    if (pairs) {
        ADACOMP_CUDA(cudaMemcpyAsync(h_idx_out, d_idx_staging, pairs * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
        ADACOMP_CUDA(cudaMemcpyAsync(h_val_out, d_val_staging, pairs * sizeof(float), cudaMemcpyDeviceToHost, st));
    }
    return ADACOMP_OK;
}

int adacomp_select_pairs_per_worker(const adacomp_select_t* h, uint64_t* pairs_out) {
    if (!h || !pairs_out) return ADACOMP_ERR_INVALID;
    *pairs_out = h->K;
    return ADACOMP_OK;
}

int adacomp_select_last_error(adacomp_select_t* h, void* cuda_stream, uint64_t* stats_out) {
    if (!h) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int status = 0;
    uint32_t len[2] = {0, 0};
    ADACOMP_CUDA(cudaMemcpyAsync(&status, h->d_status, sizeof status, cudaMemcpyDeviceToHost, st));
    ADACOMP_CUDA(cudaMemcpyAsync(len, h->d_list_len, sizeof len, cudaMemcpyDeviceToHost, st));
    ADACOMP_CUDA(cudaMemsetAsync(h->d_status, 0, sizeof(int), st));
    ADACOMP_CUDA(cudaStreamSynchronize(st));
    if (stats_out) stats_out[0] = len[0];
    return status;
}

int adacomp_select_gather(adacomp_select_t* h, const float* d_grads, uint64_t worker_stride_elems, uint32_t n_workers,
                          const uint32_t* d_idx, float* d_val_out, void* cuda_stream) {
    if (!h || !d_grads || n_workers == 0 || n_workers > h->max_workers) return ADACOMP_ERR_INVALID;
    if (worker_stride_elems < h->extent) return ADACOMP_ERR_INVALID;
    if (h->K == 0) return ADACOMP_OK;
    if (!d_idx || !d_val_out) return ADACOMP_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    const uint64_t total = static_cast<uint64_t>(h->K) * n_workers;
    uint64_t grid = (total + kThreads - 1) / kThreads;
    const uint64_t cap = static_cast<uint64_t>(h->n_sms) * 32;
    if (grid > cap) grid = cap;
    k_gather<<<static_cast<unsigned>(grid), kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        d_grads, worker_stride_elems, h->extent, d_idx, d_val_out, h->K, total, h->d_status);
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

int adacomp_select_destroy(adacomp_select_t* h) {
    if (h) {
        DeviceGuard guard(h->device);
        for (int r = 0; r < kProfileRing; ++r)
            for (const adacomp_select::Span& sp : h->spans[r]) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    }
    delete h;
    return ADACOMP_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Selection of one tensor with no workspace from the caller and no allocation by the library:
// the scratch of the general route (one layout record, one instance record, the digit
// histogram, the work list and the per-chunk counters) lives in a fixed array that is part of
// the library image on every GPU that loads it.
namespace {

constexpr uint32_t kStaticMaxN = 1u << 24;                                   // entries per call
constexpr uint32_t kStaticMaxSlots = (kStaticMaxN + 3 + kChunkElems - 1) / kChunkElems;   // 129 chunks
// byte offsets inside the array (each 256-byte aligned)
constexpr size_t kStOffLayer = 0;
constexpr size_t kStOffInst = 256;
constexpr size_t kStOffList = 512;
constexpr size_t kStOffSlotStart = 768;
constexpr size_t kStOffListLen = 1024;
constexpr size_t kStOffStatus = 1280;
constexpr size_t kStOffHist = 1536;
constexpr size_t kStOffChunk = kStOffHist + kBins * sizeof(uint32_t);
constexpr size_t kStaticScratchBytes = kStOffChunk + ((kStaticMaxSlots * sizeof(uint2) + 255) / 256) * 256;
static_assert(sizeof(Layer) <= 256 && sizeof(Inst) <= 256, "records fit their 256-byte cells");
static_assert(kStaticScratchBytes <= 16 * 1024, "the built-in scratch stays small");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Writes the layout record and clears what a selection expects to find zeroed.  Names the array
// directly: device code may.
__global__ void k_static_setup(Layer L) {
    *reinterpret_cast<Layer*>(g_static_scratch + kStOffLayer) = L;
    uint32_t* hist = reinterpret_cast<uint32_t*>(g_static_scratch + kStOffHist);
    for (int b = threadIdx.x; b < kBins; b += blockDim.x) hist[b] = 0;
    if (threadIdx.x < 2) reinterpret_cast<uint32_t*>(g_static_scratch + kStOffListLen)[threadIdx.x] = 0;
    if (threadIdx.x == 0) *reinterpret_cast<int*>(g_static_scratch + kStOffStatus) = 0;
}

// Device address of the array on each device, looked up once per device.  In host code the
// array's name is only a handle for this lookup, never an address a kernel could use.
constexpr int kMaxDevices = 64;
unsigned char* g_static_ptr[kMaxDevices] = {};
std::mutex g_static_mutex;

int static_scratch_for(int device, unsigned char** out) {      // `device` must be current
    if (device < 0 || device >= kMaxDevices) return ADACOMP_ERR_INVALID;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* ptr = nullptr;
        ADACOMP_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        g_static_ptr[device] = static_cast<unsigned char*>(ptr);
    }
    *out = g_static_ptr[device];
    return ADACOMP_OK;
}

}  // namespace

extern "C" int adacomp_select_static(const float* d_grad, uint32_t n, uint32_t k, uint32_t* d_idx_out,
                                     float* d_val_out, int device, void* cuda_stream) {
    if (n > kStaticMaxN) return ADACOMP_ERR_CAPACITY;          // beyond the built-in scratch
    if (k > n || !d_grad || (k > 0 && (!d_idx_out || !d_val_out))) return ADACOMP_ERR_INVALID;
    if (reinterpret_cast<uintptr_t>(d_grad) % 4 != 0) return ADACOMP_ERR_INVALID;
    if (k == 0) return ADACOMP_OK;
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    unsigned char* base = nullptr;
    int rc = static_scratch_for(device, &base);
    if (rc != ADACOMP_OK) return rc;
    int n_sms = 0;
    ADACOMP_CUDA(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, device));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    Layer L = {};
    L.offset = 0;
    L.out_offset = 0;
    L.n = n;
    L.k = k;
    L.n_slots = static_cast<uint32_t>((static_cast<uint64_t>(n) + 3 + kChunkElems - 1) / kChunkElems);
    L.slot_base = 0;

    SelectParams p = {};
    p.grads = d_grad;
    p.stride = n;
    p.n_workers = 1;
    p.n_layers = 1;
    p.layers = reinterpret_cast<const Layer*>(base + kStOffLayer);
    p.inst = reinterpret_cast<Inst*>(base + kStOffInst);
    p.hist = reinterpret_cast<uint32_t*>(base + kStOffHist);
    p.list = reinterpret_cast<uint32_t*>(base + kStOffList);
    p.list_slot_start = reinterpret_cast<uint32_t*>(base + kStOffSlotStart);
    p.list_len = reinterpret_cast<uint32_t*>(base + kStOffListLen);
    p.chunk_cnt = reinterpret_cast<uint2*>(base + kStOffChunk);
    p.slots_per_worker = L.n_slots;
    p.idx_out = d_idx_out;
    p.val_out = d_val_out;
    p.K = k;
    p.status = reinterpret_cast<int*>(base + kStOffStatus);

    unsigned grid = static_cast<unsigned>(n_sms) * 8;
    if (grid > L.n_slots) grid = L.n_slots;
    k_static_setup<<<1, kThreads, 0, st>>>(L);
    ADACOMP_LAUNCH_CHECK();
    k_bracket_sample<kBigFew><<<1, kBigFew, 0, st>>>(p, 1);     // general route only: resets the instance record
    ADACOMP_LAUNCH_CHECK();
    k_general_plan<<<1, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    k_general_hist<0><<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    k_general_hist<1><<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    k_general_hist<2><<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    k_general_count<<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    k_general_write<<<grid, kThreads, 0, st>>>(p);
    ADACOMP_LAUNCH_CHECK();
    return ADACOMP_OK;
}

// Companion of adacomp_select_static: the status word lives in the same built-in array, so reading it
// needs no buffer from the caller and no allocation either.
extern "C" int adacomp_select_static_last_error(int device, void* cuda_stream) {
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    unsigned char* base = nullptr;
    const int rc = static_scratch_for(device, &base);
    if (rc != ADACOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int status = 0;
    ADACOMP_CUDA(cudaMemcpyAsync(&status, base + kStOffStatus, sizeof status, cudaMemcpyDeviceToHost, st));
    ADACOMP_CUDA(cudaMemsetAsync(base + kStOffStatus, 0, sizeof(int), st));
    ADACOMP_CUDA(cudaStreamSynchronize(st));
    return status;
}
