// a3: the slot-pool expert store (Sec. 3.1 "staged" executor path; Fig. 1 streaming pool) and
// the whole layer-step (Sec. 3.2, the double shift).
//
// A pinned-host tier holds every expert record of every layer and stands in for the paper's
// SSD.  Each layer owns a fixed pool of HBM slots.  Staging is host-driven: the allocator below
// is pure integer logic; for each missing expert one cudaMemcpyAsync is enqueued on a side
// stream, ordered after the layer's last compute by an event, so that the copies of the next
// token overlap the compute of the current one.  Slots are sticky: an expert that stays routed
// is never copied again, and a step rewrites only the slots whose expert changed.
#include <chrono>
#include <new>
#include <utility>
#include <vector>

#include "edg_common.cuh"

namespace edg {

// The hot path's on-demand fetch, initiated by the device: block row k looks routed expert k up in the
// layer's slot table; a resident expert only has its slot noted; for one that is not, the SMs copy
// its record from the pinned-host tier (mapped host memory, plain 16-byte loads, four in flight per
// thread) into transient slot S_hot + k.  slots_eff[k] is what the layer kernel then runs over.
constexpr int kFetchBlocks = 32, kFetchThreads = 256;

__device__ __forceinline__ uint4 ld_host16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kFetchThreads) hot_fetch_kernel(const int32_t* inds, const int32_t* table,
                                                                  const uint8_t* host_layer, uint8_t* pool,
                                                                  int32_t* slots_eff, int E, int S_hot, int n_slots,
                                                                  size_t R) {
    const int k = blockIdx.y;
    const int e = inds[k];
    const bool first = blockIdx.x == 0 && threadIdx.x == 0;
    if (e < 0 || e >= E) {                       // the layer kernel skips and flags it
        if (first) slots_eff[k] = -1;
        return;
    }
    const int s = table[e];
    if (s >= 0 && s < n_slots) {                 // a hit: run from the hot set
        if (first) slots_eff[k] = s;
        return;
    }
    const uint4* src = reinterpret_cast<const uint4*>(host_layer + (size_t)e * R);
    uint4* dst = reinterpret_cast<uint4*>(pool + (size_t)(S_hot + k) * R);
    const size_t n16 = R / 16, stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (i + u * stride < n16) v[u] = ld_host16(src + i + u * stride);
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (i + u * stride < n16) dst[i + u * stride] = v[u];
    }
    if (first) slots_eff[k] = S_hot + k;
}

}  // namespace edg

namespace {

// ---- the default copy engine: the CUDA runtime
int32_t cu_rc(cudaError_t e) { if (e != cudaSuccess) { edg::set_cuda_error(e); return EDG_E_CUDA; } return EDG_OK; }
int32_t cu_copy(void*, void* dst, const void* src, size_t n, void* st) {
    return cu_rc(cudaMemcpyAsync(dst, src, n, cudaMemcpyHostToDevice, static_cast<cudaStream_t>(st)));
}
int32_t cu_fill(void*, void* dst, int32_t b, size_t n, void* st) { return cu_rc(cudaMemsetAsync(dst, b, n, static_cast<cudaStream_t>(st))); }
int32_t cu_ev_create(void*, void** ev) {
    cudaEvent_t e = nullptr;
    const int32_t rc = cu_rc(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    *ev = e;
    return rc;
}
int32_t cu_ev_destroy(void*, void* ev) { return cu_rc(cudaEventDestroy(static_cast<cudaEvent_t>(ev))); }
int32_t cu_ev_record(void*, void* ev, void* st) { return cu_rc(cudaEventRecord(static_cast<cudaEvent_t>(ev), static_cast<cudaStream_t>(st))); }
int32_t cu_wait(void*, void* st, void* ev) { return cu_rc(cudaStreamWaitEvent(static_cast<cudaStream_t>(st), static_cast<cudaEvent_t>(ev), 0)); }
int32_t cu_ev_sync(void*, void* ev) { return cu_rc(cudaEventSynchronize(static_cast<cudaEvent_t>(ev))); }
int32_t cu_st_sync(void*, void* st) { return cu_rc(cudaStreamSynchronize(static_cast<cudaStream_t>(st))); }
int32_t cu_halloc(void*, void** p, size_t n) { return cu_rc(cudaHostAlloc(p, n, cudaHostAllocDefault)); }
int32_t cu_hfree(void*, void* p) { return cu_rc(cudaFreeHost(p)); }
const edg_copy_engine kCudaEngine = {nullptr, cu_copy, cu_fill, cu_ev_create, cu_ev_destroy, cu_ev_record, cu_wait,
                                     cu_ev_sync, cu_st_sync, cu_halloc, cu_hfree};

#define EDG_ENG_TRY(expr)                          \
    do {                                           \
        const int32_t _rc = (expr);                \
        if (_rc != EDG_OK) return _rc;             \
    } while (0)

constexpr uint32_t kMagic = 0x45444731u;   // "EDG1"
constexpr int kRing = 64;                  // pinned staging rows for slot-table updates

struct LayerState {
    std::vector<int32_t> expert_of_slot, slot_of_expert;
    std::vector<int64_t> last_use;
    std::vector<uint8_t> taken;
    int64_t n = 0;                         // stage calls so far (the LRU clock)
    std::vector<int64_t> uses;             // hot path: times each expert has been routed
    std::vector<std::pair<int32_t, int32_t>> pending;   // hot path: (expert, slot) admissions waiting for this step's compute
    void* copy_done = nullptr;             // engine events
    void* compute_done = nullptr;
    bool copy_pending = false;             // copy_done recorded and not yet waited on by compute
    bool compute_recorded = false;
};

}  // namespace

struct edg_store {
    uint32_t magic = kMagic;
    edg_layer_desc d{};
    int n_layers = 0;
    size_t R = 0;
    std::vector<const uint8_t*> host_layers;
    uint8_t* dev_slots = nullptr;
    int32_t* dev_tables = nullptr;
    std::vector<edg_lora> loras;
    std::vector<edg_mlp_head> mlp_heads;   // per layer: the full prerouter head (W1 == null: none)
    int32_t* prev_inds = nullptr;          // dev [n_layers][K]: the routing each layer executed at its previous step (-1: none yet)
    std::vector<const void*> shared_rec;   // per layer: device record of the shared expert, or null
    std::vector<edg_lora> shared_lora;     // per layer: its adapter
    std::vector<uint8_t> shared_has_lora;
    void* copy_stream = nullptr;
    edg_copy_engine eng{};                 // what staging runs on: the CUDA runtime, or a caller's engine
    bool cuda_engine = true;
    bool whole_layer_loads = false;        // edg_store_load_whole_layer has been used: a full pool gets overwritten too
    bool hot = false;                      // the hot executor path (edg_store_set_hot)
    int admit_after = 1;
    edg_hot_stats hot_stats{};
    int32_t* slots_eff = nullptr;          // dev [n_layers][K]: slots of a hot-path step after the fetch kernel
    std::vector<LayerState> layers;
    int32_t* ring = nullptr;               // pinned [kRing][E]
    void* ring_ev[kRing] = {};
    bool ring_used[kRing] = {};
    int ring_pos = 0;
    edg_store_stats stats{};
    // chaining of consecutive batch-1 layer-steps: when a call consumes the routing that the
    // previous call on the same stream and workspace produced, its kernel is launched as a
    // programmatic dependent of that one and waits on a device flag instead of the kernel's end
    const void* chain_x_next = nullptr;    // the hidden state the last batch-1 layer-step produces for its successor, or null
    const void* chain_inds = nullptr;
    const void* chain_ws = nullptr;
    void* chain_stream = nullptr;
    int chain_flag = 0;
    const void* ring_ws = nullptr;         // workspace whose hand-off ring this store has initialised
    int ring_next = 0;                     // ring slot of the next batch-1 layer-step
    int pub_slot = -1;                     // ring slot holding logits no step has read yet, or -1
    int chaining = 0;                      // 0 off (default), 1 when the previous step is still in flight (or under capture), 2 always
    cudaEvent_t step_done = nullptr;       // recorded behind every batch-1 layer-step launched outside a capture
    bool step_done_valid = false;
    // optional measurement of the time compute streams spend waiting for staging copies: an event
    // pair around every wait that is actually enqueued
    bool time_waits = false;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> wait_events;
    size_t wait_used = 0;
    double wait_ms = 0.0;
    int64_t wait_count = 0;
};

constexpr size_t kWaitPairs = 2048;

// adds up the pairs recorded so far (synchronising on the last of them) and frees the pool
static int32_t drain_waits(edg_store* s) {
    for (size_t i = 0; i < s->wait_used; ++i) {
        EDG_CUDA_TRY(cudaEventSynchronize(s->wait_events[i].second));
        float ms = 0.f;
        EDG_CUDA_TRY(cudaEventElapsedTime(&ms, s->wait_events[i].first, s->wait_events[i].second));
        s->wait_ms += ms;
    }
    s->wait_count += (int64_t)s->wait_used;
    s->wait_used = 0;
    return EDG_OK;
}

static bool store_ok(const edg_store* s) { return s != nullptr && s->magic == kMagic; }

extern "C" int32_t edg_store_create_ex(const edg_layer_desc* desc, int32_t n_layers, const void* const* host_layers,
                                       void* dev_slots, int32_t* dev_tables, const edg_lora* loras,
                                       void* copy_stream, const edg_copy_engine* engine_opt, edg_store** out) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!host_layers || !dev_slots || !dev_tables || !out || n_layers < 1) return EDG_E_INVAL;
    if (!edg::aligned(dev_slots, 256) || !edg::aligned(dev_tables, 16)) return EDG_E_INVAL;
    for (int l = 0; l < n_layers; ++l)
        if (!host_layers[l] || !edg::aligned(host_layers[l], 16)) return EDG_E_INVAL;
    if (engine_opt != nullptr &&
        (!engine_opt->copy_h2d || !engine_opt->fill || !engine_opt->event_create || !engine_opt->event_destroy ||
         !engine_opt->event_record || !engine_opt->stream_wait_event || !engine_opt->event_synchronize ||
         !engine_opt->stream_synchronize || !engine_opt->host_alloc || !engine_opt->host_free))
        return EDG_E_INVAL;
    edg_store* s = new (std::nothrow) edg_store();
    if (!s) return EDG_E_INVAL;
    s->d = *desc;
    s->n_layers = n_layers;
    s->R = edg::record_layout(desc->H, desc->I, desc->group).bytes;
    s->host_layers.assign(reinterpret_cast<const uint8_t* const*>(host_layers),
                          reinterpret_cast<const uint8_t* const*>(host_layers) + n_layers);
    s->dev_slots = static_cast<uint8_t*>(dev_slots);
    s->dev_tables = dev_tables;
    if (loras) s->loras.assign(loras, loras + n_layers);
    s->copy_stream = copy_stream;
    s->eng = engine_opt ? *engine_opt : kCudaEngine;
    s->cuda_engine = engine_opt == nullptr;
    s->layers.resize(n_layers);
    const edg_copy_engine& g = s->eng;
    auto fail = [&](int32_t code) { edg_store_destroy(s); return code; };
    for (auto& L : s->layers) {
        L.expert_of_slot.assign(desc->n_slots, -1);
        L.slot_of_expert.assign(desc->E, -1);
        L.last_use.assign(desc->n_slots, -1);
        L.taken.assign(desc->n_slots, 0);
        L.uses.assign(desc->E, 0);
        if ((rc = g.event_create(g.ctx, &L.copy_done)) != EDG_OK) return fail(rc);
        if ((rc = g.event_create(g.ctx, &L.compute_done)) != EDG_OK) return fail(rc);
    }
    void* ring = nullptr;
    if ((rc = g.host_alloc(g.ctx, &ring, (size_t)kRing * desc->E * sizeof(int32_t))) != EDG_OK) return fail(rc);
    s->ring = static_cast<int32_t*>(ring);
    for (int i = 0; i < kRing; ++i)
        if ((rc = g.event_create(g.ctx, &s->ring_ev[i])) != EDG_OK) return fail(rc);
    // every expert starts non-resident
    if ((rc = g.fill(g.ctx, dev_tables, 0xFF, (size_t)n_layers * desc->E * sizeof(int32_t), s->copy_stream)) != EDG_OK) return fail(rc);
    if ((rc = g.stream_synchronize(g.ctx, s->copy_stream)) != EDG_OK) return fail(rc);
    *out = s;
    return EDG_OK;
}

extern "C" int32_t edg_store_create(const edg_layer_desc* desc, int32_t n_layers, const void* const* host_layers,
                                    void* dev_slots, int32_t* dev_tables, const edg_lora* loras,
                                    void* copy_stream, edg_store** out) {
    return edg_store_create_ex(desc, n_layers, host_layers, dev_slots, dev_tables, loras, copy_stream, nullptr, out);
}

extern "C" int32_t edg_store_destroy(edg_store* s) {
    if (!store_ok(s)) return EDG_E_INVAL;
    const edg_copy_engine& g = s->eng;
    g.stream_synchronize(g.ctx, s->copy_stream);
    for (auto& L : s->layers) {
        if (L.copy_done) g.event_destroy(g.ctx, L.copy_done);
        if (L.compute_done) g.event_destroy(g.ctx, L.compute_done);
    }
    for (int i = 0; i < kRing; ++i)
        if (s->ring_ev[i]) g.event_destroy(g.ctx, s->ring_ev[i]);
    if (s->ring) g.host_free(g.ctx, s->ring);
    if (s->step_done) cudaEventDestroy(s->step_done);
    if (s->slots_eff) cudaFree(s->slots_eff);
    if (s->prev_inds) cudaFree(s->prev_inds);
    for (auto& pr : s->wait_events) {
        if (pr.first) cudaEventDestroy(pr.first);
        if (pr.second) cudaEventDestroy(pr.second);
    }
    s->magic = 0;
    delete s;
    return EDG_OK;
}

extern "C" int32_t edg_store_get_stats(const edg_store* s, edg_store_stats* out) {
    if (!store_ok(s) || !out) return EDG_E_INVAL;
    *out = s->stats;
    return EDG_OK;
}

extern "C" int32_t edg_store_snapshot(const edg_store* s, int32_t layer, int32_t* expert_of_slot, int32_t* slot_of_expert) {
    if (!store_ok(s)) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    const LayerState& L = s->layers[layer];
    if (expert_of_slot) for (int i = 0; i < s->d.n_slots; ++i) expert_of_slot[i] = L.expert_of_slot[i];
    if (slot_of_expert) for (int i = 0; i < s->d.E; ++i) slot_of_expert[i] = L.slot_of_expert[i];
    return EDG_OK;
}

// Queues, on the copy stream, the copies of the given (expert, slot) pairs of a layer -- behind the
// layer's last recorded compute, which may still be reading the slots -- then the layer's new
// expert -> slot row for the device table, then the layer's copy-done event.
static int32_t queue_copies(edg_store* s, int layer, const std::pair<int32_t, int32_t>* pairs, int n_pairs) {
    if (n_pairs <= 0) return EDG_OK;
    const edg_copy_engine& g = s->eng;
    const int S = s->d.n_slots, E = s->d.E;
    LayerState& L = s->layers[layer];
    if (L.compute_recorded) EDG_ENG_TRY(g.stream_wait_event(g.ctx, s->copy_stream, L.compute_done));
    for (int i = 0; i < n_pairs; ++i)
        EDG_ENG_TRY(g.copy_h2d(g.ctx, s->dev_slots + ((size_t)layer * S + pairs[i].second) * s->R,
                               s->host_layers[layer] + (size_t)pairs[i].first * s->R, s->R, s->copy_stream));
    // publish the new expert -> slot row to the device table, after the record copies
    const int r = s->ring_pos;
    s->ring_pos = (r + 1) % kRing;
    if (s->ring_used[r]) EDG_ENG_TRY(g.event_synchronize(g.ctx, s->ring_ev[r]));
    int32_t* row = s->ring + (size_t)r * E;
    for (int e = 0; e < E; ++e) row[e] = L.slot_of_expert[e];
    EDG_ENG_TRY(g.copy_h2d(g.ctx, s->dev_tables + (size_t)layer * E, row, (size_t)E * sizeof(int32_t), s->copy_stream));
    EDG_ENG_TRY(g.event_record(g.ctx, s->ring_ev[r], s->copy_stream));
    s->ring_used[r] = true;
    EDG_ENG_TRY(g.event_record(g.ctx, L.copy_done, s->copy_stream));
    L.copy_pending = true;
    s->stats.table_updates += 1;
    s->stats.bytes_copied += (int64_t)n_pairs * (int64_t)s->R;
    return EDG_OK;
}

// least recently used slot among the first `n_pool` that this call has not spoken for, or -1
static int lru_victim(const LayerState& L, int n_pool) {
    int victim = -1;
    for (int sl = 0; sl < n_pool; ++sl)
        if (!L.taken[sl] && (victim < 0 || L.last_use[sl] < L.last_use[victim])) victim = sl;
    return victim;
}

extern "C" int32_t stage_experts_to_slots(edg_store* s, int32_t layer, const int32_t* inds, int32_t n,
                                          int32_t* slots_out, int32_t* n_miss_out) {
    if (!store_ok(s) || !inds || !slots_out) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    const int S = s->d.n_slots, E = s->d.E;
    if (n < 0) return EDG_E_INVAL;
    if (n > (s->hot ? s->d.K : S)) return EDG_E_SLOTS;
    LayerState& L = s->layers[layer];

    // validate before touching any state: in range and distinct
    for (int i = 0; i < n; ++i) {
        if (inds[i] < 0 || inds[i] >= E) return EDG_E_RANGE;
        for (int j = 0; j < i; ++j) if (inds[j] == inds[i]) return EDG_E_RANGE;
    }
    s->stats.stage_calls += 1;

    if (s->hot) {
        // The hot path: this step runs its hits from the hot set as it stands and serves its misses
        // on demand; what a miss changes in the hot set takes effect after this step's compute.
        const int S_hot = S - s->d.K;
        for (int i = 0; i < n; ++i) L.uses[inds[i]] += 1;
        for (int i = 0; i < S_hot; ++i) L.taken[i] = 0;
        for (int i = 0; i < n; ++i) {
            const int sl = L.slot_of_expert[inds[i]];
            slots_out[i] = sl;
            if (sl >= 0) { L.taken[sl] = 1; L.last_use[sl] = L.n; }
        }
        int n_miss = 0;
        for (int i = 0; i < n; ++i) {
            if (slots_out[i] >= 0) continue;
            ++n_miss;
            const int e = inds[i];
            if (L.uses[e] < s->admit_after) continue;
            const int victim = lru_victim(L, S_hot);
            if (victim < 0) continue;                      // every slot is spoken for: served only
            const int old = L.expert_of_slot[victim];
            if (old >= 0) L.slot_of_expert[old] = -1;
            L.expert_of_slot[victim] = e;
            L.slot_of_expert[e] = victim;
            L.last_use[victim] = L.n;
            L.taken[victim] = 1;
            L.pending.emplace_back(e, victim);
            s->hot_stats.admitted += 1;
        }
        L.n += 1;
        s->hot_stats.hits += n - n_miss;
        s->hot_stats.misses += n_miss;
        s->hot_stats.bytes_direct += (int64_t)n_miss * (int64_t)s->R;
        s->stats.hits += n - n_miss;
        s->stats.misses += n_miss;
        if (n_miss_out) *n_miss_out = n_miss;
        return EDG_OK;
    }

    // (i) residents keep their slot and are touched
    for (int i = 0; i < S; ++i) L.taken[i] = 0;
    for (int i = 0; i < n; ++i) {
        const int sl = L.slot_of_expert[inds[i]];
        if (sl >= 0) { L.taken[sl] = 1; L.last_use[sl] = L.n; }
    }
    // (ii) each missing expert takes the least recently used slot this call does not need
    std::pair<int32_t, int32_t> copies[1024];
    int n_miss = 0;
    for (int i = 0; i < n; ++i) {
        const int e = inds[i];
        if (L.slot_of_expert[e] >= 0) continue;
        const int victim = lru_victim(L, S);               // n <= S guarantees a free slot
        const int old = L.expert_of_slot[victim];
        if (old >= 0) L.slot_of_expert[old] = -1;
        L.expert_of_slot[victim] = e;
        L.slot_of_expert[e] = victim;
        L.last_use[victim] = L.n;
        L.taken[victim] = 1;
        copies[n_miss++] = std::make_pair(e, victim);
    }
    L.n += 1;
    for (int i = 0; i < n; ++i) slots_out[i] = L.slot_of_expert[inds[i]];
    if (n_miss_out) *n_miss_out = n_miss;
    s->stats.hits += n - n_miss;
    s->stats.misses += n_miss;
    return queue_copies(s, layer, copies, n_miss);
}

extern "C" int32_t edg_store_wait_staged(edg_store* s, int32_t layer, void* stream) {
    if (!store_ok(s)) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    LayerState& L = s->layers[layer];
    if (L.copy_pending) {
        const edg_copy_engine& g = s->eng;
        bool timed = false;
        if (s->time_waits && s->cuda_engine) {
            cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
            EDG_CUDA_TRY(cudaStreamIsCapturing(static_cast<cudaStream_t>(stream), &capturing));
            timed = capturing == cudaStreamCaptureStatusNone;
        }
        if (timed && s->wait_used == s->wait_events.size()) {
            int32_t rc = drain_waits(s);
            if (rc != EDG_OK) return rc;
        }
        if (timed) EDG_CUDA_TRY(cudaEventRecord(s->wait_events[s->wait_used].first, static_cast<cudaStream_t>(stream)));
        EDG_ENG_TRY(g.stream_wait_event(g.ctx, stream, L.copy_done));
        if (timed) {
            EDG_CUDA_TRY(cudaEventRecord(s->wait_events[s->wait_used].second, static_cast<cudaStream_t>(stream)));
            s->wait_used += 1;
        }
        L.copy_pending = false;
    }
    return EDG_OK;
}

extern "C" int32_t edg_store_time_waits(edg_store* s, int32_t enable) {
    if (!store_ok(s)) return EDG_E_INVAL;
    if (enable && s->wait_events.empty()) {
        s->wait_events.assign(kWaitPairs, std::make_pair((cudaEvent_t) nullptr, (cudaEvent_t) nullptr));
        for (auto& pr : s->wait_events) {
            EDG_CUDA_TRY(cudaEventCreate(&pr.first));
            EDG_CUDA_TRY(cudaEventCreate(&pr.second));
        }
    }
    s->time_waits = enable != 0;
    return EDG_OK;
}

extern "C" int32_t edg_store_exposed_wait_ms(edg_store* s, double* ms_out, int64_t* n_waits_out) {
    if (!store_ok(s) || !ms_out) return EDG_E_INVAL;
    int32_t rc = drain_waits(s);
    if (rc != EDG_OK) return rc;
    *ms_out = s->wait_ms;
    if (n_waits_out) *n_waits_out = s->wait_count;
    s->wait_ms = 0.0;
    s->wait_count = 0;
    return EDG_OK;
}

extern "C" int32_t edg_store_mark_computed(edg_store* s, int32_t layer, void* stream) {
    if (!store_ok(s)) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    // Only a pool that can evict needs the ordering: with n_slots == E nothing is ever overwritten.
    LayerState& L = s->layers[layer];
    if (s->d.n_slots < s->d.E || s->hot || s->whole_layer_loads) {
        const edg_copy_engine& g = s->eng;
        EDG_ENG_TRY(g.event_record(g.ctx, L.compute_done, stream));
        L.compute_recorded = true;
    }
    // hot path: the admissions decided while this step was staged go out now, behind its compute
    if (!L.pending.empty()) {
        const int32_t rc = queue_copies(s, layer, L.pending.data(), (int)L.pending.size());
        L.pending.clear();
        if (rc != EDG_OK) return rc;
    }
    return EDG_OK;
}

// The whole-layer path (Sec. 3.1, executor path 4): every expert of a layer in one shot, for prefill,
// where each expert is hit and there is nothing to predict.  The pinned-host layer is laid out as
// the pool is, so the load is ONE copy of E records (the paper's per-layer stacked layout makes it
// nine direct reads instead of 256 x 9 builds), queued on the copy stream behind the pool layer's
// last compute; the table becomes the identity.  The next layer's load runs while this layer computes.
extern "C" int32_t edg_store_load_whole_layer(edg_store* s, int32_t layer, const void* host_layer_opt) {
    if (!store_ok(s)) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    if (s->d.n_slots != s->d.E || s->hot) return EDG_E_SLOTS;
    if (host_layer_opt != nullptr && !edg::aligned(host_layer_opt, 16)) return EDG_E_INVAL;
    const edg_copy_engine& g = s->eng;
    const int E = s->d.E;
    LayerState& L = s->layers[layer];
    const uint8_t* src = host_layer_opt ? static_cast<const uint8_t*>(host_layer_opt) : s->host_layers[layer];
    s->whole_layer_loads = true;
    for (int e = 0; e < E; ++e) { L.expert_of_slot[e] = e; L.slot_of_expert[e] = e; L.last_use[e] = L.n; }
    L.n += 1;
    L.pending.clear();
    if (L.compute_recorded) EDG_ENG_TRY(g.stream_wait_event(g.ctx, s->copy_stream, L.compute_done));
    EDG_ENG_TRY(g.copy_h2d(g.ctx, s->dev_slots + (size_t)layer * E * s->R, src, (size_t)E * s->R, s->copy_stream));
    const int r = s->ring_pos;
    s->ring_pos = (r + 1) % kRing;
    if (s->ring_used[r]) EDG_ENG_TRY(g.event_synchronize(g.ctx, s->ring_ev[r]));
    int32_t* row = s->ring + (size_t)r * E;
    for (int e = 0; e < E; ++e) row[e] = e;
    EDG_ENG_TRY(g.copy_h2d(g.ctx, s->dev_tables + (size_t)layer * E, row, (size_t)E * sizeof(int32_t), s->copy_stream));
    EDG_ENG_TRY(g.event_record(g.ctx, s->ring_ev[r], s->copy_stream));
    s->ring_used[r] = true;
    EDG_ENG_TRY(g.event_record(g.ctx, L.copy_done, s->copy_stream));
    L.copy_pending = true;
    s->stats.stage_calls += 1;
    s->stats.misses += E;
    s->stats.table_updates += 1;
    s->stats.bytes_copied += (int64_t)E * (int64_t)s->R;
    return EDG_OK;
}

extern "C" int32_t edg_store_set_mlp_head(edg_store* s, int32_t layer, const edg_mlp_head* head) {
    if (!store_ok(s) || !s->cuda_engine) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    if (s->mlp_heads.empty()) s->mlp_heads.assign(s->n_layers, edg_mlp_head{});
    if (head == nullptr) { s->mlp_heads[layer] = edg_mlp_head{}; return EDG_OK; }
    if (!head->W1 || !head->W2) return EDG_E_INVAL;
    if (head->width < 8 || head->width > 4096 || head->width % 8 != 0) return EDG_E_SHAPE;
    if ((size_t)(s->d.E + s->d.H + head->width) * sizeof(float) > 48 * 1024) return EDG_E_SHAPE;
    if (s->prev_inds == nullptr) {
        const size_t n = (size_t)s->n_layers * s->d.K * sizeof(int32_t);
        EDG_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&s->prev_inds), n));
        EDG_CUDA_TRY(cudaMemset(s->prev_inds, 0xFF, n));   // no previous step yet: an empty K-hot vector
    }
    s->mlp_heads[layer] = *head;
    return EDG_OK;
}

extern "C" int32_t edg_store_reset_feedback(edg_store* s, int32_t layer) {
    if (!store_ok(s) || !s->cuda_engine) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    if (s->prev_inds != nullptr)
        EDG_CUDA_TRY(cudaMemset(s->prev_inds + (size_t)layer * s->d.K, 0xFF, (size_t)s->d.K * sizeof(int32_t)));
    return EDG_OK;
}

extern "C" int32_t edg_store_set_shared_expert(edg_store* s, int32_t layer, const void* dev_record, const edg_lora* lora_opt) {
    if (!store_ok(s)) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    if (dev_record != nullptr && !edg::aligned(dev_record, 256)) return EDG_E_INVAL;
    if (dev_record != nullptr && !edg::fused_supported(s->d)) return EDG_E_SHAPE;
    if (lora_opt != nullptr && s->d.rank > 0 &&
        (!lora_opt->A_gate || !lora_opt->B_gate || !lora_opt->A_up || !lora_opt->B_up || !lora_opt->A_down || !lora_opt->B_down))
        return EDG_E_INVAL;
    if (s->shared_rec.empty()) {
        s->shared_rec.assign(s->n_layers, nullptr);
        s->shared_lora.assign(s->n_layers, edg_lora{});
        s->shared_has_lora.assign(s->n_layers, 0);
    }
    s->shared_rec[layer] = dev_record;
    s->shared_has_lora[layer] = (dev_record != nullptr && lora_opt != nullptr && s->d.rank > 0) ? 1 : 0;
    if (s->shared_has_lora[layer]) s->shared_lora[layer] = *lora_opt;
    return EDG_OK;
}

extern "C" int32_t edg_store_set_hot(edg_store* s, int32_t enable, int32_t admit_after) {
    if (!store_ok(s)) return EDG_E_INVAL;
    if (!enable) { s->hot = false; return EDG_OK; }
    if (admit_after < 1) return EDG_E_INVAL;
    if (s->d.n_slots <= s->d.K) return EDG_E_SLOTS;
    for (const auto& L : s->layers)
        if (L.n != 0) return EDG_E_INVAL;                  // before the first staging call
    if (s->cuda_engine && s->slots_eff == nullptr)
        EDG_CUDA_TRY(cudaMalloc(reinterpret_cast<void**>(&s->slots_eff), (size_t)s->n_layers * s->d.K * sizeof(int32_t)));
    s->hot = true;
    s->admit_after = admit_after;
    return EDG_OK;
}

extern "C" int32_t edg_store_get_hot_stats(const edg_store* s, edg_hot_stats* out) {
    if (!store_ok(s) || !out) return EDG_E_INVAL;
    *out = s->hot_stats;
    return EDG_OK;
}

static int32_t layer_decode(edg_store* s, int32_t layer, const void* x,
                            const int32_t* inds_cur, const float* gates_cur,
                            const void* W_pre_next, int32_t* inds_next, float* gates_next,
                            float* logits_next_opt, int32_t* inds_next_host_mirror_opt, void* y,
                            void* x_next, float eps,
                            void* workspace, size_t workspace_bytes, void* stream) {
    if (!store_ok(s) || !x || !inds_cur || !gates_cur || !y) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    if (!s->cuda_engine) return EDG_E_INVAL;               // kernels need the real machine
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t rc = edg_store_wait_staged(s, layer, stream);
    if (rc != EDG_OK) return rc;
    const edg_lora* lora = s->loras.empty() ? nullptr : &s->loras[layer];
    // A layer with a full (MLP) head predicts with it: fc1 -> gelu -> fc2 + residual path on the feature
    // [x ; K-hot(routing executed now) ; K-hot(routing executed at this layer's previous step)].
    const bool mlp = !s->mlp_heads.empty() && s->mlp_heads[layer].W1 != nullptr && inds_next != nullptr;
    if (mlp) {
        if (!gates_next) return EDG_E_INVAL;
        int32_t* prev = s->prev_inds + (size_t)layer * s->d.K;
        rc = edg::run_prerouter_mlp(&s->d, &s->mlp_heads[layer], x, inds_cur, prev, 1, inds_next, gates_next,
                                    logits_next_opt, st, inds_next_host_mirror_opt);
        if (rc != EDG_OK) return rc;
        // what this step executes is the next step's "previous routing"
        EDG_CUDA_TRY(cudaMemcpyAsync(prev, inds_cur, (size_t)s->d.K * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
        W_pre_next = nullptr;                              // the layer kernel evaluates no head of its own
    }
    if (W_pre_next != nullptr && (!inds_next || !gates_next)) return EDG_E_INVAL;
    const void* pool = s->dev_slots + (size_t)layer * s->d.n_slots * s->R;
    const int32_t* table = s->dev_tables + (size_t)layer * s->d.E;
    const int32_t* slot_arg = inds_cur;                    // expert ids, mapped through the table by the kernels
    const int32_t* expert_arg = nullptr;
    if (s->hot) {
        // hits from the hot set, misses fetched by the SMs from the host tier into transient slots
        int32_t* eff = s->slots_eff + (size_t)layer * s->d.K;
        edg::hot_fetch_kernel<<<dim3(edg::kFetchBlocks, s->d.K), edg::kFetchThreads, 0, st>>>(
            inds_cur, table, s->host_layers[layer], s->dev_slots + (size_t)layer * s->d.n_slots * s->R, eff,
            s->d.E, s->d.n_slots - s->d.K, s->d.n_slots, s->R);
        EDG_CUDA_TRY(cudaGetLastError());
        slot_arg = eff;
        expert_arg = inds_cur;
        table = nullptr;
    }
    if (edg::fused_supported(s->d)) {
        // one launch: prerouter for the next step, take, FFN and reduce for this one
        rc = edg::check_desc(&s->d);
        if (rc != EDG_OK) return rc;
        if (!workspace || !edg::aligned(workspace, 256) || workspace_bytes < edg::workspace_layout(s->d, 1).bytes)
            return EDG_E_WORKSPACE;
        if (!edg::aligned(x, 16) || !edg::aligned(y, 16) || (W_pre_next && !edg::aligned(W_pre_next, 16))) return EDG_E_INVAL;
        bool chained = s->chaining && !s->hot && s->chain_inds != nullptr && s->chain_inds == inds_cur &&
                       s->chain_ws == workspace && s->chain_stream == stream;
        // Chaining pays when steps queue up on the device: a chained step runs as a few long-lived
        // CTAs that share the GPU with dozens of other steps.  A step that finds the GPU idle -- the
        // step before it has already finished -- is launched on its own, across all SMs, which
        // is several times faster for that one step.  Inside a stream capture nothing can be
        // asked of the device; a captured sequence is replayed back to back, so it is chained.
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        EDG_CUDA_TRY(cudaStreamIsCapturing(st, &capturing));
        if (chained && s->chaining == 1 && capturing == cudaStreamCaptureStatusNone && s->step_done_valid &&
            cudaEventQuery(s->step_done) == cudaSuccess)
            chained = false;
        // A workspace seen for the first time gets its ring cleared: counters to zero, logits to
        // "not yet written".  After that the ring looks after itself: a chained step resets the
        // slot it has read, and a step that starts over clears the slot the last head left unread.
        bool fresh = s->ring_ws != workspace;
        if (fresh) {
            uint8_t* w8 = static_cast<uint8_t*>(workspace);
            const edg::WorkspaceLayout W = edg::workspace_layout(s->d, 1);
            EDG_CUDA_TRY(cudaMemsetAsync(w8 + edg::kCtrlCounters, 0, edg::kCtrlBytes - edg::kCtrlCounters, st));
            EDG_CUDA_TRY(cudaMemsetAsync(w8 + W.logits, 0xFF, (size_t)edg::kHandoffRing * (s->d.E + edg::kPairWords) * sizeof(float), st));
            EDG_CUDA_TRY(cudaMemsetAsync(w8 + W.dep, 0, (size_t)edg::kHandoffRing * edg::kDepWords * sizeof(float), st));
            s->ring_ws = workspace;
            s->ring_next = 0;
            s->pub_slot = -1;
        }
        const bool chain = chained && !fresh;
        const int flag_in = chain ? s->chain_flag : -1;              // ring slot this step's logits arrive in
        // a chained step whose x is the state the previous step is still producing waits for it on the device
        const bool dep_chain = chain && s->chain_x_next != nullptr && s->chain_x_next == x;
        int stale = -1;
        if (!chain && s->pub_slot >= 0) stale = s->pub_slot;         // nobody will read that head's logits
        s->pub_slot = -1;
        const int ring = s->ring_next;                               // ring slot of this step's scratch and of the head it evaluates
        const int flag_out = W_pre_next != nullptr ? ring : -1;
        s->ring_next = (ring + 1) % edg::kHandoffRing;
        edg::FusedExtras extras;
        extras.inds_mirror = W_pre_next != nullptr ? inds_next_host_mirror_opt : nullptr;
        extras.x_next = x_next;
        extras.eps = eps;
        extras.dep_wait = dep_chain ? flag_in : -1;
        if (!s->shared_rec.empty() && s->shared_rec[layer] != nullptr) {
            extras.shared_rec = s->shared_rec[layer];
            extras.shared_lora = s->shared_has_lora[layer] ? &s->shared_lora[layer] : nullptr;
        }
        rc = edg::run_fused_layer(&s->d, pool, slot_arg, table, expert_arg, gates_cur, x,
                                  (lora && s->d.rank > 0) ? lora : nullptr, y, W_pre_next, inds_next, gates_next,
                                  logits_next_opt, workspace, flag_in, flag_out, ring, stale, st, &extras);
        if (W_pre_next != nullptr) s->pub_slot = flag_out;
        if (rc != EDG_OK) return rc;
        s->step_done_valid = false;
        if (capturing == cudaStreamCaptureStatusNone && s->chaining == 1) {
            if (s->step_done == nullptr) EDG_CUDA_TRY(cudaEventCreateWithFlags(&s->step_done, cudaEventDisableTiming));
            EDG_CUDA_TRY(cudaEventRecord(s->step_done, st));
            s->step_done_valid = true;
        }
        s->chain_x_next = x_next;
        s->chain_inds = W_pre_next != nullptr ? inds_next : nullptr;
        s->chain_ws = workspace;
        s->chain_stream = stream;
        s->chain_flag = flag_out;
    } else {
        if (!s->shared_rec.empty() && s->shared_rec[layer] != nullptr) return EDG_E_SHAPE;   // the shared expert rides in the fused kernel only
        rc = edg::run_ffn(&s->d, pool, 1, slot_arg, table, expert_arg, gates_cur, x, lora, y, workspace, workspace_bytes, st);
        if (rc != EDG_OK) return rc;
        if (W_pre_next != nullptr) {
            rc = edg::run_prerouter(&s->d, W_pre_next, x, 1, inds_next, gates_next, logits_next_opt, st, 0,
                                    inds_next_host_mirror_opt);
            if (rc != EDG_OK) return rc;
        }
    }
    if (x_next != nullptr && !edg::fused_supported(s->d)) {
        rc = edg_next_hidden_state(&s->d, x, y, x_next, eps, stream);
        if (rc != EDG_OK) return rc;
    }
    return edg_store_mark_computed(s, layer, stream);
}

extern "C" int32_t moe_layer_decode(edg_store* s, int32_t layer, const void* x,
                                    const int32_t* inds_cur, const float* gates_cur,
                                    const void* W_pre_next, int32_t* inds_next, float* gates_next,
                                    float* logits_next_opt, int32_t* inds_next_host_mirror_opt, void* y,
                                    void* workspace, size_t workspace_bytes, void* stream) {
    return layer_decode(s, layer, x, inds_cur, gates_cur, W_pre_next, inds_next, gates_next, logits_next_opt,
                        inds_next_host_mirror_opt, y, nullptr, 0.f, workspace, workspace_bytes, stream);
}

extern "C" int32_t moe_layer_decode_dependent(edg_store* s, int32_t layer, const void* x,
                                              const int32_t* inds_cur, const float* gates_cur,
                                              const void* W_pre_next, int32_t* inds_next, float* gates_next,
                                              float* logits_next_opt, int32_t* inds_next_host_mirror_opt, void* y,
                                              void* x_next, float eps,
                                              void* workspace, size_t workspace_bytes, void* stream) {
    if (!x_next || !edg::aligned(x_next, 16) || x_next == x) return EDG_E_INVAL;
    return layer_decode(s, layer, x, inds_cur, gates_cur, W_pre_next, inds_next, gates_next, logits_next_opt,
                        inds_next_host_mirror_opt, y, x_next, eps, workspace, workspace_bytes, stream);
}

extern "C" int32_t edg_stack_decode_token(edg_store* s, const void* x, const int32_t* inds_cur, const float* gates_cur,
                                          const void* W_pre, int32_t* inds_next, float* gates_next,
                                          float* logits_next_opt, const int32_t* mirror_cur, int32_t* mirror_next,
                                          void* y, void* workspace, size_t workspace_bytes, void* stream,
                                          int32_t prefetch, int32_t* n_miss_out) {
    if (!store_ok(s) || !x || !inds_cur || !gates_cur || !W_pre || !inds_next || !gates_next || !mirror_cur ||
        !mirror_next || !y)
        return EDG_E_INVAL;
    const int L = s->n_layers, K = s->d.K, E = s->d.E, H = s->d.H;
    // (1) the single hand-off of the token: the routing of every layer, predicted during the previous
    //     token, as the kernels have mirrored it into host memory.  Bounded wait.
    {
        const volatile int32_t* m = mirror_cur;
        const auto t0 = std::chrono::steady_clock::now();
        int done = 0;
        for (uint64_t spin = 0; done < L * K; ++spin) {
            while (done < L * K && m[done] >= 0) ++done;
            if (done < L * K && (spin & 0xFFF) == 0xFFF &&
                std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count() > 5.0)
                return EDG_E_TIMEOUT;
        }
    }
    for (int i = 0; i < L * K; ++i) {
        if (mirror_cur[i] >= E) return EDG_E_RANGE;
        mirror_next[i] = -1;
    }
    int32_t slots_tmp[32];
    int32_t miss = 0, total_miss = 0, rc;
    // (2) prediction-driven staging: every layer's missing experts are queued on the copy stream
    //     before the first layer runs, so later layers' copies overlap earlier layers' compute
    if (prefetch)
        for (int l = 0; l < L; ++l) {
            rc = stage_experts_to_slots(s, l, mirror_cur + (size_t)l * K, K, slots_tmp, &miss);
            if (rc != EDG_OK) return rc;
            total_miss += miss;
        }
    // (3) the layer-steps; the head owned by layer l predicts layer (l + 1) mod L at the next token
    const size_t wb = (size_t)E * H * (s->d.pre_dtype == EDG_F16 ? 2 : 4);
    const size_t yb = (size_t)H * (s->d.out_dtype == EDG_F32 ? 4 : 2);
    for (int l = 0; l < L; ++l) {
        if (!prefetch) {
            rc = stage_experts_to_slots(s, l, mirror_cur + (size_t)l * K, K, slots_tmp, &miss);
            if (rc != EDG_OK) return rc;
            total_miss += miss;
        }
        const int ln = (l + 1) % L;
        rc = moe_layer_decode(s, l, static_cast<const uint16_t*>(x) + (size_t)l * H, inds_cur + (size_t)l * K,
                              gates_cur + (size_t)l * K, static_cast<const uint8_t*>(W_pre) + (size_t)l * wb,
                              inds_next + (size_t)ln * K, gates_next + (size_t)ln * K,
                              logits_next_opt ? logits_next_opt + (size_t)ln * E : nullptr, mirror_next + (size_t)ln * K,
                              static_cast<uint8_t*>(y) + (size_t)l * yb, workspace, workspace_bytes, stream);
        if (rc != EDG_OK) return rc;
    }
    if (n_miss_out) *n_miss_out = total_miss;
    return EDG_OK;
}

extern "C" int32_t edg_store_set_chaining(edg_store* s, int32_t enable) {
    if (!store_ok(s)) return EDG_E_INVAL;
    s->chaining = enable < 0 ? 0 : (enable > 2 ? 2 : enable);
    return EDG_OK;
}
