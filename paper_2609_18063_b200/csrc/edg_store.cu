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

namespace {

constexpr uint32_t kMagic = 0x45444731u;   // "EDG1"
constexpr int kRing = 64;                  // pinned staging rows for slot-table updates

struct LayerState {
    std::vector<int32_t> expert_of_slot, slot_of_expert;
    std::vector<int64_t> last_use;
    std::vector<uint8_t> taken;
    int64_t n = 0;                         // stage calls so far (the LRU clock)
    cudaEvent_t copy_done = nullptr, compute_done = nullptr;
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
    cudaStream_t copy_stream = nullptr;
    std::vector<LayerState> layers;
    int32_t* ring = nullptr;               // pinned [kRing][E]
    cudaEvent_t ring_ev[kRing] = {};
    bool ring_used[kRing] = {};
    int ring_pos = 0;
    edg_store_stats stats{};
    // chaining of consecutive batch-1 layer-steps: when a call consumes the routing that the
    // previous call on the same stream and workspace produced, its kernel is launched as a
    // programmatic dependent of that one and waits on a device flag instead of the kernel's end
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

extern "C" int32_t edg_store_create(const edg_layer_desc* desc, int32_t n_layers, const void* const* host_layers,
                                    void* dev_slots, int32_t* dev_tables, const edg_lora* loras,
                                    void* copy_stream, edg_store** out) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!host_layers || !dev_slots || !dev_tables || !out || n_layers < 1) return EDG_E_INVAL;
    if (!edg::aligned(dev_slots, 256) || !edg::aligned(dev_tables, 16)) return EDG_E_INVAL;
    for (int l = 0; l < n_layers; ++l)
        if (!host_layers[l] || !edg::aligned(host_layers[l], 16)) return EDG_E_INVAL;
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
    s->copy_stream = static_cast<cudaStream_t>(copy_stream);
    s->layers.resize(n_layers);
    auto fail = [&](cudaError_t e) { edg::set_cuda_error(e); edg_store_destroy(s); return EDG_E_CUDA; };
    for (auto& L : s->layers) {
        L.expert_of_slot.assign(desc->n_slots, -1);
        L.slot_of_expert.assign(desc->E, -1);
        L.last_use.assign(desc->n_slots, -1);
        L.taken.assign(desc->n_slots, 0);
        cudaError_t e = cudaEventCreateWithFlags(&L.copy_done, cudaEventDisableTiming);
        if (e != cudaSuccess) return fail(e);
        e = cudaEventCreateWithFlags(&L.compute_done, cudaEventDisableTiming);
        if (e != cudaSuccess) return fail(e);
    }
    cudaError_t e = cudaHostAlloc(reinterpret_cast<void**>(&s->ring), (size_t)kRing * desc->E * sizeof(int32_t), cudaHostAllocDefault);
    if (e != cudaSuccess) return fail(e);
    for (int i = 0; i < kRing; ++i) {
        e = cudaEventCreateWithFlags(&s->ring_ev[i], cudaEventDisableTiming);
        if (e != cudaSuccess) return fail(e);
    }
    // every expert starts non-resident
    e = cudaMemsetAsync(dev_tables, 0xFF, (size_t)n_layers * desc->E * sizeof(int32_t), s->copy_stream);
    if (e != cudaSuccess) return fail(e);
    e = cudaStreamSynchronize(s->copy_stream);
    if (e != cudaSuccess) return fail(e);
    *out = s;
    return EDG_OK;
}

extern "C" int32_t edg_store_destroy(edg_store* s) {
    if (!store_ok(s)) return EDG_E_INVAL;
    cudaStreamSynchronize(s->copy_stream);
    for (auto& L : s->layers) {
        if (L.copy_done) cudaEventDestroy(L.copy_done);
        if (L.compute_done) cudaEventDestroy(L.compute_done);
    }
    for (int i = 0; i < kRing; ++i)
        if (s->ring_ev[i]) cudaEventDestroy(s->ring_ev[i]);
    if (s->ring) cudaFreeHost(s->ring);
    if (s->step_done) cudaEventDestroy(s->step_done);
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

extern "C" int32_t stage_experts_to_slots(edg_store* s, int32_t layer, const int32_t* inds, int32_t n,
                                          int32_t* slots_out, int32_t* n_miss_out) {
    if (!store_ok(s) || !inds || !slots_out) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    const int S = s->d.n_slots, E = s->d.E;
    if (n < 0) return EDG_E_INVAL;
    if (n > S) return EDG_E_SLOTS;
    LayerState& L = s->layers[layer];

    // validate before touching any state: in range and distinct
    for (int i = 0; i < n; ++i) {
        if (inds[i] < 0 || inds[i] >= E) return EDG_E_RANGE;
        for (int j = 0; j < i; ++j) if (inds[j] == inds[i]) return EDG_E_RANGE;
    }

    // (i) residents keep their slot and are touched
    for (int i = 0; i < S; ++i) L.taken[i] = 0;
    for (int i = 0; i < n; ++i) {
        const int sl = L.slot_of_expert[inds[i]];
        if (sl >= 0) { L.taken[sl] = 1; L.last_use[sl] = L.n; }
    }
    // (ii) each missing expert takes the least recently used slot this call does not need
    int n_miss = 0;
    bool waited = false;
    for (int i = 0; i < n; ++i) {
        const int e = inds[i];
        if (L.slot_of_expert[e] >= 0) continue;
        int victim = -1;
        for (int sl = 0; sl < S; ++sl)
            if (!L.taken[sl] && (victim < 0 || L.last_use[sl] < L.last_use[victim])) victim = sl;
        // n <= S guarantees a free slot
        const int old = L.expert_of_slot[victim];
        if (old >= 0) L.slot_of_expert[old] = -1;
        L.expert_of_slot[victim] = e;
        L.slot_of_expert[e] = victim;
        L.last_use[victim] = L.n;
        L.taken[victim] = 1;
        if (!waited && L.compute_recorded) {
            // do not overwrite a slot the layer's last compute may still be reading
            EDG_CUDA_TRY(cudaStreamWaitEvent(s->copy_stream, L.compute_done, 0));
            waited = true;
        }
        EDG_CUDA_TRY(cudaMemcpyAsync(s->dev_slots + ((size_t)layer * S + victim) * s->R,
                                     s->host_layers[layer] + (size_t)e * s->R, s->R,
                                     cudaMemcpyHostToDevice, s->copy_stream));
        ++n_miss;
    }
    L.n += 1;
    for (int i = 0; i < n; ++i) slots_out[i] = L.slot_of_expert[inds[i]];
    if (n_miss_out) *n_miss_out = n_miss;
    s->stats.stage_calls += 1;
    s->stats.hits += n - n_miss;
    s->stats.misses += n_miss;
    s->stats.bytes_copied += (int64_t)n_miss * (int64_t)s->R;

    if (n_miss > 0) {
        // publish the new expert -> slot row to the device table, after the record copies
        const int r = s->ring_pos;
        s->ring_pos = (r + 1) % kRing;
        if (s->ring_used[r]) EDG_CUDA_TRY(cudaEventSynchronize(s->ring_ev[r]));
        int32_t* row = s->ring + (size_t)r * E;
        for (int e = 0; e < E; ++e) row[e] = L.slot_of_expert[e];
        EDG_CUDA_TRY(cudaMemcpyAsync(s->dev_tables + (size_t)layer * E, row, (size_t)E * sizeof(int32_t),
                                     cudaMemcpyHostToDevice, s->copy_stream));
        EDG_CUDA_TRY(cudaEventRecord(s->ring_ev[r], s->copy_stream));
        s->ring_used[r] = true;
        EDG_CUDA_TRY(cudaEventRecord(L.copy_done, s->copy_stream));
        L.copy_pending = true;
        s->stats.table_updates += 1;
    }
    return EDG_OK;
}

extern "C" int32_t edg_store_wait_staged(edg_store* s, int32_t layer, void* stream) {
    if (!store_ok(s)) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    LayerState& L = s->layers[layer];
    if (L.copy_pending) {
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        if (s->time_waits) EDG_CUDA_TRY(cudaStreamIsCapturing(st, &capturing));
        const bool timed = s->time_waits && capturing == cudaStreamCaptureStatusNone;
        if (timed && s->wait_used == s->wait_events.size()) {
            int32_t rc = drain_waits(s);
            if (rc != EDG_OK) return rc;
        }
        if (timed) EDG_CUDA_TRY(cudaEventRecord(s->wait_events[s->wait_used].first, st));
        EDG_CUDA_TRY(cudaStreamWaitEvent(st, L.copy_done, 0));
        if (timed) {
            EDG_CUDA_TRY(cudaEventRecord(s->wait_events[s->wait_used].second, st));
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
    if (s->d.n_slots < s->d.E) {
        LayerState& L = s->layers[layer];
        EDG_CUDA_TRY(cudaEventRecord(L.compute_done, static_cast<cudaStream_t>(stream)));
        L.compute_recorded = true;
    }
    return EDG_OK;
}

extern "C" int32_t moe_layer_decode(edg_store* s, int32_t layer, const void* x,
                                    const int32_t* inds_cur, const float* gates_cur,
                                    const void* W_pre_next, int32_t* inds_next, float* gates_next,
                                    float* logits_next_opt, int32_t* inds_next_host_mirror_opt, void* y,
                                    void* workspace, size_t workspace_bytes, void* stream) {
    if (!store_ok(s) || !x || !inds_cur || !gates_cur || !y) return EDG_E_INVAL;
    if (layer < 0 || layer >= s->n_layers) return EDG_E_RANGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t rc = edg_store_wait_staged(s, layer, stream);
    if (rc != EDG_OK) return rc;
    const edg_lora* lora = s->loras.empty() ? nullptr : &s->loras[layer];
    if (W_pre_next != nullptr && (!inds_next || !gates_next)) return EDG_E_INVAL;
    const void* pool = s->dev_slots + (size_t)layer * s->d.n_slots * s->R;
    const int32_t* table = s->dev_tables + (size_t)layer * s->d.E;
    if (edg::fused_supported(s->d)) {
        // one launch: prerouter for the next step, take, FFN and reduce for this one
        rc = edg::check_desc(&s->d);
        if (rc != EDG_OK) return rc;
        if (!workspace || !edg::aligned(workspace, 256) || workspace_bytes < edg::workspace_layout(s->d, 1).bytes)
            return EDG_E_WORKSPACE;
        if (!edg::aligned(x, 16) || !edg::aligned(y, 16) || (W_pre_next && !edg::aligned(W_pre_next, 16))) return EDG_E_INVAL;
        bool chained = s->chaining && s->chain_inds != nullptr && s->chain_inds == inds_cur && s->chain_ws == workspace &&
                       s->chain_stream == stream;
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
            s->ring_ws = workspace;
            s->ring_next = 0;
            s->pub_slot = -1;
        }
        const bool chain = chained && !fresh;
        const int flag_in = chain ? s->chain_flag : -1;              // ring slot this step's logits arrive in
        int stale = -1;
        if (!chain && s->pub_slot >= 0) stale = s->pub_slot;         // nobody will read that head's logits
        s->pub_slot = -1;
        const int ring = s->ring_next;                               // ring slot of this step's scratch and of the head it evaluates
        const int flag_out = W_pre_next != nullptr ? ring : -1;
        s->ring_next = (ring + 1) % edg::kHandoffRing;
        edg::FusedExtras extras;
        extras.inds_mirror = W_pre_next != nullptr ? inds_next_host_mirror_opt : nullptr;
        rc = edg::run_fused_layer(&s->d, pool, inds_cur, table, nullptr, gates_cur, x,
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
        s->chain_inds = W_pre_next != nullptr ? inds_next : nullptr;
        s->chain_ws = workspace;
        s->chain_stream = stream;
        s->chain_flag = flag_out;
    } else {
        rc = edg::run_ffn(&s->d, pool, 1, inds_cur, table, nullptr, gates_cur, x, lora, y, workspace, workspace_bytes, st);
        if (rc != EDG_OK) return rc;
        if (W_pre_next != nullptr) {
            rc = edg::run_prerouter(&s->d, W_pre_next, x, 1, inds_next, gates_next, logits_next_opt, st, 0,
                                    inds_next_host_mirror_opt);
            if (rc != EDG_OK) return rc;
        }
    }
    return edg_store_mark_computed(s, layer, stream);
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
