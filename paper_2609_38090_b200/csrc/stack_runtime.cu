// Layer-step runtime over a stack of MoE layers with per-layer HOT + STAGE caches (host code; see include/mira.h):
// predictor call, routing, one host synchronisation for the cache manager, prefetch copies for layer + 2 on a side
// stream, wave plan with on-demand copies, the waves themselves, and the bounded HOT rebalancing.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <cstring>
#include <new>
#include <vector>
#include "mira_internal.cuh"

using namespace mira;

struct mira_stack {
    mira_ctx* ctx = nullptr;
    mira_stack_config cfg;
    int n_routed = 0, n_shared = 0, n_total = 0, n_slots = 0, stage_first = 0, max_waves = 0;
    size_t bb = 0;                                   // bytes of one compressed expert
    std::vector<const unsigned char*> host;          // [L] pinned stores
    std::vector<unsigned char*> slot;                // [L] device slot arrays
    std::vector<mira_cache*> cache;                  // [L]
    std::vector<cudaEvent_t> ready, freed;           // [L * n_slots]: slot filled / slot's last reader done
    std::vector<std::vector<int>> pending_hot;       // [L] HOT slots being refilled by a rebalancing swap
    std::vector<int64_t> win_tokens;                 // [L] tokens since the layer's last rebalancing pass
    cudaEvent_t waves_done = nullptr;
    int32_t* h_live = nullptr;                       // host-mapped: counts [n_total] | predicted ids [16] | flags [2], written by the kernels
    volatile uint32_t* h_live_flag = nullptr;
    int32_t* d_live = nullptr;                       // the same memory as the device sees it
    uint32_t* d_live_flag = nullptr;
    uint32_t seq = 0;                                // sequence number of the layer step (what the flag must show)
    std::vector<cudaEvent_t> wave0_done;             // [L] the layer's first wave of its latest step has run
    std::vector<cudaEvent_t> last_reader;            // [L * n_slots] event after the slot's last reader (null: none yet);
                                                     // one of `freed` or the layer's wave0_done
    std::vector<char> inflight;                      // [L * n_slots] a copy into the slot was issued and not yet waited for
    cudaStream_t side = nullptr;
    cudaStream_t pred_stream = nullptr;              // the predictor head runs beside the routing kernels (owned)
    cudaEvent_t fork_ev = nullptr, join_ev = nullptr;
    // device scratch (caller's memory)
    void** d_tables = nullptr;                       // [L][n_slots] slot pointers
    int32_t* d_map0 = nullptr;                       // [L][n_total] slot map of each layer's first wave, kept between steps
    int32_t* d_ring = nullptr;                       // [max_waves][n_total] slot maps of the demand waves of one step
    float* d_pooled = nullptr;                       // [E]
    int32_t* d_ids = nullptr;                        // [k_pred]
    // pinned host staging (owned)
    int32_t* h_map0 = nullptr;                       // mirror of d_map0
    int32_t* h_ring = nullptr;                       // mirror of d_ring
    std::vector<char> map0_valid;                    // [L]
    // plan outputs
    std::vector<int32_t> wave_of, copy_slot, slot_maps, pf_expert, pf_slot, sw_ev, sw_pr, sw_slot;
    // Coverage@k of the heads: ids predicted for layer l wait here until layer l has routed
    std::vector<std::vector<int32_t>> pred_for;      // [L]
    std::vector<double> cov_sum;                     // [L][k_pred]
    std::vector<int32_t> cov_n;                      // [L]
    int64_t bytes_staged = 0, swaps = 0;
};

namespace {

size_t align256(size_t v) { return (v + 255) / 256 * 256; }

struct ScratchLayout { size_t tables, map0, ring, pooled, ids, total; };
ScratchLayout scratch_layout(const mira_config& c, const mira_stack_config& s) {
    const size_t n_total = Et(c), n_slots = c.n_shared + s.n_hot + s.n_stage;
    const size_t max_waves = 1 + (n_total + s.n_stage - 1) / s.n_stage;
    ScratchLayout L;
    size_t o = 0;
    L.tables = o; o = align256(o + (size_t)s.n_layers * n_slots * sizeof(void*));
    L.map0 = o;   o = align256(o + (size_t)s.n_layers * n_total * 4);
    L.ring = o;   o = align256(o + max_waves * n_total * 4);
    L.pooled = o; o = align256(o + (size_t)c.n_experts * 4);
    L.ids = o;    o = align256(o + (size_t)kMaxTopK * 4);
    L.total = o;
    return L;
}

bool config_ok(const mira_ctx* ctx, const mira_stack_config* s) {
    if (!ctx || !s) return false;
    if (s->n_layers < 1 || s->n_hot < 0 || s->n_hot > ctx->cfg.n_experts || s->n_stage < 1) return false;
    if (s->k_pred < 0 || s->k_pred > kMaxTopK || s->k_pred > ctx->cfg.n_experts) return false;
    if (s->rebalance_every < 0 || s->max_swaps < 0) return false;
    return true;
}

cudaEvent_t& ev(std::vector<cudaEvent_t>& v, const mira_stack* s, int layer, int slot) { return v[(size_t)layer * s->n_slots + slot]; }

// Host-to-device copy of one expert into a slot on the side stream, after the slot's last reader.
mira_status stage(mira_stack* s, int layer, int e, int slot) {
    const size_t idx = (size_t)layer * s->n_slots + slot;
    if (s->last_reader[idx]) MIRA_CUDA_OK(cudaStreamWaitEvent(s->side, s->last_reader[idx], 0));
    s->inflight[idx] = 1;
    mira_status r = mira_stage_expert(s->ctx, s->host[layer] + (size_t)e * s->bb, s->slot[layer] + (size_t)slot * s->bb,
                                      s->side, ev(s->ready, s, layer, slot));
    s->bytes_staged += (int64_t)s->bb;
    return r;
}

}  // namespace

extern "C" {

size_t mira_stack_scratch_bytes(const mira_ctx* ctx, const mira_stack_config* cfg) {
    if (!config_ok(ctx, cfg)) return 0;
    return scratch_layout(ctx->cfg, *cfg).total;
}

void mira_stack_destroy(mira_stack* s) {
    if (!s) return;
    for (mira_cache* c : s->cache) mira_cache_destroy(c);
    for (cudaEvent_t e : s->ready) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : s->freed) if (e) cudaEventDestroy(e);
    if (s->waves_done) cudaEventDestroy(s->waves_done);
    if (s->h_live) cudaFreeHost(s->h_live);
    for (cudaEvent_t e : s->wave0_done) if (e) cudaEventDestroy(e);
    if (s->fork_ev) cudaEventDestroy(s->fork_ev);
    if (s->join_ev) cudaEventDestroy(s->join_ev);
    if (s->pred_stream) cudaStreamDestroy(s->pred_stream);
    if (s->h_map0) cudaFreeHost(s->h_map0);
    if (s->h_ring) cudaFreeHost(s->h_ring);
    delete s;
}

mira_status mira_stack_create(mira_ctx* ctx, const mira_stack_config* cfg, const void* const* host_blobs,
                              void* const* slot_mem, const int32_t* hot, void* dev_scratch, size_t scratch_bytes,
                              void* side_stream, void* stream, mira_stack** out) {
    if (!ctx || !cfg || !host_blobs || !slot_mem || !dev_scratch || !out || (cfg->n_hot > 0 && !hot)) return MIRA_ERR_INVALID_ARG;
    if (!config_ok(ctx, cfg)) return MIRA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(dev_scratch) & 255u) return MIRA_ERR_ALIGN;
    const ScratchLayout SL = scratch_layout(ctx->cfg, *cfg);
    if (scratch_bytes < SL.total) return MIRA_ERR_WORKSPACE;
    mira_stack* s = new (std::nothrow) mira_stack();
    if (!s) return MIRA_ERR_WORKSPACE;
    s->ctx = ctx; s->cfg = *cfg;
    const int L = cfg->n_layers;
    s->n_routed = ctx->cfg.n_experts; s->n_shared = ctx->cfg.n_shared; s->n_total = Et(ctx->cfg);
    s->n_slots = s->n_shared + cfg->n_hot + cfg->n_stage; s->stage_first = s->n_shared + cfg->n_hot;
    s->max_waves = 1 + (s->n_total + cfg->n_stage - 1) / cfg->n_stage;
    s->bb = blob_bytes(ctx->cfg);
    s->side = static_cast<cudaStream_t>(side_stream);
    char* base = static_cast<char*>(dev_scratch);
    s->d_tables = reinterpret_cast<void**>(base + SL.tables);
    s->d_map0 = reinterpret_cast<int32_t*>(base + SL.map0);
    s->d_ring = reinterpret_cast<int32_t*>(base + SL.ring);
    s->d_pooled = reinterpret_cast<float*>(base + SL.pooled);
    s->d_ids = reinterpret_cast<int32_t*>(base + SL.ids);
    auto fail = [&](mira_status code) { mira_stack_destroy(s); return code; };
    for (int l = 0; l < L; ++l) {
        if (!host_blobs[l] || !slot_mem[l] || (reinterpret_cast<uintptr_t>(slot_mem[l]) & 15u)) return fail(MIRA_ERR_INVALID_ARG);
        s->host.push_back(static_cast<const unsigned char*>(host_blobs[l]));
        s->slot.push_back(static_cast<unsigned char*>(slot_mem[l]));
        mira_cache* c = nullptr;
        mira_status r = mira_cache_create(s->n_routed, s->n_shared, hot ? hot + (size_t)l * cfg->n_hot : nullptr, cfg->n_hot,
                                          cfg->n_stage, &c);
        if (r != MIRA_OK) return fail(r);
        s->cache.push_back(c);
    }
    s->ready.assign((size_t)L * s->n_slots, nullptr);
    s->freed.assign((size_t)L * s->n_slots, nullptr);
    for (auto* v : {&s->ready, &s->freed})
        for (cudaEvent_t& e : *v)
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    if (cudaEventCreateWithFlags(&s->waves_done, cudaEventDisableTiming) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    if (cudaHostAlloc(reinterpret_cast<void**>(&s->h_live), (size_t)(s->n_total + 32) * 4, cudaHostAllocMapped) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    std::memset(s->h_live, 0, (size_t)(s->n_total + 32) * 4);
    if (cudaHostGetDevicePointer(reinterpret_cast<void**>(&s->d_live), s->h_live, 0) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    s->h_live_flag = reinterpret_cast<volatile uint32_t*>(s->h_live + s->n_total + 16);     // its own cache line
    s->d_live_flag = reinterpret_cast<uint32_t*>(s->d_live + s->n_total + 16);
    s->wave0_done.assign(L, nullptr);
    for (cudaEvent_t& e : s->wave0_done)
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    s->last_reader.assign((size_t)L * s->n_slots, nullptr);
    s->inflight.assign((size_t)L * s->n_slots, 0);
    if (cudaEventCreateWithFlags(&s->fork_ev, cudaEventDisableTiming) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    if (cudaEventCreateWithFlags(&s->join_ev, cudaEventDisableTiming) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    if (cudaStreamCreateWithFlags(&s->pred_stream, cudaStreamNonBlocking) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    if (cudaMallocHost(reinterpret_cast<void**>(&s->h_map0), (size_t)L * s->n_total * 4) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    if (cudaMallocHost(reinterpret_cast<void**>(&s->h_ring), (size_t)s->max_waves * s->n_total * 4) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    s->map0_valid.assign(L, 0);
    s->pending_hot.resize(L);
    s->win_tokens.assign(L, 0);
    s->wave_of.resize(s->n_total); s->copy_slot.resize(s->n_total);
    s->slot_maps.resize((size_t)s->max_waves * s->n_total);
    s->pf_expert.resize(cfg->n_stage); s->pf_slot.resize(cfg->n_stage);
    s->sw_ev.resize(std::max(cfg->max_swaps, 1)); s->sw_pr.resize(std::max(cfg->max_swaps, 1)); s->sw_slot.resize(std::max(cfg->max_swaps, 1));
    s->pred_for.resize(L);
    s->cov_sum.assign((size_t)L * std::max(cfg->k_pred, 1), 0.0);
    s->cov_n.assign(L, 0);
    // slot pointer tables, and the shared and HOT experts into their slots
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::vector<void*> tables((size_t)L * s->n_slots);
    std::vector<int32_t> map(s->n_total);
    for (int l = 0; l < L; ++l) {
        for (int j = 0; j < s->n_slots; ++j) tables[(size_t)l * s->n_slots + j] = s->slot[l] + (size_t)j * s->bb;
        mira_cache_slot_map(s->cache[l], map.data());
        for (int e = 0; e < s->n_total; ++e)
            if (map[e] >= 0 &&
                cudaMemcpyAsync(s->slot[l] + (size_t)map[e] * s->bb, s->host[l] + (size_t)e * s->bb, s->bb, cudaMemcpyHostToDevice, st) != cudaSuccess)
                return fail(MIRA_ERR_CUDA);
    }
    if (cudaMemcpyAsync(s->d_tables, tables.data(), tables.size() * sizeof(void*), cudaMemcpyHostToDevice, st) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    if (cudaStreamSynchronize(st) != cudaSuccess) return fail(MIRA_ERR_CUDA);
    *out = s;
    return MIRA_OK;
}

mira_status mira_stack_layer_step(mira_stack* s, int32_t layer, const void* hidden, int32_t T, const void* router_w,
                                  const float* router_bias, int32_t k, const void* pred_w, const float* pred_b,
                                  void* out, void* stream) {
    if (!s || layer < 0 || layer >= s->cfg.n_layers || !hidden || !router_w || !out || T < 1) return MIRA_ERR_INVALID_ARG;
    mira_ctx* ctx = s->ctx;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_total = s->n_total, k_pred = s->cfg.k_pred, target = layer + 2;
    const bool do_pred = pred_w && target < s->cfg.n_layers && k_pred > 0;
    mira_cache* cache = s->cache[layer];
    mira_status r;

    // The experts that are resident now start before the host knows which ones the router picks: the slot map of
    // the first wave is the cache's map as it stands, and the routing kernel writes the schedule over every routed
    // expert that has a slot. The stream first waits for what may still be landing in this layer's slots.
    for (int slot : s->pending_hot[layer]) MIRA_CUDA_OK(cudaStreamWaitEvent(st, ev(s->ready, s, layer, slot), 0));
    s->pending_hot[layer].clear();
    for (int j = s->stage_first; j < s->n_slots; ++j) {
        char& f = s->inflight[(size_t)layer * s->n_slots + j];
        if (f) { MIRA_CUDA_OK(cudaStreamWaitEvent(st, ev(s->ready, s, layer, j), 0)); f = 0; }
    }
    int32_t* h0 = s->h_map0 + (size_t)layer * n_total;
    int32_t* d0 = s->d_map0 + (size_t)layer * n_total;
    mira_cache_slot_map(cache, s->wave_of.data());                 // wave_of is scratch here
    if (!s->map0_valid[layer] || std::memcmp(h0, s->wave_of.data(), (size_t)n_total * 4) != 0) {
        std::memcpy(h0, s->wave_of.data(), (size_t)n_total * 4);  // the copy before this one was consumed at least one
        MIRA_CUDA_OK(cudaMemcpyAsync(d0, h0, (size_t)n_total * 4, cudaMemcpyHostToDevice, st));   // synchronisation ago
        s->map0_valid[layer] = 1;
    }
    void* const* tables = s->d_tables + (size_t)layer * s->n_slots;
    // The head reads only `hidden` and has its own scratch, so it runs on a stream of its own beside the routing
    // kernels; its calls are issued after the routing launches, when the device is already busy.
    if (do_pred) MIRA_CUDA_OK(cudaEventRecord(s->fork_ev, st));
    // The grouping kernel itself writes the counts to host-mapped memory and then this step's sequence number to a
    // flag there: no copy and no event sits between the routing kernel and the expert kernels, whose programmatic
    // launch edge stays intact, and the host sees the counts as soon as they exist.
    const uint32_t seq = ++s->seq;
    ctx->notify_count = s->d_live; ctx->notify_flag = s->d_live_flag; ctx->notify_seq = seq;
    r = route_and_schedule(ctx, hidden, T, router_w, router_bias, k, tables, d0, st);
    ctx->notify_count = nullptr; ctx->notify_flag = nullptr;
    if (r != MIRA_OK) return r;
    if (do_pred) {                                                  // before the expert kernels, which fill every SM
        MIRA_CUDA_OK(cudaStreamWaitEvent(s->pred_stream, s->fork_ev, 0));
        ctx->notify_ids = s->d_live + n_total; ctx->notify_ids_flag = s->d_live_flag + 1; ctx->notify_seq = seq;
        r = mira_predict(ctx, layer, hidden, T, pred_w, pred_b, s->d_pooled, nullptr, s->d_ids, k_pred, s->pred_stream);
        ctx->notify_ids = nullptr; ctx->notify_ids_flag = nullptr;
        if (r != MIRA_OK) return r;
        MIRA_CUDA_OK(cudaEventRecord(s->join_ev, s->pred_stream));
    }
    if ((r = run_scheduled_experts(ctx, T, tables, d0, st)) != MIRA_OK) return r;       // first wave: no host decision needed
    // The cache manager runs on the host while the first wave computes: it needs the counts and the predicted ids.
    {
        volatile uint32_t* flag = s->h_live_flag;
        const auto t0 = std::chrono::steady_clock::now();
        for (uint64_t spin = 0; flag[0] != seq || (do_pred && flag[1] != seq); ++spin)
            if ((spin & 0xffff) == 0xffff && std::chrono::steady_clock::now() - t0 > std::chrono::seconds(10)) return MIRA_ERR_CUDA;
        std::atomic_thread_fence(std::memory_order_acquire);
    }
    const int32_t* counts = s->h_live;
    const int32_t* pred = s->h_live + n_total;              // k_pred <= 16 ids behind the counts

    if (!s->pred_for[layer].empty()) {                 // predicted two layers back: score it on this routing
        const std::vector<int32_t>& p = s->pred_for[layer];
        int64_t total = 0;
        for (int e = 0; e < s->n_routed; ++e) total += counts[e];
        const int src = layer - 2;
        if (total > 0) {
            int64_t hit = 0;
            for (size_t j = 0; j < p.size(); ++j) {
                bool seen = false;
                for (size_t i = 0; i < j; ++i) seen |= p[i] == p[j];
                if (!seen && p[j] >= 0 && p[j] < s->n_routed) hit += counts[p[j]];
                s->cov_sum[(size_t)src * k_pred + j] += (double)hit / (double)total;
            }
        }
        s->cov_n[src] += 1;
        s->pred_for[layer].clear();
    }
    if (do_pred) {
        s->pred_for[target].assign(pred, pred + k_pred);
        const int n = mira_cache_prefetch(s->cache[target], pred, k_pred, s->pf_expert.data(), s->pf_slot.data());
        if (n < 0) return MIRA_ERR_INVALID_ARG;
        for (int i = 0; i < n; ++i)
            if ((r = stage(s, target, s->pf_expert[i], s->pf_slot[i])) != MIRA_OK) return r;
    }

    const int nw = mira_cache_plan(cache, counts, s->wave_of.data(), s->copy_slot.data(), s->slot_maps.data(), s->max_waves);
    if (nw < 1) return MIRA_ERR_INVALID_ARG;
    // Wave 0 of the plan is what is already running (the routed experts that had a slot). Its STAGE slots' last
    // reader is that wave. A plan without such a wave (nothing resident was routed) starts at its demand waves.
    bool first_recorded = false;
    auto record_first = [&]() -> cudaError_t {        // the event after the first wave, at most once per step
        if (first_recorded) return cudaSuccess;
        first_recorded = true;
        return cudaEventRecord(s->wave0_done[layer], st);
    };
    bool has_first = true;
    for (int e = 0; e < n_total; ++e) has_first = has_first && !(s->wave_of[e] == 0 && s->copy_slot[e] >= 0);
    const int32_t* map0 = s->slot_maps.data();
    if (has_first)
        for (int e = 0; e < n_total; ++e)
            if (s->wave_of[e] == 0 && map0[e] >= s->stage_first) s->last_reader[(size_t)layer * s->n_slots + map0[e]] = s->wave0_done[layer];
    int ring_pos = 0;
    if (nw > (has_first ? 1 : 0)) MIRA_CUDA_OK(record_first());     // demand copies may have to wait for the first wave
    for (int w = has_first ? 1 : 0; w < nw; ++w) {
        const int32_t* map = s->slot_maps.data() + (size_t)w * n_total;
        uint32_t mask[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int e = 0; e < n_total; ++e) {
            if (s->wave_of[e] != w) continue;
            mask[e >> 5] |= 1u << (e & 31);
            if (s->copy_slot[e] >= 0 && (r = stage(s, layer, e, s->copy_slot[e])) != MIRA_OK) return r;
        }
        for (int e = 0; e < n_total; ++e)
            if (s->wave_of[e] == w && map[e] >= s->stage_first) {
                MIRA_CUDA_OK(cudaStreamWaitEvent(st, ev(s->ready, s, layer, map[e]), 0));
                s->inflight[(size_t)layer * s->n_slots + map[e]] = 0;
            }
        int32_t* h = s->h_ring + (size_t)ring_pos * n_total;
        int32_t* d = s->d_ring + (size_t)ring_pos * n_total;
        ++ring_pos;
        std::memcpy(h, map, (size_t)n_total * 4);
        MIRA_CUDA_OK(cudaMemcpyAsync(d, h, (size_t)n_total * 4, cudaMemcpyHostToDevice, st));
        if ((r = mira_moe_experts(ctx, hidden, T, tables, d, mask, 0, nullptr, st)) != MIRA_OK) return r;
        for (int e = 0; e < n_total; ++e)
            if (s->wave_of[e] == w && map[e] >= s->stage_first) {
                cudaEvent_t f = ev(s->freed, s, layer, map[e]);
                MIRA_CUDA_OK(cudaEventRecord(f, st));
                s->last_reader[(size_t)layer * s->n_slots + map[e]] = f;
            }
    }
    if ((r = combine_only(ctx, T, out, st)) != MIRA_OK) return r;
    MIRA_CUDA_OK(record_first());                     // without demand waves it is recorded here, behind the combine,
                                                      // so nothing sits between the down kernel and the combine
    if (do_pred) MIRA_CUDA_OK(cudaStreamWaitEvent(st, s->join_ev, 0));   // later work on `stream` may overwrite `hidden`
    mira_cache_layer_done(cache, T);
    s->win_tokens[layer] += T;
    if (s->cfg.rebalance_every > 0 && s->win_tokens[layer] >= s->cfg.rebalance_every) {
        s->win_tokens[layer] = 0;
        const int n = mira_cache_rebalance(cache, s->cfg.max_swaps, s->cfg.miss_weight, s->cfg.margin, s->sw_ev.data(),
                                           s->sw_pr.data(), s->sw_slot.data());
        if (n < 0) return MIRA_ERR_INVALID_ARG;
        if (n > 0) {
            MIRA_CUDA_OK(cudaEventRecord(s->waves_done, st));           // the waves above still read the evicted experts
            MIRA_CUDA_OK(cudaStreamWaitEvent(s->side, s->waves_done, 0));
            for (int i = 0; i < n; ++i) {
                const int slot = s->sw_slot[i];
                if ((r = mira_stage_expert(ctx, s->host[layer] + (size_t)s->sw_pr[i] * s->bb, s->slot[layer] + (size_t)slot * s->bb,
                                           s->side, ev(s->ready, s, layer, slot))) != MIRA_OK) return r;
                s->bytes_staged += (int64_t)s->bb;
                s->pending_hot[layer].push_back(slot);
            }
            s->swaps += n;
        }
    }
    return MIRA_OK;
}

mira_status mira_stack_stats(const mira_stack* s, int64_t* out11, int64_t* out_bytes_staged, int64_t* out_swaps) {
    if (!s || !out11) return MIRA_ERR_INVALID_ARG;
    for (int i = 0; i < 11; ++i) out11[i] = 0;
    for (const mira_cache* c : s->cache) {
        int64_t v[11];
        mira_cache_stats(c, v);
        for (int i = 0; i < 11; ++i) out11[i] += v[i];
    }
    if (out_bytes_staged) *out_bytes_staged = s->bytes_staged;
    if (out_swaps) *out_swaps = s->swaps;
    return MIRA_OK;
}

void mira_stack_stats_reset(mira_stack* s) {
    if (!s) return;
    for (mira_cache* c : s->cache) mira_cache_stats_reset(c);
    s->bytes_staged = 0; s->swaps = 0;
    std::fill(s->cov_sum.begin(), s->cov_sum.end(), 0.0);
    std::fill(s->cov_n.begin(), s->cov_n.end(), 0);
}

mira_status mira_stack_coverage(const mira_stack* s, double* out_sum, int32_t* out_n) {
    if (!s || !out_sum || !out_n) return MIRA_ERR_INVALID_ARG;
    const int kp = s->cfg.k_pred;
    for (int l = 0; l < s->cfg.n_layers; ++l) {
        for (int j = 0; j < kp; ++j) out_sum[(size_t)l * kp + j] = s->cov_sum[(size_t)l * kp + j];
        out_n[l] = s->cov_n[l];
    }
    return MIRA_OK;
}

mira_cache* mira_stack_cache(mira_stack* s, int32_t layer) {
    return (s && layer >= 0 && layer < s->cfg.n_layers) ? s->cache[layer] : nullptr;
}

}  // extern "C"
