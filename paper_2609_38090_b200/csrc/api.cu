// extern "C" entry points of libmira: argument validation, workspace layout, kernel sequencing.
#include <algorithm>
#include <new>
#include <cstring>
#include <climits>
#include "mira_internal.cuh"

namespace mira {
namespace {

inline size_t align256(size_t v) { return (v + 255) / 256 * 256; }

bool config_ok(const mira_config* c) {
    if (!c) return false;
    if (c->hidden <= 0 || c->ffn <= 0 || c->hidden % 64 || c->ffn % 64) return false;
    if (c->hidden > 16384) return false;
    if (c->n_experts < 1 || c->n_shared < 0 || c->n_shared > 16 || c->n_experts + c->n_shared > kMaxExperts) return false;
    if (c->max_tokens < 1 || c->max_top_k < 1 || c->max_top_k > kMaxTopK || c->max_top_k > c->n_experts) return false;
    if (c->out_dtype != 0 && c->out_dtype != 1) return false;
    if (c->format != MIRA_FORMAT_SHARED && c->format != MIRA_FORMAT_PER_MATRIX) return false;
    return true;
}

int down_splits_of(int R) { return (R + kDownSlice - 1) / kDownSlice; }
int down_slice_of(int R) { int S = down_splits_of(R); return ((R / kChunk + S - 1) / S) * kChunk; }

Layout make_layout(const mira_config& c) {
    Layout L;
    const size_t T = c.max_tokens, E = c.n_experts, Etot = Et(c), kk = c.max_top_k + c.n_shared, P = T * kk;
    const size_t C = c.hidden, R = c.ffn, S = down_splits_of(c.ffn);
    size_t o = 0;
    L.status = o;    o = align256(o + 32 * sizeof(int32_t));
    L.sched = o;     o = align256(o + sizeof(Sched));
    L.logits = o;    o = align256(o + T * E * 4);
    L.idx = o;       o = align256(o + T * c.max_top_k * 4);
    L.w = o;         o = align256(o + T * c.max_top_k * 4);
    L.count = o;     o = align256(o + Etot * 4);
    L.offset = o;    o = align256(o + (Etot + 1) * 4);
    L.perm = o;      o = align256(o + P * 4);
    L.row_token = o; o = align256(o + P * 4);
    L.xscale = o;    o = align256(o + T * 4);
    L.xnorm = o;     o = align256(o + T * 4);
    L.xsum = o;      o = align256(o + T * 4);
    L.hscale = o;    o = align256(o + P * 4);
    L.hexp = o;      o = align256(o + 2 * kMaxExperts * 4);
    L.x16 = o;       o = align256(o + T * C * 2);
    L.x16p = o;      o = align256(o + (T >= (size_t)kTensorPathMinTokens ? P * C * 2 : 0));
    L.xs_pos = o;    o = align256(o + (T >= (size_t)kTensorPathMinTokens ? P * 4 : 0));
    L.hm_pos = o;    o = align256(o + (T >= (size_t)kTensorPathMinTokens ? P * 4 : 0));
    L.sum_pos = o;   o = align256(o + (T >= (size_t)kTensorPathMinTokens ? P * 4 : 0));
    L.h16 = o;       o = align256(o + P * R * 2);
    L.h16lo = o;     o = align256(o + P * R * 2);
    L.ypart = o;     o = align256(o + std::max(S * P * C * 4, R * 4));   // at least one expert's abs-max scratch for the quantizer
    L.pred = o;      o = align256(o + T * E * 4);
    L.mix = o;       o = align256(o + 8 * (C + E) * 4);
    L.tickets = o;   o = align256(o + (T / 8 + 1) * 4);
    L.total = o;
    return L;
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

RouteView ws_route(mira_ctx* ctx) {
    RouteView rv;
    rv.idx = ws_ptr<int32_t>(ctx, ctx->lay.idx); rv.w = ws_ptr<float>(ctx, ctx->lay.w);
    rv.count = ws_ptr<int32_t>(ctx, ctx->lay.count); rv.offset = ws_ptr<int32_t>(ctx, ctx->lay.offset);
    rv.perm = ws_ptr<int32_t>(ctx, ctx->lay.perm); rv.logits = ws_ptr<float>(ctx, ctx->lay.logits);
    rv.row_token = ws_ptr<int32_t>(ctx, ctx->lay.row_token);
    return rv;
}

// One launch copies every requested routing array (all are 4-byte words): blockIdx.y selects the array.
struct CopyList { const uint32_t* src[6]; uint32_t* dst[6]; unsigned n[6]; };
__global__ void k_copy_route(CopyList L) {
    const unsigned a = blockIdx.y;
    uint32_t* dst = L.dst[a];
    if (dst == nullptr) return;
    const uint32_t* src = L.src[a];
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < L.n[a]; i += gridDim.x * blockDim.x) dst[i] = src[i];
}

mira_status copy_route(mira_ctx* ctx, const mira_route_out* dst, int T, int k, cudaStream_t st) {
    if (!dst) return MIRA_OK;
    const RouteView rv = ws_route(ctx);
    const size_t E = ctx->cfg.n_experts, Etot = Et(ctx->cfg), kk = k + ctx->cfg.n_shared;
    CopyList L;
    const void* src[6] = {rv.idx, rv.w, rv.count, rv.offset, rv.perm, rv.logits};
    void* out[6] = {dst->idx, dst->w, dst->count, dst->offset, dst->perm, dst->logits};
    const size_t n[6] = {(size_t)T * k, (size_t)T * k, Etot, Etot + 1, (size_t)T * kk, (size_t)T * E};
    size_t most = 0;
    for (int i = 0; i < 6; ++i) {
        L.src[i] = static_cast<const uint32_t*>(src[i]); L.dst[i] = static_cast<uint32_t*>(out[i]); L.n[i] = (unsigned)n[i];
        if (out[i]) most = std::max(most, n[i]);
    }
    if (most == 0) return MIRA_OK;
    const unsigned blocks = (unsigned)std::min<size_t>((most + 255) / 256, 64);
    k_copy_route<<<dim3(blocks, 6), 256, 0, st>>>(L);
    ctx->launches += 1;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

mira_status check_layer_args(mira_ctx* ctx, const void* hidden, int T, int k) {
    if (!ctx) return MIRA_ERR_INVALID_ARG;
    if (T == 0 && k >= 1 && k <= ctx->cfg.n_experts) return MIRA_OK;   // nothing to read: hidden may be NULL
    if (!hidden) return MIRA_ERR_INVALID_ARG;
    if (T < 0 || k < 1 || k > ctx->cfg.n_experts) return MIRA_ERR_INVALID_ARG;
    if (k > ctx->cfg.max_top_k || T > ctx->cfg.max_tokens) return MIRA_ERR_WORKSPACE;
    if (misaligned(hidden)) return MIRA_ERR_ALIGN;
    return MIRA_OK;
}

mira_status do_route(mira_ctx* ctx, const void* hidden, int T, const void* router_w, const float* bias, int k,
                     void* const* slots, const int32_t* slot_map, int* fused_schedule, cudaStream_t st, bool quiet_schedule = false) {
    mira_status s = launch_route(ctx, hidden, T, router_w, bias, k, ws_route(ctx), ws_ptr<__half>(ctx, ctx->lay.x16),
                                 ws_ptr<float>(ctx, ctx->lay.xscale), ws_ptr<float>(ctx, ctx->lay.xnorm), slots, slot_map,
                                 fused_schedule, st, quiet_schedule);
    if (s == MIRA_OK) { ctx->route_T = T; ctx->route_k = k; }
    return s;
}

mira_status do_experts(mira_ctx* ctx, int T, void* const* slots, const int32_t* slot_map, const uint32_t* mask,
                       int final_wave, void* out, int schedule_done, cudaStream_t st) {
    mira_status s = MIRA_OK;
    if (!schedule_done && (s = launch_schedule(ctx, T, slots, slot_map, mask, mask == nullptr, st)) != MIRA_OK) return s;
    // Every wave of one routed batch takes the same kernels (T and k decide), so the partial-sum layout is consistent.
    // Per projection, the experts below the step's threshold run on the weight-streaming kernel and the others on the
    // tensor-core kernel (the schedule was written for the same thresholds); both share the fp16 intermediate's layout.
    int tc_min[2];
    step_tc_min(ctx, T, ctx->route_k, tc_min);
    if (tc_min[0] > 0 && (s = launch_up_gate(ctx, slots, slot_map, st)) != MIRA_OK) return s;
    if (tc_min[0] < INT_MAX && (s = launch_up_gate_tc(ctx, slots, slot_map, st)) != MIRA_OK) return s;
    if (tc_min[1] > 0 && (s = launch_down(ctx, slots, slot_map, st)) != MIRA_OK) return s;
    if (tc_min[1] < INT_MAX && (s = launch_down_tc(ctx, slots, slot_map, st)) != MIRA_OK) return s;
    if (final_wave) s = launch_combine(ctx, T, ctx->route_k, tc_min[1] > 0 ? ctx->down_splits : 1,
                                       tc_min[1] < INT_MAX ? down_tc_slices(ctx) : 1, tc_min[1], out, st);
    return s;
}

}  // namespace

mira_status route_and_schedule(mira_ctx* ctx, const void* hidden, int T, const void* router_w, const float* bias, int k,
                               void* const* slots, const int32_t* slot_map, cudaStream_t st) {
    mira_status s = check_layer_args(ctx, hidden, T, k);
    if (s != MIRA_OK) return s;
    if (T < 1 || !router_w || !slots || !slot_map) return MIRA_ERR_INVALID_ARG;
    if (misaligned(router_w)) return MIRA_ERR_ALIGN;
    int fused = 0;
    if ((s = do_route(ctx, hidden, T, router_w, bias, k, slots, slot_map, &fused, st, true)) != MIRA_OK) return s;
    return fused ? MIRA_OK : MIRA_ERR_UNSUPPORTED;      // every routing path writes the schedule when it has the slot map
}

mira_status run_scheduled_experts(mira_ctx* ctx, int T, void* const* slots, const int32_t* slot_map, cudaStream_t st) {
    if (!ctx || ctx->route_T != T || T < 1 || !slots || !slot_map) return MIRA_ERR_INVALID_ARG;
    return do_experts(ctx, T, slots, slot_map, nullptr, 0, nullptr, 1, st);
}

mira_status combine_only(mira_ctx* ctx, int T, void* out, cudaStream_t st) {
    if (!ctx || ctx->route_T != T || T < 1 || !out) return MIRA_ERR_INVALID_ARG;
    if (misaligned(out)) return MIRA_ERR_ALIGN;
    int tc_min[2];
    step_tc_min(ctx, T, ctx->route_k, tc_min);
    return launch_combine(ctx, T, ctx->route_k, tc_min[1] > 0 ? ctx->down_splits : 1,
                          tc_min[1] < INT_MAX ? down_tc_slices(ctx) : 1, tc_min[1], out, st);
}

// Which experts of a T-token step go to the tensor-core kernels (see Sched::tc_min). Today's rule reproduces the
// all-or-nothing switch per projection; MIRA_OPT_HYBRID_MIN_UP / _DOWN override it.
void step_tc_min(const mira_ctx* ctx, int T, int k, int out_min[2]) {
    (void)k;
    const bool tc_ok = ctx->tensor_path_ok && !ctx->force_decode_path;
    out_min[0] = (tc_ok && T >= tc_min_tokens_up(ctx->cfg)) ? 0 : INT_MAX;
    out_min[1] = (tc_ok && T >= tc_min_tokens_down(ctx->cfg)) ? 0 : INT_MAX;
    if (tc_ok && T >= kTensorPathMinTokens)
        for (int p = 0; p < 2; ++p)
            if (ctx->hybrid_min[p] >= 0) out_min[p] = ctx->hybrid_min[p];
}

}  // namespace mira

using namespace mira;

extern "C" {

size_t mira_expert_bytes(int32_t ffn, int32_t hidden) {
    if (ffn <= 0 || hidden <= 0) return 0;
    size_t raw = 3 * (size_t)ffn * hidden + 2 * (size_t)ffn;
    return (raw + 255) / 256 * 256;
}

size_t mira_expert_bytes_format(int32_t ffn, int32_t hidden, int32_t format) {
    if (format == MIRA_FORMAT_SHARED) return mira_expert_bytes(ffn, hidden);
    if (ffn <= 0 || hidden <= 0 || format != MIRA_FORMAT_PER_MATRIX) return 0;
    size_t raw = 3 * (size_t)ffn * hidden + 4 * (size_t)ffn + 2 * (size_t)hidden;
    return (raw + 255) / 256 * 256;
}

size_t mira_workspace_bytes(const mira_config* cfg) {
    if (!config_ok(cfg)) return 0;
    return make_layout(*cfg).total;
}

mira_status mira_create(const mira_config* cfg, void* dev_workspace, size_t workspace_bytes, mira_ctx** out_ctx) {
    if (!cfg || !dev_workspace || !out_ctx) return MIRA_ERR_INVALID_ARG;
    if (!config_ok(cfg)) return MIRA_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(dev_workspace) & 255u) return MIRA_ERR_ALIGN;
    Layout L = make_layout(*cfg);
    if (workspace_bytes < L.total) return MIRA_ERR_WORKSPACE;
    int dev = 0, n_sm = 0;
    MIRA_CUDA_OK(cudaGetDevice(&dev));
    MIRA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    mira_status s;
    if ((s = set_route_attributes()) != MIRA_OK) return s;
    if ((s = set_ffn_attributes()) != MIRA_OK) return s;
    if ((s = set_tc_attributes()) != MIRA_OK) return s;
    if ((s = set_mixture_attributes()) != MIRA_OK) return s;
    if ((s = set_quantize_attributes()) != MIRA_OK) return s;
    MIRA_CUDA_OK(cudaMemset(static_cast<char*>(dev_workspace) + L.status, 0, 32 * sizeof(int32_t)));
    MIRA_CUDA_OK(cudaMemset(static_cast<char*>(dev_workspace) + L.tickets, 0, ((size_t)cfg->max_tokens / 8 + 1) * 4));
    MIRA_CUDA_OK(cudaMemset(static_cast<char*>(dev_workspace) + L.sched, 0, sizeof(Sched)));   // the up/gate kernel's rehearsal pass reads it before the first schedule is written
    mira_ctx* ctx = new (std::nothrow) mira_ctx();
    if (!ctx) return MIRA_ERR_INVALID_ARG;
    ctx->cfg = *cfg;
    if (ctx->cfg.eps <= 0.f) ctx->cfg.eps = 1e-8f;
    ctx->lay = L;
    ctx->ws = static_cast<char*>(dev_workspace);
    ctx->ws_bytes = workspace_bytes;
    ctx->device = dev;
    ctx->n_sm = n_sm;
    ctx->down_splits = down_splits_of(cfg->ffn);
    ctx->down_slice = down_slice_of(cfg->ffn);
    ctx->force_decode_path = false;
    ctx->route_T = -1;
    ctx->route_k = 0;
    ctx->launches = 0;
    ctx->tensor_path_ok = tc_shape_ok(*cfg) && cfg->max_tokens >= kTensorPathMinTokens && build_tensor_maps(ctx);
    *out_ctx = ctx;
    return MIRA_OK;
}

void mira_destroy(mira_ctx* ctx) {
    if (!ctx) return;
    for (auto& r : ctx->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    delete ctx;
}

mira_status mira_profile(mira_ctx* ctx, int32_t enable) {
    if (!ctx) return MIRA_ERR_INVALID_ARG;
    ctx->prof_on = enable != 0;
    return MIRA_OK;
}

mira_status mira_profile_read(mira_ctx* ctx, float* total_ms, int64_t* launches) {
    if (!ctx || !total_ms || !launches) return MIRA_ERR_INVALID_ARG;
    MIRA_CUDA_OK(cudaDeviceSynchronize());
    for (int i = 0; i < MIRA_K_COUNT; ++i) { total_ms[i] = 0.f; launches[i] = 0; }
    for (size_t i = 0; i < ctx->prof_used; ++i) {
        const ProfRec& r = ctx->prof[i];
        float ms = 0.f;
        MIRA_CUDA_OK(cudaEventElapsedTime(&ms, r.a, r.b));
        if (r.id >= 0 && r.id < MIRA_K_COUNT) { total_ms[r.id] += ms; launches[r.id] += 1; }
    }
    ctx->prof_used = 0;
    return MIRA_OK;
}

mira_status mira_quantize_experts(mira_ctx* ctx, const void* w1, const void* w2, const void* w3, int32_t src_dtype,
                                  int32_t n, void* out_blobs, void* stream) {
    if (!ctx || !w1 || !w2 || !w3 || !out_blobs || n < 0) return MIRA_ERR_INVALID_ARG;
    if (src_dtype != 0 && src_dtype != 1) return MIRA_ERR_INVALID_ARG;
    if (misaligned(w1) || misaligned(w2) || misaligned(w3) || misaligned(out_blobs)) return MIRA_ERR_ALIGN;
    if (n == 0) return MIRA_OK;
    return launch_quantize(ctx, w1, w2, w3, src_dtype, n, out_blobs, static_cast<cudaStream_t>(stream));
}

mira_status mira_unpack_expert(mira_ctx* ctx, const void* blob, int8_t* q1, int8_t* q2, int8_t* q3, float* w1,
                               float* w2, float* w3, void* stream) {
    if (!ctx || !blob) return MIRA_ERR_INVALID_ARG;
    if (misaligned(blob)) return MIRA_ERR_ALIGN;
    return launch_unpack(ctx, blob, q1, q2, q3, w1, w2, w3, static_cast<cudaStream_t>(stream));
}

mira_status mira_stage_expert(mira_ctx* ctx, const void* pinned_host_blob, void* dev_slot, void* side_stream,
                              void* ready_event) {
    if (!ctx || !pinned_host_blob || !dev_slot) return MIRA_ERR_INVALID_ARG;
    if (misaligned(dev_slot)) return MIRA_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(side_stream);
    MIRA_CUDA_OK(cudaMemcpyAsync(dev_slot, pinned_host_blob, blob_bytes(ctx->cfg),
                                 cudaMemcpyHostToDevice, st));
    if (ready_event) MIRA_CUDA_OK(cudaEventRecord(static_cast<cudaEvent_t>(ready_event), st));
    return MIRA_OK;
}

mira_status mira_predict(mira_ctx* ctx, int32_t layer, const void* hidden, int32_t T, const void* pred_w,
                         const float* pred_b, float* out_expert_scores, float* out_token_scores,
                         int32_t* out_topk_ids, int32_t k_pred, void* stream) {
    if (!ctx || !hidden || !pred_w || !out_expert_scores || T < 1 || layer < 0) return MIRA_ERR_INVALID_ARG;
    if (ctx->cfg.n_layers > 0 && layer >= ctx->cfg.n_layers - 2) return MIRA_ERR_NO_PREDICTOR;
    if (T > ctx->cfg.max_tokens) return MIRA_ERR_WORKSPACE;
    if (out_topk_ids && (k_pred < 1 || k_pred > kMaxTopK || k_pred > ctx->cfg.n_experts)) return MIRA_ERR_INVALID_ARG;
    if (misaligned(hidden) || misaligned(pred_w)) return MIRA_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int E = ctx->cfg.n_experts;
    float* ts = out_token_scores ? out_token_scores : ws_ptr<float>(ctx, ctx->lay.pred);
    mira_status s = launch_scores(ctx, hidden, T, pred_w, pred_b, E, ts, nullptr, nullptr, nullptr, st);
    if (s != MIRA_OK) return s;
    return launch_pool(ctx, ts, T, E, out_expert_scores, out_topk_ids, out_topk_ids ? k_pred : 0, st);
}

mira_status mira_predict_mixture(mira_ctx* ctx, int32_t layer, const void* hidden, int32_t T, const float* router_logits,
                                 const int32_t* count, int32_t k_top, const mira_mixture_head* head, float* out_scores,
                                 float* out_probs, float* out_alpha, int32_t* out_topk_ids, int32_t k_pred, void* stream) {
    if (!ctx || !hidden || !router_logits || !count || !head || !out_scores || T < 1 || layer < 0) return MIRA_ERR_INVALID_ARG;
    if (!head->wa_h || !head->wa_l || !head->wh_c || !head->wh_t || !head->g_h || !head->g_l || !head->g_c) return MIRA_ERR_INVALID_ARG;
    if (ctx->cfg.n_layers > 0 && layer >= ctx->cfg.n_layers - 2) return MIRA_ERR_NO_PREDICTOR;
    if (T > ctx->cfg.max_tokens) return MIRA_ERR_WORKSPACE;
    if (k_top < 1 || k_top > ctx->cfg.n_experts) return MIRA_ERR_INVALID_ARG;
    if (out_topk_ids && (k_pred < 1 || k_pred > kMaxTopK || k_pred > ctx->cfg.n_experts)) return MIRA_ERR_INVALID_ARG;
    if (misaligned(hidden)) return MIRA_ERR_ALIGN;
    return launch_mixture(ctx, hidden, T, router_logits, count, k_top, *head, out_scores, out_probs, out_alpha,
                          out_topk_ids, out_topk_ids ? k_pred : 0, static_cast<cudaStream_t>(stream));
}

mira_status mira_moe_layer(mira_ctx* ctx, const void* hidden, int32_t T, const void* router_w,
                           const float* router_bias, void* const* expert_slots, const int32_t* slot_map, int32_t k,
                           void* out, const mira_route_out* dbg, void* stream) {
    mira_status s = check_layer_args(ctx, hidden, T, k);
    if (s != MIRA_OK) return s;
    if (T == 0) return MIRA_OK;
    if (!router_w || !expert_slots || !slot_map || !out) return MIRA_ERR_INVALID_ARG;
    if (misaligned(router_w) || misaligned(out)) return MIRA_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int fused = 0;
    if ((s = do_route(ctx, hidden, T, router_w, router_bias, k, expert_slots, slot_map, &fused, st)) != MIRA_OK) return s;
    if ((s = do_experts(ctx, T, expert_slots, slot_map, nullptr, 1, out, fused, st)) != MIRA_OK) return s;
    return copy_route(ctx, dbg, T, k, st);
}

mira_status mira_route(mira_ctx* ctx, const void* hidden, int32_t T, const void* router_w, const float* router_bias,
                       int32_t k, const mira_route_out* route, void* stream) {
    mira_status s = check_layer_args(ctx, hidden, T, k);
    if (s != MIRA_OK) return s;
    if (T == 0) { ctx->route_T = 0; ctx->route_k = k; return MIRA_OK; }
    if (!router_w) return MIRA_ERR_INVALID_ARG;
    if (misaligned(router_w)) return MIRA_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((s = do_route(ctx, hidden, T, router_w, router_bias, k, nullptr, nullptr, nullptr, st)) != MIRA_OK) return s;
    return copy_route(ctx, route, T, k, st);
}

mira_status mira_moe_experts(mira_ctx* ctx, const void* hidden, int32_t T, void* const* expert_slots,
                             const int32_t* slot_map, const uint32_t* expert_mask, int32_t final_wave, void* out,
                             void* stream) {
    if (!ctx || ctx->route_T != T || T < 0) return MIRA_ERR_INVALID_ARG;
    if (T == 0) return MIRA_OK;
    if (!hidden || !expert_slots || !slot_map) return MIRA_ERR_INVALID_ARG;
    if (final_wave && !out) return MIRA_ERR_INVALID_ARG;
    if (final_wave && misaligned(out)) return MIRA_ERR_ALIGN;
    if (T == 0) return MIRA_OK;
    uint32_t all[8];
    const uint32_t* mask = expert_mask;
    if (!mask) { for (int i = 0; i < 8; ++i) all[i] = 0xffffffffu; mask = all; }
    return do_experts(ctx, T, expert_slots, slot_map, mask, final_wave, out, 0, static_cast<cudaStream_t>(stream));
}

mira_status mira_poll_status(mira_ctx* ctx, uint32_t* miss_mask_out, void* stream) {
    if (!ctx) return MIRA_ERR_INVALID_ARG;
    MIRA_CUDA_OK(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    int32_t host[32];
    MIRA_CUDA_OK(cudaMemcpy(host, ctx->ws + ctx->lay.status, sizeof(host), cudaMemcpyDeviceToHost));
    if (host[0] == 0) return MIRA_OK;
    // status word: bit 0 = a routed expert had no slot (the miss mask says which), bit 1 = a bounded wait of a
    // tensor-core kernel ran out. The time-out is reported in preference: that step's outputs are undefined.
    const int words = (Et(ctx->cfg) + 31) / 32;
    if (miss_mask_out) {
        if (host[0] & 1) std::memcpy(miss_mask_out, host + 16, (size_t)words * 4);
        else std::memset(miss_mask_out, 0, (size_t)words * 4);
    }
    MIRA_CUDA_OK(cudaMemset(ctx->ws + ctx->lay.status, 0, 24 * sizeof(int32_t)));   // status + miss mask, not the done mask
    return (host[0] & 2) ? MIRA_ERR_TIMEOUT : MIRA_ERR_EXPERT_MISS;
}

mira_status mira_set_option(mira_ctx* ctx, int32_t option, int32_t value) {
    if (!ctx) return MIRA_ERR_INVALID_ARG;
    if (option == MIRA_OPT_FORCE_DECODE_PATH) { ctx->force_decode_path = value != 0; return MIRA_OK; }
    if (option == MIRA_OPT_TENSOR_LAYOUT && value >= 0 && value <= 5) { ctx->tc_layout = value; return MIRA_OK; }
    if (option == MIRA_OPT_UP_CONVERSION && value >= 0 && value <= 2) { ctx->up_conversion = value; return MIRA_OK; }
    if (option == MIRA_OPT_DOWN_SLICES && value >= 0 && value <= 4) { ctx->down_slices_forced = value; return MIRA_OK; }
    if (option == MIRA_OPT_TEST_WAIT_TIMEOUT) { ctx->test_wait_timeout = value != 0; return MIRA_OK; }
    if ((option == MIRA_OPT_HYBRID_MIN_UP || option == MIRA_OPT_HYBRID_MIN_DOWN) && value >= -1) {
        ctx->hybrid_min[option == MIRA_OPT_HYBRID_MIN_UP ? 0 : 1] = value;
        return MIRA_OK;
    }
    return MIRA_ERR_INVALID_ARG;
}

int64_t mira_kernel_launches(const mira_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* mira_status_string(mira_status s) {
    switch (s) {
        case MIRA_OK: return "ok";
        case MIRA_ERR_INVALID_ARG: return "invalid argument";
        case MIRA_ERR_SHAPE: return "unsupported shape";
        case MIRA_ERR_ALIGN: return "pointer not 16-byte aligned";
        case MIRA_ERR_EXPERT_MISS: return "a routed expert was not resident";
        case MIRA_ERR_NO_PREDICTOR: return "no predictor head for this layer";
        case MIRA_ERR_WORKSPACE: return "workspace too small";
        case MIRA_ERR_CUDA: return "CUDA error";
        case MIRA_ERR_UNSUPPORTED: return "unsupported";
        case MIRA_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    }
    return "unknown";
}

}  // extern "C"
