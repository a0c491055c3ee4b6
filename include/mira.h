/*
 * mira.h -- C ABI of the B200 (sm_100a) Mira MoE-layer library.
 *
 * The library runs the routed-expert FFN of one Mixture-of-Experts layer directly on expert
 * weights held in Mira's shared-scale INT8 format (Section IV-B of the paper), plus the linear
 * part of the two-layers-ahead expert predictor (Section IV-E). Every step runs in CUDA kernels
 * of this library; there is no CPU fallback.
 *
 * General conventions
 *   - "device" pointers are CUDA device addresses of the current device; "host" pointers are
 *     ordinary process memory. All memory is owned by the caller; the library never takes
 *     ownership and never allocates or frees device memory (all scratch lives in the workspace
 *     handed to mira_create).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Calls enqueue
 *     work on it and return without synchronising the host, except where stated.
 *   - The return value reports what the host can check (NULL pointers, shapes, alignment, a failed
 *     launch). Conditions only the device can see (a routed expert that is not resident) are
 *     recorded in a device status word that mira_poll_status reads back.
 *   - Shapes: C = model hidden size, R = expert hidden size, E = routed experts, k = experts per
 *     token, T = tokens in the call. Required: C % 64 == 0, R % 64 == 0, E + n_shared <= 256, n_shared <= 16,
 *     1 <= k <= min(E, 16). Device pointers must be 16-byte aligned.
 *   - Matrices are row-major. bf16 / fp16 values are passed as raw 16-bit words.
 *
 * Compressed expert ("blob", Section IV-B and the memory-layout figure):
 *     int8  W1^[R][C]  (up)   | int8 W2^[C][R] (down) | int8 W3^[R][C] (gate) | bf16 s[R]
 *   followed by zero padding to a multiple of 256 bytes. One scale s_r per expert-hidden row r is
 *   shared by row r of W1^, row r of W3^ and COLUMN r of W2^. Codes are symmetric in [-127, 127].
 *   The same bytes are used in pinned host memory and in a device cache slot.
 *
 * Format variant MIRA_FORMAT_PER_MATRIX: the per-matrix-scale ("standard") INT8 that Section IV-B contrasts
 *   the shared scale with, one bf16 scale per ROW of each stored matrix:
 *     int8 W1^[R][C] | int8 W2^[C][R] | int8 W3^[R][C] | bf16 s1[R] | bf16 s2[C] | bf16 s3[R]   (+ padding to 256)
 *   s1[r] scales row r of W1^, s3[r] row r of W3^, s2[c] row c of W2^ (output column c of the down projection).
 *   A context handles one format (mira_config.format); every call of that context reads and writes it.
 */
#ifndef MIRA_H_
#define MIRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mira_ctx mira_ctx; /* opaque, host object */

typedef enum {
    MIRA_OK = 0,
    MIRA_ERR_INVALID_ARG = 1,  /* NULL pointer, k out of range, negative size ...            */
    MIRA_ERR_SHAPE = 2,        /* a dimension violates the divisibility / range rules above   */
    MIRA_ERR_ALIGN = 3,        /* a device pointer is not 16-byte aligned                     */
    MIRA_ERR_EXPERT_MISS = 4,  /* (poll) a token was routed to an expert with no resident slot */
    MIRA_ERR_NO_PREDICTOR = 5, /* mira_predict on one of the last two layers                  */
    MIRA_ERR_WORKSPACE = 6,    /* workspace too small or T > max_tokens                       */
    MIRA_ERR_CUDA = 7,         /* a CUDA runtime call or a kernel launch failed               */
    MIRA_ERR_UNSUPPORTED = 8,
    MIRA_ERR_TIMEOUT = 9       /* (poll) a bounded wait inside a tensor-core kernel ran out; that step's output is undefined */
} mira_status;

typedef struct {
    int32_t hidden;     /* C */
    int32_t ffn;        /* R */
    int32_t n_experts;  /* E, routed experts of one layer */
    int32_t n_shared;   /* always-on shared experts (weight 1, every token); 0 for the paper's models */
    int32_t n_layers;   /* L, only used to validate mira_predict's layer argument */
    int32_t max_tokens; /* largest T of any call */
    int32_t max_top_k;  /* largest k of any call (<= 16) */
    int32_t act_on_w1;  /* 0: h = silu(W3 x) * (W1 x)  (gate matrix activated, the paper's naming)
                           1: h = silu(W1 x) * (W3 x) */
    int32_t out_dtype;  /* 0: bf16 output, 1: fp32 output (parity mode) */
    float eps;          /* epsilon of s_r = max(alpha_r, eps) / 127 ; 0 selects 1e-8 */
    int32_t format;     /* MIRA_FORMAT_SHARED (0, the paper's format) or MIRA_FORMAT_PER_MATRIX (1) */
} mira_config;

enum { MIRA_FORMAT_SHARED = 0, MIRA_FORMAT_PER_MATRIX = 1 };

/* Routing results (Section II-A; grouping is a stable counting sort by expert, tokens ascending).
 * All pointers are device pointers. */
typedef struct {
    int32_t* idx;        /* [T][k]   selected experts, best first (ties: lower index; -0 = +0; a NaN
                                     logit ranks below every number, -inf included)            */
    float* w;            /* [T][k]   softmax over the k selected logits                        */
    int32_t* count;      /* [E+n_shared]   pairs per expert (shared experts: T)                */
    int32_t* offset;     /* [E+n_shared+1] exclusive prefix sum of count                       */
    int32_t* perm;       /* [T][k+n_shared] position of pair (t, j); columns >= k are the shared experts */
    float* logits;       /* [T][E]   router logits (fp32), may be NULL                         */
} mira_route_out;

/* Bytes of one compressed expert, 3RC + 2R rounded up to 256 (Section IV-B). 0 if R or C invalid. */
size_t mira_expert_bytes(int32_t ffn, int32_t hidden);
/* The same for either format: MIRA_FORMAT_PER_MATRIX blobs hold 3RC + 4R + 2C bytes rounded up to 256.
 * 0 if R, C or the format is invalid. */
size_t mira_expert_bytes_format(int32_t ffn, int32_t hidden, int32_t format);

/* Device workspace the context needs for this configuration (bytes). 0 if the config is invalid. */
size_t mira_workspace_bytes(const mira_config* cfg);

/* Create a context on the current device. `dev_workspace` (device, 256-byte aligned, at least
 * mira_workspace_bytes(cfg) bytes) stays owned by the caller and must outlive the context. The call
 * clears the status words with a synchronous memset. */
mira_status mira_create(const mira_config* cfg, void* dev_workspace, size_t workspace_bytes,
                        mira_ctx** out_ctx);
void mira_destroy(mira_ctx* ctx);

/* Section IV-B: joint quantization of n experts. w1, w3: [n][R][C], w2: [n][C][R], device, fp32
 * (src_dtype 0) or bf16 (src_dtype 1). For every expert-hidden row r:
 *   alpha_r = max(|W1[r,:]|, |W3[r,:]|, |W2[:,r]|),  s_r = bf16(max(alpha_r, eps) / 127),
 *   code = clamp(round_half_even(w / s_r), -127, 127).
 * out_blobs: device, n * mira_expert_bytes(R, C) bytes, blob i at offset i * mira_expert_bytes.
 * Inputs must be finite (not checked).
 * In a MIRA_FORMAT_PER_MATRIX context the same rule is applied to each row of each matrix on its own
 * (alpha = abs-max of that row) and blobs are mira_expert_bytes_format(R, C, 1) bytes apart. */
mira_status mira_quantize_experts(mira_ctx* ctx, const void* w1, const void* w2, const void* w3,
                                  int32_t src_dtype, int32_t n_experts_in_call, void* out_blobs,
                                  void* stream);

/* Parity hook: unpack one blob into its integer codes (q1, q3: [R][C], q2: [C][R]) and / or its
 * dequantized fp32 weights w^ = code * s_r (Eq. 1 with zero-point 0; per-matrix format: the scale of the
 * element's row in its own matrix). Any output may be NULL. */
mira_status mira_unpack_expert(mira_ctx* ctx, const void* blob, int8_t* q1, int8_t* q2, int8_t* q3,
                               float* w1, float* w2, float* w3, void* stream);

/* Section IV-E (prefetch controller's copy): asynchronous copy of one compressed expert from pinned
 * host memory into a device cache slot on `side_stream`; if `ready_event` (a cudaEvent_t) is not
 * NULL it is recorded on that stream after the copy. The consumer stream must wait on the event
 * before a layer call uses the slot. */
mira_status mira_stage_expert(mira_ctx* ctx, const void* pinned_host_blob, void* dev_slot,
                              void* side_stream, void* ready_event);

/* Section IV-E, linear head on the hidden state: scores the experts of layer `layer + 2`.
 *   token score[t][e] = sum_c hidden[t][c] * pred_w[e][c] + pred_b[e]      (fp32 accumulation)
 *   out_expert_scores[e] = mean over t (fp32; 32 interleaved partial sums over the tokens, added pairwise, divided by T)
 *   out_topk_ids = the k_pred best pooled scores, ties to the lower id.
 * hidden [T][C] bf16, pred_w [E][C] bf16, pred_b [E] fp32 or NULL, out_token_scores [T][E] or NULL,
 * out_topk_ids [k_pred] or NULL (then k_pred is ignored). Heads exist for every layer except the
 * last two: layer >= n_layers - 2 returns MIRA_ERR_NO_PREDICTOR. */
mira_status mira_predict(mira_ctx* ctx, int32_t layer, const void* hidden, int32_t T,
                         const void* pred_w, const float* pred_b, float* out_expert_scores,
                         float* out_token_scores, int32_t* out_topk_ids, int32_t k_pred,
                         void* stream);

/* The predictor head for callers that cannot allocate device memory. (No counterpart in the paper: this
 * entry point exists for the deployment constraint below, not for a step of the method.)
 *
 * Some hosts of this library may not call cudaMalloc at all -- code running inside a CUDA-graph-only
 * serving loop whose memory plan is frozen, a plug-in that is handed tensors but no allocator, a
 * process whose device memory is fully pre-partitioned. They cannot create a mira_ctx, because a
 * context needs a caller-provided device workspace. This variant of mira_predict needs neither: it
 * takes plain input and output pointers and keeps its only scratch (the per-token scores, T * E
 * floats) in a fixed array that is part of the library image, MIRA_NOALLOC_MAX_SCORES floats
 * (256 KB) on every GPU that loads the library, held until the process exits.
 *
 *   out_expert_scores[e] = mean over t of (sum_c hidden[t][c] * pred_w[e][c] + pred_b[e]);
 *   out_topk_ids (optional) = the k_pred best, ties to the lower id -- exactly as mira_predict.
 *
 * hidden [T][hidden_size] bf16 device, pred_w [n_experts][hidden_size] bf16 device, pred_b [n_experts]
 * fp32 device or NULL, outputs device. Limits: T * n_experts <= MIRA_NOALLOC_MAX_SCORES (else
 * MIRA_ERR_WORKSPACE), hidden_size % 8 == 0 and <= 16384, n_experts <= 256, k_pred <= 16.
 * The call allocates and frees nothing, on the host allocator of CUDA or on the device. The first call
 * on each device resolves the device address of the scratch array and raises a kernel attribute; make
 * that first call outside any stream capture. All calls on one GPU share the scratch array, which
 * keeps the previous call's contents (every entry a call reads it has written first, so nothing needs
 * clearing): two calls whose kernels can overlap on the GPU (different streams) race on it -- keep
 * them on one stream or order them with events. */
#define MIRA_NOALLOC_MAX_SCORES 65536
mira_status mira_predict_noalloc(const void* hidden, int32_t T, int32_t hidden_size, const void* pred_w,
                                 const float* pred_b, int32_t n_experts, float* out_expert_scores,
                                 int32_t* out_topk_ids, int32_t k_pred, void* stream);

/* The MoE layer (Section II-A) on compressed experts (Section IV-B, "fused dequantization + FFN"):
 *   logits = hidden Wr^T + bias; per token top-k, w = softmax over the k selected logits;
 *   out[t] = sum_j w[t][j] * FFN_{idx[t][j]}(hidden[t]) + sum_{shared s} FFN_s(hidden[t]),
 *   FFN_e(x) = W2^ (silu(W3^ x) * (W1^ x)) on the dequantized weights of expert e.
 * hidden [T][C] bf16; router_w [E][C] bf16; router_bias [E] fp32 or NULL;
 * expert_slots: device array of device pointers, one per cache slot, each to a blob;
 * slot_map: device int32 [E+n_shared], expert -> slot index, or -1 if not resident. A pair whose
 *   expert is not resident contributes zero and raises MIRA_ERR_EXPERT_MISS at the next poll.
 * out [T][C] bf16 (or fp32 if out_dtype = 1). dbg: NULL, or device buffers that receive a copy of
 * the routing results (any member may be NULL). T = 0 is a no-op. */
mira_status mira_moe_layer(mira_ctx* ctx, const void* hidden, int32_t T, const void* router_w,
                           const float* router_bias, void* const* expert_slots,
                           const int32_t* slot_map, int32_t k, void* out,
                           const mira_route_out* dbg, void* stream);

/* Routing and grouping only (the first half of mira_moe_layer); results stay in the context for
 * mira_moe_experts and are also copied to `route` (may be NULL, members may be NULL). Lets a host
 * cache manager read `count` and fetch the experts a batch needs. */
mira_status mira_route(mira_ctx* ctx, const void* hidden, int32_t T, const void* router_w,
                       const float* router_bias, int32_t k, const mira_route_out* route,
                       void* stream);

/* Expert FFNs for the routing of the last mira_route call, restricted to the experts whose bit is
 * set in expert_mask (host pointer, ceil((E+n_shared)/32) words; NULL = all). May be called several
 * times with disjoint masks as experts become resident ("waves"); with final_wave != 0 the call
 * also runs the weighted combine and writes `out`. Pairs of experts that were never run, or were
 * not resident when their wave ran, contribute zero and raise MIRA_ERR_EXPERT_MISS. `hidden` and T
 * must be those of the mira_route call. */
mira_status mira_moe_experts(mira_ctx* ctx, const void* hidden, int32_t T,
                             void* const* expert_slots, const int32_t* slot_map,
                             const uint32_t* expert_mask, int32_t final_wave, void* out,
                             void* stream);

/* Synchronises `stream`, reads the device status word and clears it. Returns MIRA_OK,
 * MIRA_ERR_EXPERT_MISS (then miss_mask_out, host, ceil((E+n_shared)/32) words or NULL, receives
 * the experts that were needed but not resident), MIRA_ERR_TIMEOUT (a pipeline wait of a tensor-core kernel gave
 * up after its poll limit: every such wait is bounded, the kernel frees its tensor memory and returns, the
 * outputs of that step are undefined and the context stays usable; reported in preference to a miss, and the
 * mask is still filled if both happened) or MIRA_ERR_CUDA. */
mira_status mira_poll_status(mira_ctx* ctx, uint32_t* miss_mask_out, void* stream);

/* Profiling aid. While enabled, every kernel launch made through this context is bracketed by a
 * pair of CUDA events on the launch stream (up to MIRA_PROFILE_MAX_RECORDS launches; later ones are
 * not recorded). mira_profile_read synchronises the device, adds up the elapsed time and the
 * number of recorded launches per kernel class (index = the MIRA_K_* constants; arrays of
 * MIRA_K_COUNT entries, host) and forgets the records. Event recording perturbs timing slightly:
 * use a profiled pass for per-kernel shares, an unprofiled one for throughput. */
#define MIRA_PROFILE_MAX_RECORDS 16384
enum { MIRA_K_ROUTE = 0, MIRA_K_GROUP = 1, MIRA_K_SCHEDULE = 2, MIRA_K_UP_GATE = 3, MIRA_K_DOWN = 4,
       MIRA_K_COMBINE = 5, MIRA_K_SCORES = 6, MIRA_K_POOL = 7, MIRA_K_QUANTIZE = 8, MIRA_K_UNPACK = 9,
       MIRA_K_COUNT = 10 };
mira_status mira_profile(mira_ctx* ctx, int32_t enable);
mira_status mira_profile_read(mira_ctx* ctx, float* total_ms, int64_t* launches);

/* Section IV-E, MixtureHead: the predictor as a mixture of an activation branch and a history branch with a
 * contextual gate. The paper names the parts and the features but no sizes or non-linearities; this is the smallest
 * instance with every named part, all branches linear (E2 = experts of the predicted layer, here E2 = E):
 *   hbar = mean_t hidden[t][:]      lbar = mean_t router_logits[t][:]      (means summed in token order)
 *   hist[e] = count[e] / sum_e count[e] over the routed experts      top[e] = 1 for the k_top largest counts
 *                                                                    (ties to the lower id), else 0
 *   act = wa_h hbar + wa_l lbar + b_a          (ActHead)        his = wh_c hist + wh_t top + b_h      (HistHead)
 *   alpha = sigmoid(g_h . hbar + g_l . lbar + g_c . hist + b_g)          (contextual gate, one scalar per call)
 *   out_scores = alpha * act + (1 - alpha) * his     out_probs = softmax(out_scores)
 *   out_topk_ids = the k_pred largest of out_scores, ties to the lower id.
 * router_logits [T][E] fp32 and count [E + n_shared] int32 are the by-products of mira_route (device memory);
 * hidden [T][C] bf16. The head's matrices are bf16 row-major device arrays, the biases fp32 device arrays, the
 * struct itself is read on the host. Arithmetic is fp32. out_scores [E] required; out_probs [E], out_alpha [1],
 * out_topk_ids [k_pred] may be NULL. Errors as mira_predict, plus MIRA_ERR_INVALID_ARG for k_top outside
 * [1, E] or a NULL matrix. */
typedef struct {
    const void* wa_h;   /* [E][C] bf16 */
    const void* wa_l;   /* [E][E] bf16 */
    const float* b_a;   /* [E] */
    const void* wh_c;   /* [E][E] bf16 */
    const void* wh_t;   /* [E][E] bf16 */
    const float* b_h;   /* [E] */
    const void* g_h;    /* [C] bf16 */
    const void* g_l;    /* [E] bf16 */
    const void* g_c;    /* [E] bf16 */
    float b_g;
} mira_mixture_head;
mira_status mira_predict_mixture(mira_ctx* ctx, int32_t layer, const void* hidden, int32_t T,
                                 const float* router_logits, const int32_t* count, int32_t k_top,
                                 const mira_mixture_head* head, float* out_scores, float* out_probs,
                                 float* out_alpha, int32_t* out_topk_ids, int32_t k_pred, void* stream);

/* Options. MIRA_OPT_FORCE_DECODE_PATH (value 0/1): run S4/S5 of every batch through the weight-streaming
 * mma.sync kernels, also for the batch sizes that would take the tcgen05 kernels (used by the
 * tests to compare the two paths). MIRA_OPT_TENSOR_LAYOUT (value 0..3): 0 lets every step choose the tile layout of
 * the tcgen05 kernels from its token count (the default); 1, 2, 3 force the narrow, wide or big layout, 4 and 5 the
 * two-SM kernel (tcgen05 cta_group::2: tiles of 256 MMA rows over a cluster of two CTAs, 192 tokens x 4 ring stages
 * or 128 tokens x 8; needs ffn % 128 == 0 and hidden % 256 == 0, else the one-CTA layouts run), for tests and
 * tuning. MIRA_OPT_UP_CONVERSION (value 0..2): how the tcgen05 up/gate kernel turns int8 codes into fp16 operands
 * (the weight-streaming kernels always convert exactly). 0 and 1: exactly (the default). 2: as (code + 128) * 2^-24 with
 * the offset 128 * sum(x) taken out afterwards, 1.6 % faster at 2048 tokens; only accurate while the activations of every
 * token are close to zero-mean and every row's codes are well spread (the subtraction costs about
 * hidden size * |sum x| / (32 |x|_2) * 2^-27 relative to a row of typical codes, more for rows of small codes), which
 * the library does not check; tiles of wide-range experts convert exactly regardless.
 * MIRA_OPT_TEST_WAIT_TIMEOUT (value 1; test hook): the next tcgen05
 * up/gate launch of this context leaves out one activation load in its first CTA and gives up its waits after 4096
 * polls instead of 2^24, so that CTA takes the time-out path (status MIRA_ERR_TIMEOUT at the next poll); the option
 * clears itself with that launch. MIRA_OPT_HYBRID_MIN_UP / MIRA_OPT_HYBRID_MIN_DOWN (value >= -1): a step may split its
 * experts between the two kernel families per projection: experts routed fewer than `value` pairs run on the
 * weight-streaming kernel, the others on the tcgen05 kernel (0: all tensor-core, INT32_MAX: all streaming, -1: the
 * library's rule for the step's token count, the default). Applies to steps of at least 16 tokens of a context whose
 * shape the tensor-core kernels take; set it before the routing call of the step.
 * MIRA_OPT_DOWN_SLICES (value 0..4): reduction slices of the tcgen05 down kernel (one-CTA layouts). Each slice of
 * the expert-hidden dimension is a tile of its own and writes its own partial sums, which S6 adds in slice order, so
 * a batch with few token tiles fills the GPU's CTAs more evenly. 0 (the default): chosen per step from the batch size,
 * the top-k and the configuration, 1 when a tile layout is forced; 1..4: that many, at most ceil(ffn / 4096) (the
 * partial-sum slices the workspace holds). Set it before the first wave of a step: every wave must use the same. */
enum { MIRA_OPT_FORCE_DECODE_PATH = 1, MIRA_OPT_TENSOR_LAYOUT = 2, MIRA_OPT_UP_CONVERSION = 3, MIRA_OPT_TEST_WAIT_TIMEOUT = 4,
       MIRA_OPT_HYBRID_MIN_UP = 5, MIRA_OPT_HYBRID_MIN_DOWN = 6, MIRA_OPT_DOWN_SLICES = 7 };
mira_status mira_set_option(mira_ctx* ctx, int32_t option, int32_t value);

/* ---------------------------------------------------------------------------------------------------------------
 * Host-side HOT + STAGE cache bookkeeping of ONE layer (HOT+STAGE expert cache and adaptive rebalancing sections of
 * the paper). No CUDA calls, no copies: the caller issues the copies (mira_stage_expert) and the waves
 * (mira_moe_experts) that a plan names. Slots of a layer's slot array are numbered
 *   [0, n_shared) shared experts (always resident), [n_shared, n_shared + n_hot) HOT, then n_stage STAGE slots.
 * All pointers are host memory owned by the caller. Not thread-safe per object.
 *
 * mira_cache_prefetch: predictor ids for this layer, best first. Resident experts are skipped (a staged one is
 *   kept until the layer has run), others get a STAGE slot if one is free, else the request is declined.
 *   Writes the copies to issue to out_expert / out_slot (room for n_stage each); returns their number.
 * mira_cache_plan: counts[e] = routed pairs per expert of this step (n_routed + n_shared entries). Wave 0 holds
 *   every needed expert that is resident; the missing ones follow in waves of at most n_stage experts, each
 *   copied into a STAGE slot first. Outputs, each with n_routed + n_shared entries: wave_of[e] (-1 if the expert
 *   is not needed), copy_slot[e] (STAGE slot to copy it into before its wave, -1 if none). slot_maps receives one
 *   slot map (expert -> slot or -1, valid while that wave runs) per wave, max_waves rows; returns the number of
 *   waves, or -1 if max_waves is too small.
 * mira_cache_layer_done: the layer has run (its staged experts may be overwritten from now on); adds n_tokens to
 *   the rebalancing window.
 * mira_cache_rebalance: one pass over the window's counters (victim score = pairs routed to a HOT expert,
 *   candidate score = pairs routed + miss_weight * pairs fetched on demand; a swap only while the best candidate
 *   exceeds margin * the worst victim; at most max_swaps), then the window is reset. Returns the number of swaps
 *   written to out_evicted / out_promoted / out_slot (room for max_swaps each); the caller copies each promoted
 *   expert into its slot.
 * mira_cache_stats: 11 counters: pairs served from HOT, STAGE, on demand; experts likewise; prefetches issued,
 *   declined, skipped, useful; copies. mira_cache_stats_reset zeroes them (the rebalancing window is kept). */
typedef struct mira_cache mira_cache;
/* Byte budget -> slots per layer (HOT+STAGE cache section of the paper): what is left of vram_bytes after reserve_bytes
 * is counted in expert slots, the shared experts of every layer are set aside, and the rest is split between HOT and
 * STAGE. The paper names two regimes without numbers; the reading taken: small-VRAM mode (fewer than a quarter of the
 * routed experts fit) keeps STAGE at the prefetch window of k_stage experts (<= 0 selects 3), everything else HOT;
 * large-VRAM mode gives STAGE an eighth of the slots (at least the window), HOT never exceeds n_routed. Writes
 * out_n_hot, out_n_stage and out_small_mode (1 / 0). MIRA_ERR_INVALID_ARG for non-positive sizes, MIRA_ERR_WORKSPACE
 * if not even the shared experts and one HOT + one STAGE slot per layer fit. */
mira_status mira_cache_budget(int64_t vram_bytes, int64_t reserve_bytes, int64_t expert_bytes, int32_t n_layers,
                              int32_t n_routed, int32_t n_shared, int32_t k_stage, int32_t* out_n_hot,
                              int32_t* out_n_stage, int32_t* out_small_mode);
mira_status mira_cache_create(int32_t n_routed, int32_t n_shared, const int32_t* hot, int32_t n_hot, int32_t n_stage,
                              mira_cache** out);
void mira_cache_destroy(mira_cache* c);
mira_status mira_cache_slot_map(const mira_cache* c, int32_t* out_slot_map);
int32_t mira_cache_prefetch(mira_cache* c, const int32_t* predicted, int32_t n, int32_t* out_expert, int32_t* out_slot);
int32_t mira_cache_plan(mira_cache* c, const int32_t* counts, int32_t* wave_of, int32_t* copy_slot,
                        int32_t* slot_maps, int32_t max_waves);
void mira_cache_layer_done(mira_cache* c, int32_t n_tokens);
int32_t mira_cache_rebalance(mira_cache* c, int32_t max_swaps, float miss_weight, float margin, int32_t* out_evicted,
                             int32_t* out_promoted, int32_t* out_slot);
void mira_cache_stats(const mira_cache* c, int64_t* out11);
void mira_cache_stats_reset(mira_cache* c);

/* ---------------------------------------------------------------------------------------------------------------
 * Layer-step runtime over a stack of MoE layers with per-layer HOT + STAGE caches: the prefetch controller, the
 * cache manager and the wave executor of the predictive-staging and cache sections of the paper in one host object,
 * so that a decode loop makes one call per layer. mira_stack_layer_step does, on `stream` unless stated:
 *   1. waits for copies still landing in this layer's slots and uploads the layer's slot map if it changed;
 *   2. routes (as mira_route), the routing kernel also writing the schedule over every routed expert that has a slot,
 *      and starts the up/gate and down kernels of those experts at once: the first wave needs no host decision. The
 *      grouping kernel writes the per-expert pair counts to host-mapped memory followed by a sequence flag, which the
 *      host polls (bounded: MIRA_ERR_CUDA after 10 s), so nothing is synchronised and no copy sits in the stream;
 *   3. if pred_w != NULL and layer + 2 < n_layers and k_pred > 0: mira_predict with that head (it scores the experts
 *      of layer + 2) on a stream of the object's own beside the routing kernels, its ids reported the same way;
 *   4. mira_cache_prefetch on the cache of layer + 2: each admitted expert is copied from the pinned host store into
 *      its STAGE slot on the side stream, after the slot's last reader and followed by the slot's "ready" event;
 *   5. mira_cache_plan on this layer's cache; for every demand wave: on-demand copies on the side stream, the stream
 *      waits for the "ready" events of the STAGE slots the wave uses, mira_moe_experts runs the wave, then the slots'
 *      "last reader" events are recorded; then the weighted combine into `out`;
 *   6. mira_cache_layer_done and, every rebalance_every tokens of this layer, mira_cache_rebalance; promoted
 *      experts are copied into their HOT slots on the side stream after this step's waves, and the layer's next step
 *      waits for them.
 * The call returns when everything is enqueued; `hidden` must stay unchanged until the work enqueued on `stream` by
 * this call has run (work enqueued on `stream` afterwards is ordered behind the head's reads as well).
 * Ownership: the caller owns and keeps alive host_blobs (pinned host, per layer all E + n_shared blobs, blob e at
 * e * blob bytes), slot_mem (device, per layer n_shared + n_hot + n_stage slots one blob apart, 16-byte aligned) and
 * dev_scratch (device, 256-byte aligned, mira_stack_scratch_bytes bytes). The object allocates pinned host staging
 * memory and CUDA events, freed by mira_stack_destroy. mira_stack_create copies the shared and the initial HOT
 * experts (hot: [n_layers][n_hot] expert ids) into their slots and synchronises. One stack per context; calls are
 * not thread-safe. Errors: those of the calls above; MIRA_ERR_INVALID_ARG for a bad layer or NULL pointers.
 * mira_stack_stats: the 11 counters of mira_cache_stats summed over the layers, bytes copied host to device since
 * the last reset, HOT swaps. mira_stack_coverage: per source layer l (heads exist for l < n_layers - 2) the sum
 * over its scored steps of Coverage@k, k = 1..k_pred (share of the routed pairs of layer l + 2 that fell on the
 * first k predicted experts), and the number of scored steps; out_sum [n_layers][k_pred], out_n [n_layers].
 * mira_stack_stats_reset zeroes the counters, the byte and swap counts and the coverage sums (not the rebalancing
 * windows, nor the cache contents). */
typedef struct mira_stack mira_stack;
typedef struct {
    int32_t n_layers;
    int32_t n_hot, n_stage;     /* slots per layer */
    int32_t k_pred;             /* ids requested from each predictor head (0: no prefetching) */
    int32_t rebalance_every;    /* tokens per layer between rebalancing passes of its HOT set (0: never) */
    int32_t max_swaps;
    float miss_weight, margin;  /* see mira_cache_rebalance */
} mira_stack_config;
size_t mira_stack_scratch_bytes(const mira_ctx* ctx, const mira_stack_config* cfg);
mira_status mira_stack_create(mira_ctx* ctx, const mira_stack_config* cfg, const void* const* host_blobs,
                              void* const* slot_mem, const int32_t* hot, void* dev_scratch, size_t scratch_bytes,
                              void* side_stream, void* stream, mira_stack** out);
void mira_stack_destroy(mira_stack* s);
mira_status mira_stack_layer_step(mira_stack* s, int32_t layer, const void* hidden, int32_t T, const void* router_w,
                                  const float* router_bias, int32_t k, const void* pred_w, const float* pred_b,
                                  void* out, void* stream);
mira_status mira_stack_stats(const mira_stack* s, int64_t* out11, int64_t* out_bytes_staged, int64_t* out_swaps);
void mira_stack_stats_reset(mira_stack* s);
mira_status mira_stack_coverage(const mira_stack* s, double* out_sum, int32_t* out_n);
/* The bookkeeping object of one layer (owned by the stack; for inspection with mira_cache_slot_map / _stats). */
mira_cache* mira_stack_cache(mira_stack* s, int32_t layer);

/* Harness glue of the layer-stack workload (not a step of the paper's method): residual connection plus a
 * parameter-free RMS norm, out[t] = v * rsqrt(mean_c(v^2) + eps) with v = x[t] + moe_out[t] in fp32, rounded once to
 * bf16. x, moe_out, out: [T][hidden] bf16 device (out may alias x), hidden even and <= 16384. No context needed. */
mira_status mira_residual_rmsnorm(const void* x, const void* moe_out, int32_t T, int32_t hidden, float eps, void* out,
                                  void* stream);

/* Number of this library's kernels launched through this context since it was created. */
int64_t mira_kernel_launches(const mira_ctx* ctx);

const char* mira_status_string(mira_status s);

#ifdef __cplusplus
}
#endif
#endif /* MIRA_H_ */
