// Internal declarations shared by the translation units of libmira (not part of the C ABI).
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include <vector>
#include "../../include/mira.h"

namespace mira {

constexpr int kMaxExperts = 256;   // E + n_shared
constexpr int kMaxTopK = 16;
constexpr int kTokBlock = 32;      // tokens of one expert handled by one work item (4 MMA n-tiles)
constexpr int kChunk = 64;         // reduction-dimension bytes of one weight row per pipeline stage
constexpr int kDownSlice = 4096;   // nominal reduction length of one split of the down projection
// The fp16 intermediate v = s_r h_r 2^f of a wide-range expert is kept as two fp16 values, hi = fp16(v) and
// lo = fp16((v - hi) * 2^kLoShift), both saturating: together they hold 11 bits or more of every |v| in
// [2^-38, 2^16). The down projection multiplies both by the same weight fragments and adds the second sum scaled
// by 2^-kLoShift.
constexpr int kLoShift = 24;

// Device-resident schedule written by the grouping kernel and read by the expert kernels.
struct Sched {
    int32_t n_active;                  // experts with at least one pair AND a resident slot
    int32_t act_expert[kMaxExperts];   // active expert ids, ascending
    // A step may split its experts between the two kernel families ("hybrid" step): an active expert with fewer than
    // tc_min[p] pairs is taken by the weight-streaming kernel of projection p (0 up/gate, 1 down), the others by
    // the tcgen05 kernel (tc_min = 0: all tensor-core; INT_MAX: all streaming). The streaming kernels' work lists:
    int32_t tc_min[2];
    int32_t total_tb[2];               // token blocks of the streaming kernel of projection p
    int32_t tb_prefix[2][kMaxExperts + 1];   // exclusive prefix sum of those token blocks per active expert (0 blocks for
                                             // an expert the tensor-core kernel takes)
    // Exclusive prefix sums of the COST of the token blocks, [0] for the up/gate kernel, [1] for the down kernel.
    // A block of 1-8, 9-16, 17-24, 25-32 tokens costs block_cost(., 1..4): the streaming kernels split the work
    // between CTAs by cost, not by block count. Alone, a full block takes about 1.5x the time of an 8-token block
    // (uniform counts: 171 / 193 / 218 / 258 us up/gate, 89 / 97 / 117 / 137 us down); in a batch with mixed counts
    // the gap is wider, because the CTAs of small blocks speed up while the others are compute bound and leave
    // them memory bandwidth, so the costs are those that balanced skewed 16- and 32-token batches best.
    int32_t w_prefix[2][kMaxExperts + 1];
};
__host__ __device__ constexpr int block_cost(int which, int n_tiles) {       // which: 0 up/gate, 1 down; n_tiles 1..4
    return which == 0 ? (n_tiles <= 1 ? 16 : n_tiles == 2 ? 22 : n_tiles == 3 ? 27 : 31)
                      : (n_tiles <= 1 ? 16 : n_tiles == 2 ? 22 : n_tiles == 3 ? 27 : 32);
}

// Where the scale vectors of a compressed expert live (byte offsets from the start of the blob) and how they
// enter the FFN, for the two formats. Shared scale: one vector s[R] scales the up and gate rows and is folded
// into the intermediate h_r once more for the down projection. Per-matrix scales: s1[R] (up), s3[R] (gate),
// and s2[C] applied to the output columns of the down projection; nothing is folded into h.
struct BlobFmt {
    size_t s_up, s_gate, s_out;    // s_out is only read when fold == 0
    int fold;
};
__host__ __device__ inline BlobFmt blob_fmt(int format, int R, int C) {
    const size_t per = (size_t)R * C;
    BlobFmt f;
    f.s_up = 3 * per;
    f.s_gate = format == MIRA_FORMAT_PER_MATRIX ? 3 * per + 2 * (size_t)R + 2 * (size_t)C : 3 * per;
    f.s_out = 3 * per + 2 * (size_t)R;
    f.fold = format == MIRA_FORMAT_PER_MATRIX ? 0 : 1;
    return f;
}

// Byte offsets of the regions inside the caller's workspace.
struct Layout {
    size_t status;      // int32[16]: [0] status bits, [8] route ticket; then miss mask uint32[8], done mask uint32[8]
    size_t sched;       // Sched
    size_t logits;      // float [Tmax][E]
    size_t idx;         // int32 [Tmax][kmax]
    size_t w;           // float [Tmax][kmax]
    size_t count;       // int32 [Et]
    size_t offset;      // int32 [Et+1]
    size_t perm;        // int32 [Tmax][kmax+ns]
    size_t row_token;   // int32 [Pmax]   position -> token
    size_t xscale;      // float [Tmax]   2^p_t that undoes the fp16 pre-scaling of token t
    size_t xnorm;       // float [Tmax]   Euclidean norm of token t
    size_t xsum;        // float [Tmax]   sum of the fp16 activations of token t
    size_t hscale;      // float [Pmax]   2^-f_p that undoes the per-pair scaling of the fp16 intermediate
    size_t hexp;        // int32 [2][kMaxExperts] per expert: exponent of the intermediate's expected magnitude per unit of
                        //                |x|^2; then 1 if the expert keeps a second (lower) window of its fp16 intermediate
    size_t h16lo;       // half  [Pmax][R] the lower window of the intermediate (wide-range experts only)
    size_t x16;         // half  [Tmax][C]
    size_t x16p;        // half  [Pmax][C] activations in position order (tensor-core path only)
    size_t xs_pos;      // float [Pmax]    per position: undo factor of the token's fp16 pre-scaling (tensor-core path)
    size_t hm_pos;      // float [Pmax]    per position: 2^f applied to the fp16 intermediate (tensor-core path)
    size_t sum_pos;     // float [Pmax]    per position: sum of the token's fp16 activations (tensor-core path)
    size_t h16;         // half  [Pmax][R]
    size_t ypart;       // float [S][Pmax][C] split partial sums of the down projection
    size_t pred;        // float [Tmax][E] per-token predictor scores when the caller passes none
    size_t mix;         // float [8][C + E] partial column sums of the MixtureHead's mean features
    size_t tickets;     // uint32 [Tmax / 8 + 1] arrival counters of the 2-D score kernel, one per token group (zero at rest)
    size_t total;
};

struct RouteView {      // device pointers to one routing result
    int32_t* idx; float* w; int32_t* count; int32_t* offset; int32_t* perm; float* logits;
    int32_t* row_token;
};

}  // namespace mira

namespace mira {
struct ProfRec { int id; cudaEvent_t a, b; };
}

struct mira_ctx {
    alignas(64) unsigned char tmap_x16p[6][128];   // CUtensorMaps of x16p (tensor-core path): boxes of 32, 64, ..., 192 rows
    alignas(64) unsigned char tmap_h16[6][128];    // CUtensorMaps of h16, likewise
    alignas(64) unsigned char tmap_h16lo[6][128];  // CUtensorMaps of h16lo, likewise
    alignas(64) unsigned char tmap_half[3][6][128]; // x16p, h16, h16lo with boxes of 16, 32, ..., 96 rows (two-SM kernels)
    bool tensor_path_ok = false;
    bool force_decode_path = false;
    int tc_layout = 0;                 // 0: chosen per step; 1..3 force a tile layout of the tensor-core kernels (MIRA_OPT_TENSOR_LAYOUT)
    bool test_wait_timeout = false;    // the next tcgen05 up/gate launch drops one load and shortens its waits (MIRA_OPT_TEST_WAIT_TIMEOUT)
    int hybrid_min[2] = {-1, -1};      // MIRA_OPT_HYBRID_MIN_UP / _DOWN: -1 = chosen per step, else the pair count from which an
                                       // expert goes to the tcgen05 kernel of that projection (0: all, INT_MAX: none)
    int down_slices_forced = 0;        // MIRA_OPT_DOWN_SLICES: 0 = chosen per step, else the reduction slices of the tcgen05 down kernel
    int up_conversion = 0;             // tcgen05 up/gate kernel: 0, 1: exact code conversion; 2: offset subnormals (MIRA_OPT_UP_CONVERSION)
    bool prof_on = false;
    size_t prof_used = 0;
    std::vector<mira::ProfRec> prof;   // per-launch event pairs, reused between reads
    mira_config cfg;
    mira::Layout lay;
    char* ws;
    size_t ws_bytes;
    int device;
    int n_sm;
    int down_splits;        // S
    int down_slice;         // reduction length per split (multiple of 64)
    int route_T;            // T of the last routing call (-1: none)
    int route_k;
    int64_t launches;
    // While set (by the stack runtime, around one routing call), the grouping kernel also writes the per-expert counts
    // to this host-mapped buffer and then notify_seq to the flag (device addresses of pinned host memory).
    int32_t* notify_count = nullptr;
    uint32_t* notify_flag = nullptr;
    uint32_t notify_seq = 0;
    int32_t* notify_ids = nullptr;      // likewise for the pooling kernel's top-k ids (mira_predict)
    uint32_t* notify_ids_flag = nullptr;
};

namespace mira {

inline size_t blob_bytes(const mira_config& c) { return mira_expert_bytes_format(c.ffn, c.hidden, c.format); }
inline int Et(const mira_config& c) { return c.n_experts + c.n_shared; }
inline int Pmax(const mira_config& c) { return c.max_tokens * (c.max_top_k + c.n_shared); }

template <typename T> inline T* ws_ptr(const mira_ctx* ctx, size_t off) { return reinterpret_cast<T*>(ctx->ws + off); }

// quantize.cu
mira_status launch_quantize(mira_ctx*, const void* w1, const void* w2, const void* w3, int src_dtype,
                            int n, void* blobs, cudaStream_t);
mira_status launch_unpack(mira_ctx*, const void* blob, int8_t* q1, int8_t* q2, int8_t* q3, float* w1,
                          float* w2, float* w3, cudaStream_t);
// route.cu
mira_status launch_scores(mira_ctx*, const void* x, int T, const void* w, const float* b, int E,
                          float* scores, __half* x16, float* xscale, float* xnorm, cudaStream_t);
// (launch_route and launch_schedule write the schedule for the thresholds step_tc_min gives for (T, k))
mira_status launch_route(mira_ctx*, const void* x, int T, const void* w, const float* b, int k,
                         const RouteView& rv, __half* x16, float* xscale, float* xnorm, void* const* slots,
                         const int32_t* slot_map, int* fused_schedule, cudaStream_t, bool quiet_schedule = false);
mira_status launch_schedule(mira_ctx*, int T, void* const* slots, const int32_t* slot_map, const uint32_t* dev_expert_mask,
                            int all_experts, cudaStream_t);
mira_status launch_pool(mira_ctx*, const float* token_scores, int T, int E, float* pooled,
                        int32_t* ids, int k_pred, cudaStream_t);
// expert_ffn.cu
mira_status launch_up_gate(mira_ctx*, void* const* slots, const int32_t* slot_map, cudaStream_t);
mira_status launch_down(mira_ctx*, void* const* slots, const int32_t* slot_map, cudaStream_t);
mira_status launch_combine(mira_ctx*, int T, int k, int splits, int tc_splits, int down_tc_min, void* out, cudaStream_t);
int down_tc_slices(const mira_ctx*);     // reduction slices the tensor-core down kernel uses for the step last routed
// expert_ffn_tc.cu (tcgen05 path for prefill-sized batches)
bool tc_shape_ok(const mira_config&);
bool build_tensor_maps(mira_ctx*);
mira_status launch_up_gate_tc(mira_ctx*, void* const* slots, const int32_t* slot_map, cudaStream_t);
mira_status launch_down_tc(mira_ctx*, void* const* slots, const int32_t* slot_map, cudaStream_t);
mira_status set_tc_attributes();
// From how many tokens a step takes the tcgen05 kernel instead of the weight-streaming one, separately for the up/gate
// and the down projection (measured, us per kernel, streaming / tcgen05: Mixtral shape up/gate 40 tokens 182 / 200,
// 56 tokens 202 / 203, down 32 tokens 103 / 102, 40 tokens 115 / 104, 48 tokens 118 / 104; fine-grained shape with
// 64 experts up/gate 16 tokens 38 / 42, 32 tokens 48 / 44, down 16 tokens 26 / 23, 32 tokens 30 / 27; below these
// sizes the streaming kernels win: Mixtral shape 16 tokens 0.231 / 0.240 ms per step, fine-grained 4 tokens 0.055 /
// 0.057). The down projection switches earlier: its exact conversion costs the streaming kernel more per weight.
constexpr int kTensorPathMinTokens = 16;    // below, no buffers of the tensor path are laid out
inline int tc_min_tokens_up(const mira_config& c) { return c.n_experts + c.n_shared > 16 ? 20 : 56; }
inline int tc_min_tokens_down(const mira_config& c) { return c.n_experts + c.n_shared > 16 ? 16 : 40; }
// Per projection (0 up/gate, 1 down): the pair count from which an expert of a T-token step goes to the tcgen05
// kernel (0: every expert; INT_MAX: none). The same rule for every wave of a routed batch.
void step_tc_min(const mira_ctx* ctx, int T, int k, int out_min[2]);
mira_status set_route_attributes();
// mixture_head.cu
mira_status launch_mixture(mira_ctx*, const void* hidden, int T, const float* logits, const int32_t* count, int k_top,
                           const mira_mixture_head& head, float* out_scores, float* out_probs, float* out_alpha,
                           int32_t* out_ids, int k_pred, cudaStream_t);
mira_status set_mixture_attributes();
mira_status set_ffn_attributes();
mira_status set_quantize_attributes();

// api.cu: the pieces of a layer step for the stack runtime, which starts the resident experts before the host has
// read the routing counts. route_and_schedule = S1-S3 plus the schedule over every routed expert that slot_map
// holds (an expert without a slot is left for a later wave, not reported); run_scheduled_experts = S4 + S5 for the
// schedule in place; combine_only = S6 (pairs of experts no wave has run contribute zero and raise the miss flag).
mira_status route_and_schedule(mira_ctx*, const void* hidden, int T, const void* router_w, const float* bias, int k,
                               void* const* slots, const int32_t* slot_map, cudaStream_t);
mira_status run_scheduled_experts(mira_ctx*, int T, void* const* slots, const int32_t* slot_map, cudaStream_t);
mira_status combine_only(mira_ctx*, int T, void* out, cudaStream_t);

// Brackets one kernel launch with events when profiling is enabled (see mira_profile).
struct ProfScope {
    mira_ctx* ctx; cudaStream_t st; cudaEvent_t stop = nullptr;
    ProfScope(mira_ctx* c, int id, cudaStream_t s) : ctx(c), st(s) {
        if (!c->prof_on || c->prof_used >= MIRA_PROFILE_MAX_RECORDS) return;
        if (c->prof_used == c->prof.size()) {
            ProfRec r; r.id = id;
            if (cudaEventCreate(&r.a) != cudaSuccess) return;
            if (cudaEventCreate(&r.b) != cudaSuccess) { cudaEventDestroy(r.a); return; }
            c->prof.push_back(r);
        }
        ProfRec& r = c->prof[c->prof_used++];
        r.id = id;
        cudaEventRecord(r.a, st);
        stop = r.b;
    }
    ~ProfScope() { if (stop) cudaEventRecord(stop, st); }
};

// Programmatic dependent launch: the kernels of one layer step are launched with this attribute, so the next
// kernel's CTAs are scheduled (and run their preamble) while the previous kernel drains. Every such kernel
// executes pdl_wait() before it touches anything an earlier kernel of the stream wrote or still reads, and
// pdl_launch() only AFTER that wait, so that "the previous kernel has started" implies "everything before it
// has completed".
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
#endif

#define MIRA_CUDA_OK(expr) do { cudaError_t e__ = (expr); if (e__ != cudaSuccess) return MIRA_ERR_CUDA; } while (0)

}  // namespace mira
