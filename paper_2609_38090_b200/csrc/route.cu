// S1-S3 and S7: router / predictor scores, warp-shuffle top-k with softmax weights, grouping of the
// (token, expert) pairs by expert, and the work schedule the expert kernels read.
//
//   scores  (Section II-A, Section IV-E): score[t][e] = sum_c x[t][c] * W[e][c] + b[e], fp32.
//   top-k   (Section II-A): k best logits per token, ties to the lower index; weights = softmax over
//           the selected logits, best first.
//   group   : stable counting sort of the pairs by expert, tokens ascending (no atomics: one warp
//           walks the tokens of "its" expert in order with ballots, so the result is unique).
#include <mutex>
#include <algorithm>
#include "mira_internal.cuh"

namespace mira {
namespace {

constexpr int kScoreTok = 4;       // tokens per CTA of the score kernel
constexpr int kScoreThreads = 256;
constexpr int kFusedRouteMaxTokens = 128;   // up to here one CTA per token + last-CTA grouping is used ...
constexpr int kFusedRouteMaxTokensFewExperts = 512;   // ... and up to here with at most 16 experts, where the separate score and
                                                      // grouping launches cost more than the serial tail (256 tokens x 8 experts: 0.370 against 0.375 ms)

__device__ __forceinline__ float bf16lo(unsigned v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(unsigned v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ int expo_of(float v) { return (int)((__float_as_uint(v) >> 23) & 0xff) - 127; }

__device__ __forceinline__ float dot8(const uint4& a, const uint4& b, float acc) {
    acc = fmaf(bf16lo(a.x), bf16lo(b.x), acc); acc = fmaf(bf16hi(a.x), bf16hi(b.x), acc);
    acc = fmaf(bf16lo(a.y), bf16lo(b.y), acc); acc = fmaf(bf16hi(a.y), bf16hi(b.y), acc);
    acc = fmaf(bf16lo(a.z), bf16lo(b.z), acc); acc = fmaf(bf16hi(a.z), bf16hi(b.z), acc);
    acc = fmaf(bf16lo(a.w), bf16lo(b.w), acc); acc = fmaf(bf16hi(a.w), bf16hi(b.w), acc);
    return acc;
}

// Warp top-k over up to 256 values held 8 per lane (value j of lane l is element l + 32 j).
// Order: value descending, index ascending. Lane 0 returns through out_idx / out_val (k <= 16).
// Warps walk the router rows in rounds (row w, w + nwarps, ...). The rows of the later rounds are requested
// into L2 up front, so that after a step that streamed the experts through L2 only the first round pays DRAM
// latency.
__device__ __forceinline__ void prefetch_rows_l2(const void* W, int row_bytes, int first, int step, int n_rows, int lane) {
    for (int e = first; e < n_rows; e += step)
        for (int off = lane * 128; off < row_bytes; off += 32 * 128)
            asm volatile("prefetch.global.L2 [%0];\n" ::"l"(static_cast<const char*>(W) + (size_t)e * row_bytes + off));
}

// The selection runs on 32-bit keys that order like the logits (sign-magnitude floats mapped to unsigned; -0 counts as
// +0, a NaN ranks below every number), with two hardware warp reductions per selected expert: the largest key, then
// the lowest index that holds it. Keys: 0 = no candidate (beyond E, or already selected), 1 = NaN, else the logit.
// SLOTS = values per lane that can be occupied (2 covers 64 experts): this code runs once per token on the critical
// path of a decode step, where every instruction is fetched cold, so the short form matters.
__device__ __forceinline__ unsigned topk_key(float v) {
    if (!(v == v)) return 1u;
    const unsigned b = __float_as_uint(v + 0.f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float topk_value(unsigned key) {
    if (key <= 1u) return key ? __uint_as_float(0x7fc00000u) : -INFINITY;
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}
// One selection step: returns the winner's index and key to every lane and retires it. With nothing left the result is
// index 0 with key 0.
template <int SLOTS>
__device__ __forceinline__ void topk_step(unsigned (&key)[SLOTS], int lane, int& win_idx, unsigned& win_key) {
    unsigned bk = 0u;
#pragma unroll
    for (int i = 0; i < SLOTS; ++i) bk = max(bk, key[i]);
    win_key = __reduce_max_sync(0xffffffffu, bk);
    unsigned cand = 0xffffffffu;
#pragma unroll
    for (int i = SLOTS - 1; i >= 0; --i) if (key[i] == win_key) cand = (unsigned)(lane + 32 * i);
    const unsigned w = __reduce_min_sync(0xffffffffu, win_key ? cand : 0xffffffffu);
    win_idx = (w == 0xffffffffu) ? 0 : (int)w;
#pragma unroll
    for (int i = 0; i < SLOTS; ++i) if (win_key && lane + 32 * i == win_idx) key[i] = 0u;
}

template <int SLOTS>
__device__ __forceinline__ void warp_topk_n(const float (&v)[8], int E, int k, int lane, int* out_idx, float* out_val) {
    unsigned key[SLOTS];
#pragma unroll
    for (int i = 0; i < SLOTS; ++i) key[i] = (lane + 32 * i < E) ? topk_key(v[i]) : 0u;
#pragma unroll 1
    for (int j = 0; j < k; ++j) {
        int bi; unsigned bk;
        topk_step<SLOTS>(key, lane, bi, bk);
        if (lane == 0) { out_idx[j] = bi; out_val[j] = topk_value(bk); }
    }
}
__device__ __forceinline__ void warp_topk(float (&v)[8], int E, int k, int lane, int* out_idx, float* out_val) {
    if (E <= 64) warp_topk_n<2>(v, E, k, lane, out_idx, out_val);
    else warp_topk_n<8>(v, E, k, lane, out_idx, out_val);
}

// The same selection with the results spread over the lanes: lane j (< k) returns the j-th selection. Used by the
// single-CTA routing kernel (at most 16 experts: one slot per lane).
__device__ __forceinline__ void warp_topk_lanes(float (&v)[8], int E, int k, int lane, int& my_idx, float& my_val) {
    my_idx = 0; my_val = -INFINITY;
    unsigned key[1] = {lane < E ? topk_key(v[0]) : 0u};
#pragma unroll 1
    for (int j = 0; j < k; ++j) {
        int bi; unsigned bk;
        topk_step<1>(key, lane, bi, bk);
        if (lane == j) { my_idx = bi; my_val = topk_value(bk); }
    }
}

// Routing weight of lane j's selection: softmax over the k selected logits, the sum taken in selection order
// (the same arithmetic, in the same order, as the list form's loop on lane 0).
__device__ __forceinline__ float topk_softmax(float my_val, int k, int lane) {
    const float top = __shfl_sync(0xffffffffu, my_val, 0);
    const float p = lane < k ? expf(my_val - top) : 0.f;
    float z = 0.f;
    for (int j = 0; j < k; ++j) z += __shfl_sync(0xffffffffu, p, j);
    return p / z;
}

// One CTA scores kScoreTok tokens against all E rows of W. Optionally: writes the fp16 copy of the
// tokens pre-scaled by a power of two (so that any bf16 magnitude fits fp16 exactly) and selects
// the top-k experts with their softmax weights.
// The fp16 copy of a CTA's tokens (rows of xs in shared memory, warp w takes token w) with its per-token numbers: the
// power-of-two scale that puts the row maximum in [2^13, 2^14), the norm of the row and the sum of the fp16 values
// the expert kernels will read. Called by every thread of the CTA; n_threads = its size.
__device__ __forceinline__ void write_fp16_copy(const uint4* xs, int c8, int nt, int t0, int n_threads, float* s_scale,
                                                __half* __restrict__ x16, float* __restrict__ xscale,
                                                float* __restrict__ xnorm, float* __restrict__ xsum) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (warp < nt) {
        float m = 0.f;
        for (int i = lane; i < c8; i += 32) {
            uint4 v = xs[warp * c8 + i];
            m = fmaxf(m, fmaxf(fmaxf(fabsf(bf16lo(v.x)), fabsf(bf16hi(v.x))), fmaxf(fabsf(bf16lo(v.y)), fabsf(bf16hi(v.y)))));
            m = fmaxf(m, fmaxf(fmaxf(fabsf(bf16lo(v.z)), fabsf(bf16hi(v.z))), fmaxf(fabsf(bf16lo(v.w)), fabsf(bf16hi(v.w)))));
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        int ex = (int)((__float_as_uint(m) >> 23) & 0xff) - 127;
        ex = (m > 0.f) ? max(-100, min(127, ex)) : 13;
        const float sc_up = __uint_as_float((unsigned)(127 + 13 - ex) << 23);
        const float sc_dn = __uint_as_float((unsigned)(127 - 13 + ex) << 23);
        float ss = 0.f;     // sum of squares of the scaled row (every term <= 2^28)
        float sm = 0.f;     // sum of the fp16 values the expert kernels will read
        for (int i = lane; i < c8; i += 32) {
            uint4 v = xs[warp * c8 + i];
            const unsigned w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float a = bf16lo(w4[j]) * sc_up, b = bf16hi(w4[j]) * sc_up;
                ss = fmaf(a, a, ss); ss = fmaf(b, b, ss);
                const float2 hf = __half22float2(__floats2half2_rn(a, b));
                sm += hf.x; sm += hf.y;
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            ss += __shfl_xor_sync(0xffffffffu, ss, o);
            sm += __shfl_xor_sync(0xffffffffu, sm, o);
        }
        if (lane == 0) {
            s_scale[warp] = sc_up;
            xscale[t0 + warp] = sc_dn;
            xnorm[t0 + warp] = sqrtf(ss) * sc_dn;
            xsum[t0 + warp] = sm;
        }
    }
    __syncthreads();
    uint4* og = reinterpret_cast<uint4*>(x16) + (size_t)t0 * c8;
    for (int i = threadIdx.x; i < nt * c8; i += n_threads) {
        const float sc = s_scale[i / c8];
        uint4 v = xs[i], o;
        __half2 h;
        h = __floats2half2_rn(bf16lo(v.x) * sc, bf16hi(v.x) * sc); o.x = *reinterpret_cast<unsigned*>(&h);
        h = __floats2half2_rn(bf16lo(v.y) * sc, bf16hi(v.y) * sc); o.y = *reinterpret_cast<unsigned*>(&h);
        h = __floats2half2_rn(bf16lo(v.z) * sc, bf16hi(v.z) * sc); o.z = *reinterpret_cast<unsigned*>(&h);
        h = __floats2half2_rn(bf16lo(v.w) * sc, bf16hi(v.w) * sc); o.w = *reinterpret_cast<unsigned*>(&h);
        og[i] = o;
    }
}

__global__ void __launch_bounds__(kScoreThreads)
k_scores(const __nv_bfloat16* __restrict__ x, int T, int C, const __nv_bfloat16* __restrict__ W,
         const float* __restrict__ bias, int E, float* __restrict__ scores, __half* __restrict__ x16,
         float* __restrict__ xscale, float* __restrict__ xnorm, float* __restrict__ xsum, int k,
         int32_t* __restrict__ idx,
         float* __restrict__ wts) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint4* xs = reinterpret_cast<uint4*>(smem);                       // [kScoreTok][C/8]
    float* sc = reinterpret_cast<float*>(smem + (size_t)kScoreTok * C * 2);  // [kScoreTok][E]
    __shared__ float s_scale[kScoreTok];
    pdl_wait();            // (a no-op unless launched with programmatic serialization: the routing path of large batches)
    pdl_launch();
    const int t0 = blockIdx.x * kScoreTok;
    const int nt = min(kScoreTok, T - t0);
    const int c8 = C / 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = kScoreThreads / 32;
    const uint4* xg = reinterpret_cast<const uint4*>(x) + (size_t)t0 * c8;
    for (int i = threadIdx.x; i < kScoreTok * c8; i += kScoreThreads)
        xs[i] = (i < nt * c8) ? xg[i] : make_uint4(0, 0, 0, 0);
    __syncthreads();

    if (x16 != nullptr) write_fp16_copy(xs, c8, nt, t0, kScoreThreads, s_scale, x16, xscale, xnorm, xsum);

    // Plain scores (no top-k, no fp16 copy: the predictor) may split the experts over gridDim.y CTAs per token
    // group, so that a decode batch of a many-expert layer does not read the whole head through one SM.
    const uint4* wg = reinterpret_cast<const uint4*>(W);
    const bool split = gridDim.y > 1;
    for (int e = warp + nwarp * blockIdx.y; e < E; e += nwarp * gridDim.y) {
        float acc[kScoreTok];
#pragma unroll
        for (int j = 0; j < kScoreTok; ++j) acc[j] = 0.f;
#pragma unroll 8
        for (int i = lane; i < c8; i += 32) {
            uint4 wv = __ldg(wg + (size_t)e * c8 + i);
#pragma unroll
            for (int j = 0; j < kScoreTok; ++j) acc[j] = dot8(wv, xs[j * c8 + i], acc[j]);
        }
#pragma unroll
        for (int j = 0; j < kScoreTok; ++j) {
#pragma unroll
            for (int o = 16; o; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
        }
        if (lane == 0) {
            float b = bias ? bias[e] : 0.f;
#pragma unroll
            for (int j = 0; j < kScoreTok; ++j) {
                sc[j * E + e] = acc[j] + b;
                if (split && j < nt) scores[(size_t)(t0 + j) * E + e] = acc[j] + b;
            }
        }
    }
    if (split) return;
    __syncthreads();
    if (scores != nullptr)
        for (int i = threadIdx.x; i < nt * E; i += kScoreThreads) scores[(size_t)t0 * E + i] = sc[i];
    if (idx != nullptr && warp < nt) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (lane + 32 * i < E) ? sc[warp * E + lane + 32 * i] : -INFINITY;
        int oi[kMaxTopK]; float ov[kMaxTopK];
        warp_topk(v, E, k, lane, oi, ov);
        if (lane == 0) {
            float z = 0.f, p[kMaxTopK];
            for (int j = 0; j < k; ++j) { p[j] = expf(ov[j] - ov[0]); z += p[j]; }
            for (int j = 0; j < k; ++j) {
                idx[(size_t)(t0 + warp) * k + j] = oi[j];
                wts[(size_t)(t0 + warp) * k + j] = p[j] / z;
            }
        }
    }
}

// S3, run by ONE CTA (any multiple of 32 threads). Warp w owns experts w, w + nwarps, ...: it scans the
// tokens in ascending order, 32 at a time, and gives every pair routed to its expert the next local
// rank. Then offsets and positions. `idx` is read with L2 loads because the fused route kernel calls
// this from the last CTA to finish, on values other CTAs of the same launch wrote.
struct GroupArgs {
    const int32_t* idx; int T, k, E, ns;
    int32_t* count; int32_t* offset; int32_t* perm; int32_t* row_token; uint32_t* done_mask;
    // Optional notification of a waiting host thread: the counts are also written to host-mapped memory, then (after a
    // system-scope fence) the sequence number to the flag, so the host learns them without a copy or a
    // synchronisation call in the stream.
    int32_t* host_count; volatile uint32_t* host_flag; uint32_t host_seq;
};

// Called by every thread of the (single) grouping CTA after the counts sit in s_count.
__device__ __forceinline__ void notify_host(const GroupArgs& G, const int* s_count, int n) {
    if (G.host_count == nullptr) return;
    for (int e = threadIdx.x; e < n; e += blockDim.x) G.host_count[e] = s_count[e];
    __threadfence_system();
    __syncthreads();
    if (threadIdx.x == 0) { __threadfence_system(); *G.host_flag = G.host_seq; }     // the storing thread releases at system scope
}

// off[e] = sum of count[0..e), off[n] = the total, for n entries in shared memory, by one warp: every lane adds its run
// of consecutive entries, a shuffle scan over the lanes' sums gives each run its start. Written as short loops: the
// code runs once per step in one CTA, where instruction fetch costs more than the arithmetic (a thread walking 64
// entries took 1.3 us, and so did a fully unrolled version of this).
__device__ __forceinline__ void exclusive_offsets(const int* count, int* off, int n, int lane) {
    const int per = (n + 31) >> 5, base = lane * per, stop = min(n, base + per);
    int sum = 0;
#pragma unroll 1
    for (int i = base; i < stop; ++i) sum += count[i];
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int up = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += up; }
    int run = incl - sum;
#pragma unroll 1
    for (int i = base; i < stop; ++i) { off[i] = run; run += count[i]; }
    if (lane == 31) off[n] = incl;
}

// S3 by one CTA in O(pairs): the routed pairs, in (token, choice) order, are cut into one contiguous range per warp.
// Pass 1 builds each warp's histogram over the experts (32 pairs per step; lanes with the same expert find each
// other with match.any, the lowest one adds the group's size). An exclusive prefix over the warps turns the
// histograms into each warp's first rank per expert, the totals are the counts. Pass 2 walks the pairs again in the
// same order: rank = the warp's running rank of that expert + the number of lower lanes with the same expert. The
// order inside an expert is the token order (a stable counting sort), with no atomics.
// s_hist: nwarps * E ints of scratch.
template <bool FEW>
__device__ __forceinline__ void group_body(const GroupArgs& G, int* s_count, int* s_off, int* s_hist) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int T = G.T, k = G.k, E = G.E, ns = G.ns, kk = k + ns;
    const int P = T * k;
    if (threadIdx.x < 8) G.done_mask[threadIdx.x] = 0u;
    const unsigned lt = (1u << lane) - 1u;
    // At most 64 pairs (the decode steps of a beam or a small batch): every warp holds all pairs, up to two per lane,
    // and counts "its" experts with a ballot per half; no histograms, no prefix over the warps, one pass. This is the
    // step's critical path and is fetched cold, so the short form is worth its own branch (4 tokens x top-4 of 60
    // experts: 3.8 -> 2 us).
    constexpr bool few = FEW;            // chosen at launch: P <= 64
    int e_mine = -1, e_hi = -1;          // the experts of pairs `lane` and `lane + 32`
    if (few) {
        if (lane < P) e_mine = __ldcg(G.idx + lane);
        if (lane + 32 < P) e_hi = __ldcg(G.idx + lane + 32);
#pragma unroll 1
        for (int e = warp; e < E; e += nwarps) {
            const unsigned m = __ballot_sync(0xffffffffu, e_mine == e), mh = __ballot_sync(0xffffffffu, e_hi == e);
            if (lane == 0) s_count[e] = __popc(m) + __popc(mh);
        }
    } else {
        for (int i = threadIdx.x; i < nwarps * E; i += blockDim.x) s_hist[i] = 0;
        __syncthreads();
    }
    const int chunk = ((P + nwarps - 1) / nwarps + 31) & ~31;
    const int p0 = few ? 0 : min(P, warp * chunk), p1 = few ? 0 : min(P, p0 + chunk);
    int* hist = s_hist + warp * E;
    for (int base = p0; base < p1; base += 32) {
        const int p = base + lane;
        const bool valid = p < p1;
        const unsigned active = __ballot_sync(0xffffffffu, valid);
        if (valid) {
            const int e = __ldcg(G.idx + p);
            const unsigned m = __match_any_sync(active, e);
            if ((m & lt) == 0) hist[e] += __popc(m);
        }
        __syncwarp();
    }
    if (!few) {
        __syncthreads();
        for (int e = threadIdx.x; e < E; e += blockDim.x) {
            int run = 0;
            for (int w = 0; w < nwarps; ++w) { const int v = s_hist[w * E + e]; s_hist[w * E + e] = run; run += v; }
            s_count[e] = run;
        }
    }
    for (int s = threadIdx.x; s < ns; s += blockDim.x) s_count[E + s] = T;
    __syncthreads();
    if (warp == 0) exclusive_offsets(s_count, s_off, E + ns, lane);
    __syncthreads();
    notify_host(G, s_count, E + ns);
    for (int e = threadIdx.x; e <= E + ns; e += blockDim.x) {
        G.offset[e] = s_off[e];
        if (e < E + ns) G.count[e] = s_count[e];
    }
    if (few && warp == 0) {                  // rank inside the expert = earlier pairs with the same expert (token order)
        const int n_lo = min(P, 32), n_hi = P - n_lo;
        int below = 0;                       // pairs of the first half with the expert of this lane's second-half pair
        unsigned m = 0;
        if (lane < n_lo) m = __match_any_sync(n_lo == 32 ? 0xffffffffu : (1u << n_lo) - 1u, e_mine);
        if (n_hi > 0) {                      // through a few words of shared memory: zero, first half's group sizes, read
            if (lane < n_hi) s_hist[e_hi] = 0;
            __syncwarp();
            if (lane < n_lo && (m & lt) == 0) s_hist[e_mine] = __popc(m);
            __syncwarp();
            if (lane < n_hi) below = s_hist[e_hi];
        }
        if (lane < n_lo) {
            const int pos = s_off[e_mine] + __popc(m & lt);
            const int t = lane / k, j = lane - t * k;
            G.perm[(size_t)t * kk + j] = pos;
            G.row_token[pos] = t;
        }
        if (lane < n_hi) {
            const unsigned mh = __match_any_sync(n_hi == 32 ? 0xffffffffu : (1u << n_hi) - 1u, e_hi);
            const int pos = s_off[e_hi] + below + __popc(mh & lt);
            const int p = lane + 32, t = p / k, j = p - t * k;
            G.perm[(size_t)t * kk + j] = pos;
            G.row_token[pos] = t;
        }
    }
    for (int base = p0; base < p1; base += 32) {
        const int p = base + lane;
        const bool valid = p < p1;
        const unsigned active = __ballot_sync(0xffffffffu, valid);
        int e = 0;
        unsigned m = 0;
        if (valid) {
            e = __ldcg(G.idx + p);
            m = __match_any_sync(active, e);
            const int pos = s_off[e] + hist[e] + __popc(m & lt);
            const int t = p / k, j = p - t * k;
            G.perm[(size_t)t * kk + j] = pos;
            G.row_token[pos] = t;
        }
        __syncwarp();
        if (valid && (m & lt) == 0) hist[e] += __popc(m);
        __syncwarp();
    }
    for (int q = threadIdx.x; q < T * ns; q += blockDim.x) {       // shared experts: every token, in token order
        const int t = q / ns, sx = q - t * ns;
        const int pos = s_off[E + sx] + t;
        G.perm[(size_t)t * kk + k + sx] = pos;
        G.row_token[pos] = t;
    }
}

constexpr int kGroupScratch = 32 * kMaxExperts;      // ints: a histogram row per warp of the grouping CTA (32 KB)

struct MaskArg { uint32_t w[8]; };

// Work schedule for one wave of expert execution: which experts run (routed to, selected by the
// caller's mask, resident), how many 32-token blocks each has; records misses and completed experts.
// Run by one CTA of at least Etot threads; `count` may come from shared memory (fused) or global.
struct SchedArgs {
    const int32_t* slot_map; MaskArg mask; Sched* sched; int32_t* status; uint32_t* miss_mask; uint32_t* done_mask;
    int quiet;      // 1: a routed expert without a slot is left for a later wave, not reported as a miss
    // hexp[e]: exponent of the largest magnitude the intermediate of expert e is expected to reach per unit of |x|^2
    // (from the largest row scale of the blob in its slot), then the wide-range flags; written by the statistics CTAs.
    void* const* slots; int32_t* hexp;
    int tc_min[2];                      // hybrid thresholds of the step (see Sched)
    int T, R, C, per_matrix, n_main;    // n_main: CTAs of the launch that are not statistics CTAs
};

// Statistics CTA of expert e (every thread of the CTA calls it): the largest row scale of the blob in the expert's
// slot, as the exponent the SwiGLU epilogues use to place the fp16 intermediate. Shared scale: the intermediate
// s_r h_r grows like s^3; per-matrix scales: like s1 * s3. Experts without a slot, or outside the wave, are skipped.
__device__ __forceinline__ float max8_bf16(const uint4& v) {
    return fmaxf(fmaxf(fmaxf(bf16lo(v.x), bf16hi(v.x)), fmaxf(bf16lo(v.y), bf16hi(v.y))),
                 fmaxf(fmaxf(bf16lo(v.z), bf16hi(v.z)), fmaxf(bf16lo(v.w), bf16hi(v.w))));
}
__device__ __forceinline__ float min8_bf16(const uint4& v) {
    return fminf(fminf(fminf(bf16lo(v.x), bf16hi(v.x)), fminf(bf16lo(v.y), bf16hi(v.y))),
                 fminf(fminf(bf16lo(v.z), bf16hi(v.z)), fminf(bf16lo(v.w), bf16hi(v.w))));
}

__device__ __forceinline__ void expert_stats(const SchedArgs& S, int e) {
    __shared__ float s_m[4][32];
    const bool sel = (S.mask.w[e >> 5] >> (e & 31)) & 1u;
    const int slot = (S.slots != nullptr && S.slot_map != nullptr && sel) ? S.slot_map[e] : -1;
    if (slot < 0) return;
    const unsigned char* blob = static_cast<const unsigned char*>(S.slots[slot]);
    const BlobFmt f = blob_fmt(S.per_matrix ? MIRA_FORMAT_PER_MATRIX : MIRA_FORMAT_SHARED, S.R, S.C);
    const uint4* su = reinterpret_cast<const uint4*>(blob + f.s_up);
    const uint4* sg = reinterpret_cast<const uint4*>(blob + f.s_gate);
    float m1 = 0.f, m3 = 0.f, n1 = INFINITY, n3 = INFINITY;      // largest and smallest row scale (scales are positive)
    for (int i = threadIdx.x; i < S.R / 8; i += blockDim.x) {
        const uint4 v = __ldg(su + i);
        m1 = fmaxf(m1, max8_bf16(v)); n1 = fminf(n1, min8_bf16(v));
        if (S.per_matrix) {
            const uint4 w = __ldg(sg + i);
            m3 = fmaxf(m3, max8_bf16(w)); n3 = fminf(n3, min8_bf16(w));
        }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o)); n1 = fminf(n1, __shfl_xor_sync(0xffffffffu, n1, o));
        m3 = fmaxf(m3, __shfl_xor_sync(0xffffffffu, m3, o)); n3 = fminf(n3, __shfl_xor_sync(0xffffffffu, n3, o));
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    if (lane == 0) { s_m[0][warp] = m1; s_m[1][warp] = m3; s_m[2][warp] = n1; s_m[3][warp] = n3; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < nwarps; ++w) {
            m1 = fmaxf(m1, s_m[0][w]); m3 = fmaxf(m3, s_m[1][w]); n1 = fminf(n1, s_m[2][w]); n3 = fminf(n3, s_m[3][w]);
        }
        S.hexp[e] = S.per_matrix ? expo_of(m1) + expo_of(m3) : 3 * expo_of(m1);
        // Wide-range experts: the intermediate is placed by the LARGEST row scale, and one fp16 window holds rows
        // whose terms are up to 2^12 smaller. With the row scales spread over more than 8x (terms grow like s^3;
        // per-matrix scales: s1 * s3 over more than 64x) the rows that carry the down projection's sum may fall
        // below that window, so such experts keep a second fp16 window 2^24 lower (see kLoShift in the expert
        // kernels) and their down projection runs over both.
        S.hexp[kMaxExperts + e] = S.per_matrix ? (m1 * m3 > 64.f * n1 * n3) : (m1 > 8.f * n1);
    }
}

// Serial tail of the schedule (one thread): the active experts in ascending order with the prefix sums of their
// token blocks and of the blocks' costs. tb[i] = token blocks of expert i if it is active, else 0.
__device__ __forceinline__ void write_schedule(Sched* sched, const int* tb, const int* count, int Etot,
                                               int min_up, int min_down) {
    int n = 0, au = 0, ad = 0, wu = 0, wd = 0;
    sched->tc_min[0] = min_up; sched->tc_min[1] = min_down;
    for (int i = 0; i < Etot; ++i) {
        const int b = tb[i];
        if (b > 0) {
            sched->act_expert[n] = i;
            sched->tb_prefix[0][n] = au; sched->tb_prefix[1][n] = ad;
            sched->w_prefix[0][n] = wu; sched->w_prefix[1][n] = wd;
            const int last = (count[i] - (b - 1) * kTokBlock + 7) >> 3;          // n-tiles of the last block, 1..4
            if (count[i] < min_up) { wu += (b - 1) * block_cost(0, 4) + block_cost(0, last); au += b; }      // streaming up/gate
            if (count[i] < min_down) { wd += (b - 1) * block_cost(1, 4) + block_cost(1, last); ad += b; }    // streaming down
            ++n;
        }
    }
    sched->tb_prefix[0][n] = au; sched->tb_prefix[1][n] = ad;
    sched->w_prefix[0][n] = wu; sched->w_prefix[1][n] = wd;
    sched->n_active = n;
    sched->total_tb[0] = au; sched->total_tb[1] = ad;
}

// The same schedule written by kMaxExperts threads (thread e = expert e; b = its token blocks, 0 if it does not run):
// five exclusive prefix sums over the experts (rank among the active ones, token blocks and costs of the two streaming
// kernels), then every active expert writes its own entries. One loop body serves the five sums (the values wait in
// shared memory), because this code runs once per step and is fetched cold: with 64 experts the serial loop took 3.7
// us at the very end of the routing kernel, on the critical path of the step.
// s_tmp: kSchedScratch ints; the calling threads (exactly kMaxExperts) meet at named barrier 1.
constexpr int kSerialScheduleMax = 16;
constexpr int kSchedScratch = 5 * kMaxExperts + 5 * (kMaxExperts / 32);
__device__ __forceinline__ void write_schedule_parallel(Sched* sched, int b, int cnt, int min_up, int min_down, int* s_tmp) {
    const int e = threadIdx.x, lane = e & 31, warp = e >> 5;
    constexpr int kW = kMaxExperts / 32;
    int* s_v = s_tmp;                        // [5][kMaxExperts]: values, then their exclusive prefixes
    int* s_w = s_tmp + 5 * kMaxExperts;      // [5][kW]: totals of the warps
    {
        const int last = b > 0 ? (cnt - (b - 1) * kTokBlock + 7) >> 3 : 1;            // n-tiles of the last block, 1..4
        const bool up = b > 0 && cnt < min_up, dn = b > 0 && cnt < min_down;          // taken by the streaming kernel of that projection
        s_v[e] = b > 0 ? 1 : 0;
        s_v[kMaxExperts + e] = up ? b : 0;
        s_v[2 * kMaxExperts + e] = dn ? b : 0;
        s_v[3 * kMaxExperts + e] = up ? (b - 1) * block_cost(0, 4) + block_cost(0, last) : 0;
        s_v[4 * kMaxExperts + e] = dn ? (b - 1) * block_cost(1, 4) + block_cost(1, last) : 0;
    }
#pragma unroll 1
    for (int q = 0; q < 5; ++q) {
        const int x = s_v[q * kMaxExperts + e];
        int incl = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
        if (lane == 31) s_w[q * kW + warp] = incl;
        s_v[q * kMaxExperts + e] = incl - x;          // exclusive within the warp
    }
    asm volatile("bar.sync 1, %0;\n" ::"n"(kMaxExperts) : "memory");
    int before[5];
#pragma unroll
    for (int q = 0; q < 5; ++q) before[q] = 0;
#pragma unroll 1
    for (int w = 0; w < warp; ++w) {
#pragma unroll
        for (int q = 0; q < 5; ++q) before[q] += s_w[q * kW + w];
    }
    if (e == 0) { sched->tc_min[0] = min_up; sched->tc_min[1] = min_down; }
    if (b > 0 || e == kMaxExperts - 1) {
        // the last thread also writes the closing entry (its own exclusive prefix + its own value = the totals)
        const int n = s_v[e] + before[0];
        const int au = s_v[kMaxExperts + e] + before[1], ad = s_v[2 * kMaxExperts + e] + before[2];
        const int wu = s_v[3 * kMaxExperts + e] + before[3], wd = s_v[4 * kMaxExperts + e] + before[4];
        if (b > 0) {
            sched->act_expert[n] = e;
            sched->tb_prefix[0][n] = au; sched->tb_prefix[1][n] = ad;
            sched->w_prefix[0][n] = wu; sched->w_prefix[1][n] = wd;
        }
        if (e == kMaxExperts - 1) {
            // totals = this thread's exclusive prefixes plus its own values (recomputed: cheap, and only here)
            const int last = b > 0 ? (cnt - (b - 1) * kTokBlock + 7) >> 3 : 1;
            const bool up = b > 0 && cnt < min_up, dn = b > 0 && cnt < min_down;
            const int nt = n + (b > 0 ? 1 : 0), tu = au + (up ? b : 0), td = ad + (dn ? b : 0);
            const int cu = wu + (up ? (b - 1) * block_cost(0, 4) + block_cost(0, last) : 0);
            const int cd = wd + (dn ? (b - 1) * block_cost(1, 4) + block_cost(1, last) : 0);
            sched->tb_prefix[0][nt] = tu; sched->tb_prefix[1][nt] = td;
            sched->w_prefix[0][nt] = cu; sched->w_prefix[1][nt] = cd;
            sched->n_active = nt;
            sched->total_tb[0] = tu; sched->total_tb[1] = td;
        }
    }
}

// Called by every thread of a CTA of at least kMaxExperts threads. Thread e looks at expert e; a warp covers one word
// of the masks, so the experts that run and the misses are collected with a ballot and cost one atomic per word
// (not one per expert on the same word).
__device__ __forceinline__ void schedule_body(const SchedArgs& S, const int* count, int Etot, int* s_tb, int* s_act) {
    const int e = threadIdx.x;
    if (e < kMaxExperts) {
        int tb = 0, act = 0, miss = 0;
        if (e < Etot) {
            const int c = count[e];
            const bool sel = (S.mask.w[e >> 5] >> (e & 31)) & 1u;
            if (c > 0 && sel) {
                if (S.slot_map[e] >= 0) { act = 1; tb = (c + kTokBlock - 1) / kTokBlock; }
                else miss = 1;
            }
        }
        s_tb[e] = tb; s_act[e] = act;
        const unsigned done_w = __ballot_sync(0xffffffffu, act), miss_w = __ballot_sync(0xffffffffu, miss);
        if ((e & 31) == 0) {
            if (done_w) atomicOr(S.done_mask + (e >> 5), done_w);
            if (miss_w && !S.quiet) { atomicOr(S.miss_mask + (e >> 5), miss_w); atomicOr(S.status, 1); }
        }
    }
    __syncthreads();
    if (Etot <= kSerialScheduleMax) {        // few experts: one thread is as fast as the scans (8 experts: 0.5 us)
        if (threadIdx.x == 0) write_schedule(S.sched, s_tb, count, Etot, S.tc_min[0], S.tc_min[1]);    // s_tb is 0 for inactive experts
        return;
    }
    if (threadIdx.x >= kMaxExperts) return;
    write_schedule_parallel(S.sched, s_tb[e], e < Etot ? count[e] : 0, S.tc_min[0], S.tc_min[1], s_act);
}

// S3 for large batches, one CTA; with do_sched also the work schedule of a call that runs every routed expert.
__global__ void __launch_bounds__(1024) k_group(GroupArgs G, SchedArgs S, int do_sched) {
    __shared__ int s_count[kMaxExperts];
    __shared__ int s_off[kMaxExperts + 1];
    __shared__ int s_hist[kGroupScratch];
    pdl_wait();            // the score kernel's selections
    pdl_launch();
    if ((int)blockIdx.x >= S.n_main) { expert_stats(S, blockIdx.x - S.n_main); return; }
    group_body<false>(G, s_count, s_off, s_hist);
    if (do_sched) {
        __syncthreads();
        schedule_body(S, s_count, G.E + G.ns, s_off, s_hist);      // s_off and s_hist are free now
    }
}

__global__ void __launch_bounds__(256) k_schedule(const int32_t* __restrict__ count, int Etot, SchedArgs S) {
    __shared__ int s_tb[kMaxExperts];
    __shared__ int s_act[kSchedScratch];
    pdl_wait();            // the kernels of the wave before still read the schedule this one rewrites
    pdl_launch();
    if ((int)blockIdx.x >= S.n_main) { expert_stats(S, blockIdx.x - S.n_main); return; }
    schedule_body(S, count, Etot, s_tb, s_act);
}

// Fused S1-S3 for small batches: one CTA per token does the scores, the fp16 copy and the top-k; the
// last CTA to finish (atomic ticket, no waiting) does the grouping and, if asked, the schedule.
// Dynamic shared memory of k_route_token: the token row (2 C bytes), reused by the last CTA for the per-warp
// histograms of the grouping step and as scratch of the schedule.
constexpr int kTokenSmemBytes = 4096;
inline size_t token_smem(int C, int n_warps, int E) {
    size_t need = (size_t)C * 2;                                                  // the token row
    need = std::max(need, (size_t)n_warps * (size_t)E * 4);                       // the grouping CTA's histograms
    need = std::max(need, (size_t)kSchedScratch * 4);                             // the schedule's scratch
    return std::max(need, (size_t)kTokenSmemBytes);
}

struct TokenArgs {
    const __nv_bfloat16* x; int T, C; const __nv_bfloat16* W; const float* bias; int E;
    float* scores; __half* x16; float* xscale; float* xnorm; float* xsum; int k; int32_t* idx; float* wts;
    unsigned* ticket; int do_sched;
};

template <bool FEW, int THREADS>
__global__ void __launch_bounds__(THREADS) k_route_token(TokenArgs A, GroupArgs G, SchedArgs S) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint4* xs = reinterpret_cast<uint4*>(smem);                        // [C/8]
    __shared__ float s_red[3][32];
    __shared__ float s_sc[kMaxExperts];
    __shared__ int s_count[kMaxExperts];
    __shared__ int s_off[kMaxExperts + 1];
    __shared__ int s_last;
    const int t = blockIdx.x, C = A.C, E = A.E, c8 = C / 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;    // 8 or 32 warps
    if (t >= S.n_main) {       // statistics CTAs: one per expert, beside the token CTAs; they take no ticket
        pdl_wait();            // the previous step's kernels still read the table this CTA rewrites
        pdl_launch();
        expert_stats(S, t - S.n_main);
        return;
    }
    prefetch_rows_l2(A.W, C * 2, warp, nwarps, E, lane);     // the router is constant: ask for it under the previous kernel's tail
    pdl_wait();            // the previous step's kernels still read the buffers this kernel rewrites
    pdl_launch();
    const uint4* xg = reinterpret_cast<const uint4*>(A.x) + (size_t)t * c8;
    float m = 0.f;
    for (int i = threadIdx.x; i < c8; i += blockDim.x) {
        const uint4 v = xg[i];
        xs[i] = v;
        const unsigned w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) m = fmaxf(m, fmaxf(fabsf(bf16lo(w4[j])), fabsf(bf16hi(w4[j]))));
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) s_red[0][warp] = m;
    __syncthreads();
    m = s_red[0][0];
    for (int i = 1; i < nwarps; ++i) m = fmaxf(m, s_red[0][i]);
    int ex = expo_of(m);
    ex = (m > 0.f) ? max(-100, min(127, ex)) : 13;
    const float sc_up = __uint_as_float((unsigned)(127 + 13 - ex) << 23);   // row maximum -> [2^13, 2^14)
    const float sc_dn = __uint_as_float((unsigned)(127 - 13 + ex) << 23);
    float ss = 0.f, sm = 0.f;
    uint4* og = reinterpret_cast<uint4*>(A.x16) + (size_t)t * c8;
    for (int i = threadIdx.x; i < c8; i += blockDim.x) {
        const uint4 v = xs[i];
        const unsigned w4[4] = {v.x, v.y, v.z, v.w};
        unsigned o4[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float a = bf16lo(w4[j]) * sc_up, b = bf16hi(w4[j]) * sc_up;
            ss = fmaf(a, a, ss); ss = fmaf(b, b, ss);
            const __half2 h = __floats2half2_rn(a, b);
            const float2 hf = __half22float2(h);
            sm += hf.x; sm += hf.y;
            o4[j] = *reinterpret_cast<const unsigned*>(&h);
        }
        og[i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        ss += __shfl_xor_sync(0xffffffffu, ss, o);
        sm += __shfl_xor_sync(0xffffffffu, sm, o);
    }
    if (lane == 0) { s_red[1][warp] = ss; s_red[2][warp] = sm; }
    // scores: warp w takes experts w, w + nwarps, ...
    const uint4* wg = reinterpret_cast<const uint4*>(A.W);
    for (int e = warp; e < E; e += nwarps) {
        float acc = 0.f;
        if (THREADS <= 256) {                // few experts, registers to spare: all loads of a 4096-wide row in flight at once
            for (int i0 = 0; i0 < c8; i0 += 32 * 16) {
                uint4 wv[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int i = i0 + lane + 32 * j;
                    wv[j] = i < c8 ? __ldg(wg + (size_t)e * c8 + i) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int i = i0 + lane + 32 * j;
                    if (i < c8) acc = dot8(wv[j], xs[i], acc);
                }
            }
        } else {
#pragma unroll 8
            for (int i = lane; i < c8; i += 32) acc = dot8(__ldg(wg + (size_t)e * c8 + i), xs[i], acc);
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) s_sc[e] = acc + (A.bias ? A.bias[e] : 0.f);
    }
    __syncthreads();
    if (threadIdx.x == 32) {                 // warp 1: warp 0 has the top-k to do
        float a = 0.f, b = 0.f;
        for (int i = 0; i < nwarps; ++i) { a += s_red[1][i]; b += s_red[2][i]; }
        A.xscale[t] = sc_dn; A.xnorm[t] = sqrtf(a) * sc_dn; A.xsum[t] = b;
    }
    if (A.scores != nullptr)
        for (int i = threadIdx.x; i < E; i += blockDim.x) A.scores[(size_t)t * E + i] = s_sc[i];
    if (warp == 0) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (lane + 32 * i < E) ? s_sc[lane + 32 * i] : -INFINITY;
        int oi[kMaxTopK]; float ov[kMaxTopK];
        warp_topk(v, E, A.k, lane, oi, ov);
        if (lane == 0) {
            float z = 0.f, p[kMaxTopK];
            for (int j = 0; j < A.k; ++j) { p[j] = expf(ov[j] - ov[0]); z += p[j]; }
            for (int j = 0; j < A.k; ++j) {
                A.idx[(size_t)t * A.k + j] = oi[j];
                A.wts[(size_t)t * A.k + j] = p[j] / z;
            }
        }
    }
    // ticket: the CTA that takes the last ticket sees every other CTA's idx (fence before the atomic)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(A.ticket, 1u) == (unsigned)S.n_main - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    group_body<FEW>(G, s_count, s_off, reinterpret_cast<int*>(xs));     // the token row is no longer needed
    if (A.do_sched) {
        __syncthreads();
        schedule_body(S, s_count, E + G.ns, s_off, reinterpret_cast<int*>(xs));   // s_off and xs are free now
    }
    if (threadIdx.x == 0) *A.ticket = 0u;
}

// Fused S1-S3 (+ schedule) for decode-sized batches in ONE CTA: no ticket, no fences, no atomics on the
// common path. Requires T * C * 2 bytes of shared memory for the token rows (T <= kSingleCtaMaxTokens).
constexpr int kSingleCtaMaxTokens = 4;      // beyond, one CTA per token is faster (8 tokens x 8 experts: 23 against 18 us)
constexpr int kSingleCtaThreads = 512;

__global__ void __launch_bounds__(kSingleCtaThreads) k_route_small(TokenArgs A, GroupArgs G, SchedArgs S) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint4* xs = reinterpret_cast<uint4*>(smem);                        // [T][C/8]
    __shared__ float s_sc[kSingleCtaMaxTokens][kMaxExperts];
    __shared__ int s_idx[kSingleCtaMaxTokens][kMaxTopK];
    __shared__ int s_rank[kSingleCtaMaxTokens][kMaxTopK];
    __shared__ int s_count[kMaxExperts];
    __shared__ int s_off[kMaxExperts + 1];
    __shared__ int s_tb[kMaxExperts];
    __shared__ int s_slot[kMaxExperts];
    const int T = A.T, C = A.C, E = A.E, k = A.k, c8 = C / 8, ns = G.ns, Etot = E + ns, kk = k + ns;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = kSingleCtaThreads / 32;
    if ((int)blockIdx.x >= S.n_main) {       // statistics CTAs: one per expert, beside the routing CTA
        pdl_wait();
        pdl_launch();
        expert_stats(S, blockIdx.x - S.n_main);
        return;
    }
    prefetch_rows_l2(A.W, C * 2, warp, nwarps, E, lane);     // the router is constant: ask for it under the previous kernel's tail
    pdl_wait();            // the previous step's kernels still read the buffers this kernel rewrites
    pdl_launch();
    // Every load that does not depend on another is issued before the first barrier, so a cold L2 costs
    // one DRAM round trip, not one per step: token rows, residency of every expert, bias, and the
    // first batch of this warp's router rows.
    const uint4* xg = reinterpret_cast<const uint4*>(A.x);
    for (int i = threadIdx.x; i < T * c8; i += kSingleCtaThreads) xs[i] = xg[i];
    if (A.do_sched) for (int e = threadIdx.x; e < Etot; e += kSingleCtaThreads) s_slot[e] = S.slot_map[e];
    const uint4* wg = reinterpret_cast<const uint4*>(A.W);
    constexpr int kWB = 16;                                  // router chunks per lane held in registers
    uint4 wpre[kWB];
    {
        const int e = warp;                                  // first expert of this warp
#pragma unroll
        for (int j = 0; j < kWB; ++j) {
            const int i = lane + 32 * j;
            wpre[j] = (e < E && i < c8) ? __ldg(wg + (size_t)e * c8 + i) : make_uint4(0, 0, 0, 0);
        }
    }
    const float bpre = (A.bias && warp < E) ? A.bias[warp] : 0.f;
    __syncthreads();
    // per token (one warp each, from the last warp down: the first warps have a router row to score): power-of-two
    // fp16 scale, norm, sum, fp16 copy
    for (int t = nwarps - 1 - warp; t < T; t += nwarps) {
        float m = 0.f;
        for (int i = lane; i < c8; i += 32) {
            const uint4 v = xs[t * c8 + i];
            const unsigned w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) m = fmaxf(m, fmaxf(fabsf(bf16lo(w4[j])), fabsf(bf16hi(w4[j]))));
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        int ex = expo_of(m);
        ex = (m > 0.f) ? max(-100, min(127, ex)) : 13;
        const float sc_up = __uint_as_float((unsigned)(127 + 13 - ex) << 23);
        const float sc_dn = __uint_as_float((unsigned)(127 - 13 + ex) << 23);
        float ss = 0.f, sm = 0.f;
        uint4* og = reinterpret_cast<uint4*>(A.x16) + (size_t)t * c8;
        for (int i = lane; i < c8; i += 32) {
            const uint4 v = xs[t * c8 + i];
            const unsigned w4[4] = {v.x, v.y, v.z, v.w};
            unsigned o4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float a = bf16lo(w4[j]) * sc_up, b = bf16hi(w4[j]) * sc_up;
                ss = fmaf(a, a, ss); ss = fmaf(b, b, ss);
                const __half2 h = __floats2half2_rn(a, b);
                const float2 hf = __half22float2(h);
                sm += hf.x; sm += hf.y;
                o4[j] = *reinterpret_cast<const unsigned*>(&h);
            }
            og[i] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            ss += __shfl_xor_sync(0xffffffffu, ss, o);
            sm += __shfl_xor_sync(0xffffffffu, sm, o);
        }
        if (lane == 0) { A.xscale[t] = sc_dn; A.xnorm[t] = sqrtf(ss) * sc_dn; A.xsum[t] = sm; }
    }
    // scores: warp w takes experts w, w + nwarps, ...; one pass over the expert's row serves all tokens
    for (int e = warp; e < E; e += nwarps) {
        float acc[kSingleCtaMaxTokens];
#pragma unroll
        for (int t = 0; t < kSingleCtaMaxTokens; ++t) acc[t] = 0.f;
        for (int i0 = 0; i0 < c8; i0 += 32 * kWB) {
            if (e != warp || i0 != 0) {                      // later batches: load now (the first one is in registers)
#pragma unroll
                for (int j = 0; j < kWB; ++j) {
                    const int i = i0 + lane + 32 * j;
                    wpre[j] = (i < c8) ? __ldg(wg + (size_t)e * c8 + i) : make_uint4(0, 0, 0, 0);
                }
            }
            for (int t = 0; t < T; ++t) {
                float a = acc[0];                            // rotate so that acc[t] is addressed statically
#pragma unroll
                for (int q = 0; q < kSingleCtaMaxTokens; ++q) if (q == t) a = acc[q];
#pragma unroll
                for (int j = 0; j < kWB; ++j) {
                    const int i = i0 + lane + 32 * j;
                    if (i < c8) a = dot8(wpre[j], xs[t * c8 + i], a);
                }
#pragma unroll
                for (int q = 0; q < kSingleCtaMaxTokens; ++q) if (q == t) acc[q] = a;
            }
        }
        const float bv = (e == warp) ? bpre : (A.bias ? A.bias[e] : 0.f);
#pragma unroll
        for (int t = 0; t < kSingleCtaMaxTokens; ++t) {
            if (t < T) {
#pragma unroll
                for (int o = 16; o; o >>= 1) acc[t] += __shfl_xor_sync(0xffffffffu, acc[t], o);
                if (lane == 0) s_sc[t][e] = acc[t] + bv;
            }
        }
    }
    __syncthreads();
    if (A.scores != nullptr)
        for (int i = threadIdx.x; i < T * E; i += kSingleCtaThreads) A.scores[i] = s_sc[i / E][i % E];
    for (int t = warp; t < T; t += nwarps) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (lane + 32 * i < E) ? s_sc[t][lane + 32 * i] : -INFINITY;
        int oi; float ov;
        warp_topk_lanes(v, E, k, lane, oi, ov);
        const float wj = topk_softmax(ov, k, lane);
        if (lane < k) {
            s_idx[t][lane] = oi;
            A.idx[(size_t)t * k + lane] = oi;
            A.wts[(size_t)t * k + lane] = wj;
        }
    }
    __syncthreads();
    // grouping from shared memory (T <= 8: one ballot per expert)
    for (int e = warp; e < E; e += nwarps) {
        int jsel = -1;
        if (lane < T)
            for (int j = 0; j < k; ++j) if (s_idx[lane][j] == e) { jsel = j; break; }
        const unsigned m = __ballot_sync(0xffffffffu, jsel >= 0);
        if (jsel >= 0) s_rank[lane][jsel] = __popc(m & ((1u << lane) - 1u));
        if (lane == 0) s_count[e] = __popc(m);
    }
    for (int s = threadIdx.x; s < ns; s += kSingleCtaThreads) s_count[E + s] = T;
    __syncthreads();
    if (threadIdx.x == 0) {
        int a = 0;
        for (int e = 0; e < Etot; ++e) { s_off[e] = a; a += s_count[e]; }
        s_off[Etot] = a;
    }
    __syncthreads();
    notify_host(G, s_count, Etot);
    for (int e = threadIdx.x; e <= Etot; e += kSingleCtaThreads) {
        G.offset[e] = s_off[e];
        if (e < Etot) G.count[e] = s_count[e];
    }
    for (int p = threadIdx.x; p < T * kk; p += kSingleCtaThreads) {
        const int t = p / kk, j = p % kk;
        const int pos = (j < k) ? s_off[s_idx[t][j]] + s_rank[t][j] : s_off[E + (j - k)] + t;
        G.perm[p] = pos;
        G.row_token[pos] = t;
    }
    if (!A.do_sched) {
        if (threadIdx.x < 8) G.done_mask[threadIdx.x] = 0u;
        return;
    }
    // schedule over all experts: resident ones run, missing ones are flagged
    if (threadIdx.x < kMaxExperts) {
        const int e = threadIdx.x;
        const bool need = e < Etot && s_count[e] > 0;
        const bool res = need && s_slot[e] >= 0;
        s_tb[e] = res ? (s_count[e] + kTokBlock - 1) / kTokBlock : 0;
        const unsigned done = __ballot_sync(0xffffffffu, res), miss = __ballot_sync(0xffffffffu, need && !res);
        if (lane == 0) {
            S.done_mask[e >> 5] = done;
            if (miss && !S.quiet) { atomicOr(S.miss_mask + (e >> 5), miss); atomicOr(S.status, 1); }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) write_schedule(S.sched, s_tb, s_count, Etot, S.tc_min[0], S.tc_min[1]);
}

// S7 pooling: pooled[e] = mean_t score[t][e]; then the k_pred best pooled scores.
__global__ void __launch_bounds__(1024)
k_pool(const float* __restrict__ ts, int T, int E, float* __restrict__ pooled, int32_t* __restrict__ ids, int k_pred,
       int32_t* host_ids = nullptr, volatile uint32_t* host_flag = nullptr, uint32_t host_seq = 0) {
    __shared__ float s_pool[kMaxExperts];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int e = warp; e < E; e += 32) {
        float a = 0.f;
        for (int t = lane; t < T; t += 32) a += ts[(size_t)t * E + e];
#pragma unroll
        for (int o = 16; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) { a = a / (float)T; s_pool[e] = a; pooled[e] = a; }
    }
    __syncthreads();
    if (warp == 0 && ids != nullptr) {
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (lane + 32 * i < E) ? s_pool[lane + 32 * i] : -INFINITY;
        int oi[kMaxTopK]; float ov[kMaxTopK];
        warp_topk(v, E, k_pred, lane, oi, ov);
        if (lane == 0) {
            for (int j = 0; j < k_pred; ++j) ids[j] = oi[j];
            if (host_ids != nullptr) {             // optional notification of a waiting host thread, as in the grouping kernel
                for (int j = 0; j < k_pred; ++j) host_ids[j] = oi[j];
                __threadfence_system();
                *host_flag = host_seq;
            }
        }
    }
}

// S1 + S2 for batches too large for one CTA per token, as a 2-D grid: blockIdx.x = a group of kWideTok tokens,
// blockIdx.y = a group of kWideExp experts (one warp each). Every CTA stages its tokens once, every warp reads its
// expert's router row once (all its loads in flight) and scores all the group's tokens. The logits go to global
// memory; the CTA that finishes a token group last (a ticket per token group) does the top-k of its tokens from
// there. Same arithmetic, in the same order, as k_scores: the logits, and with them the selection, are identical.
constexpr int kWideTok = 8, kWideExp = 8, kWideThreads = 32 * kWideExp;
size_t wide_scores_smem(int C) { return (size_t)kWideTok * C * 2; }
constexpr size_t kWideSmemMax = 160 * 1024;

__global__ void __launch_bounds__(kWideThreads)
k_scores_wide(const __nv_bfloat16* __restrict__ x, int T, int C, const __nv_bfloat16* __restrict__ W,
              const float* __restrict__ bias, int E, float* __restrict__ scores, __half* __restrict__ x16,
              float* __restrict__ xscale, float* __restrict__ xnorm, float* __restrict__ xsum, int k,
              int32_t* __restrict__ idx, float* __restrict__ wts, unsigned* __restrict__ tickets) {
    extern __shared__ __align__(16) unsigned char smem[];
    uint4* xs = reinterpret_cast<uint4*>(smem);                       // [kWideTok][C/8]
    __shared__ float s_scale[kWideTok];
    __shared__ int s_last;
    pdl_wait();            // the previous step's kernels still read the buffers this kernel rewrites
    pdl_launch();
    const int t0 = blockIdx.x * kWideTok;
    const int nt = min(kWideTok, T - t0);
    const int c8 = C / 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint4* xg = reinterpret_cast<const uint4*>(x) + (size_t)t0 * c8;
    for (int i = threadIdx.x; i < kWideTok * c8; i += kWideThreads)
        xs[i] = (i < nt * c8) ? xg[i] : make_uint4(0, 0, 0, 0);
    __syncthreads();

    // the fp16 copy of the tokens and its per-token numbers, once per token group
    if (x16 != nullptr && blockIdx.y == 0) write_fp16_copy(xs, c8, nt, t0, kWideThreads, s_scale, x16, xscale, xnorm, xsum);

    const int e = blockIdx.y * kWideExp + warp;
    if (e < E) {
        const uint4* wg = reinterpret_cast<const uint4*>(W) + (size_t)e * c8;
        float acc[kWideTok];
#pragma unroll
        for (int j = 0; j < kWideTok; ++j) acc[j] = 0.f;
#pragma unroll 8
        for (int i = lane; i < c8; i += 32) {
            const uint4 wv = __ldg(wg + i);
#pragma unroll
            for (int j = 0; j < kWideTok; ++j) acc[j] = dot8(wv, xs[j * c8 + i], acc[j]);
        }
#pragma unroll
        for (int j = 0; j < kWideTok; ++j) {
#pragma unroll
            for (int o = 16; o; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
        }
        if (lane == 0) {
            const float b = bias ? bias[e] : 0.f;
#pragma unroll
            for (int j = 0; j < kWideTok; ++j) if (j < nt) scores[(size_t)(t0 + j) * E + e] = acc[j] + b;
        }
    }
    if (idx == nullptr) return;
    // the last CTA of this token group sees every other CTA's logits (fence before the ticket)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool last = atomicAdd(tickets + blockIdx.x, 1u) == gridDim.y - 1;
        if (last) tickets[blockIdx.x] = 0u;
        s_last = last;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (warp < nt) {
        const float* row = scores + (size_t)(t0 + warp) * E;
        float v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = (lane + 32 * i < E) ? __ldcg(row + lane + 32 * i) : -INFINITY;
        int oi[kMaxTopK]; float ov[kMaxTopK];
        warp_topk(v, E, k, lane, oi, ov);
        if (lane == 0) {
            float z = 0.f, p[kMaxTopK];
            for (int j = 0; j < k; ++j) { p[j] = expf(ov[j] - ov[0]); z += p[j]; }
            for (int j = 0; j < k; ++j) {
                idx[(size_t)(t0 + warp) * k + j] = oi[j];
                wts[(size_t)(t0 + warp) * k + j] = p[j] / z;
            }
        }
    }
}

size_t scores_smem(int C, int E) { return (size_t)kScoreTok * C * 2 + (size_t)kScoreTok * E * 4; }

}  // namespace

mira_status launch_scores(mira_ctx* ctx, const void* x, int T, const void* w, const float* b, int E,
                          float* scores, __half* x16, float* xscale, float* xnorm, cudaStream_t st) {
    // plain scores (predictor): no top-k
    const int C = ctx->cfg.hidden;
    ProfScope ps(ctx, MIRA_K_SCORES, st);
    const int n_tok_ctas = (T + kScoreTok - 1) / kScoreTok;
    int ysplit = 1;                                      // experts over several CTAs while the grid is below two waves
    if (x16 == nullptr && scores != nullptr)
        ysplit = std::max(1, std::min((E + kScoreThreads / 32 - 1) / (kScoreThreads / 32), 2 * ctx->n_sm / n_tok_ctas));
    k_scores<<<dim3(n_tok_ctas, ysplit), kScoreThreads, scores_smem(C, E), st>>>(
        (const __nv_bfloat16*)x, T, C, (const __nv_bfloat16*)w, b, E, scores, x16, xscale, xnorm, nullptr, 0, nullptr, nullptr);
    ctx->launches += 1;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

namespace {
GroupArgs group_args(mira_ctx* ctx, int T, int k, const RouteView& rv) {
    GroupArgs G;
    G.idx = rv.idx; G.T = T; G.k = k; G.E = ctx->cfg.n_experts; G.ns = ctx->cfg.n_shared;
    G.count = rv.count; G.offset = rv.offset; G.perm = rv.perm; G.row_token = rv.row_token;
    G.done_mask = ws_ptr<uint32_t>(ctx, ctx->lay.status) + 16 + 8;
    G.host_count = ctx->notify_count; G.host_flag = ctx->notify_flag; G.host_seq = ctx->notify_seq;
    return G;
}
SchedArgs sched_args(mira_ctx* ctx, void* const* slots, const int32_t* slot_map, const uint32_t* host_mask, int T, int k, int n_main,
                     bool quiet = false) {
    SchedArgs S;
    S.quiet = quiet ? 1 : 0;
    S.slots = slots; S.hexp = ws_ptr<int32_t>(ctx, ctx->lay.hexp);
    S.T = T; S.R = ctx->cfg.ffn; S.C = ctx->cfg.hidden; S.per_matrix = ctx->cfg.format == MIRA_FORMAT_PER_MATRIX; S.n_main = n_main;
    step_tc_min(ctx, T, k, S.tc_min);
    const int Etot = Et(ctx->cfg);
    for (int i = 0; i < 8; ++i) S.mask.w[i] = (host_mask == nullptr) ? 0xffffffffu : (i < (Etot + 31) / 32 ? host_mask[i] : 0u);
    S.slot_map = slot_map;
    S.sched = ws_ptr<Sched>(ctx, ctx->lay.sched);
    S.status = ws_ptr<int32_t>(ctx, ctx->lay.status);
    S.miss_mask = reinterpret_cast<uint32_t*>(S.status) + 16;
    S.done_mask = S.miss_mask + 8;
    return S;
}
}  // namespace

// S1-S3. If slot_map is given and the batch is small, the schedule of a run over ALL experts is
// produced by the same launch (*fused_schedule = 1) and the caller must not launch it again.
mira_status launch_route(mira_ctx* ctx, const void* x, int T, const void* w, const float* b, int k,
                         const RouteView& rv, __half* x16, float* xscale, float* xnorm, void* const* slots,
                         const int32_t* slot_map, int* fused_schedule, cudaStream_t st, bool quiet_schedule) {
    const int C = ctx->cfg.hidden, E = ctx->cfg.n_experts;
    const int n_stat = (slots != nullptr && slot_map != nullptr) ? Et(ctx->cfg) : 0;      // statistics CTAs, one per expert
    if (fused_schedule) *fused_schedule = 0;
    GroupArgs G = group_args(ctx, T, k, rv);
    if (T <= (E > 16 ? kFusedRouteMaxTokens : kFusedRouteMaxTokensFewExperts)) {
        // one CTA for everything only while its T * E dot products stay cheap for a single SM
        const bool single = T <= kSingleCtaMaxTokens && E <= 16 && (size_t)T * C * 2 <= 96 * 1024;
        TokenArgs A;
        A.x = (const __nv_bfloat16*)x; A.T = T; A.C = C; A.W = (const __nv_bfloat16*)w; A.bias = b; A.E = E;
        A.scores = rv.logits; A.x16 = x16; A.xscale = xscale; A.xnorm = xnorm; A.xsum = ws_ptr<float>(ctx, ctx->lay.xsum);
        A.k = k; A.idx = rv.idx; A.wts = rv.w;
        A.ticket = ws_ptr<unsigned>(ctx, ctx->lay.status) + 8;
        A.do_sched = slot_map != nullptr;
        SchedArgs S = sched_args(ctx, slots, slot_map, nullptr, T, k, single ? 1 : T, quiet_schedule);
        ProfScope ps(ctx, MIRA_K_ROUTE, st);
        if (single) MIRA_CUDA_OK(launch_pdl(k_route_small, dim3(1 + n_stat), dim3(kSingleCtaThreads), (size_t)T * C * 2, st, A, G, S));
        else if (E > 16) {                   // a warp per expert and round
            if (T * k <= 64) MIRA_CUDA_OK(launch_pdl(k_route_token<true, 1024>, dim3(T + n_stat), dim3(1024), token_smem(C, 32, E), st, A, G, S));
            else MIRA_CUDA_OK(launch_pdl(k_route_token<false, 1024>, dim3(T + n_stat), dim3(1024), token_smem(C, 32, E), st, A, G, S));
        } else {
            if (T * k <= 64) MIRA_CUDA_OK(launch_pdl(k_route_token<true, 256>, dim3(T + n_stat), dim3(256), token_smem(C, 8, E), st, A, G, S));
            else MIRA_CUDA_OK(launch_pdl(k_route_token<false, 256>, dim3(T + n_stat), dim3(256), token_smem(C, 8, E), st, A, G, S));
        }
        ctx->launches += 1;
        if (fused_schedule) *fused_schedule = A.do_sched;
        MIRA_CUDA_OK(cudaGetLastError());
        return MIRA_OK;
    }
    {
        ProfScope ps(ctx, MIRA_K_ROUTE, st);
        if (E > kWideExp && wide_scores_smem(C) <= kWideSmemMax)      // several expert groups: the 2-D grid pays (27 against 39 us at 1024 tokens x 60 experts)
            MIRA_CUDA_OK(launch_pdl(k_scores_wide, dim3((T + kWideTok - 1) / kWideTok, (E + kWideExp - 1) / kWideExp), dim3(kWideThreads), wide_scores_smem(C), st,
                (const __nv_bfloat16*)x, T, C, (const __nv_bfloat16*)w, b, E, rv.logits, x16, xscale, xnorm,
                ws_ptr<float>(ctx, ctx->lay.xsum), k, rv.idx, rv.w, ws_ptr<unsigned>(ctx, ctx->lay.tickets)));
        else
            MIRA_CUDA_OK(launch_pdl(k_scores, dim3((T + kScoreTok - 1) / kScoreTok), dim3(kScoreThreads), scores_smem(C, E), st,
                (const __nv_bfloat16*)x, T, C, (const __nv_bfloat16*)w, b, E, rv.logits, x16, xscale, xnorm, ws_ptr<float>(ctx, ctx->lay.xsum), k, rv.idx, rv.w));
    }
    {
        // the schedule of a run over all experts comes out of the same launch
        const int do_sched = slot_map != nullptr;
        SchedArgs S = sched_args(ctx, slots, slot_map, nullptr, T, k, 1, quiet_schedule);
        ProfScope ps(ctx, MIRA_K_GROUP, st);
        MIRA_CUDA_OK(launch_pdl(k_group, dim3(1 + n_stat), dim3(1024), 0, st, G, S, do_sched));
        if (fused_schedule) *fused_schedule = do_sched;
    }
    ctx->launches += 2;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

mira_status launch_schedule(mira_ctx* ctx, int T, void* const* slots, const int32_t* slot_map, const uint32_t* host_mask,
                            int all_experts, cudaStream_t st) {
    SchedArgs S = sched_args(ctx, slots, slot_map, all_experts ? nullptr : host_mask, T, ctx->route_k, 1);
    ProfScope ps(ctx, MIRA_K_SCHEDULE, st);
    MIRA_CUDA_OK(launch_pdl(k_schedule, dim3(1 + (slots != nullptr ? Et(ctx->cfg) : 0)), dim3(256), 0, st,
                            (const int32_t*)ws_ptr<int32_t>(ctx, ctx->lay.count), Et(ctx->cfg), S));
    ctx->launches += 1;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

mira_status launch_pool(mira_ctx* ctx, const float* token_scores, int T, int E, float* pooled,
                        int32_t* ids, int k_pred, cudaStream_t st) {
    ProfScope ps(ctx, MIRA_K_POOL, st);
    k_pool<<<1, 1024, 0, st>>>(token_scores, T, E, pooled, ids, k_pred, ids ? ctx->notify_ids : nullptr, ctx->notify_ids_flag,
                               ctx->notify_seq);
    ctx->launches += 1;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

mira_status set_route_attributes() {
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_scores, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_scores_wide, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWideSmemMax));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_route_token<true, 1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_route_token<false, 1024>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_route_token<true, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_route_token<false, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_route_small, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024));
    return MIRA_OK;
}

}  // namespace mira

// ---------------------------------------------------------------------------------------------
// mira_predict_noalloc: the predictor head for callers that have no device allocator.
// ---------------------------------------------------------------------------------------------
namespace {

// Scratch for the per-token scores of mira_predict_noalloc. It is part of the library image: every
// GPU that loads libmira holds these 256 KB until the process exits, used or not.
static __device__ __align__(256) float g_noalloc_token_scores[MIRA_NOALLOC_MAX_SCORES];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
float* g_noalloc_scores_addr[kMaxDevices];   // device address of the array above, per device (nullptr: not set up)

// Once per device, with that device current: resolve the DEVICE address of the scratch array. In host
// code the name `g_noalloc_token_scores` is only a host-side handle of the symbol; handing it to a
// kernel would make the kernel touch the wrong memory.
mira_status noalloc_setup(int dev, float** scratch) {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_scores_addr[dev] == nullptr) {
        float* p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_token_scores) != cudaSuccess || p == nullptr)
            return MIRA_ERR_CUDA;
        if (cudaFuncSetAttribute(mira::k_scores, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
            return MIRA_ERR_CUDA;
        g_noalloc_scores_addr[dev] = p;
    }
    *scratch = g_noalloc_scores_addr[dev];
    return MIRA_OK;
}

}  // namespace

extern "C" mira_status mira_predict_noalloc(const void* hidden, int32_t T, int32_t hidden_size, const void* pred_w,
                                            const float* pred_b, int32_t n_experts, float* out_expert_scores,
                                            int32_t* out_topk_ids, int32_t k_pred, void* stream) {
    using namespace mira;
    if (!hidden || !pred_w || !out_expert_scores || T < 1 || hidden_size < 1 || n_experts < 1) return MIRA_ERR_INVALID_ARG;
    if (hidden_size % 8 || hidden_size > 16384 || n_experts > kMaxExperts) return MIRA_ERR_SHAPE;
    if ((long)T * n_experts > (long)MIRA_NOALLOC_MAX_SCORES) return MIRA_ERR_WORKSPACE;   // beyond the built-in scratch
    if (out_topk_ids && (k_pred < 1 || k_pred > kMaxTopK || k_pred > n_experts)) return MIRA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(hidden) | reinterpret_cast<uintptr_t>(pred_w)) & 15u) return MIRA_ERR_ALIGN;
    int dev = 0;
    MIRA_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return MIRA_ERR_UNSUPPORTED;
    float* scratch = nullptr;
    mira_status s = noalloc_setup(dev, &scratch);
    if (s != MIRA_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // every token score of this call is written before it is read, so nothing has to be cleared
    k_scores<<<(T + kScoreTok - 1) / kScoreTok, kScoreThreads, scores_smem(hidden_size, n_experts), st>>>(
        (const __nv_bfloat16*)hidden, T, hidden_size, (const __nv_bfloat16*)pred_w, pred_b, n_experts, scratch,
        nullptr, nullptr, nullptr, nullptr, 0, nullptr, nullptr);
    k_pool<<<1, 1024, 0, st>>>(scratch, T, n_experts, out_expert_scores, out_topk_ids, out_topk_ids ? k_pred : 0);
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

