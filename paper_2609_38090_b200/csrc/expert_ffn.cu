// S4-S6 for decode-sized groups: the expert FFN computed directly on the compressed expert
// ("fused dequantization + FFN", Section IV-A step 4 and Section IV-F), as two weight-streaming
// kernels plus the weighted combine (Section II-A).
//
// The shared scale s_r (Section IV-B) indexes the OUTPUT row of W1^/W3^ and the REDUCTION index of
// W2^, so no weight is ever multiplied by its scale one by one:
//     U_r = sum_c q1[r][c] x_c,  G_r = sum_c q3[r][c] x_c        (integer codes, exact in fp16)
//     h_r = silu(s_r G_r) * (s_r U_r)
//     y_c = sum_r q2[c][r] * (s_r h_r)
// The scale is applied three times per (token, row) in the epilogue of the up/gate kernel; the
// weight stream itself only needs the int8 -> fp16 conversion. The intermediate s_r h_r is stored
// in fp16 after multiplication by a per-(token, expert) power of two that puts its typical
// magnitude near 1; the down kernel undoes that power of two on its fp32 accumulators.
//
// Both kernels stream the int8 rows with cp.async, turn them into fp16 MMA fragments in registers
// (XOR 0x80, byte permute into the mantissa of 1024.0, subtract 1152: five ALU operations per four
// weights) and use mma.sync m16n8k16 with the weights as the M operand and up to 32 tokens of the
// expert as the N operand. The reduction index inside one MMA is permuted (the same way for both
// operands) so that a thread's 16 consecutive weight bytes feed four MMAs without any shuffle.
//
// Work is derived on the device from the schedule the grouping step wrote; the host never reads
// routing results.
#include <algorithm>
#include "mira_internal.cuh"

namespace mira {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kPairs = kWarps / 2;
// Ring depth: 3 stages when the activation tile is small (<= 8 tokens), else 2, so that two CTAs fit one SM.
__host__ __device__ constexpr int stages_for(int nt) { return nt == 1 ? 3 : 2; }
constexpr int kMT = 2;            // MMA m-tiles per unit

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma16816(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Four int8 codes (one 32-bit word, already XOR-ed with 0x80808080 so each byte is u = code + 128) -> two half2 of
// the signed codes, exactly: the byte goes into the mantissa of 1024.0 (0x6400 | u = 1024 + u) and 1152 = 1024 + 128
// is subtracted. Five ALU operations per four weights (one XOR, two byte permutes, two half2 subtractions).
// (Feeding u * 2^-24 as an fp16 subnormal and subtracting 128 * sum(x) afterwards saves the two subtractions, but
// the tensor cores add in fp32 with truncation, so the subtracted term costs accuracy as soon as a token's
// activations have a mean: measured 6e-3 instead of 1e-3 at hidden size 4096 with mean = spread. It also needs the
// token sums in the epilogue. Measured on the Mixtral shape the exact form is as fast at 1 and 8 tokens and 0.5 %
// slower at 32, so the streaming kernels always convert exactly; the tcgen05 up/gate kernel keeps the offset form
// as an option.)
__device__ __forceinline__ unsigned cvt_exact_lo(unsigned u) {
    unsigned v = __byte_perm(u, 0x64646464u, 0x4140);
    __half2 r = __hsub2(*reinterpret_cast<__half2*>(&v), __half2half2(__ushort_as_half(0x6480)));
    return *reinterpret_cast<unsigned*>(&r);
}
__device__ __forceinline__ unsigned cvt_exact_hi(unsigned u) {
    unsigned v = __byte_perm(u, 0x64646464u, 0x4342);
    __half2 r = __hsub2(*reinterpret_cast<__half2*>(&v), __half2half2(__ushort_as_half(0x6480)));
    return *reinterpret_cast<unsigned*>(&r);
}

// fp32 -> fp16, round to nearest even, values beyond the fp16 range go to +-65504 instead of infinity
__device__ __forceinline__ unsigned short f32_to_f16_sat(float v) {
    unsigned short h;
    asm("cvt.rn.satfinite.f16.f32 %0, %1;\n" : "=h"(h) : "f"(v));
    return h;
}
__device__ __forceinline__ float silu(float z) { return z / (1.f + __expf(-z)); }
__device__ __forceinline__ float pow2i(int e) { return __uint_as_float((unsigned)(max(-126, min(127, e)) + 127) << 23); }
__device__ __forceinline__ int expo(float v) { return (int)((__float_as_uint(v) >> 23) & 0xff) - 127; }

struct ItemTable {             // the schedule, copied to shared memory once per CTA
    int n_active, total_tb;
    int tb_prefix[kMaxExperts + 1];
    int w_prefix[kMaxExperts + 1];     // cost prefix of this kernel (up/gate or down)
    uint8_t act_expert[kMaxExperts];
};

__device__ __forceinline__ void load_table(ItemTable& tab, const Sched* __restrict__ sched, int which) {
    // the token blocks and costs of THIS projection's streaming work: an expert that the tensor-core kernel takes has
    // none, and the searches below skip such zero-length entries
    // (clamped: the up/gate kernel's rehearsal pass may read a schedule that is being rewritten, or was never written)
    if (threadIdx.x == 0) { tab.n_active = max(0, min(sched->n_active, kMaxExperts)); tab.total_tb = sched->total_tb[which]; }
    for (int i = threadIdx.x; i < kMaxExperts; i += blockDim.x) tab.act_expert[i] = (uint8_t)sched->act_expert[i];
    for (int i = threadIdx.x; i <= kMaxExperts; i += blockDim.x) {
        tab.tb_prefix[i] = sched->tb_prefix[which][i];
        tab.w_prefix[i] = sched->w_prefix[which][i];
    }
    __syncthreads();
}

// Units are weighted by the cost of their token block. Returns the first unit at or after cost position x, where
// x counts cost * units (0 <= x <= total cost * per_tb); monotonic in x, so consecutive CTAs get adjoining ranges.
// I: the integer type of unit numbers and cost positions. The launcher takes 32 bits whenever the largest cost
// position (cost * units * CTAs) fits: 64-bit divisions are long software routines, and this code runs cold at the
// start of every CTA, where instruction fetch from memory is what it costs.
template <typename I>
__device__ __forceinline__ I unit_at(const ItemTable& tab, I x, I per_tb, int w_full) {
    const int n = tab.n_active;
    if (x >= (I)tab.w_prefix[n] * per_tb) return (I)tab.total_tb * per_tb;
    const int xb = (int)(x / per_tb);
    int lo = 0, hi = n - 1;                                // largest a with w_prefix[a] <= xb
    while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (tab.w_prefix[mid] <= xb) lo = mid; else hi = mid - 1; }
    const I local = x - (I)tab.w_prefix[lo] * per_tb;
    const int ntb = tab.tb_prefix[lo + 1] - tab.tb_prefix[lo];
    const I full_block = (I)w_full * per_tb;
    const I full_span = (I)(ntb - 1) * full_block;
    I blk, in_blk;
    if (local < full_span) {
        blk = local / full_block;
        in_blk = (local - blk * full_block) / w_full;
    } else {
        const int w_last = tab.w_prefix[lo + 1] - tab.w_prefix[lo] - (ntb - 1) * w_full;
        blk = ntb - 1;
        in_blk = (local - full_span) / w_last;
    }
    return ((I)tab.tb_prefix[lo] + blk) * per_tb + in_blk;
}

struct FfnArgs {
    void* const* slots;
    const int32_t* slot_map;
    const Sched* sched;
    const int32_t* count;
    const int32_t* offset;
    const int32_t* row_token;
    const float* xscale;
    const float* xnorm;
    const int32_t* hexp;        // per expert: exponent of the intermediate's expected magnitude per unit of |x|^2
    float* hscale;
    const __half* x16;
    __half* h16;
    __half* h16lo;              // lower window of the intermediate, written and read for wide-range experts only
    float* ypart;
    int R, C, act_on_w1;
    int down_splits, down_slice;
    int per_matrix;             // blob format: 0 shared scale, 1 per-matrix scales (see BlobFmt)
    int n_all;                  // routed + shared experts
    long ypart_stride;          // elements between two splits = P * C
};

// ---------------------------------------------------------------------------------------------
// S4 (up + gate) and S5 (down) share one pipeline.
//
// Unit of work: 32 weight rows (two MMA m-tiles) x one block of <= 32 tokens of one expert, done by
// a PAIR of warps that split the reduction index between them and add their partial sums at the
// end of the unit (fixed order, so results are bit-repeatable).
//   S4: an m-tile holds 8 rows of W1^ in MMA rows 0-7 and the SAME 8 rows of W3^ in MMA rows 8-15, so
//       one thread ends up with U and G of the same (row, token) and the SwiGLU is thread-local;
//       a unit is 16 expert-hidden rows over the whole reduction (C).
//   S5: ordinary m-tiles of W2^; a unit is 32 model-hidden rows over one slice of the reduction (R);
//       partial sums of the slices go to ypart[slice].
// Units are numbered (expert, token block, [slice,] row group). Every CTA takes an equal contiguous
// range of units and walks it in steps of up to 4 units (one per warp pair) that belong to the same
// (expert, token block, slice), so the pairs of a step share one activation tile.
//
// Memory pipeline, per stage of 256 reduction elements:
//   weights     : each pair copies its 32 rows x 256 bytes with cp.async, two rows per instruction,
//                 so every request is 256 contiguous bytes of one row (64-byte pieces reach only
//                 ~75 % of HBM bandwidth on B200, 256-byte pieces reach all of it). The tile is
//                 XOR-swizzled so the MMA fragment reads are conflict free.
//   activations : the CTA copies the <= 32 token rows x 512 bytes (fp16) once for all its warps.
// ---------------------------------------------------------------------------------------------
constexpr int kSeg = 256;                           // reduction elements (= weight bytes per row) per stage
constexpr int kSegChunks = kSeg / kChunk;           // 4 MMA k-groups of 64 per stage, 2 per warp of a pair
constexpr int kATile = 32 * kSeg;                   // bytes of one pair's weight tile
constexpr int kBRow = kSeg * 2 + 16;                // bytes per activation row in shared memory (padded)
__host__ __device__ constexpr size_t ring_bytes(int nt) {
    return (size_t)stages_for(nt) * (kPairs * kATile + nt * 8 * kBRow);
}
// After the ring comes the exchange area of the pair reduction, 4 slots (one per pair) of 512 NT bytes.
__host__ __device__ constexpr size_t step_smem(int nt) { return ring_bytes(nt) + (size_t)kPairs * 512 * nt; }
constexpr size_t kSmemBytes = step_smem(1) > step_smem(4) ? step_smem(1) : step_smem(4);
static_assert(step_smem(2) <= kSmemBytes && step_smem(3) <= kSmemBytes, "ring geometry");
static_assert(kSmemBytes + sizeof(ItemTable) + 1024 <= 116736, "two CTAs per SM (228 KB, 1 KB reserved per CTA)");

__device__ __forceinline__ void lds128(unsigned (&v)[4], unsigned saddr) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(saddr));
}
__device__ __forceinline__ void cp_async16_s(unsigned saddr, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(saddr), "l"(gmem_src) : "memory");
}
// One step of a CTA: up to kPairs units of the same (expert, token block, slice).
struct StepDesc {
    const unsigned char* blob;
    int row0, k0, klen, split, pos0, ntok, nt, nstep, hexp;
    bool active, valid;
    bool wide;          // wide-range expert: the intermediate has a second, lower fp16 window (h16lo)
    bool last_half;     // S5 of a wide-range expert takes a 32-token block as two halves of 16 (see k_ffn)
};

// Per-thread state of the copies of one step (geometry follows the step's NT).
struct CopyState {
    const unsigned char* w0;       // S4: W1^ rows; S5: W2^ rows 0-7 of this warp's half tile
    const unsigned char* w1;       // S4: W3^ rows; S5: W2^ rows 8-15
    const unsigned char* b;        // activation row of this thread
    unsigned a_cp, b_cp, ld2, b_tile;
    int nchunk;
    bool active, bvalid;
};

template <bool DOWN>
__device__ __forceinline__ CopyState setup_copy(const FfnArgs& A, const StepDesc& d, unsigned sA) {
    CopyState c;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int pair = warp >> 1, half = warp & 1, crow = lane >> 4, ccol = lane & 15;
    const size_t per = (size_t)A.R * A.C;
    const unsigned ld = DOWN ? A.R : A.C;
    // weight copy: this warp moves tile rows [16 half, 16 half + 16); instruction i moves rows 2i, 2i+1 of
    // those; this lane moves 16 bytes of row 2i + (lane >> 4)
    if (DOWN) {
        c.w0 = d.blob + per + (size_t)(d.row0 + half * 16 + crow) * ld + d.k0 + ccol * 16;
        c.w1 = c.w0 + (size_t)8 * ld;
    } else {
        c.w0 = d.blob + (size_t)(d.row0 + half * 8 + crow) * ld + d.k0 + ccol * 16;
        c.w1 = c.w0 + 2 * per;
    }
    c.ld2 = 2 * ld;
    c.a_cp = sA + pair * kATile + (half * 16 + crow) * kSeg + ((ccol ^ (crow << 2)) << 4);
    // activation copy: thread t moves pieces (t % 8) + 8 q, q = 0..3, of token t / 8 (512 bytes per token and stage)
    const int bcol = threadIdx.x & 7, btok = threadIdx.x >> 3;
    c.b_tile = d.nt * 8 * kBRow;
    c.b_cp = sA + stages_for(d.nt) * (kPairs * kATile) + btok * kBRow + bcol * 16;
    {
        // S5 of a wide-range expert: the tile's first nt / 2 n-tiles hold the upper window of the <= 16 tokens, the
        // other nt / 2 the lower window of the same tokens, so one pass over the weight fragments serves both
        int trow = btok;
        const __half* src = DOWN ? A.h16 : A.x16;
        if (DOWN && d.wide) {
            const int hr = d.nt * 4;               // rows of one window: 8 * (nt / 2)
            if (btok >= hr) { trow = btok - hr; src = A.h16lo; }
            c.bvalid = trow < d.ntok && btok < 2 * hr;
        } else {
            c.bvalid = btok < d.ntok;
        }
        const int tok = min(trow, d.ntok - 1);     // rows beyond ntok alias the last valid row and are not copied
        const size_t rowi = DOWN ? (size_t)(d.pos0 + tok) : (size_t)A.row_token[d.pos0 + tok];
        c.b = reinterpret_cast<const unsigned char*>(src + rowi * ld + d.k0) + bcol * 16;
    }
    c.nchunk = d.klen / kChunk;
    c.active = d.active;
    return c;
}

// Issue the copies of stage sg into ring buffer `buf`; advances the source pointers by one stage.
// WEIGHTS / ACTS select the half of the stage to issue (both by default).
template <bool WEIGHTS = true, bool ACTS = true>
__device__ __forceinline__ void issue_stage(CopyState& c, int sg, int buf) {
    const int left = c.nchunk - sg * kSegChunks;                // chunks valid in this stage
    if (WEIGHTS) {
        if (c.active && (int)(threadIdx.x & 15) < left * 4) {
            const unsigned dst = c.a_cp + buf * (kPairs * kATile);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                cp_async16_s(dst + (2 * i) * kSeg, c.w0 + i * c.ld2);          // S4: W1^ rows; S5: rows 0-7
                cp_async16_s(dst + (8 + 2 * i) * kSeg, c.w1 + i * c.ld2);      // S4: W3^ rows; S5: rows 8-15
            }
        }
        c.w0 += kSeg; c.w1 += kSeg;
    }
    if (ACTS) {
        if (c.bvalid) {
            const unsigned dst = c.b_cp + buf * c.b_tile;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (q < left) cp_async16_s(dst + q * 128, c.b + q * 128);
        }
        c.b += kSeg * 2;
    }
}

// The first stages of a step (as many as its ring holds), one cp.async group each.
template <bool DOWN>
__device__ __forceinline__ CopyState start_step(const FfnArgs& A, const StepDesc& d, unsigned sA) {
    CopyState c = setup_copy<DOWN>(A, d, sA);
    const int nstage = (c.nchunk + kSegChunks - 1) / kSegChunks, ks = stages_for(d.nt);
    for (int s = 0; s < ks; ++s) {
        if (s < nstage) issue_stage(c, s, s);
        cp_async_commit();
    }
    return c;
}

// The same in two halves, for a kernel whose weights do not depend on the kernel before it but whose activations do:
// the weight copies of the first stages go out before the wait on that kernel (one group, older than all others),
// the activation copies after it, one group per stage in the places where start_step commits its groups, so the
// group counts that the step's waits rely on are the same.
template <bool DOWN>
__device__ __forceinline__ CopyState start_step_weights(const FfnArgs& A, const StepDesc& d, unsigned sA) {
    CopyState c = setup_copy<DOWN>(A, d, sA);
    const int nstage = (c.nchunk + kSegChunks - 1) / kSegChunks, ks = stages_for(d.nt);
    for (int s = 0; s < ks; ++s)
        if (s < nstage) issue_stage<true, false>(c, s, s);
    cp_async_commit();
    return c;
}
__device__ __forceinline__ void start_step_acts(CopyState& c, const StepDesc& d) {
    const int nstage = (c.nchunk + kSegChunks - 1) / kSegChunks, ks = stages_for(d.nt);
    for (int s = 0; s < ks; ++s) {
        if (s < nstage) issue_stage<false, true>(c, s, s);
        cp_async_commit();
    }
}

// Runs one step whose first stages are already in flight (start_step), then starts the next step's first
// stages before its own epilogue, so the memory system never idles between steps.
template <bool DOWN, int NT>
__device__ __forceinline__ void ffn_step(const FfnArgs& A, const StepDesc& d, CopyState& cs, const StepDesc& next,
                                         CopyState& cs_next, unsigned char* ringA) {
    constexpr int kStages = stages_for(NT);
    constexpr int kBTile = NT * 8 * kBRow;
    const unsigned char* blob = d.blob;
    const int row0 = d.row0, split = d.split, pos0 = d.pos0, ntok = d.ntok;
    const bool active = d.active;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, tq = lane & 3;
    const int pair = warp >> 1, half = warp & 1;
    const int C = A.C, R = A.R;
    const size_t per = (size_t)R * C;
    const unsigned sA = (unsigned)__cvta_generic_to_shared(ringA), sB = sA + kStages * (kPairs * kATile);
    // shared-memory byte addresses; everything that varies inside the loops is a compile-time offset
    const unsigned gpar = g & 1;
    const unsigned a_rd0 = sA + pair * kATile + g * kSeg + half * 128 + gpar * 64 + tq * 16;          // first chunk of this warp
    const unsigned a_rd1 = sA + pair * kATile + g * kSeg + half * 128 + (gpar ^ 1) * 64 + tq * 16;    // second chunk
    const unsigned b_rd = sB + g * kBRow + half * 256 + tq * 32;

    float acc[kMT][NT][4];
#pragma unroll
    for (int mt = 0; mt < kMT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;

    const int nchunk = cs.nchunk;
    const int nstage = (nchunk + kSegChunks - 1) / kSegChunks;
    // one 64-wide chunk: B fragments of all n-tiles, A fragments of both m-tiles, 8 NT MMAs
    auto chunk = [&](unsigned a_rd, unsigned b_at) {
        unsigned bf[NT][8];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            unsigned lo[4], hi[4];
            lds128(lo, b_at + nt * 8 * kBRow);
            lds128(hi, b_at + nt * 8 * kBRow + 16);
#pragma unroll
            for (int i = 0; i < 4; ++i) { bf[nt][i] = lo[i]; bf[nt][4 + i] = hi[i]; }
        }
#pragma unroll
        for (int mt = 0; mt < kMT; ++mt) {
            unsigned wa[4], wb[4];
            lds128(wa, a_rd + (mt * 16) * kSeg);           // MMA rows 0-7
            lds128(wb, a_rd + (mt * 16 + 8) * kSeg);       // MMA rows 8-15
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const unsigned ua = wa[j] ^ 0x80808080u, ub = wb[j] ^ 0x80808080u;
                unsigned f0, f1, f2, f3;
                f0 = cvt_exact_lo(ua); f2 = cvt_exact_hi(ua); f1 = cvt_exact_lo(ub); f3 = cvt_exact_hi(ub);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) mma16816(acc[mt][nt], f0, f1, f2, f3, bf[nt][2 * j], bf[nt][2 * j + 1]);
            }
        }
    };
    for (int sg = 0; sg < nstage; ++sg) {
        const int buf = sg % kStages;
        cp_async_wait<kStages - 1>();
        __syncthreads();                 // stage sg has landed for every thread of the CTA
        if (active) {
            const unsigned ao = buf * (kPairs * kATile), bo = buf * kBTile;
            const int nch = nchunk - sg * kSegChunks - half * 2;     // chunks of this warp that are valid (>= 2: both)
            if (nch >= 2) {
                chunk(a_rd0 + ao, b_rd + bo);
                chunk(a_rd1 + ao, b_rd + bo + 128);
            } else if (nch == 1) {
                chunk(a_rd0 + ao, b_rd + bo);
            }
        }
        __syncthreads();                 // every warp is done with the tiles of stage sg
        if (sg + kStages < nstage) issue_stage(cs, sg + kStages, buf);
        cp_async_commit();
    }
    cp_async_wait<0>();
    // The ring is idle now. If the next step has the same ring geometry its first stages start here, under
    // the reduction and the epilogue of this step; otherwise they start after the reduction, whose exchange
    // area (behind this step's ring) a larger ring would overlap.
    const bool early = next.valid && next.nt == NT;
    if (early) cs_next = start_step<DOWN>(A, next, sA);

    // Add the two halves of the reduction in two passes through the pair's exchange slot: warp `half` keeps
    // m-tile `half` and receives the other warp's partial sums of that m-tile; always (warp 0 part) + (warp 1 part).
    float* slot = reinterpret_cast<float*>(ringA + ring_bytes(NT)) + (size_t)pair * 128 * NT;
    float sum[NT][4];
    if (active && half == 1) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) slot[(nt * 4 + i) * 32 + lane] = acc[0][nt][i];
    }
    __syncthreads();
    if (active && half == 0) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                sum[nt][i] = acc[0][nt][i] + slot[(nt * 4 + i) * 32 + lane];
                slot[(nt * 4 + i) * 32 + lane] = acc[1][nt][i];          // second pass: this warp's part of m-tile 1
            }
    }
    __syncthreads();
    if (active && half == 1) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) sum[nt][i] = slot[(nt * 4 + i) * 32 + lane] + acc[1][nt][i];
    }
    if (next.valid && !early) {
        __syncthreads();                 // the exchange slots have been read
        cs_next = start_step<DOWN>(A, next, sA);
    }
    if (!active) return;
    const int mt = half;

    if (DOWN) {
        float* yp = A.ypart + (size_t)split * A.ypart_stride;
        float so0 = 1.f, so1 = 1.f;          // per-matrix format: the scale of the output column (row of W2^)
        if (A.per_matrix) {
            const __nv_bfloat16* so = reinterpret_cast<const __nv_bfloat16*>(blob + blob_fmt(1, R, C).s_out);
            so0 = __bfloat162float(so[row0 + mt * 16 + g]);
            so1 = __bfloat162float(so[row0 + mt * 16 + g + 8]);
        }
        if (NT % 2 == 0 && d.wide) {         // upper window in n-tiles [0, NT / 2), lower window of the same tokens behind
            constexpr int H = NT / 2;
            const float lo_scale = pow2i(-kLoShift);
#pragma unroll
            for (int nt = 0; nt < H; ++nt)
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int n = nt * 8 + tq * 2 + i;
                    if (n < ntok) {
                        const float hs = A.hscale[pos0 + n];
                        yp[(size_t)(pos0 + n) * C + row0 + mt * 16 + g] = fmaf(sum[nt + H][i], lo_scale, sum[nt][i]) * hs * so0;
                        yp[(size_t)(pos0 + n) * C + row0 + mt * 16 + g + 8] = fmaf(sum[nt + H][2 + i], lo_scale, sum[nt][2 + i]) * hs * so1;
                    }
                }
            return;
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int n = nt * 8 + tq * 2 + i;
                if (n < ntok) {
                    const float hs = A.hscale[pos0 + n];
                    yp[(size_t)(pos0 + n) * C + row0 + mt * 16 + g] = sum[nt][i] * hs * so0;
                    yp[(size_t)(pos0 + n) * C + row0 + mt * 16 + g + 8] = sum[nt][2 + i] * hs * so1;
                }
            }
        return;
    }

    // S4 epilogue: thread holds U (sum[.][0..1]) and G (sum[.][2..3]) of row r for tokens 2tq, 2tq+1 of each n-tile.
    // Per-pair power of two 2^f for the fp16 intermediate s_r h_r: |u|, |g| ~ s * 32 * |x| (codes have
    // rms ~ 127/4) and |h| ~ u g / 2, so s h ~ s^3 * 512 |x|^2 for the row with the LARGEST scale of the expert
    // (d.hexp = exponent of that s^3, from the routing kernel's statistics CTAs). That magnitude is placed at 2^-2:
    // what matters to the down projection is the error relative to its largest terms, so the rows that carry the
    // sum keep 11 bits with room for values 2^17 above the estimate, rows whose scale is much smaller may fall
    // into fp16's subnormals (absolute error 2^-25 against terms near 2^-2), and nothing overflows (the store
    // saturates).
    const __nv_bfloat16* sc = reinterpret_cast<const __nv_bfloat16*>(blob + 3 * per);
    const int r = row0 + mt * 8 + g;
    // s_u, s_g: scales of the up and gate rows; s_h: what is folded into the intermediate for the down projection.
    // Shared format: all three are s_r and s h ~ s^3; per-matrix: s1, s3 and 1, so h ~ s^2.
    const float s_u = __bfloat162float(sc[r]);
    const float s_g = A.per_matrix ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(blob + blob_fmt(1, R, C).s_gate)[r]) : s_u;
    const float s_h = A.per_matrix ? 1.f : s_u;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int n = nt * 8 + tq * 2 + i;
            if (n < ntok) {
                const int pos = pos0 + n;
                const int tok = A.row_token[pos];
                const int f = max(-120, min(120, -(d.hexp + 11 + 2 * expo(A.xnorm[tok]))));
                if (row0 == 0 && mt == 0 && g == 0) A.hscale[pos] = pow2i(-f);
                const float xs = A.xscale[tok];
                const float u = sum[nt][i] * (xs * s_u), gt = sum[nt][2 + i] * (xs * s_g);
                const float h = A.act_on_w1 ? silu(u) * gt : silu(gt) * u;
                const float v = h * s_h * pow2i(f);
                const unsigned short hi = f32_to_f16_sat(v);
                reinterpret_cast<unsigned short*>(A.h16)[(size_t)pos * R + r] = hi;
                if (d.wide)
                    reinterpret_cast<unsigned short*>(A.h16lo)[(size_t)pos * R + r] =
                        f32_to_f16_sat((v - __half2float(__ushort_as_half(hi))) * pow2i(kLoShift));
            }
        }
    }
}

template <bool DOWN, typename I, bool REHEARSE = false>
__global__ void __launch_bounds__(kThreads, 2) k_ffn(FfnArgs A) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ ItemTable tab;
    unsigned char* ringA = smem;
    // The schedule comes from the routing kernel, which has completed once the up/gate kernel has started; the
    // down kernel may therefore read it before its own wait (the up/gate kernel may not).
    // The down kernel goes further before its wait: it also issues the weight copies of its first step, which depend
    // on the routing alone, so the weight stream restarts while the up/gate kernel drains. Every CTA still waits
    // before it exits or signals its dependents.
    const int pair = threadIdx.x >> 6;
    const int S = DOWN ? A.down_splits : 1;
    const I n_mg = DOWN ? A.C / (16 * kMT) : A.R / (8 * kMT);
    const I per_tb = n_mg * S;
    const int w_full = block_cost(DOWN ? 1 : 0, 4);
    I u = 0, u1 = 0;
    const unsigned sA = (unsigned)__cvta_generic_to_shared(ringA);

    // Describes the step that starts at unit v (valid = false past the end of this CTA's range). S5 of a wide-range
    // expert carries two fp16 windows per token, so a block of more than 16 tokens is taken as two steps over the
    // same units: half 0 = its first 16 tokens, half 1 = the rest.
    auto decode = [&](I v, int half) {
        StepDesc d;
        d.valid = v < u1;
        d.nstep = 0; d.nt = 0; d.active = false; d.blob = nullptr; d.hexp = 0; d.wide = false; d.last_half = true;
        d.row0 = d.k0 = d.klen = d.split = d.pos0 = d.ntok = 0;
        if (!d.valid) return d;
        const int tbg = (int)(v / per_tb);
        int lo = 0, hi = tab.n_active - 1;                  // largest a with tb_prefix[a] <= tbg
        while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (tab.tb_prefix[mid] <= tbg) lo = mid; else hi = mid - 1; }
        const int e = min((int)tab.act_expert[lo], A.n_all - 1);     // (the clamp only matters to the rehearsal pass)
        const int tb = tbg - tab.tb_prefix[lo];
        const int rem = (int)(v - (I)tbg * per_tb);            // < per_tb = row groups x slices
        d.split = rem / (int)n_mg;
        const int mg = rem - d.split * (int)n_mg;
        const I left = u1 - v, in_group = n_mg - mg;
        const I steps = (left + kPairs - 1) / kPairs;
        d.nstep = (int)min(in_group, (left + steps - 1) / steps);
        const int cnt = A.count[e];
        d.pos0 = A.offset[e] + tb * kTokBlock;
        d.ntok = min(kTokBlock, cnt - tb * kTokBlock);
        d.nt = (d.ntok + 7) >> 3;
        d.wide = A.hexp[kMaxExperts + e] != 0;
        if (DOWN && d.wide) {
            d.last_half = half == 1 || d.ntok <= kTokBlock / 2;
            d.pos0 += half * (kTokBlock / 2);
            d.ntok = min(kTokBlock / 2, d.ntok - half * (kTokBlock / 2));
            d.nt = 2 * ((d.ntok + 7) >> 3);
        }
        d.blob = static_cast<const unsigned char*>(A.slots[max(A.slot_map[e], 0)]);     // (an active expert has a slot)
        if (!DOWN) d.hexp = A.hexp[e];
        d.k0 = DOWN ? d.split * A.down_slice : 0;
        d.klen = DOWN ? min(A.down_slice, A.R - d.k0) : A.C;
        d.row0 = (mg + pair) * (DOWN ? 16 * kMT : 8 * kMT);
        d.active = pair < d.nstep;
        return d;
    };

    // Table, partition and the description of the first step. The up/gate kernel runs this twice: once as a rehearsal
    // BEFORE its wait, on whatever the schedule memory holds (results discarded; every index it forms is clamped or
    // stays inside the table), then for real. The CTAs sit in that wait for most of the routing kernel anyway, and the
    // step streams more than the L2 holds, so each kernel's instructions come from DRAM again every step: the rehearsal
    // takes those misses off the critical path (same loop body, so the same instruction addresses). Steps of up to 16
    // tokens do it (fine-grained layer, 4 / 16 tokens: 0.0540 -> 0.0532 / 0.0703 -> 0.0690 ms per step); alone, without
    // a predecessor to wait for, the kernel is 1.7 us slower for it, and from 32 tokens on the step gains nothing.
    int half = 0;
    StepDesc cur;
    I total = 0;
#pragma unroll 1
    for (int pass = REHEARSE ? 0 : 1; pass < 2; ++pass) {
        if (!DOWN && pass == 1) { if (REHEARSE) __syncthreads(); pdl_wait(); pdl_launch(); }
        load_table(tab, A.sched, DOWN ? 1 : 0);
        total = (I)tab.total_tb * per_tb;
        const I cost = (I)tab.w_prefix[tab.n_active] * per_tb;
        u = unit_at<I>(tab, cost * (I)blockIdx.x / (I)gridDim.x, per_tb, w_full);
        u1 = unit_at<I>(tab, cost * (I)(blockIdx.x + 1) / (I)gridDim.x, per_tb, w_full);
        cur = decode(u, 0);
    }
    if (total == 0 || !cur.valid) { if (DOWN) { pdl_wait(); pdl_launch(); } return; }
    CopyState cs = DOWN ? start_step_weights<DOWN>(A, cur, sA) : start_step<DOWN>(A, cur, sA);
    if (DOWN) {
        pdl_wait();
        pdl_launch();
        start_step_acts(cs, cur);
    }
    while (cur.valid) {
        if (cur.last_half) { u += cur.nstep; half = 0; } else half = 1;
        const StepDesc next = decode(u, half);
        CopyState cs_next = cs;
        switch (cur.nt) {
            case 1: ffn_step<DOWN, 1>(A, cur, cs, next, cs_next, ringA); break;
            case 2: ffn_step<DOWN, 2>(A, cur, cs, next, cs_next, ringA); break;
            case 3: ffn_step<DOWN, 3>(A, cur, cs, next, cs_next, ringA); break;
            default: ffn_step<DOWN, 4>(A, cur, cs, next, cs_next, ringA); break;
        }
        cur = next;
        cs = cs_next;
    }
}

// ---------------------------------------------------------------------------------------------
// S6: out[t] = sum_j w[t][j] * y(t,j) + sum_shared y(t,s), y = sum over the reduction slices, all in
// a fixed order; rounded once to bf16 (or stored as fp32 in parity mode).
// ---------------------------------------------------------------------------------------------
struct CombineArgs {
    const int32_t* idx; const float* w; const int32_t* perm; const float* ypart;
    const uint32_t* done_mask; uint32_t* miss_mask; int32_t* status;
    void* out; int T, C, k, ns, E, S, out_fp32; long ypart_stride;
    const int32_t* count; int down_tc_min;      // terms of experts with count >= down_tc_min come from the tensor-core down kernel ...
    int tpb;                                    // tokens per CTA
    int S_stream, S_tc;                         // ... in this many slices; S = the larger of the two kernels' slice counts in use
};

constexpr int kCombineThreads = 128;
constexpr int kCombineMaxTerms = kMaxTopK + 16;     // routed choices + shared experts handled per token
constexpr int kCombineTokens = 4;                   // tokens per CTA for large batches: one metadata round trip serves four rows

__global__ void __launch_bounds__(kCombineThreads) k_combine(CombineArgs A) {
    __shared__ int s_pos_all[kCombineTokens][kCombineMaxTerms];
    __shared__ int s_S_all[kCombineTokens][kCombineMaxTerms];
    __shared__ float s_w_all[kCombineTokens][kCombineMaxTerms];
    const int t0 = blockIdx.y * A.tpb;                    // a CTA takes tpb tokens (1 for decode batches, kCombineTokens for large ones)
    const int c = (blockIdx.x * kCombineThreads + threadIdx.x) * 4;
    const int kk = A.k + A.ns;
    // one round of independent loads for the per-term metadata of all the CTA's tokens
    for (int q = threadIdx.x; q < A.tpb * kk; q += kCombineThreads) {
        const int tt = q / kk, j = q - tt * kk, t = t0 + tt;
        if (t < A.T) {
            const int e = (j < A.k) ? A.idx[(size_t)t * A.k + j] : A.E + (j - A.k);
            const float wj = (j < A.k) ? A.w[(size_t)t * A.k + j] : 1.f;
            const int pos = A.perm[(size_t)t * kk + j];
            const bool done = (A.done_mask[e >> 5] >> (e & 31)) & 1u;
            if (!done && blockIdx.x == 0) { atomicOr(A.miss_mask + (e >> 5), 1u << (e & 31)); atomicOr(A.status, 1); }
            s_pos_all[tt][j] = done ? pos : -1;
            s_S_all[tt][j] = (A.count[e] >= A.down_tc_min) ? A.S_tc : A.S_stream;
            s_w_all[tt][j] = wj;
        }
    }
    pdl_wait();            // the routing results above are older than the kernel before this one; the partial sums are not
    pdl_launch();
    __syncthreads();
    if (c >= A.C) return;
#pragma unroll 1
    for (int tt = 0; tt < A.tpb; ++tt) {
    const int t = t0 + tt;
    if (t >= A.T) break;
    const int* s_pos = s_pos_all[tt];
    const int* s_S = s_S_all[tt];
    const float* s_w = s_w_all[tt];
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (A.S == 1) {
        // one slice per term (the tensor-core path): the loads of up to 8 terms go out together, added in term order
        for (int j0 = 0; j0 < kk; j0 += 8) {
            float4 v[8];
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                const int pos = (j0 + jj < kk) ? s_pos[j0 + jj] : -1;
                v[jj] = pos >= 0 ? __ldcs(reinterpret_cast<const float4*>(A.ypart + (size_t)pos * A.C + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                const float wj = (j0 + jj < kk) ? s_w[j0 + jj] : 0.f;
                acc.x = fmaf(wj, v[jj].x, acc.x); acc.y = fmaf(wj, v[jj].y, acc.y);
                acc.z = fmaf(wj, v[jj].z, acc.z); acc.w = fmaf(wj, v[jj].w, acc.w);
            }
        }
    } else
    // loads of two terms x up to 8 reduction slices are issued together; sums keep the fixed order
    for (int j0 = 0; j0 < kk; j0 += 2) {
        for (int s0 = 0; s0 < A.S; s0 += 8) {
            float4 v[2][8];
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                const int pos = (j0 + jj < kk) ? s_pos[j0 + jj] : -1;
                const int Sj = (j0 + jj < kk) ? s_S[j0 + jj] : 0;
                const float* yp = A.ypart + (size_t)max(pos, 0) * A.C + c;
#pragma unroll
                for (int s = 0; s < 8; ++s)
                    v[jj][s] = (pos >= 0 && s0 + s < Sj)
                        ? __ldcs(reinterpret_cast<const float4*>(yp + (size_t)(s0 + s) * A.ypart_stride))
                        : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int s = 0; s < 8; ++s) { y.x += v[jj][s].x; y.y += v[jj][s].y; y.z += v[jj][s].z; y.w += v[jj][s].w; }
                const float wj = (j0 + jj < kk) ? s_w[j0 + jj] : 0.f;
                acc.x = fmaf(wj, y.x, acc.x); acc.y = fmaf(wj, y.y, acc.y);
                acc.z = fmaf(wj, y.z, acc.z); acc.w = fmaf(wj, y.w, acc.w);
            }
        }
    }
    if (A.out_fp32) {
        *reinterpret_cast<float4*>(static_cast<float*>(A.out) + (size_t)t * A.C + c) = acc;
    } else {
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 o = make_uint2(*reinterpret_cast<unsigned*>(&lo), *reinterpret_cast<unsigned*>(&hi));
        *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(A.out) + (size_t)t * A.C + c) = o;
    }
    }
}

FfnArgs make_args(mira_ctx* ctx, void* const* slots, const int32_t* slot_map) {
    FfnArgs A;
    A.slots = slots; A.slot_map = slot_map;
    A.sched = ws_ptr<Sched>(ctx, ctx->lay.sched);
    A.count = ws_ptr<int32_t>(ctx, ctx->lay.count);
    A.offset = ws_ptr<int32_t>(ctx, ctx->lay.offset);
    A.row_token = ws_ptr<int32_t>(ctx, ctx->lay.row_token);
    A.xscale = ws_ptr<float>(ctx, ctx->lay.xscale);
    A.xnorm = ws_ptr<float>(ctx, ctx->lay.xnorm);
    A.hscale = ws_ptr<float>(ctx, ctx->lay.hscale);
    A.hexp = ws_ptr<int32_t>(ctx, ctx->lay.hexp);
    A.x16 = ws_ptr<__half>(ctx, ctx->lay.x16);
    A.h16 = ws_ptr<__half>(ctx, ctx->lay.h16);
    A.h16lo = ws_ptr<__half>(ctx, ctx->lay.h16lo);
    A.ypart = ws_ptr<float>(ctx, ctx->lay.ypart);
    A.R = ctx->cfg.ffn; A.C = ctx->cfg.hidden; A.act_on_w1 = ctx->cfg.act_on_w1;
    A.down_splits = ctx->down_splits; A.down_slice = ctx->down_slice;
    A.per_matrix = ctx->cfg.format == MIRA_FORMAT_PER_MATRIX;
    A.n_all = ctx->cfg.n_experts + ctx->cfg.n_shared;
    A.ypart_stride = (long)ctx->route_T * (ctx->route_k + ctx->cfg.n_shared) * ctx->cfg.hidden;
    return A;
}

// Whether every cost position of a step fits 31 bits: cost of all token blocks (at most 32 per block; a step has at
// most pairs / 32 + experts blocks) x units per block x CTAs.
bool fits_32(const mira_ctx* ctx, long long per_tb) {
    const long long pairs = (long long)ctx->route_T * (ctx->route_k + ctx->cfg.n_shared);
    const long long blocks = pairs / kTokBlock + ctx->cfg.n_experts + ctx->cfg.n_shared;
    return blocks * 32 * per_tb * (2LL * ctx->n_sm + 1) < (1LL << 31);
}

}  // namespace

mira_status launch_up_gate(mira_ctx* ctx, void* const* slots, const int32_t* slot_map, cudaStream_t st) {
    FfnArgs A = make_args(ctx, slots, slot_map);
    ProfScope ps(ctx, MIRA_K_UP_GATE, st);
    if (ctx->route_T <= 16 && fits_32(ctx, ctx->cfg.ffn / (8 * kMT)))        // small steps rehearse their start-up code, see k_ffn
        MIRA_CUDA_OK(launch_pdl(k_ffn<false, int, true>, dim3(ctx->n_sm * 2), dim3(kThreads), kSmemBytes, st, A));
    else if (fits_32(ctx, ctx->cfg.ffn / (8 * kMT))) MIRA_CUDA_OK(launch_pdl(k_ffn<false, int>, dim3(ctx->n_sm * 2), dim3(kThreads), kSmemBytes, st, A));
    else MIRA_CUDA_OK(launch_pdl(k_ffn<false, long long>, dim3(ctx->n_sm * 2), dim3(kThreads), kSmemBytes, st, A));
    ctx->launches += 1;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

mira_status launch_down(mira_ctx* ctx, void* const* slots, const int32_t* slot_map, cudaStream_t st) {
    FfnArgs A = make_args(ctx, slots, slot_map);
    ProfScope ps(ctx, MIRA_K_DOWN, st);
    if (fits_32(ctx, (long long)(ctx->cfg.hidden / (16 * kMT)) * ctx->down_splits)) MIRA_CUDA_OK(launch_pdl(k_ffn<true, int>, dim3(ctx->n_sm * 2), dim3(kThreads), kSmemBytes, st, A));
    else MIRA_CUDA_OK(launch_pdl(k_ffn<true, long long>, dim3(ctx->n_sm * 2), dim3(kThreads), kSmemBytes, st, A));
    ctx->launches += 1;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

mira_status launch_combine(mira_ctx* ctx, int T, int k, int splits, int tc_splits, int down_tc_min, void* out, cudaStream_t st) {
    CombineArgs A;
    A.idx = ws_ptr<int32_t>(ctx, ctx->lay.idx); A.w = ws_ptr<float>(ctx, ctx->lay.w);
    A.perm = ws_ptr<int32_t>(ctx, ctx->lay.perm); A.ypart = ws_ptr<float>(ctx, ctx->lay.ypart);
    A.status = ws_ptr<int32_t>(ctx, ctx->lay.status);
    A.miss_mask = reinterpret_cast<uint32_t*>(A.status) + 16;
    A.done_mask = A.miss_mask + 8;
    A.out = out; A.T = T; A.C = ctx->cfg.hidden; A.k = k; A.ns = ctx->cfg.n_shared; A.E = ctx->cfg.n_experts;
    A.S_stream = splits; A.S_tc = tc_splits; A.S = std::max(splits, tc_splits); A.out_fp32 = ctx->cfg.out_dtype;
    A.count = ws_ptr<int32_t>(ctx, ctx->lay.count); A.down_tc_min = down_tc_min;
    A.ypart_stride = (long)T * (k + ctx->cfg.n_shared) * ctx->cfg.hidden;
    A.tpb = T >= 1024 ? kCombineTokens : 1;      // (256 tokens x 8 terms: 10.6 against 8.6 us with four; 2048 tokens x 2 terms: 30 against 34 us)
    dim3 grid((ctx->cfg.hidden / 4 + kCombineThreads - 1) / kCombineThreads, (T + A.tpb - 1) / A.tpb);
    ProfScope ps(ctx, MIRA_K_COMBINE, st);
    MIRA_CUDA_OK(launch_pdl(k_combine, grid, dim3(kCombineThreads), 0, st, A));
    ctx->launches += 1;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

mira_status set_ffn_attributes() {
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn<false, int>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemBytes)));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn<false, int, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemBytes)));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn<true, int>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemBytes)));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn<false, long long>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemBytes)));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn<true, long long>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemBytes)));
    return MIRA_OK;
}

}  // namespace mira
