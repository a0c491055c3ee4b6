// S4 / S5 for prefill-sized groups: the grouped expert GEMM on the 5th-generation tensor cores
// (tcgen05.mma, accumulators and the weight operand in TENSOR MEMORY), still directly on the compressed
// expert (Section IV-B): int8 codes are converted to fp16 in registers on their way from HBM to the MMA
// operand, the shared scale s_r is applied to the [token, row] intermediate in the epilogue, no weight is
// dequantized to memory (Section IV-A step 4, Section IV-F).
//
// Persistent CTAs (one or two per SM, see TileCfg) over tiles of 128 MMA rows x up to 128 / 192 tokens of one expert:
//   rows    : S4: 64 expert-hidden rows, MMA row 2m = W1^ row, 2m+1 = W3^ row, so U and G of one
//             (row, token) sit in neighbouring TMEM lanes and meet with one warp shuffle;
//             S5: 128 model-hidden rows of W2^ over the whole reduction.
//   columns : consecutive positions of the grouping step (the tokens of one expert).
// Warp roles, in this order:
//   converters  one or two groups of four warps taking K-blocks of 64 in turn. Thread t of a group owns MMA row
//               t: the group streams its rows' int8 codes with cp.async (8 rows x 64 B per request), each thread
//               converts its 64 codes (XOR 0x80, byte permute into the mantissa of 1024.0, subtract 1152:
//               exact) and writes them with one tcgen05.st into the A operand ring in tensor memory (TMEM
//               lane = MMA row), so converted weights never touch shared memory.
//   epilogue    four warps read the finished accumulator from TMEM, apply scales / SwiGLU, store. With two
//               accumulators the next tile's MMAs overlap; with one, the SM's other CTA fills the gap.
//   TMA warp    one lane issues one TMA tensor load (no multicast) per K-block: a box of 128 / 192 positions x
//               64 fp16 of the position-ordered activations, written in the 128-byte-swizzled K-major layout;
//               the warp also allocates / frees TMEM.
//   MMA warp    one lane issues tcgen05.mma (4 per K-block, K = 16 each; A from TMEM, B from shared memory)
//               and one tcgen05.commit per K-block; it tests the next stage's barrier between the MMAs, so
//               that its own wait costs nothing when the stage is already full.
// The A ring (TMEM) and the B ring (shared memory) have the same depth and share one 'full' barrier per stage
// (4 converter warps + the TMA transaction) and one 'empty' barrier (the commit), so the single issuing
// thread pays one wait and one commit per K-block. Every wait is bounded: a wait that runs out
// sets an error bit in the device status word and every role leaves through the common exit, where TMEM
// is always freed.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <type_traits>
#include <cuda.h>
#include "mira_internal.cuh"

namespace mira {
namespace {

constexpr int kTileM = 128;          // MMA rows per tile
constexpr int kKB = 64;              // reduction elements per pipeline stage (4 MMAs of K = 16)
constexpr int kWStages = 4;          // int8 weight ring of each converter group
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr int kWRow = 80;            // bytes per int8 row in the weight ring: 64 + 16 pad (conflict-free row reads)
constexpr int kWWarp = 32 * kWRow;   // one warp's 32 rows
constexpr int kWStage = 4 * kWWarp;  // the four warps of a converter group

// Kernel layout.
//   TN      tokens per tile (at most); NS = depth of the A ring (TMEM) and of the B ring (shared memory), which share
//           their barriers
//   GROUPS  converter groups of four warps; group g takes the K-blocks with index = g (mod GROUPS)
//   ACC     accumulator buffers in TMEM (2: the epilogue of a tile overlaps the next tile's MMAs)
//   CTAS    CTAs per SM (2: one CTA's hand-overs and epilogue hide behind the other CTA's MMAs)
//   ISSUERS MMA-issuing warps (2: they take the K-blocks in turn, so one thread's barrier waits and commit overlap
//           the other's MMAs; a turn barrier keeps the MMAs of a tile in K order)
// TMEM columns of one CTA: ACC * TN + 32 NS, a power of two, CTAS of them in the SM's 512.
template <int TN, int NS, int GROUPS, int ACC, int CTAS, int ISSUERS = 1, int WST = kWStages> struct TileCfg {
    static constexpr int kTileN = TN, kStages = NS, kGroups = GROUPS, kAccBufs = ACC, kCtasPerSm = CTAS, kIssuers = ISSUERS;
    static constexpr int kWRing = WST;           // depth of each converter group's int8 weight ring (cp.async stages)
    static constexpr int kEpiWarp0 = 4 * GROUPS, kTmaWarp = kEpiWarp0 + 4, kMmaWarp = kEpiWarp0 + 5;
    static constexpr int kThreads = (kMmaWarp + ISSUERS) * 32;
    static constexpr uint32_t kTmemCols = ACC * TN + NS * 32;
    static constexpr int kBTileBytes = TN * kKB * 2;
    static constexpr size_t kSmem = (size_t)NS * kBTileBytes + (size_t)GROUPS * WST * kWStage + 1024;
    static_assert(kTmemCols == 256 || kTmemCols == 512, "TMEM allocations are powers of two");
    static_assert(kTmemCols * CTAS <= 512, "TMEM has 512 columns per SM");
    static_assert((kSmem + 8 * 1024) * CTAS <= 227 * 1024, "shared memory per SM");
    static_assert(TN % 32 == 0, "the epilogue reads 32 columns at a time");
};
// Measured on the Mixtral shape (same run, us up/gate + down): 256 tokens 318 + 170 (Big) vs 261 + 118 (Narrow);
// 1024: 580 + 342 (Big) vs 602 + 292 (Wide); 2048: 1000 + 539 (Big) vs 1035 + 469 (Wide); fine-grained shape,
// 1024 tokens over 60 experts: 239 + 110 (Big), 228 + 104 (Wide), 211 + 97 (Narrow). The up/gate kernel has
// short tiles with a heavy epilogue and gains from the second accumulator; the down kernel has long tiles and
// gains from the second CTA.
using BigTile = TileCfg<192, 4, 2, 2, 1, 2>;    // one CTA per SM, two converter groups, two accumulators, two issuers
using WideTile = TileCfg<192, 2, 1, 1, 2>;      // two CTAs per SM
using NarrowTile = TileCfg<128, 4, 1, 1, 2>;    // two CTAs per SM, deeper ring
// (Tried for batches with few tokens per expert and dropped: 64-token tiles with a weight ring of 7 stages instead of
// 4, and the same tiles with two converter groups per CTA -- 4 groups per SM, 72 registers per thread: Mixtral shape, 64
// tokens, up/gate 228 and 217 against 226 us; fine-grained 1024 tokens 237 and 239 against 215 us. Neither the weight
// bytes in flight nor the converters' throughput is what sets the K-block period. Three CTAs per SM -- 64-token tiles,
// two ring stages, 64 registers per thread -- lost 9 to 20 %. Weight copies running ahead across tile boundaries, so
// that a tile does not start with an empty weight ring: down kernel of the fine-grained layer at 1024 tokens 99 against
// 102 us, up/gate of the Mixtral shape at 128 tokens 226 against 218 us, nothing elsewhere; the stages already converted
// cover the restart. 64-token tiles with six ring stages instead of four, two CTAs per SM: identical times at 24 to 64
// tokens (fine-grained 58.2 against 58.3 us), so with one converter group the period is that group's serial chain per
// K-block, not the depth of the ring; two groups at 64 tokens spill at the 72 registers two CTAs of 14 warps allow
// (76.8 against 58.4 us), and without the spills -- half a row converted and stored at a time, 16-column epilogue chunks --
// measure 59.7 us: the same. So neither the ring nor the converters set the period of narrow tiles: what fits all of
// it, per SM and K-block of four MMAs, is 440 - 450 cycles at 32 to 128 tokens and 397 at 192 tokens, where the
// arithmetic itself needs 384. It is not a floor of the tensor pipe: a stand-alone loop of tcgen05.mma (M = 128, K =
// 16, A from tensor memory) issues one every 51 cycles from one thread at N <= 64 and at the arithmetic rate from
// N = 128 on (two threads: at the arithmetic rate from N = 64). Clock stamps in the issuing thread: per K-block 260 -
// 290 cycles for the four MMAs, 75 - 85 for the commit, 80 for the look-ahead test, 60 - 150 in the wait: the thread
// is busy 560 of the 870 cycles, yet a second issuing thread in the narrow layout made every size 5 - 10 % slower
// (fine-grained 64 tokens 61.3 against 58.5 us; the turn hand-over costs what the sharing saves). Ring stages of two
// K-blocks for the narrow layout (one wait, one commit and one look-ahead per eight MMAs; built as a template
// parameter, correct, removed): 58.2 against 58.5 us. Weight requests of 128 contiguous bytes per row (the converters'
// ring in pairs of K-blocks) instead of 64: Mixtral shape 64 tokens 214.7 against 204.5 us, 2048 tokens up/gate + 1 %,
// down - 3 %: not the request size either. The converter warps taking every other 32-column chunk of the epilogue in
// the one-accumulator layouts (they wait for the accumulator with the next tile's first weight copies already
// issued; eight arrivals free it): wide layout, 2048 tokens, up/gate 1137 against 1145 us, narrow layout 4 - 9 %
// slower at every size: the epilogue's time is not what the other CTA of the SM cannot hide. 160-token tiles with
// three ring stages (the most that two CTAs per SM leave room for in tensor memory) against the wide layout's 192 x 2:
// up/gate 489 against 518 us at 768 tokens, 603 against 630 at 1024, 1129 against 1116 at 2048: the third stage is
// worth 4 - 5 % where the tile count stays the same and loses where 160-token tiles are more tiles; not kept.)
constexpr int kMaxDownSlices = 4;               // reduction slices of the tensor-core down projection (see plan_down)
constexpr int kBigMinPerExpert = 640;            // up/gate: ... from which the big layout is used. Re-measured with the exact code conversion (Mixtral
                                                // shape, us big / wide): 1024 tokens (256 per expert) 695 / 626, 1536 tokens 942 / 873, 2048 tokens 1182 /
                                                // 1154, 3072 tokens (768 per expert) 1737 / 1785; Mixtral-8x22B shape 1024 tokens 1148 / 991
constexpr int kWideMinPerExpert = 144;          // up/gate: average routed tokens per expert from which the wide tiles are used (640 tokens
                                                // over 8 experts: narrow 434, wide 424, big 414 us; 512 tokens: 359 / 380 / 373)

// The B tile is loaded with the smallest box that covers the tile's tokens: boxes of 32, 64, ..., 192 positions.
constexpr int kBoxStep = 32, kBoxMaps = 6;
struct TileMaps { CUtensorMap m[kBoxMaps]; };

struct TcArgs {
    void* const* slots; const int32_t* slot_map; const Sched* sched;
    const int32_t* count; const int32_t* offset;
    const float* xs_pos; const float* hm_pos; const float* sum_pos; const float* hscale;
    const int32_t* hexp;        // [2][kMaxExperts]: exponent of the intermediate's magnitude, then the wide-range flag
    __half* h16; __half* h16lo; float* ypart;
    int32_t* status;
    int R, C, act_on_w1;
    int per_matrix;             // blob format: 0 shared scale, 1 per-matrix scales (see BlobFmt)
    int up_conversion;          // up/gate codes: 0, 1 exact conversion; 2 offset subnormals
    uint32_t spin_limit;        // polls after which a barrier wait gives up (kSpinLimit; shortened by MIRA_OPT_TEST_WAIT_TIMEOUT)
    int down_splits;            // S5, one-CTA layouts: slices of the reduction, each its own tile and its own ypart slice
    long ypart_stride;          // elements between two slices of ypart
    int drop_first_load;        // test hook: CTA 0 leaves out the activation load of its first K-block, so the waits on that
                                // stage run out and the kernel leaves through its time-out path
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {      // non-blocking
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait. Returns false (and raises the abort flag) if the barrier did not flip in time.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit) {
    for (uint32_t spin = 0; spin < limit; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void cp_async16_s(uint32_t saddr, const void* g) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(saddr), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }

// Shared-memory matrix descriptor of the B tile: K-major, 128-byte swizzle (rows of 128 bytes, 8-row groups of
// 1024 bytes, the layout the TMA unit writes); a K = 16 step advances the start address by 32 bytes.
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;                          // leading byte offset: unused for swizzled K-major
    d |= (uint64_t)((1024 >> 4) & 0x3FFF) << 32;     // stride between 8-row groups
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;                          // 128-byte swizzle
    return d;
}
// Instruction descriptor, kind::f16: D fp32, A and B fp16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t make_idesc(int n) {
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}\n"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const unsigned (&v)[32]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
                 :: "r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                    "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
                    "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
                    "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
                 : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
}

// The up/gate kernel can feed the codes as fp16 subnormals (code + 128) * 2^-24 and undo offset and scale in its
// epilogue with the per-token sum of the activations: two fewer instructions per four weights in the converters
// (1.6 % of the kernel at 2048 tokens). It is an option, not the default (MIRA_OPT_UP_CONVERSION = 2): the tensor
// cores add in fp32 with truncation, so the subtracted term 128 * sum(x) costs accuracy in proportion to
// |sum x| / (rms of the row's codes * |x|_2) and to the hidden size. With Gaussian weights and zero-mean activations
// that is invisible up to a hidden size of about 8000; a mean of the order of the spread costs 6e-3 at 4096, and a
// row triple whose scale is set by another matrix's row (codes of a few units) fails at a mean of 0.3 even at 512.
// Neither can be seen from the scales, so the default converts exactly. The tiles of wide-range experts always do.
__device__ __forceinline__ unsigned cvt_exact_lo(unsigned u) {      // bytes 0,1 of (code + 128) -> half2 of codes
    unsigned v = __byte_perm(u, 0x64646464u, 0x4140);
    __half2 r = __hsub2(*reinterpret_cast<__half2*>(&v), __half2half2(__ushort_as_half(0x6480)));
    return *reinterpret_cast<unsigned*>(&r);
}
__device__ __forceinline__ unsigned cvt_exact_hi(unsigned u) {      // bytes 2,3
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
__device__ __forceinline__ float pow2_f(int e) { return __uint_as_float((unsigned)(max(-126, min(127, e)) + 127) << 23); }
__device__ __forceinline__ int expo_f(float v) { return (int)((__float_as_uint(v) >> 23) & 0xff) - 127; }

struct Tile { int pos0, ntok, row0, wide, kb0, nkb, split; const unsigned char* blob; };

// One MMA row's 64 codes of a K-block (shared memory, 64 bytes) -> 32 half2 in k order. SUB: as the fp16
// subnormals (code + 128) * 2^-24, no subtraction here; else the signed codes, exactly.
template <bool SUB>
__device__ __forceinline__ void convert_row(unsigned (&f)[32], uint32_t saddr) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        unsigned w4[4];
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(w4[0]), "=r"(w4[1]), "=r"(w4[2]), "=r"(w4[3]) : "r"(saddr + q * 16));
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const unsigned u = w4[jj] ^ 0x80808080u;
            if (SUB) {
                f[q * 8 + jj * 2] = __byte_perm(u, 0u, 0x4140);
                f[q * 8 + jj * 2 + 1] = __byte_perm(u, 0u, 0x4342);
            } else {
                f[q * 8 + jj * 2] = cvt_exact_lo(u);
                f[q * 8 + jj * 2 + 1] = cvt_exact_hi(u);
            }
        }
    }
}

template <bool DOWN, typename TC>
__global__ void __launch_bounds__(TC::kThreads, TC::kCtasPerSm) k_ffn_tc(TcArgs A, const __grid_constant__ TileMaps bmaps, const __grid_constant__ TileMaps bmaps_lo) {
    constexpr int kTileN = TC::kTileN, kAStages = TC::kStages, kBStages = TC::kStages, kBTileBytes = TC::kBTileBytes;
    constexpr int kGroups = TC::kGroups, kAccBufs = TC::kAccBufs, kWRing = TC::kWRing;
    constexpr int kEpiWarp0 = TC::kEpiWarp0, kTmaWarp = TC::kTmaWarp, kMmaWarp = TC::kMmaWarp, kIssuers = TC::kIssuers;
    constexpr uint32_t kTmemCols = TC::kTmemCols;
    constexpr uint32_t kTmemA = kAccBufs * kTileN;      // first column of the A ring
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ uint64_t s_bar[2 * kAStages + 6];   // full, empty, acc_full[2], acc_empty[2], turn[2]
    __shared__ uint32_t s_tmem;
    __shared__ volatile int s_abort;
    __shared__ int s_ntile[kMaxExperts + 1];          // exclusive prefix of token tiles per active expert
    __shared__ int s_cnt[kMaxExperts], s_off[kMaxExperts];
    __shared__ int s_wide[kMaxExperts];               // wide-range expert: two fp16 windows of the intermediate (see kLoShift)
    __shared__ const unsigned char* s_blob[kMaxExperts];
    __shared__ int s_nact;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int C = A.C, R = A.R;
    const int K = DOWN ? R : C;                       // reduction length
    const int nkb = K / kKB;
    const int n_mb = DOWN ? C / kTileM : R / (kTileM / 2);
    // S5 may cut the reduction into slices, each a tile of its own whose sums go to its own slice of ypart (the combine
    // adds the slices in order). The down projection has only C / 128 row tiles, so with few token tiles the CTAs run
    // a round and a fraction: slices make the rounds shorter. The number of slices depends on the batch size alone,
    // so every wave of a step uses the same arithmetic.
    const int S = DOWN ? A.down_splits : 1;
    const int per_e = n_mb * S;                       // tiles per token tile of an expert (tile counts fit 32 bits: checked by the launcher)
    const size_t per = (size_t)R * C;

    const uint32_t b_s = smem_u32(smem);                                          // [stage] B tile
    const uint32_t w_s = b_s + kBStages * kBTileBytes;                            // [group][stage] int8 rows
    const uint32_t bar0 = smem_u32(s_bar);
    auto a_full = [&](int s) { return bar0 + 8u * s; };
    auto a_empty = [&](int s) { return bar0 + 8u * (kAStages + s); };
    auto b_full = a_full;        // one 'full' barrier per stage: 4 converter warps + the TMA transaction
    auto b_empty = a_empty;      // one 'empty' barrier per stage: one tcgen05.commit
    auto acc_full = [&](int b) { return bar0 + 8u * (2 * kAStages + b); };
    auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kAStages + 2 + b); };
    auto turn = [&](int q) { return bar0 + 8u * (2 * kAStages + 4 + q); };

    // per-expert table: one round of parallel loads, then a serial prefix over shared memory
    const int n_active = A.sched->n_active;
    const bool sub_batch = !DOWN && A.up_conversion == 2;
    if (tid < kMaxExperts && tid < n_active) {
        const int e = A.sched->act_expert[tid];
        s_cnt[tid] = A.count[e];
        s_off[tid] = A.offset[e];
        s_wide[tid] = A.hexp[kMaxExperts + e];
        s_blob[tid] = static_cast<const unsigned char*>(A.slots[A.slot_map[e]]);
    }
    if (tid == 0) {
        for (int s = 0; s < kAStages; ++s) { mbar_init(a_full(s), 4 + 1); mbar_init(a_empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), kIssuers); mbar_init(acc_empty(b), 4); mbar_init(turn(b), 1); }
        s_abort = 0;
        s_nact = n_active;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == kTmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        // S5 of a wide-range expert holds both windows of a token in one tile: half as many tokens per tile
        const int tc_min = A.sched->tc_min[DOWN ? 1 : 0];      // hybrid step: experts with fewer pairs belong to the streaming kernel
        for (int a = 0; a < n_active; ++a) {
            const int tn = (DOWN && s_wide[a]) ? kTileN / 2 : kTileN;
            s_ntile[a] = acc; acc += s_cnt[a] >= tc_min ? (s_cnt[a] + tn - 1) / tn : 0;
        }
        s_ntile[n_active] = acc;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const long total = (long)s_ntile[s_nact] * per_e;     // < 2^31
    // Everything above read only what the routing kernels wrote, and those had completed before the kernel in front
    // of this one started (it waited for them before letting this one launch). The activations come from that
    // kernel itself.
    pdl_wait();
    pdl_launch();

    // tile order: (expert, slice, row block, token tile) with the token tile fastest, so CTAs working at the same
    // time share weight rows through L2
    auto decode = [&](long tile_l) {
        Tile t;
        const int tile = (int)tile_l;
        int lo = 0, hi = s_nact - 1;
        while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (s_ntile[mid] * per_e <= tile) lo = mid; else hi = mid - 1; }
        const int nt_e = s_ntile[lo + 1] - s_ntile[lo];
        const int local = tile - s_ntile[lo] * per_e;
        const int rest = local / nt_e, nb = local - rest * nt_e;
        int mb = rest;
        t.split = 0; t.kb0 = 0; t.nkb = nkb;
        if (DOWN && S > 1) {
            t.split = rest / n_mb; mb = rest - t.split * n_mb;
            t.kb0 = t.split * nkb / S;
            t.nkb = (t.split + 1) * nkb / S - t.kb0;
        }
        t.wide = s_wide[lo];
        const int tn = (DOWN && t.wide) ? kTileN / 2 : kTileN;
        t.pos0 = s_off[lo] + nb * tn;
        t.ntok = min(tn, s_cnt[lo] - nb * tn);
        t.row0 = mb * (DOWN ? kTileM : kTileM / 2);
        t.blob = s_blob[lo];
        return t;
    };
    // Ring bookkeeping: K-blocks are numbered over the whole life of the CTA (g = blocks of earlier tiles + kb);
    // block g uses A stage g % kAStages for the (g / kAStages)-th time, likewise for B.

    if (warp < kEpiWarp0) {
        // ------------------------------------------------ converters: group (warp >> 2) takes the blocks with g % kGroups == group
        const int group = warp >> 2, gw = warp & 3, row = gw * 32 + lane;     // MMA row of this thread
        const uint32_t w_g = w_s + group * (kWRing * kWStage) + gw * kWWarp;
        const uint32_t w_cp = w_g + (lane & 7) * kWRow + (lane >> 3) * 16;   // + stage * kWStage + i * 8 * kWRow
        const uint32_t w_rd = w_g + lane * kWRow;                             // + stage * kWStage + q * 16
        uint32_t gbase = 0;                                                   // K-blocks of this CTA's earlier tiles
        for (long tile = blockIdx.x; tile < total && !s_abort; tile += gridDim.x) {
            const Tile t = decode(tile);
            const int nkb = t.nkb;                              // K-blocks of this tile (a slice of the reduction in S5)
            const bool sub = sub_batch && !t.wide;              // offset subnormals or exact codes: per tile, see above
            // source of the row this lane copies in instruction 0 (MMA row 32 gw + (lane & 7)); instruction i is 8 MMA
            // rows further: + 8 rows of W2^ (S5) or + 4 expert-hidden rows of W1^ / W3^ (S4)
            const unsigned char* src;
            size_t src_step;
            {
                const int mrow = gw * 32 + (lane & 7);
                if (DOWN) { src = t.blob + per + (size_t)(t.row0 + mrow) * R + (lane >> 3) * 16 + (size_t)t.kb0 * kKB; src_step = (size_t)8 * R; }
                else { src = t.blob + ((mrow & 1) ? 2 * per : 0) + (size_t)(t.row0 + (mrow >> 1)) * C + (lane >> 3) * 16; src_step = (size_t)4 * C; }
            }
            const int kb0 = (int)(((uint32_t)group + kGroups - gbase % kGroups) % kGroups);   // first K-block of this tile that belongs to the group
            const int nmine = (nkb - kb0 + kGroups - 1) / kGroups;                               // its blocks: kb0, kb0 + kGroups, ...
#pragma unroll
            for (int s = 0; s < kWRing - 1; ++s) {
                if (s < nmine) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) cp_async16_s(w_cp + s * kWStage + i * 8 * kWRow, src + i * src_step + (size_t)(kb0 + kGroups * s) * kKB);
                }
                cp_async_commit();
            }
            bool ok = true;
            for (int j = 0; j < nmine; ++j) {
                const int pre = j + kWRing - 1;
                if (pre < nmine) {
                    const int ws = pre % kWRing;
#pragma unroll
                    for (int i = 0; i < 4; ++i) cp_async16_s(w_cp + ws * kWStage + i * 8 * kWRow, src + i * src_step + (size_t)(kb0 + kGroups * pre) * kKB);
                }
                cp_async_commit();
                cp_async_wait<kWRing - 1>();
                __syncwarp();                                     // the other lanes' copies of this stage have landed too
                const int ws = j % kWRing;
                unsigned f[32];                                   // 64 codes as fp16, in k order
                if (sub) convert_row<true>(f, w_rd + ws * kWStage);
                else convert_row<false>(f, w_rd + ws * kWStage);
                const uint32_t g = gbase + (uint32_t)(kb0 + kGroups * j);
                const uint32_t st = g % kAStages;
                if (!mbar_wait(a_empty(st), ((g / kAStages) & 1u) ^ 1u, &s_abort, A.spin_limit)) { ok = false; break; }
                tc_fence_after();
                __syncwarp();
                tmem_st32(tmem + ((uint32_t)(gw * 32) << 16) + kTmemA + st * 32, f);   // TMEM lane = MMA row
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(a_full(st));
            }
            cp_async_wait<0>();
            (void)row;
            if (!ok) break;
            gbase += (uint32_t)nkb;
        }
    } else if (warp < kTmaWarp) {
        // ------------------------------------------------ epilogue (thread = MMA row = TMEM lane)
        const int q4 = warp & 3, row = q4 * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(q4 * 32) << 16);
        long it = 0;
        for (long tile = blockIdx.x; tile < total && !s_abort; tile += gridDim.x, ++it) {
            const Tile t = decode(tile);
            const int buf = (int)(it % kAccBufs);
            if (!mbar_wait(acc_full(buf), (uint32_t)((it / kAccBufs) & 1), &s_abort, A.spin_limit)) break;
            tc_fence_after();
            const uint32_t acc_t = lane_base + buf * kTileN;
            const int ncol = (t.ntok + 31) & ~31;
            if (DOWN) {
                const int c = t.row0 + row;
                // per-matrix format: the scale of output column c (row c of W2^)
                const float so = A.per_matrix ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(t.blob + blob_fmt(1, R, C).s_out)[c]) : 1.f;
                float* yp = A.ypart + (size_t)t.split * A.ypart_stride;
                auto store = [&](auto wide_c) {       // compiled with and without the second window, chosen per tile
                    constexpr bool kWide = decltype(wide_c)::value;
                    for (int c0 = 0; c0 < ncol; c0 += 32) {
                        uint32_t v[32];
                        __syncwarp();
                        tmem_ld32(acc_t + c0, v);
                        if (kWide) {                  // the lower window's sums sit one box further, scaled by 2^kLoShift
                            uint32_t w[32];
                            __syncwarp();
                            tmem_ld32(acc_t + ncol + c0, w);
                            const float lo_scale = pow2_f(-kLoShift);
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(fmaf(__uint_as_float(w[j]), lo_scale, __uint_as_float(v[j])));
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int n = c0 + j;
                            if (n < t.ntok) yp[(size_t)(t.pos0 + n) * C + c] = __uint_as_float(v[j]) * (__ldg(A.hscale + t.pos0 + n) * so);
                        }
                    }
                };
                if (t.wide) store(std::integral_constant<bool, true>{});
                else store(std::integral_constant<bool, false>{});
            } else {
                // Even lanes hold U (W1^ row), odd lanes G (W3^ row) of the same expert-hidden row. Of every pair of
                // columns the even lane finishes the even one and the odd lane the odd one, branch-free.
                const int r = t.row0 + (row >> 1);
                const float s_u = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(t.blob + 3 * per)[r]);
                const float s_g = A.per_matrix ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(t.blob + blob_fmt(1, R, C).s_gate)[r]) : s_u;
                const float s_h = A.per_matrix ? 1.f : s_u;          // folded into the intermediate (shared format only)
                const int odd = row & 1;
                // The loop is compiled in three forms (offset subnormals / exact codes; one or two fp16 windows) and
                // the form is chosen per tile, so that no per-element branch sits in it.
                auto finish = [&](auto sub_c, auto wide_c) {
                    constexpr bool kSub = decltype(sub_c)::value, kWide = decltype(wide_c)::value;
                    for (int c0 = 0; c0 < ncol; c0 += 32) {
                        uint32_t v[32];
                        __syncwarp();
                        tmem_ld32(acc_t + c0, v);
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const float a = __uint_as_float(v[2 * jj]), b = __uint_as_float(v[2 * jj + 1]);
                            // one exchange per pair: the even lane needs its neighbour's G of the even column, the odd lane
                            // its neighbour's U of the odd column
                            const float other = __shfl_xor_sync(0xffffffffu, odd ? a : b, 1);
                            const int n = c0 + 2 * jj + odd;
                            const int pc = t.pos0 + min(n, t.ntok - 1);
                            const float xs = __ldg(A.xs_pos + pc);
                            float ru = odd ? other : a, rg = odd ? b : other;
                            if (kSub) {                       // undo the 2^-24 and the +128 offset of the codes
                                const float off = -128.f * __ldg(A.sum_pos + pc);
                                ru = fmaf(ru, 16777216.f, off); rg = fmaf(rg, 16777216.f, off);
                            }
                            const float u = ru * (xs * s_u), g = rg * (xs * s_g);
                            const float act = A.act_on_w1 ? u : g, lin = A.act_on_w1 ? g : u;
                            const float h = __fdividef(act, 1.f + __expf(-act)) * lin;
                            const float val = h * s_h * __ldg(A.hm_pos + pc);
                            const unsigned short hi16 = f32_to_f16_sat(val);
                            if (n < t.ntok) {
                                reinterpret_cast<unsigned short*>(A.h16)[(size_t)(t.pos0 + n) * R + r] = hi16;
                                if (kWide)
                                    reinterpret_cast<unsigned short*>(A.h16lo)[(size_t)(t.pos0 + n) * R + r] =
                                        f32_to_f16_sat((val - __half2float(__ushort_as_half(hi16))) * pow2_f(kLoShift));
                            }
                        }
                    }
                };
                using T1 = std::integral_constant<bool, true>;
                using T0 = std::integral_constant<bool, false>;
                if (t.wide) finish(T0{}, T1{});               // wide-range experts always take the exact codes
                else if (sub_batch) finish(T1{}, T0{});
                else finish(T0{}, T0{});
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(buf));
        }
    } else if (warp == kTmaWarp) {
        // ------------------------------------------------ activation producer: one lane, one TMA load per K-block
        // The box is the smallest of 32, 64, ... positions that covers the tile's tokens; its rows past the expert's
        // tokens are other positions or zero fill, and their accumulator columns are never read.
        if (lane == 0) {
            uint32_t st = 0, ph = 1;                     // ring stage and the parity of its 'empty' barrier to wait for
            for (long tile = blockIdx.x; tile < total && !s_abort; tile += gridDim.x) {
                const Tile t = decode(tile);
                const int hi = (t.ntok + kBoxStep - 1) / kBoxStep - 1;              // box of 32 (hi + 1) positions
                const uint64_t map = reinterpret_cast<uint64_t>(&bmaps.m[hi]);
                const uint64_t map_lo = reinterpret_cast<uint64_t>(&bmaps_lo.m[hi]);
                const uint32_t box_bytes = (uint32_t)(hi + 1) * kBoxStep * kKB * 2;
                const bool two = DOWN && t.wide;                                    // second box: the lower window, behind the first
                bool ok = true;
                for (int kb = 0; kb < t.nkb; ++kb) {
                    if (!mbar_wait(b_empty(st), ph, &s_abort, A.spin_limit)) { ok = false; break; }
                    if (A.drop_first_load && blockIdx.x == 0 && tile == blockIdx.x && kb == 0) {    // test hook, see TcArgs
                        if (++st == kBStages) { st = 0; ph ^= 1u; }
                        continue;
                    }
                    const uint32_t dst = b_s + st * kBTileBytes, bar = b_full(st);
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(two ? 2 * box_bytes : box_bytes) : "memory");
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                                 ::"r"(dst), "l"(map), "r"((t.kb0 + kb) * kKB), "r"(t.pos0), "r"(bar) : "memory");
                    if (two)
                        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                                     ::"r"(dst + box_bytes), "l"(map_lo), "r"((t.kb0 + kb) * kKB), "r"(t.pos0), "r"(bar) : "memory");
                    if (++st == kBStages) { st = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
        }
    } else {
        // ------------------------------------------------ MMA issuers (one lane each). With two, issuer q takes the
        // K-blocks with running index g = q (mod 2); before its MMAs it waits for the other issuer's turn signal, so
        // the MMAs of a tile reach the tensor pipe in K order, and its own waits and commit run under the other's MMAs.
        if (lane == 0) {
            const int q = warp - kMmaWarp;
            uint32_t g = 0;                              // running K-block index over the life of the CTA
            uint32_t nmine = 0;                          // K-blocks this issuer has issued
            uint32_t buf = 0, pacc = 1;                  // accumulator buffer and the parity of its 'empty' barrier
            const uint64_t bdesc0 = make_desc_sw128(b_s);
            bool ready = false;                          // this issuer's next stage was already seen full
            for (long tile = blockIdx.x; tile < total && !s_abort; tile += gridDim.x) {
                const Tile t = decode(tile);
                // columns of the MMA: the tile's tokens, or for a wide-range expert's down projection both boxes
                const uint32_t idesc = make_idesc((DOWN && t.wide) ? 2 * ((t.ntok + kBoxStep - 1) / kBoxStep) * kBoxStep : (t.ntok + 15) & ~15);
                if (!mbar_wait(acc_empty(buf), pacc, &s_abort, A.spin_limit)) break;   // its previous epilogue is done
                tc_fence_after();
                const uint32_t d_t = tmem + buf * kTileN;
                bool ok = true;
                for (int kb = 0; kb < t.nkb; ++kb, ++g) {
                    if (kIssuers == 2 && (int)(g & 1u) != q) continue;
                    const uint32_t sa = g % kAStages, pa = (g / kAStages) & 1u;
                    if (!ready && !mbar_wait(a_full(sa), pa, &s_abort, A.spin_limit)) { ok = false; break; }
                    if (kIssuers == 2 && g > 0) {            // the other issuer has issued K-block g - 1
                        const uint32_t n_other = (q == 0) ? nmine - 1 : nmine;      // its blocks before this one, minus one
                        if (!mbar_wait(turn(q), n_other & 1u, &s_abort, A.spin_limit)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const uint32_t a_t = tmem + kTmemA + sa * 32;
                    const uint64_t bdesc = bdesc0 + (uint64_t)(sa * (kBTileBytes >> 4));
                    umma_ts(d_t, a_t, bdesc, idesc, kb ? 1u : 0u);
                    umma_ts(d_t, a_t + 8, bdesc + 2, idesc, 1u);               // +32 bytes per K step of 16
                    umma_ts(d_t, a_t + 16, bdesc + 4, idesc, 1u);
                    umma_ts(d_t, a_t + 24, bdesc + 6, idesc, 1u);
                    if (kIssuers == 2) mbar_arrive(turn(q ^ 1));           // issued: the other issuer may go
                    umma_commit(a_empty(sa));              // both rings' stages are free once these MMAs have read them
                    ++nmine;
                    // look at this issuer's next stage while the tensor pipe is busy, so that the wait above is
                    // skipped when the stage is already full
                    const uint32_t gn = g + kIssuers;
                    ready = mbar_test(a_full(gn % kAStages), (gn / kAStages) & 1u);
                }
                if (!ok) break;
                umma_commit(acc_full(buf));
                if (++buf == kAccBufs) { buf = 0; pacc ^= 1u; }
            }
        }
    }
    // ---------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (s_abort && tid == 0) atomicOr(A.status, 2);      // after the barrier: the role that gave up may be the last to arrive
    if (warp == kTmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------------------------
// The same grouped GEMM with the MMA spread over a PAIR of SMs (tcgen05 cta_group::2): a cluster of two CTAs works
// on tiles of 256 MMA rows x up to 192 tokens. Each CTA converts ITS 128 weight rows into its own tensor memory and
// loads ITS half of the activation tile (the tile's first / second half of the positions, one plain TMA tensor load
// per K-block and CTA, no multicast) into its own shared memory; one thread of the even CTA (the leader) issues
// the MMAs for both SMs. Per SM and K-block the activation tile costs half the shared-memory traffic of the one-CTA
// kernels (they are bound by it with two CTAs per SM), and one issuing thread's waits and commits serve two SMs.
// Measured on B200 (Mixtral shape, 2048 tokens, us per kernel, pair / one-CTA layouts): up/gate 1111 / 1143, down
// 630 / 541; 512 tokens 435 / 373 and 300 / 198. The pair's K-block period (0.46 us for 256 x 192 x 64) is that of
// the one-CTA kernel per SM, whatever the ring depth (4 or 8 stages) and the tile width (128 or 192 tokens), and as
// a one-CTA-per-SM cluster kernel it cannot overlap its neighbours in the stream. It is therefore not chosen by
// default (MIRA_OPT_TENSOR_LAYOUT 4 and 5 select it); what it needed to run at all: remote arrivals as plain
// mbarrier.arrive (a .release.cluster arrival per K-block cost 40 % of the kernel), one tcgen05.commit per CTA's
// barrier, the peer's TMA load completing its bytes on the leader's barrier.
//   barriers   full[s]      leader only: its 4 converter warps + the peer's 4 (remote arrivals) + the leader's
//                           expect_tx; both CTAs' loads complete their bytes on it
//              empty[s]     one in each CTA, each signalled by a tcgen05.commit of the leader: the stage of the A
//                           ring (TMEM) and of the B ring (shared memory) of that CTA is free
//              acc_full[b]  one in each CTA, likewise: the accumulator half in that CTA's TMEM is complete
//              acc_empty[b] leader only: 4 local + 4 remote epilogue warps have drained their halves
// Every wait is bounded as in the one-CTA kernels; both CTAs meet at a cluster barrier before tensor memory is
// freed, because the leader's MMAs write the peer's tensor memory and read its shared memory.
constexpr int kPairGroups = 2, kPairAcc = 2;
constexpr int kPairEpiWarp0 = 4 * kPairGroups, kPairTmaWarp = kPairEpiWarp0 + 4, kPairMmaWarp = kPairEpiWarp0 + 5;
constexpr int kPairIssuers = 2;                       // MMA-issuing warps of the leader, taking the K-blocks in turn
constexpr int kPairThreads = (kPairMmaWarp + kPairIssuers) * 32;
constexpr uint32_t kPairTmemCols = 512;
constexpr int kHalfBoxStep = 16, kHalfBoxMaps = 6;                    // half-tile boxes of 16, 32, ..., 96 positions
// TN tokens per tile, NS ring stages (A ring in TMEM, B ring in shared memory): two accumulators of TN columns and
// NS stages of 32 columns fill the 512 TMEM columns either as (192, 4) or as (128, 8).
template <int TN, int NS> struct PairCfg {
    static constexpr int kTileN = TN, kStages = NS;
    static constexpr uint32_t kTmemA = kPairAcc * TN;
    static constexpr int kBHalfBytes = (TN / 2) * kKB * 2;           // one CTA's half of the activation tile, per stage
    static constexpr size_t kSmem = (size_t)NS * kBHalfBytes + (size_t)kPairGroups * kWStages * kWStage + 1024;
    static_assert(kTmemA + NS * 32 <= kPairTmemCols, "TMEM columns");
    static_assert(TN / 2 <= kHalfBoxStep * kHalfBoxMaps && TN % 64 == 0, "boxes cover a half tile");
};
using PairWide = PairCfg<192, 4>;
using PairDeep = PairCfg<128, 8>;

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {       // shared::cluster address of saddr in CTA `rank`
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];\n" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void umma2_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}\n"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma2_commit(uint32_t cluster_bar) {                   // a barrier of either CTA of the pair
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ uint32_t make_idesc_m(int m, int n) {
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct HalfMaps { CUtensorMap m[kHalfBoxMaps]; };

template <bool DOWN, typename PC>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
k_ffn_tc_pair(TcArgs A, const __grid_constant__ HalfMaps bmaps, const __grid_constant__ HalfMaps bmaps_lo) {
    constexpr int kPairTileN = PC::kTileN, kPairStages = PC::kStages, kPairBHalfBytes = PC::kBHalfBytes;
    constexpr uint32_t kPairTmemA = PC::kTmemA;
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ uint64_t s_bar[2 * kPairStages + 6];   // full, empty, acc_full[2], acc_empty[2], turn[2]
    __shared__ uint32_t s_tmem;
    __shared__ volatile int s_abort;
    __shared__ int s_ntile[kMaxExperts + 1];
    __shared__ int s_cnt[kMaxExperts], s_off[kMaxExperts], s_wide[kMaxExperts];
    __shared__ const unsigned char* s_blob[kMaxExperts];
    __shared__ int s_nact;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_rank();             // 0: leader (issues the MMAs), 1: peer
    const bool leader = rank == 0;
    const int C = A.C, R = A.R;
    const int K = DOWN ? R : C;
    const int nkb = K / kKB;
    const int n_mb = DOWN ? C / (2 * kTileM) : R / kTileM;       // row blocks of 256 MMA rows
    const size_t per = (size_t)R * C;
    const uint32_t b_s = smem_u32(smem);
    const uint32_t w_s = b_s + kPairStages * kPairBHalfBytes;
    const uint32_t bar0 = smem_u32(s_bar);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (kPairStages + s); };
    auto acc_full = [&](int b) { return bar0 + 8u * (2 * kPairStages + b); };
    auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kPairStages + 2 + b); };
    auto turn = [&](int q) { return bar0 + 8u * (2 * kPairStages + 4 + q); };

    const int n_active = A.sched->n_active;
    const bool sub_batch = !DOWN && A.up_conversion == 2;
    if (tid < kMaxExperts && tid < n_active) {
        const int e = A.sched->act_expert[tid];
        s_cnt[tid] = A.count[e];
        s_off[tid] = A.offset[e];
        s_wide[tid] = A.hexp[kMaxExperts + e];
        s_blob[tid] = static_cast<const unsigned char*>(A.slots[A.slot_map[e]]);
    }
    if (tid == 0) {
        for (int s = 0; s < kPairStages; ++s) { mbar_init(full(s), 4 + 4 + 1); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), kPairIssuers); mbar_init(acc_empty(b), 4 + 4); mbar_init(turn(b), 1); }
        s_abort = 0;
        s_nact = n_active;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == kPairTmaWarp) {                        // the same warp of both CTAs, as the pair allocation requires
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&s_tmem)), "r"(kPairTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;\n" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        const int tc_min = A.sched->tc_min[DOWN ? 1 : 0];
        for (int a = 0; a < n_active; ++a) {
            const int tn = (DOWN && s_wide[a]) ? kPairTileN / 2 : kPairTileN;
            s_ntile[a] = acc; acc += s_cnt[a] >= tc_min ? (s_cnt[a] + tn - 1) / tn : 0;
        }
        s_ntile[n_active] = acc;
    }
    tc_fence_before();
    cluster_sync_all();                                // barriers of both CTAs are initialised before any remote arrival
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const long total = (long)s_ntile[s_nact] * n_mb;
    const long pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    pdl_wait();
    pdl_launch();

    auto decode = [&](long tile) {
        Tile t;
        int lo = 0, hi = s_nact - 1;
        while (lo < hi) { int mid = (lo + hi + 1) >> 1; if ((long)s_ntile[mid] * n_mb <= tile) lo = mid; else hi = mid - 1; }
        const int nt_e = s_ntile[lo + 1] - s_ntile[lo];
        const long local = tile - (long)s_ntile[lo] * n_mb;
        const int nb = (int)(local % nt_e), mb = (int)(local / nt_e);
        t.wide = s_wide[lo];
        const int tn = (DOWN && t.wide) ? kPairTileN / 2 : kPairTileN;
        t.pos0 = s_off[lo] + nb * tn;
        t.ntok = min(tn, s_cnt[lo] - nb * tn);
        t.row0 = mb * (DOWN ? 2 * kTileM : kTileM) + (int)rank * (DOWN ? kTileM : kTileM / 2);   // this CTA's first row
        t.blob = s_blob[lo];
        return t;
    };
    // Columns of the pair's MMA and what each CTA loads for them. Ordinary tile: N = the tokens rounded up to 32, the
    // leader holds positions [0, N / 2), the peer [N / 2, N). Down projection of a wide-range expert: the leader holds
    // the upper window of the tile's (at most 96) tokens, the peer the lower window of the same tokens, N / 2 each.
    auto half_rows = [&](const Tile& t) {
        return (DOWN && t.wide) ? ((t.ntok + 31) / 32) * 32 : ((t.ntok + 31) / 32) * 16;
    };

    if (warp < kPairEpiWarp0) {
        // ------------------------------------------------ converters (as in the one-CTA kernel; the 'full' arrival goes to the leader)
        const int group = warp >> 2, gw = warp & 3;
        const uint32_t w_g = w_s + group * (kWStages * kWStage) + gw * kWWarp;
        const uint32_t w_cp = w_g + (lane & 7) * kWRow + (lane >> 3) * 16;
        const uint32_t w_rd = w_g + lane * kWRow;
        uint32_t gbase = 0;
        for (long tile = pair_id; tile < total && !s_abort; tile += n_pairs, gbase += (uint32_t)nkb) {
            const Tile t = decode(tile);
            const bool sub = sub_batch && !t.wide;
            const unsigned char* src;
            size_t src_step;
            {
                const int mrow = gw * 32 + (lane & 7);
                if (DOWN) { src = t.blob + per + (size_t)(t.row0 + mrow) * R + (lane >> 3) * 16; src_step = (size_t)8 * R; }
                else { src = t.blob + ((mrow & 1) ? 2 * per : 0) + (size_t)(t.row0 + (mrow >> 1)) * C + (lane >> 3) * 16; src_step = (size_t)4 * C; }
            }
            const int kb0 = (int)(((uint32_t)group + kPairGroups - gbase % kPairGroups) % kPairGroups);
            const int nmine = (nkb - kb0 + kPairGroups - 1) / kPairGroups;
#pragma unroll
            for (int s = 0; s < kWStages - 1; ++s) {
                if (s < nmine) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) cp_async16_s(w_cp + s * kWStage + i * 8 * kWRow, src + i * src_step + (size_t)(kb0 + kPairGroups * s) * kKB);
                }
                cp_async_commit();
            }
            bool ok = true;
            for (int j = 0; j < nmine; ++j) {
                const int pre = j + kWStages - 1;
                if (pre < nmine) {
                    const int ws = pre % kWStages;
#pragma unroll
                    for (int i = 0; i < 4; ++i) cp_async16_s(w_cp + ws * kWStage + i * 8 * kWRow, src + i * src_step + (size_t)(kb0 + kPairGroups * pre) * kKB);
                }
                cp_async_commit();
                cp_async_wait<kWStages - 1>();
                __syncwarp();
                const int ws = j % kWStages;
                unsigned f[32];
                if (sub) convert_row<true>(f, w_rd + ws * kWStage);
                else convert_row<false>(f, w_rd + ws * kWStage);
                const uint32_t g = gbase + (uint32_t)(kb0 + kPairGroups * j);
                const uint32_t st = g % kPairStages;
                if (!mbar_wait(empty(st), ((g / kPairStages) & 1u) ^ 1u, &s_abort, A.spin_limit)) { ok = false; break; }
                tc_fence_after();
                __syncwarp();
                tmem_st32(tmem + ((uint32_t)(gw * 32) << 16) + kPairTmemA + st * 32, f);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(full(st), 0));
            }
            cp_async_wait<0>();
            if (!ok) break;
        }
    } else if (warp < kPairTmaWarp) {
        // ------------------------------------------------ epilogue of this CTA's 128 accumulator rows
        const int q4 = warp & 3, row = q4 * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(q4 * 32) << 16);
        long it = 0;
        for (long tile = pair_id; tile < total && !s_abort; tile += n_pairs, ++it) {
            const Tile t = decode(tile);
            const int buf = (int)(it % kPairAcc);
            if (!mbar_wait(acc_full(buf), (uint32_t)((it / kPairAcc) & 1), &s_abort, A.spin_limit)) break;
            tc_fence_after();
            const uint32_t acc_t = lane_base + buf * kPairTileN;
            const int hr = half_rows(t);
            if (DOWN) {
                const int c = t.row0 + row;
                const float so = A.per_matrix ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(t.blob + blob_fmt(1, R, C).s_out)[c]) : 1.f;
                const int ncol = t.wide ? hr : 2 * hr;            // columns that hold tokens (wide: the lower window follows)
                auto store = [&](auto wide_c) {
                    constexpr bool kWide = decltype(wide_c)::value;
                    for (int c0 = 0; c0 < ncol; c0 += 32) {
                        uint32_t v[32];
                        __syncwarp();
                        tmem_ld32(acc_t + c0, v);
                        if (kWide) {
                            uint32_t w[32];
                            __syncwarp();
                            tmem_ld32(acc_t + hr + c0, w);
                            const float lo_scale = pow2_f(-kLoShift);
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(fmaf(__uint_as_float(w[j]), lo_scale, __uint_as_float(v[j])));
                        }
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int n = c0 + j;
                            if (n < t.ntok) A.ypart[(size_t)(t.pos0 + n) * C + c] = __uint_as_float(v[j]) * (__ldg(A.hscale + t.pos0 + n) * so);
                        }
                    }
                };
                if (t.wide) store(std::integral_constant<bool, true>{});
                else store(std::integral_constant<bool, false>{});
            } else {
                const int r = t.row0 + (row >> 1);
                const float s_u = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(t.blob + 3 * per)[r]);
                const float s_g = A.per_matrix ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(t.blob + blob_fmt(1, R, C).s_gate)[r]) : s_u;
                const float s_h = A.per_matrix ? 1.f : s_u;
                const int odd = row & 1;
                const int ncol = 2 * hr;
                auto finish = [&](auto sub_c, auto wide_c) {
                    constexpr bool kSub = decltype(sub_c)::value, kWide = decltype(wide_c)::value;
                    for (int c0 = 0; c0 < ncol; c0 += 32) {
                        uint32_t v[32];
                        __syncwarp();
                        tmem_ld32(acc_t + c0, v);
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const float a = __uint_as_float(v[2 * jj]), b = __uint_as_float(v[2 * jj + 1]);
                            const float oa = __shfl_xor_sync(0xffffffffu, a, 1), ob = __shfl_xor_sync(0xffffffffu, b, 1);
                            const int n = c0 + 2 * jj + odd;
                            const int pc = t.pos0 + min(n, t.ntok - 1);
                            const float xs = __ldg(A.xs_pos + pc);
                            float ru = odd ? ob : a, rg = odd ? b : oa;
                            if (kSub) {
                                const float off = -128.f * __ldg(A.sum_pos + pc);
                                ru = fmaf(ru, 16777216.f, off); rg = fmaf(rg, 16777216.f, off);
                            }
                            const float u = ru * (xs * s_u), g = rg * (xs * s_g);
                            const float act = A.act_on_w1 ? u : g, lin = A.act_on_w1 ? g : u;
                            const float h = __fdividef(act, 1.f + __expf(-act)) * lin;
                            const float val = h * s_h * __ldg(A.hm_pos + pc);
                            const unsigned short hi16 = f32_to_f16_sat(val);
                            if (n < t.ntok) {
                                reinterpret_cast<unsigned short*>(A.h16)[(size_t)(t.pos0 + n) * R + r] = hi16;
                                if (kWide)
                                    reinterpret_cast<unsigned short*>(A.h16lo)[(size_t)(t.pos0 + n) * R + r] =
                                        f32_to_f16_sat((val - __half2float(__ushort_as_half(hi16))) * pow2_f(kLoShift));
                            }
                        }
                    }
                };
                using T1 = std::integral_constant<bool, true>;
                using T0 = std::integral_constant<bool, false>;
                if (t.wide) finish(T0{}, T1{});
                else if (sub_batch) finish(T1{}, T0{});
                else finish(T0{}, T0{});
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty(buf), 0));
        }
    } else if (warp == kPairTmaWarp) {
        // ------------------------------------------------ this CTA's half of the activation tile, one load per K-block
        if (lane == 0) {
            uint32_t st = 0, ph = 1;
            const uint32_t full0 = map_to_cta(full(0), 0);        // the leader's 'full' barriers (8 bytes apart)
            for (long tile = pair_id; tile < total && !s_abort; tile += n_pairs) {
                const Tile t = decode(tile);
                const int hr = half_rows(t);
                const int mi = hr / kHalfBoxStep - 1;
                const bool lo_window = DOWN && t.wide && !leader;
                const uint64_t map = reinterpret_cast<uint64_t>(lo_window ? &bmaps_lo.m[mi] : &bmaps.m[mi]);
                const int pos = (DOWN && t.wide) ? t.pos0 : t.pos0 + (int)rank * hr;
                const uint32_t half_bytes = (uint32_t)hr * kKB * 2;
                bool ok = true;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!mbar_wait(empty(st), ph, &s_abort, A.spin_limit)) { ok = false; break; }
                    const uint32_t dst = b_s + st * kPairBHalfBytes, bar = full0 + 8u * st;
                    if (leader)
                        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(full(st)), "r"(2 * half_bytes) : "memory");
                    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                                 ::"r"(dst), "l"(map), "r"(kb * kKB), "r"(pos), "r"(bar) : "memory");
                    if (++st == kPairStages) { st = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
        }
    } else if (leader) {
        // ------------------------------------------------ MMA issuers of the pair (one lane each, in the leader). Issuer q
        // takes the K-blocks with running index g = q (mod 2); a turn barrier keeps the MMAs of a tile in K order, and
        // one issuer's waits and commits run under the other's MMAs.
        if (lane == 0) {
            const int q = warp - kPairMmaWarp;
            uint32_t g = 0, nmine = 0, buf = 0, pacc = 1;
            const uint64_t bdesc0 = make_desc_sw128(b_s);
            const uint32_t empty_peer0 = map_to_cta(empty(0), 1), acc_full_peer0 = map_to_cta(acc_full(0), 1);
            bool ready = false;
            for (long tile = pair_id; tile < total && !s_abort; tile += n_pairs) {
                const Tile t = decode(tile);
                const uint32_t idesc = make_idesc_m(2 * kTileM, 2 * half_rows(t));
                if (!mbar_wait(acc_empty(buf), pacc, &s_abort, A.spin_limit)) break;
                tc_fence_after();
                const uint32_t d_t = tmem + buf * kPairTileN;
                bool ok = true;
                for (int kb = 0; kb < nkb; ++kb, ++g) {
                    if (kPairIssuers == 2 && (int)(g & 1u) != q) continue;
                    const uint32_t sa = g % kPairStages, pa = (g / kPairStages) & 1u;
                    if (!ready && !mbar_wait(full(sa), pa, &s_abort, A.spin_limit)) { ok = false; break; }
                    if (kPairIssuers == 2 && g > 0) {         // the other issuer has issued K-block g - 1
                        const uint32_t n_other = (q == 0) ? nmine - 1 : nmine;
                        if (!mbar_wait(turn(q), n_other & 1u, &s_abort, A.spin_limit)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const uint32_t a_t = tmem + kPairTmemA + sa * 32;
                    const uint64_t bdesc = bdesc0 + (uint64_t)(sa * (kPairBHalfBytes >> 4));
                    umma2_ts(d_t, a_t, bdesc, idesc, kb ? 1u : 0u);
                    umma2_ts(d_t, a_t + 8, bdesc + 2, idesc, 1u);
                    umma2_ts(d_t, a_t + 16, bdesc + 4, idesc, 1u);
                    umma2_ts(d_t, a_t + 24, bdesc + 6, idesc, 1u);
                    if (kPairIssuers == 2) mbar_arrive(turn(q ^ 1));
                    umma2_commit(empty(sa));                       // both CTAs' stages are free once these MMAs have read them
                    umma2_commit(empty_peer0 + 8u * sa);
                    ++nmine;
                    const uint32_t gn = g + kPairIssuers;
                    ready = mbar_test(full(gn % kPairStages), (gn / kPairStages) & 1u);
                }
                if (!ok) break;
                umma2_commit(acc_full(buf));
                umma2_commit(acc_full_peer0 + 8u * buf);
                if (++buf == kPairAcc) { buf = 0; pacc ^= 1u; }
            }
        }
    }
    // ---------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (s_abort && tid == 0) atomicOr(A.status, 2);
    cluster_sync_all();                                // the peer's tensor and shared memory are no longer in use by this CTA
    if (warp == kPairTmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kPairTmemCols) : "memory");
    }
}

// Position-ordered inputs of the tensor path, one block per position: x16p[pos] = x16[row_token[pos]] (so the
// tokens of one expert are consecutive rows and one TMA box covers a token tile) and the per-position factors
// of the SwiGLU epilogue: the undo factor of the token's fp16 pre-scaling and the power of two 2^f that places
// the fp16 intermediate (same rule as the streaming kernels: |s h| ~ s^3 * 512 |x|^2 with s the largest row scale
// of the expert, whose exponent the routing kernel's statistics CTAs left in hexp; that magnitude goes to 2^-2).
struct GatherArgs {
    const __half* x16; const int32_t* row_token; __half* x16p; const int32_t* offset; void* const* slots;
    const int32_t* slot_map; const float* xscale; const float* xnorm; const float* xsum; float* xs_pos; float* hm_pos;
    float* sum_pos; float* hscale; const int32_t* hexp; const Sched* sched;
    int C, R, Etot;
};

__global__ void __launch_bounds__(128) k_gather_x16p(GatherArgs G) {
    __shared__ int s_e;
    pdl_wait();            // the routing kernels' results; see launch_pdl
    pdl_launch();
    const int pos = blockIdx.x, tok = G.row_token[pos];
    for (int e = threadIdx.x; e < G.Etot; e += 128)
        if (G.offset[e] <= pos && pos < G.offset[e + 1]) s_e = e;
    __syncthreads();
    if (G.offset[s_e + 1] - G.offset[s_e] < G.sched->tc_min[0]) return;     // hybrid step: this expert's up/gate is the streaming kernel's
    const uint4* src = reinterpret_cast<const uint4*>(G.x16 + (size_t)tok * G.C);
    uint4* dst = reinterpret_cast<uint4*>(G.x16p + (size_t)pos * G.C);
    for (int i = threadIdx.x; i < G.C / 8; i += 128) dst[i] = src[i];
    if (threadIdx.x == 0) {
        if (G.slot_map[s_e] < 0) return;                        // expert not resident: its pairs are skipped everywhere
        const int f = max(-120, min(120, -(G.hexp[s_e] + 11 + 2 * expo_f(G.xnorm[tok]))));
        G.xs_pos[pos] = G.xscale[tok];
        G.sum_pos[pos] = G.xsum[tok];
        G.hm_pos[pos] = pow2_f(f);
        G.hscale[pos] = pow2_f(-f);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool encode_map(EncodeTiledFn fn, void* out, void* base, size_t rows, size_t cols, int box_rows) {
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kKB, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(reinterpret_cast<CUtensorMap*>(out), CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base, gdim, gstride, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

TcArgs make_tc_args(mira_ctx* ctx, void* const* slots, const int32_t* slot_map) {
    TcArgs A;
    A.slots = slots; A.slot_map = slot_map;
    A.sched = ws_ptr<Sched>(ctx, ctx->lay.sched);
    A.count = ws_ptr<int32_t>(ctx, ctx->lay.count);
    A.offset = ws_ptr<int32_t>(ctx, ctx->lay.offset);
    A.xs_pos = ws_ptr<float>(ctx, ctx->lay.xs_pos);
    A.hm_pos = ws_ptr<float>(ctx, ctx->lay.hm_pos);
    A.sum_pos = ws_ptr<float>(ctx, ctx->lay.sum_pos);
    A.hscale = ws_ptr<float>(ctx, ctx->lay.hscale);
    A.h16 = ws_ptr<__half>(ctx, ctx->lay.h16);
    A.h16lo = ws_ptr<__half>(ctx, ctx->lay.h16lo);
    A.hexp = ws_ptr<int32_t>(ctx, ctx->lay.hexp);
    A.ypart = ws_ptr<float>(ctx, ctx->lay.ypart);
    A.status = ws_ptr<int32_t>(ctx, ctx->lay.status);
    A.R = ctx->cfg.ffn; A.C = ctx->cfg.hidden; A.act_on_w1 = ctx->cfg.act_on_w1;
    A.per_matrix = ctx->cfg.format == MIRA_FORMAT_PER_MATRIX;
    A.up_conversion = ctx->up_conversion;
    A.spin_limit = kSpinLimit;
    A.drop_first_load = 0;
    A.down_splits = 1;
    A.ypart_stride = (long)ctx->route_T * (ctx->route_k + ctx->cfg.n_shared) * ctx->cfg.hidden;
    return A;
}

}  // namespace

bool tc_shape_ok(const mira_config& c) { return c.hidden % 128 == 0 && c.ffn % 64 == 0; }

// Tensor maps of the two activation matrices the TMA unit reads (both live in the caller's workspace, whose
// address is fixed at mira_create). Returns false if the driver entry point is unavailable.
bool build_tensor_maps(mira_ctx* ctx) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || fn == nullptr ||
        q != cudaDriverEntryPointSuccess)
        return false;
    const size_t P = (size_t)Pmax(ctx->cfg);
    const EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(fn);
    __half* x16p = ws_ptr<__half>(ctx, ctx->lay.x16p);
    __half* h16 = ws_ptr<__half>(ctx, ctx->lay.h16);
    __half* h16lo = ws_ptr<__half>(ctx, ctx->lay.h16lo);
    for (int i = 0; i < kBoxMaps; ++i)
        if (!encode_map(enc, ctx->tmap_x16p[i], x16p, P, ctx->cfg.hidden, (i + 1) * kBoxStep) ||
            !encode_map(enc, ctx->tmap_h16[i], h16, P, ctx->cfg.ffn, (i + 1) * kBoxStep) ||
            !encode_map(enc, ctx->tmap_h16lo[i], h16lo, P, ctx->cfg.ffn, (i + 1) * kBoxStep))
            return false;
    for (int i = 0; i < kHalfBoxMaps; ++i)              // half-tile boxes of the two-SM kernels
        if (!encode_map(enc, ctx->tmap_half[0][i], x16p, P, ctx->cfg.hidden, (i + 1) * kHalfBoxStep) ||
            !encode_map(enc, ctx->tmap_half[1][i], h16, P, ctx->cfg.ffn, (i + 1) * kHalfBoxStep) ||
            !encode_map(enc, ctx->tmap_half[2][i], h16lo, P, ctx->cfg.ffn, (i + 1) * kHalfBoxStep))
            return false;
    return true;
}

// Kernel layout of a step.
template <bool DOWN, typename TC>
static void launch_cfg(mira_ctx* ctx, const TcArgs& A, const unsigned char (*maps)[128], cudaStream_t st) {
    static_assert(TC::kTileN <= kBoxStep * kBoxMaps, "no box covers the tile");
    static_assert((TC::kTileN / 2) % kBoxStep == 0, "a wide-range expert's half tile is a whole number of boxes");
    TileMaps tm, tm_lo;
    memcpy(&tm, maps, sizeof(tm));
    memcpy(&tm_lo, ctx->tmap_h16lo, sizeof(tm_lo));          // only the down projection of wide-range experts reads it
    launch_pdl(k_ffn_tc<DOWN, TC>, dim3(ctx->n_sm * TC::kCtasPerSm), dim3(TC::kThreads), TC::kSmem, st, A, tm, tm_lo);
}

// Estimated cost of a down projection in a 2-CTA layout with tiles of `tn` tokens: the kernel has few row tiles
// (C / 128), so what counts is how many ROUNDS of tiles its CTAs run, times the cost of a tile relative to a narrow
// one (a wide tile covers 1.5 times the tokens at 1.3 times the time: 224 K-blocks take 115 us narrow, 150 us wide).
// Token-tile columns: exact for the shared experts, tokens / tn plus half a ragged tile per expert for the routed ones
// (at least one per expert that can be routed to).
static double down_cost(const mira_ctx* ctx, int tn, double tile_cost, int slices = 1) {
    const double T = ctx->route_T, E = ctx->cfg.n_experts, pairs = T * ctx->route_k;
    const double cols = std::max(std::min(E, pairs), pairs / tn + 0.5 * std::min(E, pairs)) + ctx->cfg.n_shared * std::ceil(T / tn);
    const double tiles = cols * (ctx->cfg.hidden / kTileM) * slices;
    return std::ceil(tiles / (2.0 * ctx->n_sm)) * tile_cost;
}

// The two-SM kernel: one cluster of two CTAs per pair of SMs.
template <bool DOWN>
static void launch_pair(mira_ctx* ctx, const TcArgs& A, cudaStream_t st) {
    static_assert(sizeof(HalfMaps) == sizeof(ctx->tmap_half[0]), "tensor map storage");
    HalfMaps tm, tm_lo;
    memcpy(&tm, ctx->tmap_half[DOWN ? 1 : 0], sizeof(tm));
    memcpy(&tm_lo, ctx->tmap_half[2], sizeof(tm_lo));
    if (ctx->tc_layout == 5) launch_pdl(k_ffn_tc_pair<DOWN, PairDeep>, dim3(ctx->n_sm / 2 * 2), dim3(kPairThreads), PairDeep::kSmem, st, A, tm, tm_lo);
    else launch_pdl(k_ffn_tc_pair<DOWN, PairWide>, dim3(ctx->n_sm / 2 * 2), dim3(kPairThreads), PairWide::kSmem, st, A, tm, tm_lo);
}
static bool pair_shape_ok(const mira_config& c) { return c.ffn % kTileM == 0 && c.hidden % (2 * kTileM) == 0; }

// Layout and number of reduction slices of the down projection of the step last routed. Both follow from the batch
// size, the top-k and the configuration alone, so every wave of a step gets the same plan (the slices change the
// order of the additions). Cost model, in K-blocks: rounds of tiles x (K-blocks of a tile x the layout's relative
// K-block time + 26 for the epilogue and the hand-over of the accumulator, fitted to the times below); a tile of S
// slices has 1/S of the K-blocks. Measured on the Mixtral shape at 512 tokens (us, down kernel + combine, 1 / 2 / 3 /
// 4 slices): 240 + 15 / 198 + 18 / 208 + 20 / 233 + 22; Mixtral-8x22B shape at 256 tokens 284 + 14 / 254 + 17; at other
// sizes (128 to 2048 tokens) slices bring nothing and one is chosen.
struct DownPlan { int layout, splits; };
static DownPlan plan_down(const mira_ctx* ctx) {
    const long avg = (long)ctx->route_T * ctx->route_k / (ctx->cfg.n_experts > 0 ? ctx->cfg.n_experts : 1);
    DownPlan p;
    p.layout = ctx->tc_layout;                             // 0 unless a layout is forced (MIRA_OPT_TENSOR_LAYOUT)
    p.splits = 1;
    const bool narrow_only = 2 * avg < NarrowTile::kTileN;
    if (p.layout == 0)
        // wide only when the estimate is clearly lower: near a tie the narrow layout is the safer one (1536 tokens: 429 / 460)
        // (with fewer than half a narrow tile of tokens per expert on average no expert fills a wide tile: narrow.
        // Fine-grained layer, 128 tokens: 39 against 45 us)
        p.layout = (narrow_only || 0.9 * down_cost(ctx, NarrowTile::kTileN, 1.0) <= down_cost(ctx, WideTile::kTileN, 1.3)) ? 1 : 2;
    if ((p.layout == 4 || p.layout == 5) && !pair_shape_ok(ctx->cfg)) p.layout = 2;
    if (p.layout >= 4) return p;                           // the two-SM kernel takes whole reductions
    const int nkb = ctx->cfg.ffn / kKB;
    const int max_s = std::min(std::min(ctx->down_splits, kMaxDownSlices), std::max(1, nkb / 16));
    if (ctx->down_slices_forced > 0) { p.splits = std::min(ctx->down_slices_forced, std::min(ctx->down_splits, nkb)); return p; }
    if (ctx->tc_layout != 0) return p;                     // a forced layout keeps whole reductions unless slices are forced too
    auto cost = [&](int tn, double w, int S) { return down_cost(ctx, tn, 1.0, S) * (w * nkb / S + 26.0); };
    const double w0 = p.layout == 1 ? 1.0 : 1.3;
    double best = cost(p.layout == 1 ? NarrowTile::kTileN : WideTile::kTileN, w0, 1);
    for (int S = 2; S <= max_s; ++S)
        for (int lay = 1; lay <= (narrow_only ? 1 : 2); ++lay) {
            const double c = cost(lay == 1 ? NarrowTile::kTileN : WideTile::kTileN, lay == 1 ? 1.0 : 1.3, S);
            if (c < 0.93 * best) { best = c; p.layout = lay; p.splits = S; }     // slices cost partial-sum traffic: only for a clear gain
        }
    return p;
}

int down_tc_slices(const mira_ctx* ctx) { return plan_down(ctx).splits; }

template <bool DOWN>
static void launch_tc(mira_ctx* ctx, TcArgs& A, const unsigned char (*maps)[128], cudaStream_t st) {
    // Up/gate has many row tiles (R / 64), so its time follows the number of tiles: narrow tiles while an expert gets
    // fewer tokens than fill wide ones on average, then wide, and with few experts and many tokens the big layout.
    // The down projection is chosen by the estimated number of rounds (measured on the Mixtral shape, us narrow /
    // wide: 384 tokens 186 / 160, 896 tokens 229 / 300, 1024 tokens 311 / 291, 3072 tokens 730 / 664: the estimate
    // picks the faster one in each case).
    const long avg = (long)ctx->route_T * ctx->route_k / (ctx->cfg.n_experts > 0 ? ctx->cfg.n_experts : 1);
    int layout = ctx->tc_layout;                          // 0 unless a layout is forced (MIRA_OPT_TENSOR_LAYOUT)
    if (layout == 0 && !DOWN) {
        layout = avg < kWideMinPerExpert ? 1 : (avg >= kBigMinPerExpert && ctx->cfg.n_experts <= 16) ? 3 : 2;
    }
    if (DOWN) { const DownPlan p = plan_down(ctx); layout = p.layout; A.down_splits = p.splits; }
    if ((layout == 4 || layout == 5) && !pair_shape_ok(ctx->cfg)) layout = DOWN ? 2 : 3;
    if (layout >= 4) launch_pair<DOWN>(ctx, A, st);
    else if (layout == 1) launch_cfg<DOWN, NarrowTile>(ctx, A, maps, st);
    else if (layout == 3) launch_cfg<DOWN, BigTile>(ctx, A, maps, st);
    else launch_cfg<DOWN, WideTile>(ctx, A, maps, st);
}

mira_status launch_up_gate_tc(mira_ctx* ctx, void* const* slots, const int32_t* slot_map, cudaStream_t st) {
    TcArgs A = make_tc_args(ctx, slots, slot_map);
    GatherArgs G;
    G.x16 = ws_ptr<__half>(ctx, ctx->lay.x16); G.row_token = ws_ptr<int32_t>(ctx, ctx->lay.row_token);
    G.x16p = ws_ptr<__half>(ctx, ctx->lay.x16p); G.offset = A.offset; G.slots = slots; G.slot_map = slot_map;
    G.xscale = ws_ptr<float>(ctx, ctx->lay.xscale); G.xnorm = ws_ptr<float>(ctx, ctx->lay.xnorm);
    G.xs_pos = ws_ptr<float>(ctx, ctx->lay.xs_pos); G.hm_pos = ws_ptr<float>(ctx, ctx->lay.hm_pos);
    G.sum_pos = ws_ptr<float>(ctx, ctx->lay.sum_pos); G.xsum = ws_ptr<float>(ctx, ctx->lay.xsum);
    G.hscale = ws_ptr<float>(ctx, ctx->lay.hscale); G.hexp = ws_ptr<int32_t>(ctx, ctx->lay.hexp); G.sched = A.sched;
    G.C = ctx->cfg.hidden; G.R = ctx->cfg.ffn; G.Etot = Et(ctx->cfg);
    if (ctx->test_wait_timeout) {          // one launch whose waits run out (MIRA_OPT_TEST_WAIT_TIMEOUT)
        A.spin_limit = 1u << 12;
        A.drop_first_load = 1;
        ctx->test_wait_timeout = false;
    }
    ProfScope ps(ctx, MIRA_K_UP_GATE, st);
    const int P = ctx->route_T * (ctx->route_k + ctx->cfg.n_shared);
    MIRA_CUDA_OK(launch_pdl(k_gather_x16p, dim3(P), dim3(128), 0, st, G));
    launch_tc<false>(ctx, A, ctx->tmap_x16p, st);
    ctx->launches += 2;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

mira_status launch_down_tc(mira_ctx* ctx, void* const* slots, const int32_t* slot_map, cudaStream_t st) {
    TcArgs A = make_tc_args(ctx, slots, slot_map);
    ProfScope ps(ctx, MIRA_K_DOWN, st);
    launch_tc<true>(ctx, A, ctx->tmap_h16, st);
    ctx->launches += 1;
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}

template <typename TC> static cudaError_t set_smem_attr() {
    cudaError_t e = cudaFuncSetAttribute(k_ffn_tc<false, TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC::kSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(k_ffn_tc<true, TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC::kSmem);
}

mira_status set_tc_attributes() {
    MIRA_CUDA_OK(set_smem_attr<BigTile>());
    MIRA_CUDA_OK(set_smem_attr<WideTile>());
    MIRA_CUDA_OK(set_smem_attr<NarrowTile>());
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn_tc_pair<false, PairWide>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairWide::kSmem));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn_tc_pair<true, PairWide>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairWide::kSmem));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn_tc_pair<false, PairDeep>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairDeep::kSmem));
    MIRA_CUDA_OK(cudaFuncSetAttribute(k_ffn_tc_pair<true, PairDeep>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairDeep::kSmem));
    return MIRA_OK;
}

}  // namespace mira
