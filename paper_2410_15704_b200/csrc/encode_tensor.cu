// Tensor-core encode for group_dim 32 (Section 2.2, Algorithm 1).
//
// One persistent CTA per SM takes a contiguous run of 128-row tiles and works
// through it in rounds of up to three tiles (one row per thread, 12 epilogue
// warps; rounds are sized evenly, e.g. 7 tiles = 3 + 2 + 2) plus four role
// warps: one MMA issuer per tile (the warp runs its loop as one, a single lane
// issues) and the operand loader.  The role warps give registers up
// (setmaxnreg 40) and the epilogue warps take them (152).
//   - Scores ||e||^2 - 2 z.e of a 128-row tile against 128 codewords are one
//     tcgen05.mma chain (M=128, N=128, seven K=16 steps over the split
//     half-precision operands described in prepare.cu), accumulated in float32
//     in TMEM.
//   - The B operand (128 codewords per slot) streams from the prepared block
//     through a ring of shared-memory slots filled by cp.async.bulk; every
//     slot serves all three tiles.
//   - Epilogue threads read their row's 128 scores with four tcgen05.ld of 32
//     columns issued together, hand the accumulator back to the issuer as soon
//     as they have landed, and fold them afterwards while the next chain runs.
//     The fold keeps running minima over four partitions of the stage's
//     columns: by 128-column chunk (a short list of the chunks that come within
//     the error window of the running minimum), by 32-column block of a chunk,
//     by half of a block, and by place within a half (16 places): 36 minimum
//     operations per 32 scores.  At the stage end the sets of chunks, blocks,
//     halves and places whose minimum lies inside the window bound where the
//     exact argmin can be: when each set has one member the column is known
//     and only that codeword is fetched; otherwise the warp re-scores every
//     column in the product of the sets exactly in float32 against the float32
//     codebook (direct form, lowest index on ties), and a full exact scan
//     covers list overflow.  The emitted code is the exact-L2 choice.
//   - The A operand (the residual split into half-precision head and remainder)
//     lives in TMEM next to its tile's scores, so the tensor core fetches only B
//     from shared memory; the constant (1 1 1 0 ...) rows that pick up the
//     squared norms are one small shared-memory tile used by every MMA chain.
//   - The float32 residual lives in registers between stages and is parked in
//     shared memory during a stage's sweep; x is read once and only codes and
//     the half-precision deviation are written.
//   - With the EMA statistics asked for (Section 3), every stage's rows join the bins of their codes:
//     the stage's output, parked for the next sweep, is added by the tile's MMA issuer warp between
//     two chains of that sweep (count x codeword is added back by the caller's finishing kernel); the
//     last stage's input is added by the epilogue warps.
// TMEM columns of tile t: scores [160 t, 160 t + 128), A operand
// [160 t + 128, 160 t + 160) (16 columns of head, 16 of remainder).
// Every wait is bounded; a wait that gives up sets status->wait_timeouts and
// the kernel drains and returns.
#include "prepared.cuh"

namespace rvq {

namespace {

constexpr int kTiles = 3;
constexpr int kRowsPerPass = 128 * kTiles;
constexpr int kEpiThreads = kRowsPerPass;
constexpr int kThreads = kEpiThreads + 32 * (kTiles + 1);  // + one MMA issuer warp per tile + loader warp
constexpr int kRing = 6;                                  // operand slots in flight
constexpr int kTileCols = 160;                            // TMEM columns per tile: 128 scores + 32 of A operand
constexpr int kOnesBytes = 2 * 128 * 16;                  // the constant A cells (1 1 1 0 ...) and (0 ...)
constexpr int kListCap = 8;
constexpr uint32_t kWaitLimit = 4u * 1000u * 1000u;

constexpr int kOffB = 0;
constexpr int kOffA = kOffB + kRing * kSlotBytes;                    
constexpr int kOffZ = kOffA + kOnesBytes;                             // parked residuals, float [32][rows]
constexpr int kOffListV = kOffZ + 32 * kRowsPerPass * 4;              
constexpr int kOffListI = kOffListV + (kListCap + 1) * kRowsPerPass * 4;   
constexpr int kOffCodes = kOffListI + (kListCap + 1) * kRowsPerPass * 2;   
constexpr int kOffBars = kOffCodes + kRowsPerPass * 16 * 2;          
constexpr int kOffFlags = kOffBars + 256;                             // per row of the round: bit 0 valid, bit 1 degenerate
constexpr int kSmemBytes = kOffFlags + 512;
constexpr int kDeferMinSlots = 5;                                     // chunks a stage needs for its issuers to take the statistics

// barrier slots
constexpr int kBarFull = 0, kBarEmpty = kRing, kBarAReady = 2 * kRing, kBarAccFull = 2 * kRing + kTiles,
              kBarAccFree = 2 * kRing + 2 * kTiles, kNumBars = 2 * kRing + 3 * kTiles;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait; returns false (and raises the CTA's abort flag) when it gives up.  A phase that has
// completed already is recognised by the non-blocking test (a plain shared-memory read); only a
// phase still pending goes through the suspending form.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t limit = kWaitLimit)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
#pragma unroll 1
    for (uint32_t it = 0; it < limit; ++it) {
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1u;
    return false;
}

__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    // K-major, no swizzle: 8x16-byte core matrices; LBO steps along the
    // contraction, SBO along rows; descriptor version 1.
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | ((uint64_t)1 << 46);
}

__device__ __forceinline__ void mma_f16_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ float min3(float a, float b, float c)
{
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

#define RVQ_R32(u) u[0], u[1], u[2], u[3], u[4], u[5], u[6], u[7], u[8], u[9], u[10], u[11], u[12], u[13], u[14], u[15], \
    u[16], u[17], u[18], u[19], u[20], u[21], u[22], u[23], u[24], u[25], u[26], u[27], u[28], u[29], u[30], u[31]
#define RVQ_OUT32(u) "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), \
    "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), \
    "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), \
    "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
#define RVQ_INOUT32(u) "+r"(u[0]), "+r"(u[1]), "+r"(u[2]), "+r"(u[3]), "+r"(u[4]), "+r"(u[5]), "+r"(u[6]), "+r"(u[7]), \
    "+r"(u[8]), "+r"(u[9]), "+r"(u[10]), "+r"(u[11]), "+r"(u[12]), "+r"(u[13]), "+r"(u[14]), "+r"(u[15]), \
    "+r"(u[16]), "+r"(u[17]), "+r"(u[18]), "+r"(u[19]), "+r"(u[20]), "+r"(u[21]), "+r"(u[22]), "+r"(u[23]), \
    "+r"(u[24]), "+r"(u[25]), "+r"(u[26]), "+r"(u[27]), "+r"(u[28]), "+r"(u[29]), "+r"(u[30]), "+r"(u[31])
#define RVQ_IN32(u) "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), \
    "r"(u[8]), "r"(u[9]), "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]), \
    "r"(u[16]), "r"(u[17]), "r"(u[18]), "r"(u[19]), "r"(u[20]), "r"(u[21]), "r"(u[22]), "r"(u[23]), \
    "r"(u[24]), "r"(u[25]), "r"(u[26]), "r"(u[27]), "r"(u[28]), "r"(u[29]), "r"(u[30]), "r"(u[31])

// Start loading 32 consecutive TMEM columns of this thread's lane.  The
// registers are not valid until tmem_ld_wait() has been given the same array.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&u)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : RVQ_OUT32(u) : "r"(taddr));
}
// Waits for every tcgen05.ld of this thread; the arrays pass through so that no
// use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait4(uint32_t (&u)[32], uint32_t (&v)[32], uint32_t (&w)[32], uint32_t (&x)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" : RVQ_INOUT32(u) : : "memory");
    asm volatile("" : RVQ_INOUT32(v) : : "memory");
    asm volatile("" : RVQ_INOUT32(w) : : "memory");
    asm volatile("" : RVQ_INOUT32(x) : : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&u)[32])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 : : "r"(taddr), RVQ_IN32(u) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Per-row state of one stage's sweep over the scores.
struct Sweep {
    float m1, thr, win;      // running minimum of the block minima, threshold(m1), error window
    float zz;                // squared norm of the scaled residual: m1 + zz is the best squared distance
    int cnt;                 // listed chunks (kListCap + 1: the list overflowed)
    float bb[4];             // minimum per 32-column block position inside its 128-column chunk
    float h[2];              // minimum per half (columns 0-15, 16-31) of a block
    float d[16];             // minimum per column position inside its half
};

// One 32-column block of scores (block `b` of its chunk) folded into the running minima of three
// partitions of its columns: the 16 places inside a half (one three-input minimum takes in the two
// columns of a place), the two halves, and the block itself; returns the block minimum.  Together
// with the chunk list a column that could be the argmin is pinned to (listed chunk) x (block of the
// chunk) x (half) x (place): when every one of the four lists has a single entry, to one column.
// 36 minimum operations per 32 scores: they run on the narrow integer/compare pipe, which this sweep
// keeps about as busy as the tensor pipe, so their number per score is what the sweep's speed
// hangs on.
__device__ __forceinline__ float fold_block(Sweep &w, const uint32_t (&u)[32], int b)
{
#pragma unroll
    for (int c = 0; c < 16; ++c) w.d[c] = min3(w.d[c], __uint_as_float(u[c]), __uint_as_float(u[c + 16]));
    float hm[2];
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        const uint32_t *v = u + 16 * hf;
        const float a0 = min3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
        const float a1 = min3(__uint_as_float(v[3]), __uint_as_float(v[4]), __uint_as_float(v[5]));
        const float a2 = min3(__uint_as_float(v[6]), __uint_as_float(v[7]), __uint_as_float(v[8]));
        const float a3 = min3(__uint_as_float(v[9]), __uint_as_float(v[10]), __uint_as_float(v[11]));
        const float a4 = min3(__uint_as_float(v[12]), __uint_as_float(v[13]), __uint_as_float(v[14]));
        hm[hf] = fminf(min3(a0, a1, a2), min3(a3, a4, __uint_as_float(v[15])));
    }
    w.h[0] = fminf(w.h[0], hm[0]);
    w.h[1] = fminf(w.h[1], hm[1]);
    const float m = fminf(hm[0], hm[1]);
    w.bb[b] = fminf(w.bb[b], m);
    return m;
}

// A column can only be the exact-L2 choice (in real arithmetic, and in the float32 direct-form
// arithmetic of the all-float32 kernel, whose relative error on a distance is below 34 * 2^-24) if its
// approximate score is at most threshold(m1): the window covers the approximation error of both
// scores, the last term the float32 evaluation error of both distances (2 * 34 * 2^-24 < 2^-17.5).
__device__ __forceinline__ float threshold(const Sweep &w, float m1)
{
    return m1 + w.win + 5.4e-6f * (fmaxf(m1 + w.zz, 0.0f) + w.win);
}

__device__ __forceinline__ void list_block(Sweep &w, float cb_min, int block, float *list_v, uint16_t *list_i,
                                           int stride)
{
    const bool app = cb_min <= w.thr;
    w.m1 = fminf(w.m1, cb_min);
    w.thr = threshold(w, w.m1);
    if (app && w.cnt == kListCap) {
        // full: drop entries that left the window as the minimum came down
        int keep = 0;
        for (int e = 0; e < kListCap; ++e) {
            const float fv = list_v[e * stride];
            const uint16_t fi = list_i[e * stride];
            if (fv <= w.thr) { list_v[keep * stride] = fv; list_i[keep * stride] = fi; ++keep; }
        }
        w.cnt = keep;
    }
    const int slot = min(w.cnt, kListCap);
    list_v[slot * stride] = cb_min;
    list_i[slot * stride] = (uint16_t)block;
    w.cnt += app ? 1 : 0;
}

// 32-byte read-only global load: a codeword row costs four of these, and for
// row-per-lane gathers it is the number of load instructions that the L1 pays for.
__device__ __forceinline__ void ldg256(const float *p, float (&v)[8])
{
    asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p));
}

// Exact squared distance, direct form, same operation order as the scalar kernel.
__device__ __forceinline__ float exact_distance(const float (&z)[32], const float *__restrict__ e)
{
    float acc = 0.0f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float ev[8];
        ldg256(e + 8 * q, ev);
#pragma unroll
        for (int k = 0; k < 8; ++k) { const float t = z[8 * q + k] - ev[k]; acc = fmaf(t, t, acc); }
    }
    return acc;
}

struct Params {
    Shape s;
    const void *x;
    int64_t n, stride;
    const float *cb;
    const uint8_t *prepared;
    void *codes;
    uint16_t *std16;
    rvq_status *st;
    int tiles;          // 128-row tiles in the whole problem
    uint32_t *stat_cnt; // optional EMA statistics of this batch: counts [R][K] ...
    float *stat_sum;    // ... and sums of the stage inputs [R][K][32]; both null when not wanted
    float *energy;      // optional [R]: sum over the rows of the squared norm of what each stage leaves
    uint32_t wait_limit;   // polls after which a wait gives up (kWaitLimit; smaller only in the timeout self-test)
    int drop_last_chain;   // timeout self-test: 1 = tile 0's issuer leaves out the CTA's very last chain; else 0
    int defer_stats;       // 1 = the statistics of every stage but the last are added by the MMA issuer warps (below)
};

// The tiles of one CTA: a contiguous run, done in `rounds` rounds of nearly equal size (<= kTiles).
struct Work {
    int first, count, rounds;
    __device__ __forceinline__ int round_size(int k) const { return count / rounds + (k < count % rounds ? 1 : 0); }
    __device__ __forceinline__ int round_first(int k) const { return first + k * (count / rounds) + min(k, count % rounds); }
};

// 16 warps, launched with 128 registers per thread; the four role warps then keep 40 each and the
// twelve epilogue warps take 152 (4 x 40 + 12 x 152 = 1984 of the 2048 per lane).
__global__ void __launch_bounds__(kThreads, 1)
encode_tensor_kernel(const Params p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kOffBars);
    uint32_t *tmem_word = reinterpret_cast<uint32_t *>(smem + kOffBars + kNumBars * 8);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + kOffBars + kNumBars * 8 + 4);

    const Shape &s = p.s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = slots_per_stage(s.K);
    Work work;
    {
        const int per = p.tiles / (int)gridDim.x, rem = p.tiles % (int)gridDim.x, b = (int)blockIdx.x;
        work.count = per + (b < rem ? 1 : 0);
        work.first = b * per + min(b, rem);
        work.rounds = (work.count + kTiles - 1) / kTiles;
    }
    const int my_passes = work.rounds;
    const StageParams *sp = reinterpret_cast<const StageParams *>(p.prepared + kPreparedParamsOffset);
    const uint8_t *image = p.prepared + kPreparedImageOffset;
    const uint32_t bar0 = smem_u32(bars);
    auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        for (int i = 0; i < kRing; ++i) { mbar_init(BAR(kBarFull + i), 1); mbar_init(BAR(kBarEmpty + i), kTiles); }
        for (int t = 0; t < kTiles; ++t) {
            mbar_init(BAR(kBarAReady + t), 128); mbar_init(BAR(kBarAccFull + t), 1); mbar_init(BAR(kBarAccFree + t), 128);
        }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kEpiThreads / 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_word)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    // constant A cells shared by all tiles: (1, 1, 1, 0...) per row, then zeros
    if (tid < 128) {
        uint8_t *a = smem + kOffA + tid * 16;
        *reinterpret_cast<uint4 *>(a) = make_uint4(0x3C003C00u, 0x00003C00u, 0u, 0u);
        *reinterpret_cast<uint4 *>(a + 2048) = make_uint4(0u, 0u, 0u, 0u);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_word;

    // The four role warps run one lane each and need few registers; their share goes to the
    // epilogue warps, which hold three 32-column blocks of scores at a time
    // (12 warps x 32 x 152 + 4 warps x 32 x 40 = 63488 of the 65536 the block was launched with).
    if (warp >= kEpiThreads / 32) asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    else asm volatile("setmaxnreg.inc.sync.aligned.u32 152;");

    if (warp == kEpiThreads / 32 + kTiles) {
        // ------------------------------------------------------------ operand loader
        // One thread streams the B slots of every (pass, stage) through the ring; a slot is
        // free again once the MMA chains of all tiles that read it have completed.
        if (lane == 0 && my_passes > 0) {
            const uint32_t total = (uint32_t)my_passes * (uint32_t)s.R * (uint32_t)S;
            const uint32_t per_pass = (uint32_t)s.R * (uint32_t)S;
            uint32_t slot = 0, rs = 0, empty_par = 1;          // parity of the previous completion of empty[slot]
            bool ok = true;
            for (uint32_t nl = 0; nl < total && ok; ++nl) {
                if (nl >= (uint32_t)kRing) ok = mbar_wait(BAR(kBarEmpty + slot), empty_par, abort_flag);
                if (!ok) break;
                mbar_expect_tx(BAR(kBarFull + slot), kSlotBytes);
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(smem_u32(smem + kOffB) + slot * (uint32_t)kSlotBytes), "l"(image + (size_t)rs * kSlotBytes),
                               "r"((uint32_t)kSlotBytes), "r"(BAR(kBarFull + slot)) : "memory");
                if (++rs == per_pass) rs = 0;
                if (++slot == (uint32_t)kRing) { slot = 0; empty_par ^= 1u; }
            }
        }
    } else if (warp >= kEpiThreads / 32) {
        // ------------------------------------------------------------ MMA issuer of tile t
        // One thread per tile, each in a warp of its own so that the tiles' waits overlap.
        // Whatever it does between two tcgen05.mma chains delays its tile, so descriptors
        // are built once and all counters advance by increments.
        // (The whole warp runs the loop with warp-uniform values and one lane issues: operands that the
        // compiler knows to be uniform can stay in uniform registers, which tcgen05.mma reads directly.)
        if (my_passes > 0) {
            const int t = __shfl_sync(0xFFFFFFFFu, warp, 0) - kEpiThreads / 32;
            const uint32_t total = (uint32_t)my_passes * (uint32_t)s.R * (uint32_t)S;
            const uint32_t idesc = (1u << 4) | ((128u >> 3) << 17) | ((128u >> 4) << 24);   // f16 x f16 -> f32, M=N=128
            // Seven K=16 steps: hi.hi (2), hi.lo (2), lo.hi (2) with A in TMEM (8 columns per
            // step), then 1.norm with the constant A cells from shared memory.  A B cell is
            // 128 codewords x 16 bytes = 2048 bytes = 128 descriptor address units.
            const uint64_t bdesc0 = make_smem_desc(smem_u32(smem + kOffB), kSlotCodewords * 16, 128);
            const uint64_t ones_desc = make_smem_desc(smem_u32(smem + kOffA), 2048, 128);
            const uint32_t acc = tmem + t * kTileCols, a0 = acc + 128;
            const uint32_t bar_ready = BAR(kBarAReady + t), bar_free = BAR(kBarAccFree + t), bar_acc = BAR(kBarAccFull + t);
            const uint32_t per_round = (uint32_t)s.R * (uint32_t)S;
            uint32_t slot = 0, full_par = 0, s_in = 0, ready_par = 0, free_par = 1, in_round = 0, stage = 0;
            int round = 0;
            // Deferred statistics (Section 3's EMA sums): while stage r+1 is swept, its input z_{r+1} -- what stage r
            // left -- sits parked in shared memory, and this warp, idle between two chains, adds it to the bins of
            // the stage-r codes, one group of 32 rows after each of the chains 1..4 of the stage.  The sum of a
            // bin's stage-r INPUTS is that plus count * codeword (z_r = z_{r+1} + C_r[j]), which the caller adds
            // afterwards.  Ordering: the epilogue parks z_{r+1} and has written the stage-r codes before it hands
            // chunk 0's accumulator back, which this warp has waited for before chain 1; and it cannot finish the
            // stage, and park anew, before the chains that this warp issues after the additions.
            const float *zp = reinterpret_cast<const float *>(smem + kOffZ);
            const uint16_t *codes_s = reinterpret_cast<const uint16_t *>(smem + kOffCodes);
            const uint8_t *flags_s = smem + kOffFlags;
            bool ok = true, first = true, active = t < work.round_size(0);
            for (uint32_t q = 0; q < total && ok; ++q) {
                ok = mbar_wait(BAR(kBarFull + slot), full_par, abort_flag);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!active) {
                    // this tile sits the round out, but the slot still waits for its release
                    if (ok && lane == 0) mbar_arrive(BAR(kBarEmpty + slot));
                    if (++slot == (uint32_t)kRing) { slot = 0; full_par ^= 1u; }
                    if (++in_round == per_round) { in_round = 0; ++round; active = round < work.rounds && t < work.round_size(round); }
                    continue;                                       // (an idle round keeps `stage` at 0: it is only read while active)
                }
                if (ok && s_in == 0) ok = mbar_wait(bar_ready, ready_par, abort_flag);
                if (ok && !first) ok = mbar_wait(bar_free, free_par, abort_flag);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                first = false;
                tc_fence_after();
                const uint64_t bd = bdesc0 + (uint64_t)(slot * (uint32_t)(kSlotBytes >> 4));
                // (self-test of the give-up path: the chain that nothing comes after is left out, so that the
                // epilogue's wait for it runs out with no copy or MMA of this CTA still in flight)
                if (p.drop_last_chain && t == 0 && q == total - 1) break;
                if (lane == 0) {
                    mma_f16_ts(acc, a0, bd, idesc, 0);                      // hi[0:16]  . hi cells 0-1
                    mma_f16_ts(acc, a0 + 8, bd + 2 * 128, idesc, 1);        // hi[16:32] . hi cells 2-3
                    mma_f16_ts(acc, a0, bd + 4 * 128, idesc, 1);            // hi[0:16]  . lo cells 4-5
                    mma_f16_ts(acc, a0 + 8, bd + 6 * 128, idesc, 1);        // hi[16:32] . lo cells 6-7
                    mma_f16_ts(acc, a0 + 16, bd, idesc, 1);                 // lo[0:16]  . hi cells 0-1
                    mma_f16_ts(acc, a0 + 24, bd + 2 * 128, idesc, 1);       // lo[16:32] . hi cells 2-3
                    mma_f16_ss(acc, ones_desc, bd + 8 * 128, idesc, 1);     // (1 1 1 0..) . norm cells 8-9
                    mma_commit(bar_acc);
                    mma_commit(BAR(kBarEmpty + slot));
                }
                __syncwarp();
                if (p.defer_stats && stage >= 1u && s_in >= 1u && s_in <= 4u) {
                    const int rl = t * 128 + (int)(s_in - 1u) * 32 + lane;
                    const uint32_t fl = flags_s[rl];
                    if (fl & 1u) {
                        const size_t bin = (size_t)(stage - 1u) * s.K + codes_s[rl * 16 + (int)(stage - 1u)];
                        atomicAdd(p.stat_cnt + bin, 1u);
                        if (!(fl & 2u)) {
                            float4 *m = reinterpret_cast<float4 *>(p.stat_sum + bin * 32);
#pragma unroll
                            for (int q4 = 0; q4 < 8; ++q4)
                                atomicAdd(m + q4, make_float4(zp[(4 * q4) * kRowsPerPass + rl], zp[(4 * q4 + 1) * kRowsPerPass + rl],
                                                              zp[(4 * q4 + 2) * kRowsPerPass + rl], zp[(4 * q4 + 3) * kRowsPerPass + rl]));
                        }
                    }
                    __syncwarp();
                }
                free_par ^= 1u;
                if (++slot == (uint32_t)kRing) { slot = 0; full_par ^= 1u; }
                if (++s_in == (uint32_t)S) { s_in = 0; ready_par ^= 1u; ++stage; }
                if (++in_round == per_round) { in_round = 0; stage = 0; ++round; active = round < work.rounds && t < work.round_size(round); }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int tile = warp >> 2, q4 = warp & 3;
        const int rloc = tile * 128 + q4 * 32 + lane;
        const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(tile * kTileCols);
        float *z_park = reinterpret_cast<float *>(smem + kOffZ) + rloc;                    // [i][row]
        float *list_v = reinterpret_cast<float *>(smem + kOffListV) + rloc;              // [e][row]
        uint16_t *list_i = reinterpret_cast<uint16_t *>(smem + kOffListI) + rloc;         // [e][row]
        uint16_t *codes_s = reinterpret_cast<uint16_t *>(smem + kOffCodes);                // [row][R]
        const int G = s.G;
        uint32_t chunk_use = 0;
        uint32_t n_rescored = 0, n_exhaustive = 0, n_degenerate = 0, n_stdrange = 0;
        bool ok = true;

        for (int pass = 0; pass < my_passes && ok; ++pass) {
            if (tile >= work.round_size(pass)) continue;            // this tile sits the round out
            const int64_t row0 = (int64_t)(work.round_first(pass) + tile) * 128;   // first row of this tile
            const int64_t grow = row0 + q4 * 32 + lane;
            const int64_t v = grow / G;
            const int g = (int)(grow - v * G);
            const bool valid = v < p.n;

            // The warp's 32 / G head vectors (1024 elements) come in as 16-byte pieces through the
            // warp's share of the parking area: word k sits at [k / 32][k % 32], and piece c of
            // vector vl at position c ^ (vl mod 8) of its vector so that the reads below spread over the banks.
            float z[32];
            {
                const int eb = s.elem_bytes, ppv = s.dim * eb / 16;          // pieces per vector (>= 4)
                const int64_t v_first = (row0 + q4 * 32) / G;
                float *scr = reinterpret_cast<float *>(smem + kOffZ) + (rloc - lane);
                // (four loads in flight per lane: a 16-bit head vector of 128 channels is 16 pieces, so the
                // 8 vectors of a warp are 4 pieces per lane)
                const int npieces = (32 / G) * ppv;
                for (int c0 = 0; c0 < npieces; c0 += 128) {
                    uint4 val[4];
                    int kk[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int c = c0 + 32 * u + lane;
                        const int vl = c / ppv, off = c - vl * ppv;
                        const int64_t vv = v_first + vl;
                        val[u] = make_uint4(0u, 0u, 0u, 0u);
                        if (c < npieces && vv < p.n)
                            val[u] = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const uint8_t *>(p.x) + vv * p.stride * eb) + off);
                        kk[u] = (vl * ppv + (off ^ (vl & 7 & (ppv - 1)))) * 4;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (c0 + 32 * u + lane < npieces)
                            *reinterpret_cast<uint4 *>(scr + (kk[u] >> 5) * kRowsPerPass + (kk[u] & 31)) = val[u];
                }
                __syncwarp();
                const int vl = lane / G, sw = vl & 7 & (ppv - 1);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int b = channel_of(s.layout, G, 32, g, i) * eb;      // byte within the vector
                    const int k = (vl * ppv + ((b >> 4) ^ sw)) * 4 + ((b & 15) >> 2);
                    const uint32_t word = __float_as_uint(scr[(k >> 5) * kRowsPerPass + (k & 31)]);
                    float val;
                    if (s.dtype == RVQ_F32) val = __uint_as_float(word);
                    else {
                        const uint16_t h = (b & 2) ? (uint16_t)(word >> 16) : (uint16_t)(word & 0xFFFFu);
                        val = s.dtype == RVQ_BF16 ? __uint_as_float((uint32_t)h << 16) : __half2float(__ushort_as_half(h));
                    }
                    z[i] = valid ? val : 0.0f;
                }
                __syncwarp();
            }
            // deviation over the G lanes of this head vector, same summation order as the scalar kernel
            float dev;
            {
                float a = 0.0f;
#pragma unroll
                for (int i = 0; i < 32; ++i) a += z[i];
                const int base = lane - g;
                float mu = 0.0f;
                for (int k = 0; k < G; ++k) mu += __shfl_sync(0xFFFFFFFFu, a, base + k);
                mu /= (float)s.dim;
                float b = 0.0f;
#pragma unroll
                for (int i = 0; i < 32; ++i) b += (z[i] - mu) * (z[i] - mu);
                float ss = 0.0f;
                for (int k = 0; k < G; ++k) ss += __shfl_sync(0xFFFFFFFFu, b, base + k);
                dev = sqrtf(ss / (float)(s.dim - s.ddof));
            }
            // (raw rows are stage inputs already: taken as they are, no deviation stored)
            const bool deg = s.raw ? !valid : (deviation_is_degenerate(dev) || !valid);
            if (p.defer_stats) smem[kOffFlags + rloc] = (uint8_t)((valid ? 1 : 0) | (deg ? 2 : 0));
#pragma unroll
            for (int i = 0; i < 32; ++i) z[i] = deg ? 0.0f : (s.raw ? z[i] : z[i] / dev);
            if (valid && g == 0 && !s.raw) {
                const uint16_t hb = deviation_is_degenerate(dev) ? (uint16_t)0 : __half_as_ushort(__float2half_rn(dev));
                p.std16[v] = hb;
                if (deviation_is_degenerate(dev)) ++n_degenerate;
                else if ((hb & 0x7FFFu) == 0 || (hb & 0x7FFFu) >= 0x7C00u) ++n_stdrange;
            }

#pragma unroll 1
            for (int r = 0; r < s.R && ok; ++r) {
                const StageParams prm = sp[r];
                const float *cbr = p.cb + (size_t)r * s.K * 32;
                // scaled half-precision copy of the residual -> A operand row; error window of this row
                float zz = 0.0f, zmax = 0.0f;
                {
                    uint32_t ab[32];                       // 16 words of head, 16 of remainder
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float z0 = z[2 * i] * prm.scale, z1 = z[2 * i + 1] * prm.scale;
                        zz = fmaf(z0, z0, zz); zz = fmaf(z1, z1, zz);
                        zmax = fmaxf(zmax, fmaxf(fabsf(z0), fabsf(z1)));
                        const __half2 h2 = __floats2half2_rn(z0, z1);
                        const float2 hf = __half22float2(h2);
                        const __half2 l2 = __floats2half2_rn(z0 - hf.x, z1 - hf.y);
                        ab[i] = *reinterpret_cast<const uint32_t *>(&h2);
                        ab[16 + i] = *reinterpret_cast<const uint32_t *>(&l2);
                    }
                    tmem_st32(taddr + 128, ab);
                }
                tc_fence_before();
                mbar_arrive(BAR(kBarAReady + tile));
                // park the float32 residual in shared memory for the sweep
#pragma unroll
                for (int i = 0; i < 32; ++i) z_park[i * kRowsPerPass] = z[i];
                Sweep w;
                w.win = 2.125f * (prm.a * sqrtf(zz) * 1.0001f + prm.b);    // 2 * bound, with slack for this arithmetic
                w.zz = zz;
                w.m1 = INFINITY; w.thr = INFINITY; w.cnt = 0;
#pragma unroll
                for (int q = 0; q < 16; ++q) w.d[q] = INFINITY;
                w.h[0] = w.h[1] = INFINITY;
                w.bb[0] = w.bb[1] = w.bb[2] = w.bb[3] = INFINITY;
                const bool force_scan = !(zmax < 60000.0f) || !(w.win < INFINITY);

#pragma unroll 1
                for (int c = 0; c < S && ok; ++c) {
                    if (c == S - 1 && w.cnt > 0) {
                        // Before the last chunk the running winner is the final one most of the time:
                        // start fetching its codeword while the MMA chain runs.
                        int pb = 0, pq = 0, ph = 0, pbb = 0;
#pragma unroll
                        for (int e = kListCap - 1; e >= 0; --e)
                            if (e < w.cnt && list_v[e * kRowsPerPass] == w.m1) pb = list_i[e * kRowsPerPass];
#pragma unroll
                        for (int q = 15; q >= 0; --q)
                            if (w.d[q] == w.m1) pq = q;
                        if (w.h[1] == w.m1 && w.h[0] != w.m1) ph = 1;
#pragma unroll
                        for (int i = 3; i > 0; --i)
                            if (w.bb[i] == w.m1) pbb = i;
                        const int pj = min(pb * 128 + pbb * 32 + 16 * ph + pq, s.K - 1);
                        asm volatile("prefetch.global.L1 [%0];" ::"l"(cbr + (size_t)pj * 32));
                    }
                    ok = mbar_wait(BAR(kBarAccFull + tile), chunk_use & 1u, abort_flag, p.wait_limit);
                    ok = __all_sync(0xFFFFFFFFu, ok);          // tcgen05.ld below needs the whole warp
                    ++chunk_use;
                    if (!ok) break;
                    tc_fence_after();
                    // All four 32-column blocks are asked for at once and the accumulator goes back to
                    // the MMA issuer as soon as they have landed: the reduction below runs while the
                    // next chain computes.
                    uint32_t ua[32], ub[32], uc[32], ud[32];
                    tmem_ld32_issue(taddr, ua);
                    tmem_ld32_issue(taddr + 32, ub);
                    tmem_ld32_issue(taddr + 64, uc);
                    tmem_ld32_issue(taddr + 96, ud);
                    tmem_ld_wait4(ua, ub, uc, ud);
                    tc_fence_before();
                    mbar_arrive(BAR(kBarAccFree + tile));        // the accumulator may be overwritten
                    const float c0 = fold_block(w, ua, 0);
                    const float c1 = fold_block(w, ub, 1);
                    const float c2 = fold_block(w, uc, 2);
                    const float c3 = fold_block(w, ud, 3);
                    list_block(w, fminf(min3(c0, c1, c2), c3), c, list_v, list_i, kRowsPerPass);
                }
                if (!ok) break;
                // take the residual back
#pragma unroll
                for (int i = 0; i < 32; ++i) z[i] = z_park[i * kRowsPerPass];
                const float m1 = w.m1;
                const int cnt = w.cnt;

                // ---- stage end: the columns that can still be the exact argmin are those of a listed
                // chunk, in a listed block of the chunk, in a listed half, at a listed place.  When each of
                // the four lists has one entry (almost always) that column is the choice: every other
                // column is farther than the approximation and float32 evaluation errors can bridge.
                const float lim = threshold(w, m1);
                int b1 = 0, nlisted = 0;
                {
                    bool found = false;
#pragma unroll
                    for (int e = 0; e < kListCap; ++e) {
                        const float fv = list_v[e * kRowsPerPass];
                        const int fi = list_i[e * kRowsPerPass];
                        const bool live = e < cnt;
                        if (live && fv <= lim) ++nlisted;
                        if (live && !found && fv == m1) { found = true; b1 = fi; }
                    }
                }
                uint32_t qmask = 0u, hmask = 0u, bmask = 0u;
                int q1 = 0, h1 = 0, bb1 = 0;
#pragma unroll
                for (int i = 3; i >= 0; --i) {
                    if (w.bb[i] <= lim) bmask |= 1u << i;
                    if (w.bb[i] == m1) bb1 = i;
                }
#pragma unroll
                for (int q = 15; q >= 0; --q) {
                    if (w.d[q] <= lim) qmask |= 1u << q;
                    if (w.d[q] == m1) q1 = q;
                }
#pragma unroll
                for (int c = 1; c >= 0; --c) {
                    if (w.h[c] <= lim) hmask |= 1u << c;
                    if (w.h[c] == m1) h1 = c;
                }
                const int j1 = b1 * 128 + bb1 * 32 + 16 * h1 + q1;
                // (a padded column scores 60000: if nothing real scored less, scan everything)
                const bool scan_all = force_scan || cnt == 0 || cnt > kListCap || !(m1 < 59000.0f);
                const bool unique = nlisted == 1 && (qmask & (qmask - 1u)) == 0u && (hmask & (hmask - 1u)) == 0u &&
                                    (bmask & (bmask - 1u)) == 0u && j1 < s.K;
                const bool flagged = !deg && (scan_all || !unique);
                int bj = j1 < s.K ? j1 : 0;
                // Rows with more than one candidate: the whole warp re-scores the candidate columns of
                // every listed block of one such row at a time (lane = place in the block; all columns
                // when the list overflowed) exactly in float32, direct form, then reduces to the
                // smallest distance, lowest index on ties.
                uint32_t todo = __ballot_sync(0xFFFFFFFFu, flagged);
                while (todo) {
                    const int src = __ffs(todo) - 1;
                    todo &= todo - 1;
                    float zs[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) zs[i] = z_park[i * kRowsPerPass + (src - lane)];
                    const float lim_s = __shfl_sync(0xFFFFFFFFu, lim, src);
                    const int cnt_s = __shfl_sync(0xFFFFFFFFu, cnt, src);
                    const uint32_t qmask_s = __shfl_sync(0xFFFFFFFFu, qmask, src);
                    const uint32_t hmask_s = __shfl_sync(0xFFFFFFFFu, hmask, src);
                    const uint32_t bmask_s = __shfl_sync(0xFFFFFFFFu, bmask, src);
                    const bool all_s = __shfl_sync(0xFFFFFFFFu, (int)scan_all, src) != 0;
                    const int row_s = rloc - lane + src;
                    const bool mine = ((qmask_s >> (lane & 15)) & 1u) && ((hmask_s >> (lane >> 4)) & 1u);
                    float bv = INFINITY;
                    int bi = 0x7FFFFFFF;
                    if (all_s) {
                        for (int j = lane; j < s.K; j += 32) {
                            const float dj = exact_distance(zs, cbr + (size_t)j * 32);
                            if (dj < bv) { bv = dj; bi = j; }
                        }
                    } else {
                        for (int e = 0; e < cnt_s; ++e) {
                            const float fv = reinterpret_cast<const float *>(smem + kOffListV)[e * kRowsPerPass + row_s];
                            if (!(fv <= lim_s)) continue;                              // warp-uniform
                            const int j0 = (int)reinterpret_cast<const uint16_t *>(smem + kOffListI)[e * kRowsPerPass + row_s] * 128 + lane;
                            for (int i = 0; i < 4; ++i) {
                                const int j = j0 + 32 * i;
                                if (((bmask_s >> i) & 1u) && mine && j < s.K) {     // (the block test is warp-uniform)
                                    const float dj = exact_distance(zs, cbr + (size_t)j * 32);
                                    if (dj < bv) { bv = dj; bi = j; }
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) {
                        const float ov = __shfl_xor_sync(0xFFFFFFFFu, bv, off);
                        const int oi = __shfl_xor_sync(0xFFFFFFFFu, bi, off);
                        if (ov < bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                    }
                    if (lane == src) {
                        bj = bi < s.K ? bi : 0;
                        if (all_s) ++n_exhaustive; else ++n_rescored;
                    }
                }
                if (deg) bj = 0;
                if (p.stat_sum && valid && !(p.defer_stats && r < s.R - 1)) {
                    // EMA statistics (Section 3): this row's stage input joins the bin of its code
                    // (all stages but the last are the issuer warps' when deferred)
                    const size_t bin = (size_t)r * s.K + bj;
                    atomicAdd(p.stat_cnt + bin, 1u);
                    if (!deg) {
                        float4 *m = reinterpret_cast<float4 *>(p.stat_sum + bin * 32);
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            atomicAdd(m + q, make_float4(z[4 * q], z[4 * q + 1], z[4 * q + 2], z[4 * q + 3]));
                    }
                }
                if (!deg) {
                    const float *ew = cbr + (size_t)bj * 32;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float ev[8];
                        ldg256(ew + 8 * q, ev);
#pragma unroll
                        for (int k = 0; k < 8; ++k) z[8 * q + k] -= ev[k];
                    }
                }
                if (p.energy) {
                    // squared norm of the residual leaving this stage (scaled units), summed over the
                    // warp's rows: one atomic per warp and stage
                    float e2 = 0.0f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) e2 = fmaf(z[i], z[i], e2);
                    if (!valid) e2 = 0.0f;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) e2 += __shfl_xor_sync(0xFFFFFFFFu, e2, off);
                    if (lane == 0) atomicAdd(p.energy + r, e2);
                }
                codes_s[rloc * 16 + r] = (uint16_t)bj;
            }
            if (!ok) break;

            // ---- emit the codes of this pass (Section 3.2 storage)
            __syncwarp();
            if (s.bits == 16) {
                if (valid) {
                    uint16_t *o = reinterpret_cast<uint16_t *>(p.codes) + (v * G + g) * s.R;
                    if (s.R == 8) {
                        *reinterpret_cast<uint4 *>(o) = *reinterpret_cast<const uint4 *>(codes_s + rloc * 16);
                    } else {
                        for (int r = 0; r < s.R; ++r) o[r] = codes_s[rloc * 16 + r];
                    }
                }
            } else {
                // lanes of this warp hold 32 / G whole head vectors; one 32-bit word per lane and step
                const int words = s.code_bytes / 4, vec_per_warp = 32 / G;
                const int wrow0 = rloc - lane;
                for (int t = lane; t < vec_per_warp * words; t += 32) {
                    const int vl = t / words, w = t - vl * words;
                    const int64_t vv = (row0 + q4 * 32) / G + vl;
                    if (vv >= p.n) continue;
                    uint32_t word = 0;
                    const int k_lo = (32 * w) / s.bits, k_hi = min(s.per_vector - 1, (32 * w + 31) / s.bits);
                    for (int k = k_lo; k <= k_hi; ++k) {
                        const int gg = k / s.R, rr = k - gg * s.R;
                        const uint32_t val = codes_s[(wrow0 + vl * G + gg) * 16 + rr];
                        const int sh = k * s.bits - 32 * w;
                        word |= sh >= 0 ? (val << sh) : (val >> (-sh));
                    }
                    reinterpret_cast<uint32_t *>(p.codes)[vv * words + w] = word;
                }
            }
            __syncwarp();
        }
        if (p.st) {
            if (n_rescored) atomicAdd(&p.st->rescored_rows, n_rescored);
            if (n_exhaustive) atomicAdd(&p.st->exhaustive_rows, n_exhaustive);
            if (n_degenerate) atomicAdd(&p.st->degenerate_vectors, n_degenerate);
            if (n_stdrange) atomicAdd(&p.st->std_out_of_half, n_stdrange);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kEpiThreads / 32) {
        tc_fence_after();
        if (lane == 0 && *abort_flag && p.st) atomicAdd(&p.st->wait_timeouts, 1u);
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
    }
}

}  // namespace

bool encode_tensor_supported(const Shape &s)
{
    return s.gd == 32 && s.G <= 32 && (s.G & (s.G - 1)) == 0 && slots_per_stage(s.K) * 4 <= 65535;
}

// Stages 0 .. this - 1 of the fused statistics hold the sums of what those stages LEFT (their bins' inputs
// minus count * codeword): the caller adds count * codeword (launch_stats_finish).
int encode_tensor_deferred_stages(const Shape &s)
{
    return encode_tensor_supported(s) && slots_per_stage(s.K) >= kDeferMinSlots && s.R > 1 ? s.R - 1 : 0;
}

int launch_encode_tensor(const Shape &s, const void *x, int64_t n, int64_t stride, const float *cb,
                         const void *prepared, void *codes, uint16_t *std16, rvq_status *st,
                         cudaStream_t stream, uint32_t *stat_cnt, float *stat_sum, float *energy,
                         uint32_t wait_limit, int drop_last_chain)
{
    if (n == 0) return RVQ_OK;
    const int64_t rows = n * s.G;
    const int64_t tiles = (rows + 127) / 128;
    if (tiles > 0x7FFFFFFF) return RVQ_ERR_UNSUPPORTED;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return RVQ_ERR_DEVICE;
    if (cudaFuncSetAttribute(encode_tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
        return RVQ_ERR_LAUNCH;
    Params p{s, x, n, stride, cb, reinterpret_cast<const uint8_t *>(prepared), codes, std16, st, (int)tiles, stat_cnt, stat_sum,
             energy, wait_limit ? wait_limit : kWaitLimit, drop_last_chain,
             stat_sum != nullptr && encode_tensor_deferred_stages(s) > 0 ? 1 : 0};
    const int64_t groups = (tiles + kTiles - 1) / kTiles;
    const int grid = (int)(groups < sms ? groups : sms);
    encode_tensor_kernel<<<grid, kThreads, kSmemBytes, stream>>>(p);
    return check_launch();
}

}  // namespace rvq
