// Stage 2 as one persistent kernel (bf16, head_dim 128, window 32, four query heads per KV
// head, i.e. the 128 window rows of a KV head fill one tcgen05 tile).
//
// The softmax normaliser of a window row (Eq. 2) depends on every key, so the scores need two
// sweeps over K: sweep A accumulates, per window row, sum_j exp(logit_j) over its causal keys;
// sweep B recomputes the logits, normalises, and reduces over heads and window positions per
// token (Eqs. 3, 4 and the per-token entropy of Eq. 6).  The kernel walks "phases" = (problem,
// KV head).  A CTA owns a fixed set of token tiles of its problem and, for phase n, interleaves
// sweep A of phase n with sweep B of phase n-1, so that the second read of a KV head's keys
// (33.5 MB at 128K tokens) comes out of L2 shortly after the first one pulled them from HBM.
// Between the sweeps the row sums of all CTAs of the problem are merged into log-sum-exps by
// dedicated merge warps; CTAs hand over through two counters per phase in global memory,
// every wait on them bounded.
//
// Both sweeps are the same 128 x 128 x 128 product on the tensor cores with the operand roles
// swapped: sweep A computes Q_g K^T (TMEM lane = window row, the running sum is thread-local),
// sweep B computes K Q_g^T (TMEM lane = token, the sums over heads and window positions are
// thread-local).  The head-summed attention \bar A[w, t] of the CTA's tokens lives in tensor
// memory (32 columns per token tile) across the KV heads of a layer, so neither the H x W x T
// attention tensor nor \bar A ever reaches shared or global memory.
//
// CTA = 11 warps: warp 0 TMA producer, warp 1 MMA issuer (owns tensor memory), warps 2-9
// epilogue (two warps per 32-lane quarter of tensor memory; in sweep A they split a tile's
// 128 token columns, in sweep B the 32 window positions), warp 10 merges row statistics.
#pragma once
#include "common.cuh"
#include "score_simt.cuh"
#include "score_tc.cuh"

namespace sab {

constexpr int kFuThreads = 352;
constexpr int kFuEpiWarp0 = 2;
constexpr int kFuEpiThreads = 256;
constexpr int kFuMergeWarp = 10;
constexpr int kFuStages = 4;                 // K tile ring
constexpr int kFuMaxTilesPerCta = 7;         // \bar A slots in tensor memory: 7 x 32 columns
constexpr int kFuAbarCol0 = 256;             // columns [0, 256): two logit accumulators
constexpr int kFuTmemCols = 512;
constexpr int kFuLead = 3;                   // sweep A runs this many tiles ahead of sweep B
constexpr int kFuPartSlots = 4;              // ring of per-phase partial buffers
constexpr int kFuMaxCtasDev = 256;           // upper bound on the CTAs of one launch
constexpr int kFuTileBytes = 2 * kAtomBytes; // 128 rows x 128 bf16
constexpr int kFuSmemBytes = 1024 + (2 + kFuStages) * kFuTileBytes;

struct FusedArgs {
    int cpp;                 // CTAs per group (one group works on one problem at a time)
    int n_groups;
    int n_prob;
    float c2;                // log2(e) / sqrt(D)
    float eps;
    float2* part;            // [n_groups][kFuPartSlots][cpp][2][128] row statistics (m, l)
    float* lse2;             // [n_prob][Hkv * 128] log2-sum-exp2 per window row
    int* arrive;             // [n_prob][Hkv]
    int* done;               // [n_prob][Hkv]
    float* s_out;            // [n_layers][total_tokens]
    float* e_out;
    int* status;
};

// Optional cycle-stamp trace of a few CTAs (compiled in with -DSABLOCK_TRACE; off otherwise):
// role 0 = TMA producer, 1 = MMA issuer, 2 / 3 = leader thread of epilogue set 0 / 1.
#ifdef SABLOCK_TRACE
constexpr int kTraceOps = 600;
__device__ long long g_trace[4][4][kTraceOps][4];   // [traced CTA][role][op][event]
#define FU_TRACE(role, n, ev)                                                                 \
    do {                                                                                      \
        if (tslot >= 0 && (n) < kTraceOps) g_trace[tslot][role][n][ev] = clock64();           \
    } while (0)
#else
#define FU_TRACE(role, n, ev) do { } while (0)
#endif

struct FuBarriers {
    uint64_t full[kFuStages];
    uint64_t empty[kFuStages];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint64_t qfull[2];
    uint64_t qempty[2];
    uint64_t sbar[2];        // the four warps of one epilogue set
    uint32_t tmem_base;
    int abort_flag;
};

// One step of a CTA's work list.
enum { kOpA = 0, kOpB = 1, kOpPairEnd = 2, kOpStop = 3 };

// What a role needs to know about one phase = (problem, KV head).
struct FuPhase {
    int phase;       // phase counter of the group; -1 = none
    int prob, j;     // problem index and KV head
    int layer, seq;
    int L, Tn;       // sequence length and compressible length
    int tok_base;    // first packed token row of the sequence
    int n_tiles;     // tiles of this CTA in the sweep in question
};

struct FuOp {
    int kind;
    int k;           // which of the CTA's tiles (slot of \bar A in tensor memory)
    int tile;        // token tile index inside the sequence
    int last;        // last tile of this kind for this CTA in this phase
    int pair;        // for kOpPairEnd: the pair that ended
};

// Deterministic walk over the work list; every role of the CTA runs its own copy.  Pair n holds
// the sweep A tiles of phase n (`pa`) and the sweep B tiles of phase n - 1 (`pb`); all divisions
// happen when a pair begins, the per-tile step is a few adds and compares.
struct FuIter {
    const Geo& g;
    int cpp, n_groups, group, rank;
    int n_phases;            // phases of this group
    int pair, ia, ib;
    FuPhase pa, pb;
    __device__ FuIter(const Geo& geo, const FusedArgs& a) : g(geo), cpp(a.cpp), n_groups(a.n_groups)
    {
        group = blockIdx.x / cpp;
        rank = blockIdx.x % cpp;
        const int my_probs = group < n_groups ? (a.n_prob - group + n_groups - 1) / n_groups : 0;
        n_phases = my_probs * g.Hkv;
        pair = 0; ia = ib = 0;
        pb.phase = -1; pb.n_tiles = 0;
        load_a();
    }
    __device__ int my_tiles(int n) const { return rank < n ? (n - rank + cpp - 1) / cpp : 0; }
    __device__ void load_a()
    {
        pa.phase = pair;
        pa.n_tiles = 0;
        if (pair >= n_phases) { pa.phase = -1; return; }
        pa.prob = group + (pair / g.Hkv) * n_groups;
        pa.j = pair % g.Hkv;
        pa.layer = pa.prob / g.n_seqs;
        pa.seq = pa.prob % g.n_seqs;
        pa.tok_base = g.cu[pa.seq];
        pa.L = g.cu[pa.seq + 1] - pa.tok_base;
        pa.Tn = pa.L - g.window;
        if (pa.L > g.n_out) pa.n_tiles = my_tiles((pa.L + kTcTile - 1) / kTcTile);   // else: returned unchanged
    }
    __device__ void next_pair()
    {
        pb = pa;
        pb.n_tiles = (pa.phase >= 0 && pa.L > g.n_out) ? my_tiles((pa.Tn + kTcTile - 1) / kTcTile) : 0;
        ++pair; ia = ib = 0;
        load_a();
    }
    __device__ FuOp next()
    {
        FuOp op;
        op.pair = pair;
        if (pair > n_phases) { op.kind = kOpStop; return op; }
        const bool take_a = ia < pa.n_tiles && (ia < ib + kFuLead || ib >= pb.n_tiles);
        if (take_a) {
            op.kind = kOpA; op.k = ia; op.last = ia == pa.n_tiles - 1;
            op.tile = rank + ia * cpp;
            ++ia;
            return op;
        }
        if (ib < pb.n_tiles) {
            op.kind = kOpB; op.k = ib; op.last = ib == pb.n_tiles - 1;
            op.tile = rank + ib * cpp;
            ++ib;
            return op;
        }
        op.kind = kOpPairEnd;
        next_pair();
        return op;
    }
};

// ---- small PTX helpers used only here -------------------------------------------------------
// Barrier among a fixed group of threads built on an mbarrier, so that the wait is bounded and
// gives up when the CTA is aborting.  `n` counts the uses of this barrier by the calling thread.
__device__ __forceinline__ bool group_sync(uint64_t* bar, int& n, volatile int* abort_flag)
{
    mbar_arrive(smem_u32(bar));
    const bool ok = mbar_wait(smem_u32(bar), (uint32_t)(n & 1), abort_flag);
    ++n;
    return ok && !*abort_flag;
}
__device__ __forceinline__ int ld_acquire(const int* p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
          "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
          "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
          "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
          "r"(__float_as_uint(v[15]))
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
          "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
          "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
          "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
          "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])),
          "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])),
          "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
          "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])),
          "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])),
          "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait()
{
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Bounded wait until *ctr >= target.  Gives up after about a second, or as soon as another
// role of the CTA or another CTA has reported a failure.
__device__ __forceinline__ bool wait_counter(const int* ctr, int target, volatile int* abort_flag, const int* status)
{
    if (ld_acquire(ctr) >= target) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (true) {
        if (ld_acquire(ctr) >= target) return true;
        __nanosleep(64);
        if ((++spins & 15) == 0) {
            if (*abort_flag || ld_acquire(status) != 0 || clock64() - t0 > kWaitLimitCycles) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}

// Sum of exp2(v * c2 - m) over 32 logits of one window row.
__device__ __forceinline__ float chunk_expsum(const uint32_t (&r)[32], float c2, float m)
{
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        s0 += ex2_approx(fmaf(__uint_as_float(r[i + 0]), c2, -m));
        s1 += ex2_approx(fmaf(__uint_as_float(r[i + 1]), c2, -m));
        s2 += ex2_approx(fmaf(__uint_as_float(r[i + 2]), c2, -m));
        s3 += ex2_approx(fmaf(__uint_as_float(r[i + 3]), c2, -m));
    }
    return (s0 + s1) + (s2 + s3);
}
__device__ __forceinline__ float chunk_max(const uint32_t (&r)[32])
{
    float a = fmaxf(__uint_as_float(r[0]), __uint_as_float(r[1]));
    float b = fmaxf(__uint_as_float(r[2]), __uint_as_float(r[3]));
#pragma unroll
    for (int i = 4; i < 32; i += 2) {
        a = fmaxf(a, __uint_as_float(r[i]));
        b = fmaxf(b, __uint_as_float(r[i + 1]));
    }
    return fmaxf(a, b);
}
// Causal mask of 32 logits of window row w: keys beyond position lim = T + w do not exist for it.
__device__ __forceinline__ void chunk_mask(uint32_t (&r)[32], int tok0, int lim)
{
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if (tok0 + i > lim) r[i] = 0xff800000u;       // -inf
}

// Running sum of exp2 over the keys of one window row, kept as l * 2^m with an integer-valued
// reference exponent m that only moves when the sum would leave the fp32 range.
struct RowSum {
    float m, l;
    bool have_m;
    __device__ void reset() { m = 0.f; l = 0.f; have_m = false; }
    __device__ void add(const uint32_t (&r0)[32], const uint32_t (&r1)[32], float c2)
    {
        if (!have_m) {
            const float mx = fmaxf(chunk_max(r0), chunk_max(r1)) * c2;
            m = (mx == -INFINITY) ? 0.f : ceilf(mx);
            have_m = true;
        }
        float c = chunk_expsum(r0, c2, m) + chunk_expsum(r1, c2, m);
        if (!(l + c < 1.8e19f)) {                          // far above the reference: move it
            const float mx = fmaxf(chunk_max(r0), chunk_max(r1)) * c2;
            const float m_new = fmaxf(m, ceilf(mx));
            l *= exp2f(m - m_new);
            m = m_new;
            c = chunk_expsum(r0, c2, m) + chunk_expsum(r1, c2, m);
        }
        l += c;
    }
};

// accw[w] += exp2(logit * c2 - lse) for two heads' 32 window positions each (64 logits).
__device__ __forceinline__ void accumulate_heads(float (&accw)[32], const uint32_t (&r0)[32], const uint32_t (&r1)[32],
                                                 const float* lse0, float c2)
{
    const float4* l4 = reinterpret_cast<const float4*>(lse0);
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        const float4 ls = l4[i >> 2];
        accw[i + 0] += ex2_approx(fmaf(__uint_as_float(r0[i + 0]), c2, -ls.x));
        accw[i + 1] += ex2_approx(fmaf(__uint_as_float(r0[i + 1]), c2, -ls.y));
        accw[i + 2] += ex2_approx(fmaf(__uint_as_float(r0[i + 2]), c2, -ls.z));
        accw[i + 3] += ex2_approx(fmaf(__uint_as_float(r0[i + 3]), c2, -ls.w));
    }
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        const float4 ls = l4[8 + (i >> 2)];
        accw[i + 0] += ex2_approx(fmaf(__uint_as_float(r1[i + 0]), c2, -ls.x));
        accw[i + 1] += ex2_approx(fmaf(__uint_as_float(r1[i + 1]), c2, -ls.y));
        accw[i + 2] += ex2_approx(fmaf(__uint_as_float(r1[i + 2]), c2, -ls.z));
        accw[i + 3] += ex2_approx(fmaf(__uint_as_float(r1[i + 3]), c2, -ls.w));
    }
}

__global__ void __launch_bounds__(kFuThreads, 1)
score_fused_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const Geo g,
               const FusedArgs fa)
{
    extern __shared__ uint8_t dyn_smem[];
    __shared__ FuBarriers sh;
    __shared__ __align__(16) float lse_s[2][2][128];     // [epilogue set][phase parity][window row]
    const uint32_t base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    const uint32_t q_smem = base;                                  // two query blocks
    const uint32_t k_smem = base + 2 * kFuTileBytes;               // K tile ring

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0 && lane == 0) {
        for (int i = 0; i < kFuStages; ++i) {
            mbar_init(smem_u32(&sh.full[i]), 1);
            mbar_init(smem_u32(&sh.empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh.tfull[i]), 1);
            mbar_init(smem_u32(&sh.tempty[i]), 128);
            mbar_init(smem_u32(&sh.qfull[i]), 1);
            mbar_init(smem_u32(&sh.qempty[i]), 1);
            mbar_init(smem_u32(&sh.sbar[i]), 128);
        }
        sh.abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        __syncwarp();
        tmem_alloc(smem_u32(&sh.tmem_base), kFuTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort_flag;
    constexpr int R = 128;                           // window rows per KV head
#ifdef SABLOCK_TRACE
    const int tslot = blockIdx.x == 0 ? 0 : blockIdx.x == 5 ? 1 : blockIdx.x == 77 ? 2 : blockIdx.x == gridDim.x - 1 ? 3 : -1;
#endif

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            const uint64_t pol_a = l2_policy_evict_last();     // first read: keep for sweep B
            const uint64_t pol_b = l2_policy_evict_first();    // second read: last use
            const uint64_t pol_q = l2_policy_evict_last();
            FuIter it(g, fa);
            int n_ops = 0, qloads[2] = {0, 0}, q_phase = -1;
            while (true) {
                const FuOp op = it.next();
                if (op.kind == kOpStop) break;
                if (op.kind == kOpPairEnd) continue;
                const FuPhase& ph = op.kind == kOpA ? it.pa : it.pb;
                if (op.kind == kOpA && ph.phase != q_phase) {      // first tile of a phase: its query block
                    q_phase = ph.phase;
                    const int b = ph.phase & 1;
                    if (qloads[b] > 0 && !mbar_wait(smem_u32(&sh.qempty[b]), (qloads[b] - 1) & 1, abort_flag)) break;
                    ++qloads[b];
                    mbar_expect_tx(smem_u32(&sh.qfull[b]), kFuTileBytes);
                    for (int a = 0; a < 2; ++a)
                        tma_load_2d(q_smem + b * kFuTileBytes + a * kAtomBytes, &tmQ, smem_u32(&sh.qfull[b]), a * 64,
                                    ph.prob * g.H * g.window + ph.j * R, pol_q);
                }
                const int st = n_ops % kFuStages, par = (n_ops / kFuStages) & 1;
                FU_TRACE(0, n_ops, 0);
                if (!mbar_wait(smem_u32(&sh.empty[st]), par ^ 1, abort_flag)) break;
                FU_TRACE(0, n_ops, 1);
                mbar_expect_tx(smem_u32(&sh.full[st]), kFuTileBytes);
                for (int a = 0; a < 2; ++a)
                    tma_load_4d(k_smem + st * kFuTileBytes + a * kAtomBytes, &tmK, smem_u32(&sh.full[st]), a * 64, ph.j,
                                ph.tok_base + op.tile * kTcTile, ph.layer, op.kind == kOpA ? pol_a : pol_b);
                ++n_ops;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            FuIter it(g, fa);
            int n_ops = 0, qwaits[2] = {0, 0}, q_phase = -1;
            bool q_used[2] = {false, false};     // does the phase of that parity hold a query block
            while (true) {
                const FuOp op = it.next();
                if (op.kind == kOpStop) break;
                if (op.kind == kOpPairEnd) {
                    // the query block of phase (pair - 1) has seen its last product
                    const int b = (op.pair - 1) & 1;
                    if (op.pair >= 1 && q_used[b]) {
                        tc_commit(smem_u32(&sh.qempty[b]));
                        q_used[b] = false;
                    }
                    continue;
                }
                const FuPhase& ph = op.kind == kOpA ? it.pa : it.pb;
                const int b = ph.phase & 1;
                if (op.kind == kOpA && ph.phase != q_phase) {
                    q_phase = ph.phase;
                    if (!mbar_wait(smem_u32(&sh.qfull[b]), qwaits[b] & 1, abort_flag)) break;
                    ++qwaits[b];
                    q_used[b] = true;
                }
                const int st = n_ops % kFuStages, par = (n_ops / kFuStages) & 1;
                const int acc = n_ops & 1, aph = (n_ops >> 1) & 1;
                FU_TRACE(1, n_ops, 0);
                if (!mbar_wait(smem_u32(&sh.tempty[acc]), aph ^ 1, abort_flag)) break;
                FU_TRACE(1, n_ops, 1);
                if (!mbar_wait(smem_u32(&sh.full[st]), par, abort_flag)) break;
                FU_TRACE(1, n_ops, 2);
                tc_fence_after();
                const uint32_t kt = k_smem + st * kFuTileBytes, qt = q_smem + b * kFuTileBytes;
                if (op.kind == kOpA) tc_issue_tile(tmem, acc, qt, kt, 8);     // rows = window rows
                else                 tc_issue_tile(tmem, acc, kt, qt, 8);     // rows = tokens
                tc_commit(smem_u32(&sh.empty[st]));
                tc_commit(smem_u32(&sh.tfull[acc]));
                ++n_ops;
            }
        }
    } else if (warp == kFuMergeWarp) {
        // ------------------------------------------------------------------ row-statistics merge
        FuIter it(g, fa);
        const int group = it.group, rank = it.rank;
        for (int phase = 0; phase < it.n_phases; ++phase) {
            const int prob = group + (phase / g.Hkv) * fa.n_groups, j = phase % g.Hkv, seq = prob % g.n_seqs;
            if (geo_identity(g, seq)) continue;
            const int nt1 = (geo_L(g, seq) + kTcTile - 1) / kTcTile;
            const int n_src = 2 * min(fa.cpp, nt1);             // (CTA that holds tiles, epilogue set)
            if (rank >= R) continue;
            bool ok = true;
            if (lane == 0) ok = wait_counter(fa.arrive + prob * g.Hkv + j, n_src, abort_flag, fa.status);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            const float2* pp = fa.part + ((size_t)group * kFuPartSlots + (phase % kFuPartSlots)) * fa.cpp * 2 * R;
            for (int row = rank; row < R; row += fa.cpp) {
                // partial i = (source CTA, epilogue set), merged in index order; all loads of a
                // lane are issued before the first use so that their latencies overlap
                constexpr int kPer = 2 * kFuMaxCtasDev / 32;
                float2 v[kPer];
#pragma unroll
                for (int u = 0; u < kPer; ++u) {
                    const int i = lane + 32 * u;
                    v[u] = i < n_src ? __ldcg(pp + (size_t)i * R + row) : make_float2(0.f, 0.f);
                }
                float m = -INFINITY;
#pragma unroll
                for (int u = 0; u < kPer; ++u)
                    if (v[u].y > 0.f) m = fmaxf(m, v[u].x);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                float l = 0.f;
#pragma unroll
                for (int u = 0; u < kPer; ++u)
                    if (v[u].y > 0.f) l += v[u].y * exp2f(v[u].x - m);
                l = warp_sum(l);
                if (lane == 0) fa.lse2[(size_t)prob * g.H * g.window + j * R + row] = m + log2f(l);
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence();
                atomicAdd(fa.done + prob * g.Hkv + j, 1);
            }
        }
    } else if (warp >= kFuEpiWarp0 && warp < kFuEpiWarp0 + 8) {
        // ------------------------------------------------------------------ epilogue
        // Two sets of four warps; set s takes the tiles whose logits land in accumulator s, so
        // the sets run half a tile out of step and one computes while the other waits and loads.
        const int ew = warp - kFuEpiWarp0;
        const int q4 = warp & 3;                       // tensor-memory lane quarter of this warp
        const int set = ew >> 2;
        const int row = q4 * 32 + lane;                // TMEM lane: window row (sweep A) or token (sweep B)
        const bool leader = (ew & 3) == 0 && lane == 0;
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t acc_addr = lane_addr + (uint32_t)set * 128u;
        const float c2 = fa.c2;
        const float inv_H = 1.f / (float)g.H;
        const int n_mergers = min(fa.cpp, R);
        FuIter it(g, fa);
        const int group = it.group, rank = it.rank;
        RowSum rs;                                     // sweep A state of this window row in this set
        rs.reset();
        int n_ops = 0, n_mine = 0, lse_phase = -1, n_sync = 0;
        while (true) {
            const FuOp op = it.next();
            if (op.kind == kOpStop) break;
            if (op.kind == kOpPairEnd) continue;
            const bool mine = (n_ops & 1) == set;
            ++n_ops;
            if (op.kind == kOpA) {
                const FuPhase& ph = it.pa;
                if (mine) {
                    if (leader) FU_TRACE(2 + set, n_mine, 0);
                    if (!mbar_wait(smem_u32(&sh.tfull[set]), n_mine & 1, abort_flag)) break;
                    if (leader) FU_TRACE(2 + set, n_mine, 1);
                    tc_fence_after();
                    const int tok0 = op.tile * kTcTile;
                    const int lim = ph.Tn + (row & 31);            // causal: key index <= T + w (Eq. 2)
                    const bool need_mask = tok0 + 127 > ph.Tn;
                    uint32_t r0[32], r1[32];
                    tmem_ld32_issue(acc_addr, r0);
                    tmem_ld32_issue(acc_addr + 32, r1);
                    tmem_ld_wait();
                    if (need_mask) { chunk_mask(r0, tok0, lim); chunk_mask(r1, tok0 + 32, lim); }
                    rs.add(r0, r1, c2);
                    tmem_ld32_issue(acc_addr + 64, r0);
                    tmem_ld32_issue(acc_addr + 96, r1);
                    tmem_ld_wait();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&sh.tempty[set]));        // logits are in registers: release the accumulator
                    if (leader) FU_TRACE(2 + set, n_mine, 2);
                    if (need_mask) { chunk_mask(r0, tok0 + 64, lim); chunk_mask(r1, tok0 + 96, lim); }
                    rs.add(r0, r1, c2);
                    if (leader) FU_TRACE(2 + set, n_mine, 3);
                    ++n_mine;
                }
                if (op.last) {
                    // Publish this set's row sums of the phase.  The partial buffers are a ring over
                    // phases: the slot is free once every merge of the phase that used it last is
                    // done.  (A CTA that also runs sweep B is throttled by it anyway; one that owns
                    // only a window tile is not.)
                    if (leader && ph.phase >= kFuPartSlots) {
                        const int old = ph.phase - kFuPartSlots;
                        wait_counter(fa.done + (group + (old / g.Hkv) * fa.n_groups) * g.Hkv + old % g.Hkv, n_mergers,
                                     abort_flag, fa.status);
                    }
                    if (!group_sync(&sh.sbar[set], n_sync, abort_flag)) break;
                    float2* pp = fa.part + ((size_t)group * kFuPartSlots + (ph.phase % kFuPartSlots)) * fa.cpp * 2 * R;
                    pp[((size_t)rank * 2 + set) * R + row] = make_float2(rs.m, rs.l);
                    __threadfence();
                    if (!group_sync(&sh.sbar[set], n_sync, abort_flag)) break;
                    if (leader) atomicAdd(fa.arrive + ph.prob * g.Hkv + ph.j, 1);
                    rs.reset();
                }
            } else if (mine) {
                const FuPhase& ph = it.pb;
                if (ph.phase != lse_phase) {                       // log-sum-exps of this phase
                    lse_phase = ph.phase;
                    if (leader) wait_counter(fa.done + ph.prob * g.Hkv + ph.j, n_mergers, abort_flag, fa.status);
                    if (!group_sync(&sh.sbar[set], n_sync, abort_flag)) break;
                    lse_s[set][ph.phase & 1][row] = __ldcg(fa.lse2 + (size_t)ph.prob * g.H * g.window + ph.j * R + row);
                    if (!group_sync(&sh.sbar[set], n_sync, abort_flag)) break;
                }
                if (leader) FU_TRACE(2 + set, n_mine, 0);
                if (!mbar_wait(smem_u32(&sh.tfull[set]), n_mine & 1, abort_flag)) break;
                if (leader) FU_TRACE(2 + set, n_mine, 1);
                tc_fence_after();
                const float* lj = lse_s[set][ph.phase & 1];
                float accw[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) accw[i] = 0.f;
                uint32_t r0[32], r1[32];
                tmem_ld32_issue(acc_addr, r0);                     // query heads 0, 1 of the group
                tmem_ld32_issue(acc_addr + 32, r1);
                tmem_ld_wait();
                accumulate_heads(accw, r0, r1, lj, c2);
                tmem_ld32_issue(acc_addr + 64, r0);                // query heads 2, 3
                tmem_ld32_issue(acc_addr + 96, r1);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(smem_u32(&sh.tempty[set]));
                if (leader) FU_TRACE(2 + set, n_mine, 2);
                accumulate_heads(accw, r0, r1, lj + 64, c2);
                const int n_this = n_mine;
                ++n_mine;
                // \bar A of this token tile, summed over the KV heads seen so far
                const uint32_t abar_addr = lane_addr + (uint32_t)(kFuAbarCol0 + op.k * 32);
                if (ph.j > 0) {
                    tmem_ld32_issue(abar_addr, r0);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) accw[i] += __uint_as_float(r0[i]);
                }
                if (ph.j < g.Hkv - 1) {
                    tmem_st32(abar_addr, accw);
                    tmem_st_wait();
                    tc_fence_before();         // the next head's update may come from the other set's warps
                } else {
                    // last KV head of the layer: s_t (Eqs. 3, 4) and the entropy of Eq. 6
                    float t0 = 0.f, t1 = 0.f, t2 = 0.f, t3 = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; i += 4) { t0 += accw[i]; t1 += accw[i + 1]; t2 += accw[i + 2]; t3 += accw[i + 3]; }
                    const float tot = (t0 + t1) + (t2 + t3);
                    float ent = 0.f;
                    if (tot > 0.f) {
                        const float inv = 1.f / tot;
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float ah = accw[i] * inv;                       // \hat A (Eq. 6)
                            ent -= ah * (lg2_approx(ah + fa.eps) * 0.6931471805599453f);
                        }
                    }
                    const int t = op.tile * kTcTile + row;
                    if (t < ph.Tn) {
                        const size_t off = (size_t)ph.layer * g.total_tokens + ph.tok_base;
                        fa.s_out[off + t] = tot * inv_H;
                        fa.e_out[off + t] = ent;
                    }
                }
                if (leader) FU_TRACE(2 + set, n_this, 3);
                (void)n_this;
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (sh.abort_flag) {
        if (threadIdx.x == 0) atomicOr(fa.status, kStatTimeout);
        long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }       // let copies and products in flight land
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, kFuTmemCols);
    }
}

}  // namespace sab
