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
constexpr int kFuLead = 2;                   // sweep A runs this many tiles ahead of sweep B
constexpr int kFuPartSlots = 4;              // ring of per-phase partial buffers
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

struct FuBarriers {
    uint64_t full[kFuStages];
    uint64_t empty[kFuStages];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint64_t qfull[2];
    uint64_t qempty[2];
    uint64_t ebar;           // all epilogue threads
    uint64_t pbar[4];        // the two warps of one tensor-memory lane quarter
    uint32_t tmem_base;
    int abort_flag;
};

// One step of a CTA's work list.
enum { kOpA = 0, kOpB = 1, kOpPairEnd = 2, kOpStop = 3 };
struct FuOp {
    int kind;
    int phase;       // phase counter of the group (problem slot * Hkv + KV head)
    int prob, j;     // problem index and KV head of that phase
    int k;           // which of the CTA's tiles (slot of \bar A in tensor memory)
    int tile;        // token tile index inside the sequence
    int first, last; // first / last tile of this kind for this CTA in this phase
    int pair;        // for kOpPairEnd: the pair that ended
};

// Deterministic walk over the work list; every role of the CTA runs its own copy.
struct FuIter {
    const Geo& g;
    int cpp, n_groups, n_prob, group, rank;
    int n_phases;            // phases of this group
    int pair, ia, ib, nA, nB;
    __device__ FuIter(const Geo& geo, const FusedArgs& a)
        : g(geo), cpp(a.cpp), n_groups(a.n_groups), n_prob(a.n_prob)
    {
        group = blockIdx.x / cpp;
        rank = blockIdx.x % cpp;
        const int my_probs = group < n_groups ? (n_prob - group + n_groups - 1) / n_groups : 0;
        n_phases = my_probs * g.Hkv;
        pair = 0; ia = ib = 0;
        load_pair();
    }
    __device__ int prob_of(int phase) const { return group + (phase / g.Hkv) * n_groups; }
    __device__ int tiles_of(int phase, bool sweep_b) const
    {
        if (phase < 0 || phase >= n_phases) return 0;
        const int seq = prob_of(phase) % g.n_seqs;
        if (geo_identity(g, seq)) return 0;
        const int L = geo_L(g, seq);
        const int n = sweep_b ? (L - g.window + kTcTile - 1) / kTcTile : (L + kTcTile - 1) / kTcTile;
        return rank < n ? (n - rank + cpp - 1) / cpp : 0;
    }
    __device__ void load_pair()
    {
        nA = tiles_of(pair, false);
        nB = tiles_of(pair - 1, true);
    }
    __device__ FuOp next()
    {
        FuOp op;
        op.pair = pair;
        if (pair > n_phases) { op.kind = kOpStop; return op; }
        const bool take_a = ia < nA && (ia < ib + kFuLead || ib >= nB);
        if (take_a || ib < nB) {
            op.kind = take_a ? kOpA : kOpB;
            op.phase = take_a ? pair : pair - 1;
            op.k = take_a ? ia : ib;
            const int n = take_a ? nA : nB;
            op.first = op.k == 0;
            op.last = op.k == n - 1;
            op.tile = rank + op.k * cpp;
            op.prob = prob_of(op.phase);
            op.j = op.phase % g.Hkv;
            if (take_a) ++ia; else ++ib;
            return op;
        }
        op.kind = kOpPairEnd;
        ++pair; ia = ib = 0;
        load_pair();
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

__global__ void __launch_bounds__(kFuThreads, 1)
score_fused_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const Geo g,
               const FusedArgs fa)
{
    extern __shared__ uint8_t dyn_smem[];
    __shared__ FuBarriers sh;
    __shared__ __align__(16) float lse_s[2][128];
    __shared__ float xch[2][2][2][128];          // [op parity][tot | ent][half][token row]
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
            mbar_init(smem_u32(&sh.tempty[i]), kFuEpiThreads);
            mbar_init(smem_u32(&sh.qfull[i]), 1);
            mbar_init(smem_u32(&sh.qempty[i]), 1);
        }
        mbar_init(smem_u32(&sh.ebar), kFuEpiThreads);
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&sh.pbar[i]), 64);
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
    const int R = 128;                               // window rows per KV head

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
            bool ok = true;
            while (ok) {
                const FuOp op = it.next();
                if (op.kind == kOpStop) break;
                if (op.kind == kOpPairEnd) continue;
                if (op.kind == kOpA && op.phase != q_phase) {      // first tile of a phase: its query block
                    q_phase = op.phase;
                    const int b = op.phase & 1;
                    if (qloads[b] > 0 && !mbar_wait(smem_u32(&sh.qempty[b]), (qloads[b] - 1) & 1, abort_flag)) break;
                    ++qloads[b];
                    mbar_expect_tx(smem_u32(&sh.qfull[b]), kFuTileBytes);
                    for (int a = 0; a < 2; ++a)
                        tma_load_2d(q_smem + b * kFuTileBytes + a * kAtomBytes, &tmQ, smem_u32(&sh.qfull[b]), a * 64,
                                    op.prob * g.H * g.window + op.j * R, pol_q);
                }
                const int st = n_ops % kFuStages, ph = (n_ops / kFuStages) & 1;
                if (!mbar_wait(smem_u32(&sh.empty[st]), ph ^ 1, abort_flag)) break;
                mbar_expect_tx(smem_u32(&sh.full[st]), kFuTileBytes);
                const int layer = op.prob / g.n_seqs, seq = op.prob % g.n_seqs;
                for (int a = 0; a < 2; ++a)
                    tma_load_4d(k_smem + st * kFuTileBytes + a * kAtomBytes, &tmK, smem_u32(&sh.full[st]), a * 64, op.j,
                                g.cu[seq] + op.tile * kTcTile, layer, op.kind == kOpA ? pol_a : pol_b);
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
                const int b = op.phase & 1;
                if (op.kind == kOpA && op.phase != q_phase) {
                    q_phase = op.phase;
                    if (!mbar_wait(smem_u32(&sh.qfull[b]), qwaits[b] & 1, abort_flag)) break;
                    ++qwaits[b];
                    q_used[b] = true;
                }
                const int st = n_ops % kFuStages, ph = (n_ops / kFuStages) & 1;
                const int acc = n_ops & 1, aph = (n_ops >> 1) & 1;
                if (!mbar_wait(smem_u32(&sh.tempty[acc]), aph ^ 1, abort_flag)) break;
                if (!mbar_wait(smem_u32(&sh.full[st]), ph, abort_flag)) break;
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
            const int prob = it.prob_of(phase), j = phase % g.Hkv, seq = prob % g.n_seqs;
            if (geo_identity(g, seq)) continue;
            const int nt1 = (geo_L(g, seq) + kTcTile - 1) / kTcTile;
            const int n_src = min(fa.cpp, nt1);                 // CTAs that hold tiles of this problem
            if (rank >= R) continue;
            bool ok = true;
            if (lane == 0) ok = wait_counter(fa.arrive + prob * g.Hkv + j, n_src, abort_flag, fa.status);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            const float2* pp = fa.part + ((size_t)group * kFuPartSlots + (phase % kFuPartSlots)) * fa.cpp * 2 * R;
            for (int row = rank; row < R; row += fa.cpp) {
                // partial i = (source CTA, column half); merged in index order
                float m = -INFINITY;
                for (int i = lane; i < 2 * n_src; i += 32) {
                    const float2 v = __ldcg(pp + (size_t)i * R + row);
                    if (v.y > 0.f) m = fmaxf(m, v.x);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                float l = 0.f;
                for (int i = lane; i < 2 * n_src; i += 32) {
                    const float2 v = __ldcg(pp + (size_t)i * R + row);
                    if (v.y > 0.f) l += v.y * exp2f(v.x - m);
                }
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
        const int ew = warp - kFuEpiWarp0;
        const int q4 = warp & 3;                       // tensor-memory lane quarter of this warp
        const int half = ew >> 2;                      // which half of the columns / window positions
        const int row = q4 * 32 + lane;                // TMEM lane: window row (sweep A) or token (sweep B)
        const int et = ew * 32 + lane;                 // thread index among the epilogue threads
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const float c2 = fa.c2;
        const float inv_H = 1.f / (float)g.H;
        FuIter it(g, fa);
        const int group = it.group, rank = it.rank;
        float m_ref = 0.f, l_run = 0.f;                // sweep A state of (row, half)
        bool have_m = false;
        int n_ops = 0, n_fin = 0, lse_phase = -1, n_esync = 0, n_psync = 0;
        while (true) {
            const FuOp op = it.next();
            if (op.kind == kOpStop) break;
            if (op.kind == kOpPairEnd) continue;
            const int seq = op.prob % g.n_seqs, layer = op.prob / g.n_seqs;
            const int L = geo_L(g, seq), Tn = L - g.window;
            const int acc = n_ops & 1, aph = (n_ops >> 1) & 1;
            const uint32_t acc_addr = lane_addr + (uint32_t)acc * 128u;
            if (op.kind == kOpA) {
                if (op.first) { have_m = false; m_ref = 0.f; l_run = 0.f; }
                if (!mbar_wait(smem_u32(&sh.tfull[acc]), aph, abort_flag)) break;
                tc_fence_after();
                const int tok0 = op.tile * kTcTile + half * 64;
                const int lim = Tn + (row & 31);                   // causal: key index <= T + w (Eq. 2)
                const bool need_mask = tok0 + 63 > Tn;
                uint32_t r0[32], r1[32];
                tmem_ld32_issue(acc_addr + half * 64, r0);
                tmem_ld32_issue(acc_addr + half * 64 + 32, r1);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(smem_u32(&sh.tempty[acc]));            // logits are in registers: release the accumulator
                if (need_mask) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (tok0 + i > lim) r0[i] = 0xff800000u;       // -inf
                        if (tok0 + 32 + i > lim) r1[i] = 0xff800000u;
                    }
                }
                if (!have_m) {                                     // reference exponent of this row
                    const float mx = fmaxf(chunk_max(r0), chunk_max(r1)) * c2;
                    m_ref = (mx == -INFINITY) ? 0.f : ceilf(mx);
                    have_m = true;
                }
                float c = chunk_expsum(r0, c2, m_ref) + chunk_expsum(r1, c2, m_ref);
                if (!(l_run + c < 1.8e19f)) {                      // far above the reference: move it
                    const float mx = fmaxf(chunk_max(r0), chunk_max(r1)) * c2;
                    const float m_new = fmaxf(m_ref, ceilf(mx));
                    l_run *= exp2f(m_ref - m_new);
                    m_ref = m_new;
                    c = chunk_expsum(r0, c2, m_ref) + chunk_expsum(r1, c2, m_ref);
                }
                l_run += c;
                if (op.last) {
                    // The partial buffers are a ring over phases: the slot is free once every merge
                    // of the phase that used it last is done.  (A CTA that also runs sweep B is
                    // throttled by it anyway; one that owns only a window tile is not.)
                    if (et == 0 && op.phase >= kFuPartSlots) {
                        const int old = op.phase - kFuPartSlots;
                        wait_counter(fa.done + it.prob_of(old) * g.Hkv + old % g.Hkv, min(fa.cpp, R), abort_flag, fa.status);
                    }
                    if (!group_sync(&sh.ebar, n_esync, abort_flag)) break;
                    float2* pp = fa.part + ((size_t)group * kFuPartSlots + (op.phase % kFuPartSlots)) * fa.cpp * 2 * R;
                    pp[((size_t)rank * 2 + half) * R + row] = make_float2(m_ref, l_run);
                    __threadfence();
                    if (!group_sync(&sh.ebar, n_esync, abort_flag)) break;
                    if (et == 0) atomicAdd(fa.arrive + op.prob * g.Hkv + op.j, 1);
                }
            } else {
                if (op.phase != lse_phase) {                       // log-sum-exps of this phase
                    lse_phase = op.phase;
                    if (et == 0) wait_counter(fa.done + op.prob * g.Hkv + op.j, min(fa.cpp, R), abort_flag, fa.status);
                    if (!group_sync(&sh.ebar, n_esync, abort_flag)) break;
                    if (et < R) lse_s[op.phase & 1][et] = __ldcg(fa.lse2 + (size_t)op.prob * g.H * g.window + op.j * R + et);
                    if (!group_sync(&sh.ebar, n_esync, abort_flag)) break;
                }
                if (!mbar_wait(smem_u32(&sh.tfull[acc]), aph, abort_flag)) break;
                tc_fence_after();
                uint32_t v[4][16];                                 // head hl of the group, 16 window positions
#pragma unroll
                for (int hl = 0; hl < 4; ++hl) tmem_ld16_issue(acc_addr + hl * 32 + half * 16, v[hl]);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(smem_u32(&sh.tempty[acc]));
                const float* lj = lse_s[op.phase & 1];
                float accw[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) accw[i] = 0.f;
#pragma unroll
                for (int hl = 0; hl < 4; ++hl) {
                    const float4* l4 = reinterpret_cast<const float4*>(lj + hl * 32 + half * 16);
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        const float4 ls = l4[i >> 2];
                        accw[i + 0] += ex2_approx(fmaf(__uint_as_float(v[hl][i + 0]), c2, -ls.x));
                        accw[i + 1] += ex2_approx(fmaf(__uint_as_float(v[hl][i + 1]), c2, -ls.y));
                        accw[i + 2] += ex2_approx(fmaf(__uint_as_float(v[hl][i + 2]), c2, -ls.z));
                        accw[i + 3] += ex2_approx(fmaf(__uint_as_float(v[hl][i + 3]), c2, -ls.w));
                    }
                }
                // \bar A of this token tile, summed over the KV heads seen so far
                const uint32_t abar_addr = lane_addr + (uint32_t)(kFuAbarCol0 + op.k * 32 + half * 16);
                if (op.j > 0) {
                    uint32_t prev[16];
                    tmem_ld16_issue(abar_addr, prev);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) accw[i] += __uint_as_float(prev[i]);
                }
                if (op.j < g.Hkv - 1) {
                    tmem_st16(abar_addr, accw);
                    tmem_st_wait();
                } else {
                    // last KV head of the layer: s_t (Eqs. 3, 4) and the entropy of Eq. 6
                    const int par = n_fin & 1;
                    ++n_fin;
                    float tot_h = 0.f;
#pragma unroll
                    for (int i = 0; i < 16; ++i) tot_h += accw[i];
                    xch[par][0][half][row] = tot_h;
                    if (!group_sync(&sh.pbar[q4], n_psync, abort_flag)) break;
                    const float tot = xch[par][0][0][row] + xch[par][0][1][row];
                    float ent_h = 0.f;
                    if (tot > 0.f) {
                        const float inv = 1.f / tot;
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const float ah = accw[i] * inv;                       // \hat A (Eq. 6)
                            ent_h -= ah * (lg2_approx(ah + fa.eps) * 0.6931471805599453f);
                        }
                    }
                    xch[par][1][half][row] = ent_h;
                    if (!group_sync(&sh.pbar[q4], n_psync, abort_flag)) break;
                    const int t = op.tile * kTcTile + row;
                    if (half == 0 && t < Tn) {
                        const size_t off = (size_t)layer * g.total_tokens + g.cu[seq];
                        fa.s_out[off + t] = tot * inv_H;
                        fa.e_out[off + t] = xch[par][1][0][row] + xch[par][1][1][row];
                    }
                }
            }
            ++n_ops;
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
