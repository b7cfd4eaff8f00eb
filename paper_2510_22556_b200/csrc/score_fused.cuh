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
// Between the sweeps the row sums of all CTAs of the problem are merged into log-sum-exps; CTAs
// hand over through two counters per phase in global memory, every wait on them bounded.
//
// Both sweeps are the same 128 x 128 x 128 product on the tensor cores with the operand roles
// swapped: sweep A computes Q_g K^T (TMEM lane = window row, the running sum is thread-local),
// sweep B computes K Q_g^T (TMEM lane = token, the sums over heads and window positions are
// thread-local).  The head-summed attention \bar A[w, t] of the CTA's tokens lives in tensor
// memory (32 columns per token tile) across the KV heads of a layer, so neither the H x W x T
// attention tensor nor \bar A ever reaches shared or global memory.
//
// CTA = 19 warps.  Warp 0: one thread walks the work list, posts every tile step to a small ring
// in shared memory and issues the TMA loads.  Warp 1: one thread issues every tcgen05.mma (the
// warp owns tensor memory).  Warps 2-17: epilogue, two sets of eight warps; set s
// takes the steps whose logits land in accumulator s, so one set computes while the other waits
// and loads.  Inside a set two warps share each 32-lane quarter of tensor memory: in sweep A they
// split the tile's 128 token columns, in sweep B the 32 window positions.  Warp 18: hand-over
// between CTAs (publishes this CTA's row sums, merges its share of the rows of all CTAs, fetches
// the finished log-sum-exps), so that no epilogue thread ever waits on global memory.
//
// Single-sweep mode: when the caller passes the log of every window row's normaliser (the prefill's
// attention kernel keeps it, Sec. 4.1), sweep A, the hand-over warp and the waits between CTAs drop
// out: the producer posts sweep-B steps only and brings each phase's 128 log-sum-exps into shared
// memory with a bulk copy, one phase ahead; MMA issuer and epilogue are the same code.
//
// A launch works on the sequences of one length class (FusedArgs::sel): the host starts one launch
// per class so that a problem's group has about ceil(tiles / 7) CTAs and every CTA several tiles.
#pragma once
#include "common.cuh"
#include "score_simt.cuh"
#include "score_tc.cuh"

namespace sab {

constexpr int kFuThreads = 608;
constexpr int kFuEpiWarp0 = 2;
constexpr int kFuEpiWarps = 16;
constexpr int kFuHelpWarp = 18;
constexpr int kFuStages = 3;                 // K tile ring
constexpr int kFuQBufs = 3;                  // query-block buffers: phases n - 1 (sweep B), n (sweep A), n + 1 (loading ahead)
constexpr int kFuMaxTilesPerCta = 7;         // \bar A slots in tensor memory: 7 x 32 columns
constexpr int kFuAbarCol0 = 256;             // columns [0, 256): two logit accumulators
constexpr int kFuTmemCols = 512;
constexpr int kFuLead = 2;                   // sweep A runs at least this many tiles ahead of sweep B
constexpr int kFuPartSlots = 4;              // ring of per-phase partial buffers in global memory
constexpr int kFuLseSlots = 16;              // ring of log-sum-exp buffers in shared memory
constexpr int kFuMaxCtasDev = 256;           // upper bound on the CTAs of one launch
constexpr int kFuTileBytes = 2 * kAtomBytes; // 128 rows x 128 bf16
constexpr int kFuSmemBytes = 1024 + (kFuQBufs + kFuStages) * kFuTileBytes;
// The two epilogue sets take turns at the exponentials.  The special-function unit is the busiest
// unit of the kernel; two sets that share it freely end up in lockstep, both computing and then
// both going through the latencies between two steps (step record, accumulator barrier,
// tensor-memory loads) with the unit idle.  With turns, set s starts the exponentials of its k-th
// step only when the other set is well into those of its own preceding step (halfway in sweep A,
// three heads of four in sweep B), which keeps the sets apart: while one goes through the
// latencies the other has the unit.  An epilogue set hands its accumulator back to the MMA issuer
// as soon as the logits are in registers.

struct FusedArgs {
    int cpp;                 // CTAs per group (one group works on one problem at a time)
    int n_groups;
    int n_prob;              // problems of this launch: n_layers x n_sel, numbered layer * n_sel + k
    int n_sel;               // sequences this launch works on (a call is split into launches by sequence length,
    unsigned char sel[kMaxSeqs];   // so that short sequences get small groups): their indices
    float c2;                // log2(e) / sqrt(D)
    float eps;
    float2* part;            // [n_groups][kFuPartSlots][cpp][128] row statistics (m, l)
    float* lse2;             // [n_prob][Hkv * 128] log2-sum-exp2 per window row
    int fixed_schedule;      // two sweeps: the order of the tile steps ignores when the log-sum-exps arrive
    const float* neg_lse2;   // single-sweep mode: minus the log2-sum-exp2 of every window row, known beforehand
                             // (same layout as lse2; NULL = two sweeps, the kernel works the normalisers out itself)
    int* arrive;             // [n_prob][Hkv]
    int* done;               // [n_prob][Hkv]
    float* s_out;            // [n_layers][total_tokens]
    float* e_out;
    int* status;
};

// Problem v of a launch -> layer, sequence, and the problem's index in the call (layer * n_seqs + seq).
struct FuProb { int layer, seq, prob; };
__device__ __forceinline__ FuProb fu_prob(const FusedArgs& fa, const Geo& g, int v)
{
    FuProb r;
    r.layer = v / fa.n_sel;
    r.seq = fa.sel[v - r.layer * fa.n_sel];
    r.prob = r.layer * g.n_seqs + r.seq;
    return r;
}

struct FuBarriers {
    uint64_t full[kFuStages];
    uint64_t empty[kFuStages];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint64_t qfull[kFuQBufs];
    uint64_t qempty[kFuQBufs];
    uint64_t pbar[2][4];     // the two warps of one set that share a tensor-memory lane quarter
    uint64_t pub_full[2];    // row sums of a phase are in shared memory (all epilogue threads)
    uint64_t lse_full[kFuLseSlots];
    uint64_t xu[2];          // turn of epilogue set s at the exponentials
    uint64_t adone[2][2];    // epilogue set s has finished its k-th step (k & 1 picks the barrier), its update of
                             // the head-summed attention included
    uint32_t tmem_base;
    int abort_flag;
};

// ---- the work list ----------------------------------------------------------------------------
enum { kOpA = 0, kOpB = 1, kOpPairEnd = 2, kOpStop = 3 };

// What the producer needs to know about one phase = (problem, KV head).
struct FuPhase {
    int vp;          // problem number inside the launch
    int prob, j;     // problem index in the call and KV head
    int layer;
    int Tn;          // compressible length of the sequence
    int tok_base;    // first packed token row of the sequence
    int n_a, n_b;    // tiles of this CTA in sweep A and in sweep B
    int qpar;        // parity of the load of this phase's query block into its buffer
};

struct FuOp {
    int kind;
    int phase;
    int k;           // which of the CTA's tiles (slot of \bar A in tensor memory)
    int tile;        // token tile index inside the sequence
    int last;        // last tile of this kind for this CTA in this phase
    int released;    // kOpPairEnd: the query-block buffer of the phase whose sweep B just ended, or -1
};

// Walk over the work list of one CTA (run by the producer thread only) with two cursors: sweep A
// at phase `a_ph`, sweep B behind it at phase `b_ph` < a_ph.  Normally sweep B follows one phase
// behind and sweep A leads by at least kFuLead tiles inside that phase.  While the log-sum-exps of
// sweep B's phase are not in yet (`b_ready` false: another CTA is late) sweep A simply runs on,
// up to two phases ahead (three query-block buffers), instead of idling; the second read of K then
// comes a little later, which costs L2 hits only while it lasts.
struct FuIter {
    const Geo& g;
    const FusedArgs& fa;
    int cpp, n_groups, group, rank;
    int n_phases;            // phases of this group
    int a_ph, ia, b_ph, ib;
    int a_buf, b_buf;        // a_ph % 3 and b_ph % 3 (query-block buffers), kept without divisions
    FuPhase pa;              // phase a_ph
    FuPhase q0, q1;          // phases b_ph and b_ph + 1 where those lie behind sweep A
    __device__ FuIter(const Geo& geo, const FusedArgs& a) : g(geo), fa(a), cpp(a.cpp), n_groups(a.n_groups)
    {
        group = blockIdx.x / cpp;
        rank = blockIdx.x % cpp;
        const int my_probs = group < n_groups ? (a.n_prob - group + n_groups - 1) / n_groups : 0;
        n_phases = my_probs * g.Hkv;
        a_ph = ia = b_ph = ib = a_buf = b_buf = 0;
        pa.vp = group; pa.prob = 0; pa.j = -1; pa.n_a = pa.n_b = 0;
        if (n_phases > 0) load_next();
    }
    __device__ int my_tiles(int n) const { return rank < n ? (n - rank + cpp - 1) / cpp : 0; }
    // Turns pa into the next phase.  Consecutive phases of a problem differ only in the KV head;
    // the divisions are paid once per problem.
    __device__ void load_next()
    {
        if (pa.j >= 0 && pa.j + 1 < g.Hkv) { ++pa.j; return; }
        if (pa.j >= 0) pa.vp += n_groups;
        pa.j = 0;
        const FuProb m = fu_prob(fa, g, pa.vp);
        pa.layer = m.layer;
        pa.prob = m.prob;
        const int seq = m.seq;
        pa.tok_base = g.cu[seq];
        const int L = g.cu[seq + 1] - pa.tok_base;
        pa.Tn = L - g.window;
        pa.n_a = L > g.n_out ? my_tiles((L + kTcTile - 1) / kTcTile) : 0;       // else: returned unchanged
        pa.n_b = pa.n_a > 0 ? my_tiles((pa.Tn + kTcTile - 1) / kTcTile) : 0;
    }
    __device__ bool b_pending() const { return b_ph < a_ph && ib < q0.n_b; }
    __device__ FuOp next(bool b_ready)
    {
        FuOp op;
        op.released = -1;
        // sweep B leaves a phase when its tiles are done (at once if it has none)
        if (b_ph < a_ph && ib >= q0.n_b) {
            op.kind = kOpPairEnd;
            op.released = q0.n_a > 0 ? b_buf : -1;
            q0 = q1;
            ++b_ph; ib = 0;
            b_buf = b_buf == kFuQBufs - 1 ? 0 : b_buf + 1;
            return op;
        }
        // sweep A moves on to the next phase when its tiles are done and a buffer is free for it
        if (a_ph < n_phases && ia >= pa.n_a && a_ph + 1 <= b_ph + kFuQBufs - 1) {
            if (a_ph == b_ph) q0 = pa; else q1 = pa;
            ++a_ph; ia = 0;
            a_buf = a_buf == kFuQBufs - 1 ? 0 : a_buf + 1;
            if (a_ph < n_phases) load_next();
            op.kind = kOpPairEnd;
            return op;
        }
        const bool can_a = a_ph < n_phases && ia < pa.n_a && a_ph <= b_ph + 1;
        const bool can_b = b_ph < a_ph && ib < q0.n_b;
        if (!can_a && !can_b) { op.kind = kOpStop; return op; }
        const bool lead_needed = a_ph == b_ph + 1 && ia < ib + kFuLead;
        if (can_a && (!can_b || !b_ready || lead_needed)) {
            op.kind = kOpA; op.phase = a_ph; op.k = ia; op.last = ia == pa.n_a - 1;
            op.tile = rank + ia * cpp;
            ++ia;
            return op;
        }
        op.kind = kOpB; op.phase = b_ph; op.k = ib; op.last = ib == q0.n_b - 1;
        op.tile = rank + ib * cpp;
        ++ib;
        return op;
    }
};

// One tile step as the other roles see it: 16 bytes in the shared-memory ring.
constexpr int kStepB = 1 << 0;          // sweep B (else sweep A)
constexpr int kStepLastA = 1 << 1;      // last sweep A step of its phase for this CTA: row sums are due
constexpr int kStepPrevLastA = 1 << 2;  // (epilogue rings) the step before this one, taken by the other set, was a kStepLastA step
constexpr int kStepLseWait = 1 << 3;    // (epilogue rings) first sweep B step of its phase for this set: wait for the log-sum-exps
constexpr int kStepKShift = 4;          // bits 4-6: slot of the tile among the CTA's tiles
constexpr int kStepHead0 = 1 << 7;      // first KV head of the layer (sweep B starts \bar A afresh)
constexpr int kStepHeadLast = 1 << 8;   // last KV head of the layer (sweep B emits s and the entropy)
constexpr int kStepQBufShift = 9;       // bits 9-10: which query-block buffer the step's phase uses
constexpr int kStepQPar = 1 << 11;      // parity of that buffer's load
constexpr int kStepRelShift = 12;       // bits 12-14: before this step, query-block buffer i has seen its last product
constexpr int kStepMask = 1 << 15;      // sweep A tile that reaches the causal boundary
constexpr int kStepNewQ = 1 << 16;      // first step that uses this load of the query block
constexpr int kStepLseShift = 17;       // (epilogue rings) bits 17-20: log-sum-exp buffer of the phase, bit 21: parity of its fill
constexpr int kStepStop = 1 << 22;      // (epilogue rings) no further step for this set
constexpr int kStepTagShift = 24;       // (epilogue rings) bits 24-31: which use of the ring slot this is (never 0)

constexpr int kFuRing = 16;
constexpr int kFuSetRing = 8;
struct FuSched {
    // Every step, for the MMA issuer: one tagged flags word (the issuer needs nothing else; ring
    // position, K stage and parities follow from the step's number).  The tag in bits 24-31 counts
    // the uses of the slot and is never 0, so one look at the word says whether step n is posted.
    int ring[kFuRing];
    // The steps of each epilogue set once more, in a ring of its own: {flags, first token of the
    // tile, T of the sequence, row offset of the outputs}.  A set reads only its own steps (what it
    // must know about the other set's steps is folded into the flags); the flags word is tagged in
    // the same way and is published after the payload.
    int4 sring[2][kFuSetRing];
    volatile int lse_fetched;   // log-sum-exp buffers filled so far (helper warp)
    volatile int pub_done;      // phases whose row sums the helper warp has taken out of shared memory
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

// 2^d for an integer d <= 0, built from the exponent field (d below -126 gives 2^-126: the
// product with any row sum is then far below one unit of the result).
__device__ __forceinline__ float pow2_nonpos(int d)
{
    return __int_as_float((127 + max(d, -126)) << 23);
}
__device__ __forceinline__ int redux_max_s32(int v)
{
    int r;
    asm volatile("redux.sync.max.s32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
    return r;
}
__device__ __forceinline__ unsigned redux_max_u32(unsigned v)
{
    unsigned r;
    asm volatile("redux.sync.max.u32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
    return r;
}
__device__ __forceinline__ unsigned redux_add_u32(unsigned v)
{
    unsigned r;
    asm volatile("redux.sync.add.u32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v));
    return r;
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


// Hand-over of the step rings and the small counters of FuSched between threads of the CTA.  A
// word that stands for itself (a tagged flags word, a counter) is written and read relaxed.  Where
// a reader goes on to read what the writer stored BEFORE that word (the payload of a step, the
// buffer a counter announces), the writer publishes the word with a release store and the reader
// puts an acquire fence between seeing the word and reading the rest.
__device__ __forceinline__ void st_release_cta(const volatile void* p, int v)
{
    asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32((const void*)p)), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_cta(const volatile void* p)
{
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32((const void*)p)) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed_cta(const volatile void* p)
{
    int v;
    asm volatile("ld.relaxed.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32((const void*)p)) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_cta(const volatile void* p, int v)
{
    asm volatile("st.relaxed.cta.shared.s32 [%0], %1;" ::"r"(smem_u32((const void*)p)), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_acquire_cta()
{
    asm volatile("fence.acq_rel.cta;" ::: "memory");
}

__device__ __forceinline__ int sched_tag(int idx, int ring_len) { return (((idx / ring_len) & 0x7f) + 1) << kStepTagShift; }
__device__ __forceinline__ bool sched_posted(int fl, int idx, int ring_len)
{
    return (fl & (0xff << kStepTagShift)) == sched_tag(idx, ring_len);
}

// Main ring (MMA issuer): a single word per step.
__device__ __forceinline__ void sched_post(FuSched& sc, int idx, int flags)
{
    st_relaxed_cta(&sc.ring[idx % kFuRing], flags | sched_tag(idx, kFuRing));
}
__device__ __forceinline__ int sched_peek(FuSched& sc, int idx) { return ld_relaxed_cta(&sc.ring[idx % kFuRing]); }
// Waits (bounded) until step `idx` is posted and returns its flags; false when the wait gave up.
__device__ __forceinline__ bool sched_get(FuSched& sc, int idx, int& flags, volatile int* abort_flag)
{
    long long t0 = 0;
    int spins = 0;
    while (true) {
        flags = sched_peek(sc, idx);
        if (sched_posted(flags, idx, kFuRing)) return true;
        if (spins++ == 0) t0 = clock64();
        if ((spins & 15) == 0 && (*abort_flag || clock64() - t0 > kWaitLimitCycles)) { *abort_flag = 1; return false; }
    }
}

// Posts the k-th step of an epilogue set: payload first, then the tagged flags word (release).
__device__ __forceinline__ void sched_post_set(FuSched& sc, int set, int k, int4 step)
{
    const uint32_t dst = smem_u32(&sc.sring[set][k % kFuSetRing]);
    asm volatile("st.relaxed.cta.shared.s32 [%0], %1;" ::"r"(dst + 4), "r"(step.y) : "memory");
    asm volatile("st.relaxed.cta.shared.v2.s32 [%0], {%1, %2};" ::"r"(dst + 8), "r"(step.z), "r"(step.w) : "memory");
    st_release_cta(&sc.sring[set][k % kFuSetRing], step.x | sched_tag(k, kFuSetRing));
}
// The flags word of the k-th step of an epilogue set as it stands (posted or not), and whether a
// flags word read that way is the posted k-th step.
__device__ __forceinline__ int sched_peek_flags(FuSched& sc, int set, int k)
{
    return ld_relaxed_cta(&sc.sring[set][k % kFuSetRing]);
}
__device__ __forceinline__ bool sched_flags_posted(int fl, int k) { return sched_posted(fl, k, kFuSetRing); }
// Payload (.y, .z, .w) of a step whose flags word has been seen posted: the fence orders the read
// after that sighting.
__device__ __forceinline__ void sched_payload(FuSched& sc, int set, int k, int4& out)
{
    fence_acquire_cta();
    const uint32_t src = smem_u32(&sc.sring[set][k % kFuSetRing]);
    asm volatile("ld.relaxed.cta.shared.s32 %0, [%1];" : "=r"(out.y) : "r"(src + 4) : "memory");
    asm volatile("ld.relaxed.cta.shared.v2.s32 {%0, %1}, [%2];" : "=r"(out.z), "=r"(out.w) : "r"(src + 8) : "memory");
}
// Waits (bounded) until the k-th step of an epilogue set is posted and returns its flags.
__device__ __forceinline__ bool sched_get_set(FuSched& sc, int set, int k, int& flags, volatile int* abort_flag)
{
    long long t0 = 0;
    int spins = 0;
    while (true) {
        flags = sched_peek_flags(sc, set, k);
        if (sched_flags_posted(flags, k)) return true;
        if (spins++ == 0) t0 = clock64();
        if ((spins & 15) == 0 && (*abort_flag || clock64() - t0 > kWaitLimitCycles)) { *abort_flag = 1; return false; }
    }
}

#define FU_WAIT(code, expr) ((expr) ? true : (note_giveup(fa.status, code), false))

// One 128 x 128 x 128 product into the accumulator at tensor-memory address `d`: eight
// tcgen05.mma.  `a_lo` / `b_lo` are the start-address fields (shared-memory address / 16) of the
// operands' descriptors; the rest of a descriptor is constant (128-byte swizzle, eight-row groups
// 1024 bytes apart, version 1).  A k-step moves the start address by 32 bytes inside the 128-byte
// row, the second 64-column atom follows after the fourth step.
__device__ __forceinline__ void fu_issue_tile(uint32_t d, uint32_t a_lo, uint32_t b_lo)
{
    constexpr uint32_t idesc = umma_idesc_bf16(128, 128);
    constexpr uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);     // bits 32-63 of umma_desc_sw128()
    static_assert((kAtomBytes >> 4) == 1024, "start-address step of the second atom");
#define FU_MMA_STEP(OFF, PRED)                                                        \
        "add.u32 ta, %1, " #OFF ";\n\tadd.u32 tb, %2, " #OFF ";\n\t"                  \
        "mov.b64 da, {ta, %3};\n\tmov.b64 db, {tb, %3};\n\t"                          \
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, " #PRED ";\n\t"
    asm volatile(
        "{\n\t.reg .pred yes, no;\n\t.reg .b32 ta, tb;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 no, 0, 0;\n\tsetp.eq.b32 yes, 0, 0;\n\t"
        FU_MMA_STEP(0, no) FU_MMA_STEP(2, yes) FU_MMA_STEP(4, yes) FU_MMA_STEP(6, yes)
        FU_MMA_STEP(1024, yes) FU_MMA_STEP(1026, yes) FU_MMA_STEP(1028, yes) FU_MMA_STEP(1030, yes)
        "}"
        ::"r"(d), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc)
        : "memory");
#undef FU_MMA_STEP
}

// ---- arithmetic of the epilogue ---------------------------------------------------------------
// Packed fp32 pairs (one instruction for two lanes of arithmetic: the epilogue is short of issue
// slots, not of fp32 throughput).
// Sum of exp2(v * c2 - m) over 32 logits of one window row.
__device__ __forceinline__ float chunk_expsum(const uint32_t (&r)[32], float c2, float m)
{
    const uint64_t cc = pack2(c2, c2), mm = pack2(-m, -m);
    uint64_t s0 = pack2(0.f, 0.f), s1 = s0;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        float a, b, c, d;
        unpack2(fma2(pack2u(r[i + 0], r[i + 1]), cc, mm), a, b);
        unpack2(fma2(pack2u(r[i + 2], r[i + 3]), cc, mm), c, d);
        s0 = add2(s0, pack2(ex2_approx(a), ex2_approx(b)));
        s1 = add2(s1, pack2(ex2_approx(c), ex2_approx(d)));
    }
    float a, b, c, d;
    unpack2(s0, a, b);
    unpack2(s1, c, d);
    return (a + b) + (c + d);
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
    __device__ void add(const uint32_t (&r)[32], float c2)
    {
        if (!have_m) {
            const float mx = chunk_max(r) * c2;
            if (mx == -INFINITY) return;                   // nothing visible yet
            m = ceilf(mx);
            have_m = true;
        }
        // one copy of the summation code: the loop repeats only when the sum would leave the
        // fp32 range, after moving the reference exponent up to the chunk's maximum
#pragma unroll 1
        while (true) {
            const float c = chunk_expsum(r, c2, m);
            if (l + c < 1.8e19f || !(c == c)) { l += c; break; }
            const float m_new = fmaxf(m, ceilf(chunk_max(r) * c2));
            if (!(m_new > m)) { l += c; break; }            // cannot be improved (non-finite logits)
            l *= exp2f(m - m_new);
            m = m_new;
        }
    }
};

// accw[i] += exp2(logit * c2 - lse) for 16 window positions of one query head; `lse` holds -lse.
__device__ __forceinline__ void accumulate_head16(float (&accw)[16], const uint32_t (&r)[16], const float* lse, float c2)
{
    const float4* l4 = reinterpret_cast<const float4*>(lse);
    const uint64_t cc = pack2(c2, c2);
#pragma unroll
    for (int i = 0; i < 16; i += 4) {
        const float4 ls = l4[i >> 2];
        float a, b, c, d;
        unpack2(fma2(pack2u(r[i + 0], r[i + 1]), cc, pack2(ls.x, ls.y)), a, b);
        unpack2(fma2(pack2u(r[i + 2], r[i + 3]), cc, pack2(ls.z, ls.w)), c, d);
        unpack2(add2(pack2(accw[i + 0], accw[i + 1]), pack2(ex2_approx(a), ex2_approx(b))), accw[i + 0], accw[i + 1]);
        unpack2(add2(pack2(accw[i + 2], accw[i + 3]), pack2(ex2_approx(c), ex2_approx(d))), accw[i + 2], accw[i + 3]);
    }
}

// ---- producer of the single-sweep mode ----------------------------------------------------------
// With the log-sum-exp of every window row known beforehand there is no sweep A and no hand-over
// between CTAs: the producer walks the phases = (problem, KV head) in which this CTA has token
// tiles and posts one sweep-B step per tile.  The query block and the 128 log-sum-exps of a phase
// are fetched one phase ahead: the former into query-block buffer a % 3 (a counts this CTA's
// phases with tiles), the latter by a bulk copy into log-sum-exp buffer a % 16.  The copy for phase
// a + 1 is issued together with that phase's query block, i.e. once the query-block buffer of phase
// a - 2 is free: every product up to that phase's last step is complete then.  With one step per
// phase (the tightest case) those are the products of step n - 2 when step n is being posted; they
// were issued after the epilogue of step n - 4 had handed its accumulator back, which it does
// BEFORE its exponentials, and the other set may likewise still be inside step n - 5.  The oldest
// buffer that can still be read is therefore that of phase a - 5, six buffers from the one being
// written; sixteen leave a wide margin.
struct FuSinglePhase {
    int phase, vp, prob, j, layer, tok_base, Tn, n_b;
};

__device__ __forceinline__ void fu_single_advance(FuSinglePhase& c, const Geo& g, const FusedArgs& fa, int group, int n_groups,
                                                  int rank, int cpp, int n_phases)
{
    while (true) {
        ++c.phase;
        if (c.phase >= n_phases) { c.phase = n_phases; return; }
        if (c.j >= 0 && c.j + 1 < g.Hkv) {             // same problem, next KV head
            ++c.j;
        } else {                                       // next problem of the group: the divisions are paid here
            c.vp = c.j < 0 ? group : c.vp + n_groups;
            c.j = 0;
            const FuProb m = fu_prob(fa, g, c.vp);
            c.layer = m.layer;
            c.prob = m.prob;
            const int seq = m.seq;
            c.tok_base = g.cu[seq];
            const int L = g.cu[seq + 1] - c.tok_base;
            c.Tn = L - g.window;
            const int nt = (c.Tn + kTcTile - 1) / kTcTile;
            c.n_b = (L > g.n_out && rank < nt) ? (nt - rank + cpp - 1) / cpp : 0;    // else: returned unchanged, or no tile here
        }
        if (c.n_b > 0) return;
    }
}

__device__ __forceinline__ void fu_produce_single(const CUtensorMap* tmQ, const CUtensorMap* tmK, const Geo& g,
                                                  const FusedArgs& fa, FuBarriers& sh, FuSched& sched, uint32_t q_smem,
                                                  uint32_t k_smem, uint32_t lse_smem, volatile int* abort_flag)
{
    constexpr int R = 128;
    const uint64_t pol_k = l2_policy_evict_first();        // every K tile is read once
    const uint64_t pol_q = l2_policy_evict_last();
    const int group = blockIdx.x / fa.cpp, rank = blockIdx.x % fa.cpp;
    const int my_probs = group < fa.n_groups ? (fa.n_prob - group + fa.n_groups - 1) / fa.n_groups : 0;
    const int n_phases = my_probs * g.Hkv;
    FuSinglePhase cur;
    cur.phase = -1; cur.vp = 0; cur.prob = 0; cur.j = -1; cur.layer = 0; cur.tok_base = 0; cur.Tn = 0; cur.n_b = 0;
    fu_single_advance(cur, g, fa, group, fa.n_groups, rank, fa.cpp, n_phases);
    FuSinglePhase nxt = cur;
    if (cur.phase < n_phases) fu_single_advance(nxt, g, fa, group, fa.n_groups, rank, fa.cpp, n_phases);

    // Loads of this CTA's a-th phase with tiles: query block and log-sum-exps.  The buffers must be free.
    auto issue_phase_loads = [&](const FuSinglePhase& ph, int qb, int ls) {
        mbar_expect_tx(smem_u32(&sh.qfull[qb]), kFuTileBytes);
        for (int a = 0; a < 2; ++a)
            tma_load_2d(q_smem + qb * kFuTileBytes + a * kAtomBytes, tmQ, smem_u32(&sh.qfull[qb]), a * 64,
                        ph.prob * g.H * g.window + ph.j * R, pol_q);
        mbar_expect_tx(smem_u32(&sh.lse_full[ls]), R * (uint32_t)sizeof(float));
        bulk_load_1d(lse_smem + ls * R * (uint32_t)sizeof(float), fa.neg_lse2 + (size_t)ph.prob * g.H * g.window + ph.j * R,
                     R * (uint32_t)sizeof(float), smem_u32(&sh.lse_full[ls]));
    };

    int n_steps = 0, pending_rel = 0;
    int a_idx = 0, qb = 0, ls = 0;                        // this phase: its count, query-block buffer, log-sum-exp buffer
    unsigned q_uses = 0;                                   // per query-block buffer: parity of the number of loads so far
    unsigned ls_par = 0;                                   // parity of a_idx / kFuLseSlots
    int sb0 = -1, sb1 = -1;                                // last phase in which set 0 / set 1 had a step
    bool ok = true;
    if (cur.phase < n_phases) {
        issue_phase_loads(cur, 0, 0);
        q_uses ^= 1u;
    }
    while (ok && cur.phase < n_phases) {
        const int qb_n = qb == kFuQBufs - 1 ? 0 : qb + 1, ls_n = (ls + 1) & (kFuLseSlots - 1);
        const bool have_next = nxt.phase < n_phases;
        bool next_loaded = !have_next;
        const int qpar = ((q_uses >> qb) & 1u) ^ 1u;       // parity of the load this phase uses (q_uses already counts it)
        for (int k = 0; k < cur.n_b; ++k) {
            // the next phase's loads, as soon as its query-block buffer is free (probe only; the
            // blocking wait comes after the last step of this phase)
            if (!next_loaded) {
                const bool fresh = a_idx + 1 < kFuQBufs;
                if (fresh || mbar_test_wait(smem_u32(&sh.qempty[qb_n]), ((q_uses >> qb_n) & 1u) ^ 1u)) {
                    issue_phase_loads(nxt, qb_n, ls_n);
                    q_uses ^= 1u << qb_n;
                    next_loaded = true;
                }
            }
            int flags = pending_rel | kStepB | (k << kStepKShift) | (qb << kStepQBufShift);
            pending_rel = 0;
            if (cur.j == 0) flags |= kStepHead0;
            if (cur.j == g.Hkv - 1) flags |= kStepHeadLast;
            if (k == 0) flags |= kStepNewQ;
            if (qpar) flags |= kStepQPar;
            const int tok0 = (rank + k * fa.cpp) * kTcTile;
            const int4 rec = make_int4(flags, tok0, cur.Tn, cur.layer * g.total_tokens + cur.tok_base);
            sched_post(sched, n_steps, flags);
            {
                const int eset = n_steps & 1;
                int ef = (flags & ~(7 << kStepRelShift)) | ((ls | ((int)ls_par << 4)) << kStepLseShift);
                if ((eset ? sb1 : sb0) != a_idx) {
                    if (eset) sb1 = a_idx; else sb0 = a_idx;
                    ef |= kStepLseWait;
                }
                sched_post_set(sched, eset, n_steps >> 1, make_int4(ef, rec.y, rec.z, rec.w));
            }
            const int st = n_steps % kFuStages, par = (n_steps / kFuStages) & 1;
            if (!FU_WAIT(2, mbar_wait(smem_u32(&sh.empty[st]), par ^ 1, abort_flag))) { ok = false; break; }
            mbar_expect_tx(smem_u32(&sh.full[st]), kFuTileBytes);
            for (int a = 0; a < 2; ++a)
                tma_load_4d(k_smem + st * kFuTileBytes + a * kAtomBytes, tmK, smem_u32(&sh.full[st]), a * 64, cur.j,
                            cur.tok_base + tok0, cur.layer, pol_k);
            ++n_steps;
        }
        if (!ok) break;
        if (!next_loaded) {
            if (!FU_WAIT(1, mbar_wait(smem_u32(&sh.qempty[qb_n]), ((q_uses >> qb_n) & 1u) ^ 1u, abort_flag))) break;
            issue_phase_loads(nxt, qb_n, ls_n);
            q_uses ^= 1u << qb_n;
        }
        pending_rel = 1 << (kStepRelShift + qb);           // this phase's query block has seen its last product
        cur = nxt;
        if (have_next) fu_single_advance(nxt, g, fa, group, fa.n_groups, rank, fa.cpp, n_phases);
        ++a_idx;
        qb = qb_n;
        ls = ls_n;
        if (ls == 0) ls_par ^= 1u;
    }
    sched_post(sched, n_steps, kStepStop);
    for (int es = 0; es < 2; ++es)
        sched_post_set(sched, es, (n_steps + 1 - es) >> 1, make_int4(kStepStop, 0, 0, 0));
}


__global__ void __launch_bounds__(kFuThreads, 1)
score_fused_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const Geo g,
               const FusedArgs fa)
{
    extern __shared__ uint8_t dyn_smem[];
    __shared__ FuBarriers sh;
    __shared__ __align__(16) FuSched sched;
    __shared__ __align__(16) float lse_s[kFuLseSlots][128];      // minus the log2-sum-exp2 of the window rows of a phase
    __shared__ float2 pub_s[2][4][128];                          // [phase parity][set * 2 + half][window row]
    __shared__ float xch[2][2][2][2][128];                       // [set][use parity][tot | ent][half][token]
    const uint32_t base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    const uint32_t q_smem = base;                                  // query blocks
    const uint32_t k_smem = base + kFuQBufs * kFuTileBytes;        // K tile ring

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0 && lane == 0) {
        for (int i = 0; i < kFuStages; ++i) {
            mbar_init(smem_u32(&sh.full[i]), 1);
            mbar_init(smem_u32(&sh.empty[i]), 1);
        }
        for (int i = 0; i < kFuQBufs; ++i) {
            mbar_init(smem_u32(&sh.qfull[i]), 1);
            mbar_init(smem_u32(&sh.qempty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh.tfull[i]), 1);
            mbar_init(smem_u32(&sh.tempty[i]), 256);
            mbar_init(smem_u32(&sh.pub_full[i]), kFuEpiWarps * 32);
            for (int q = 0; q < 4; ++q) mbar_init(smem_u32(&sh.pbar[i][q]), 64);
        }
        for (int i = 0; i < kFuLseSlots; ++i) mbar_init(smem_u32(&sh.lse_full[i]), 1);
        for (int i = 0; i < 2; ++i) mbar_init(smem_u32(&sh.xu[i]), kFuEpiWarps * 16);
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&sh.adone[i >> 1][i & 1]), kFuEpiWarps * 16);
        sh.abort_flag = 0;
        for (int i = 0; i < kFuRing; ++i) sched.ring[i] = 0;
        for (int i = 0; i < 2 * kFuSetRing; ++i) (&sched.sring[0][0])[i] = make_int4(0, 0, 0, 0);
        sched.lse_fetched = 0;
        sched.pub_done = 0;
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

    if (warp == 0) {
        // ------------------------------------------------------------------ scheduler + TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            if (fa.neg_lse2 != nullptr) {
                fu_produce_single(&tmQ, &tmK, g, fa, sh, sched, q_smem, k_smem, smem_u32(&lse_s[0][0]), abort_flag);
            } else {
            const uint64_t pol_a = l2_policy_evict_last();     // first read: keep for sweep B
            const uint64_t pol_b = l2_policy_evict_first();    // second read: last use
            const uint64_t pol_q = l2_policy_evict_last();
            FuIter it(g, fa);
            // Query blocks are loaded a phase ahead of their first use: phase p goes to buffer p % 3
            // as soon as that buffer's previous tenant (phase p - 3) has seen its last product.
            int ql_phase = 0, ql_buf = 0, ql_vp = it.group, ql_prob = 0, ql_j = 0;      // ql_prob: index in the call of problem ql_vp
            unsigned ql_used = 0, ql_par = 0;                  // per buffer: ever loaded, parity of its load count
            bool ql_tiles = false;
            if (it.n_phases > 0) {
                const FuProb m = fu_prob(fa, g, ql_vp);
                const int L = geo_L(g, m.seq);
                ql_prob = m.prob;
                ql_tiles = L > g.n_out && it.rank < (L + kTcTile - 1) / kTcTile;
            }
            unsigned fq_par = 0;                               // the same parities as the work list sees them
            int q_phase = -1, pending_rel = 0, b_idx = -1, b_counted = -1, n_steps = 0;
            int sb0 = -1, sb1 = -1;                            // last sweep B phase in which set 0 / set 1 had a step
            bool ok = true, prev_last_a = false;
            while (ok) {
                // ---- next step of the work list
                if (it.b_pending() && b_counted != it.b_ph) {  // sweep B entered a phase: it needs the helper's next fetch
                    b_counted = it.b_ph;
                    ++b_idx;
                }
                const FuOp op = it.next(fa.fixed_schedule != 0 || ld_relaxed_cta(&sched.lse_fetched) > b_idx);   // a hint: the epilogue waits on the buffer's barrier
                if (op.kind == kOpStop) break;
                if (op.kind == kOpPairEnd) {
                    // the query block of a phase whose sweep B ended has seen its last product
                    if (op.released >= 0) pending_rel |= 1 << (kStepRelShift + op.released);
                    continue;
                }
                const bool is_b = op.kind == kOpB;
                FuPhase& ph = is_b ? it.q0 : it.pa;
                const int b = is_b ? it.b_buf : it.a_buf;
                int flags = pending_rel | (op.k << kStepKShift) | (b << kStepQBufShift);
                pending_rel = 0;
                if (!is_b) {
                    if (op.last) flags |= kStepLastA;
                    if (op.tile * kTcTile + kTcTile - 1 > ph.Tn) flags |= kStepMask;
                    if (op.phase != q_phase) {                 // first tile of a phase: its query block
                        q_phase = op.phase;
                        ph.qpar = (fq_par >> b) & 1;
                        fq_par ^= 1u << b;
                        flags |= kStepNewQ;
                    }
                } else {
                    flags |= kStepB;
                    if (ph.j == 0) flags |= kStepHead0;
                    if (ph.j == g.Hkv - 1) flags |= kStepHeadLast;
                }
                if (ph.qpar) flags |= kStepQPar;
                const int tok0 = op.tile * kTcTile;
                const int4 rec = make_int4(flags, tok0, ph.Tn, ph.layer * g.total_tokens + ph.tok_base);
                sched_post(sched, n_steps, flags);
                {
                    const int eset = n_steps & 1;
                    int ef = flags & ~(7 << kStepRelShift);
                    if (prev_last_a) ef |= kStepPrevLastA;
                    if (is_b) {
                        ef |= ((b_idx % kFuLseSlots) | (((b_idx / kFuLseSlots) & 1) << 4)) << kStepLseShift;
                        if ((eset ? sb1 : sb0) != b_idx) {
                            if (eset) sb1 = b_idx; else sb0 = b_idx;
                            ef |= kStepLseWait;
                        }
                    }
                    sched_post_set(sched, eset, n_steps >> 1, make_int4(ef, rec.y, rec.z, rec.w));
                    prev_last_a = !is_b && op.last;
                }
                // ---- query blocks: this step's must be on its way (blocking); the next phase's is
                // started if its buffer is free (probe only)
                while (ql_phase < it.n_phases && ql_phase <= op.phase + 1) {
                    if (ql_tiles) {
                        if ((ql_used >> ql_buf) & 1) {
                            const uint32_t par = ((ql_par >> ql_buf) & 1) ^ 1;
                            if (ql_phase <= op.phase) {
                                if (!FU_WAIT(1, mbar_wait(smem_u32(&sh.qempty[ql_buf]), par, abort_flag))) { ok = false; break; }
                            } else if (!mbar_test_wait(smem_u32(&sh.qempty[ql_buf]), par)) {
                                break;
                            }
                        }
                        ql_used |= 1u << ql_buf;
                        ql_par ^= 1u << ql_buf;
                        mbar_expect_tx(smem_u32(&sh.qfull[ql_buf]), kFuTileBytes);
                        for (int a = 0; a < 2; ++a)
                            tma_load_2d(q_smem + ql_buf * kFuTileBytes + a * kAtomBytes, &tmQ, smem_u32(&sh.qfull[ql_buf]), a * 64,
                                        ql_prob * g.H * g.window + ql_j * R, pol_q);
                    }
                    ++ql_phase;
                    ql_buf = ql_buf == kFuQBufs - 1 ? 0 : ql_buf + 1;
                    if (++ql_j == g.Hkv) {
                        ql_j = 0;
                        ql_vp += it.n_groups;
                        if (ql_phase < it.n_phases) {
                            const FuProb m = fu_prob(fa, g, ql_vp);
                            const int L = geo_L(g, m.seq);
                            ql_prob = m.prob;
                            ql_tiles = L > g.n_out && it.rank < (L + kTcTile - 1) / kTcTile;
                        }
                    }
                }
                if (!ok) break;
                // ---- the K tile of the step
                const int st = n_steps % kFuStages, par = (n_steps / kFuStages) & 1;
                if (!FU_WAIT(2, mbar_wait(smem_u32(&sh.empty[st]), par ^ 1, abort_flag))) break;
                mbar_expect_tx(smem_u32(&sh.full[st]), kFuTileBytes);
                for (int a = 0; a < 2; ++a)
                    tma_load_4d(k_smem + st * kFuTileBytes + a * kAtomBytes, &tmK, smem_u32(&sh.full[st]), a * 64, ph.j,
                                ph.tok_base + tok0, ph.layer, is_b ? pol_b : pol_a);
                ++n_steps;
            }
            sched_post(sched, n_steps, kStepStop);
            // the end of each epilogue set's list (also after a wait that gave up: the sets then
            // leave through the abort flag)
            for (int es = 0; es < 2; ++es) {
                const int k = (n_steps + 1 - es) >> 1;         // steps set es has had
                const bool other_was_last = prev_last_a && ((n_steps - 1) & 1) != es;
                sched_post_set(sched, es, k, make_int4(kStepStop | (other_was_last ? kStepPrevLastA : 0), 0, 0, 0));
            }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // One thread issues every product (the two accumulators alternate with the steps).  Issuing
        // blocks for about as long as the tensor core needs for the tile, so everything else this
        // thread does per step is kept short: no state in local memory, barrier probes whose
        // latencies overlap, the next step's record fetched while the products are issued.
        // It runs at a fraction of an instruction per clock (four epilogue warps share its
        // scheduler), so the loop keeps its own arithmetic to a minimum: ring positions, parities and
        // the start-address fields of the descriptors are carried along instead of recomputed.
        if (lane == 0) {
            const uint32_t q_lo0 = (q_smem & 0x3FFFFu) >> 4, k_lo0 = (k_smem & 0x3FFFFu) >> 4;    // descriptor start-address fields
            constexpr uint32_t kTileLo = kFuTileBytes >> 4;
            const uint32_t bar_full0 = smem_u32(&sh.full[0]), bar_empty0 = smem_u32(&sh.empty[0]);
            const uint32_t bar_tfull0 = smem_u32(&sh.tfull[0]), bar_tempty0 = smem_u32(&sh.tempty[0]);
            int n = 0, flags = 0, flags_next = 0;
            uint32_t st = 0, kpar = 0;                         // K stage of the step and the parity of its fill
            bool have_next = false;
            while (true) {
                if (have_next) {
                    flags = flags_next;
                } else if (!sched_get(sched, n, flags, abort_flag)) {
                    break;
                }
                have_next = false;
                if (flags & kStepStop) break;
                if (flags & (7 << kStepRelShift)) {
#pragma unroll
                    for (int i = 0; i < kFuQBufs; ++i)
                        if (flags & (1 << (kStepRelShift + i))) tc_commit(smem_u32(&sh.qempty[i]));
                }
                const uint32_t b = (uint32_t)(flags >> kStepQBufShift) & 3u;
                const uint32_t acc = (uint32_t)n & 1u;             // accumulator of the step
                const uint32_t te_par = (((uint32_t)n >> 1) & 1u) ^ 1u;
                const uint32_t bar_te = bar_tempty0 + acc * 8u, bar_k = bar_full0 + st * 8u;
                // both barriers are probed before either result is looked at, so that their
                // latencies overlap; only a barrier that is not complete yet is waited for
                bool te_ok, k_ok;
                mbar_test_wait2(bar_te, te_par, bar_k, kpar, te_ok, k_ok);
                // the first product that uses a load of the query block waits for it
                if ((flags & kStepNewQ) && !FU_WAIT(3, mbar_wait(smem_u32(&sh.qfull[b]), (flags & kStepQPar) ? 1u : 0u, abort_flag))) break;
                if (!te_ok && !FU_WAIT(4, mbar_wait(bar_te, te_par, abort_flag))) break;
                if (!k_ok && !FU_WAIT(5, mbar_wait(bar_k, kpar, abort_flag))) break;
                tc_fence_after();
                // the next step's flags, if it is posted, come in while the products are issued
                flags_next = sched_peek(sched, n + 1);
                have_next = sched_posted(flags_next, n + 1, kFuRing);
                const uint32_t k_lo = k_lo0 + st * kTileLo, q_lo = q_lo0 + b * kTileLo;
                const bool is_b = (flags & kStepB) != 0;
                fu_issue_tile(tmem + acc * 128u, is_b ? k_lo : q_lo, is_b ? q_lo : k_lo);   // rows = tokens (B) or window rows (A)
                tc_commit(bar_empty0 + st * 8u);
                tc_commit(bar_tfull0 + acc * 8u);
                ++n;
                if (++st == kFuStages) { st = 0; kpar ^= 1u; }
            }
        }
    } else if (warp == kFuHelpWarp && fa.neg_lse2 == nullptr) {
        // ------------------------------------------------------------------ hand-over between CTAs
        // Per phase, in this order: publish this CTA's row sums (the epilogue left the four (set, half)
        // partial sums of every window row in shared memory), merge the sums of all CTAs for this
        // CTA's share of the rows, fetch the finished log-sum-exps for this CTA's sweep B.
        const int group = blockIdx.x / fa.cpp, rank = blockIdx.x % fa.cpp;
        const int my_probs = group < fa.n_groups ? (fa.n_prob - group + fa.n_groups - 1) / fa.n_groups : 0;
        const int n_phases = my_probs * g.Hkv;
        const int n_mergers = min(fa.cpp, R);
        int n_fetch = 0, n_pub = 0;
        for (int phase = 0; phase < n_phases; ++phase) {
            const FuProb pm = fu_prob(fa, g, group + (phase / g.Hkv) * fa.n_groups);
            const int prob = pm.prob, j = phase % g.Hkv, seq = pm.seq;
            if (geo_identity(g, seq)) continue;
            const int L = geo_L(g, seq);
            const int nt1 = (L + kTcTile - 1) / kTcTile, nt2 = (L - g.window + kTcTile - 1) / kTcTile;
            const int n_src = min(fa.cpp, nt1);                 // CTAs that hold tiles of this problem
            bool ok = true;
            if (rank < nt1) {
                // the slot of the partial ring is free once the phase that used it last is merged
                if (lane == 0 && phase >= kFuPartSlots) {
                    const int old = phase - kFuPartSlots;
                    const int old_prob = fu_prob(fa, g, group + (old / g.Hkv) * fa.n_groups).prob;
                    ok = FU_WAIT(11, wait_counter(fa.done + old_prob * g.Hkv + old % g.Hkv, n_mergers, abort_flag, fa.status));
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                const int buf = n_pub & 1;
                if (!FU_WAIT(6, mbar_wait(smem_u32(&sh.pub_full[buf]), (uint32_t)((n_pub >> 1) & 1), abort_flag))) break;
                float2* dst = fa.part + (((size_t)group * kFuPartSlots + (phase % kFuPartSlots)) * fa.cpp + rank) * R;
                // all partial sums of this lane's four rows first (the loads overlap), then the merges;
                // the reference exponents are integers, so the rescaling is exact
                float2 pv[4][4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int x = 0; x < 4; ++x) pv[u][x] = pub_s[buf][x][lane + 32 * u];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float m = -INFINITY;
#pragma unroll
                    for (int x = 0; x < 4; ++x)
                        if (pv[u][x].y > 0.f) m = fmaxf(m, pv[u][x].x);
                    float l = 0.f;
#pragma unroll
                    for (int x = 0; x < 4; ++x)
                        if (pv[u][x].y > 0.f) l += pv[u][x].y * pow2_nonpos((int)(pv[u][x].x - m));
                    dst[lane + 32 * u] = make_float2(l > 0.f ? m : 0.f, l);
                }
                __threadfence();
                __syncwarp();
                ++n_pub;
                if (lane == 0) {
                    st_release_cta(&sched.pub_done, n_pub);
                    if (!(SAB_HOOK(2) && blockIdx.x == 0 && phase == 0)) atomicAdd(fa.arrive + prob * g.Hkv + j, 1);
                }
            }
            if (rank < R) {
                if (lane == 0) ok = FU_WAIT(12, wait_counter(fa.arrive + prob * g.Hkv + j, n_src, abort_flag, fa.status));
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                const float2* pp = fa.part + ((size_t)group * kFuPartSlots + (phase % kFuPartSlots)) * fa.cpp * R;
                for (int row = rank; row < R; row += fa.cpp) {
                    // one partial per source CTA, merged in index order; all loads of a lane are issued
                    // before the first use so that their latencies overlap
                    constexpr int kPer = kFuMaxCtasDev / 32;
                    float2 v[kPer];
#pragma unroll
                    for (int u = 0; u < kPer; ++u) {
                        const int i = lane + 32 * u;
                        v[u] = i < n_src ? __ldcg(pp + (size_t)i * R + row) : make_float2(0.f, 0.f);
                    }
                    // Reference exponents are integer-valued: their maximum over the warp is an integer
                    // reduction.  The sum over the warp is taken in fixed point relative to the
                    // largest lane sum (26 bits each, 31 in all), so that it does not depend on an
                    // order and needs one reduction instead of five exchanges.
                    int mi = INT_MIN;
#pragma unroll
                    for (int u = 0; u < kPer; ++u)
                        if (v[u].y > 0.f) mi = max(mi, (int)v[u].x);
                    mi = redux_max_s32(mi);
                    const float m = (float)mi;
                    float l = 0.f;
#pragma unroll
                    for (int u = 0; u < kPer; ++u)
                        if (v[u].y > 0.f) l += v[u].y * pow2_nonpos((int)v[u].x - mi);
                    const unsigned lmax = redux_max_u32(__float_as_uint(l));      // l >= 0: bit pattern orders like the value
                    if (lmax != 0u) {
                        const int ex = min(max((int)(lmax >> 23) - 127, -100), 100);   // 2^ex <= largest lane sum < 2^(ex + 1)
                        const float up = __int_as_float((127 + 25 - ex) << 23), down = __int_as_float((127 - 25 + ex) << 23);
                        const unsigned q = (unsigned)(l * up + 0.5f);                 // < 2^26
                        l = (float)redux_add_u32(q) * down;
                    }
                    if (lane == 0) fa.lse2[(size_t)prob * g.H * g.window + j * R + row] = m + log2f(l);
                }
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    atomicAdd(fa.done + prob * g.Hkv + j, 1);
                }
            }
            // the finished log-sum-exps, if this CTA runs sweep B for the phase
            if (rank < nt2) {
                if (lane == 0) ok = FU_WAIT(13, wait_counter(fa.done + prob * g.Hkv + j, n_mergers, abort_flag, fa.status));
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                const int slot = n_fetch % kFuLseSlots;
                const float* src = fa.lse2 + (size_t)prob * g.H * g.window + j * R;
#pragma unroll
                for (int u = 0; u < 4; ++u) lse_s[slot][lane + 32 * u] = -__ldcg(src + lane + 32 * u);   // negated: the epilogue adds it
                __syncwarp();
                ++n_fetch;
                if (lane == 0) {
                    mbar_arrive(smem_u32(&sh.lse_full[slot]));
                    st_release_cta(&sched.lse_fetched, n_fetch);
                }
            }
        }
    } else if (warp >= kFuEpiWarp0 && warp < kFuEpiWarp0 + kFuEpiWarps) {
        // ------------------------------------------------------------------ epilogue
        const int ew = warp - kFuEpiWarp0;
        const int q4 = warp & 3;                       // tensor-memory lane quarter of this warp
        const int set = (ew >> 2) & 1;
        const int half = ew >> 3;
        const int row = q4 * 32 + lane;                // TMEM lane: window row (sweep A) or token (sweep B)
        const uint32_t lane_addr = tmem + ((uint32_t)(q4 * 32) << 16);
        const uint32_t acc_addr = lane_addr + (uint32_t)set * 128u;
        const float c2 = fa.c2;
        const float inv_H = 1.f / (float)g.H;
        RowSum rs;                                     // sweep A state of (window row, set, half)
        rs.reset();
        int n_mine = 0, n_pub = 0, n_psync = 0, n_fin = 0;
        // Hands this thread's row sum of a phase to the helper warp (no waiting unless the helper is
        // two phases behind).
        auto publish = [&]() -> bool {
            const int buf = n_pub & 1;
            if (n_pub >= 2 && ld_acquire_cta(&sched.pub_done) < n_pub - 1) {
                const long long t0 = clock64();
                while (ld_acquire_cta(&sched.pub_done) < n_pub - 1) {
                    if (*abort_flag || clock64() - t0 > kWaitLimitCycles) { note_giveup(fa.status, 21); *abort_flag = 1; break; }
                }
                if (*abort_flag) return false;
            }
            pub_s[buf][set * 2 + half][row] = make_float2(rs.m, rs.l);
            mbar_arrive(smem_u32(&sh.pub_full[buf]));
            ++n_pub;
            rs.reset();
            return true;
        };
        int4 e;
        // Read ahead during a step's exponentials, so that the latencies do not add up between two
        // steps: the flags of the set's next step, and whether its accumulator is complete already.
        int ahead_flags = 0;
        bool ahead_tfull = false;
        while (true) {
            if (sched_flags_posted(ahead_flags, n_mine)) {
                e.x = ahead_flags;
            } else {
                if (!sched_get_set(sched, set, n_mine, e.x, abort_flag)) break;
                ahead_tfull = false;
            }
            const int flags = e.x;
            // the other set took the last sweep A step of a phase: this thread's row sums are due too
            if ((flags & kStepPrevLastA) && !publish()) break;
            if (flags & kStepStop) break;
            if (!(flags & kStepB)) {
                {
                    if (!ahead_tfull && !FU_WAIT(7, mbar_wait(smem_u32(&sh.tfull[set]), (uint32_t)(n_mine & 1), abort_flag))) break;
                    tc_fence_after();
                    uint32_t r0[32], r1[32];
                    tmem_ld32_issue(acc_addr + half * 64, r0);
                    tmem_ld32_issue(acc_addr + half * 64 + 32, r1);
                    tmem_ld_wait();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&sh.tempty[set]));   // logits are in registers
                    if (flags & kStepMask) {
                        sched_payload(sched, set, n_mine, e);
                        const int tok0 = e.y + half * 64;
                        const int lim = e.z + (row & 31);          // causal: key index <= T + w (Eq. 2)
                        chunk_mask(r0, tok0, lim);
                        chunk_mask(r1, tok0 + 32, lim);
                    }
                    if (!FU_WAIT(9, mbar_wait(smem_u32(&sh.xu[set]), (uint32_t)((n_mine & 1) ^ (set ^ 1)), abort_flag))) break;
                    rs.add(r0, c2);
                    mbar_arrive(smem_u32(&sh.xu[set ^ 1]));
                    ahead_flags = sched_peek_flags(sched, set, n_mine + 1);
                    rs.add(r1, c2);
                    ahead_tfull = mbar_test_wait(smem_u32(&sh.tfull[set]), (uint32_t)((n_mine + 1) & 1));
                    mbar_arrive(smem_u32(&sh.adone[set][n_mine & 1]));      // every step counts, so that the parities below hold
                    ++n_mine;
                }
                if ((flags & kStepLastA) && !publish()) break;
            } else {
                {
                    const int lse_slot = (flags >> kStepLseShift) & (kFuLseSlots - 1);
                    if (flags & kStepLseWait) {                    // log-sum-exps of this phase (fetched by warp 18)
                        if (!FU_WAIT(8, mbar_wait(smem_u32(&sh.lse_full[lse_slot]), (uint32_t)((flags >> (kStepLseShift + 4)) & 1), abort_flag)))
                            break;
                    }
                    if (!ahead_tfull && !FU_WAIT(7, mbar_wait(smem_u32(&sh.tfull[set]), (uint32_t)(n_mine & 1), abort_flag))) break;
                    tc_fence_after();
                    const float* lj = lse_s[lse_slot] + half * 16;
                    float accw[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) accw[i] = 0.f;
                    uint32_t v0[16], v1[16], v2[16], v3[16];       // query head hl of the group, 16 window positions
                    tmem_ld16_issue(acc_addr + half * 16, v0);
                    tmem_ld16_issue(acc_addr + 32 + half * 16, v1);
                    tmem_ld16_issue(acc_addr + 64 + half * 16, v2);
                    tmem_ld16_issue(acc_addr + 96 + half * 16, v3);
                    tmem_ld_wait();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&sh.tempty[set]));
                    if (!FU_WAIT(9, mbar_wait(smem_u32(&sh.xu[set]), (uint32_t)((n_mine & 1) ^ (set ^ 1)), abort_flag))) break;
                    accumulate_head16(accw, v0, lj, c2);
                    accumulate_head16(accw, v1, lj + 32, c2);
                    ahead_flags = sched_peek_flags(sched, set, n_mine + 1);
                    accumulate_head16(accw, v2, lj + 64, c2);
                    mbar_arrive(smem_u32(&sh.xu[set ^ 1]));
                    accumulate_head16(accw, v3, lj + 96, c2);
                    ahead_tfull = mbar_test_wait(smem_u32(&sh.tfull[set]), (uint32_t)((n_mine + 1) & 1));
                    // \bar A of this token tile, summed over the KV heads seen so far.  The step before this
                    // one belongs to the other set and may have updated the same tile's columns (a CTA with
                    // one tile per phase alternates the sets on it): wait until that set is through its step.
                    // Set 0's k-th step follows set 1's (k - 1)-th, set 1's k-th follows set 0's k-th.  A set's
                    // steps alternate between two barriers, so that the other set being one step ahead
                    // (it cannot be two) does not make the awaited phase ambiguous.
                    if (set == 1 || n_mine > 0) {
                        const int ko = n_mine - (set ^ 1);             // the other set's step that precedes this one
                        if (!FU_WAIT(22, mbar_wait(smem_u32(&sh.adone[set ^ 1][ko & 1]), (uint32_t)((ko >> 1) & 1), abort_flag))) break;
                        tc_fence_after();
                    }
                    const uint32_t abar_addr = lane_addr + (uint32_t)(kFuAbarCol0 + ((flags >> kStepKShift) & 7) * 32 + half * 16);
                    if (!(flags & kStepHead0)) {
                        tmem_ld16_issue(abar_addr, v0);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i) accw[i] += __uint_as_float(v0[i]);
                    }
                    if (!(flags & kStepHeadLast)) {
                        tmem_st16(abar_addr, accw);
                        tmem_st_wait();
                        tc_fence_before();         // the next head's update may come from the other set's warps
                    } else {
                        // last KV head of the layer: s_t (Eqs. 3, 4) and the entropy of Eq. 6; the two warps
                        // that hold the halves of a token's window positions exchange partial sums
                        const int par = n_fin & 1;
                        ++n_fin;
                        float t0 = 0.f, t1 = 0.f;
#pragma unroll
                        for (int i = 0; i < 16; i += 2) { t0 += accw[i]; t1 += accw[i + 1]; }
                        xch[set][par][0][half][row] = t0 + t1;
                        if (!FU_WAIT(20, group_sync(&sh.pbar[set][q4], n_psync, abort_flag))) break;
                        const float tot = xch[set][par][0][0][row] + xch[set][par][0][1][row];
                        float ent_h = 0.f;
                        if (tot > 0.f) {
                            const float inv = 1.f / tot;
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const float ah = accw[i] * inv;                       // \hat A (Eq. 6)
                                ent_h -= ah * (lg2_approx(ah + fa.eps) * 0.6931471805599453f);
                            }
                        }
                        xch[set][par][1][half][row] = ent_h;
                        if (!FU_WAIT(20, group_sync(&sh.pbar[set][q4], n_psync, abort_flag))) break;
                        sched_payload(sched, set, n_mine, e);
                        const int t = e.y + row;
                        if (half == 0 && t < e.z) {
                            const unsigned o = (unsigned)e.w + (unsigned)t;            // row of the [layer][token] outputs
                            if (o < (unsigned)g.n_layers * (unsigned)g.total_tokens) {
                                fa.s_out[o] = tot * inv_H;
                                fa.e_out[o] = xch[set][par][1][0][row] + xch[set][par][1][1][row];
                            } else {
                                atomicOr(fa.status, kStatInternal);                    // a step record that cannot be right
                            }
                        }
                    }
                    mbar_arrive(smem_u32(&sh.adone[set][n_mine & 1]));
                    ++n_mine;
                }
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
