// Decoding over a (compacted) cache: attention of one new query token per problem against the
// cache rows, grouped-query attention (Eqs. 1-2 with a single query row; Sec. 4.4 measures
// decoding over the compressed cache against the full one).  The work is a stream over K and V
// with 2 * G flops per loaded element (G = query heads per KV head, 4 for Llama-3-8B), far below
// the tensor-core ridge, so it runs on plain FMAs with 16-byte coalesced loads.
//
// grid = (splits, KV heads, problems).  Inside a CTA a row of K or V is read by the 8, 16 or 32
// lanes that together hold its 128, 256 or 512 bytes; each such group of lanes runs an online
// softmax over its share of the split's rows and the groups are merged at the end.  The splits of
// a problem leave (accumulator, max, sum) in scratch; a second kernel merges them in split order.
// Every merge has a fixed order: results are reproducible.
#pragma once
#include "common.cuh"

namespace sab {

constexpr int kDecThreads = 256;
constexpr int kDecMaxSplits = 512;
constexpr int kDecMaxD = 256;
constexpr int kDecMaxG = 4;

struct DecodeArgs {
    const void* q;                                   // [n_prob][H][D]
    const void* k;                                   // [n_prob][n_rows][Hkv][D] through the strides below (elements)
    const void* v;
    long long k_prob, k_row, k_head, v_prob, v_row, v_head;
    const int* n_valid;                              // optional [n_prob]: rows of each problem that count
    int n_rows, n_splits, rows_per_split;
    int H, Hkv, D;
    float c2;                                        // log2(e) / sqrt(D)
    float* part;                                     // [n_prob][H][n_splits][D + 2]: accumulator, max (log2 units), sum
    float* out;                                      // [n_prob][H][D]
    float* lse;                                      // optional [n_prob][H]: natural log of the normaliser
};

// 16-byte asynchronous copy global -> shared (cp.async), grouped and waited for per thread.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// A 16-byte piece of a row as packed fp32 pairs.
template <typename T> struct DecVec;
template <> struct DecVec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static void unpack(const uint4 u, uint64_t (&x)[4])
    {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) x[i] = pack2u(w[i] << 16, w[i] & 0xffff0000u);   // bf16 -> fp32 is a shift of the bit pattern
    }
};
template <> struct DecVec<float> {
    static constexpr int kElems = 4;
    __device__ static void unpack(const uint4 u, uint64_t (&x)[2])
    {
        x[0] = pack2u(u.x, u.y);
        x[1] = pack2u(u.z, u.w);
    }
};

// D is the head dimension (compile time: the loops over a row unroll).  LPK = lanes that share a
// row: each lane owns one 16-byte piece of it, for K and for V alike, so a row is one coalesced
// load of LPK lanes and a warp holds 32 / LPK rows at a time.  A group of LPK lanes walks rows
// group, group + n_groups, ... of the split, kRowsPer rows per turn (that many loads in flight),
// and keeps its own running maximum, sum and accumulator (online softmax); nothing is shared
// between groups until the end, so the main loop has no barrier.  The pieces travel by cp.async
// into a ring of kDecStages turns in shared memory that each thread fills and reads for itself, so
// that the bytes in flight (what hides the DRAM latency) do not cost registers.
constexpr int kDecRowsPer = 4;
constexpr int kDecStages = 3;                        // turns in flight per thread (ring in shared memory)
constexpr int kDecSmemBytes = kDecStages * 2 * kDecRowsPer * kDecThreads * 16;

template <typename T, int G, int D>
__global__ void __launch_bounds__(kDecThreads, 2)
decode_partial_kernel(DecodeArgs a)
{
    constexpr int E = DecVec<T>::kElems;             // elements per 16-byte vector
    constexpr int LPK = D / E;                       // 8, 16 or 32
    constexpr int kGroups = kDecThreads / LPK;
    constexpr int R = kDecRowsPer;
    static_assert(LPK == 8 || LPK == 16 || LPK == 32, "row of 128, 256 or 512 bytes");
    const int split = blockIdx.x, j = blockIdx.y, p = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.n_valid ? min(a.n_valid[p], a.n_rows) : a.n_rows;
    const int r0 = split * a.rows_per_split, r1 = min(r0 + a.rows_per_split, n);
    const int group = tid / LPK, piece = tid % LPK;

    __shared__ float ms[kDecThreads / 32][G], ls[kDecThreads / 32][G];

    // the G queries in log2 units; a lane reads its own piece of them from shared memory every turn
    // (registers are better spent on loads in flight)
    __shared__ __align__(16) float qs[G][D];
    {
        const T* qg = static_cast<const T*>(a.q) + ((size_t)p * a.H + (size_t)j * G) * D;
        for (int i = tid; i < G * D; i += kDecThreads) qs[i / D][i % D] = ld_as_float(qg + i) * a.c2;
    }
    __syncthreads();
    const T* kb = static_cast<const T*>(a.k) + (size_t)p * a.k_prob + (size_t)j * a.k_head + piece * E;
    const T* vb = static_cast<const T*>(a.v) + (size_t)p * a.v_prob + (size_t)j * a.v_head + piece * E;

    constexpr int E2 = E / 2;
    float m[G], l[G];
    uint64_t acc[G][E2];                             // packed pairs of the accumulator
#pragma unroll
    for (int h = 0; h < G; ++h) {
        m[h] = -INFINITY;
        l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < E2; ++e) acc[h][e] = pack2(0.f, 0.f);
    }

    // Every lane of the CTA makes the same number of turns (the shuffles below involve whole warps);
    // a group whose turn lies beyond the split's last row works on masked rows.
    const int n_turns = r1 > r0 ? (r1 - r0 + kGroups * R - 1) / (kGroups * R) : 0;
    extern __shared__ __align__(16) uint8_t dec_ring[];
    uint4* ring = reinterpret_cast<uint4*>(dec_ring);      // [stage][piece 0 .. 2R)[thread] x 16 bytes
    // Copies of turn t into its stage of the ring (rows beyond the split read its last row and are
    // masked later); an empty group once the turns are used up keeps the group count in step.
    auto issue = [&](int t) {
        if (t < n_turns) {
            const int b = r0 + (t * kGroups + group) * R;
            const uint32_t dst = smem_u32(ring + (size_t)(t % kDecStages) * (2 * R) * kDecThreads + tid);
#pragma unroll
            for (int r = 0; r < R; ++r) cp_async16(dst + r * kDecThreads * 16, kb + (size_t)min(b + r, r1 - 1) * a.k_row);
#pragma unroll
            for (int r = 0; r < R; ++r) cp_async16(dst + (R + r) * kDecThreads * 16, vb + (size_t)min(b + r, r1 - 1) * a.v_row);
        }
        cp_async_commit();
    };
#pragma unroll
    for (int t = 0; t < kDecStages - 1; ++t) issue(t);
    for (int turn = 0; turn < n_turns; ++turn) {
        const int base = r0 + (turn * kGroups + group) * R;
        // ---- ask for the turn kDecStages - 1 ahead, then wait for this turn's 2 R pieces
        issue(turn + kDecStages - 1);
        cp_async_wait<kDecStages - 1>();
        uint64_t xk[R][E2], x[R][E2];
        float s[R][G];
        {
            const uint4* slot = ring + (size_t)(turn % kDecStages) * (2 * R) * kDecThreads + tid;
#pragma unroll
            for (int r = 0; r < R; ++r) DecVec<T>::unpack(slot[(size_t)r * kDecThreads], xk[r]);
#pragma unroll
            for (int r = 0; r < R; ++r) DecVec<T>::unpack(slot[(size_t)(R + r) * kDecThreads], x[r]);
        }
        // ---- logits: partial dot products of this lane's piece, summed over the group's lanes
#pragma unroll
        for (int h = 0; h < G; ++h) {
            uint64_t qf[E2];
#pragma unroll
            for (int e = 0; e < E2; e += 2) {
                const float4 t = *reinterpret_cast<const float4*>(&qs[h][piece * E + 2 * e]);
                qf[e] = pack2(t.x, t.y);
                qf[e + 1] = pack2(t.z, t.w);
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                uint64_t d = mul2(qf[0], xk[r][0]);
#pragma unroll
                for (int e = 1; e < E2; ++e) d = fma2(qf[e], xk[r][e], d);
                float lo, hi;
                unpack2(d, lo, hi);
                s[r][h] = lo + hi;
            }
        }
#pragma unroll
        for (int o = 1; o < LPK; o <<= 1)
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int h = 0; h < G; ++h) s[r][h] += __shfl_xor_sync(0xffffffffu, s[r][h], o);
        // ---- online softmax over the R rows, then the weighted V rows
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float mx = m[h];
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (base + r < r1) mx = fmaxf(mx, s[r][h]);
            const float scale = m[h] == -INFINITY ? 0.f : exp2f(m[h] - mx);      // mx is finite once a row has counted
            m[h] = mx;
            float sum = 0.f;
            uint64_t w2[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float w = base + r < r1 ? exp2f(s[r][h] - mx) : 0.f;
                w2[r] = pack2(w, w);
                sum += w;
            }
            l[h] = l[h] * scale + sum;
            const uint64_t sc2 = pack2(scale, scale);
#pragma unroll
            for (int e = 0; e < E2; ++e) {
                uint64_t v = mul2(acc[h][e], sc2);
#pragma unroll
                for (int r = 0; r < R; ++r) v = fma2(w2[r], x[r][e], v);
                acc[h][e] = v;
            }
        }
    }

    // ---- merge the groups of a warp (shuffles), then the warps (shared memory), in a fixed order.
    // The warps' accumulators go where the ring was: every copy has landed and, after the barrier,
    // every thread has read its last turn.
    cp_async_wait<0>();
    __syncthreads();
    float (*accs)[G][D] = reinterpret_cast<float (*)[G][D]>(dec_ring);
    static_assert(sizeof(float) * (kDecThreads / 32) * G * D <= kDecSmemBytes, "accumulators fit in the ring");
    float accf[G][E];
#pragma unroll
    for (int h = 0; h < G; ++h)
#pragma unroll
        for (int e = 0; e < E2; ++e) unpack2(acc[h][e], accf[h][2 * e], accf[h][2 * e + 1]);
#pragma unroll
    for (int o = LPK; o < 32; o <<= 1) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const float m_o = __shfl_xor_sync(0xffffffffu, m[h], o), l_o = __shfl_xor_sync(0xffffffffu, l[h], o);
            const float mx = fmaxf(m[h], m_o);
            const float w_me = m[h] == -INFINITY ? 0.f : exp2f(m[h] - mx), w_o = m_o == -INFINITY ? 0.f : exp2f(m_o - mx);
            l[h] = l[h] * w_me + l_o * w_o;
            m[h] = mx;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const float a_o = __shfl_xor_sync(0xffffffffu, accf[h][e], o);
                accf[h][e] = accf[h][e] * w_me + a_o * w_o;
            }
        }
    }
    if (lane < LPK) {
#pragma unroll
        for (int h = 0; h < G; ++h) {
            if (lane == 0) { ms[warp][h] = m[h]; ls[warp][h] = l[h]; }
#pragma unroll
            for (int e = 0; e < E; ++e) accs[warp][h][lane * E + e] = accf[h][e];
        }
    }
    __syncthreads();
    constexpr int kWarps = kDecThreads / 32;
    for (int i = tid; i < G * D; i += kDecThreads) {
        const int h = i / D, d = i - h * D;
        float mx = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) mx = fmaxf(mx, ms[w][h]);
        float sum = 0.f, lsum = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float wt = ms[w][h] == -INFINITY ? 0.f : exp2f(ms[w][h] - mx);
            sum += accs[w][h][d] * wt;
            lsum += ls[w][h] * wt;
        }
        float* dst = a.part + (((size_t)p * a.H + (size_t)j * G + h) * a.n_splits + split) * (D + 2);
        dst[d] = sum;
        if (d == 0) { dst[D] = mx; dst[D + 1] = lsum; }
    }
}

// out[p][h][:] = sum over the splits of acc * 2^(m - M) / sum over the splits of l * 2^(m - M).  The
// weights go through shared memory so that the loads of the D-wide sums are independent of one
// another; four slices of threads take every fourth split each and are added in slice order, so
// the summation order is fixed.  blockDim = kDecMergeSlices * dpad, dpad = D rounded up to 32.
constexpr int kDecMergeSlices = 4;

__global__ void __launch_bounds__(kDecMergeSlices * kDecMaxD)
decode_merge_kernel(DecodeArgs a)
{
    const int h = blockIdx.x, p = blockIdx.y, tid = threadIdx.x;
    const int D = a.D, ns = a.n_splits;
    const int dpad = blockDim.x / kDecMergeSlices, slice = tid / dpad, d = tid - slice * dpad;
    const float* base = a.part + ((size_t)p * a.H + h) * ns * (D + 2);
    __shared__ float w_s[kDecMaxSplits], lw_s[kDecMaxSplits];
    __shared__ float red[kDecMergeSlices * kDecMaxD / 32];
    __shared__ float num_s[kDecMergeSlices][kDecMaxD];
    float mx = -INFINITY;
    for (int s = tid; s < ns; s += blockDim.x) mx = fmaxf(mx, base[(size_t)s * (D + 2) + D]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((tid & 31) == 0) red[tid >> 5] = mx;
    __syncthreads();
    float M = -INFINITY;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) M = fmaxf(M, red[w]);
    for (int s = tid; s < ns; s += blockDim.x) {
        const float ms = base[(size_t)s * (D + 2) + D];
        const float w = (ms == -INFINITY || M == -INFINITY) ? 0.f : exp2f(ms - M);      // a split without rows weighs nothing
        w_s[s] = w;
        lw_s[s] = base[(size_t)s * (D + 2) + D + 1] * w;
    }
    __syncthreads();
    float num = 0.f;
    if (d < D) {
#pragma unroll 8
        for (int s = slice; s < ns; s += kDecMergeSlices) num = fmaf(base[(size_t)s * (D + 2) + d], w_s[s], num);
        num_s[slice][d] = num;
    }
    __syncthreads();
    if (slice == 0 && d < D) {
        float den = 0.f;
        for (int s = 0; s < ns; ++s) den += lw_s[s];
        float tot = 0.f;
#pragma unroll
        for (int q = 0; q < kDecMergeSlices; ++q) tot += num_s[q][d];
        a.out[((size_t)p * a.H + h) * D + d] = den > 0.f ? tot / den : 0.f;
        if (a.lse && d == 0) a.lse[(size_t)p * a.H + h] = den > 0.f ? (M + log2f(den)) * 0.6931471805599453f : -INFINITY;
    }
}

}  // namespace sab
