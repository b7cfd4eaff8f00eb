// Decoding over a (compacted) cache: attention of one new query token per problem against the
// cache rows, grouped-query attention (Eqs. 1-2 with a single query row; Sec. 4.4 measures
// decoding over the compressed cache against the full one).  The work is a stream over K and V
// with 2 * G flops per loaded element (G = query heads per KV head, 4 for Llama-3-8B), far below
// the tensor-core ridge, so it runs on plain FMAs with 16-byte coalesced loads.
//
// grid = (splits, KV heads, problems).  A CTA walks its share of the rows in chunks of 256:
//   1. thread = row: the G logits of the row (K row read as 16-byte vectors, queries in shared
//      memory, pre-scaled to log2 units);
//   2. CTA-wide running maximum and sum per head (online softmax), weights to shared memory;
//   3. thread = (row slice, 16-byte piece of the head dimension): weighted sum of the V rows, each
//      V row read by consecutive lanes.
// The splits of a problem leave (accumulator, max, sum) in scratch; a second kernel merges them in
// split order (fixed order: results are reproducible).
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

template <typename T> struct DecVec;
template <> struct DecVec<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static void load(const __nv_bfloat16* p, float (&x)[8])
    {
        const uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {                // bf16 -> fp32 is a shift of the bit pattern
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};
template <> struct DecVec<float> {
    static constexpr int kElems = 4;
    __device__ static void load(const float* p, float (&x)[4])
    {
        const float4 u = __ldg(reinterpret_cast<const float4*>(p));
        x[0] = u.x; x[1] = u.y; x[2] = u.z; x[3] = u.w;
    }
};

template <typename T, int G>
__global__ void __launch_bounds__(kDecThreads)
decode_partial_kernel(DecodeArgs a)
{
    constexpr int E = DecVec<T>::kElems;             // elements per 16-byte vector
    const int split = blockIdx.x, j = blockIdx.y, p = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int D = a.D;
    const int n = a.n_valid ? min(a.n_valid[p], a.n_rows) : a.n_rows;
    const int r0 = split * a.rows_per_split, r1 = min(r0 + a.rows_per_split, n);
    const int lpk = D / E;                           // lanes that share one V row (8, 16 or 32)
    const int n_slices = kDecThreads / lpk;          // row slices of step 3
    const int slice = tid / lpk, piece = tid - slice * lpk;

    __shared__ __align__(16) float qs[G][kDecMaxD];
    __shared__ __align__(16) float ps[kDecThreads][G];
    __shared__ float red[2][kDecThreads / 32][G];
    __shared__ __align__(16) float accs[kDecThreads / 32][G][kDecMaxD];

    const T* qg = static_cast<const T*>(a.q) + ((size_t)p * a.H + (size_t)j * G) * D;
    for (int i = tid; i < G * D; i += kDecThreads) qs[i / D][i % D] = ld_as_float(qg + i) * a.c2;
    __syncthreads();

    const T* kb = static_cast<const T*>(a.k) + (size_t)p * a.k_prob + (size_t)j * a.k_head;
    const T* vb = static_cast<const T*>(a.v) + (size_t)p * a.v_prob + (size_t)j * a.v_head;

    float m[G], l[G], acc[G][E];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        m[h] = -INFINITY;
        l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[h][e] = 0.f;
    }

    for (int c0 = r0; c0 < r1; c0 += kDecThreads) {
        // ---- 1. logits of this thread's row
        const int row = c0 + tid;
        const bool valid = row < r1;
        float s[G];
#pragma unroll
        for (int h = 0; h < G; ++h) s[h] = 0.f;
        if (valid) {
            const T* kr = kb + (size_t)row * a.k_row;
            for (int d0 = 0; d0 < D; d0 += E) {
                float x[E];
                DecVec<T>::load(kr + d0, x);
#pragma unroll
                for (int h = 0; h < G; ++h)
#pragma unroll
                    for (int e = 0; e < E; ++e) s[h] = fmaf(qs[h][d0 + e], x[e], s[h]);
            }
        }
        // ---- 2. running maximum and sum per head over the CTA
        float wmax[G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float x = valid ? s[h] : -INFINITY;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
            wmax[h] = x;
        }
        if (lane == 0) {
#pragma unroll
            for (int h = 0; h < G; ++h) red[0][warp][h] = wmax[h];
        }
        __syncthreads();
        float scale[G], pr[G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float mx = m[h];
#pragma unroll
            for (int w = 0; w < kDecThreads / 32; ++w) mx = fmaxf(mx, red[0][w][h]);
            // the chunk has at least one row, so mx is finite from the first chunk on
            scale[h] = m[h] == -INFINITY ? 0.f : exp2f(m[h] - mx);
            pr[h] = valid ? exp2f(s[h] - mx) : 0.f;
            m[h] = mx;
        }
        {
            float* pw = ps[tid];
#pragma unroll
            for (int h = 0; h < G; ++h) pw[h] = pr[h];
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float x = pr[h];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            if (lane == 0) red[1][warp][h] = x;
        }
        __syncthreads();
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < kDecThreads / 32; ++w) sum += red[1][w][h];
            l[h] = l[h] * scale[h] + sum;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[h][e] *= scale[h];
        }
        // ---- 3. weighted sum of the V rows: rows slice, slice + n_slices, ... of the chunk
        const int rows_here = min(kDecThreads, r1 - c0);
        for (int i = slice; i < rows_here; i += n_slices) {
            float x[E];
            DecVec<T>::load(vb + (size_t)(c0 + i) * a.v_row + piece * E, x);
            const float* pw = ps[i];
#pragma unroll
            for (int h = 0; h < G; ++h) {
                const float w = pw[h];
#pragma unroll
                for (int e = 0; e < E; ++e) acc[h][e] = fmaf(w, x[e], acc[h][e]);
            }
        }
        __syncthreads();                             // ps and red are written again by the next chunk
    }

    // ---- the CTA's result: sum of the row slices (slices of one warp by shuffles, warps through shared memory)
    for (int o = lpk; o < 32; o <<= 1) {
#pragma unroll
        for (int h = 0; h < G; ++h)
#pragma unroll
            for (int e = 0; e < E; ++e) acc[h][e] += __shfl_xor_sync(0xffffffffu, acc[h][e], o);
    }
    if (lane < lpk) {
#pragma unroll
        for (int h = 0; h < G; ++h)
#pragma unroll
            for (int e = 0; e < E; ++e) accs[warp][h][lane * E + e] = acc[h][e];
    }
    __syncthreads();
    for (int i = tid; i < G * D; i += kDecThreads) {
        const int h = i / D, d = i - h * D;
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < kDecThreads / 32; ++w) sum += accs[w][h][d];
        a.part[(((size_t)p * a.H + (size_t)j * G + h) * a.n_splits + split) * (D + 2) + d] = sum;
    }
    if (tid < G) {
        float* dst = a.part + (((size_t)p * a.H + (size_t)j * G + tid) * a.n_splits + split) * (D + 2) + D;
        // every thread holds the same m and l
        float mm = -INFINITY, ll = 0.f;
#pragma unroll
        for (int h = 0; h < G; ++h)
            if (h == tid) { mm = m[h]; ll = l[h]; }
        dst[0] = mm;
        dst[1] = ll;
    }
}

// out[p][h][:] = sum over the splits of acc * 2^(m - M) / sum over the splits of l * 2^(m - M), in split order.
__global__ void decode_merge_kernel(DecodeArgs a)
{
    const int h = blockIdx.x, p = blockIdx.y, d = threadIdx.x;
    const int D = a.D;
    const float* base = a.part + ((size_t)p * a.H + h) * a.n_splits * (D + 2);
    float M = -INFINITY;
    for (int s = 0; s < a.n_splits; ++s) M = fmaxf(M, base[(size_t)s * (D + 2) + D]);
    float num = 0.f, den = 0.f;
    if (M != -INFINITY) {
        for (int s = 0; s < a.n_splits; ++s) {
            const float* ps = base + (size_t)s * (D + 2);
            const float ms = ps[D];
            if (ms == -INFINITY) continue;           // a split without rows
            const float w = exp2f(ms - M);
            den += ps[D + 1] * w;
            if (d < D) num += ps[d] * w;
        }
    }
    if (d < D) a.out[((size_t)p * a.H + h) * D + d] = den > 0.f ? num / den : 0.f;
    if (a.lse && d == 0) a.lse[(size_t)p * a.H + h] = den > 0.f ? (M + log2f(den)) * 0.6931471805599453f : -INFINITY;
}

}  // namespace sab
