// Stage 2 with plain fp32 FMAs (any head_dim / window the tensor-core kernels do not take,
// and fp32 inputs).  Two sweeps over K: pass 1 produces the log-sum-exp of every window
// row (h, w) over its causal keys (Eq. 2), pass 2 recomputes the logits, normalises, and
// reduces over heads and window positions per token (Eqs. 3, 4 and the inner sum of Eq. 6).
// Logits are kept in log2 units: x2 = (q . k) * log2(e) / sqrt(D).
#pragma once
#include "common.cuh"

namespace sab {

constexpr int kSimtThreads = 128;
constexpr int kSimtWChunk = 16;
constexpr int kSimtMaxW = 64;
constexpr int kSimtMaxD = 256;

// Partial row statistics of pass 1: (m, l) with m the running maximum (log2 units) and
// l = sum exp2(x2 - m) over the keys seen.
struct ScoreBufs {
    float2* part;          // [n_prob][H*W][n_chunks]   (SIMT)  or [n_prob][Hkv][n_chunks][128] (tensor)
    float* lse2;           // [n_prob][H*W]
    int n_chunks;
};

// Single-sweep mode: the caller knows ln sum_j exp(logit_j) of every window row (the prefill's
// attention kernel keeps it).  Converts it to the log2 units the score kernels work in, once as it
// is and once negated (the persistent kernel adds it).
__global__ void lse_import_kernel(const float* __restrict__ row_lse, float* __restrict__ lse2,
                                  float* __restrict__ neg_lse2, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float v = row_lse[i] * 1.4426950408889634f;
    lse2[i] = v;
    neg_lse2[i] = -v;
}

template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
score_p1_simt(Geo g, const T* __restrict__ q, const T* __restrict__ k, long long ks_tok, long long ks_head,
              long long ks_layer, float c2, ScoreBufs sb)
{
    const int p = blockIdx.z, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const int L = geo_L(g, seq), Tn = L - g.window, W = g.window, D = g.D;
    const int chunk = blockIdx.x, h = blockIdx.y;
    if (chunk * kSimtThreads >= L) return;
    const int j = h / g.G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    extern __shared__ float smem[];
    float* qs = smem;                                   // [W][D]
    float* wm = smem + W * D;                           // [4][W] warp maxima
    float* wl = wm + (kSimtThreads / 32) * W;           // [4][W] warp sums
    const T* qh = q + ((size_t)p * g.H + h) * W * D;
    for (int i = tid; i < W * D; i += kSimtThreads) qs[i] = ld_as_float(qh + i);
    __syncthreads();
    const int i_key = chunk * kSimtThreads + tid;
    const bool in_seq = i_key < L;
    const T* kr = k + (size_t)layer * ks_layer + ((size_t)g.cu[seq] + (in_seq ? i_key : 0)) * ks_tok +
                  (size_t)j * ks_head;
    for (int w0 = 0; w0 < W; w0 += kSimtWChunk) {
        float acc[kSimtWChunk];
#pragma unroll
        for (int u = 0; u < kSimtWChunk; ++u) acc[u] = 0.f;
        for (int d = 0; d < D; ++d) {
            const float kd = ld_as_float(kr + d);
#pragma unroll
            for (int u = 0; u < kSimtWChunk; ++u)
                if (w0 + u < W) acc[u] = fmaf(qs[(w0 + u) * D + d], kd, acc[u]);
        }
#pragma unroll
        for (int u = 0; u < kSimtWChunk; ++u) {
            const int w = w0 + u;
            if (w >= W) break;
            const bool valid = in_seq && i_key <= Tn + w;        // causal (Eq. 2)
            const float x2 = valid ? acc[u] * c2 : -INFINITY;
            float m = x2;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            const float ms = (m == -INFINITY) ? 0.f : m;
            float l = valid ? exp2f(x2 - ms) : 0.f;
            l = warp_sum(l);
            if (lane == 0) {
                wm[warp * W + w] = m;
                wl[warp * W + w] = l;
            }
        }
    }
    __syncthreads();
    if (tid < W) {
        float m = -INFINITY;
        for (int x = 0; x < kSimtThreads / 32; ++x) m = fmaxf(m, wm[x * W + tid]);
        const float ms = (m == -INFINITY) ? 0.f : m;
        float l = 0.f;
        for (int x = 0; x < kSimtThreads / 32; ++x) l += wl[x * W + tid] * exp2f(wm[x * W + tid] - ms);
        sb.part[((size_t)p * g.H * W + (size_t)h * W + tid) * sb.n_chunks + chunk] = make_float2(m, l);
    }
}

// lse2[row] = log2 sum_j exp2(x2_j) from the per-chunk partials, merged in chunk order.
__global__ void lse_merge_simt(Geo g, ScoreBufs sb)
{
    const int p = blockIdx.y, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const int rows = g.H * g.window;
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    const int L = geo_L(g, seq);
    const int nch = (L + kSimtThreads - 1) / kSimtThreads;
    const float2* pr = sb.part + ((size_t)p * rows + row) * sb.n_chunks;
    float m = -INFINITY;
    for (int c = 0; c < nch; ++c) m = fmaxf(m, pr[c].x);
    float l = 0.f;
    for (int c = 0; c < nch; ++c) l += pr[c].y * exp2f(pr[c].x - m);
    sb.lse2[(size_t)p * rows + row] = m + log2f(l);
}

template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
score_p2_simt(Geo g, const T* __restrict__ q, const T* __restrict__ k, long long ks_tok, long long ks_head,
              long long ks_layer, float c2, float eps, ScoreBufs sb, float* __restrict__ s_out,
              float* __restrict__ e_out)
{
    const int p = blockIdx.y, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const int L = geo_L(g, seq), Tn = L - g.window, W = g.window, D = g.D, H = g.H;
    if (blockIdx.x * kSimtThreads >= Tn) return;
    const int tid = threadIdx.x;
    const int t = blockIdx.x * kSimtThreads + tid;
    const bool live = t < Tn;
    extern __shared__ float smem[];
    float* qs = smem;                                   // [kSimtWChunk][D]
    float* ls = smem + kSimtWChunk * D;                 // [kSimtWChunk]
    const float* lse = sb.lse2 + (size_t)p * H * W;
    const size_t tok = (size_t)g.cu[seq] + (live ? t : 0);
    float abar[kSimtMaxW];
#pragma unroll
    for (int w = 0; w < kSimtMaxW; ++w) abar[w] = 0.f;
#pragma unroll
    for (int wc = 0; wc < kSimtMaxW / kSimtWChunk; ++wc) {
        const int w0 = wc * kSimtWChunk;
        if (w0 >= W) break;
        float a16[kSimtWChunk];
#pragma unroll
        for (int u = 0; u < kSimtWChunk; ++u) a16[u] = 0.f;
        for (int h = 0; h < H; ++h) {
            __syncthreads();
            const T* qh = q + (((size_t)p * H + h) * W + w0) * D;
            const int nw = min(kSimtWChunk, W - w0);
            for (int i = tid; i < nw * D; i += kSimtThreads) qs[i] = ld_as_float(qh + i);
            if (tid < nw) ls[tid] = lse[h * W + w0 + tid];
            __syncthreads();
            const T* kr = k + (size_t)layer * ks_layer + tok * ks_tok + (size_t)(h / g.G) * ks_head;
            float acc[kSimtWChunk];
#pragma unroll
            for (int u = 0; u < kSimtWChunk; ++u) acc[u] = 0.f;
            for (int d = 0; d < D; ++d) {
                const float kd = ld_as_float(kr + d);
#pragma unroll
                for (int u = 0; u < kSimtWChunk; ++u)
                    if (u < nw) acc[u] = fmaf(qs[u * D + d], kd, acc[u]);
            }
#pragma unroll
            for (int u = 0; u < kSimtWChunk; ++u)
                if (u < nw) a16[u] += exp2f(acc[u] * c2 - ls[u]);      // A[h, w, t]
        }
#pragma unroll
        for (int u = 0; u < kSimtWChunk; ++u) abar[w0 + u] = a16[u];
    }
    if (!live) return;
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kSimtMaxW; ++w)
        if (w < W) tot += abar[w];
    float ent = 0.f;
    if (tot > 0.f) {
        const float inv = 1.f / tot;
#pragma unroll
        for (int w = 0; w < kSimtMaxW; ++w)
            if (w < W) {
                const float ah = abar[w] * inv;                          // \hat A (Eq. 6)
                ent -= ah * logf(ah + eps);
            }
    }
    const size_t off = (size_t)layer * g.total_tokens + g.cu[seq];
    s_out[off + t] = tot / (float)H;                                     // Eqs. 3, 4
    e_out[off + t] = ent;
}

}  // namespace sab
