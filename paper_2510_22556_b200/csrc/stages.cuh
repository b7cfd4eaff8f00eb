// Stages 1, 3, 4, 5 of the compression pass: segmentation scan, segment-guided refinement,
// global Top-B radix select, per-segment block-size search, index list and K/V compaction.
// Each kernel is batched over problems (layer, sequence) through its grid.
#pragma once
#include "common.cuh"

namespace sab {

// ---------------------------------------------------------------------------------------
// Stage 1: segmentation (Sec. 3.1).  seg_id[t] = number of delimiters among tokens [0, t),
// i.e. an inclusive prefix sum of the "a segment starts here" flags f[t] = delim(t-1).
// Single pass over the tokens with a decoupled look-back between tiles: each tile publishes
// its aggregate, then its inclusive prefix, in one 64-bit word {flag, value}.
// ---------------------------------------------------------------------------------------
constexpr int kSegThreads = 256;
constexpr int kSegItems = 8;
constexpr int kSegTile = kSegThreads * kSegItems;

__device__ __forceinline__ int is_delim(int id, const unsigned* bitmap, int vocab)
{
    if (id < 0 || id >= vocab) return 0;
    return (__ldg(bitmap + (id >> 5)) >> (id & 31)) & 1u;
}

__global__ void __launch_bounds__(kSegThreads)
segment_kernel(Geo g, const int* __restrict__ token_ids, const unsigned* __restrict__ bitmap, int vocab,
               int* __restrict__ seg_id, int* __restrict__ seg_start, int* __restrict__ n_seg,
               unsigned long long* tile_state, int* ticket, int max_tiles, int* status, int* giveup)
{
    const int seq = blockIdx.y;
    const int T = geo_L(g, seq) - g.window;
    const int tid = threadIdx.x;
    if (T <= 0) {
        if (blockIdx.x == 0 && tid == 0) n_seg[seq] = 0;
        return;
    }
    const int ntiles = (T + kSegTile - 1) / kSegTile;
    __shared__ int s_tile, s_prefix;
    __shared__ int s_warp[kSegThreads / 32];
    // Tiles are handed out in launch order so that every predecessor of a running tile is
    // itself running or done: the look-back below always makes progress.
    if (tid == 0) s_tile = atomicAdd(&ticket[seq], 1);
    __syncthreads();
    const int tile = s_tile;
    if (tile >= ntiles) return;

    const int* ids = token_ids + g.cu[seq];
    int* sid = seg_id + g.cu[seq];
    int* sst = seg_start + g.cu[seq] + seq;
    unsigned long long* state = tile_state + (size_t)seq * max_tiles;

    const int base = tile * kSegTile + tid * kSegItems;
    int f[kSegItems];
    int cnt = 0;
#pragma unroll
    for (int i = 0; i < kSegItems; ++i) {
        int t = base + i;
        f[i] = (t >= 1 && t < T) ? is_delim(__ldg(ids + t - 1), bitmap, vocab) : 0;
        cnt += f[i];
    }
    // block-wide exclusive scan of cnt
    const int lane = tid & 31, warp = tid >> 5;
    int inc = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    int woff = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kSegThreads / 32; ++w) {
        int v = s_warp[w];
        if (w < warp) woff += v;
        total += v;
    }
    const int excl = woff + inc - cnt;

    if (tid == 0) {
        int prefix = 0;
        const bool withheld = SAB_HOOK(0) && tile == 1;       // test builds: this tile never publishes
        if (tile == 0) {
            *(volatile unsigned long long*)&state[0] = (2ull << 32) | (unsigned)total;
        } else {
            if (!withheld) *(volatile unsigned long long*)&state[tile] = (1ull << 32) | (unsigned)total;
            int j = tile - 1;
            const long long t0 = clock64();
            while (j >= 0) {
                unsigned long long st = *(volatile unsigned long long*)&state[j];
                unsigned flag = (unsigned)(st >> 32);
                if (flag == 0) {
                    if (clock64() - t0 > kWaitLimitCycles) {   // bounded: report and carry on
                        atomicOr(status, kStatTimeout);
                        if (giveup) atomicCAS(giveup, 0, kGiveupSegment | ((int)blockIdx.x << 8));
                        break;
                    }
                    __nanosleep(40);
                    continue;
                }
                prefix += (int)(unsigned)st;
                if (flag == 2) break;
                --j;
            }
            if (!withheld) *(volatile unsigned long long*)&state[tile] = (2ull << 32) | (unsigned)(prefix + total);
        }
        s_prefix = prefix;
    }
    __syncthreads();
    int run = s_prefix + excl;
#pragma unroll
    for (int i = 0; i < kSegItems; ++i) {
        int t = base + i;
        if (t < T) {
            run += f[i];
            sid[t] = run;
            if (f[i] || t == 0) sst[run] = t;
            if (t == T - 1) {
                n_seg[seq] = run + 1;
                sst[run + 1] = T;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Optional pooling of s_t over a clipped window (not part of the method's equations).
// ---------------------------------------------------------------------------------------
__global__ void pool_kernel(Geo g, const float* __restrict__ s_in, float* __restrict__ s_out, int kernel, int mode)
{
    const int p = blockIdx.y, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const int T = geo_L(g, seq) - g.window;
    const size_t off = (size_t)layer * g.total_tokens + g.cu[seq];
    const int half = kernel / 2;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < T; t += gridDim.x * blockDim.x) {
        int lo = max(t - half, 0), hi = min(t + half, T - 1);
        float acc = s_in[off + lo];
        for (int i = lo + 1; i <= hi; ++i) {
            float v = s_in[off + i];
            acc = mode == 0 ? fmaxf(acc, v) : acc + v;
        }
        s_out[off + t] = mode == 0 ? acc : acc / (float)(hi - lo + 1);
    }
}

// ---------------------------------------------------------------------------------------
// Stage 3: segment-guided refinement (Algorithm 1, Eqs. 5-8).  One warp per segment; lanes
// stride over the segment's tokens and combine with a butterfly, so the summation order is
// fixed and every lane ends with the same value.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum(int v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(256)
refine_kernel(Geo g, const float* __restrict__ s, const float* __restrict__ e,
              const int* __restrict__ seg_start, const int* __restrict__ n_seg, float alpha, float eta,
              float* __restrict__ s_ref, float* __restrict__ stats, int stats_stride)
{
    const int p = blockIdx.y, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const size_t off = (size_t)layer * g.total_tokens + g.cu[seq];
    const int* sst = seg_start + g.cu[seq] + seq;
    const int ns = n_seg[seq];
    const int lane = threadIdx.x & 31;
    const int wpb = blockDim.x >> 5;
    for (int k = blockIdx.x * wpb + (threadIdx.x >> 5); k < ns; k += gridDim.x * wpb) {
        const int a = sst[k], z = sst[k + 1];
        float si = 0.f, sd = 0.f;
        for (int t = a + lane; t < z; t += 32) {
            si += s[off + t];
            sd += e[off + t];
        }
        si = warp_sum(si);
        sd = warp_sum(sd);
        const float n = (float)(z - a);
        const float I = si / n;                    // Eq. 5
        const float Dk = sd / n;                   // Eq. 6
        const float om = I * (1.f + eta * Dk);     // Eq. 7
        const float fac = 1.f + alpha * om;        // Eq. 8
        for (int t = a + lane; t < z; t += 32) s_ref[off + t] = s[off + t] * fac;
        if (stats && lane == 0) {
            stats[k] = I;
            stats[stats_stride + k] = Dk;
            stats[2 * stats_stride + k] = om;
        }
    }
}

// ---------------------------------------------------------------------------------------
// Stage 4a: global Top-B (Eq. 9) by a most-significant-digit radix select on the
// order-preserving integer image of the fp32 scores.  One CTA per problem.  Result:
// the threshold key and a cut-off index; token t is in the Top-B set iff
// key(t) > thr, or key(t) == thr and t <= cut (ties go to the lower index).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned order_key(float f)
{
    unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kTopThreads = 1024;
constexpr int kTopMaxCtas = 8;         // CTAs that may share one problem

// Scratch of the multi-CTA select, per problem (zeroed before the launch).
struct TopScratch {
    int hist[4][256];                  // digit histograms of the four passes, summed over the CTAs
    int arrived[5];                    // CTAs that have added their share (passes 0-3, tie count)
    int eq_count[kTopMaxCtas];         // keys equal to the threshold in each CTA's slice
};

// Bounded wait until every CTA of the problem has contributed; false if it gave up.
__device__ __forceinline__ bool top_wait(const int* ctr, int target, int* status)
{
    const long long t0 = clock64();
    while (true) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
        if (v >= target) return true;
        if (clock64() - t0 > kWaitLimitCycles) {
            atomicOr(status, kStatTimeout);
            note_giveup(status, kGiveupTopB);
            return false;
        }
        __nanosleep(100);
    }
}

// grid = (ctas per problem, problems).  The CTAs of a problem each histogram a slice of the
// scores and combine through integer atomics (sums of integers: the result does not depend on the
// order), so all of them see the same digit counts and walk the same path.  The CTAs of a problem
// wait for one another: the launch must keep them co-resident (the host launches cooperatively
// when there is more than one per problem).
__global__ void __launch_bounds__(kTopThreads)
topb_kernel(Geo g, const float* __restrict__ s_ref, unsigned* __restrict__ sel_thr, int* __restrict__ sel_cut,
            TopScratch* __restrict__ scratch, int* status)
{
    const int p = blockIdx.y, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const int T = geo_L(g, seq) - g.window;
    const float* x = s_ref + (size_t)layer * g.total_tokens + g.cu[seq];
    const int tid = threadIdx.x, lane = tid & 31;
    const int n_cta = gridDim.x, cta = blockIdx.x;
    // this CTA's slice [a0, z0), a multiple of the block size long except for the last
    const int per = ((T + n_cta - 1) / n_cta + kTopThreads - 1) / kTopThreads * kTopThreads;
    const int a0 = min(cta * per, T), z0 = min(a0 + per, T);
    TopScratch* sc = scratch + p;
    __shared__ int hist[256];
    __shared__ unsigned s_prefix;
    __shared__ int s_k, s_neq, s_ok;
    __shared__ int s_scan[kTopThreads / 32];

    unsigned prefix = 0, mask = 0;
    int k = g.B;                                   // rank (1-based, descending) still to locate
    int n_eq = 0;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int i0 = a0; i0 < z0; i0 += kTopThreads) {
            const int i = i0 + tid;
            int bin = 256;
            if (i < z0) {
                unsigned u = order_key(x[i]);
                if ((u & mask) == prefix) bin = (u >> shift) & 255;
            }
            // one shared-memory atomic per distinct digit per warp
            if (__any_sync(0xffffffffu, bin < 256)) {
                unsigned peers = __match_any_sync(0xffffffffu, bin);
                if (bin < 256 && lane == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
            }
        }
        __syncthreads();
        if (n_cta > 1) {
            if (tid < 256 && hist[tid]) atomicAdd(&sc->hist[pass][tid], hist[tid]);
            __threadfence();
            __syncthreads();
            if (tid == 0) {
                if (!(SAB_HOOK(1) && cta == 0 && pass == 0)) atomicAdd(&sc->arrived[pass], 1);
                s_ok = top_wait(&sc->arrived[pass], n_cta, status) ? 1 : 0;
            }
            __syncthreads();
            if (!s_ok) return;
            if (tid < 256) hist[tid] = __ldcg(&sc->hist[pass][tid]);
            __syncthreads();
        }
        if (tid < 32) {
            // the digit that holds the k-th key: lane l looks at digits 255 - 8 l ... 248 - 8 l, highest first
            int c[8], mine = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[i] = hist[255 - (8 * lane + i)]; mine += c[i]; }
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            int above = incl - mine;
            const int total = __shfl_sync(0xffffffffu, incl, 31);
            // fewer than k keys left (only with non-finite scores that do not order): the lowest digit
            if (lane == 31 && total < k) { s_k = k - (total - c[7]); s_neq = c[7]; s_prefix = prefix; }
            if (above < k && k <= incl) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (above + c[i] >= k) {
                        s_k = k - above;
                        s_neq = c[i];
                        s_prefix = prefix | ((unsigned)(255 - (8 * lane + i)) << shift);
                        break;
                    }
                    above += c[i];
                }
            }
        }
        __syncthreads();
        k = s_k;
        n_eq = s_neq;
        prefix = s_prefix;
        mask |= 0xFFu << shift;
        __syncthreads();
    }
    // k of the n_eq tokens whose key equals the threshold are taken, lowest indices first.
    int cut = T;                                   // all of them
    if (k < n_eq) {
        const int len = z0 - a0;
        const int chunk = (len + kTopThreads - 1) / kTopThreads;
        const int a = a0 + tid * chunk, z = min(a + chunk, z0);
        int c = 0;
        for (int i = a; i < z; ++i) c += (order_key(x[i]) == prefix);
        int inc = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        if (lane == 31) s_scan[tid >> 5] = inc;
        __syncthreads();
        int woff = 0, total = 0;
        for (int w = 0; w < kTopThreads / 32; ++w) {
            if (w < (tid >> 5)) woff += s_scan[w];
            total += s_scan[w];
        }
        int before = 0;                            // equal keys in the slices of the CTAs before this one
        if (n_cta > 1) {
            if (tid == 0) {
                sc->eq_count[cta] = total;
                __threadfence();
                atomicAdd(&sc->arrived[4], 1);
                s_ok = top_wait(&sc->arrived[4], n_cta, status) ? 1 : 0;
            }
            __syncthreads();
            if (!s_ok) return;
            for (int i = 0; i < cta; ++i) before += __ldcg(&sc->eq_count[i]);
        }
        const int excl = before + woff + inc - c;
        if (excl < k && k <= excl + c) {           // the k-th equal key lies in this thread's chunk
            int seen = excl;
            for (int i = a; i < z; ++i)
                if (order_key(x[i]) == prefix && ++seen == k) { sel_cut[p] = i; break; }
        }
        if (cta == 0 && tid == 0) sel_thr[p] = prefix;
        return;
    }
    if (cta == 0 && tid == 0) {
        sel_thr[p] = prefix;
        sel_cut[p] = cut;
    }
}

// ---------------------------------------------------------------------------------------
// Stage 4b: implicit budgets (Eq. 10) and the per-segment block-size search of Algorithm 2.
// One warp per segment; the segment's refined scores and its block scores live in shared
// memory.  Block scores and the two fidelity sums are accumulated in double, in an order
// fixed by token position, so that the decisions (block order, Score_k(g) >= tau *
// Score_base) are reproducible and depend only on the fp32 scores.
// Segments longer than kSegShort tokens are queued for search_long_kernel.
// ---------------------------------------------------------------------------------------
constexpr int kSegShort = 512;
constexpr int kSearchWarps = 4;

struct SearchOut {
    unsigned* keep;        // [n_prob][keep_words] bitmask over t in [0, T)
    int keep_words;
    int* seg_g;            // optional [n_prob][seg_stride]
    int* seg_b;            // optional
    int seg_stride;
    int* long_list;        // [n_prob][long_cap]
    int* long_count;       // [n_prob]
    int long_cap;
};

__device__ __forceinline__ bool in_topb(float v, int t, unsigned thr, int cut)
{
    unsigned u = order_key(v);
    return u > thr || (u == thr && t <= cut);
}

// Greedy fill of Alg. 2 for block size g, evaluated in closed form from the block ranks:
// all blocks have g tokens except the last (rem tokens, rank rl).  Returns the first rank
// that does not fit (nb if every block fits) and the tokens still missing at that point.
__device__ __forceinline__ void greedy_cut(int nb, int g, int rem, int rl, int b, int& r_star, int& m_take)
{
    // tokens covered by ranks [0, r): g * r, minus (g - rem) once the short block is included
    // fits(r)  <=>  covered(r) + size(r) <= b; monotone in r
    int lo = 0, hi = nb;                       // first r in [0, nb) with !fits(r)
    while (lo < hi) {
        int r = (lo + hi) >> 1;
        int covered_incl = g * (r + 1) - ((rl <= r) ? (g - rem) : 0);
        if (covered_incl <= b) lo = r + 1; else hi = r;
    }
    r_star = lo;
    int covered = g * r_star - ((rl < r_star) ? (g - rem) : 0);
    m_take = (r_star < nb) ? b - covered : 0;
}

__global__ void __launch_bounds__(kSearchWarps * 32)
search_kernel(Geo g, Cands cands, const float* __restrict__ s_ref, const int* __restrict__ seg_start,
              const int* __restrict__ n_seg, const unsigned* __restrict__ sel_thr,
              const int* __restrict__ sel_cut, float tau, SearchOut out)
{
    const int p = blockIdx.y, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const float* x = s_ref + (size_t)layer * g.total_tokens + g.cu[seq];
    const int* sst = seg_start + g.cu[seq] + seq;
    const int ns = n_seg[seq];
    const unsigned thr = sel_thr[p];
    const int cut = sel_cut[p];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned* keep = out.keep + (size_t)p * out.keep_words;

    __shared__ float sv_all[kSearchWarps][kSegShort];
    __shared__ double phi_all[kSearchWarps][kSegShort / 2];
    __shared__ short rank_all[kSearchWarps][kSegShort / 2];
    float* sv = sv_all[warp];
    double* phi = phi_all[warp];
    short* rank = rank_all[warp];

    for (int k = blockIdx.x * kSearchWarps + warp; k < ns; k += gridDim.x * kSearchWarps) {
        const int a = sst[k], z = sst[k + 1], n = z - a;
        // implicit budget b_k and the token-level baseline Score_base
        int b = 0;
        double base = 0.0;
        for (int i = lane; i < n; i += 32) {
            float v = x[a + i];
            if (in_topb(v, a + i, thr, cut)) { ++b; base += (double)v; }
        }
        b = warp_sum(b);
        if (out.seg_b && lane == 0) out.seg_b[(size_t)p * out.seg_stride + k] = b;
        if (b == 0) {                               // most segments at small budgets: nothing to search
            if (out.seg_g && lane == 0) out.seg_g[(size_t)p * out.seg_stride + k] = 0;
            continue;
        }
        base = warp_sum(base);
        if (n > kSegShort) {
            if (lane == 0) {
                int slot = atomicAdd(&out.long_count[p], 1);
                if (slot < out.long_cap) out.long_list[(size_t)p * out.long_cap + slot] = k;
            }
            continue;
        }
        for (int i = lane; i < n; i += 32) sv[i] = x[a + i];
        __syncwarp();
        const int lim = min(n, b);
        int g_acc = 1;
        unsigned taken_bits = 0;                   // bit i: token lane + 32 i is retained
        for (int ci = cands.n - 1; ci >= 0; --ci) {
            const int gs = cands.g[ci];
            if (gs > lim) continue;
            if (gs == 1) {                         // T_k(1) = T_topB within the segment; R_k(1) = 1
                taken_bits = 0;
                for (int i = lane, q = 0; i < n; i += 32, ++q)
                    if (in_topb(sv[i], a + i, thr, cut)) taken_bits |= 1u << q;
                g_acc = 1;
                break;
            }
            const int nb = (n + gs - 1) / gs;
            const int rem = n - (nb - 1) * gs;
            for (int m = lane; m < nb; m += 32) {  // block scores Phi, tokens in index order
                int t0 = m * gs, t1 = min(t0 + gs, n);
                double acc = 0.0;
                for (int t = t0; t < t1; ++t) acc += (double)sv[t];
                phi[m] = acc;
            }
            __syncwarp();
            for (int m = lane; m < nb; m += 32) {  // rank by (Phi desc, index asc)
                double pm = phi[m];
                int r = 0;
                for (int m2 = 0; m2 < nb; ++m2) {
                    double q = phi[m2];
                    r += (q > pm) || (q == pm && m2 < m);
                }
                rank[m] = (short)r;
            }
            __syncwarp();
            int r_star, m_take;
            greedy_cut(nb, gs, rem, rank[nb - 1], b, r_star, m_take);
            int mp = -1;                           // the block that is truncated
            if (m_take > 0)
                for (int m = 0; m < nb; ++m) if (rank[m] == r_star) { mp = m; break; }
            double score = 0.0;
            unsigned bits = 0;
            for (int i = lane, q = 0; i < n; i += 32, ++q) {
                int m = i / gs;
                int rk = rank[m];
                bool take = rk < r_star;
                if (m == mp) {                     // top m_take tokens of the block, (score desc, index asc)
                    int t0 = mp * gs, t1 = min(t0 + gs, n);
                    float vi = sv[i];
                    int tr = 0;
                    for (int t = t0; t < t1; ++t) tr += (sv[t] > vi) || (sv[t] == vi && t < i);
                    take = tr < m_take;
                }
                if (take) { bits |= 1u << q; score += (double)sv[i]; }
            }
            score = warp_sum(score);
            __syncwarp();
            if (score >= (double)tau * base) {     // R_k(g) >= tau (Eqs. 11, 12)
                taken_bits = bits;
                g_acc = gs;
                break;
            }
        }
        for (int i = lane, q = 0; i < n; i += 32, ++q)
            if (taken_bits & (1u << q)) atomicOr(&keep[(a + i) >> 5], 1u << ((a + i) & 31));
        if (out.seg_g && lane == 0) out.seg_g[(size_t)p * out.seg_stride + k] = g_acc;
        __syncwarp();
    }
}

// Same search for one long segment per CTA.  A prompt with few delimiters can be one segment of
// the whole compressible region, so nothing here is quadratic in the segment: Algorithm 2's greedy
// fill takes blocks in descending (Phi, then lower index) order and stops at the first one that
// does not fit, and since all blocks but the last have g tokens, where it stops (r*) follows from
// the rank of the short last block alone.  The retained blocks are then the r* best ones, found
// by a radix select of the (r* + 1)-th block on the order-preserving integer image of the double
// block scores (ties to the lower index), which also names the block that is truncated.  Block
// scores live in global scratch indexed by absolute token position (disjoint between segments).
constexpr int kLongThreads = 1024;

__device__ __forceinline__ unsigned long long order_key64(double f)
{
    unsigned long long u = (unsigned long long)__double_as_longlong(f);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

struct LongShared {
    double red[kLongThreads / 32];
    int hist[256];
    int scan[kLongThreads / 32];
    int b, k, digit, mp;
};

__device__ __forceinline__ double block_sum_double(double v, LongShared& sm)
{
    const int tid = threadIdx.x;
    v = warp_sum(v);
    if ((tid & 31) == 0) sm.red[tid >> 5] = v;
    __syncthreads();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < kLongThreads / 32; ++w) tot += sm.red[w];
    __syncthreads();
    return tot;
}

__device__ __forceinline__ int block_sum_int(int v, LongShared& sm)
{
    const int tid = threadIdx.x;
    v = warp_sum(v);
    if ((tid & 31) == 0) sm.scan[tid >> 5] = v;
    __syncthreads();
    int tot = 0;
#pragma unroll
    for (int w = 0; w < kLongThreads / 32; ++w) tot += sm.scan[w];
    __syncthreads();
    return tot;
}

// The k-th (1-based) of phi[0..nb) in descending order, ties to the lower index: its key and its
// index.  Block m then ranks before it iff key(m) > thr, or key(m) == thr and m < mp.  Called by
// every thread of the CTA.
__device__ __forceinline__ void long_select(const double* __restrict__ phi, int nb, int k, LongShared& sm,
                                            unsigned long long& thr, int& mp)
{
    const int tid = threadIdx.x, lane = tid & 31;
    unsigned long long prefix = 0, mask = 0;
    for (int pass = 0; pass < 8; ++pass) {
        const int shift = 56 - 8 * pass;
        if (tid < 256) sm.hist[tid] = 0;
        __syncthreads();
        for (int m0 = 0; m0 < nb; m0 += kLongThreads) {
            const int m = m0 + tid;
            int bin = 256;
            if (m < nb) {
                const unsigned long long u = order_key64(phi[m]);
                if ((u & mask) == prefix) bin = (int)((u >> shift) & 255);
            }
            if (__any_sync(0xffffffffu, bin < 256)) {          // one shared-memory atomic per distinct digit per warp
                const unsigned peers = __match_any_sync(0xffffffffu, bin);
                if (bin < 256 && lane == __ffs(peers) - 1) atomicAdd(&sm.hist[bin], __popc(peers));
            }
        }
        __syncthreads();
        if (tid < 32) {
            // lane l looks at digits 255 - 8 l ... 248 - 8 l, highest first
            int c[8], mine = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[i] = sm.hist[255 - (8 * lane + i)]; mine += c[i]; }
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            int above = incl - mine;
            if (above < k && k <= incl) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (above + c[i] >= k) { sm.digit = 255 - (8 * lane + i); sm.k = k - above; break; }
                    above += c[i];
                }
            }
        }
        __syncthreads();
        k = sm.k;
        prefix |= (unsigned long long)sm.digit << shift;
        mask |= 0xFFull << shift;
    }
    // the k-th block, in index order, among those whose key equals the threshold
    const int chunk = (nb + kLongThreads - 1) / kLongThreads;
    const int a = min(tid * chunk, nb), z = min(a + chunk, nb);
    int c = 0;
    for (int m = a; m < z; ++m) c += (order_key64(phi[m]) == prefix);
    int inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) sm.scan[tid >> 5] = inc;
    __syncthreads();
    int woff = 0;
    for (int w = 0; w < (tid >> 5); ++w) woff += sm.scan[w];
    const int excl = woff + inc - c;
    if (excl < k && k <= excl + c) {
        int seen = excl;
        for (int m = a; m < z; ++m)
            if (order_key64(phi[m]) == prefix && ++seen == k) { sm.mp = m; break; }
    }
    __syncthreads();
    thr = prefix;
    mp = sm.mp;
    __syncthreads();
}

__global__ void __launch_bounds__(kLongThreads)
search_long_kernel(Geo g, Cands cands, const float* __restrict__ s_ref, const int* __restrict__ seg_start,
                   const unsigned* __restrict__ sel_thr, const int* __restrict__ sel_cut, float tau,
                   SearchOut out, double* __restrict__ phi_ws)
{
    const int p = blockIdx.y, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const int count = min(out.long_count[p], out.long_cap);
    const size_t off = (size_t)layer * g.total_tokens + g.cu[seq];
    const float* x = s_ref + off;
    const int* sst = seg_start + g.cu[seq] + seq;
    const unsigned thr_top = sel_thr[p];
    const int cut = sel_cut[p];
    unsigned* keep = out.keep + (size_t)p * out.keep_words;
    const int tid = threadIdx.x;
    __shared__ LongShared sm;

    for (int li = blockIdx.x; li < count; li += gridDim.x) {
        const int k = out.long_list[(size_t)p * out.long_cap + li];
        const int a = sst[k], z = sst[k + 1], n = z - a;
        const float* sv = x + a;
        double* phi = phi_ws + off + a;
        int bl = 0;
        double base = 0.0;
        for (int i = tid; i < n; i += kLongThreads) {
            const float v = sv[i];
            if (in_topb(v, a + i, thr_top, cut)) { ++bl; base += (double)v; }
        }
        const int b = block_sum_int(bl, sm);
        base = block_sum_double(base, sm);
        const int lim = min(n, b);
        int g_acc = 1;
        for (int ci = cands.n - 1; ci >= 0; --ci) {
            const int gs = cands.g[ci];
            if (gs > lim) continue;
            if (gs == 1) {                         // T_k(1) = T_topB within the segment; R_k(1) = 1
                for (int i = tid; i < n; i += kLongThreads)
                    if (in_topb(sv[i], a + i, thr_top, cut)) atomicOr(&keep[(a + i) >> 5], 1u << ((a + i) & 31));
                g_acc = 1;
                break;
            }
            const int nb = (n + gs - 1) / gs;
            const int rem = n - (nb - 1) * gs;
            for (int m = tid; m < nb; m += kLongThreads) {     // block scores Phi, tokens in index order
                const int t0 = m * gs, t1 = min(t0 + gs, n);
                double acc = 0.0;
                for (int t = t0; t < t1; ++t) acc += (double)sv[t];
                phi[m] = acc;
            }
            __syncthreads();
            int rl = nb - 1;                                   // rank of the short last block (only matters if it is short)
            if (rem != gs) {
                const double pl = phi[nb - 1];
                int c = 0;
                for (int m = tid; m < nb - 1; m += kLongThreads) c += phi[m] >= pl;    // earlier index wins a tie
                rl = block_sum_int(c, sm);
            }
            int r_star, m_take;
            greedy_cut(nb, gs, rem, rl, b, r_star, m_take);
            unsigned long long thr = 0;
            int mp = -1;                                       // the block that is truncated
            if (r_star < nb) long_select(phi, nb, r_star + 1, sm, thr, mp);
            const bool all = r_star >= nb;
            // Retained tokens: the blocks ranked before r*, and the top m_take tokens of block mp
            // by (score desc, index asc).
            auto retained = [&](int i) -> bool {
                const int m = i / gs;
                if (all) return true;
                if (m == mp) {
                    if (m_take <= 0) return false;
                    const int t0 = mp * gs, t1 = min(t0 + gs, n);
                    const float vi = sv[i];
                    int tr = 0;
                    for (int t = t0; t < t1; ++t) tr += (sv[t] > vi) || (sv[t] == vi && t < i);
                    return tr < m_take;
                }
                const unsigned long long u = order_key64(phi[m]);
                return u > thr || (u == thr && m < mp);
            };
            double score = 0.0;
            for (int i = tid; i < n; i += kLongThreads)
                if (retained(i)) score += (double)sv[i];
            score = block_sum_double(score, sm);
            if (score >= (double)tau * base) {                 // R_k(g) >= tau (Eqs. 11, 12)
                for (int i = tid; i < n; i += kLongThreads)
                    if (retained(i)) atomicOr(&keep[(a + i) >> 5], 1u << ((a + i) & 31));
                g_acc = gs;
                break;
            }
            __syncthreads();
        }
        if (out.seg_g && tid == 0) out.seg_g[(size_t)p * out.seg_stride + k] = g_acc;
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------
// Stage 5a: T* as an ascending index list (Eq. 13) followed by the W window positions.
// One CTA per problem: ordered prefix sum over the popcounts of the bitmask words.
// ---------------------------------------------------------------------------------------
constexpr int kIdxThreads = 1024;

__global__ void __launch_bounds__(kIdxThreads)
index_kernel(Geo g, const unsigned* __restrict__ keep_all, int keep_words, int* __restrict__ out_idx,
             int* __restrict__ out_n_keep, int* status)
{
    const int p = blockIdx.x, seq = p % g.n_seqs;
    const int L = geo_L(g, seq), T = L - g.window;
    int* oi = out_idx + (size_t)p * g.n_out;
    const int tid = threadIdx.x, lane = tid & 31;
    if (geo_identity(g, seq)) {
        for (int i = tid; i < L; i += kIdxThreads) oi[i] = i;
        if (tid == 0) out_n_keep[p] = L;
        return;
    }
    const unsigned* keep = keep_all + (size_t)p * keep_words;
    const int words = (T + 31) >> 5;
    const int wpt = (words + kIdxThreads - 1) / kIdxThreads;
    const int w0 = tid * wpt, w1 = min(w0 + wpt, words);
    int c = 0;
    for (int w = w0; w < w1; ++w) c += __popc(keep[w]);
    __shared__ int s_scan[kIdxThreads / 32];
    int inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) s_scan[tid >> 5] = inc;
    __syncthreads();
    int woff = 0, total = 0;
    for (int w = 0; w < kIdxThreads / 32; ++w) {
        int v = s_scan[w];
        if (w < (tid >> 5)) woff += v;
        total += v;
    }
    int pos = woff + inc - c;
    for (int w = w0; w < w1; ++w) {
        unsigned bits = keep[w];
        while (bits) {
            int bit = __ffs(bits) - 1;
            bits &= bits - 1;
            if (pos < g.B) oi[pos] = (w << 5) + bit;
            ++pos;
        }
    }
    for (int i = tid; i < g.window; i += kIdxThreads) oi[g.B + i] = T + i;
    // |T*| = B (Eq. 13) whenever the scores are finite.  If the search retained fewer (scores
    // that do not order, e.g. NaN), the rest of the list still gets valid positions, so that the
    // gather that follows stays inside the cache, and the status word reports it.
    for (int i = total + tid; i < g.B; i += kIdxThreads) oi[i] = 0;
    if (tid == 0) {
        out_n_keep[p] = g.B + g.window;
        if (total != g.B) atomicOr(status, kStatInternal);
    }
}

// ---------------------------------------------------------------------------------------
// Stage 5b: compaction.  Row i of the output is row out_idx[i] of the input; rows are moved
// as 16-byte vectors, one per thread, consecutive threads on consecutive vectors.
// ---------------------------------------------------------------------------------------
struct CompactArgs {
    const char* k; const char* v;
    char* out_k; char* out_v;
    long long k_tok, k_head, k_layer;     // byte strides
    long long v_tok, v_head, v_layer;
    int head_bytes;                        // D * element size (multiple of 16)
    int rows_per_cta;
};

__global__ void __launch_bounds__(256)
compact_kernel(Geo g, CompactArgs c, const int* __restrict__ out_idx, const int* __restrict__ out_n_keep,
               int n_keep_fixed)
{
    const int p = blockIdx.y, layer = p / g.n_seqs, seq = p % g.n_seqs;
    const bool is_v = blockIdx.z != 0;
    const int n_keep = out_n_keep ? out_n_keep[p] : n_keep_fixed;
    const char* src = (is_v ? c.v : c.k) + (size_t)layer * (is_v ? c.v_layer : c.k_layer);
    char* dst = is_v ? c.out_v : c.out_k;
    const long long s_tok = is_v ? c.v_tok : c.k_tok, s_head = is_v ? c.v_head : c.k_head;
    const int vec_per_head = c.head_bytes >> 4;
    const int vec_per_row = vec_per_head * g.Hkv;
    const int row0 = blockIdx.x * c.rows_per_cta;
    const int* oi = out_idx + (size_t)p * g.n_out;
    const size_t out_row_bytes = (size_t)g.Hkv * c.head_bytes;
    for (int i = threadIdx.x; i < c.rows_per_cta * vec_per_row; i += blockDim.x) {
        const int r = row0 + i / vec_per_row;
        if (r >= n_keep) break;
        const int vi = i % vec_per_row;
        const int h = vi / vec_per_head, x = vi % vec_per_head;
        const int pos = oi[r];
        if ((unsigned)pos >= (unsigned)geo_L(g, seq)) continue;     // not a position of this sequence: row left as is
        const long long tok = (long long)g.cu[seq] + pos;
        const uint4 val = __ldg(reinterpret_cast<const uint4*>(src + tok * s_tok + (long long)h * s_head) + x);
        reinterpret_cast<uint4*>(dst + ((size_t)p * g.n_out + r) * out_row_bytes)[vi] = val;
    }
}

}  // namespace sab
