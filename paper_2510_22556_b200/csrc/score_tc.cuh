// Stage 2 on the sm_100a tensor cores (bf16 inputs, head_dim 64 or 128, window 8/16/32,
// (H / Hkv) * W <= 128).  The window-Q x K^T logits are tcgen05.mma tiles of 128 x 128 with
// fp32 accumulators in tensor memory; K tiles and the query block arrive by TMA into
// 128-byte-swizzled shared memory; softmax statistics, normalisation, the head / window
// reductions and the per-token entropy are done by the epilogue warps straight from tensor
// memory, so the H x W x T attention matrix never exists in HBM (Eqs. 2-4, 6).
//
// CTA = 6 warps: warp 0 issues TMA loads, warp 1 owns tensor memory and issues the MMAs,
// warps 2-5 are the epilogue (each reads its own 32-lane quarter of tensor memory).
//
// Pass 1 (row statistics): D[row = query (h_local, w)][col = token] = Q_g . K_tile^T; every
// epilogue thread owns one query row and keeps its running (max, sum) in registers.
// Pass 2 (scores): D[row = token][col = query (h_local, w)] = K_tile . Q_g^T; every epilogue
// thread owns one token and keeps the W head-summed weights in registers across all KV
// heads, then emits s_t and the entropy.  No cross-thread reduction, no atomics.
#pragma once
#include "common.cuh"
#include "score_simt.cuh"

namespace sab {

constexpr int kTcThreads = 192;
constexpr int kTcTile = 128;                 // tokens per tile = MMA M or N
constexpr int kAtomBytes = 128 * 128;        // 128 rows x 64 bf16 (one 128-byte-swizzle atom column)
constexpr int kTmemCols = 256;               // two 128-column fp32 accumulators
constexpr int kTcMaxStages = 4;

struct TcBarriers {
    uint64_t full[kTcMaxStages];
    uint64_t empty[kTcMaxStages];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint64_t qfull;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ void tc_setup(TcBarriers& sh, int nst, int warp, int lane)
{
    if (warp == 0 && lane == 0) {
        for (int i = 0; i < nst; ++i) {
            mbar_init(smem_u32(&sh.full[i]), 1);
            mbar_init(smem_u32(&sh.empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh.tfull[i]), 1);
            mbar_init(smem_u32(&sh.tempty[i]), 128);
        }
        mbar_init(smem_u32(&sh.qfull), 1);
        sh.abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        __syncwarp();
        tmem_alloc(smem_u32(&sh.tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
}

__device__ __forceinline__ void tc_teardown(TcBarriers& sh, uint32_t tmem, int warp, int* status)
{
    tc_fence_before();
    __syncthreads();
    if (sh.abort_flag) {
        // A bounded wait ran out: report it, give copies and MMAs in flight time to land,
        // then release tensor memory as usual.
        if (threadIdx.x == 0) atomicOr(status, kStatTimeout);
        long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// One 128 x 128 x D product into accumulator `acc` of tensor memory.
__device__ __forceinline__ void tc_issue_tile(uint32_t tmem, int acc, uint32_t a_base, uint32_t b_base, int ksteps)
{
    constexpr uint32_t idesc = umma_idesc_bf16(128, 128);
    for (int kk = 0; kk < ksteps; ++kk) {
        const uint32_t off = (uint32_t)(kk >> 2) * kAtomBytes + (uint32_t)(kk & 3) * 32u;
        tc_mma_bf16(tmem + (uint32_t)acc * 128u, umma_desc_sw128(a_base + off), umma_desc_sw128(b_base + off),
                    idesc, kk > 0 ? 1u : 0u);
    }
}

// ---------------------------------------------------------------------------------------
// Pass 1.  grid = (chunks, Hkv, problems); a CTA covers `tiles_per_cta` consecutive key
// tiles of one KV head and writes the (max, sum) of each of its 128 query rows.
// ---------------------------------------------------------------------------------------
template <int NST>
__global__ void __launch_bounds__(kTcThreads)
score_p1_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, Geo g, float c2,
            ScoreBufs sb, int tiles_per_cta, int* status)
{
    const int p = blockIdx.z, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const int L = geo_L(g, seq), Tn = L - g.window;
    const int ntiles = (L + kTcTile - 1) / kTcTile;
    const int chunk = blockIdx.x, j = blockIdx.y;
    const int tile0 = chunk * tiles_per_cta;
    if (tile0 >= ntiles) return;
    const int ntl = min(tiles_per_cta, ntiles - tile0);
    const int n_atoms = g.D >> 6, ksteps = g.D >> 4;
    const int R = g.G * g.window;

    extern __shared__ uint8_t dyn_smem[];
    __shared__ TcBarriers sh;
    const uint32_t base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    const uint32_t q_smem = base;
    const uint32_t k_smem = base + (uint32_t)n_atoms * kAtomBytes;
    const uint32_t stage_bytes = (uint32_t)n_atoms * kAtomBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    tc_setup(sh, NST, warp, lane);
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            const uint64_t pol = l2_policy_normal();
            mbar_expect_tx(smem_u32(&sh.qfull), stage_bytes);
            for (int a = 0; a < n_atoms; ++a)
                tma_load_2d(q_smem + a * kAtomBytes, &tmQ, smem_u32(&sh.qfull), a * 64, p * g.H * g.window + j * R, pol);
            for (int it = 0; it < ntl; ++it) {
                const int st = it % NST, ph = (it / NST) & 1;
                if (!mbar_wait(smem_u32(&sh.empty[st]), ph ^ 1, abort_flag)) break;
                mbar_expect_tx(smem_u32(&sh.full[st]), stage_bytes);
                for (int a = 0; a < n_atoms; ++a)
                    tma_load_4d(k_smem + st * stage_bytes + a * kAtomBytes, &tmK, smem_u32(&sh.full[st]), a * 64, j,
                                g.cu[seq] + (tile0 + it) * kTcTile, layer, pol);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = mbar_wait(smem_u32(&sh.qfull), 0, abort_flag);
            for (int it = 0; ok && it < ntl; ++it) {
                const int st = it % NST, ph = (it / NST) & 1;
                const int acc = it & 1, aph = (it >> 1) & 1;
                if (!mbar_wait(smem_u32(&sh.tempty[acc]), aph ^ 1, abort_flag)) break;
                if (!mbar_wait(smem_u32(&sh.full[st]), ph, abort_flag)) break;
                tc_fence_after();
                tc_issue_tile(tmem, acc, q_smem, k_smem + st * stage_bytes, ksteps);
                tc_commit(smem_u32(&sh.empty[st]));
                tc_commit(smem_u32(&sh.tfull[acc]));
            }
        }
    } else {
        const int q4 = warp & 3;
        const int row = q4 * 32 + lane;
        const int lim = Tn + (row % g.window);          // causal: key index <= T + w (Eq. 2)
        float m2 = -INFINITY, l = 0.f;
        for (int it = 0; it < ntl; ++it) {
            const int acc = it & 1, aph = (it >> 1) & 1;
            if (!mbar_wait(smem_u32(&sh.tfull[acc]), aph, abort_flag)) break;
            tc_fence_after();
            const int tok0 = (tile0 + it) * kTcTile;
            const bool need_mask = tok0 + kTcTile - 1 > Tn;
            const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)acc * 128u;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                float v[32];
                tmem_ld32(taddr + c * 32, v);
                if (need_mask) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (tok0 + c * 32 + i > lim) v[i] = -INFINITY;
                }
                float cm0 = fmaxf(v[0], v[1]), cm1 = fmaxf(v[2], v[3]);
#pragma unroll
                for (int i = 4; i < 32; i += 2) {
                    cm0 = fmaxf(cm0, v[i]);
                    cm1 = fmaxf(cm1, v[i + 1]);
                }
                const float m_new = fmaxf(m2, fmaxf(cm0, cm1) * c2);
                const float ms = (m_new == -INFINITY) ? 0.f : m_new;
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    s0 += ex2_approx(fmaf(v[i], c2, -ms));
                    s1 += ex2_approx(fmaf(v[i + 1], c2, -ms));
                    s2 += ex2_approx(fmaf(v[i + 2], c2, -ms));
                    s3 += ex2_approx(fmaf(v[i + 3], c2, -ms));
                }
                l = l * ex2_approx(m2 - ms) + ((s0 + s1) + (s2 + s3));
                m2 = m_new;
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&sh.tempty[acc]));
        }
        sb.part[(((size_t)p * g.Hkv + j) * sb.n_chunks + chunk) * 128 + row] = make_float2(m2, l);
    }
    tc_teardown(sh, tmem, warp, status);
}

// Merge of the per-chunk row statistics into lse2[p][h*W + w] (log2 units), in chunk order.
__global__ void lse_merge_tc(Geo g, ScoreBufs sb, int tiles_per_cta)
{
    const int p = blockIdx.y, seq = p % g.n_seqs, j = blockIdx.x;
    if (geo_identity(g, seq)) return;
    const int R = g.G * g.window;
    const int row = threadIdx.x;
    if (row >= R) return;
    const int ntiles = (geo_L(g, seq) + kTcTile - 1) / kTcTile;
    const int nch = (ntiles + tiles_per_cta - 1) / tiles_per_cta;
    const float2* pr = sb.part + (((size_t)p * g.Hkv + j) * sb.n_chunks) * 128 + row;
    float m = -INFINITY;
    for (int c = 0; c < nch; ++c) m = fmaxf(m, pr[(size_t)c * 128].x);
    float l = 0.f;
    for (int c = 0; c < nch; ++c) {
        const float2 v = pr[(size_t)c * 128];
        l += v.y * exp2f(v.x - m);
    }
    sb.lse2[(size_t)p * g.H * g.window + j * R + row] = m + log2f(l);
}

// ---------------------------------------------------------------------------------------
// Pass 2.  grid = (token chunks, problems); a CTA covers `tiles_per_cta` consecutive token
// tiles and, for each, walks all KV heads (one pipeline stage = K tile + that head's
// query block).
// ---------------------------------------------------------------------------------------
template <int W, int NST>
__global__ void __launch_bounds__(kTcThreads)
score_p2_tc(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, Geo g, float c2,
            float eps, ScoreBufs sb, int tiles_per_cta, float* __restrict__ s_out, float* __restrict__ e_out,
            int* status)
{
    const int p = blockIdx.y, layer = p / g.n_seqs, seq = p % g.n_seqs;
    if (geo_identity(g, seq)) return;
    const int L = geo_L(g, seq), Tn = L - W;
    const int ntiles = (Tn + kTcTile - 1) / kTcTile;
    const int tile0 = blockIdx.x * tiles_per_cta;
    if (tile0 >= ntiles) return;
    const int ntl = min(tiles_per_cta, ntiles - tile0);
    const int n_atoms = g.D >> 6, ksteps = g.D >> 4;
    const int R = g.G * W, Hkv = g.Hkv;
    const int n_it = ntl * Hkv;

    extern __shared__ uint8_t dyn_smem[];
    __shared__ TcBarriers sh;
    __shared__ __align__(16) float lse_s[2048];
    const uint32_t base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    const uint32_t op_bytes = (uint32_t)n_atoms * kAtomBytes;
    const uint32_t stage_bytes = 2 * op_bytes;           // K tile then Q block

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < g.H * W; i += kTcThreads) lse_s[i] = sb.lse2[(size_t)p * g.H * W + i];
    tc_setup(sh, NST, warp, lane);
    const uint32_t tmem = sh.tmem_base;
    volatile int* abort_flag = &sh.abort_flag;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            const uint64_t pol_k = l2_policy_normal();
            const uint64_t pol_q = l2_policy_evict_last();
            for (int it = 0; it < n_it; ++it) {
                const int st = it % NST, ph = (it / NST) & 1;
                const int tile = tile0 + it / Hkv, j = it % Hkv;
                if (!mbar_wait(smem_u32(&sh.empty[st]), ph ^ 1, abort_flag)) break;
                mbar_expect_tx(smem_u32(&sh.full[st]), stage_bytes);
                const uint32_t dst = base + st * stage_bytes;
                for (int a = 0; a < n_atoms; ++a)
                    tma_load_4d(dst + a * kAtomBytes, &tmK, smem_u32(&sh.full[st]), a * 64, j,
                                g.cu[seq] + tile * kTcTile, layer, pol_k);
                for (int a = 0; a < n_atoms; ++a)
                    tma_load_2d(dst + op_bytes + a * kAtomBytes, &tmQ, smem_u32(&sh.full[st]), a * 64,
                                p * g.H * W + j * R, pol_q);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            for (int it = 0; it < n_it; ++it) {
                const int st = it % NST, ph = (it / NST) & 1;
                const int acc = it & 1, aph = (it >> 1) & 1;
                if (!mbar_wait(smem_u32(&sh.tempty[acc]), aph ^ 1, abort_flag)) break;
                if (!mbar_wait(smem_u32(&sh.full[st]), ph, abort_flag)) break;
                tc_fence_after();
                const uint32_t src = base + st * stage_bytes;
                tc_issue_tile(tmem, acc, src, src + op_bytes, ksteps);
                tc_commit(smem_u32(&sh.empty[st]));
                tc_commit(smem_u32(&sh.tfull[acc]));
            }
        }
    } else {
        const int q4 = warp & 3;
        const int row = q4 * 32 + lane;
        const size_t off = (size_t)layer * g.total_tokens + g.cu[seq];
        const float inv_H = 1.f / (float)g.H;
        float accw[W];
        bool ok = true;
        for (int tl = 0; ok && tl < ntl; ++tl) {
#pragma unroll
            for (int w = 0; w < W; ++w) accw[w] = 0.f;
            for (int j = 0; j < Hkv; ++j) {
                const int it = tl * Hkv + j;
                const int acc = it & 1, aph = (it >> 1) & 1;
                if (!mbar_wait(smem_u32(&sh.tfull[acc]), aph, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem + ((uint32_t)(q4 * 32) << 16) + (uint32_t)acc * 128u;
                const float* lj = lse_s + j * R;
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    if (c * 32 >= R) break;
                    float v[32];
                    tmem_ld32(taddr + c * 32, v);
                    const float4* l4 = reinterpret_cast<const float4*>(lj + c * 32);
                    if (c * 32 + 32 <= R) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            const float4 ls = l4[i >> 2];
                            accw[(i + 0) % W] += ex2_approx(fmaf(v[i + 0], c2, -ls.x));
                            accw[(i + 1) % W] += ex2_approx(fmaf(v[i + 1], c2, -ls.y));
                            accw[(i + 2) % W] += ex2_approx(fmaf(v[i + 2], c2, -ls.z));
                            accw[(i + 3) % W] += ex2_approx(fmaf(v[i + 3], c2, -ls.w));
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (c * 32 + i < R) accw[i % W] += ex2_approx(fmaf(v[i], c2, -lj[c * 32 + i]));
                    }
                }
                tc_fence_before();
                mbar_arrive(smem_u32(&sh.tempty[acc]));
            }
            if (!ok) break;
            const int t = (tile0 + tl) * kTcTile + row;
            if (t < Tn) {
                float tot = 0.f;
#pragma unroll
                for (int w = 0; w < W; ++w) tot += accw[w];
                float ent = 0.f;
                if (tot > 0.f) {
                    const float inv = 1.f / tot;
#pragma unroll
                    for (int w = 0; w < W; ++w) {
                        const float ah = accw[w] * inv;                       // \hat A (Eq. 6)
                        ent -= ah * (lg2_approx(ah + eps) * 0.6931471805599453f);
                    }
                }
                s_out[off + t] = tot * inv_H;                                // Eqs. 3, 4
                e_out[off + t] = ent;
            }
        }
    }
    tc_teardown(sh, tmem, warp, status);
}

}  // namespace sab
