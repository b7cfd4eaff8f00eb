/*
 * SABlock prefill-time KV-cache compression: plain float64 CPU checker.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the compression pass computes, written from the paper's definitions
 * (Sec. 3.1-3.3, Eqs. 2-13, Algorithms 1 and 2).  Only the tests, the smoke check
 * and the benchmark's CPU-baseline leg may call it; the CUDA library shares no code
 * with it and never calls it.
 *
 * Inputs are the stored values (fp32, or bf16 widened exactly to fp32); every
 * arithmetic step is done in double.  Loops follow the paper's order and notation;
 * there is no blocking, fusion or reordering.  OpenMP, if enabled, only splits the
 * outermost independent loop (over window positions), which does not change any
 * summation order.
 *
 * Readings of points the paper leaves open (each also listed in the design notes):
 *  - a delimiter token is the last token of its segment (Sec. 3.1);
 *  - the attention weights are the model's causal softmax over all keys j <= T+w
 *    (Eq. 2), of which only columns t < T are scored (Sec. 3.2);
 *  - H in Eq. 3 counts query heads; each uses the KV head of its group (GQA);
 *  - log in Eq. 6 is the natural log; a token with s_t = 0 has zero entropy;
 *  - blocks are aligned to the segment start, the last block may be short (Alg. 2);
 *  - every ordering breaks ties by the lower index;
 *  - the greedy fill stops at the first block that does not fit (Alg. 2's break);
 *  - R_k(g) >= tau is evaluated as Score_k(g) >= tau * Score_base (no division);
 *    g = 1 is always accepted (R_k(1) = 1).
 *
 * Parity unpinned: absolute score values on random inputs (the paper prints no
 * worked numeric example); everything else is pinned by the CPU tests.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int sabo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void sabo_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ------------------------------------------------------------------ Sec. 3.1 */
/* Compressible region = first T = L - W tokens.  seg_id[t] = number of delimiters in
 * [0, t).  seg_start has n_seg + 1 entries, seg_start[n_seg] = T.  Returns n_seg. */
int sabo_segment(const int32_t *token_ids, int L, int W, const uint32_t *bitmap, int vocab,
                 int32_t *seg_id, int32_t *seg_start)
{
    int T = L - W;
    if (T <= 0) return 0;
    int cur = 0;
    seg_start[0] = 0;
    for (int t = 0; t < T; ++t) {
        seg_id[t] = cur;
        int id = token_ids[t];
        int is_delim = 0;
        if (id >= 0 && id < vocab) is_delim = (bitmap[id >> 5] >> (id & 31)) & 1u;
        if (is_delim && t + 1 < T) {
            ++cur;
            seg_start[cur] = t + 1;
        }
    }
    seg_start[cur + 1] = T;
    return cur + 1;
}

/* ------------------------------------------------------------------ Eq. 2 */
/* Logits of window query (h, w) against keys 0..n_keys-1 of its KV head. */
static void row_logits(const float *q, const float *k, int h, int w, int n_keys, int H, int Hkv,
                       int D, int W, long long ks_tok, long long ks_head, double *logit)
{
    (void)H;
    int G = H / Hkv;
    int j = h / G;
    const float *qr = q + ((size_t)h * W + w) * D;
    double inv = 1.0 / sqrt((double)D);
    for (int i = 0; i < n_keys; ++i) {
        const float *kr = k + (size_t)i * ks_tok + (size_t)j * ks_head;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += (double)qr[d] * (double)kr[d];
        logit[i] = acc * inv;
    }
}

/* Full attention tensor A[h][w][t], t < T (small inputs only; used by the pins). */
void sabo_attention(const float *q, const float *k, int L, int H, int Hkv, int D, int W,
                    long long ks_tok, long long ks_head, double *A)
{
    int T = L - W;
    double *logit = (double *)malloc(sizeof(double) * (size_t)L);
    for (int h = 0; h < H; ++h)
        for (int w = 0; w < W; ++w) {
            int n_keys = T + w + 1; /* causal: query at position T+w sees keys 0..T+w */
            row_logits(q, k, h, w, n_keys, H, Hkv, D, W, ks_tok, ks_head, logit);
            double mx = logit[0];
            for (int i = 1; i < n_keys; ++i) if (logit[i] > mx) mx = logit[i];
            double sum = 0.0;
            for (int i = 0; i < n_keys; ++i) sum += exp(logit[i] - mx);
            double *row = A + ((size_t)h * W + w) * T;
            for (int t = 0; t < T; ++t) row[t] = exp(logit[t] - mx) / sum;
        }
    free(logit);
}

/* ------------------------------------------------------------------ Eqs. 3, 4, 6 */
/* abar[w][t] (Eq. 3), s[t] (Eq. 4), e[t] = -sum_w Ahat log(Ahat + eps) (inner sum of Eq. 6). */
void sabo_scores(const float *q, const float *k, int L, int H, int Hkv, int D, int W,
                 long long ks_tok, long long ks_head, double eps,
                 double *abar, double *s, double *e)
{
    int T = L - W;
    if (T <= 0) return;
#pragma omp parallel for schedule(dynamic, 1)
    for (int w = 0; w < W; ++w) {
        double *logit = (double *)malloc(sizeof(double) * (size_t)L);
        double *row = abar + (size_t)w * T;
        for (int t = 0; t < T; ++t) row[t] = 0.0;
        int n_keys = T + w + 1;
        for (int h = 0; h < H; ++h) {
            row_logits(q, k, h, w, n_keys, H, Hkv, D, W, ks_tok, ks_head, logit);
            double mx = logit[0];
            for (int i = 1; i < n_keys; ++i) if (logit[i] > mx) mx = logit[i];
            double sum = 0.0;
            for (int i = 0; i < n_keys; ++i) sum += exp(logit[i] - mx);
            for (int t = 0; t < T; ++t) row[t] += exp(logit[t] - mx) / sum;
        }
        for (int t = 0; t < T; ++t) row[t] /= (double)H;
        free(logit);
    }
    for (int t = 0; t < T; ++t) {
        double st = 0.0;
        for (int w = 0; w < W; ++w) st += abar[(size_t)w * T + t];
        s[t] = st;
        double ent = 0.0;
        if (st > 0.0) {
            for (int w = 0; w < W; ++w) {
                double ah = abar[(size_t)w * T + t] / st;
                ent -= ah * log(ah + eps);
            }
        }
        e[t] = ent;
    }
}

/* Optional pooling of s (not part of the method's equations; Sec. 2.2 mentions it as
 * SnapKV's device).  Window [t - k/2, t + k/2] clipped to [0, T).  mode 0 = max, 1 = mean. */
void sabo_pool(const double *s, int T, int kernel, int mode, double *out)
{
    int half = kernel / 2;
    for (int t = 0; t < T; ++t) {
        int lo = t - half < 0 ? 0 : t - half;
        int hi = t + half >= T ? T - 1 : t + half;
        double acc = s[lo];
        for (int i = lo + 1; i <= hi; ++i) {
            if (mode == 0) { if (s[i] > acc) acc = s[i]; }
            else acc += s[i];
        }
        out[t] = mode == 0 ? acc : acc / (double)(hi - lo + 1);
    }
}

/* ------------------------------------------------------------------ Eqs. 5, 6, 7, 8 */
void sabo_refine(const double *s, const double *e, const int32_t *seg_start, int n_seg,
                 double alpha, double eta, double *I, double *Dk, double *omega, double *s_ref)
{
    for (int k = 0; k < n_seg; ++k) {
        int a = seg_start[k], b = seg_start[k + 1];
        double si = 0.0, sd = 0.0;
        for (int t = a; t < b; ++t) { si += s[t]; sd += e[t]; }
        double n = (double)(b - a);
        I[k] = si / n;                              /* Eq. 5 */
        Dk[k] = sd / n;                             /* Eq. 6 */
        omega[k] = I[k] * (1.0 + eta * Dk[k]);      /* Eq. 7 */
        for (int t = a; t < b; ++t) s_ref[t] = s[t] * (1.0 + alpha * omega[k]);   /* Eq. 8 */
    }
}

/* ------------------------------------------------------------------ Algorithm 2 */
typedef struct { double key; int idx; } kv_t;

static int cmp_desc(const void *pa, const void *pb)
{
    const kv_t *a = (const kv_t *)pa, *b = (const kv_t *)pb;
    if (a->key > b->key) return -1;
    if (a->key < b->key) return 1;
    return a->idx < b->idx ? -1 : (a->idx > b->idx ? 1 : 0);
}

static void note_margin(double *slot, double hi, double lo)
{
    if (!slot) return;
    double ref = fabs(hi) > fabs(lo) ? fabs(hi) : fabs(lo);
    double m = ref > 0.0 ? fabs(hi - lo) / ref : 0.0;
    if (m < *slot) *slot = m;
}

/* One segment, one block size g: the greedy block fill of Alg. 2's inner loop.
 * sv[0..n): refined scores of the segment; b: implicit budget (1 <= b <= n).
 * taken[i] = 1 for retained tokens.  Returns Score_k(g).  If blocks != NULL, the
 * (start, end) of every block that contributed tokens is appended (segment-local). */
double sabo_segment_fill(const double *sv, int n, int b, int g, uint8_t *taken,
                         int32_t *blocks, int *n_blocks, double *margins)
{
    int nb = (n + g - 1) / g;
    kv_t *blk = (kv_t *)malloc(sizeof(kv_t) * (size_t)nb);
    for (int m = 0; m < nb; ++m) {
        int a = m * g, z = a + g < n ? a + g : n;
        double phi = 0.0;
        for (int t = a; t < z; ++t) phi += sv[t];
        blk[m].key = phi;
        blk[m].idx = m;
    }
    qsort(blk, (size_t)nb, sizeof(kv_t), cmp_desc);
    memset(taken, 0, (size_t)n);
    int cnt = 0, nbk = 0;
    for (int r = 0; r < nb; ++r) {
        int m = blk[r].idx;
        int a = m * g, z = a + g < n ? a + g : n;
        int sz = z - a;
        if (margins && r + 1 < nb) note_margin(&margins[1], blk[r].key, blk[r + 1].key);
        if (cnt + sz <= b) {
            for (int t = a; t < z; ++t) taken[t] = 1;
            cnt += sz;
            if (blocks) { blocks[2 * nbk] = a; blocks[2 * nbk + 1] = z; }
            ++nbk;
        } else {
            int need = b - cnt;
            if (need > 0) {
                kv_t *tok = (kv_t *)malloc(sizeof(kv_t) * (size_t)sz);
                for (int t = a; t < z; ++t) { tok[t - a].key = sv[t]; tok[t - a].idx = t; }
                qsort(tok, (size_t)sz, sizeof(kv_t), cmp_desc);
                for (int i = 0; i < need; ++i) taken[tok[i].idx] = 1;
                if (margins) note_margin(&margins[2], tok[need - 1].key, tok[need].key);
                free(tok);
                if (blocks) { blocks[2 * nbk] = a; blocks[2 * nbk + 1] = z; }
                ++nbk;
            }
            break;
        }
    }
    free(blk);
    double score = 0.0;
    for (int t = 0; t < n; ++t) if (taken[t]) score += sv[t];
    if (n_blocks) *n_blocks = nbk;
    return score;
}

/* Algorithm 2 over all segments.
 *  sr[T]      refined scores; B token budget for the compressible region (0 <= B <= T)
 *  keep[B]    retained indices, ascending (Eq. 13)
 *  g_star[k]  chosen block size (0 where b_k = 0); b_k[k] implicit budgets (Eq. 10)
 *  margins[4] (optional, in/out minima; initialise to +inf): relative gap of
 *             [0] the Top-B boundary, [1] adjacent blocks in a block ordering,
 *             [2] the partial-block token boundary, [3] Score(g) vs tau*Score_base
 *  blocks     (optional) [2*B] absolute (start, end) of the blocks that contributed,
 *             n_blocks_out their count
 * Returns the number of retained indices (= B). */
int sabo_select(const double *sr, int T, const int32_t *seg_start, int n_seg, int B,
                const int32_t *cand, int n_cand, double tau,
                int32_t *keep, int32_t *g_star, int32_t *b_k, double *margins,
                int32_t *blocks, int32_t *n_blocks_out)
{
    /* Eq. 9: Top-B by a full sort, ties to the lower index. */
    kv_t *all = (kv_t *)malloc(sizeof(kv_t) * (size_t)(T > 0 ? T : 1));
    for (int t = 0; t < T; ++t) { all[t].key = sr[t]; all[t].idx = t; }
    qsort(all, (size_t)T, sizeof(kv_t), cmp_desc);
    uint8_t *in_top = (uint8_t *)calloc((size_t)(T > 0 ? T : 1), 1);
    for (int i = 0; i < B; ++i) in_top[all[i].idx] = 1;
    if (margins && B > 0 && B < T) note_margin(&margins[0], all[B - 1].key, all[B].key);
    free(all);

    uint8_t *keep_flag = (uint8_t *)calloc((size_t)(T > 0 ? T : 1), 1);
    int total_blocks = 0;
    for (int k = 0; k < n_seg; ++k) {
        int a = seg_start[k], z = seg_start[k + 1], n = z - a;
        int b = 0;
        for (int t = a; t < z; ++t) b += in_top[t];             /* Eq. 10 */
        b_k[k] = b;
        g_star[k] = 0;
        if (b == 0) continue;
        double base = 0.0;                                       /* Score_base */
        for (int t = a; t < z; ++t) if (in_top[t]) base += sr[t];
        int lim = n < b ? n : b;
        uint8_t *taken = (uint8_t *)malloc((size_t)n);
        int32_t *blk_tmp = blocks ? (int32_t *)malloc(sizeof(int32_t) * 2 * (size_t)(n + 1)) : NULL;
        for (int ci = n_cand - 1; ci >= 0; --ci) {               /* descending g */
            int g = cand[ci];
            if (g > lim) continue;
            int nbk = 0;
            double score = sabo_segment_fill(sr + a, n, b, g, taken, blk_tmp, &nbk, margins);
            double thr = tau * base;
            if (margins && g != 1) note_margin(&margins[3], score, thr);
            if (g == 1 || score >= thr) {                        /* Eqs. 11, 12 */
                g_star[k] = g;
                for (int t = 0; t < n; ++t) if (taken[t]) keep_flag[a + t] = 1;
                if (blocks)
                    for (int i = 0; i < nbk; ++i) {
                        blocks[2 * total_blocks] = a + blk_tmp[2 * i];
                        blocks[2 * total_blocks + 1] = a + blk_tmp[2 * i + 1];
                        ++total_blocks;
                    }
                break;
            }
        }
        free(taken);
        free(blk_tmp);
    }
    int n_keep = 0;
    for (int t = 0; t < T; ++t) if (keep_flag[t]) keep[n_keep++] = t;   /* Eq. 13 */
    free(keep_flag);
    free(in_top);
    if (n_blocks_out) *n_blocks_out = total_blocks;
    return n_keep;
}

/* ------------------------------------------------------------------ merge + gather */
/* Rows of `src` (row_bytes each, token stride stride_bytes) at idx[0..n) copied to dst. */
void sabo_gather(const uint8_t *src, long long stride_bytes, long long row_bytes,
                 const int32_t *idx, int n, uint8_t *dst)
{
    for (int i = 0; i < n; ++i)
        memcpy(dst + (size_t)i * row_bytes, src + (size_t)idx[i] * stride_bytes, (size_t)row_bytes);
}

/* ------------------------------------------------------------------ decoding over a cache */
/* Attention of ONE new query token over a cache of n entries (Eqs. 1-2 with a single query row;
 * Sec. 4.4 measures decoding over the compressed cache): for every query head h, with the KV head
 * of its group,  out[h] = sum_i softmax_i(q[h] . k[i] / sqrt(D)) * v[i].  Every entry is visible to
 * the new token.  q [H][D]; k, v [n][Hkv][D]; out [H][D]; lse [H] = ln of the normaliser. */
void sabo_decode_attention(const float *q, const float *k, const float *v, int n, int H, int Hkv, int D,
                           double *out, double *lse)
{
    int G = H / Hkv;
    double inv = 1.0 / sqrt((double)D);
    double *logit = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    for (int h = 0; h < H; ++h) {
        int j = h / G;
        const float *qr = q + (size_t)h * D;
        for (int d = 0; d < D; ++d) out[(size_t)h * D + d] = 0.0;
        if (n <= 0) { if (lse) lse[h] = -INFINITY; continue; }
        for (int i = 0; i < n; ++i) {
            const float *kr = k + ((size_t)i * Hkv + j) * D;
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += (double)qr[d] * (double)kr[d];
            logit[i] = acc * inv;
        }
        double mx = logit[0];
        for (int i = 1; i < n; ++i) if (logit[i] > mx) mx = logit[i];
        double sum = 0.0;
        for (int i = 0; i < n; ++i) sum += exp(logit[i] - mx);
        for (int i = 0; i < n; ++i) {
            double w = exp(logit[i] - mx) / sum;
            const float *vr = v + ((size_t)i * Hkv + j) * D;
            for (int d = 0; d < D; ++d) out[(size_t)h * D + d] += w * (double)vr[d];
        }
        if (lse) lse[h] = mx + log(sum);
    }
    free(logit);
}

/* ------------------------------------------------------------------ whole pass */
/* One (layer, sequence).  Outputs: out_idx[n_keep] (ascending positions in the
 * compressible region, then the W window positions), and optionally the stage results.
 * Eq. 13 fixes |T*| = B and the text after it adds the recent tokens on top, but the paper
 * does not say whether a quoted "budget" counts them.  budget_includes_window = 1: budget
 * counts all retained entries, window included, so B = budget - W; 0: B = budget and
 * budget + W entries are retained.  If the entries to retain are >= L everything is kept.
 * Returns n_keep. */
int sabo_compress(const float *q, const float *k, const int32_t *token_ids, int L,
                  int H, int Hkv, int D, int W, long long ks_tok, long long ks_head,
                  const uint32_t *bitmap, int vocab,
                  double alpha, double eta, double eps, double tau,
                  int pool_kernel, int pool_mode,
                  int budget, int budget_includes_window, const int32_t *cand, int n_cand,
                  int32_t *out_idx, int32_t *seg_id, int32_t *seg_start, int32_t *n_seg_out,
                  double *s_out, double *e_out, double *s_ref_out,
                  int32_t *g_star, int32_t *b_k, double *margins)
{
    int T = L - W;
    int n_out = budget_includes_window ? budget : budget + W;
    if (n_out >= L) {
        for (int i = 0; i < L; ++i) out_idx[i] = i;
        return L;
    }
    int B = n_out - W;
    int n_seg = sabo_segment(token_ids, L, W, bitmap, vocab, seg_id, seg_start);
    if (n_seg_out) *n_seg_out = n_seg;
    double *abar = (double *)malloc(sizeof(double) * (size_t)W * T);
    double *s = (double *)malloc(sizeof(double) * (size_t)T);
    double *e = (double *)malloc(sizeof(double) * (size_t)T);
    sabo_scores(q, k, L, H, Hkv, D, W, ks_tok, ks_head, eps, abar, s, e);
    free(abar);
    if (pool_kernel > 1) {
        double *sp = (double *)malloc(sizeof(double) * (size_t)T);
        sabo_pool(s, T, pool_kernel, pool_mode, sp);
        memcpy(s, sp, sizeof(double) * (size_t)T);
        free(sp);
    }
    double *I = (double *)malloc(sizeof(double) * (size_t)n_seg);
    double *Dk = (double *)malloc(sizeof(double) * (size_t)n_seg);
    double *om = (double *)malloc(sizeof(double) * (size_t)n_seg);
    double *sr = (double *)malloc(sizeof(double) * (size_t)T);
    sabo_refine(s, e, seg_start, n_seg, alpha, eta, I, Dk, om, sr);
    int n = sabo_select(sr, T, seg_start, n_seg, B, cand, n_cand, tau, out_idx, g_star, b_k,
                        margins, NULL, NULL);
    for (int w = 0; w < W; ++w) out_idx[n + w] = T + w;      /* window always kept (Sec. 3.1) */
    if (s_out) memcpy(s_out, s, sizeof(double) * (size_t)T);
    if (e_out) memcpy(e_out, e, sizeof(double) * (size_t)T);
    if (s_ref_out) memcpy(s_ref_out, sr, sizeof(double) * (size_t)T);
    free(I); free(Dk); free(om); free(sr); free(s); free(e);
    return n + W;
}
