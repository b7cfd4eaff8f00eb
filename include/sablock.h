/*
 * sablock.h -- C ABI of the B200 (sm_100a) implementation of SABlock's prefill-time
 * KV-cache compression pass (semantic segmentation, observation-window scoring,
 * segment-guided refinement, budget-driven adaptive block-size search, top-k selection
 * and compaction of the retained K/V rows).
 *
 * Conventions (all entry points):
 *  - "dev" pointers are CUDA device pointers owned by the caller; "host" pointers are
 *    ordinary host memory.  The library never allocates or frees device memory: all
 *    scratch comes from the caller's workspace `ws` (size from sablock_workspace_bytes).
 *  - Device work is enqueued asynchronously on `stream` (a cudaStream_t passed as void*).
 *    The return code reports host-side validation and launch errors only; on any error
 *    nothing further is enqueued.  Conditions detected on the device (a bounded wait that
 *    ran out, an internal consistency check) are written to a device status word that the
 *    caller may read after synchronising (see sablock_read_status).
 *  - Positions: a prompt has L tokens; the last W = `window` tokens are the observation
 *    window and are never evicted; T = L - W is the compressible region (Sec. 3.1).
 *  - Layouts: q_win [H, W, D]; k, v [L, Hkv, D] with element strides given in the
 *    parameter block; all score vectors are fp32 of length T; indices are int32.
 *  - `budget` counts every retained entry.  With budget_includes_window = 1 (default) the
 *    W window entries are part of it, so Algorithm 2 runs with B = budget - W and exactly
 *    `budget` rows are produced; with 0, B = budget and budget + W rows are produced.
 *    If the rows to produce would be >= L the cache is returned unchanged (identity).
 */
#ifndef SABLOCK_H
#define SABLOCK_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SABLOCK_OK = 0,
    SABLOCK_ERR_INVALID_ARG = 1,
    SABLOCK_ERR_UNSUPPORTED = 2,
    SABLOCK_ERR_WORKSPACE_TOO_SMALL = 3,
    SABLOCK_ERR_CUDA = 4,
    SABLOCK_ERR_TIMEOUT = 5,
    SABLOCK_ERR_INTERNAL = 6
} sablock_status_t;

typedef enum { SABLOCK_F32 = 0, SABLOCK_BF16 = 1 } sablock_dtype_t;

/* Which kernel family computes the attention scores.  AUTO picks, in this order, the
 * persistent tensor-core kernel (bf16, head_dim 128, window 32, four query heads per KV head,
 * at most 7 token tiles of 128 per CTA; two sweeps over K, or one when row_lse is given), the
 * two-launch tensor-core kernels (bf16, head_dim 64/128, window 8/16/32), and the SIMT kernels
 * otherwise (with row_lse these run their second pass only).  FUSED and TENSOR force the first
 * and the second and fail with SABLOCK_ERR_UNSUPPORTED where they cannot run. */
typedef enum { SABLOCK_SCORE_AUTO = 0, SABLOCK_SCORE_SIMT = 1, SABLOCK_SCORE_TENSOR = 2, SABLOCK_SCORE_FUSED = 3 }
    sablock_score_impl_t;

#define SABLOCK_MAX_SEQS 64        /* sequences per batched call              */
#define SABLOCK_MAX_CANDIDATES 16  /* block-size candidates                   */

typedef void *sablock_stream_t;    /* a cudaStream_t */

/* Plain-data parameter block, passed by const pointer.  Fill it with
 * sablock_params_default() and then set the shape fields. */
typedef struct sablock_params {
    int n_q_heads;                 /* H   query heads (Eq. 3 averages over these)               */
    int n_kv_heads;                /* Hkv key/value heads; H % Hkv == 0 (grouped-query attention) */
    int head_dim;                  /* D                                                         */
    int window;                    /* W = n_rcnt, observation window (Sec. 3.1)                 */
    int dtype;                     /* sablock_dtype_t of q_win, k, v, out_k, out_v              */
    long long k_stride_token;      /* element strides of k; 0 = contiguous [L, Hkv, D]          */
    long long k_stride_head;
    long long k_stride_layer;      /* batched call only; 0 = total_tokens * k_stride_token      */
    long long v_stride_token;      /* same for v                                                */
    long long v_stride_head;
    long long v_stride_layer;
    float alpha;                   /* Eq. 8, default 0.9                                        */
    float eta;                     /* Eq. 7, default 1.0                                        */
    float eps;                     /* Eq. 6, default 1e-6                                       */
    float tau;                     /* Eq. 12 fidelity threshold, default 0.85                   */
    int pool_kernel;               /* 1 = no pooling (the paper's method); odd k > 1 pools s_t  */
    int pool_mode;                 /* 0 = max, 1 = mean                                         */
    int budget_includes_window;    /* default 1                                                 */
    const unsigned *delim_bitmap;  /* dev: bit (id % 32) of word (id / 32) set <=> id delimits  */
    int vocab_size;                /* ids outside [0, vocab_size) never delimit                 */
    int score_impl;                /* sablock_score_impl_t                                      */
    int debug_sync;                /* diagnostic aid, default 0: non-zero makes sablock_compress_layers
                                      wait for the stream after every stage, so that a device fault
                                      is reported (sablock_last_cuda_error) with the stage that
                                      raised it; it serialises host and device                  */
    /* Optional, dev f32 [n_layers, n_seqs, H, W] (single-problem calls: [H, W]), or NULL.
     * row_lse[h][w] = ln sum_{j <= T+w} exp(q_{h,w} . k_j / sqrt(D)): the log of the softmax
     * normaliser of Eq. 2 for the query at position T + w, over its causal keys, as the prefill's
     * attention kernel leaves it for every query row (the pass runs right after a FlashAttention
     * prefill, Sec. 4.1, which keeps this value per row).  When given, the scores are computed in
     * ONE sweep over K: A = exp(logit - row_lse) needs no normalising sweep of its own.  The values
     * are trusted: a row_lse that is not the normaliser of the q_win and k passed in scales that
     * row's attention weights by exp(true - given).  The values of sequences that are returned
     * unchanged are ignored. */
    const float *row_lse;
    /* Default 0.  The persistent score kernel in its two-sweep mode lets the sweep that accumulates
     * the softmax normalisers run ahead while the other waits for another CTA; which of its two
     * groups of warps then sums which token tile depends on timing, so the normalisers (sums of up
     * to 131072 fp32 terms) can differ in their last bit from run to run, and the scores with them
     * by about 1e-7 relative.  Non-zero fixes the order of the tile steps: scores are then identical
     * bit for bit across runs, at about 17 % more time for the score stage on a 128K-token prompt.
     * Every other mode and kernel (row_lse given, the two-launch and SIMT kernels, all other stages)
     * is bit-reproducible as it is. */
    int reproducible;
    int reserved[5];
} sablock_params_t;

void sablock_params_default(sablock_params_t *p);
const char *sablock_status_string(sablock_status_t st);
int sablock_version(void);
/* Text of the most recent CUDA runtime error an entry point of this thread ran into (which call,
 * after how many kernel launches of that entry point, and the runtime's message); "" if none.
 * See debug_sync in the parameter block for the stage that raised a device fault. */
const char *sablock_last_cuda_error(void);
size_t sablock_params_sizeof(void);   /* sizeof(sablock_params_t) as the library was built */

/* Bytes of device scratch needed for a call over n_layers x n_seqs problems whose
 * sequences have at most max_L tokens and total_tokens tokens in all.  Single-problem
 * entry points use n_layers = n_seqs = 1, total_tokens = max_L = L.  Returns 0 on
 * invalid arguments. */
size_t sablock_workspace_bytes(const sablock_params_t *p, long long total_tokens, int max_L,
                               int n_seqs, int n_layers);

/* Where a fused call leaves its intermediate results inside the workspace, for diagnostics
 * and tests: name is one of "s", "e", "s_refined" (f32 [n_layers][total_tokens], token row
 * cu_seqlens[i] + t), "seg_id" (int32 [total_tokens]), "seg_start" (int32, sequence i at
 * element cu_seqlens[i] + i), "n_seg" (int32 [n_seqs]).  Stores the byte offset and size;
 * same arguments as sablock_workspace_bytes.  Returns SABLOCK_ERR_INVALID_ARG for an
 * unknown name. */
sablock_status_t sablock_workspace_region(const sablock_params_t *p, long long total_tokens, int max_L,
                                          int n_seqs, int n_layers, const char *name,
                                          size_t *offset, size_t *bytes);

/* Reads (synchronously: it waits for `stream`) the device status word kept at the start of
 * the workspace.  Returns SABLOCK_OK, SABLOCK_ERR_TIMEOUT or SABLOCK_ERR_INTERNAL; the raw
 * word is stored to *raw (host) if not NULL. */
sablock_status_t sablock_read_status(const void *ws, sablock_stream_t stream, int *raw);

/* The same, with the word that follows the status word: raw2 (host int[2]) receives the status
 * word and, if a bounded wait ran out, which one gave up first:
 * code | (CTA index << 8) | (warp index << 20).  Codes 1-29 are waits of the persistent score kernel
 * (1 query-block buffer free, 2 K stage free, 3 query block loaded, 4 accumulator free, 5 K tile
 * loaded, 6 row sums of a phase in shared memory, 7 accumulator complete, 8 log-sum-exps fetched,
 * 9 turn at the exponentials, 11 partial-sum slot free, 12 row sums of all CTAs, 13 merged
 * log-sum-exps, 20 / 21 exchanges inside the epilogue, 22 the other epilogue set's previous step), 30 the look-back of the segmentation scan,
 * 31 the CTAs of one problem in the Top-B select.  Every such wait is limited to about a second of
 * device time; the kernel that gave up returns, the later stages still run on whatever was
 * produced and stay inside their buffers. */
sablock_status_t sablock_read_status_detail(const void *ws, sablock_stream_t stream, int *raw2);

/* Stage 1 -- semantic segmentation (Sec. 3.1, "Semantic-Aware Segmentation").
 * A token whose id is in the delimiter set is the last token of its segment.
 *  token_ids dev int32[L]; seg_id dev int32[T] (segment index of each token);
 *  seg_start dev int32[T+1] (first n_seg+1 entries valid, seg_start[n_seg] = T);
 *  n_seg dev int32[1]. */
sablock_status_t sablock_segment(const sablock_params_t *p, const int *token_ids, int L,
                                 int *seg_id, int *seg_start, int *n_seg,
                                 void *ws, size_t ws_bytes, sablock_stream_t stream);

/* Stage 1 again, for callers that have no device memory to spare for scratch and no way to get
 * any.  (The paper has no counterpart; this is a service of this library.)  Some hosts of this
 * code may not allocate: an inference server whose memory pool is sized once and then frozen, a
 * plug-in that is handed only its input and output buffers, a latency-critical loop in which
 * cudaMalloc's implicit device synchronisation is not acceptable.  This variant needs no
 * workspace: the look-back state of the segmentation scan lives in a fixed 8.25 KB array inside the
 * library's device image (every GPU that loads the library holds it until the process exits).
 * Same arguments and results as sablock_segment, minus the workspace.
 *  - Limit: T = L - W <= SABLOCK_SEGMENT_STATIC_MAX_T tokens; longer inputs are rejected with
 *    SABLOCK_ERR_UNSUPPORTED and nothing is enqueued.
 *  - status: dev int32[1] or NULL.  If given it must be zero before the call; a bounded wait that
 *    ran out sets bit 0 (as in the workspace status word).  With NULL the word is kept inside the
 *    static array and cannot be read back.
 *  - The first call on each device looks up the array's device address (no allocation); make
 *    that first call outside any stream capture.
 *  - Every call on a device shares the one array.  The call clears what it needs on `stream`
 *    before the kernel, so back-to-back calls on one stream are fine; two calls whose device work
 *    overlaps (different streams, or different host threads on different streams) race on it and
 *    give wrong segment ids.
 *  - Calls no cudaMalloc / cudaFree and no allocating library routine. */
#define SABLOCK_SEGMENT_STATIC_MAX_T (1024 * 2048)
sablock_status_t sablock_segment_static(const sablock_params_t *p, const int *token_ids, int L,
                                        int *seg_id, int *seg_start, int *n_seg, int *status,
                                        sablock_stream_t stream);

/* Stages 2+3 -- observation-window scoring (Sec. 3.2, Eqs. 2-4 and the per-token entropy of
 * Eq. 6) followed by segment-guided refinement (Eqs. 5-8, Algorithm 1).
 *  q_win dev [H, W, D]: queries of the last W prompt positions; k dev [L, Hkv, D];
 *  seg_start / n_seg: from sablock_segment;
 *  s dev f32[T] window score s_t (after pooling if enabled); e dev f32[T] or NULL: per-token
 *  entropy; s_refined dev f32[T]; seg_stats dev f32[3*T] or NULL: I_k, D_k, omega_k in rows
 *  of length T (first n_seg entries of each valid). */
sablock_status_t sablock_score(const sablock_params_t *p, const void *q_win, const void *k, int L,
                               const int *seg_start, const int *n_seg,
                               float *s, float *e, float *s_refined, float *seg_stats,
                               void *ws, size_t ws_bytes, sablock_stream_t stream);

/* Stage 4 + index list -- Algorithm 2 (Sec. 3.3, Eqs. 9-13): global Top-B, implicit
 * budgets, per-segment block-size search, aggregation.
 *  block_candidates host int[n_candidates], strictly ascending, first entry 1;
 *  out_idx dev int32[n_out]: retained positions, ascending, the W window positions last,
 *  where n_out = budget (or budget + W, see budget_includes_window) or L for identity;
 *  out_seg_block dev int32[T] or NULL: g*_k (0 where b_k = 0); out_seg_budget dev int32[T]
 *  or NULL: b_k. */
sablock_status_t sablock_select(const sablock_params_t *p, const float *s_refined, int L,
                                const int *seg_start, const int *n_seg, int budget,
                                const int *block_candidates, int n_candidates,
                                int *out_idx, int *out_seg_block, int *out_seg_budget,
                                void *ws, size_t ws_bytes, sablock_stream_t stream);

/* Stage 5 -- merge with the recent tokens and compact (end of Sec. 3.3): copies rows
 * out_idx[0..n_keep) of k and v into out_k, out_v dev [n_keep, Hkv, D] (contiguous). */
sablock_status_t sablock_compact(const sablock_params_t *p, const void *k, const void *v, int L,
                                 const int *out_idx, int n_keep, void *out_k, void *out_v,
                                 sablock_stream_t stream);

/* The whole pass for one layer of one sequence (Fig. 5 steps 1-4).
 *  out_k, out_v dev [n_out, Hkv, D]; out_idx dev int32[n_out]; out_n_keep dev int32[1]. */
sablock_status_t sablock_compress(const sablock_params_t *p, const void *q_win, const void *k,
                                  const void *v, const int *token_ids, int L, int budget,
                                  const int *block_candidates, int n_candidates,
                                  void *out_k, void *out_v, int *out_idx, int *out_n_keep,
                                  void *ws, size_t ws_bytes, sablock_stream_t stream);

/* The whole pass for n_layers layers of n_seqs packed sequences in one launch sequence.
 *  cu_seqlens host int[n_seqs+1], cu_seqlens[0] = 0: sequence i occupies packed token rows
 *  [cu_seqlens[i], cu_seqlens[i+1]);
 *  q_win dev [n_layers, n_seqs, H, W, D]; k, v dev [n_layers, total_tokens, Hkv, D] (strides
 *  from the parameter block); token_ids dev int32[total_tokens] (shared by all layers);
 *  out_k, out_v dev [n_layers, n_seqs, n_out, Hkv, D]; out_idx dev int32[n_layers, n_seqs,
 *  n_out] (positions local to each sequence); out_n_keep dev int32[n_layers, n_seqs].
 *  Sequences with L_i <= n_out are returned unchanged in their first L_i rows. */
sablock_status_t sablock_compress_layers(const sablock_params_t *p, int n_layers, int n_seqs,
                                         const void *q_win, const void *k, const void *v,
                                         const int *token_ids, const int *cu_seqlens, int budget,
                                         const int *block_candidates, int n_candidates,
                                         void *out_k, void *out_v, int *out_idx, int *out_n_keep,
                                         void *ws, size_t ws_bytes, sablock_stream_t stream);

/* Same pass with HOST inputs and outputs (the end-to-end path): copies q_win, k and token_ids
 * from host memory into the caller's device staging buffers (dev_*; same shapes as above), runs
 * sablock_compress_layers, copies out_k, out_v, out_idx, out_n_keep back to host memory and waits
 * for `stream`.  The pass reads every key but only the retained rows of v: if h_v is page-locked
 * (pinned) host memory the gather reads those rows from it in place and dev_v is not written;
 * otherwise v is copied to dev_v first.  Pinned host memory also makes the copies asynchronous
 * with respect to each other; pageable memory works too.  All arguments are validated before the
 * first copy is enqueued. */
sablock_status_t sablock_compress_layers_host(const sablock_params_t *p, int n_layers, int n_seqs,
                                              const void *h_q_win, const void *h_k, const void *h_v,
                                              const int *h_token_ids, const int *cu_seqlens, int budget,
                                              const int *block_candidates, int n_candidates,
                                              void *h_out_k, void *h_out_v, int *h_out_idx, int *h_out_n_keep,
                                              void *dev_q_win, void *dev_k, void *dev_v, int *dev_token_ids,
                                              void *dev_out_k, void *dev_out_v, int *dev_out_idx,
                                              int *dev_out_n_keep,
                                              void *ws, size_t ws_bytes, sablock_stream_t stream);

/* Decoding over the compacted cache (Sec. 4.4 measures its latency and memory against the full
 * cache): the attention of ONE new query token per problem over the rows of a cache, Eqs. 1-2 with
 * a single query row, grouped-query attention as in the scores:
 *   out[h] = sum_i softmax_i(q[h] . k[i, kv(h)] / sqrt(D)) * v[i, kv(h)],  every row visible.
 * n_prob problems (layers x sequences, or one layer at a time as a decoder runs them);
 *  q dev [n_prob, H, D] (dtype of the parameter block); k_cache, v_cache dev [n_prob, n_rows, Hkv, D]:
 *  what sablock_compress_layers wrote (n_rows = n_out), or a full cache (n_rows = L); element
 *  strides from the parameter block's k_/v_stride_token, _head, and _layer (between problems),
 *  0 = contiguous; n_valid dev int32[n_prob] or NULL: rows of each problem that count (out_n_keep),
 *  NULL = all n_rows; out dev f32 [n_prob, H, D]; lse dev f32 [n_prob, H] or NULL: natural log of
 *  the softmax normaliser.  Scratch from ws (sablock_decode_workspace_bytes; returns 0 on invalid
 *  arguments).  Supported: 1, 2 or 4 query heads per KV head, head_dim * element size of 128, 256
 *  or 512 bytes.  Accumulation is fp32 in a fixed order (row splits merged in index order). */
size_t sablock_decode_workspace_bytes(const sablock_params_t *p, int n_prob, int n_rows);
sablock_status_t sablock_decode_attention(const sablock_params_t *p, int n_prob, const void *q,
                                          const void *k_cache, const void *v_cache, int n_rows,
                                          const int *n_valid, float *out, float *lse,
                                          void *ws, size_t ws_bytes, sablock_stream_t stream);

/* Per-stage timing (optional, for benchmarks).  While enabled, every fused call of this
 * thread records CUDA events on its stream between the stages, into the next of `slots`
 * event sets (round robin; the events are created on first use and kept until exit).
 * sablock_profile_read(slot, ...) waits for that slot's last event and stores the
 * milliseconds of each stage interval; it returns the number of intervals (0 if the slot
 * was never used).  sablock_profile_stage_name(i) names interval i.  The stages are:
 * segment, score_pass1, score_merge, score_pass2, refine, topb, search, index, compact. */
#define SABLOCK_PROFILE_MAX_SLOTS 512
sablock_status_t sablock_profile_enable(int slots);   /* 0 disables; resets the slot counter */
int sablock_profile_read(int slot, float *ms_out, int max_n);
const char *sablock_profile_stage_name(int i);

/* Number of kernels the most recent entry-point call of this thread enqueued (for
 * launch accounting in benchmarks). */
int sablock_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SABLOCK_H */
