// C ABI of the SABlock compression library (see include/sablock.h): argument validation,
// workspace planning, TMA tensor maps and kernel launches.  Every step of the pass runs in
// the kernels of stages.cuh / score_simt.cuh / score_tc.cuh; there is no host fallback.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "stages.cuh"
#include "score_simt.cuh"
#include "score_tc.cuh"
#include "score_fused.cuh"
#include "decode.cuh"

using namespace sab;

namespace {

thread_local int t_launches = 0;

// ---- optional per-stage event timing ---------------------------------------------------
constexpr int kProfStages = 9;
const char* const kProfNames[kProfStages] = {"segment", "score_pass1", "score_merge", "score_pass2", "refine",
                                             "topb", "search", "index", "compact"};
struct ProfState {
    int slots = 0, next = 0, cur = -1;
    cudaEvent_t ev[SABLOCK_PROFILE_MAX_SLOTS][kProfStages + 1] = {};
    bool used[SABLOCK_PROFILE_MAX_SLOTS] = {};
};
thread_local ProfState* t_prof = nullptr;

void prof_begin_call(cudaStream_t st)
{
    if (!t_prof || t_prof->slots <= 0) return;
    ProfState& ps = *t_prof;
    ps.cur = ps.next;
    ps.next = (ps.next + 1) % ps.slots;
    for (int i = 0; i <= kProfStages; ++i)
        if (!ps.ev[ps.cur][i]) cudaEventCreate(&ps.ev[ps.cur][i]);
    ps.used[ps.cur] = true;
    cudaEventRecord(ps.ev[ps.cur][0], st);
}
void prof_mark(int stage_done, cudaStream_t st)      // after stage `stage_done` (0-based)
{
    if (!t_prof || t_prof->slots <= 0 || t_prof->cur < 0) return;
    cudaEventRecord(t_prof->ev[t_prof->cur][stage_done + 1], st);
}
void prof_end_call()
{
    if (t_prof) t_prof->cur = -1;
}

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

struct Plan {
    // geometry
    Geo geo;
    int n_prob, max_L;
    bool use_tc;
    bool use_fused;            // the persistent two-sweep kernel (Llama-shaped problems)
    int fu_cpp, fu_groups;     // its CTAs per problem group and number of groups
    int tpc1, tpc2;            // tiles per CTA of the tensor-core passes
    int n_chunks;              // pass-1 partials per row
    int keep_words, long_cap, seg_tiles;
    // workspace offsets
    size_t o_status, o_ticket, o_long_count, o_tile_state, o_keep, o_arrive, o_done, o_top, control_bytes;
    size_t o_seg_id, o_seg_start, o_n_seg, o_s_raw, o_s, o_e, o_sr, o_part, o_lse, o_neg_lse, o_thr, o_cut, o_long_list,
        o_phi, o_fpart, total;
};

bool tc_eligible(const sablock_params_t* p)
{
    if (p->dtype != SABLOCK_BF16) return false;
    if (p->head_dim != 64 && p->head_dim != 128) return false;
    if (p->window != 8 && p->window != 16 && p->window != 32) return false;
    const int G = p->n_q_heads / p->n_kv_heads;
    if (G * p->window > 128) return false;
    return true;
}

// The persistent kernel takes the shape whose 128 window rows per KV head fill one MMA tile.
bool fused_eligible(const sablock_params_t* p)
{
    return tc_eligible(p) && p->head_dim == 128 && p->window == 32 && p->n_q_heads / p->n_kv_heads == 4;
}

constexpr int kFuMaxCtas = kFuMaxCtasDev;   // upper bound on the CTAs of the persistent kernel (workspace sizing)

// CTAs the persistent kernel may use on the current device: one per SM, all co-resident.
int fused_cta_limit()
{
    static int cached[64];
    static bool have[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!have[dev]) {
        int sms = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        if (cudaFuncSetAttribute(score_fused_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kFuSmemBytes) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, score_fused_tc, kFuThreads, kFuSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
        cached[dev] = per_sm >= 1 ? (sms < kFuMaxCtas ? sms : kFuMaxCtas) : 0;
        have[dev] = true;
    }
    return cached[dev];
}

// SMs of the current device; 148, a B200's count, where no device can be asked (sizing a
// workspace on a host without a GPU).  The tiles per CTA of the two-launch score kernels, and with
// them the size of their partial-sum scratch, follow from it: size a workspace with the device
// current that will use it.
int sm_count()
{
    static int cached[64];
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
    if (cached[dev] > 0) return cached[dev];
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        cudaGetLastError();
        return 148;
    }
    return cached[dev] = sms;
}

sablock_status_t validate_params(const sablock_params_t* p)
{
    if (!p) return SABLOCK_ERR_INVALID_ARG;
    if (p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->n_q_heads % p->n_kv_heads) return SABLOCK_ERR_INVALID_ARG;
    if (p->head_dim <= 0 || p->window <= 0) return SABLOCK_ERR_INVALID_ARG;
    if (p->dtype != SABLOCK_F32 && p->dtype != SABLOCK_BF16) return SABLOCK_ERR_INVALID_ARG;
    if (p->pool_kernel < 1 || (p->pool_kernel & 1) == 0) return SABLOCK_ERR_INVALID_ARG;
    if (p->pool_mode != 0 && p->pool_mode != 1) return SABLOCK_ERR_INVALID_ARG;
    if (p->score_impl < 0 || p->score_impl > 3) return SABLOCK_ERR_INVALID_ARG;
    if (!(p->tau >= 0.f) || !(p->alpha >= 0.f) || !(p->eta >= 0.f) || !(p->eps >= 0.f)) return SABLOCK_ERR_INVALID_ARG;
    if (p->k_stride_token < 0 || p->k_stride_head < 0 || p->k_stride_layer < 0 || p->v_stride_token < 0 ||
        p->v_stride_head < 0 || p->v_stride_layer < 0)
        return SABLOCK_ERR_INVALID_ARG;
    if (p->window > kSimtMaxW || p->head_dim > kSimtMaxD) return SABLOCK_ERR_UNSUPPORTED;
    if ((long long)p->n_q_heads * p->window > 2048) return SABLOCK_ERR_UNSUPPORTED;
    const int es = p->dtype == SABLOCK_BF16 ? 2 : 4;
    if ((p->head_dim * es) % 16) return SABLOCK_ERR_UNSUPPORTED;
    if (p->score_impl == SABLOCK_SCORE_TENSOR && !tc_eligible(p)) return SABLOCK_ERR_UNSUPPORTED;
    if (p->score_impl == SABLOCK_SCORE_FUSED && !fused_eligible(p)) return SABLOCK_ERR_UNSUPPORTED;
    return SABLOCK_OK;
}

int elem_size(const sablock_params_t* p) { return p->dtype == SABLOCK_BF16 ? 2 : 4; }

struct Strides { long long tok, head, layer; };
Strides k_strides(const sablock_params_t* p, long long total_tokens)
{
    Strides s;
    s.head = p->k_stride_head ? p->k_stride_head : p->head_dim;
    s.tok = p->k_stride_token ? p->k_stride_token : (long long)p->n_kv_heads * p->head_dim;
    s.layer = p->k_stride_layer ? p->k_stride_layer : total_tokens * s.tok;
    return s;
}
Strides v_strides(const sablock_params_t* p, long long total_tokens)
{
    Strides s;
    s.head = p->v_stride_head ? p->v_stride_head : p->head_dim;
    s.tok = p->v_stride_token ? p->v_stride_token : (long long)p->n_kv_heads * p->head_dim;
    s.layer = p->v_stride_layer ? p->v_stride_layer : total_tokens * s.tok;
    return s;
}

// Builds geometry + workspace layout.  cu == NULL means one sequence of max_L tokens.
sablock_status_t make_plan(const sablock_params_t* p, int n_layers, int n_seqs, const int* cu, long long total_tokens,
                           int max_L, int n_out, Plan* pl)
{
    sablock_status_t st = validate_params(p);
    if (st != SABLOCK_OK) return st;
    if (n_layers < 1 || n_seqs < 1 || n_seqs > kMaxSeqs || max_L < 1 || total_tokens < max_L) return SABLOCK_ERR_INVALID_ARG;
    if (total_tokens > 0x7fffffffLL || (long long)n_layers * total_tokens > (1LL << 40)) return SABLOCK_ERR_UNSUPPORTED;
    memset(pl, 0, sizeof(*pl));
    Geo& g = pl->geo;
    g.n_layers = n_layers; g.n_seqs = n_seqs; g.total_tokens = (int)total_tokens; g.window = p->window;
    g.H = p->n_q_heads; g.Hkv = p->n_kv_heads; g.D = p->head_dim; g.G = g.H / g.Hkv;
    g.n_out = n_out; g.B = n_out - p->window;
    if (cu) {
        for (int i = 0; i <= n_seqs; ++i) g.cu[i] = cu[i];
    } else {
        g.cu[0] = 0; g.cu[1] = max_L;
    }
    pl->n_prob = n_layers * n_seqs;
    pl->max_L = max_L;
    // The TMA boxes are 128 rows tall: tensors with fewer rows go to the SIMT kernels.
    const bool tc_rows_ok = total_tokens >= kTcTile && (long long)n_layers * n_seqs * g.H * g.window >= kTcTile;
    pl->use_tc = p->score_impl == SABLOCK_SCORE_TENSOR || p->score_impl == SABLOCK_SCORE_FUSED ||
                 (p->score_impl == SABLOCK_SCORE_AUTO && tc_eligible(p) && tc_rows_ok);
    const long long tiles = (max_L + kTcTile - 1) / kTcTile;
    pl->use_fused = pl->use_tc && p->score_impl != SABLOCK_SCORE_TENSOR && fused_eligible(p);
    if (pl->use_tc) {
        long long work1 = tiles * g.Hkv * pl->n_prob, work2 = tiles * pl->n_prob;
        const int sms = sm_count();
        pl->tpc1 = (int)fmin(8.0, fmax(1.0, (double)(work1 / (sms * 4))));
        pl->tpc2 = (int)fmin(4.0, fmax(1.0, (double)(work2 / (sms * 4))));
        pl->n_chunks = (int)((tiles + pl->tpc1 - 1) / pl->tpc1);
    } else {
        pl->tpc1 = pl->tpc2 = 1;
        pl->n_chunks = (max_L + kSimtThreads - 1) / kSimtThreads;
    }
    pl->keep_words = (max_L + 31) / 32;
    pl->long_cap = max_L / kSegShort + 1;
    pl->seg_tiles = (max_L + kSegTile - 1) / kSegTile;

    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes); return r; };
    pl->o_status = take(64);
    pl->o_ticket = take(sizeof(int) * n_seqs);
    pl->o_long_count = take(sizeof(int) * pl->n_prob);
    pl->o_tile_state = take(sizeof(unsigned long long) * (size_t)n_seqs * pl->seg_tiles);
    pl->o_keep = take(sizeof(unsigned) * (size_t)pl->n_prob * pl->keep_words);
    pl->o_arrive = take(sizeof(int) * (size_t)pl->n_prob * g.Hkv);
    pl->o_done = take(sizeof(int) * (size_t)pl->n_prob * g.Hkv);
    pl->o_top = take(sizeof(TopScratch) * (size_t)pl->n_prob);
    pl->control_bytes = o;
    const size_t ntok = (size_t)n_layers * total_tokens;
    pl->o_seg_id = take(sizeof(int) * total_tokens);
    pl->o_seg_start = take(sizeof(int) * (total_tokens + n_seqs));
    pl->o_n_seg = take(sizeof(int) * n_seqs);
    pl->o_s_raw = take(p->pool_kernel > 1 ? sizeof(float) * ntok : 0);
    pl->o_s = take(sizeof(float) * ntok);
    pl->o_e = take(sizeof(float) * ntok);
    pl->o_sr = take(sizeof(float) * ntok);
    const size_t part_n = pl->use_tc ? (size_t)pl->n_prob * g.Hkv * pl->n_chunks * 128
                                     : (size_t)pl->n_prob * g.H * g.window * pl->n_chunks;
    pl->o_part = take(sizeof(float2) * part_n);
    pl->o_lse = take(sizeof(float) * (size_t)pl->n_prob * g.H * g.window);
    pl->o_neg_lse = take(sizeof(float) * (size_t)pl->n_prob * g.H * g.window);
    pl->o_thr = take(sizeof(unsigned) * pl->n_prob);
    pl->o_cut = take(sizeof(int) * pl->n_prob);
    pl->o_long_list = take(sizeof(int) * (size_t)pl->n_prob * pl->long_cap);
    pl->o_phi = take(sizeof(double) * ntok);
    pl->o_fpart = take(pl->use_fused ? sizeof(float2) * (size_t)kFuMaxCtas * kFuPartSlots * 128 : 0);
    pl->total = o;
    return SABLOCK_OK;
}

template <typename T> T* at(void* ws, size_t off) { return reinterpret_cast<T*>(static_cast<char*>(ws) + off); }

thread_local char t_cuda_error[160] = "";

// Remembers what the CUDA runtime said, for sablock_last_cuda_error().
sablock_status_t note_cuda_error(cudaError_t err, const char* where)
{
    snprintf(t_cuda_error, sizeof(t_cuda_error), "%s after launch %d: %s", where, t_launches, cudaGetErrorString(err));
    return SABLOCK_ERR_CUDA;
}

sablock_status_t check_launch()
{
    ++t_launches;
    const cudaError_t err = cudaGetLastError();
    return err == cudaSuccess ? SABLOCK_OK : note_cuda_error(err, "kernel launch");
}
#define SAB_TRY(expr) do { sablock_status_t _s = (expr); if (_s != SABLOCK_OK) return _s; } while (0)

// Diagnostic aid: with debug_sync set in the parameter block the pipeline waits for the stream
// after every stage, so that a device fault is reported with the stage that raised it.
sablock_status_t debug_sync(const sablock_params_t* p, const char* stage, cudaStream_t stream)
{
    if (!p->debug_sync) return SABLOCK_OK;
    const cudaError_t err = cudaStreamSynchronize(stream);
    return err == cudaSuccess ? SABLOCK_OK : note_cuda_error(err, stage);
}

sablock_status_t zero_control(const Plan& pl, void* ws, cudaStream_t stream)
{
    const cudaError_t err = cudaMemsetAsync(ws, 0, pl.control_bytes, stream);
    return err == cudaSuccess ? SABLOCK_OK : note_cuda_error(err, "clearing the control words");
}

// ------------------------------------------------------------------ stage launchers
sablock_status_t run_segment(const Plan& pl, const sablock_params_t* p, const int* token_ids, int* seg_id,
                             int* seg_start, int* n_seg, void* ws, cudaStream_t stream)
{
    if (!token_ids || !seg_id || !seg_start || !n_seg || !p->delim_bitmap || p->vocab_size <= 0)
        return SABLOCK_ERR_INVALID_ARG;
    dim3 grid(pl.seg_tiles, pl.geo.n_seqs);
    segment_kernel<<<grid, kSegThreads, 0, stream>>>(pl.geo, token_ids, p->delim_bitmap, p->vocab_size, seg_id,
                                                     seg_start, n_seg, at<unsigned long long>(ws, pl.o_tile_state),
                                                     at<int>(ws, pl.o_ticket), pl.seg_tiles, at<int>(ws, pl.o_status),
                                                     at<int>(ws, pl.o_status) + 1);
    return check_launch();
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

sablock_status_t make_tensor_maps(const Plan& pl, const sablock_params_t* p, const void* q, const void* k,
                                  CUtensorMap* tmQ, CUtensorMap* tmK)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return SABLOCK_ERR_CUDA;
    const Geo& g = pl.geo;
    const Strides ks = k_strides(p, g.total_tokens);
    if (g.total_tokens < kTcTile || (long long)pl.n_prob * g.H * g.window < kTcTile) return SABLOCK_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(k) & 15) || (ks.head * 2) % 16 ||
        (ks.tok * 2) % 16 || (ks.layer * 2) % 16)
        return SABLOCK_ERR_UNSUPPORTED;
    {   // queries as rows: [n_prob * H * W, D]
        cuuint64_t dims[2] = {(cuuint64_t)g.D, (cuuint64_t)pl.n_prob * g.H * g.window};
        cuuint64_t strides[1] = {(cuuint64_t)g.D * 2};
        cuuint32_t box[2] = {64, 128};
        cuuint32_t estr[2] = {1, 1};
        if (enc(tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(q), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return SABLOCK_ERR_CUDA;
    }
    {   // keys: [layer][token][kv head][D]
        cuuint64_t dims[4] = {(cuuint64_t)g.D, (cuuint64_t)g.Hkv, (cuuint64_t)g.total_tokens, (cuuint64_t)g.n_layers};
        cuuint64_t strides[3] = {(cuuint64_t)ks.head * 2, (cuuint64_t)ks.tok * 2, (cuuint64_t)ks.layer * 2};
        cuuint32_t box[4] = {64, 1, 128, 1};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc(tmK, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(k), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return SABLOCK_ERR_CUDA;
    }
    return SABLOCK_OK;
}

template <int W>
sablock_status_t launch_p2_tc(const Plan& pl, const CUtensorMap& tmQ, const CUtensorMap& tmK, float c2, float eps,
                              ScoreBufs sb, float* s, float* e, int* status, cudaStream_t stream)
{
    constexpr int NST = 3;
    const int n_atoms = pl.geo.D / 64;
    const int smem = 1024 + NST * 2 * n_atoms * kAtomBytes;
    auto kern = score_p2_tc<W, NST>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return SABLOCK_ERR_CUDA;
    const int tiles = (pl.max_L + kTcTile - 1) / kTcTile;
    dim3 grid((tiles + pl.tpc2 - 1) / pl.tpc2, pl.n_prob);
    kern<<<grid, kTcThreads, smem, stream>>>(tmQ, tmK, pl.geo, c2, eps, sb, pl.tpc2, s, e, status);
    return check_launch();
}

// Stage 2: window scores s (pre-pooling) and per-token entropy e.
sablock_status_t run_score(const Plan& pl, const sablock_params_t* p, const void* q, const void* k, float* s,
                           float* e, void* ws, cudaStream_t stream)
{
    if (!q || !k || !s || !e) return SABLOCK_ERR_INVALID_ARG;
    const Geo& g = pl.geo;
    const float c2 = (float)(1.4426950408889634 / sqrt((double)g.D));
    ScoreBufs sb;
    sb.part = at<float2>(ws, pl.o_part);
    sb.lse2 = at<float>(ws, pl.o_lse);
    sb.n_chunks = pl.n_chunks;
    int* status = at<int>(ws, pl.o_status);
    const Strides ks = k_strides(p, g.total_tokens);
    // Single-sweep mode (Sec. 4.1: the pass follows a prefill whose attention kernel keeps the
    // log of Eq. 2's normaliser per query row): no pass over K for the row statistics.
    const bool have_lse = p->row_lse != nullptr;
    float* neg_lse2 = at<float>(ws, pl.o_neg_lse);
    if (have_lse) {
        if (reinterpret_cast<uintptr_t>(p->row_lse) & 3) return SABLOCK_ERR_INVALID_ARG;
        const size_t n = (size_t)pl.n_prob * g.H * g.window;
        lse_import_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(p->row_lse, sb.lse2, neg_lse2, n);
        SAB_TRY(check_launch());
    }
    if (pl.use_tc) {
        CUtensorMap tmQ, tmK;
        SAB_TRY(make_tensor_maps(pl, p, q, k, &tmQ, &tmK));
        // Persistent two-sweep kernel: groups of CTAs each walk their share of the problems.
        const int tiles_max = (pl.max_L + kTcTile - 1) / kTcTile;
        const int min_cpp = (tiles_max + kFuMaxTilesPerCta - 1) / kFuMaxTilesPerCta;
        const int n_cta = pl.use_fused ? fused_cta_limit() : 0;
        if (pl.use_fused && n_cta >= min_cpp && (long long)g.n_layers * g.total_tokens < 0x7fffffffLL) {
            // A CTA holds at most kFuMaxTilesPerCta token tiles of a problem, so a problem needs a
            // group of ceil(tiles / 7) CTAs; a group that is larger than that leaves its CTAs with
            // one or two tiles per (problem, KV head) and the hand-over between phases dominates.
            // The sequences of the call are therefore sorted into classes by the group size they need
            // (powers of two up to 64, then whatever the longest needs) and every class gets a launch
            // of its own.  Sequences that are returned unchanged need no scores.
            int cls_of[kMaxSeqs], cls_need[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            for (int i = 0; i < g.n_seqs; ++i) {
                const int L = g.cu[i + 1] - g.cu[i];
                cls_of[i] = -1;
                if (L <= g.n_out) continue;
                const int need = ((L + kTcTile - 1) / kTcTile + kFuMaxTilesPerCta - 1) / kFuMaxTilesPerCta;
                int c = 0;
                while (c < 7 && (1 << c) < need) ++c;               // 1, 2, 4, ..., 64, then the rest
                cls_of[i] = c;
                if (need > cls_need[c]) cls_need[c] = need;
            }
            FusedArgs fa;
            fa.c2 = c2; fa.eps = p->eps;
            fa.part = at<float2>(ws, pl.o_fpart);
            fa.lse2 = sb.lse2;
            fa.neg_lse2 = have_lse ? neg_lse2 : nullptr;
            fa.fixed_schedule = p->reproducible ? 1 : 0;
            fa.arrive = at<int>(ws, pl.o_arrive);
            fa.done = at<int>(ws, pl.o_done);
            fa.s_out = s; fa.e_out = e; fa.status = status;
            for (int c = 0; c < 8; ++c) {
                if (!cls_need[c]) continue;
                int n_sel = 0, cls_tiles = 0;
                for (int i = 0; i < g.n_seqs; ++i)
                    if (cls_of[i] == c) {
                        fa.sel[n_sel++] = (unsigned char)i;
                        const int t = (g.cu[i + 1] - g.cu[i] + kTcTile - 1) / kTcTile;
                        if (t > cls_tiles) cls_tiles = t;
                    }
                fa.n_sel = n_sel;
                fa.n_prob = g.n_layers * n_sel;
                int groups = n_cta / cls_need[c];
                if (groups > fa.n_prob) groups = fa.n_prob;
                int cpp = n_cta / groups;
                if (cpp > cls_tiles) cpp = cls_tiles;
                fa.cpp = cpp; fa.n_groups = groups;
                Geo geo = g;
                void* args[] = {&tmQ, &tmK, &geo, &fa};
                const cudaError_t err = cudaLaunchCooperativeKernel((const void*)score_fused_tc, dim3(groups * cpp),
                                                                    dim3(kFuThreads), args, kFuSmemBytes, stream);
                if (err != cudaSuccess) {
                    cudaGetLastError();
                    return note_cuda_error(err, "cooperative launch of the score kernel");
                }
                ++t_launches;
            }
            prof_mark(1, stream);
            prof_mark(2, stream);
            return SABLOCK_OK;
        }
        if (p->score_impl == SABLOCK_SCORE_FUSED) return SABLOCK_ERR_UNSUPPORTED;
        constexpr int NST1 = 2;
        const int n_atoms = g.D / 64;
        const int smem1 = 1024 + (1 + NST1) * n_atoms * kAtomBytes;
        auto k1 = score_p1_tc<NST1>;
        if (cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, smem1) != cudaSuccess)
            return SABLOCK_ERR_CUDA;
        dim3 grid1(pl.n_chunks, g.Hkv, pl.n_prob);
        if (!have_lse) {
            k1<<<grid1, kTcThreads, smem1, stream>>>(tmQ, tmK, g, c2, sb, pl.tpc1, status);
            SAB_TRY(check_launch());
        }
        prof_mark(1, stream);
        if (!have_lse) {
            lse_merge_tc<<<dim3(g.Hkv, pl.n_prob), 128, 0, stream>>>(g, sb, pl.tpc1);
            SAB_TRY(check_launch());
        }
        prof_mark(2, stream);
        switch (g.window) {
            case 8: return launch_p2_tc<8>(pl, tmQ, tmK, c2, p->eps, sb, s, e, status, stream);
            case 16: return launch_p2_tc<16>(pl, tmQ, tmK, c2, p->eps, sb, s, e, status, stream);
            case 32: return launch_p2_tc<32>(pl, tmQ, tmK, c2, p->eps, sb, s, e, status, stream);
            default: return SABLOCK_ERR_UNSUPPORTED;
        }
    }
    const int smem1 = (g.window * g.D + 2 * (kSimtThreads / 32) * g.window) * (int)sizeof(float);
    const int smem2 = (kSimtWChunk * g.D + kSimtWChunk) * (int)sizeof(float);
    dim3 grid1(pl.n_chunks, g.H, pl.n_prob);
    dim3 grid2((pl.max_L + kSimtThreads - 1) / kSimtThreads, pl.n_prob);
    dim3 gridm((g.H * g.window + 127) / 128, pl.n_prob);
    if (p->dtype == SABLOCK_BF16) {
        auto k1 = score_p1_simt<__nv_bfloat16>;
        if (cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, smem1) != cudaSuccess)
            return SABLOCK_ERR_CUDA;
        if (!have_lse) {
            k1<<<grid1, kSimtThreads, smem1, stream>>>(g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, ks.tok, ks.head,
                                                       ks.layer, c2, sb);
            SAB_TRY(check_launch());
        }
        prof_mark(1, stream);
        if (!have_lse) {
            lse_merge_simt<<<gridm, 128, 0, stream>>>(g, sb);
            SAB_TRY(check_launch());
        }
        prof_mark(2, stream);
        score_p2_simt<__nv_bfloat16><<<grid2, kSimtThreads, smem2, stream>>>(
            g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, ks.tok, ks.head, ks.layer, c2, p->eps, sb, s, e);
    } else {
        auto k1 = score_p1_simt<float>;
        if (cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, smem1) != cudaSuccess)
            return SABLOCK_ERR_CUDA;
        if (!have_lse) {
            k1<<<grid1, kSimtThreads, smem1, stream>>>(g, (const float*)q, (const float*)k, ks.tok, ks.head, ks.layer, c2, sb);
            SAB_TRY(check_launch());
        }
        prof_mark(1, stream);
        if (!have_lse) {
            lse_merge_simt<<<gridm, 128, 0, stream>>>(g, sb);
            SAB_TRY(check_launch());
        }
        prof_mark(2, stream);
        score_p2_simt<float><<<grid2, kSimtThreads, smem2, stream>>>(g, (const float*)q, (const float*)k, ks.tok,
                                                                     ks.head, ks.layer, c2, p->eps, sb, s, e);
    }
    return check_launch();
}

// Stage 3 (with optional pooling first): s_raw -> s (pooled) -> s_refined.
#ifndef SABLOCK_SEG_GRID_PER_2K
#define SABLOCK_SEG_GRID_PER_2K 8
#endif
constexpr int kSegGridPer2K = SABLOCK_SEG_GRID_PER_2K;   // CTAs of the per-segment kernels per 2048 tokens of a sequence
constexpr int kSegGridMax = 32 * kSegGridPer2K;

sablock_status_t run_refine(const Plan& pl, const sablock_params_t* p, const float* s_raw, float* s, const float* e,
                            const int* seg_start, const int* n_seg, float* s_ref, float* stats, int stats_stride,
                            cudaStream_t stream)
{
    const int gx = (int)fmin(32.0, fmax(1.0, (double)((pl.max_L + 2047) / 2048)));
    if (p->pool_kernel > 1) {
        pool_kernel<<<dim3(gx * 4, pl.n_prob), 256, 0, stream>>>(pl.geo, s_raw, s, p->pool_kernel, p->pool_mode);
        SAB_TRY(check_launch());
    }
    // one warp per segment, a few dependent loads each: the kernel is latency-bound, so it gets
    // enough warps to keep every SM's warp slots full (about ten segments per warp)
    const int gr = (int)fmin((double)kSegGridMax, fmax(1.0, (double)((pl.max_L + 2047) / 2048) * kSegGridPer2K));
    refine_kernel<<<dim3(gr, pl.n_prob), 256, 0, stream>>>(pl.geo, s, e, seg_start, n_seg, p->alpha, p->eta, s_ref,
                                                           stats, stats_stride);
    return check_launch();
}

sablock_status_t check_candidates(const int* cand, int n, Cands* out)
{
    if (!cand || n < 1 || n > kMaxCand || cand[0] != 1) return SABLOCK_ERR_INVALID_ARG;
    for (int i = 1; i < n; ++i)
        if (cand[i] <= cand[i - 1]) return SABLOCK_ERR_INVALID_ARG;
    out->n = n;
    for (int i = 0; i < n; ++i) out->g[i] = cand[i];
    return SABLOCK_OK;
}

// Stage 4 + index list.
sablock_status_t run_select(const Plan& pl, const sablock_params_t* p, const float* s_ref, const int* seg_start,
                            const int* n_seg, const Cands& cands, int* out_idx, int* out_n_keep, int* seg_g,
                            int* seg_b, int seg_stride, void* ws, cudaStream_t stream)
{
    const Geo& g = pl.geo;
    unsigned* thr = at<unsigned>(ws, pl.o_thr);
    int* cut = at<int>(ws, pl.o_cut);
    {
        // Several CTAs per problem when the problems are few and long; they wait for one another,
        // hence the cooperative launch (all CTAs co-resident or an error).
        int ctas = 1;
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) {
            // all CTAs of the launch must be co-resident: as many per SM as the kernel's occupancy allows
            int per_sm = 1;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, topb_kernel, kTopThreads, 0) != cudaSuccess || per_sm < 1)
                per_sm = 1;
            ctas = sms * per_sm / pl.n_prob;
            const int by_len = (pl.max_L + 4 * kTopThreads - 1) / (4 * kTopThreads);      // at least four rounds each
            if (ctas > by_len) ctas = by_len;
            if (ctas > kTopMaxCtas) ctas = kTopMaxCtas;
            if (ctas < 1) ctas = 1;
        }
        TopScratch* tsc = at<TopScratch>(ws, pl.o_top);
        int* status = at<int>(ws, pl.o_status);
        if (ctas > 1) {
            Geo geo = g;
            const float* sr = s_ref;
            void* args[] = {&geo, &sr, &thr, &cut, &tsc, &status};
            const cudaError_t err =
                cudaLaunchCooperativeKernel((const void*)topb_kernel, dim3(ctas, pl.n_prob), dim3(kTopThreads), args, 0, stream);
            if (err != cudaSuccess) {
                cudaGetLastError();
                return note_cuda_error(err, "cooperative launch of the top-B kernel");
            }
            ++t_launches;
        } else {
            topb_kernel<<<dim3(1, pl.n_prob), kTopThreads, 0, stream>>>(g, s_ref, thr, cut, tsc, status);
            SAB_TRY(check_launch());
        }
    }
    prof_mark(5, stream);
    SearchOut so;
    so.keep = at<unsigned>(ws, pl.o_keep);
    so.keep_words = pl.keep_words;
    so.seg_g = seg_g; so.seg_b = seg_b; so.seg_stride = seg_stride;
    so.long_list = at<int>(ws, pl.o_long_list);
    so.long_count = at<int>(ws, pl.o_long_count);
    so.long_cap = pl.long_cap;
    const int gx = (int)fmin((double)kSegGridMax, fmax(1.0, (double)((pl.max_L + 2047) / 2048) * kSegGridPer2K));
    search_kernel<<<dim3(gx, pl.n_prob), kSearchWarps * 32, 0, stream>>>(g, cands, s_ref, seg_start, n_seg, thr, cut,
                                                                        p->tau, so);
    SAB_TRY(check_launch());
    search_long_kernel<<<dim3(8, pl.n_prob), kLongThreads, 0, stream>>>(g, cands, s_ref, seg_start, thr, cut, p->tau, so,
                                                                       at<double>(ws, pl.o_phi));
    SAB_TRY(check_launch());
    prof_mark(6, stream);
    index_kernel<<<pl.n_prob, kIdxThreads, 0, stream>>>(g, so.keep, pl.keep_words, out_idx, out_n_keep,
                                                        at<int>(ws, pl.o_status));
    return check_launch();
}

sablock_status_t run_compact(const Geo& g, int n_prob, const sablock_params_t* p, const void* k, const void* v,
                             const int* out_idx, const int* out_n_keep, int n_keep_fixed, void* out_k, void* out_v,
                             cudaStream_t stream)
{
    if (!k || !v || !out_idx || !out_k || !out_v) return SABLOCK_ERR_INVALID_ARG;
    const int es = elem_size(p);
    const Strides ks = k_strides(p, g.total_tokens), vs = v_strides(p, g.total_tokens);
    CompactArgs c;
    c.k = (const char*)k; c.v = (const char*)v; c.out_k = (char*)out_k; c.out_v = (char*)out_v;
    c.k_tok = ks.tok * es; c.k_head = ks.head * es; c.k_layer = ks.layer * es;
    c.v_tok = vs.tok * es; c.v_head = vs.head * es; c.v_layer = vs.layer * es;
    c.head_bytes = g.D * es;
    c.rows_per_cta = (long long)g.n_out * n_prob >= 16384 ? 8 : 4;     // larger CTAs once there are thousands of them
    const long long all[] = {c.k_tok, c.k_head, c.k_layer, c.v_tok, c.v_head, c.v_layer};
    for (long long x : all)
        if (x % 16) return SABLOCK_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(out_k) |
         reinterpret_cast<uintptr_t>(out_v)) & 15)
        return SABLOCK_ERR_UNSUPPORTED;
    dim3 grid((g.n_out + c.rows_per_cta - 1) / c.rows_per_cta, n_prob, 2);
    compact_kernel<<<grid, 256, 0, stream>>>(g, c, out_idx, out_n_keep, n_keep_fixed);
    return check_launch();
}

// ---- decoding over a cache: launch plan ----------------------------------------------------
struct DecodePlan { int n_splits, rows_per_split; size_t bytes; };

sablock_status_t decode_plan(const sablock_params_t* p, int n_prob, int n_rows, DecodePlan* dp)
{
    SAB_TRY(validate_params(p));
    if (n_prob < 1 || n_rows < 1) return SABLOCK_ERR_INVALID_ARG;
    const int G = p->n_q_heads / p->n_kv_heads;
    const int row_bytes = p->head_dim * elem_size(p);
    if ((G != 1 && G != 2 && G != 4) || p->head_dim > kDecMaxD || (row_bytes != 128 && row_bytes != 256 && row_bytes != 512))
        return SABLOCK_ERR_UNSUPPORTED;
    // Row splits: at least 256 rows each, and no more CTAs than two waves of the device (two CTAs
    // per SM are resident): the merge that follows reads one partial result per split.
    int splits = (n_rows + kDecThreads - 1) / kDecThreads;
    const long long ctas_wanted = 4LL * sm_count();
    const long long per_split = (long long)p->n_kv_heads * n_prob;
    const int cap = (int)fmax(1.0, (double)(ctas_wanted / per_split));
    if (splits > cap) splits = cap;
    if (splits > kDecMaxSplits) splits = kDecMaxSplits;
    dp->n_splits = splits;
    dp->rows_per_split = (n_rows + splits - 1) / splits;
    dp->bytes = align_up(sizeof(float) * (size_t)n_prob * p->n_q_heads * splits * (p->head_dim + 2));
    return SABLOCK_OK;
}

template <typename T, int D>
sablock_status_t launch_decode_d(const DecodeArgs& a, int G, dim3 grid, cudaStream_t st)
{
    void (*kern)(DecodeArgs) = nullptr;
    switch (G) {
        case 1: kern = decode_partial_kernel<T, 1, D>; break;
        case 2: kern = decode_partial_kernel<T, 2, D>; break;
        case 4: kern = decode_partial_kernel<T, 4, D>; break;
        default: return SABLOCK_ERR_UNSUPPORTED;
    }
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecSmemBytes) != cudaSuccess)
        return note_cuda_error(cudaGetLastError(), "shared memory of the decode kernel");
    kern<<<grid, kDecThreads, kDecSmemBytes, st>>>(a);
    return check_launch();
}

// head_dim * element size is 128, 256 or 512 bytes (checked by decode_plan)
sablock_status_t launch_decode(const DecodeArgs& a, bool bf16, int G, dim3 grid, cudaStream_t st)
{
    if (bf16) {
        switch (a.D) {
            case 64: return launch_decode_d<__nv_bfloat16, 64>(a, G, grid, st);
            case 128: return launch_decode_d<__nv_bfloat16, 128>(a, G, grid, st);
            case 256: return launch_decode_d<__nv_bfloat16, 256>(a, G, grid, st);
        }
    } else {
        switch (a.D) {
            case 32: return launch_decode_d<float, 32>(a, G, grid, st);
            case 64: return launch_decode_d<float, 64>(a, G, grid, st);
            case 128: return launch_decode_d<float, 128>(a, G, grid, st);
        }
    }
    return SABLOCK_ERR_UNSUPPORTED;
}

int rows_out(const sablock_params_t* p, int budget) { return p->budget_includes_window ? budget : budget + p->window; }

}  // namespace

// ---------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------
extern "C" {

void sablock_params_default(sablock_params_t* p)
{
    if (!p) return;
    memset(p, 0, sizeof(*p));
    p->dtype = SABLOCK_BF16;
    p->alpha = 0.9f; p->eta = 1.0f; p->eps = 1e-6f; p->tau = 0.85f;     // Sec. 4.1, implementation details
    p->pool_kernel = 1; p->pool_mode = 0;
    p->budget_includes_window = 1;
    p->score_impl = SABLOCK_SCORE_AUTO;
}

const char* sablock_last_cuda_error(void) { return t_cuda_error; }

const char* sablock_status_string(sablock_status_t st)
{
    switch (st) {
        case SABLOCK_OK: return "ok";
        case SABLOCK_ERR_INVALID_ARG: return "invalid argument";
        case SABLOCK_ERR_UNSUPPORTED: return "unsupported shape, dtype or alignment";
        case SABLOCK_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case SABLOCK_ERR_CUDA: return "CUDA runtime or driver error";
        case SABLOCK_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case SABLOCK_ERR_INTERNAL: return "internal consistency check failed on the device";
    }
    return "unknown status";
}

int sablock_version(void) { return 100; }

size_t sablock_params_sizeof(void) { return sizeof(sablock_params_t); }

int sablock_last_launch_count(void) { return t_launches; }

sablock_status_t sablock_profile_enable(int slots)
{
    if (slots < 0 || slots > SABLOCK_PROFILE_MAX_SLOTS) return SABLOCK_ERR_INVALID_ARG;
    if (!t_prof) {
        if (slots == 0) return SABLOCK_OK;
        t_prof = new ProfState();
    }
    t_prof->slots = slots;
    t_prof->next = 0;
    t_prof->cur = -1;
    for (int i = 0; i < SABLOCK_PROFILE_MAX_SLOTS; ++i) t_prof->used[i] = false;
    return SABLOCK_OK;
}

int sablock_profile_read(int slot, float* ms_out, int max_n)
{
    if (!t_prof || slot < 0 || slot >= SABLOCK_PROFILE_MAX_SLOTS || !t_prof->used[slot] || !ms_out) return 0;
    ProfState& ps = *t_prof;
    if (cudaEventSynchronize(ps.ev[slot][kProfStages]) != cudaSuccess) return 0;
    int n = max_n < kProfStages ? max_n : kProfStages;
    for (int i = 0; i < n; ++i)
        if (cudaEventElapsedTime(&ms_out[i], ps.ev[slot][i], ps.ev[slot][i + 1]) != cudaSuccess) ms_out[i] = -1.f;
    return n;
}

const char* sablock_profile_stage_name(int i) { return (i >= 0 && i < kProfStages) ? kProfNames[i] : ""; }

size_t sablock_workspace_bytes(const sablock_params_t* p, long long total_tokens, int max_L, int n_seqs, int n_layers)
{
    Plan pl;
    if (n_seqs < 1 || n_seqs > kMaxSeqs) return 0;
    int cu[kMaxSeqs + 1];
    // Offsets depend on totals only, not on where the sequence boundaries fall.
    for (int i = 0; i <= n_seqs; ++i) cu[i] = 0;
    cu[n_seqs] = (int)total_tokens;
    if (make_plan(p, n_layers, n_seqs, cu, total_tokens, max_L, p ? p->window + 1 : 1, &pl) != SABLOCK_OK) return 0;
    return pl.total;
}

sablock_status_t sablock_workspace_region(const sablock_params_t* p, long long total_tokens, int max_L, int n_seqs,
                                          int n_layers, const char* name, size_t* offset, size_t* bytes)
{
    if (!name || !offset || !bytes || n_seqs < 1 || n_seqs > kMaxSeqs) return SABLOCK_ERR_INVALID_ARG;
    Plan pl;
    int cu[kMaxSeqs + 1];
    for (int i = 0; i <= n_seqs; ++i) cu[i] = 0;
    cu[n_seqs] = (int)total_tokens;
    SAB_TRY(make_plan(p, n_layers, n_seqs, cu, total_tokens, max_L, p->window + 1, &pl));
    const size_t ntok = (size_t)n_layers * total_tokens;
    struct { const char* n; size_t off, sz; } tab[] = {
        {"s", pl.o_s, sizeof(float) * ntok},           {"e", pl.o_e, sizeof(float) * ntok},
        {"s_refined", pl.o_sr, sizeof(float) * ntok},  {"seg_id", pl.o_seg_id, sizeof(int) * (size_t)total_tokens},
        {"seg_start", pl.o_seg_start, sizeof(int) * (size_t)(total_tokens + n_seqs)},
        {"n_seg", pl.o_n_seg, sizeof(int) * (size_t)n_seqs},
    };
    for (auto& t : tab)
        if (!strcmp(t.n, name)) { *offset = t.off; *bytes = t.sz; return SABLOCK_OK; }
    return SABLOCK_ERR_INVALID_ARG;
}

sablock_status_t sablock_read_status(const void* ws, sablock_stream_t stream, int* raw)
{
    if (!ws) return SABLOCK_ERR_INVALID_ARG;
    int word = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SABLOCK_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SABLOCK_ERR_CUDA;
    if (raw) *raw = word;
    if (word & kStatTimeout) return SABLOCK_ERR_TIMEOUT;
    if (word & kStatInternal) return SABLOCK_ERR_INTERNAL;
    return SABLOCK_OK;
}

sablock_status_t sablock_read_status_detail(const void* ws, sablock_stream_t stream, int* raw2)
{
    if (!ws || !raw2) return SABLOCK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(raw2, ws, 2 * sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SABLOCK_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SABLOCK_ERR_CUDA;
    if (raw2[0] & kStatTimeout) return SABLOCK_ERR_TIMEOUT;
    if (raw2[0] & kStatInternal) return SABLOCK_ERR_INTERNAL;
    return SABLOCK_OK;
}

#ifdef SABLOCK_TEST_HOOKS
// Test builds only: sets the word that makes one producer withhold its post (see common.cuh).
int sablock_test_set_hooks(int hooks)
{
    return (int)cudaMemcpyToSymbol(sab::g_test_hooks, &hooks, sizeof(int));
}
#endif

sablock_status_t sablock_segment(const sablock_params_t* p, const int* token_ids, int L, int* seg_id, int* seg_start,
                                 int* n_seg, void* ws, size_t ws_bytes, sablock_stream_t stream)
{
    t_launches = 0;
    if (!p || L <= p->window) return SABLOCK_ERR_INVALID_ARG;
    Plan pl;
    SAB_TRY(make_plan(p, 1, 1, nullptr, L, L, p->window + 1, &pl));
    if (!ws || ws_bytes < pl.total) return SABLOCK_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SAB_TRY(zero_control(pl, ws, st));
    return run_segment(pl, p, token_ids, seg_id, seg_start, n_seg, ws, st);
}

// ---- segmentation without a workspace ---------------------------------------------------
// Scratch of sablock_segment_static: one look-back word per 2048-token tile, then the ticket
// counter and a private status word.  In host code this name is only a handle for the symbol
// look-up below; the kernel gets the device address from cudaGetSymbolAddress.
constexpr int kStaticSegTiles = SABLOCK_SEGMENT_STATIC_MAX_T / kSegTile;
static __device__ __align__(256) unsigned long long g_segment_scratch[kStaticSegTiles + 32];

sablock_status_t sablock_segment_static(const sablock_params_t* p, const int* token_ids, int L, int* seg_id,
                                        int* seg_start, int* n_seg, int* status, sablock_stream_t stream)
{
    t_launches = 0;
    if (!p || L <= p->window) return SABLOCK_ERR_INVALID_ARG;
    SAB_TRY(validate_params(p));
    if (!token_ids || !seg_id || !seg_start || !n_seg || !p->delim_bitmap || p->vocab_size <= 0)
        return SABLOCK_ERR_INVALID_ARG;
    const long long T = (long long)L - p->window;
    if (T > SABLOCK_SEGMENT_STATIC_MAX_T) return SABLOCK_ERR_UNSUPPORTED;
    // device address of the static array, looked up once per device with that device current
    static unsigned long long* addr[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SABLOCK_ERR_CUDA;
    if (!addr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_segment_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return SABLOCK_ERR_CUDA;
        }
        addr[dev] = static_cast<unsigned long long*>(ptr);
    }
    unsigned long long* scratch = addr[dev];
    const int n_tiles = (int)((T + kSegTile - 1) / kSegTile);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps the previous call's contents: tile states, ticket and private status restart at zero
    if (cudaMemsetAsync(scratch, 0, sizeof(unsigned long long) * (size_t)n_tiles, st) != cudaSuccess ||
        cudaMemsetAsync(scratch + kStaticSegTiles, 0, 2 * sizeof(unsigned long long), st) != cudaSuccess)
        return SABLOCK_ERR_CUDA;
    int* ticket = reinterpret_cast<int*>(scratch + kStaticSegTiles);
    int* own_status = reinterpret_cast<int*>(scratch + kStaticSegTiles + 1);
    Geo g;
    memset(&g, 0, sizeof(g));
    g.n_layers = g.n_seqs = 1; g.total_tokens = L; g.window = p->window;
    g.H = p->n_q_heads; g.Hkv = p->n_kv_heads; g.D = p->head_dim; g.G = g.H / g.Hkv;
    g.cu[0] = 0; g.cu[1] = L;
    segment_kernel<<<dim3(n_tiles, 1), kSegThreads, 0, st>>>(g, token_ids, p->delim_bitmap, p->vocab_size, seg_id, seg_start,
                                                             n_seg, scratch, ticket, n_tiles, status ? status : own_status,
                                                             nullptr);
    return check_launch();
}

sablock_status_t sablock_score(const sablock_params_t* p, const void* q_win, const void* k, int L, const int* seg_start,
                               const int* n_seg, float* s, float* e, float* s_refined, float* seg_stats, void* ws,
                               size_t ws_bytes, sablock_stream_t stream)
{
    t_launches = 0;
    if (!p || L <= p->window || !seg_start || !n_seg || !s || !s_refined) return SABLOCK_ERR_INVALID_ARG;
    Plan pl;
    // no budget here: "output rows" = the window alone, so that no sequence with a compressible
    // token (L > W) counts as one that is returned unchanged
    SAB_TRY(make_plan(p, 1, 1, nullptr, L, L, p->window, &pl));
    if (!ws || ws_bytes < pl.total) return SABLOCK_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SAB_TRY(zero_control(pl, ws, st));
    float* e_buf = e ? e : at<float>(ws, pl.o_e);
    float* s_raw = p->pool_kernel > 1 ? at<float>(ws, pl.o_s_raw) : s;
    SAB_TRY(run_score(pl, p, q_win, k, s_raw, e_buf, ws, st));
    return run_refine(pl, p, s_raw, s, e_buf, seg_start, n_seg, s_refined, seg_stats, L - p->window, st);
}

sablock_status_t sablock_select(const sablock_params_t* p, const float* s_refined, int L, const int* seg_start,
                                const int* n_seg, int budget, const int* block_candidates, int n_candidates,
                                int* out_idx, int* out_seg_block, int* out_seg_budget, void* ws, size_t ws_bytes,
                                sablock_stream_t stream)
{
    t_launches = 0;
    if (!p || L < 1 || !s_refined || !seg_start || !n_seg || !out_idx) return SABLOCK_ERR_INVALID_ARG;
    if (budget <= (p->budget_includes_window ? p->window : 0)) return SABLOCK_ERR_INVALID_ARG;
    Cands cands;
    SAB_TRY(check_candidates(block_candidates, n_candidates, &cands));
    Plan pl;
    SAB_TRY(make_plan(p, 1, 1, nullptr, L, L, rows_out(p, budget), &pl));
    if (!ws || ws_bytes < pl.total) return SABLOCK_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SAB_TRY(zero_control(pl, ws, st));
    // the retained count is written to workspace (n_seg slot is free here)
    return run_select(pl, p, s_refined, seg_start, n_seg, cands, out_idx, at<int>(ws, pl.o_n_seg), out_seg_block,
                      out_seg_budget, L > p->window ? L - p->window : 1, ws, st);
}

sablock_status_t sablock_compact(const sablock_params_t* p, const void* k, const void* v, int L, const int* out_idx,
                                 int n_keep, void* out_k, void* out_v, sablock_stream_t stream)
{
    t_launches = 0;
    if (!p || L < 1 || n_keep < 1 || n_keep > L) return SABLOCK_ERR_INVALID_ARG;
    SAB_TRY(validate_params(p));
    Geo g;
    memset(&g, 0, sizeof(g));
    g.n_layers = g.n_seqs = 1; g.total_tokens = L; g.window = p->window;
    g.H = p->n_q_heads; g.Hkv = p->n_kv_heads; g.D = p->head_dim; g.G = g.H / g.Hkv;
    g.n_out = n_keep; g.B = n_keep - p->window;
    g.cu[0] = 0; g.cu[1] = L;
    return run_compact(g, 1, p, k, v, out_idx, nullptr, n_keep, out_k, out_v, static_cast<cudaStream_t>(stream));
}

sablock_status_t sablock_compress_layers(const sablock_params_t* p, int n_layers, int n_seqs, const void* q_win,
                                         const void* k, const void* v, const int* token_ids, const int* cu_seqlens,
                                         int budget, const int* block_candidates, int n_candidates, void* out_k,
                                         void* out_v, int* out_idx, int* out_n_keep, void* ws, size_t ws_bytes,
                                         sablock_stream_t stream)
{
    t_launches = 0;
    if (!p || !cu_seqlens || n_seqs < 1 || n_seqs > kMaxSeqs || n_layers < 1) return SABLOCK_ERR_INVALID_ARG;
    if (!q_win || !k || !v || !token_ids || !out_k || !out_v || !out_idx || !out_n_keep) return SABLOCK_ERR_INVALID_ARG;
    if (budget <= (p->budget_includes_window ? p->window : 0)) return SABLOCK_ERR_INVALID_ARG;
    if (cu_seqlens[0] != 0) return SABLOCK_ERR_INVALID_ARG;
    int max_L = 0;
    for (int i = 0; i < n_seqs; ++i) {
        const int L = cu_seqlens[i + 1] - cu_seqlens[i];
        if (L < 1) return SABLOCK_ERR_INVALID_ARG;
        if (L > max_L) max_L = L;
    }
    Cands cands;
    SAB_TRY(check_candidates(block_candidates, n_candidates, &cands));
    Plan pl;
    SAB_TRY(make_plan(p, n_layers, n_seqs, cu_seqlens, cu_seqlens[n_seqs], max_L, rows_out(p, budget), &pl));
    if (!ws || ws_bytes < pl.total) return SABLOCK_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    prof_begin_call(st);
    SAB_TRY(zero_control(pl, ws, st));
    int* seg_id = at<int>(ws, pl.o_seg_id);
    int* seg_start = at<int>(ws, pl.o_seg_start);
    int* n_seg = at<int>(ws, pl.o_n_seg);
    float* s = at<float>(ws, pl.o_s);
    float* e = at<float>(ws, pl.o_e);
    float* sr = at<float>(ws, pl.o_sr);
    float* s_raw = p->pool_kernel > 1 ? at<float>(ws, pl.o_s_raw) : s;
    SAB_TRY(run_segment(pl, p, token_ids, seg_id, seg_start, n_seg, ws, st));
    prof_mark(0, st);
    SAB_TRY(debug_sync(p, "stage segment", st));
    SAB_TRY(run_score(pl, p, q_win, k, s_raw, e, ws, st));
    prof_mark(3, st);
    SAB_TRY(debug_sync(p, "stage score", st));
    SAB_TRY(run_refine(pl, p, s_raw, s, e, seg_start, n_seg, sr, nullptr, 0, st));
    prof_mark(4, st);
    SAB_TRY(debug_sync(p, "stage refine", st));
    SAB_TRY(run_select(pl, p, sr, seg_start, n_seg, cands, out_idx, out_n_keep, nullptr, nullptr, 0, ws, st));
    prof_mark(7, st);
    SAB_TRY(debug_sync(p, "stage select", st));
    sablock_status_t rc = run_compact(pl.geo, pl.n_prob, p, k, v, out_idx, out_n_keep, 0, out_k, out_v, st);
    prof_mark(8, st);
    prof_end_call();
    if (rc == SABLOCK_OK) rc = debug_sync(p, "stage compact", st);
    return rc;
}

sablock_status_t sablock_compress(const sablock_params_t* p, const void* q_win, const void* k, const void* v,
                                  const int* token_ids, int L, int budget, const int* block_candidates,
                                  int n_candidates, void* out_k, void* out_v, int* out_idx, int* out_n_keep, void* ws,
                                  size_t ws_bytes, sablock_stream_t stream)
{
    if (L < 1) return SABLOCK_ERR_INVALID_ARG;
    const int cu[2] = {0, L};
    return sablock_compress_layers(p, 1, 1, q_win, k, v, token_ids, cu, budget, block_candidates, n_candidates, out_k,
                                   out_v, out_idx, out_n_keep, ws, ws_bytes, stream);
}

// ---- decoding over a cache ---------------------------------------------------------------
size_t sablock_decode_workspace_bytes(const sablock_params_t* p, int n_prob, int n_rows)
{
    DecodePlan dp;
    return decode_plan(p, n_prob, n_rows, &dp) == SABLOCK_OK ? dp.bytes : 0;
}

sablock_status_t sablock_decode_attention(const sablock_params_t* p, int n_prob, const void* q, const void* k_cache,
                                          const void* v_cache, int n_rows, const int* n_valid, float* out, float* lse,
                                          void* ws, size_t ws_bytes, sablock_stream_t stream)
{
    t_launches = 0;
    if (!p || !q || !k_cache || !v_cache || !out) return SABLOCK_ERR_INVALID_ARG;
    DecodePlan dp;
    SAB_TRY(decode_plan(p, n_prob, n_rows, &dp));
    if (!ws || ws_bytes < dp.bytes) return SABLOCK_ERR_WORKSPACE_TOO_SMALL;
    const int es = elem_size(p);
    DecodeArgs a;
    a.q = q; a.k = k_cache; a.v = v_cache;
    a.k_head = p->k_stride_head ? p->k_stride_head : p->head_dim;
    a.k_row = p->k_stride_token ? p->k_stride_token : (long long)p->n_kv_heads * p->head_dim;
    a.k_prob = p->k_stride_layer ? p->k_stride_layer : (long long)n_rows * a.k_row;
    a.v_head = p->v_stride_head ? p->v_stride_head : p->head_dim;
    a.v_row = p->v_stride_token ? p->v_stride_token : (long long)p->n_kv_heads * p->head_dim;
    a.v_prob = p->v_stride_layer ? p->v_stride_layer : (long long)n_rows * a.v_row;
    const long long strides[] = {a.k_head, a.k_row, a.k_prob, a.v_head, a.v_row, a.v_prob};
    for (long long x : strides)
        if ((x * es) % 16) return SABLOCK_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(k_cache) | reinterpret_cast<uintptr_t>(v_cache)) & 15) return SABLOCK_ERR_UNSUPPORTED;
    a.n_valid = n_valid;
    a.n_rows = n_rows; a.n_splits = dp.n_splits; a.rows_per_split = dp.rows_per_split;
    a.H = p->n_q_heads; a.Hkv = p->n_kv_heads; a.D = p->head_dim;
    a.c2 = (float)(1.4426950408889634 / sqrt((double)p->head_dim));
    a.part = static_cast<float*>(ws);
    a.out = out; a.lse = lse;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dim3 grid(dp.n_splits, p->n_kv_heads, n_prob);
    const int G = p->n_q_heads / p->n_kv_heads;
    SAB_TRY(launch_decode(a, p->dtype == SABLOCK_BF16, G, grid, st));
    const int mt = kDecMergeSlices * ((p->head_dim + 31) / 32 * 32);
    decode_merge_kernel<<<dim3(p->n_q_heads, n_prob), mt, 0, st>>>(a);
    return check_launch();
}

sablock_status_t sablock_compress_layers_host(const sablock_params_t* p, int n_layers, int n_seqs, const void* h_q_win,
                                              const void* h_k, const void* h_v, const int* h_token_ids,
                                              const int* cu_seqlens, int budget, const int* block_candidates,
                                              int n_candidates, void* h_out_k, void* h_out_v, int* h_out_idx,
                                              int* h_out_n_keep, void* dev_q_win, void* dev_k, void* dev_v,
                                              int* dev_token_ids, void* dev_out_k, void* dev_out_v, int* dev_out_idx,
                                              int* dev_out_n_keep, void* ws, size_t ws_bytes, sablock_stream_t stream)
{
    if (!p || !cu_seqlens || n_seqs < 1 || n_seqs > kMaxSeqs || n_layers < 1) return SABLOCK_ERR_INVALID_ARG;
    if (!h_q_win || !h_k || !h_v || !h_token_ids || !h_out_k || !h_out_v || !h_out_idx || !h_out_n_keep ||
        !dev_q_win || !dev_k || !dev_v || !dev_token_ids || !dev_out_k || !dev_out_v || !dev_out_idx || !dev_out_n_keep)
        return SABLOCK_ERR_INVALID_ARG;
    if (p->k_stride_token || p->k_stride_head || p->k_stride_layer || p->v_stride_token || p->v_stride_head ||
        p->v_stride_layer)
        return SABLOCK_ERR_UNSUPPORTED;            // host staging assumes contiguous tensors
    // Everything the copies below are sized from is checked first: nothing is enqueued on bad arguments.
    if (budget <= (p->budget_includes_window ? p->window : 0)) return SABLOCK_ERR_INVALID_ARG;
    if (cu_seqlens[0] != 0) return SABLOCK_ERR_INVALID_ARG;
    {
        int max_L = 0;
        for (int i = 0; i < n_seqs; ++i) {
            const int L = cu_seqlens[i + 1] - cu_seqlens[i];
            if (L < 1) return SABLOCK_ERR_INVALID_ARG;
            if (L > max_L) max_L = L;
        }
        Cands cands;
        SAB_TRY(check_candidates(block_candidates, n_candidates, &cands));
        Plan pl;
        SAB_TRY(make_plan(p, n_layers, n_seqs, cu_seqlens, cu_seqlens[n_seqs], max_L, rows_out(p, budget), &pl));
        if (!ws || ws_bytes < pl.total) return SABLOCK_ERR_WORKSPACE_TOO_SMALL;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t es = elem_size(p);
    const size_t total = (size_t)cu_seqlens[n_seqs];
    const size_t kv_bytes = (size_t)n_layers * total * p->n_kv_heads * p->head_dim * es;
    const size_t q_bytes = (size_t)n_layers * n_seqs * p->n_q_heads * p->window * p->head_dim * es;
    const int n_out = rows_out(p, budget);
    const size_t n_prob = (size_t)n_layers * n_seqs;
    const size_t okv_bytes = n_prob * n_out * p->n_kv_heads * p->head_dim * es;
    // The pass reads every key but only the retained rows of V.  If h_v is pinned (page-locked,
    // device-accessible) memory the gather reads those rows from it in place; otherwise V is staged
    // like the rest.
    const void* v_src = dev_v;
    {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, h_v) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer)
            v_src = attr.devicePointer;
        else
            cudaGetLastError();
    }
    if (cudaMemcpyAsync(dev_token_ids, h_token_ids, total * sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dev_q_win, h_q_win, q_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dev_k, h_k, kv_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        (v_src == dev_v && cudaMemcpyAsync(dev_v, h_v, kv_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess))
        return SABLOCK_ERR_CUDA;
    SAB_TRY(sablock_compress_layers(p, n_layers, n_seqs, dev_q_win, dev_k, v_src, dev_token_ids, cu_seqlens, budget,
                                    block_candidates, n_candidates, dev_out_k, dev_out_v, dev_out_idx, dev_out_n_keep,
                                    ws, ws_bytes, stream));
    if (cudaMemcpyAsync(h_out_k, dev_out_k, okv_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(h_out_v, dev_out_v, okv_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(h_out_idx, dev_out_idx, n_prob * n_out * sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(h_out_n_keep, dev_out_n_keep, n_prob * sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return SABLOCK_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? SABLOCK_OK : SABLOCK_ERR_CUDA;
}

}  // extern "C"
