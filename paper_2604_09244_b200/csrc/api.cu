// C-ABI layer: argument validation, host-side budget arithmetic, workspace and smoothed state,
// tensor-map construction, launch sequencing.  No stream synchronisation anywhere.
#include "common.cuh"

#include <cudaTypedefs.h>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>
#include <cstdio>

#include <nvtx3/nvToolsExt.h>

using namespace mvla;

namespace {
constexpr int kSets = 6;            // scratch sets = prune steps that may be in flight at once
#ifndef MVLA_TAIL_CTAS_PER_SM
#define MVLA_TAIL_CTAS_PER_SM 2
#endif
constexpr int kTailCtasPerSm = MVLA_TAIL_CTAS_PER_SM;   // grid of the selection + row copy kernel

// Tracing and logging, both on the host and off the device's path: every public call is an NVTX range (a profiler
// shows the call and, inside mvla_prune_step, its phases around the kernels they enqueue; without a profiler
// attached a range costs a few nanoseconds), and with MVLA_LOG=1 in the environment every call prints one line
// with its arguments and its result to stderr.
struct ApiRange {
    explicit ApiRange(const char* name) { nvtxRangePushA(name); }
    ~ApiRange() { nvtxRangePop(); }
    ApiRange(const ApiRange&) = delete;
    ApiRange& operator=(const ApiRange&) = delete;
};
// The phases of a step inside the call's range: mark() closes the phase before it.
struct PhaseRange {
    bool open = false;
    void mark(const char* name)
    {
        if (open) nvtxRangePop();
        nvtxRangePushA(name);
        open = true;
    }
    ~PhaseRange() { if (open) nvtxRangePop(); }
};
bool log_enabled()
{
    static const bool on = [] {
        const char* e = std::getenv("MVLA_LOG");
        return e && *e && *e != '0';
    }();
    return on;
}
}

struct mvla_ctx {
    mvla_config cfg;
    int n_slots;
    int max_vis;
    size_t elem;                 // bytes per element of hidden
    size_t qk_elem;              // bytes per element of q, k, v (1 for e4m3, else = elem)
    int hidden_dtype;            // MVLA_DTYPE_BF16 or MVLA_DTYPE_FP32
    bool use_umma;               // bf16 tensor-core salience path
    int kv_heads;                // key / value heads (== n_heads unless grouped)
    float* part;                 // [H][max_batch * max_vis] per-head partial scores
    int64_t part_stride;
    float* l1_ws;                // [kSets][max_batch * max_vis] feature norms, one set per step in flight
    float* ahat_state;           // [n_prune_points][n_slots][2][max_vis]: the copy step t reads and the one it writes
    float* mhat_state;           // [n_prune_points][n_slots][2][4]
    unsigned long long* acc64;   // [kSets][max_batch * max_vis] fixed-point score accumulators, zero between
                                 // calls; the sets rotate from step to step (a step's scoring may run beside
                                 // the selections of the steps before it)
    int32_t* tail_list;          // [kSets][rows_all] kept list as the copying CTAs read it (-1 between launches)
    unsigned int* tail_ticket;   // [kSets] ticket counters of the patch-by-patch tail (zero between launches)
    unsigned long long* patch_rec;   // [kSets][vis_all / 2][3] hand-over words of the patch-by-patch tail (all ones between launches)
    size_t rows_all;             // max_batch * (kHandWords + max_text + max_vis)
    int sm_count;                // multiprocessors of the device
    // reuse of the previous step's logits (cfg.logit_cache)
    float* lcache;               // [n_prune_points * n_slots][H][max_vis][cache_cols] raw dot products
    int cache_cols;              // round16(max_text)
    struct CacheSig { bool valid; int32_t n_txt, n_2d, n_3d; };
    std::vector<CacheSig> cache_sig;   // per (prune point, slot): does the cache hold the last step's logits, and of what shape
    int64_t tiles_computed, tiles_reused;
    cudaEvent_t stage_event;     // measurement aid: recorded between scoring and selection + copy (null: off)
    unsigned long long* stamps;  // measurement aid: device buffer [2][kStampSlots][2] of per-CTA time stamps (null: off)
    size_t vis_all;              // max_batch * max_vis
    // patch-by-patch path (cfg.patch_path): attention copy [H][max_text][vis_all], per-patch smoothed
    // indicators [n_prune_points][n_slots][max_patch][4], and the scratch between its kernels
    float* alpha_ws;             // [patch_sets] copies: steps in flight beside one another each have their own
    float* xhat_patch;
    float* patch_x_ws;           // [patch_sets][vis_all / 2 + 1][4]
    float* patch_attn_ws;        // [patch_sets][vis_all]
    int patch_sets;              // kSets when the attention copies fit a modest budget, else 1 (then no overlap)
    int32_t* nout_ws;            // [max_batch] kept rows, [max_batch] ready flags, [1] finished-CTA counter
    int max_patch;
    unsigned step_parity;        // index of the scratch set of the current step
    // Scoring and selection of a step whose inputs are promised stable run on the side stream of the
    // step's scratch set, beside the selection and row copy of the steps before; the row copy stays
    // on the caller's stream and waits for ev_sel of the step.
    cudaStream_t aux[kSets];                   // one per scratch set, so that consecutive steps do not serialise
    cudaEvent_t ev_fork, ev_sel[kSets];        // ev_sel[p]: after the selection that last used scratch set p
    cudaEvent_t ev_copy[kSets];                // ev_copy[p]: after the row copy of that same step
    bool sel_valid[kSets];
    // Buffers that the side-stream steps still possibly in flight write (selection outputs, copied rows),
    // one entry per scratch set.  A step whose side-stream work reads or writes any of them (its inputs,
    // its selection outputs) is ordered after everything enqueued on the caller's stream instead.
    struct Range { const char* lo; const char* hi; };
    Range hist[kSets][16];
    int n_hist[kSets];
    bool hist_unknown;                         // the stream ran other work of this context since: order after it
    // Smoothed states (prune point x slot) that the step last run on each scratch set reads and writes:
    // a later selection touching one of them waits for that selection, others need not.
    int32_t state_of[kSets][kMaxChunk];
    int n_state_of[kSets];
    unsigned long long sel_capture[kSets];         // capture sequence the event belongs to (0: none)
    std::vector<int32_t> t_host; // [n_prune_points][n_slots] steps absorbed so far
    int* status_host;            // mapped pinned word written by kernels whose bounded wait gave up
    int* status_dev;
    cudaError_t last_cuda;
    PFN_cuTensorMapEncodeTiled_v12000 encode;
    // tensor maps are cached per (pointer, rows)
    const void* tm_ptr[2];
    int64_t tm_rows[2];
    CUtensorMap tm[2];
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

inline int32_t rhu(double x) { return static_cast<int32_t>(std::floor(x + 0.5)); }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int32_t fail_cuda(mvla_ctx* ctx, cudaError_t e)
{
    ctx->last_cuda = e;
    return e == cudaErrorMemoryAllocation ? MVLA_ERR_OOM : MVLA_ERR_CUDA;
}

int32_t validate_samples(const mvla_ctx* ctx, int32_t batch, const mvla_sample* samples, int32_t mode,
                         int64_t rows)
{
    if (batch < 1 || !samples) return MVLA_ERR_INVALID_ARG;
    if (batch > ctx->cfg.max_batch) return MVLA_ERR_CAPACITY;
    if (mode != MVLA_MODE_FIXED && mode != MVLA_MODE_ADAPTIVE) return MVLA_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b) {
        const mvla_sample& s = samples[b];
        if (s.n_txt < 1 || s.n_2d < 0 || s.n_3d < 0 || s.n_2d + s.n_3d < 1 || s.seq_off < 0) return MVLA_ERR_INVALID_ARG;
        if (s.n_txt > ctx->cfg.max_text || s.n_2d > ctx->cfg.max_2d || s.n_3d > ctx->cfg.max_3d) return MVLA_ERR_CAPACITY;
        const int seq = s.n_txt + s.n_2d + s.n_3d;
        const int off[3] = {s.off_txt, s.off_2d, s.off_3d}, len[3] = {s.n_txt, s.n_2d, s.n_3d};
        for (int i = 0; i < 3; ++i) {
            if (off[i] < 0 || off[i] + len[i] > seq) return MVLA_ERR_INVALID_ARG;
            for (int j = i + 1; j < 3; ++j)
                if (len[i] > 0 && len[j] > 0 && off[i] < off[j] + len[j] && off[j] < off[i] + len[i])
                    return MVLA_ERR_INVALID_ARG;       // segments overlap
        }
        if (rows >= 0 && static_cast<int64_t>(s.seq_off) + seq > rows) return MVLA_ERR_INVALID_ARG;
        if (s.state_slot < 0 || s.state_slot >= ctx->n_slots) return MVLA_ERR_STATE;
        const double keeps[3] = {s.keep_2d, s.keep_3d, s.keep_total};
        for (double kq : keeps)
            if (!(kq >= 0.0) || !std::isfinite(kq)) return MVLA_ERR_INVALID_ARG;
    }
    return MVLA_OK;
}

// Everything about a call that the host can decide: layout offsets, budgets, state addressing,
// the smoothing weights of this action step.
struct Plan {
    std::vector<SampleDev> s;
    int32_t total_vis = 0;
    int32_t total_out = 0;
};

int32_t make_plan(mvla_ctx* ctx, int32_t prune_point, int32_t batch, const mvla_sample* samples, int32_t mode,
                  uint32_t flags, bool with_state, Plan* plan)
{
    plan->s.resize(batch);
    const mvla_config& c = ctx->cfg;
    if (with_state) {
        if (prune_point < 0 || prune_point >= c.n_prune_points) return MVLA_ERR_STATE;
        for (int b = 0; b < batch; ++b)
            for (int b2 = b + 1; b2 < batch; ++b2)
                if (samples[b].state_slot == samples[b2].state_slot) return MVLA_ERR_STATE;   // two writers of one state
    }
    int32_t vis_off = 0, out_off = 0, cap_off = 0;
    for (int b = 0; b < batch; ++b) {
        const mvla_sample& in = samples[b];
        SampleDev d;
        std::memset(&d, 0, sizeof d);
        d.seq_off = in.seq_off; d.off_txt = in.off_txt; d.n_txt = in.n_txt;
        d.off_2d = in.off_2d; d.n_2d = in.n_2d; d.off_3d = in.off_3d; d.n_3d = in.n_3d;
        const int nv = in.n_2d + in.n_3d;
        d.vis_off = vis_off;
        d.cap_off = cap_off;
        cap_off += kHandWords + in.n_txt + nv;
        vis_off += nv;
        d.k_2d_fixed = -1;
        d.cache_state = -1;
        d.tile_compute = 0xFFFFFFFFu;
        d.t = 1; d.update_state = 0; d.c_prev = 0.f; d.c_new = 1.f;
        if (with_state) {
            const int sidx = prune_point * ctx->n_slots + in.state_slot;
            const int t_prev = (flags & MVLA_FLAG_RESET_STATE) ? 0 : ctx->t_host[sidx];
            const int t = t_prev + 1;
            d.t = t;
            // two copies of every state: step t reads the one step t - 1 wrote, writes the other
            d.state_off = (sidx * 2 + (t_prev & 1)) * ctx->max_vis;
            d.state_off_w = (sidx * 2 + (t & 1)) * ctx->max_vis;
            d.mstate_off = sidx * 2 + (t_prev & 1);
            d.mstate_off_w = sidx * 2 + (t & 1);
            d.slot_index = sidx;
            d.update_state = (flags & MVLA_FLAG_NO_STATE_UPDATE) ? 0 : 1;
            if (t <= 1) { d.c_prev = 0.f; d.c_new = 1.f; }                                   // X^_1 = X_1
            else if (t < c.window_k) {                                                        // Eq. 8
                d.c_prev = static_cast<float>(static_cast<double>(t - 1) / t);
                d.c_new = static_cast<float>(1.0 / t);
            } else {                                                                          // Eq. 9
                d.c_prev = static_cast<float>(c.beta);
                d.c_new = static_cast<float>(1.0 - c.beta);
            }
            if (t == 1 && c.cold_start_full_keep) {                                           // Alg. 1 cold start
                d.budget = nv;
                d.k_2d_fixed = in.n_2d;
            } else if (mode == MVLA_MODE_FIXED) {
                const int k2 = std::min(in.n_2d, rhu(in.keep_2d * in.n_2d));
                const int k3 = std::min(in.n_3d, rhu(in.keep_3d * in.n_3d));
                d.budget = k2 + k3;
                d.k_2d_fixed = k2;
            } else {
                const int B = std::min(nv, rhu(in.keep_total * nv));
                d.budget = B;
                d.kmin_2d = std::min(static_cast<int>(std::ceil(c.floor_ratio * in.n_2d)),
                                     static_cast<int>(std::floor(static_cast<double>(B) * in.n_2d / nv)));
                d.kmin_3d = std::min(static_cast<int>(std::ceil(c.floor_ratio * in.n_3d)),
                                     static_cast<int>(std::floor(static_cast<double>(B) * in.n_3d / nv)));
            }
            d.n_out = in.n_txt + d.budget;
            d.out_off = out_off;
            out_off += d.n_out;
        }
        plan->s[b] = d;
    }
    plan->total_vis = vis_off;
    plan->total_out = out_off;
    return MVLA_OK;
}

void commit_steps(mvla_ctx* ctx, int32_t prune_point, const Plan& plan, const mvla_sample* samples)
{
    for (size_t b = 0; b < plan.s.size(); ++b)
        if (plan.s[b].update_state) ctx->t_host[prune_point * ctx->n_slots + samples[b].state_slot] = plan.s[b].t;
}

BatchDesc chunk_of(const Plan& plan, int first, int n)
{
    BatchDesc bd;
    std::memset(&bd, 0, sizeof bd);
    bd.n = n;
    for (int i = 0; i < n; ++i) bd.s[i] = plan.s[first + i];
    return bd;
}

int tiles_of(const SampleDev& s)
{
    return (s.n_2d + kKeyTile - 1) / kKeyTile + (s.n_3d + kKeyTile - 1) / kKeyTile;
}

// 3-D view (head_dim, heads, rows) of a token-major [rows, H, d] bf16 or e4m3 tensor; boxes of 128 bytes x 1 x
// `box_rows` land in shared memory as `box_rows` rows of 128 bytes with the 128-byte swizzle.
int32_t tensor_map(mvla_ctx* ctx, int which, const void* ptr, int64_t rows, int box_rows, const CUtensorMap** out)
{
    if (ctx->tm_ptr[which] == ptr && ctx->tm_rows[which] == rows) {
        *out = &ctx->tm[which];
        return MVLA_OK;
    }
    const mvla_config& c = ctx->cfg;
    const cuuint64_t heads = static_cast<cuuint64_t>(which == 1 ? ctx->kv_heads : c.n_heads);   // map 1 is the key tensor
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(c.head_dim), heads, static_cast<cuuint64_t>(rows)};
    const cuuint64_t es = static_cast<cuuint64_t>(ctx->qk_elem);
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(c.head_dim) * es, static_cast<cuuint64_t>(c.head_dim) * heads * es};
    cuuint32_t box[3] = {static_cast<cuuint32_t>(128 / es), 1, static_cast<cuuint32_t>(box_rows)};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapDataType dt = es == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult r = ctx->encode(&ctx->tm[which], dt, 3, const_cast<void*>(ptr), dims,
                                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->tm_ptr[which] = nullptr;
        return MVLA_ERR_CUDA;
    }
    ctx->tm_ptr[which] = ptr;
    ctx->tm_rows[which] = rows;
    *out = &ctx->tm[which];
    return MVLA_OK;
}

int32_t check_sticky(mvla_ctx* ctx)
{
    return (ctx->status_host && *reinterpret_cast<volatile int*>(ctx->status_host) != 0) ? MVLA_ERR_TIMEOUT : MVLA_OK;
}

// Salience of one chunk (+ L1 norms into `l1` when asked).  The per-head contributions land in
// ctx->part, or, when `want_acc64` and the register-resident tensor-core kernel covers the shape, in the
// fixed-point accumulators ctx->acc64 (*used_acc64 = true).
int32_t run_salience_chunk(mvla_ctx* ctx, const BatchDesc& bd, const void* q, const void* k, int64_t rows,
                           const void* hidden, float* l1, unsigned long long* acc64, bool* used_acc64,
                           bool free_running, cudaStream_t st, AlphaOut alpha = AlphaOut{nullptr, 0, 0},
                           int32_t* rearm = nullptr, bool norms_beside = false, unsigned long long* stamps = nullptr,
                           bool with_cache = false, unsigned long long* rearm_rec = nullptr)
{
    if (used_acc64) *used_acc64 = false;
    const mvla_config& c = ctx->cfg;
    int max_tiles = 1, max_txt = 1;
    for (int b = 0; b < bd.n; ++b) {
        max_tiles = std::max(max_tiles, tiles_of(bd.s[b]));
        max_txt = std::max(max_txt, bd.s[b].n_txt);
    }
    const int tiles_per_cta = (max_tiles + kMaxCluster - 1) / kMaxCluster;
    const int cluster = (max_tiles + tiles_per_cta - 1) / tiles_per_cta;
    const int npad = (max_txt + 15) / 16 * 16;
    const CUtensorMap *tq = nullptr, *tk = nullptr;
    if (ctx->use_umma) {
        int32_t r = tensor_map(ctx, 0, q, rows, 16, &tq);
        if (r != MVLA_OK) return r;
        r = tensor_map(ctx, 1, k, rows, kKeyTile, &tk);
        if (r != MVLA_OK) return r;
    }
    cudaError_t e;
    const bool fast = ctx->use_umma && fast_salience_supported(tiles_per_cta);
    // The norms do not depend on the scores: with `norms_beside` (fast kernel only) they are launched AFTER
    // the scoring kernel and run beside it instead of in front of it.
    norms_beside = norms_beside && fast;
    if (hidden && l1 && !norms_beside) {
        e = launch_l1norm(bd, ctx->hidden_dtype, c.d_model, hidden, l1, false, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    if (fast) {
        e = launch_salience_fast(bd, c.n_heads, c.n_heads / ctx->kv_heads, c.head_dim, static_cast<int>(ctx->qk_elem), tq, tk,
                                 tiles_per_cta, cluster, npad,
                                 alpha.ptr && !acc64 ? nullptr : ctx->part,     // the patch path reads the attention copy only
                                 ctx->part_stride, acc64, ctx->status_dev, free_running, alpha, rearm, rearm_rec, stamps,
                                 with_cache ? ctx->lcache : nullptr, ctx->max_vis, ctx->cache_cols, st);
        if (used_acc64) *used_acc64 = acc64 != nullptr;
    } else {
        e = launch_salience(bd, c.dtype, c.n_heads, c.n_heads / ctx->kv_heads, c.head_dim, q, k, tq, tk, ctx->use_umma, tiles_per_cta,
                            cluster, npad, ctx->part, ctx->part_stride, ctx->status_dev, alpha, st);
    }
    if (e == cudaErrorInvalidConfiguration) return MVLA_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    if (hidden && l1 && norms_beside) {
        e = launch_l1norm(bd, ctx->hidden_dtype, c.d_model, hidden, l1, true, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    return MVLA_OK;
}

mvla_ctx::Range range_of(const void* p, size_t bytes)
{
    const char* c = static_cast<const char*>(p);
    return {c, c ? c + bytes : c};
}

bool chunk_is_fast(const mvla_ctx* ctx, const BatchDesc& bd)
{
    int max_tiles = 1;
    for (int b = 0; b < bd.n; ++b) max_tiles = std::max(max_tiles, tiles_of(bd.s[b]));
    return ctx->use_umma && fast_salience_supported((max_tiles + kMaxCluster - 1) / kMaxCluster);
}

GateParams gate_params(const mvla_ctx* ctx, int32_t mode, bool has_l1)
{
    GateParams gp;
    gp.tau_2d = static_cast<float>(ctx->cfg.tau_2d);
    gp.tau_3d = static_cast<float>(ctx->cfg.tau_3d);
    gp.eps_3d = static_cast<float>(ctx->cfg.eps_3d);
    gp.adaptive = mode == MVLA_MODE_ADAPTIVE;
    gp.has_l1 = has_l1;
    return gp;
}

// A launch of the step failed after the scoring kernel was enqueued: the fixed-point accumulators of the
// chunk must not keep this step's sums (the selection that clears them will not run).
void clear_accumulators(unsigned long long* acc64, const BatchDesc& bd, cudaStream_t st)
{
    const SampleDev& first = bd.s[0];
    const SampleDev& last = bd.s[bd.n - 1];
    const size_t n = static_cast<size_t>(last.vis_off + last.n_2d + last.n_3d - first.vis_off);
    cudaMemsetAsync(acc64 + first.vis_off, 0, n * sizeof(unsigned long long), st);
}

// ---- overlap of neighbouring prune steps (MVLA_FLAG_INPUTS_STABLE) ----
// With stable inputs, scoring and selection of a step go to the side stream of the step's scratch set
// (`par`); only the row copy stays on the caller's stream.  What the side-stream work of step k must follow:
//   * selection and row copy of step k - kSets (same scratch set; the copy also frees that step's
//     output buffers, so at most kSets - 1 earlier copies can still be running);
//   * every selection of the kSets - 1 steps before that touches a smoothed state (prune point,
//     slot) this step touches: a state is updated in call order.  Steps on other slots -- independent
//     requests -- are not waited for;
//   * if it reads or writes a buffer that one of those kSets - 1 steps writes, or if the stream has
//     run other work of this context since: everything enqueued on the caller's stream so far.
// Events recorded under another stream capture cannot be waited on; then, too, the step starts
// after everything enqueued so far.
struct ForkPlan {
    bool ordered_after_all = false;
    unsigned dep_mask = 0;               // scratch sets whose selection event this step's selection waits for
    unsigned long long cap_id = 0;       // stream capture the events of this step belong to (0: none)
};

// `side`: buffers the side-stream work reads or writes, the first `n_side_written` of them written by it;
// `copied`: buffers the row copy writes.  Enqueues the wait that opens the side stream and records what the
// step writes and which states it touches.
int32_t plan_fork(mvla_ctx* ctx, cudaStream_t st, unsigned par, int32_t prune_point, int32_t batch,
                  const mvla_sample* samples, const mvla_ctx::Range* side, int n_side, int n_side_written,
                  const mvla_ctx::Range* copied, int n_copied, ForkPlan* fp)
{
    cudaStreamCaptureStatus cst = cudaStreamCaptureStatusNone;
    if (cudaStreamGetCaptureInfo(st, &cst, &fp->cap_id) != cudaSuccess) return fail_cuda(ctx, cudaGetLastError());
    if (cst != cudaStreamCaptureStatusActive) fp->cap_id = 0;
    bool clash = ctx->hist_unknown;
    for (unsigned s = 0; !clash && s < kSets; ++s) {
        if (s == par) continue;
        for (int i = 0; !clash && i < n_side; ++i)
            for (int j = 0; !clash && j < ctx->n_hist[s]; ++j)
                clash = side[i].lo && side[i].lo < ctx->hist[s][j].hi && ctx->hist[s][j].lo < side[i].hi;
    }
    // earlier selections still possibly in flight that touch a smoothed state this step touches: the
    // state is updated in call order, so this step's selection waits for the most recent one per
    // state (dep_mask; that one has in turn waited for those before it).  Steps older than
    // kSets - 1 calls are ordered through the row-copy event or the stream itself.
    const bool own_ok = ctx->sel_valid[par] && ctx->sel_capture[par] == fp->cap_id;
    bool stale = false;
    bool covered[kMaxChunk] = {};            // per sample of this step: most recent toucher of its state found
    for (unsigned back = 1; back < kSets; ++back) {          // most recent step first
        const unsigned s = (par + kSets - back) % kSets;
        bool hit = false;
        for (int b = 0; b < batch; ++b) {
            if (covered[b]) continue;        // an even later step touches it and has waited for this one
            const int32_t mine = prune_point * ctx->n_slots + samples[b].state_slot;
            for (int i = 0; i < ctx->n_state_of[s]; ++i)
                if (ctx->state_of[s][i] == mine) { covered[b] = hit = true; break; }
        }
        if (!hit) continue;
        if (ctx->sel_valid[s] && ctx->sel_capture[s] == fp->cap_id) fp->dep_mask |= 1u << s;
        else stale = true;                   // its event cannot be waited on from here
    }
    fp->ordered_after_all = clash || !own_ok || stale;
    cudaError_t e;
    if (fp->ordered_after_all) {
        e = cudaEventRecord(ctx->ev_fork, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->aux[par], ctx->ev_fork, 0);
        if (ctx->hist_unknown) {
            for (int& n : ctx->n_hist) n = 0;
            for (int& n : ctx->n_state_of) n = 0;
        }
    } else {
        e = cudaStreamWaitEvent(ctx->aux[par], ctx->ev_copy[par], 0);
    }
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    // remember what this step writes
    int m = 0;
    for (int i = 0; i < n_side_written; ++i) if (side[i].lo) ctx->hist[par][m++] = side[i];
    for (int i = 0; i < n_copied; ++i) if (copied[i].lo) ctx->hist[par][m++] = copied[i];
    ctx->n_hist[par] = m;
    ctx->hist_unknown = false;
    for (int b = 0; b < batch; ++b) ctx->state_of[par][b] = prune_point * ctx->n_slots + samples[b].state_slot;
    ctx->n_state_of[par] = batch;
    return MVLA_OK;
}

// Selection of a forked step: wait for the earlier selections on the same states.
int32_t wait_state_deps(mvla_ctx* ctx, const ForkPlan& fp, cudaStream_t sel_stream)
{
    for (unsigned s = 0; !fp.ordered_after_all && s < kSets; ++s)
        if ((fp.dep_mask >> s & 1u) && cudaStreamWaitEvent(sel_stream, ctx->ev_sel[s], 0) != cudaSuccess)
            return fail_cuda(ctx, cudaGetLastError());
    return MVLA_OK;
}

// Join of a forked step: the row copy on the caller's stream (and whatever the caller enqueues next) follows the selection.
int32_t join_selection(mvla_ctx* ctx, const ForkPlan& fp, unsigned par, cudaStream_t sel_stream, cudaStream_t st)
{
    if (cudaEventRecord(ctx->ev_sel[par], sel_stream) != cudaSuccess ||
        cudaStreamWaitEvent(st, ctx->ev_sel[par], 0) != cudaSuccess)
        return fail_cuda(ctx, cudaGetLastError());
    ctx->sel_valid[par] = true;
    ctx->sel_capture[par] = fp.cap_id;
    return MVLA_OK;
}

// ---- patch-by-patch path ----
int32_t validate_patch(const mvla_ctx* ctx, int32_t batch, const mvla_sample* samples)
{
    if (!ctx->cfg.patch_path) return MVLA_ERR_UNSUPPORTED;        // its state and scratch were not allocated
    for (int b = 0; b < batch; ++b)
        if (samples[b].n_2d != samples[b].n_3d || samples[b].n_2d < 1) return MVLA_ERR_INVALID_ARG;   // a patch owns one token of each
    return MVLA_OK;
}

// Layout of the attention copy: [head][visual token of the batch][text query, padded to whole 128-byte lines]
int64_t alpha_row(const mvla_ctx* ctx) { return (static_cast<int64_t>(ctx->cfg.max_text) + 31) / 32 * 32; }
size_t alpha_floats(const mvla_ctx* ctx)
{
    return static_cast<size_t>(ctx->cfg.n_heads) * ctx->vis_all * static_cast<size_t>(alpha_row(ctx));
}

AlphaOut alpha_of(const mvla_ctx* ctx, unsigned set)
{
    return AlphaOut{ctx->alpha_ws + set * alpha_floats(ctx), static_cast<int64_t>(ctx->vis_all) * alpha_row(ctx), alpha_row(ctx)};
}

PatchParams patch_params(const mvla_ctx* ctx)
{
    const mvla_config& c = ctx->cfg;
    PatchParams pp;
    pp.tau_2d = c.tau_2d; pp.tau_3d = c.tau_3d; pp.eps_3d = c.eps_3d;
    pp.obj_2d_min = c.obj_2d_min > 0.0 ? c.obj_2d_min : 0.5;
    pp.bg_prune_prob = 1.0 - c.floor_ratio;
    pp.kmeans_max_iter = c.kmeans_max_iter > 0 ? c.kmeans_max_iter : 32;
    pp.cold_start_full_keep = c.cold_start_full_keep;
    pp.max_patch = std::max(ctx->max_patch, 1);
    return pp;
}

// Salience with the attention copy, feature norms, head sum, per-patch indicators.
int32_t run_patch_indicators(mvla_ctx* ctx, unsigned set, const Plan& plan, int32_t batch, const void* q, const void* k,
                             const void* hidden, int64_t rows, float* attn_out, float* x_out, cudaStream_t st)
{
    const AlphaOut alpha = alpha_of(ctx, set);
    for (int first = 0; first < batch; first += kMaxChunk) {
        const BatchDesc bd = chunk_of(plan, first, std::min(kMaxChunk, batch - first));
        const int32_t rc = run_salience_chunk(ctx, bd, q, k, rows, nullptr, nullptr, nullptr, nullptr, false, st, alpha);
        if (rc != MVLA_OK) return rc;
    }
    for (int first = 0; first < batch; first += kMaxChunk) {
        const BatchDesc bd = chunk_of(plan, first, std::min(kMaxChunk, batch - first));
        const cudaError_t e = launch_patch_indicators(bd, ctx->cfg.n_heads, alpha, ctx->hidden_dtype, ctx->cfg.d_model, hidden,
                                                      x_out, attn_out, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    return MVLA_OK;
}

int32_t run_patch_select(mvla_ctx* ctx, unsigned set, const Plan& plan, int32_t batch, const float* attn, const float* x,
                         const float* rand_u, int32_t* kept_idx, int32_t* out_offsets, int32_t* counts,
                         float* xhat_out, int32_t* info_out, mvla_patch_diag* diag, cudaStream_t st)
{
    const PatchParams pp = patch_params(ctx);
    PatchIO io;
    std::memset(&io, 0, sizeof io);
    io.attn = attn; io.x = x; io.rand_u = rand_u;
    io.xhat_state = ctx->xhat_patch; io.xhat_out = xhat_out; io.info_out = info_out; io.diag = diag;
    int32_t* ws = ctx->nout_ws + set * (2 * static_cast<size_t>(ctx->cfg.max_batch) + 1);
    io.counts = counts; io.nout_ws = ws; io.ready_ws = ws + ctx->cfg.max_batch;
    io.done_ws = ws + 2 * ctx->cfg.max_batch; io.status = ctx->status_dev;
    io.kept_idx = kept_idx; io.out_offsets = out_offsets; io.batch_total = batch;
    for (int first = 0; first < batch; first += kMaxChunk) {
        const BatchDesc bd = chunk_of(plan, first, std::min(kMaxChunk, batch - first));
        io.chunk_first = first;
        const cudaError_t e = launch_patch_select(bd, pp, io, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    return MVLA_OK;
}

int32_t prune_step_patch(mvla_ctx* ctx, int32_t prune_point, int32_t batch, const mvla_sample* samples, uint32_t flags,
                         const mvla_tensors* in, const mvla_outputs* out, int32_t* total_kept_out, void* stream)
{
    PhaseRange ph;
    if (!in->hidden || !in->rand_u) return MVLA_ERR_INVALID_ARG;
    if (flags & ~(MVLA_FLAG_RESET_STATE | MVLA_FLAG_NO_STATE_UPDATE | MVLA_FLAG_INPUTS_STABLE)) return MVLA_ERR_INVALID_ARG;
    const void* src[3] = {in->hidden, in->k, in->v};
    void* dst[3] = {out->out_hidden, out->out_k, out->out_v};
    if (!aligned16(in->q) || !aligned16(out->patch_x) || !aligned16(out->patch_xhat)) return MVLA_ERR_INVALID_ARG;
    for (int i = 0; i < 3; ++i) {
        if (!aligned16(src[i]) || !aligned16(dst[i])) return MVLA_ERR_INVALID_ARG;
        if (dst[i] && (!src[i] || src[i] == dst[i])) return MVLA_ERR_INVALID_ARG;
    }
    int32_t rc = check_sticky(ctx);
    if (rc != MVLA_OK) return rc;
    rc = validate_samples(ctx, batch, samples, MVLA_MODE_ADAPTIVE, in->rows);
    if (rc != MVLA_OK) return rc;
    rc = validate_patch(ctx, batch, samples);
    if (rc != MVLA_OK) return rc;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    Plan plan;
    rc = make_plan(ctx, prune_point, batch, samples, MVLA_MODE_ADAPTIVE, flags, true, &plan);
    if (rc != MVLA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int64_t cap = 0;                               // the row count is known only on the device: cover the capacity
    for (int b = 0; b < batch; ++b) cap += samples[b].n_txt + samples[b].n_2d + samples[b].n_3d;
    CompactJob job;
    const int32_t kv_bytes = static_cast<int32_t>(ctx->kv_heads * ctx->cfg.head_dim * ctx->qk_elem);
    for (int i = 0; i < 3; ++i) { job.src[i] = src[i]; job.dst[i] = dst[i]; job.row_bytes[i] = kv_bytes; }
    job.row_bytes[0] = static_cast<int32_t>(ctx->cfg.d_model * ctx->elem);

    // Scratch set of this step; with stable inputs its scoring, indicators and selection run on that set's
    // side stream beside the steps before (plan_fork), the row copy stays on the caller's stream.
    ctx->step_parity = (ctx->step_parity + 1u) % kSets;
    const unsigned par = ctx->step_parity;
    bool forked = false;
    ForkPlan fp;
    if ((flags & MVLA_FLAG_INPUTS_STABLE) && ctx->patch_sets == kSets && batch <= kMaxChunk &&
        chunk_is_fast(ctx, chunk_of(plan, 0, batch))) {
        forked = true;
        const size_t nvis_b = static_cast<size_t>(plan.total_vis), npat_b = nvis_b / 2, in_rows = static_cast<size_t>(in->rows);
        const size_t hb = static_cast<size_t>(ctx->cfg.d_model) * ctx->elem, kb = static_cast<size_t>(kv_bytes);
        const size_t qb = static_cast<size_t>(ctx->cfg.n_heads) * ctx->cfg.head_dim * ctx->qk_elem;
        const mvla_ctx::Range side[12] = {
            range_of(out->kept_idx, static_cast<size_t>(cap) * 4), range_of(out->out_offsets, (batch + 1) * 4u),
            range_of(out->budgets, batch * 8u), range_of(out->attn, nvis_b * 4), range_of(out->patch_x, npat_b * 16),
            range_of(out->patch_xhat, npat_b * 16), range_of(out->patch_info, npat_b * 4),
            range_of(out->patch_diag, batch * sizeof(mvla_patch_diag)),
            range_of(in->q, in_rows * qb), range_of(in->k, in_rows * kb), range_of(in->hidden, in_rows * hb),
            range_of(in->rand_u, npat_b * 4)};
        const mvla_ctx::Range copied[3] = {range_of(out->out_hidden, static_cast<size_t>(cap) * hb),
                                           range_of(out->out_k, static_cast<size_t>(cap) * kb),
                                           range_of(out->out_v, static_cast<size_t>(cap) * kb)};
        rc = plan_fork(ctx, st, par, prune_point, batch, samples, side, 12, 8, copied, 3, &fp);
        if (rc != MVLA_OK) return rc;
    } else {
        ctx->hist_unknown = true;
        ctx->sel_valid[par] = false;               // this set is used outside the event chain
    }
    const unsigned set = forked ? par : 0;
    cudaStream_t side_stream = forked ? ctx->aux[par] : st;
    float* attn = out->attn ? out->attn : ctx->patch_attn_ws + set * ctx->vis_all;
    float* x = out->patch_x ? out->patch_x : ctx->patch_x_ws + set * (ctx->vis_all / 2 + 1) * 4;
    const BatchDesc whole = chunk_of(plan, 0, std::min(batch, kMaxChunk));
    if (!forked && batch <= kMaxChunk && chunk_is_fast(ctx, whole) && patch_tail_supported(whole)) {
        // two kernels: scoring (leaves the attention copy, re-arms the hand-over words), then indicators,
        // stages 1-4 and the row copy in one
        int32_t* list = ctx->tail_list + par * ctx->rows_all;
        unsigned long long* rec = ctx->patch_rec + par * (ctx->vis_all / 2 + 1) * 3;
        const AlphaOut alpha = alpha_of(ctx, set);
        ph.mark("mvla: scoring (+ attention copy)");
        rc = run_salience_chunk(ctx, whole, in->q, in->k, in->rows, nullptr, nullptr, nullptr, nullptr, false, st, alpha,
                                list, false, nullptr, false, rec);
        if (rc != MVLA_OK) return rc;
        const PatchParams pp = patch_params(ctx);
        PatchIO io;
        std::memset(&io, 0, sizeof io);
        io.rand_u = in->rand_u;
        io.xhat_state = ctx->xhat_patch; io.xhat_out = out->patch_xhat; io.info_out = out->patch_info; io.diag = out->patch_diag;
        int32_t* ws = ctx->nout_ws + set * (2 * static_cast<size_t>(ctx->cfg.max_batch) + 1);
        io.counts = out->budgets; io.nout_ws = ws; io.ready_ws = ws + ctx->cfg.max_batch;
        io.done_ws = ws + 2 * ctx->cfg.max_batch; io.status = ctx->status_dev;
        io.kept_idx = out->kept_idx; io.out_offsets = out->out_offsets; io.batch_total = batch;
        io.chunk_first = 0;
        ph.mark("mvla: indicators + stages 1-4 + row copy");
        const cudaError_t e = launch_patch_tail(whole, ctx->cfg.n_heads, alpha, ctx->hidden_dtype, ctx->cfg.d_model, in->hidden,
                                                x, attn, rec, pp, io, job, list, ctx->sm_count, ctx->tail_ticket + par, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        commit_steps(ctx, prune_point, plan, samples);
        if (total_kept_out) *total_kept_out = static_cast<int32_t>(cap);
        return MVLA_OK;
    }
    ph.mark("mvla: scoring + indicators");
    rc = run_patch_indicators(ctx, set, plan, batch, in->q, in->k, in->hidden, in->rows, attn, x, side_stream);
    if (rc != MVLA_OK) return rc;
    if (forked) {
        rc = wait_state_deps(ctx, fp, side_stream);
        if (rc != MVLA_OK) return rc;
    }
    ph.mark("mvla: stages 1-4");
    rc = run_patch_select(ctx, set, plan, batch, attn, x, in->rand_u, out->kept_idx, out->out_offsets, out->budgets,
                          out->patch_xhat, out->patch_info, out->patch_diag, side_stream);
    if (rc != MVLA_OK) return rc;
    if (forked) {
        rc = join_selection(ctx, fp, par, side_stream, st);
        if (rc != MVLA_OK) return rc;
    }
    for (int first = 0; first < batch; first += kMaxChunk) {
        const BatchDesc bd = chunk_of(plan, first, std::min(kMaxChunk, batch - first));
        ph.mark("mvla: row copy");
        const cudaError_t e = launch_compact(bd, job, out->kept_idx, static_cast<int32_t>(cap), 0, out->out_offsets, first, batch, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    if (forked && cudaEventRecord(ctx->ev_copy[par], st) != cudaSuccess) return fail_cuda(ctx, cudaGetLastError());
    commit_steps(ctx, prune_point, plan, samples);
    if (total_kept_out) *total_kept_out = static_cast<int32_t>(cap);
    return MVLA_OK;
}

}  // namespace

extern "C" {

static int32_t mvla_prune_create_impl(const mvla_config* cfg, mvla_ctx** out)
{
    if (!cfg || !out) return MVLA_ERR_INVALID_ARG;
    *out = nullptr;
    const mvla_config& c = *cfg;
    if (c.n_heads < 1 || c.d_model < 1 || c.max_batch < 1 || c.max_text < 1 || c.max_2d < 0 || c.max_3d < 0 ||
        c.max_2d + c.max_3d < 1 || c.n_prune_points < 1 || c.n_state_slots < 0 || c.window_k < 1 || c.device < 0)
        return MVLA_ERR_INVALID_ARG;
    if (!(c.beta >= 0.0 && c.beta <= 1.0) || !(c.floor_ratio >= 0.0 && c.floor_ratio <= 1.0) ||
        !std::isfinite(c.tau_2d) || !std::isfinite(c.tau_3d) || !std::isfinite(c.eps_3d))
        return MVLA_ERR_INVALID_ARG;
    if (c.dtype != MVLA_DTYPE_BF16 && c.dtype != MVLA_DTYPE_FP32 && c.dtype != MVLA_DTYPE_FP8_E4M3) return MVLA_ERR_UNSUPPORTED;
    if (c.dtype == MVLA_DTYPE_FP8_E4M3 && (c.salience_path == MVLA_SALIENCE_FMA || c.patch_path)) return MVLA_ERR_UNSUPPORTED;
    if (c.salience_path != MVLA_SALIENCE_AUTO && c.salience_path != MVLA_SALIENCE_FMA) return MVLA_ERR_INVALID_ARG;
    if (c.logit_cache != 0 && c.logit_cache != 1) return MVLA_ERR_INVALID_ARG;
    if (c.logit_cache && (c.dtype == MVLA_DTYPE_FP32 || c.salience_path == MVLA_SALIENCE_FMA || c.patch_path))
        return MVLA_ERR_UNSUPPORTED;          // the cache lives in the tensor-core scoring kernel of the budgeted path
    if ((c.patch_path != 0 && c.patch_path != 1) || c.kmeans_max_iter < 0 || !(c.obj_2d_min >= 0.0 && c.obj_2d_min <= 1.0))
        return MVLA_ERR_INVALID_ARG;
    if (c.head_dim < 64 || c.head_dim > 256 || c.head_dim % 32 != 0) return MVLA_ERR_UNSUPPORTED;
    if (c.n_kv_heads < 0 || (c.n_kv_heads > 0 && (c.n_kv_heads > c.n_heads || c.n_heads % c.n_kv_heads != 0))) return MVLA_ERR_INVALID_ARG;
    if (c.patch_path && c.n_kv_heads > 0 && c.n_kv_heads != c.n_heads) return MVLA_ERR_UNSUPPORTED;   // the patch path is built for ungrouped keys
    if (c.max_text > kMaxText || c.max_2d + c.max_3d > kMaxVis || c.max_batch > 64) return MVLA_ERR_UNSUPPORTED;
    const size_t elem = c.dtype == MVLA_DTYPE_FP32 ? 4 : 2;       // hidden: fp32, or bf16 (also beside e4m3 q / k / v)
    if ((static_cast<size_t>(c.d_model) * elem) % 16 != 0) return MVLA_ERR_UNSUPPORTED;

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || c.device >= ndev) {
        cudaGetLastError();
        return MVLA_ERR_CUDA;
    }
    DeviceGuard guard(c.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c.device) != cudaSuccess) return MVLA_ERR_CUDA;
    if (prop.major != 10) return MVLA_ERR_UNSUPPORTED;        // built for sm_100a only

    mvla_ctx* ctx = new (std::nothrow) mvla_ctx();
    if (!ctx) return MVLA_ERR_OOM;
    ctx->cfg = c;
    ctx->n_slots = c.n_state_slots > 0 ? c.n_state_slots : c.max_batch;
    ctx->max_vis = c.max_2d + c.max_3d;
    ctx->elem = elem;
    ctx->qk_elem = c.dtype == MVLA_DTYPE_FP8_E4M3 ? 1 : elem;
    ctx->hidden_dtype = c.dtype == MVLA_DTYPE_FP32 ? MVLA_DTYPE_FP32 : MVLA_DTYPE_BF16;
    ctx->use_umma = c.dtype != MVLA_DTYPE_FP32;
    ctx->kv_heads = c.n_kv_heads > 0 ? c.n_kv_heads : c.n_heads;
    if (c.salience_path == MVLA_SALIENCE_FMA) ctx->use_umma = false;
    ctx->part = ctx->l1_ws = ctx->ahat_state = ctx->mhat_state = nullptr;
    ctx->acc64 = nullptr;
    ctx->tail_list = nullptr;
    ctx->tail_ticket = nullptr;
    ctx->patch_rec = nullptr;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->stage_event = nullptr;
    ctx->stamps = nullptr;
    ctx->lcache = nullptr;
    ctx->cache_cols = (c.max_text + 15) / 16 * 16;
    ctx->tiles_computed = ctx->tiles_reused = 0;
    ctx->alpha_ws = ctx->xhat_patch = ctx->patch_x_ws = ctx->patch_attn_ws = nullptr;
    ctx->patch_sets = 1;
    ctx->nout_ws = nullptr;
    ctx->max_patch = std::min(c.max_2d, c.max_3d);
    ctx->ev_fork = nullptr;
    for (int i = 0; i < kSets; ++i) {
        ctx->aux[i] = nullptr;
        ctx->ev_sel[i] = ctx->ev_copy[i] = nullptr;
        ctx->n_hist[i] = 0;
        ctx->n_state_of[i] = 0;
        ctx->sel_valid[i] = false;
        ctx->sel_capture[i] = 0;
    }
    ctx->hist_unknown = true;
    ctx->status_host = ctx->status_dev = nullptr;
    ctx->last_cuda = cudaSuccess;
    ctx->tm_ptr[0] = ctx->tm_ptr[1] = nullptr;
    ctx->tm_rows[0] = ctx->tm_rows[1] = -1;
    ctx->encode = nullptr;
    ctx->t_host.assign(static_cast<size_t>(c.n_prune_points) * ctx->n_slots, 0);

    const size_t vis_all = static_cast<size_t>(c.max_batch) * ctx->max_vis;
    ctx->part_stride = static_cast<int64_t>(vis_all);
    const size_t n_state = static_cast<size_t>(c.n_prune_points) * ctx->n_slots;
    cudaError_t e = cudaSuccess;
    auto alloc = [&](float** p, size_t n) {
        if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(float));
        if (e == cudaSuccess) e = cudaMemset(*p, 0, n * sizeof(float));
    };
    alloc(&ctx->part, vis_all * c.n_heads);
    alloc(&ctx->l1_ws, kSets * vis_all);
    ctx->vis_all = vis_all;
    ctx->step_parity = 0;
    alloc(&ctx->ahat_state, 2 * n_state * ctx->max_vis);
    alloc(&ctx->mhat_state, 2 * n_state * 4);
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->acc64), kSets * vis_all * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(ctx->acc64, 0, kSets * vis_all * sizeof(unsigned long long));
    ctx->rows_all = static_cast<size_t>(c.max_batch) * (kHandWords + c.max_text + ctx->max_vis);
    // (+ 1: a word that no launch ever writes, for mvla_selftest_wait_timeout)
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->tail_list), (kSets * ctx->rows_all + 1) * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->tail_list, 0xFF, (kSets * ctx->rows_all + 1) * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->tail_ticket), kSets * sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMemset(ctx->tail_ticket, 0, kSets * sizeof(unsigned int));
    if (c.logit_cache) {
        ctx->cache_sig.assign(n_state, mvla_ctx::CacheSig{false, 0, 0, 0});
        alloc(&ctx->lcache, n_state * static_cast<size_t>(c.n_heads) * ctx->max_vis * ctx->cache_cols);
    }
    if (c.patch_path) {
        const size_t alpha_n = alpha_floats(ctx);
        ctx->patch_sets = alpha_n * sizeof(float) * kSets <= (size_t(1) << 30) ? kSets : 1;   // at most 1 GiB of attention copies
        alloc(&ctx->alpha_ws, alpha_n * ctx->patch_sets);
        alloc(&ctx->xhat_patch, n_state * std::max(ctx->max_patch, 1) * 4);
        alloc(&ctx->patch_x_ws, (vis_all / 2 + 1) * 4 * ctx->patch_sets);
        alloc(&ctx->patch_attn_ws, vis_all * ctx->patch_sets);
        const size_t nrec = kSets * (vis_all / 2 + 1) * 3 * sizeof(unsigned long long);
        if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->patch_rec), nrec);
        if (e == cudaSuccess) e = cudaMemset(ctx->patch_rec, 0xFF, nrec);
        const size_t nws = (2 * static_cast<size_t>(c.max_batch) + 1) * sizeof(int32_t) * ctx->patch_sets;
        if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->nout_ws), nws);
        if (e == cudaSuccess) e = cudaMemset(ctx->nout_ws, 0, nws);
    }
    for (cudaStream_t* sp = ctx->aux; sp != ctx->aux + kSets; ++sp)
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(sp, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
    for (cudaEvent_t* ev = ctx->ev_sel; ev != ctx->ev_sel + kSets; ++ev)
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
    for (cudaEvent_t* ev = ctx->ev_copy; ev != ctx->ev_copy + kSets; ++ev)
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaHostAlloc(reinterpret_cast<void**>(&ctx->status_host), sizeof(int), cudaHostAllocMapped);
    if (e == cudaSuccess) {
        *ctx->status_host = 0;
        e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&ctx->status_dev), ctx->status_host, 0);
    }
    if (e == cudaSuccess && ctx->use_umma) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres);
        if (e == cudaSuccess && (qres != cudaDriverEntryPointSuccess || !fn)) e = cudaErrorNotSupported;
        ctx->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    }
    if (e != cudaSuccess) {
        const int32_t rc = e == cudaErrorMemoryAllocation ? MVLA_ERR_OOM : MVLA_ERR_CUDA;
        cudaGetLastError();
        mvla_prune_destroy(ctx);
        return rc;
    }
    *out = ctx;
    return MVLA_OK;
}

void mvla_prune_destroy(mvla_ctx* ctx)
{
    if (!ctx) return;
    DeviceGuard guard(ctx->cfg.device);
    cudaFree(ctx->part);
    cudaFree(ctx->l1_ws);
    cudaFree(ctx->ahat_state);
    cudaFree(ctx->mhat_state);
    cudaFree(ctx->acc64);
    cudaFree(ctx->tail_list);
    cudaFree(ctx->tail_ticket);
    cudaFree(ctx->patch_rec);
    cudaFree(ctx->lcache);
    cudaFree(ctx->alpha_ws);
    cudaFree(ctx->xhat_patch);
    cudaFree(ctx->patch_x_ws);
    cudaFree(ctx->patch_attn_ws);
    cudaFree(ctx->nout_ws);
    for (cudaStream_t sp : ctx->aux)
        if (sp) {
            cudaStreamSynchronize(sp);
            cudaStreamDestroy(sp);
        }
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    for (cudaEvent_t ev : ctx->ev_sel)
        if (ev) cudaEventDestroy(ev);
    for (cudaEvent_t ev : ctx->ev_copy)
        if (ev) cudaEventDestroy(ev);
    if (ctx->status_host) cudaFreeHost(ctx->status_host);
    delete ctx;
}

static int32_t mvla_salience_impl(mvla_ctx* ctx, int32_t batch, const mvla_sample* samples, const void* q, const void* k,
                      const void* hidden, int64_t rows, float* attn_out, float* l1_out, void* stream)
{
    if (!ctx || !q || !k || !attn_out || rows < 1) return MVLA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(hidden)) return MVLA_ERR_INVALID_ARG;
    int32_t rc = check_sticky(ctx);
    if (rc != MVLA_OK) return rc;
    rc = validate_samples(ctx, batch, samples, MVLA_MODE_FIXED, rows);
    if (rc != MVLA_OK) return rc;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    ctx->hist_unknown = true;                        // what the stream ran last is no longer a known prune step
    Plan plan;
    rc = make_plan(ctx, 0, batch, samples, MVLA_MODE_FIXED, 0, false, &plan);
    if (rc != MVLA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool want_l1 = hidden && l1_out;
    for (int first = 0; first < batch; first += kMaxChunk) {
        const BatchDesc bd = chunk_of(plan, first, std::min(kMaxChunk, batch - first));
        rc = run_salience_chunk(ctx, bd, q, k, rows, want_l1 ? hidden : nullptr, l1_out, nullptr, nullptr, false, st);
        if (rc != MVLA_OK) return rc;
    }
    const cudaError_t e = launch_head_reduce(ctx->part, ctx->part_stride, ctx->cfg.n_heads, plan.total_vis, attn_out, st);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    return MVLA_OK;
}

static int32_t mvla_select_impl(mvla_ctx* ctx, int32_t prune_point, int32_t batch, const mvla_sample* samples, int32_t mode,
                    uint32_t flags, const float* attn, const float* l1, int32_t* kept_idx, int32_t* out_offsets,
                    int32_t* budgets, float* ahat_out, float* z_out, mvla_diag* diag, void* stream)
{
    if (!ctx || !attn || !kept_idx || !out_offsets) return MVLA_ERR_INVALID_ARG;
    if (flags & ~(MVLA_FLAG_RESET_STATE | MVLA_FLAG_NO_STATE_UPDATE)) return MVLA_ERR_INVALID_ARG;
    int32_t rc = check_sticky(ctx);
    if (rc != MVLA_OK) return rc;
    rc = validate_samples(ctx, batch, samples, mode, -1);
    if (rc != MVLA_OK) return rc;
    if (mode == MVLA_MODE_ADAPTIVE && !l1) return MVLA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    ctx->hist_unknown = true;                        // what the stream ran last is no longer a known prune step
    Plan plan;
    rc = make_plan(ctx, prune_point, batch, samples, mode, flags, true, &plan);
    if (rc != MVLA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const GateParams gp = gate_params(ctx, mode, l1 != nullptr);
    for (int first = 0; first < batch; first += kMaxChunk) {
        const int n = std::min(kMaxChunk, batch - first);
        const BatchDesc bd = chunk_of(plan, first, n);
        SelectIO io;
        std::memset(&io, 0, sizeof io);
        io.attn = attn; io.n_heads = ctx->cfg.n_heads; io.l1 = l1;
        io.ahat_state = ctx->ahat_state; io.mhat_state = ctx->mhat_state;
        io.kept_idx = kept_idx; io.out_offsets = out_offsets; io.budgets = budgets;
        io.ahat_out = ahat_out; io.z_out = z_out; io.diag = diag;
        io.chunk_first = first; io.total_out = plan.total_out; io.write_total = first + n == batch;
        io.n_in_launch = n;
        const cudaError_t e = launch_select(bd, gp, io, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    commit_steps(ctx, prune_point, plan, samples);
    return MVLA_OK;
}

static int32_t mvla_compact_impl(mvla_ctx* ctx, int32_t batch, const mvla_sample* samples, const int32_t* kept_idx,
                     const int32_t* out_offsets, int32_t total_kept, const void* hidden, const void* k,
                     const void* v, void* out_hidden, void* out_k, void* out_v, void* stream)
{
    if (!ctx || !kept_idx || !out_offsets || total_kept < 0) return MVLA_ERR_INVALID_ARG;
    const void* src[3] = {hidden, k, v};
    void* dst[3] = {out_hidden, out_k, out_v};
    for (int i = 0; i < 3; ++i) {
        if (!src[i] || !dst[i]) continue;
        if (!aligned16(src[i]) || !aligned16(dst[i]) || src[i] == dst[i]) return MVLA_ERR_INVALID_ARG;
    }
    int32_t rc = check_sticky(ctx);
    if (rc != MVLA_OK) return rc;
    rc = validate_samples(ctx, batch, samples, MVLA_MODE_FIXED, -1);
    if (rc != MVLA_OK) return rc;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    ctx->hist_unknown = true;                        // what the stream ran last is no longer a known prune step
    Plan plan;
    rc = make_plan(ctx, 0, batch, samples, MVLA_MODE_FIXED, 0, false, &plan);
    if (rc != MVLA_OK) return rc;
    CompactJob job;
    const int32_t kv_bytes = static_cast<int32_t>(ctx->kv_heads * ctx->cfg.head_dim * ctx->qk_elem);
    for (int i = 0; i < 3; ++i) { job.src[i] = src[i]; job.dst[i] = dst[i]; job.row_bytes[i] = kv_bytes; }
    job.row_bytes[0] = static_cast<int32_t>(ctx->cfg.d_model * ctx->elem);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int first = 0; first < batch; first += kMaxChunk) {
        const BatchDesc bd = chunk_of(plan, first, std::min(kMaxChunk, batch - first));
        const cudaError_t e = launch_compact(bd, job, kept_idx, total_kept, 0, out_offsets, first, batch, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
    }
    return MVLA_OK;
}

int32_t mvla_set_stage_event(mvla_ctx* ctx, void* event)
{
    if (!ctx) return MVLA_ERR_INVALID_ARG;
    ctx->stage_event = static_cast<cudaEvent_t>(event);
    return MVLA_OK;
}

int32_t mvla_logit_cache_stats(mvla_ctx* ctx, int64_t* tiles_computed, int64_t* tiles_reused)
{
    if (!ctx) return MVLA_ERR_INVALID_ARG;
    if (tiles_computed) *tiles_computed = ctx->tiles_computed;
    if (tiles_reused) *tiles_reused = ctx->tiles_reused;
    return MVLA_OK;
}

int32_t mvla_set_kernel_stamps(mvla_ctx* ctx, uint64_t* device_buffer)
{
    if (!ctx || (reinterpret_cast<uintptr_t>(device_buffer) & 7u)) return MVLA_ERR_INVALID_ARG;
    ctx->stamps = reinterpret_cast<unsigned long long*>(device_buffer);
    return MVLA_OK;
}

int32_t mvla_selftest_wait_timeout(mvla_ctx* ctx, uint32_t limit_us, void* stream)
{
    if (!ctx || limit_us < 1 || limit_us > 1000000u) return MVLA_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    // the last word of the kept-list scratch is never an output row of any launch: it stays -1
    const int32_t* never_set = ctx->tail_list + kSets * ctx->rows_all;
    const cudaError_t e = launch_wait_probe(never_set, static_cast<uint64_t>(limit_us) * 1000ull, ctx->status_dev,
                                            static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    return MVLA_OK;
}

static int32_t mvla_patch_indicators_impl(mvla_ctx* ctx, int32_t batch, const mvla_sample* samples, const void* q, const void* k,
                              const void* hidden, int64_t rows, float* attn_out, float* x_out, void* stream)
{
    if (!ctx || !q || !k || !hidden || !attn_out || !x_out || rows < 1) return MVLA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(hidden) || !aligned16(x_out)) return MVLA_ERR_INVALID_ARG;
    int32_t rc = check_sticky(ctx);
    if (rc != MVLA_OK) return rc;
    rc = validate_samples(ctx, batch, samples, MVLA_MODE_FIXED, rows);
    if (rc != MVLA_OK) return rc;
    rc = validate_patch(ctx, batch, samples);
    if (rc != MVLA_OK) return rc;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    ctx->hist_unknown = true;
    Plan plan;
    rc = make_plan(ctx, 0, batch, samples, MVLA_MODE_FIXED, 0, false, &plan);
    if (rc != MVLA_OK) return rc;
    return run_patch_indicators(ctx, 0, plan, batch, q, k, hidden, rows, attn_out, x_out, static_cast<cudaStream_t>(stream));
}

static int32_t mvla_patch_select_impl(mvla_ctx* ctx, int32_t prune_point, int32_t batch, const mvla_sample* samples, uint32_t flags,
                          const float* attn, const float* x, const float* rand_u, int32_t* kept_idx,
                          int32_t* out_offsets, int32_t* counts, float* xhat_out, int32_t* info_out,
                          mvla_patch_diag* diag, void* stream)
{
    if (!ctx || !attn || !x || !rand_u || !kept_idx || !out_offsets) return MVLA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(xhat_out)) return MVLA_ERR_INVALID_ARG;
    if (flags & ~(MVLA_FLAG_RESET_STATE | MVLA_FLAG_NO_STATE_UPDATE)) return MVLA_ERR_INVALID_ARG;
    int32_t rc = check_sticky(ctx);
    if (rc != MVLA_OK) return rc;
    rc = validate_samples(ctx, batch, samples, MVLA_MODE_ADAPTIVE, -1);
    if (rc != MVLA_OK) return rc;
    rc = validate_patch(ctx, batch, samples);
    if (rc != MVLA_OK) return rc;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    ctx->hist_unknown = true;
    Plan plan;
    rc = make_plan(ctx, prune_point, batch, samples, MVLA_MODE_ADAPTIVE, flags, true, &plan);
    if (rc != MVLA_OK) return rc;
    rc = run_patch_select(ctx, 0, plan, batch, attn, x, rand_u, kept_idx, out_offsets, counts, xhat_out, info_out, diag,
                          static_cast<cudaStream_t>(stream));
    if (rc != MVLA_OK) return rc;
    commit_steps(ctx, prune_point, plan, samples);
    return MVLA_OK;
}

static int32_t mvla_prune_step_impl(mvla_ctx* ctx, int32_t prune_point, int32_t batch, const mvla_sample* samples,
                        int32_t mode, uint32_t flags, const mvla_tensors* in, const mvla_outputs* out,
                        int32_t* total_kept_out, void* stream)
{
    if (!ctx || !in || !out || !in->q || !in->k || !out->kept_idx || !out->out_offsets || in->rows < 1)
        return MVLA_ERR_INVALID_ARG;
    PhaseRange ph;
    if (mode == MVLA_MODE_PATCH)
        return prune_step_patch(ctx, prune_point, batch, samples, flags, in, out, total_kept_out, stream);
    if (flags & ~(MVLA_FLAG_RESET_STATE | MVLA_FLAG_NO_STATE_UPDATE | MVLA_FLAG_INPUTS_STABLE)) return MVLA_ERR_INVALID_ARG;
    if (mode == MVLA_MODE_ADAPTIVE && !in->hidden) return MVLA_ERR_INVALID_ARG;
    const void* src[3] = {in->hidden, in->k, in->v};
    void* dst[3] = {out->out_hidden, out->out_k, out->out_v};
    if (!aligned16(in->q)) return MVLA_ERR_INVALID_ARG;
    for (int i = 0; i < 3; ++i) {
        if (!aligned16(src[i]) || !aligned16(dst[i])) return MVLA_ERR_INVALID_ARG;
        if (dst[i] && (!src[i] || src[i] == dst[i])) return MVLA_ERR_INVALID_ARG;
    }
    int32_t rc = check_sticky(ctx);
    if (rc != MVLA_OK) return rc;
    rc = validate_samples(ctx, batch, samples, mode, in->rows);
    if (rc != MVLA_OK) return rc;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return MVLA_ERR_CUDA;
    Plan plan;
    rc = make_plan(ctx, prune_point, batch, samples, mode, flags, true, &plan);
    if (rc != MVLA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool adaptive = mode == MVLA_MODE_ADAPTIVE;
    const GateParams gp = gate_params(ctx, mode, adaptive);
    CompactJob job;
    const int32_t kv_bytes = static_cast<int32_t>(ctx->kv_heads * ctx->cfg.head_dim * ctx->qk_elem);
    for (int i = 0; i < 3; ++i) { job.src[i] = src[i]; job.dst[i] = dst[i]; job.row_bytes[i] = kv_bytes; }
    job.row_bytes[0] = static_cast<int32_t>(ctx->cfg.d_model * ctx->elem);

    // Reuse of the previous step's logits: which key tiles of which sample must be computed (host decision
    // from the caller's changed_rows), for steps that are not overlapped with their neighbours.
    const bool cache_on = ctx->lcache != nullptr && !(flags & MVLA_FLAG_INPUTS_STABLE);
    for (int b = 0; b < batch; ++b) {
        SampleDev& d = plan.s[b];
        d.cache_state = -1;
        d.tile_compute = 0xFFFFFFFFu;
        if (!ctx->lcache) continue;
        const mvla_sample& sm = samples[b];
        const int sidx = prune_point * ctx->n_slots + sm.state_slot;
        mvla_ctx::CacheSig& sig = ctx->cache_sig[sidx];
        const int tiles = tiles_of(d);
        const bool fits = sm.n_2d + sm.n_3d <= 2048 && batch <= kMaxChunk;
        if (!cache_on || !fits || (flags & MVLA_FLAG_NO_STATE_UPDATE)) {
            // the step runs without the cache; a dry run leaves it as it is, anything else makes it stale
            if (!(flags & MVLA_FLAG_NO_STATE_UPDATE)) sig.valid = false;
            continue;
        }
        d.cache_state = sidx;
        bool all = !sig.valid || (flags & MVLA_FLAG_RESET_STATE) || !in->changed_rows || sig.n_txt != sm.n_txt ||
                   sig.n_2d != sm.n_2d || sig.n_3d != sm.n_3d;
        const uint8_t* ch = in->changed_rows ? in->changed_rows + sm.seq_off : nullptr;
        for (int i = 0; i < sm.n_txt && !all; ++i) all = ch[sm.off_txt + i] != 0;   // a changed query changes every logit
        if (!all) {
            uint32_t mask = 0;
            const int t2 = (sm.n_2d + kKeyTile - 1) / kKeyTile;
            for (int t = 0; t < tiles; ++t) {
                const int off = t < t2 ? sm.off_2d + t * kKeyTile : sm.off_3d + (t - t2) * kKeyTile;
                const int n = t < t2 ? std::min(kKeyTile, sm.n_2d - t * kKeyTile) : std::min(kKeyTile, sm.n_3d - (t - t2) * kKeyTile);
                bool any = false;
                for (int i = 0; i < n && !any; ++i) any = ch[off + i] != 0;
                if (any) mask |= 1u << t;
            }
            d.tile_compute = mask;
        }
        for (int t = 0; t < tiles; ++t) ((d.tile_compute >> t) & 1u ? ctx->tiles_computed : ctx->tiles_reused) += 1;
        sig = mvla_ctx::CacheSig{true, sm.n_txt, sm.n_2d, sm.n_3d};
    }

    // scratch set of this step
    ctx->step_parity = (ctx->step_parity + 1u) % kSets;
    unsigned long long* acc64 = ctx->acc64 + ctx->step_parity * ctx->vis_all;
    float* l1_ws = ctx->l1_ws + ctx->step_parity * ctx->vis_all;
    // With stable inputs (and the fast scoring kernel, whose scratch rotates over kSets sets) scoring and
    // selection go to the side stream of this step's scratch set (see plan_fork).
    bool forked = false;
    ForkPlan fp;
    const unsigned par = ctx->step_parity;
    const size_t nvis_b = static_cast<size_t>(plan.total_vis), nout_b = static_cast<size_t>(plan.total_out);
    const size_t hb = static_cast<size_t>(ctx->cfg.d_model) * ctx->elem, kb = static_cast<size_t>(kv_bytes);
    const size_t qb = static_cast<size_t>(ctx->cfg.n_heads) * ctx->cfg.head_dim * ctx->qk_elem;
    if ((flags & MVLA_FLAG_INPUTS_STABLE) && batch <= kMaxChunk && chunk_is_fast(ctx, chunk_of(plan, 0, batch))) {
        forked = true;
        // buffers the side-stream work touches: selection outputs, and the inputs of scoring
        const size_t in_rows = static_cast<size_t>(in->rows);
        const mvla_ctx::Range side[10] = {
            range_of(out->kept_idx, nout_b * 4), range_of(out->out_offsets, (batch + 1) * 4u),
            range_of(out->budgets, batch * 8u), range_of(out->attn, nvis_b * 4), range_of(out->ahat, nvis_b * 4),
            range_of(out->z, nvis_b * 4), range_of(out->diag, batch * sizeof(mvla_diag)),
            range_of(in->q, in_rows * qb), range_of(in->k, in_rows * kb),
            range_of(adaptive ? in->hidden : nullptr, in_rows * hb)};
        const mvla_ctx::Range copied[3] = {range_of(out->out_hidden, nout_b * hb), range_of(out->out_k, nout_b * kb),
                                           range_of(out->out_v, nout_b * kb)};
        rc = plan_fork(ctx, st, par, prune_point, batch, samples, side, 10, 7, copied, 3, &fp);
        if (rc != MVLA_OK) return rc;
    } else {
        ctx->hist_unknown = true;
    }
    for (int first = 0; first < batch; first += kMaxChunk) {
        const int n = std::min(kMaxChunk, batch - first);
        const BatchDesc bd = chunk_of(plan, first, n);
        bool used_acc64 = false;
        // the fused selection + copy kernel (below) wants its list words re-armed by the scoring kernel
        const bool tail = !forked && select_copy_supported(bd);
        ph.mark("mvla: scoring");
        rc = run_salience_chunk(ctx, bd, in->q, in->k, in->rows, adaptive ? in->hidden : nullptr, l1_ws, acc64,
                                &used_acc64, false, forked ? ctx->aux[par] : st, AlphaOut{nullptr, 0, 0},
                                tail ? ctx->tail_list + par * ctx->rows_all : nullptr, tail, tail ? ctx->stamps : nullptr,
                                cache_on);
        if (rc != MVLA_OK) return rc;
        if (ctx->stage_event && !forked) {
            // under stream capture the record must become an event-record node of the graph (an "external"
            // record): only then can the event be timed after a replay
            cudaStreamCaptureStatus cst = cudaStreamCaptureStatusNone;
            cudaStreamIsCapturing(st, &cst);
            const unsigned how = cst == cudaStreamCaptureStatusActive ? cudaEventRecordExternal : cudaEventRecordDefault;
            if (cudaEventRecordWithFlags(ctx->stage_event, st, how) != cudaSuccess) return fail_cuda(ctx, cudaGetLastError());
        }
        cudaStream_t sel_stream = st;
        if (forked) {
            sel_stream = ctx->aux[par];
            rc = wait_state_deps(ctx, fp, sel_stream);
            if (rc != MVLA_OK) return rc;
        }
        SelectIO io;
        std::memset(&io, 0, sizeof io);
        io.n_heads = ctx->cfg.n_heads;
        if (used_acc64) io.acc64 = acc64;
        else { io.part = ctx->part; io.part_stride = ctx->part_stride; }
        io.l1 = adaptive ? l1_ws : nullptr;
        io.ahat_state = ctx->ahat_state; io.mhat_state = ctx->mhat_state;
        io.kept_idx = out->kept_idx; io.out_offsets = out->out_offsets; io.budgets = out->budgets;
        io.attn_out = out->attn; io.ahat_out = out->ahat; io.z_out = out->z; io.diag = out->diag;
        io.chunk_first = first; io.total_out = plan.total_out; io.write_total = first + n == batch;
        io.n_in_launch = n;
        if (!forked && used_acc64 && select_copy_supported(bd)) {
            // one kernel for selection and row copy: every CTA repeats its sample's selection, then copies
            ctx->sel_valid[par] = false;             // this set was used outside the event chain
            const bool copying = (job.src[0] && job.dst[0]) || (job.src[1] && job.dst[1]) || (job.src[2] && job.dst[2]);
            (void)copying;
            ph.mark("mvla: selection + row copy");
            const cudaError_t e2 = launch_select_copy(bd, gp, io, job, ctx->tail_list + par * ctx->rows_all,
                                                      ctx->status_dev, ctx->sm_count * kTailCtasPerSm - n,
                                                      ctx->stamps ? ctx->stamps + 2 * kStampSlots : nullptr, st);
            if (e2 != cudaSuccess) {
                clear_accumulators(acc64, bd, st);
                return fail_cuda(ctx, e2);
            }
            continue;
        }
        ph.mark("mvla: selection");
        cudaError_t e = launch_select(bd, gp, io, sel_stream);
        if (e != cudaSuccess) {
            if (used_acc64) clear_accumulators(acc64, bd, sel_stream);
            return fail_cuda(ctx, e);
        }
        if (forked) {                                // join: the row copy, and whatever the caller enqueues next
            rc = join_selection(ctx, fp, par, sel_stream, st);
            if (rc != MVLA_OK) return rc;
        } else {
            ctx->sel_valid[par] = false;             // this set was used outside the event chain
        }
        const int32_t row0 = bd.s[0].out_off;
        const int32_t nrows = bd.s[n - 1].out_off + bd.s[n - 1].n_out - row0;
        ph.mark("mvla: row copy");
        e = launch_compact(bd, job, out->kept_idx, nrows, row0, nullptr, first, batch, st);
        if (e != cudaSuccess) return fail_cuda(ctx, e);
        if (forked && cudaEventRecord(ctx->ev_copy[par], st) != cudaSuccess) return fail_cuda(ctx, cudaGetLastError());
    }
    commit_steps(ctx, prune_point, plan, samples);
    if (total_kept_out) *total_kept_out = plan.total_out;
    return MVLA_OK;
}

// ---- the public entry points: an NVTX range around each call, and with MVLA_LOG=1 a line on stderr per call

int32_t mvla_prune_create(const mvla_config* cfg, mvla_ctx** out)
{
    ApiRange range("mvla_prune_create");
    const int32_t rc = mvla_prune_create_impl(cfg, out);
    if (log_enabled()) std::fprintf(stderr, "[mvla] mvla_prune_create(heads %lld x %lld, d_model %lld, dtype %lld, max batch %lld, text %lld, 2D %lld, 3D %lld) -> %d\n", static_cast<long long>(cfg ? cfg->n_heads : -1), static_cast<long long>(cfg ? cfg->head_dim : -1), static_cast<long long>(cfg ? cfg->d_model : -1), static_cast<long long>(cfg ? cfg->dtype : -1), static_cast<long long>(cfg ? cfg->max_batch : -1), static_cast<long long>(cfg ? cfg->max_text : -1), static_cast<long long>(cfg ? cfg->max_2d : -1), static_cast<long long>(cfg ? cfg->max_3d : -1), rc);
    return rc;
}

int32_t mvla_salience(mvla_ctx* ctx, int32_t batch, const mvla_sample* samples, const void* q, const void* k,
                      const void* hidden, int64_t rows, float* attn_out, float* l1_out, void* stream)
{
    ApiRange range("mvla_salience");
    const int32_t rc = mvla_salience_impl(ctx, batch, samples, q, k, hidden, rows, attn_out, l1_out, stream);
    if (log_enabled()) std::fprintf(stderr, "[mvla] mvla_salience(batch %lld, rows %lld) -> %d\n", static_cast<long long>(batch), static_cast<long long>(rows), rc);
    return rc;
}

int32_t mvla_select(mvla_ctx* ctx, int32_t prune_point, int32_t batch, const mvla_sample* samples, int32_t mode,
                    uint32_t flags, const float* attn, const float* l1, int32_t* kept_idx, int32_t* out_offsets,
                    int32_t* budgets, float* ahat_out, float* z_out, mvla_diag* diag, void* stream)
{
    ApiRange range("mvla_select");
    const int32_t rc = mvla_select_impl(ctx, prune_point, batch, samples, mode, flags, attn, l1, kept_idx, out_offsets, budgets, ahat_out, z_out, diag, stream);
    if (log_enabled()) std::fprintf(stderr, "[mvla] mvla_select(prune_point %lld, batch %lld, mode %lld, flags %lld) -> %d\n", static_cast<long long>(prune_point), static_cast<long long>(batch), static_cast<long long>(mode), static_cast<long long>(flags), rc);
    return rc;
}

int32_t mvla_compact(mvla_ctx* ctx, int32_t batch, const mvla_sample* samples, const int32_t* kept_idx,
                     const int32_t* out_offsets, int32_t total_kept, const void* hidden, const void* k,
                     const void* v, void* out_hidden, void* out_k, void* out_v, void* stream)
{
    ApiRange range("mvla_compact");
    const int32_t rc = mvla_compact_impl(ctx, batch, samples, kept_idx, out_offsets, total_kept, hidden, k, v, out_hidden, out_k, out_v, stream);
    if (log_enabled()) std::fprintf(stderr, "[mvla] mvla_compact(batch %lld) -> %d\n", static_cast<long long>(batch), rc);
    return rc;
}

int32_t mvla_patch_indicators(mvla_ctx* ctx, int32_t batch, const mvla_sample* samples, const void* q, const void* k,
                              const void* hidden, int64_t rows, float* attn_out, float* x_out, void* stream)
{
    ApiRange range("mvla_patch_indicators");
    const int32_t rc = mvla_patch_indicators_impl(ctx, batch, samples, q, k, hidden, rows, attn_out, x_out, stream);
    if (log_enabled()) std::fprintf(stderr, "[mvla] mvla_patch_indicators(batch %lld, rows %lld) -> %d\n", static_cast<long long>(batch), static_cast<long long>(rows), rc);
    return rc;
}

int32_t mvla_patch_select(mvla_ctx* ctx, int32_t prune_point, int32_t batch, const mvla_sample* samples, uint32_t flags,
                          const float* attn, const float* x, const float* rand_u, int32_t* kept_idx,
                          int32_t* out_offsets, int32_t* counts, float* xhat_out, int32_t* info_out,
                          mvla_patch_diag* diag, void* stream)
{
    ApiRange range("mvla_patch_select");
    const int32_t rc = mvla_patch_select_impl(ctx, prune_point, batch, samples, flags, attn, x, rand_u, kept_idx, out_offsets, counts, xhat_out, info_out, diag, stream);
    if (log_enabled()) std::fprintf(stderr, "[mvla] mvla_patch_select(prune_point %lld, batch %lld, flags %lld) -> %d\n", static_cast<long long>(prune_point), static_cast<long long>(batch), static_cast<long long>(flags), rc);
    return rc;
}

int32_t mvla_prune_step(mvla_ctx* ctx, int32_t prune_point, int32_t batch, const mvla_sample* samples,
                        int32_t mode, uint32_t flags, const mvla_tensors* in, const mvla_outputs* out,
                        int32_t* total_kept_out, void* stream)
{
    ApiRange range("mvla_prune_step");
    const int32_t rc = mvla_prune_step_impl(ctx, prune_point, batch, samples, mode, flags, in, out, total_kept_out, stream);
    if (log_enabled()) std::fprintf(stderr, "[mvla] mvla_prune_step(prune_point %lld, batch %lld, mode %lld, flags %lld, rows %lld) -> %d\n", static_cast<long long>(prune_point), static_cast<long long>(batch), static_cast<long long>(mode), static_cast<long long>(flags), static_cast<long long>(in ? in->rows : -1), rc);
    return rc;
}

}  // extern "C"
