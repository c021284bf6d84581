// Internal declarations shared by the kernels and the C-ABI layer.
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "mvla_prune.h"

namespace mvla {

// Hand-over words of the patch-by-patch tail, per sample from word cap_off on: kHandLines lines of 32 words
// (identical copies, so that the copying CTAs do not all poll one line of the L2: word 0 "the list is about
// to be written", word 1 the sample's first output row), then one word per row of the sample.
constexpr int kHandLines = 8;
constexpr int kHandWords = kHandLines * 32;
constexpr int kMaxChunk = 32;        // samples carried by one launch (descriptors travel as kernel parameters)
constexpr int kKeyTile = 128;        // visual keys per tile = rows of one MMA
constexpr int kMaxCluster = 8;       // portable cluster size
constexpr int kMaxText = 64;
constexpr int kMaxVis = 4096;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr unsigned kStampSlots = 4096;      // CTAs per kernel that leave time stamps when asked to (mvla_set_kernel_stamps)   // bounded device-side waits (each try sleeps, see wait loops)

// Device-side view of one sample; everything the host can compute is computed there.
struct SampleDev {
    int32_t seq_off, off_txt, n_txt, off_2d, n_2d, off_3d, n_3d;
    int32_t vis_off;        // offset of the sample in packed [sum n_vis] arrays
    int32_t cap_off;        // sum of (kHandWords + n_txt + n_vis) over the samples before this one: its hand-over words in the patch-by-patch tail
    int32_t out_off;        // first output row
    int32_t n_out;          // kept rows = n_txt + budget
    int32_t budget;         // kept visual tokens (host known)
    int32_t k_2d_fixed;     // >= 0: host-decided split (FIXED mode or cold start); -1: split on device
    int32_t kmin_2d, kmin_3d;   // ADAPTIVE floors
    // The smoothed state of a (prune point, slot) is kept twice: step t reads the copy that step t - 1
    // wrote and writes the other one, so that several CTAs may read the previous state while one writes.
    int32_t state_off;      // per-token state array: offset of the copy this step READS
    int32_t state_off_w;    // ... and of the copy it WRITES
    int32_t mstate_off;     // indicator state array (x4 floats): index of the copy this step reads
    int32_t mstate_off_w;   // ... and writes
    int32_t slot_index;     // prune point * slots + slot: addresses the per-patch state (updated in place by one CTA)
    // reuse of the previous step's logits (Sec. 4.3 / 5.2); cache_state < 0: off for this sample
    int32_t cache_state;    // which (prune point, slot) block of the logit cache
    uint32_t tile_compute;  // bit t: key tile t must be computed from K (and its logits stored); clear: reuse the cached logits
    int32_t t;              // 1-based action step this call is
    int32_t update_state;   // 0: dry run
    float c_prev, c_new;    // state update weights: xhat = c_prev * xhat + c_new * x
};

struct BatchDesc {
    SampleDev s[kMaxChunk];
    int32_t n;
};

struct GateParams {
    float tau_2d, tau_3d, eps_3d;
    int32_t adaptive;       // mode
    int32_t has_l1;
};

// Scores arrive either as fp32 (`attn`), as per-head fp32 partials (`part`), or as 64-bit fixed-point
// sums over heads (`acc64`, scale 2^60, exact and order independent; cleared after reading).
struct SelectIO {
    const float* attn;
    const float* part;
    int64_t part_stride;
    int n_heads;
    unsigned long long* acc64;
    const float* l1;
    float* ahat_state;
    float* mhat_state;
    int32_t* kept_idx;
    int32_t* out_offsets;
    int32_t* budgets;
    float* attn_out;
    float* ahat_out;
    float* z_out;
    mvla_diag* diag;
    int32_t chunk_first;     // index of the launch's first sample in the whole batch
    int32_t total_out;
    int32_t write_total;     // this launch holds the batch's last sample
    int32_t n_in_launch;
};

// Launch attribute that lets a kernel begin before its stream predecessor has drained (the kernel
// itself waits with griddepcontrol.wait before it touches anything the predecessor wrote).
inline cudaLaunchAttribute pdl_attribute()
{
    cudaLaunchAttribute a = {};
    a.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    a.val.programmaticStreamSerializationAllowed = 1;
    return a;
}

// Multiprocessors of the current device (looked up once per device).
int sm_count_of_current_device();

// ---- launchers (each enqueues on `stream` and returns the launch status) ----

// bf16 tensor-core salience with logits held in registers (one or two key tiles per CTA).  With
// `acc64` the per-head contributions are added into 64-bit fixed-point accumulators (scale 2^60, one
// per visual token, zero on entry); without it they go to part[h][vis] as in launch_salience (nowhere when
// `part` is null too: only the attention copy is wanted).
// `free_running`: the kernel does not wait for the kernel before it in its stream (the caller orders
// everything it depends on with events).
// `lcache`: logit cache [state][head][cache_vis][cache_cols] fp32 (raw dot products), or null; which tiles are
// computed and stored and which are read back is in the descriptors (cache_state, tile_compute).
// `stamps`: when not null, CTA c (linear index, below kStampSlots) writes the global timer when it was free to
// start its loads to stamps[2 c] and when it ended to stamps[2 c + 1].
// `rearm`: when not null, words [out_off, out_off + n_out) of every sample are set to -1 (the kept list that
// launch_select_copy's CTAs exchange, see there).  With `rearm_rec` (the patch-by-patch tail, launch_patch_tail)
// it is words [cap_off, cap_off + kHandWords + n_txt + n_vis) instead, and the three 8-byte words of every patch in
// `rearm_rec` ([vis_off / 2 + p][3]) are set to all ones.
// Optional copy of the attention itself for the patch-by-patch path, the text queries of a (head, token)
// next to one another (what the scoring kernel's thread holds, and what the indicators of a patch read):
// ptr[(h * stride_h) + (vis_off + j) * stride_j + i] = alpha[h, i, j]   (null: not written).
// stride_j is a multiple of 4 and ptr 16-byte aligned; entries i in [n_txt, stride_j) may be overwritten.
struct AlphaOut {
    float* ptr;
    int64_t stride_h, stride_j;
};

bool fast_salience_supported(int tiles_per_cta);
// `kv_group`: query heads per key head (1 unless the keys are grouped); the key tensor map then has
// n_heads / kv_group heads.
// `esize`: bytes per element of q and k (2: bf16, 1: e4m3).
cudaError_t launch_salience_fast(const BatchDesc& bd, int n_heads, int kv_group, int head_dim, int esize, const CUtensorMap* tmap_q,
                                 const CUtensorMap* tmap_k, int tiles_per_cta, int cluster, int npad,
                                 float* part, int64_t part_stride, unsigned long long* acc64, int* status,
                                 bool free_running, AlphaOut alpha, int32_t* rearm, unsigned long long* rearm_rec, unsigned long long* stamps,
                                 float* lcache, int cache_vis, int cache_cols, cudaStream_t stream);


// Salience: per-head partial scores part[h][vis] (already scaled by 1/(H n_t)).
// `use_umma`: tensor-core path (bf16 only).  tmaps: device-usable tensor maps (passed by value).
cudaError_t launch_salience(const BatchDesc& bd, int dtype, int n_heads, int kv_group, int head_dim,
                            const void* q, const void* k, const CUtensorMap* tmap_q,
                            const CUtensorMap* tmap_k, bool use_umma, int tiles_per_cta,
                            int cluster, int npad, float* part, int64_t part_stride,
                            int* status, AlphaOut alpha, cudaStream_t stream);

// attn[j] = sum_h part[h][j]  (fixed head order).
cudaError_t launch_head_reduce(const float* part, int64_t part_stride, int n_heads, int total_vis,
                               float* attn, cudaStream_t stream);

// L1 feature norms of the visual rows.  `beside_predecessor`: the kernel is launched right after a scoring
// kernel that releases its dependents only once ITS predecessor is complete (launch_salience_fast): it then
// runs beside the scoring kernel and completes after it.
cudaError_t launch_l1norm(const BatchDesc& bd, int dtype, int d_model, const void* hidden,
                          float* l1, bool beside_predecessor, cudaStream_t stream);

// Carry-over + budget + top-k + emission; one CTA per sample (io.n_in_launch = bd.n).
cudaError_t launch_select(const BatchDesc& bd, const GateParams& gp, const SelectIO& io, cudaStream_t stream);

// Row gather of up to three tensors.
struct CompactJob {
    const void* src[3];
    void* dst[3];
    int32_t row_bytes[3];
};
// The same as the kernels see it: rows cut into 2 KB segments (one warp moves one segment).
constexpr int kSegBytes = 2048;     // 32 lanes x 4 x 16 B
struct CompactArgs {
    const uint8_t* src[3];
    uint8_t* dst[3];
    int32_t row_bytes[3];
    int32_t segs[3];          // 2 KB segments per row
    int32_t seg_begin[4];     // prefix sums of segs per row over the (up to) three tensors
};
inline CompactArgs compact_args(const CompactJob& job)
{
    CompactArgs a;
    int total = 0;
    for (int i = 0; i < 3; ++i) {
        const bool on = job.src[i] && job.dst[i];
        a.src[i] = static_cast<const uint8_t*>(job.src[i]);
        a.dst[i] = static_cast<uint8_t*>(job.dst[i]);
        a.row_bytes[i] = job.row_bytes[i];
        a.segs[i] = on ? (job.row_bytes[i] + kSegBytes - 1) / kSegBytes : 0;
        a.seg_begin[i] = total;
        total += a.segs[i];
    }
    a.seg_begin[3] = total;
    return a;
}
// Rows [chunk_row0, chunk_row0 + chunk_rows) of the output.  With `out_offsets` (device) the owning
// sample of a row is looked up there over the whole batch and rows of samples outside this launch's
// descriptors are skipped; without it the descriptors' host-computed out_off is used.
cudaError_t launch_compact(const BatchDesc& bd, const CompactJob& job, const int32_t* kept_idx,
                           int32_t chunk_rows, int32_t chunk_row0, const int32_t* out_offsets,
                           int32_t chunk_first, int32_t batch_total, cudaStream_t stream);

// Tail of the fused step for samples of up to 2048 visual tokens: carry-over + budget + top-k (as in
// launch_select) AND the row copy in one kernel.  One CTA per sample selects; the other CTAs copy the
// text rows at once, then take the kept rows word by word from `list` as the selecting CTA writes them
// (bounded waits, MVLA_ERR_TIMEOUT into `status` when one runs out): no kernel boundary, fence or flag lies
// between selection and copy.  `list`: one int per output row of the batch, all -1 when the kernel starts
// (the scoring kernel before it re-arms them, see launch_salience_fast).
// `ctas`: copying CTAs to aim for (every sample gets at least one); together with the selecting CTAs no more than
// fit on the device at once, see the kernel.  `stamps`: as in launch_salience_fast
// (start: past the wait for the kernel before; the selecting CTA's end is when the list is written).
bool select_copy_supported(const BatchDesc& bd);
cudaError_t launch_select_copy(const BatchDesc& bd, const GateParams& gp, const SelectIO& io, const CompactJob& job,
                               int32_t* list, int* status, int ctas, unsigned long long* stamps, cudaStream_t stream);

// One warp runs the copying CTAs' bounded wait on `never_set` (a word that holds -1 and stays so) with the
// given limit and reports MVLA_ERR_TIMEOUT into `status` when it runs out.
cudaError_t launch_wait_probe(const int32_t* never_set, uint64_t limit_ns, int* status, cudaStream_t stream);

// ---- patch-by-patch path (Alg. 1 taken literally) ----
struct PatchParams {
    double tau_2d, tau_3d, eps_3d, obj_2d_min, bg_prune_prob;
    int32_t kmeans_max_iter;
    int32_t cold_start_full_keep;
    int32_t max_patch;       // stride (in patches) of one (prune point, slot) in the per-patch state
};
struct PatchIO {
    const float* attn;       // [sum 2P] per-token scores
    const float* x;          // [sum P][4] instantaneous indicators
    const float* rand_u;     // [sum P]
    float* xhat_state;       // [points * slots][max_patch][4]
    float* xhat_out;         // nullable
    int32_t* info_out;       // nullable
    mvla_patch_diag* diag;   // nullable
    int32_t* counts;         // [batch][2] nullable
    int32_t* nout_ws;        // [batch] kept rows per sample (scratch)
    int32_t* ready_ws;       // [batch] "count published" flags, zero between launches
    int32_t* done_ws;        // CTAs of the launch that have finished waiting, zero between launches
    int* status;             // word that receives MVLA_ERR_TIMEOUT when a bounded wait gives up
    int32_t* kept_idx;
    int32_t* out_offsets;
    int32_t chunk_first, batch_total;
};
// x[p] = per-patch indicators from the attention copy and the L1 norms of the hidden rows; attn = per-token scores.
cudaError_t launch_patch_indicators(const BatchDesc& bd, int n_heads, AlphaOut alpha, int dtype, int d_model,
                                    const void* hidden, float* x_out, float* attn_out, cudaStream_t stream);
// Stages 1-4 of Alg. 1 for every patch, output offsets over the batch, ordered kept-position lists.
cudaError_t launch_patch_select(const BatchDesc& bd, const PatchParams& pp, const PatchIO& io, cudaStream_t stream);
// Indicators, stages 1-4 and the row copy of the patch-by-patch step in one kernel behind the scoring kernel
// (which must have re-armed `list` and `rec`, see launch_salience_fast).  `rec`: [sum P][3] 8-byte words;
// `list`: 4-byte words, kHandWords + n_txt + n_vis per sample from cap_off on.  io.x / io.attn are not read.
// `ticket_counter`: one word, zero before the first launch, used by one launch at a time (it returns to zero with
// every launch): the CTAs take their roles in the order in which they start (copy_impl.cuh: cta_ticket).
bool patch_tail_supported(const BatchDesc& bd);
cudaError_t launch_patch_tail(const BatchDesc& bd, int n_heads, AlphaOut alpha, int dtype, int d_model, const void* hidden,
                              float* x_out, float* attn_out, unsigned long long* rec, const PatchParams& pp, const PatchIO& io,
                              const CompactJob& job, int32_t* list, int sm_count, unsigned int* ticket_counter, cudaStream_t stream);

}  // namespace mvla
