// Tail of the patch-by-patch step (Alg. 1 taken literally) as ONE kernel after the scoring kernel:
//   * CTAs [0, n_ind): indicators of a block of patches each (Eq. 3-1, Eq. 3-4, Eq. P2D, Eq. P3D) from the
//     attention copy that the scoring kernel left in L2; each patch's result also goes, as three 8-byte
//     words, to the CTA that runs the stages after it;
//   * one CTA per sample: temporal predictor, dual threshold, K-Means, semantic rules, fusion, masks
//     (stages 1-4), reading each patch's words as they appear; it writes the kept list as 4-byte words;
//   * the remaining CTAs copy the surviving rows, each warp polling the word of the row it is to move.
// No kernel boundary, fence or flag lies between the three roles: every word is its own signal, re-armed
// (all ones) by the scoring kernel of the same step.  The roles go by ticket (cta_ticket: the order in which the
// CTAs started), so a consumer only ever waits for CTAs that are already running; every wait is bounded all the same.
#include "copy_impl.cuh"
#include "patch_impl.cuh"

#include <algorithm>

namespace mvla {
namespace {

constexpr int kTailThreads = kIndThreads;

struct PatchTailPlan {
    int16_t ind0[kMaxChunk + 1];      // first indicator CTA of every sample; ind0[n] = their number
    int16_t cta0[kMaxChunk + 1];      // first copying CTA of every sample (counted from 0); cta0[n] = their number
};

template <typename T, int PP>
__global__ void __launch_bounds__(kTailThreads, 1)
patch_tail_kernel(const __grid_constant__ BatchDesc bd, const __grid_constant__ PatchTailPlan tp, int n_heads,
                  const AlphaOut alpha, const T* __restrict__ hidden, int d_model, float* __restrict__ x_out,
                  float* __restrict__ attn_out, unsigned long long* rec, const PatchParams pp, const PatchIO io,
                  const __grid_constant__ CompactArgs ca, int32_t* list, unsigned int* ticket_counter)
{
    const int n_ind = tp.ind0[bd.n];
    int c = cta_ticket(ticket_counter);
    if (c < n_ind) {
        int b = 0;
        while (b + 1 < bd.n && c >= tp.ind0[b + 1]) ++b;
        patch_indicators_block<T, PP>(bd.s[b], c - tp.ind0[b], n_heads, alpha, hidden, d_model, x_out, attn_out, rec, true);
        return;
    }
    c -= n_ind;
    if (c < bd.n) {
        __shared__ PatchSmemT<kTailThreads> sm;
        const SampleDev& s = bd.s[c];
        const bool copying = tp.cta0[bd.n] > 0;
        patch_select_block<kTailThreads>(s, c, bd.n, pp, io, sm, rec, copying ? list + s.cap_off : nullptr);
        return;
    }
    // ---- row copy
    c -= bd.n;
    int b = 0;
    while (b + 1 < bd.n && c >= tp.cta0[b + 1]) ++b;
    const SampleDev& s = bd.s[b];
    const int tid = threadIdx.x, lane = tid & 31;
    const int part = c - tp.cta0[b], nparts = tp.cta0[b + 1] - tp.cta0[b];
    const int w = part * (kTailThreads / 32) + (tid >> 5), nw = nparts * (kTailThreads / 32);
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the words were re-armed by the kernel before this one
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // One warp of the CTA waits, at a low rate, for the hint that the list is about to be written and for the
    // sample's first output row (its own copy of both); only then do all warps poll the words of their rows.
    // Thousands of warps polling while the selecting CTA works would slow that CTA's own memory traffic.
    __shared__ int s_first, s_rows;
    const int32_t* words = list + s.cap_off;
    const uint64_t t0 = global_ns();
    constexpr uint64_t kLimitNs = 1000000000ull;
    if (tid < 32) {
        const int32_t* mine = words + 32 * (part % kHandLines);
        int hint = -1, first = -1, n_rows = -1;
        for (uint32_t it = 0; it < kSpinLimit; ++it) {
            if (hint < 0) hint = ld_relaxed_gpu(mine);
            if (hint >= 0 && first < 0) first = ld_relaxed_gpu(mine + 1);
            if (first >= 0) n_rows = ld_relaxed_gpu(mine + 2);
            if (n_rows >= 0) break;
            if ((it & 63u) == 63u && global_ns() - t0 > kLimitNs) break;
            __nanosleep(hint < 0 ? 200 : 40);
        }
        if (lane == 0) { s_first = first; s_rows = n_rows; }
    }
    __syncthreads();
    const int out_off = s_first, n_rows = s_rows;           // first output row of the sample, rows it keeps
    if (out_off < 0 || n_rows < 0) {
        if (tid == 0) *reinterpret_cast<volatile int*>(io.status) = MVLA_ERR_TIMEOUT;
        return;
    }
    words += kHandWords;
    copy_rows(ca, n_rows, w, nw, lane, [&](int i, int64_t& srow, int64_t& drow) {
        const int v = poll_word(words + i, t0, kLimitNs);     // the whole warp reads one word: one request
        if (v < 0) {                                                   // gave up: report, leave the row alone
            *reinterpret_cast<volatile int*>(io.status) = MVLA_ERR_TIMEOUT;
            return false;
        }
        srow = static_cast<int64_t>(s.seq_off) + v;
        drow = static_cast<int64_t>(out_off) + i;
        return true;
    });
}

}  // namespace

bool patch_tail_supported(const BatchDesc& bd)
{
    int blocks = 0;
    for (int b = 0; b < bd.n; ++b) blocks += (bd.s[b].n_2d + 1) / 2;
    return bd.n >= 1 && blocks + bd.n < 30000;
}

cudaError_t launch_patch_tail(const BatchDesc& bd, int n_heads, AlphaOut alpha, int dtype, int d_model, const void* hidden,
                              float* x_out, float* attn_out, unsigned long long* rec, const PatchParams& pp, const PatchIO& io,
                              const CompactJob& job, int32_t* list, int sm_count, unsigned int* ticket_counter, cudaStream_t stream)
{
    if (!patch_tail_supported(bd)) return cudaErrorInvalidConfiguration;
    // as many patches per CTA as still give every multiprocessor a CTA
    int per = 8;
    auto blocks_at = [&](int p) {
        int n = 0;
        for (int b = 0; b < bd.n; ++b) n += (bd.s[b].n_2d + p - 1) / p;
        return n;
    };
    while (per > 2 && blocks_at(per) < sm_count) per >>= 1;
    PatchTailPlan tp;
    int next = 0;
    for (int b = 0; b < bd.n; ++b) {
        tp.ind0[b] = static_cast<int16_t>(next);
        next += (bd.s[b].n_2d + per - 1) / per;
    }
    for (int b = bd.n; b <= kMaxChunk; ++b) tp.ind0[b] = static_cast<int16_t>(next);
    const CompactArgs ca = compact_args(job);
    int copiers = 0;
    if (ca.seg_begin[3] > 0) {
        // copying CTAs per sample in proportion to the rows it may keep, at least one each; together with the
        // selecting CTAs they fill the multiprocessors once the indicator CTAs have retired
        const int want = std::max(sm_count - bd.n, bd.n);
        int64_t rows = 0;
        for (int b = 0; b < bd.n; ++b) rows += bd.s[b].n_txt + bd.s[b].n_2d + bd.s[b].n_3d;
        for (int b = 0; b < bd.n; ++b) {
            tp.cta0[b] = static_cast<int16_t>(copiers);
            const int64_t mine = bd.s[b].n_txt + bd.s[b].n_2d + bd.s[b].n_3d;
            copiers += static_cast<int>(std::max<int64_t>(1, (static_cast<int64_t>(want) * mine + rows / 2) / std::max<int64_t>(rows, 1)));
        }
    } else {
        for (int b = 0; b < bd.n; ++b) tp.cta0[b] = 0;
    }
    for (int b = bd.n; b <= kMaxChunk; ++b) tp.cta0[b] = static_cast<int16_t>(copiers);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(next + bd.n + copiers));
    cfg.blockDim = dim3(kTailThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
#define MVLA_TAIL(T, PPV)                                                                                     \
    if (per == PPV)                                                                                           \
        return cudaLaunchKernelEx(&cfg, patch_tail_kernel<T, PPV>, bd, tp, n_heads, alpha,                    \
                                  static_cast<const T*>(hidden), d_model, x_out, attn_out, rec, pp, io, ca, list, ticket_counter);
    if (dtype == MVLA_DTYPE_BF16) { MVLA_TAIL(__nv_bfloat16, 8) MVLA_TAIL(__nv_bfloat16, 4) MVLA_TAIL(__nv_bfloat16, 2) }
    else { MVLA_TAIL(float, 8) MVLA_TAIL(float, 4) MVLA_TAIL(float, 2) }
#undef MVLA_TAIL
    return cudaErrorInvalidConfiguration;
}

}  // namespace mvla
