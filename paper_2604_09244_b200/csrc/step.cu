// Tail of the fused prune step: carry-over, gates, budget split, top-k selection (Alg. 1 stages 1-4,
// Eqs. 8-10) AND the compaction of the surviving rows (Sec. 4.4) in one kernel.
//
// A step on one sample is a chain of latencies, not a bandwidth problem: a kernel boundary costs a
// microsecond or two, a device-wide fence about one.  Here one CTA per sample runs the selection and the
// other CTAs of the grid copy rows:
//   * while the scores are still being computed the copying CTAs move the text rows, whose output
//     positions the host knows;
//   * the selecting CTA writes every entry of the kept list as one 4-byte word into library scratch; a
//     copying warp polls the word of the row it is to move (-1: not yet known) and starts the moment the
//     word is there.  No fence, flag or barrier lies between the two roles: each word is its own signal;
//   * what nobody waits for (smoothed state, indicators and diagnostics when the budgets came from the
//     host, optional score outputs) is written after the list.
// The scoring kernel that runs before this one re-arms the words, so nothing is left to do at the end.
#include "common.cuh"
#include "device_utils.cuh"
#include "copy_impl.cuh"
#include "select_impl.cuh"

#include <algorithm>

namespace mvla {
namespace {

struct TailPlan {
    int16_t cta0[kMaxChunk + 1];      // first CTA of every sample; cta0[n] = grid size
};

// The same wait on a word that nothing ever sets, with a short limit: lets a test (or a health check) see
// the whole failure path -- the wait gives up, the kernel returns, the status word holds the error --
// without any kernel being made to hang.
__global__ void wait_probe_kernel(const int* never_set, uint64_t limit_ns, int* status)
{
    if (poll_word(never_set, global_ns(), limit_ns) < 0) *reinterpret_cast<volatile int*>(status) = MVLA_ERR_TIMEOUT;
}

// grid: CTAs 0 .. n-1 select (CTA b for sample b of the launch), the CTAs after them copy; tp.cta0[b] is the
// first copying CTA of sample b.  `list`: the kept list in library scratch (one word per output row of the
// launch's samples, -1 = not yet known; the scoring kernel before this one has set them all to -1).
// The roles go by block index.  The launcher never asks for more CTAs than fit on the device together
// (`ctas` = multiprocessors x CTAs per multiprocessor), and the kernel after this one cannot start before
// every CTA of this one has started, so all CTAs of the grid become resident whatever order they are
// dispatched in: a copying CTA never keeps its selecting CTA from running.  (Taking the roles in the order
// in which the CTAs start, by a ticket from an atomic counter as the patch-by-patch tail does, cost 0.4 us per
// step here: 296 atomics on one word.)  All waits are bounded all the same.
template <int NT, int CAP>
__global__ void __launch_bounds__(NT)
select_copy_kernel(const __grid_constant__ BatchDesc bd, const __grid_constant__ TailPlan tp, const GateParams gp,
                   const SelectIO io, const __grid_constant__ CompactArgs ca, int32_t* __restrict__ list, int* status,
                   unsigned long long* __restrict__ stamps)
{
    const int tid = threadIdx.x, lane = tid & 31;
    const int cta = blockIdx.x;
    if (cta < bd.n) {
        // ---- selection of one sample, by one CTA
        __shared__ SelectSmem<NT, CAP> sm;
        const int b = cta;
        SelectRole role;
        role.late_pdl = true;
        role.l1_late = true;                                // the norms may come from a kernel that ran beside the scoring
        if (tp.cta0[bd.n] > 0) role.kept_sm = list + bd.s[b].out_off;   // every word is its own "ready" signal
        select_sample<NT, CAP>(bd.s[b], b, gp, io, sm, role, [&]() {}, [&]() {
            if (stamps && tid == 0 && cta < kStampSlots) stamps[2 * cta + 1] = global_ns();
        });
        if (stamps && tid == 0 && cta < kStampSlots) stamps[2 * cta] = stamps[2 * cta + 1];   // placeholder start, see the copiers
        return;
    }
    // ---- row copy
    const int c = cta - bd.n;
    int b = 0;
    while (b + 1 < bd.n && c >= tp.cta0[b + 1]) ++b;
    const int part = c - tp.cta0[b], nparts = tp.cta0[b + 1] - tp.cta0[b];
    const SampleDev& s = bd.s[b];
    const int w = part * (NT / 32) + (tid >> 5), nw = nparts * (NT / 32);

    // Output position of the text rows: known on the host when the split is (FIXED budgets, cold start),
    // or when the text segment lies before or behind both visual segments (then only the total counts).
    const bool b2 = s.n_2d > 0 && s.off_2d < s.off_txt, b3 = s.n_3d > 0 && s.off_3d < s.off_txt;
    int baset = -1;
    if (s.k_2d_fixed >= 0) baset = (b2 ? s.k_2d_fixed : 0) + (b3 ? s.budget - s.k_2d_fixed : 0);
    else if (b2 == b3) baset = b2 ? s.budget : 0;
    const bool text_early = baset >= 0;
    if (text_early)                                         // while the scores are still being computed
        copy_rows(ca, s.n_txt, w, nw, lane, [&](int i, int64_t& srow, int64_t& drow) {
            srow = static_cast<int64_t>(s.seq_off) + s.off_txt + i;
            drow = static_cast<int64_t>(s.out_off) + baset + i;
            return true;
        });
    asm volatile("griddepcontrol.wait;" ::: "memory");      // keeps the chain of dependencies whole: the kernel after
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // this one may rely on the one before it being complete
    if (stamps && tid == 0 && cta < kStampSlots) stamps[2 * cta] = global_ns();

    {
        const int n_rows = s.n_out - (text_early ? s.n_txt : 0);
        const int32_t* kept = list + s.out_off;
        const uint64_t t0 = global_ns();
        copy_rows(ca, n_rows, w, nw, lane, [&](int i, int64_t& srow, int64_t& drow) {
            const int r = (text_early && i >= baset) ? i + s.n_txt : i;       // skip the text rows copied before
            const int v = poll_word(kept + r, t0, 1000000000ull);   // the whole warp reads one word: one request
            if (v < 0) {                                    // gave up: report, leave the row alone
                *reinterpret_cast<volatile int*>(status) = MVLA_ERR_TIMEOUT;
                return false;
            }
            srow = static_cast<int64_t>(s.seq_off) + v;
            drow = static_cast<int64_t>(s.out_off) + r;
            return true;
        });
    }
    if (stamps && cta < kStampSlots) {
        __syncthreads();
        if (tid == 0) stamps[2 * cta + 1] = global_ns();
    }
}

template <int NT, int CAP>
cudaError_t launch_t(const BatchDesc& bd, const TailPlan& tp, const GateParams& gp, const SelectIO& io, const CompactArgs& ca,
                     int32_t* list, int* status, unsigned long long* stamps, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(bd.n + tp.cta0[bd.n]));
    cfg.blockDim = dim3(NT);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, select_copy_kernel<NT, CAP>, bd, tp, gp, io, ca, list, status, stamps);
}

int max_vis_of(const BatchDesc& bd)
{
    int m = 0;
    for (int b = 0; b < bd.n; ++b) m = std::max(m, bd.s[b].n_2d + bd.s[b].n_3d);
    return m;
}

}  // namespace

bool select_copy_supported(const BatchDesc& bd) { return max_vis_of(bd) <= 2048; }

cudaError_t launch_wait_probe(const int32_t* never_set, uint64_t limit_ns, int* status, cudaStream_t stream)
{
    wait_probe_kernel<<<1, 32, 0, stream>>>(never_set, limit_ns, status);
    return cudaGetLastError();
}

cudaError_t launch_select_copy(const BatchDesc& bd, const GateParams& gp, const SelectIO& io, const CompactJob& job,
                               int32_t* list, int* status, int ctas, unsigned long long* stamps, cudaStream_t stream)
{
    if (bd.n < 1 || !select_copy_supported(bd)) return cudaErrorInvalidConfiguration;
    const CompactArgs ca = compact_args(job);
    TailPlan tp;
    int next = 0;
    if (ca.seg_begin[3] > 0) {
        // copying CTAs per sample in proportion to its kept rows (rounded down), at least one each, and never more
        // than `ctas` in all -- the grid must fit on the device at once, see the kernel -- unless there are more
        // samples than that
        ctas = std::min(std::max(ctas, bd.n), 30000);
        int64_t rows = 0;
        for (int b = 0; b < bd.n; ++b) rows += bd.s[b].n_out;
        int share[kMaxChunk];
        int total = 0;
        for (int b = 0; b < bd.n; ++b) {
            share[b] = static_cast<int>(std::max<int64_t>(1, rows > 0 ? static_cast<int64_t>(ctas) * bd.s[b].n_out / rows : 1));
            total += share[b];
        }
        while (total > ctas) {                               // the minimum of one pushed it over: take from the largest
            int big = 0;
            for (int b = 1; b < bd.n; ++b) big = share[b] > share[big] ? b : big;
            if (share[big] <= 1) break;
            --share[big];
            --total;
        }
        for (int b = 0; b < bd.n; ++b) {
            tp.cta0[b] = static_cast<int16_t>(next);
            next += share[b];
        }
    } else {
        for (int b = 0; b < bd.n; ++b) tp.cta0[b] = 0;       // nothing to copy: selection only
    }
    for (int b = bd.n; b <= kMaxChunk; ++b) tp.cta0[b] = static_cast<int16_t>(next);
    if (max_vis_of(bd) <= 1024) return launch_t<512, 1024>(bd, tp, gp, io, ca, list, status, stamps, stream);
    return launch_t<512, 2048>(bd, tp, gp, io, ca, list, status, stamps, stream);
}

}  // namespace mvla
