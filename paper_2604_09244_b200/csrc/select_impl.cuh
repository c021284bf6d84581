// Carry-over, budget split and top-k selection of ONE sample by one CTA of NT threads
// (Alg. 1 of the paper, stages 1-4; Eqs. 8, 9, 10).
//
// The work is a few KB, so the kernel is a chain of latencies; it is written around the number of
// block-wide barriers on that chain (five on the usual path):
//   1. every thread issues ALL its global loads (scores, previous state, norms) before any dependent
//      work, then smooths the scores (Eq. 8 / Eq. 9 as  xhat = c_prev xhat + c_new x) and builds
//      order-preserving 32-bit keys, kept in registers.  Each warp leaves its partial sums and the
//      smallest and largest key of each modality in shared memory                        [barrier A]
//   2. modality sums -> the four indicators, smoothed too; dual threshold (Sec. 4.1), target-object
//      rule (Sec. 4.2), fusion (Sec. 4.4), budget split: one thread, while the others already count
//      their keys into a histogram of 1024 bins per modality laid over the RANGE of the keys
//      (bin = (key - smallest) >> shift), so one pass separates a few hundred scores     [barrier B]
//   3. one warp per modality finds the bin that holds the k-th largest key (two 32-way scans)
//                                                                                         [barrier C]
//   4. keys in higher bins are kept, keys in lower bins dropped.  The few keys inside the bin are
//      ranked against one another by (key, lower index first) from a short list          [barrier D];
//      a crowded bin is split again with a finer histogram (only then: more barriers); keys that
//      are all equal are ranked by index during the emission;
//   5. emission merged with all text positions: warp ballots rank the kept tokens, the per-warp
//      counts meet in shared memory                                                       [barrier E]
#pragma once

#include "common.cuh"

#include <math_constants.h>

namespace mvla {

constexpr float kFixScale = 1152921504606846976.f;          // 2^60
constexpr float kFixInv = 1.f / 1152921504606846976.f;      // 2^-60, exact

constexpr int kSelBins = 1024;      // histogram bins per modality
constexpr int kSelBinBits = 10;
constexpr int kCandMax = 32;        // keys of the threshold bin ranked from a list; above that the bin is split again

// what happens to the keys of the threshold bin of a modality
enum : int {
    SEL_NONE = 0,     // budget 0: nothing is kept
    SEL_ALL = 1,      // budget = count: everything is kept
    SEL_BIN_ALL = 2,  // higher bins and the whole threshold bin are kept
    SEL_LIST = 3,     // threshold bin ranked from the candidate list
    SEL_TIES = 4,     // threshold bin holds equal keys only: the first `need` of them by index are kept
    SEL_REFINE = 5,   // threshold bin crowded: another histogram over its range
};

// Cost model behind the layout below: on this chain a shuffle, a shared-memory access or a shared-memory
// atomic costs a warp about 20 cycles whether or not anything else runs, so what is counted is the number
// of such instructions a warp issues between two barriers, and 16-byte accesses are used wherever possible.
template <int NT, int CAP = kMaxVis>
struct SelectSmem {
    // bin r (0 = largest keys) of lane r / 32 lives at hist_pos(r): the 32 bins of a lane are eight int4, and
    // for each of the eight the 32 lanes read consecutive int4 (no bank conflict)
    alignas(16) int hist[2][kSelBins];
    alignas(16) float red[NT / 32][8];       // per-warp partial sums: scores 2D, 3D; norms 2D, 3D; smoothed scores 2D, 3D
    alignas(16) uint32_t ext[NT / 32][4];    // per-warp smallest / largest key: min 2D, max 2D, min 3D, max 3D
    alignas(16) uint32_t cand_key[2][kCandMax];
    alignas(16) int cand_idx[2][kCandMax];
    int cand_rank[2][kCandMax];              // rank of every listed key among the listed keys of its modality
    alignas(16) int ctl[8];                  // mode 2D, 3D; threshold bin 2D, 3D; keys to take from it 2D, 3D; budgets 2D, 3D
    int wtot[CAP / NT][NT / 32];             // emission: kept tokens (low half) and index-ranked ties (high half) per slice and warp
    int ncand[2];
    int krem[2];                             // still to be taken from the keys under examination
    float zf[2];                             // factors of the optional normalised scores
};
__device__ __forceinline__ int hist_pos(int r)
{
    return (((r & 31) >> 2) << 7) + ((r >> 5) << 2) + (r & 3);
}

// fp32 -> uint32 whose unsigned order is the float order; NaN sorts below everything.
__device__ __forceinline__ uint32_t order_key(float x)
{
    if (x != x) return 0u;
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

__device__ __forceinline__ int warp_incl_scan(int x, int lane)
{
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, x, off);
        if (lane >= off) x += n;
    }
    return x;
}

// Sums 8 per-thread values over the 32 lanes of a warp in 9 shuffles (a butterfly that halves the number
// of values a lane carries at each of its first three stages).  On return the lanes whose bits 4..2 spell
// c hold the sum of column c.  The order of the additions is fixed.
__device__ __forceinline__ float warp_sum8(float (&v)[8], int lane)
{
#pragma unroll
    for (int w = 4; w >= 1; w >>= 1) {
        const int off = w * 4;                               // 16, 8, 4
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < w; ++i) {
            const float send = up ? v[i] : v[i + w];
            const float keep = up ? v[i + w] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    v[0] += __shfl_xor_sync(0xffffffffu, v[0], 2);
    v[0] += __shfl_xor_sync(0xffffffffu, v[0], 1);
    return v[0];
}

// Exclusive block scan of one int per thread (used by the patch-by-patch emission).
template <int NT>
__device__ __forceinline__ int block_exscan(int x, int* warp_tot, int* total)
{
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int inc = warp_incl_scan(x, lane);
    __syncthreads();                                       // previous users of warp_tot are done
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int t = lane < NW ? warp_tot[lane] : 0;
        const int winc = warp_incl_scan(t, lane);
        if (lane < NW) warp_tot[lane] = winc - t;          // exclusive prefix of the warp totals
        if (lane == 31) warp_tot[NW] = winc;               // grand total
    }
    __syncthreads();
    *total = warp_tot[NW];
    return warp_tot[warp] + inc - x;
}

// How one CTA takes part in the selection of a sample.
//   leader   : this CTA writes the global results (kept list, budgets, smoothed state, diagnostics).  Several
//              CTAs may run the same selection redundantly (each needs the kept list for its share of the
//              row copy); exactly one of them is the leader.
//   kept_sm  : optional copy of the kept list in shared memory (n_txt + budget entries).
//   clear_acc: zero the fixed-point accumulators after reading them (only when a single CTA reads them).
//   late_pdl : false: the next kernel in the stream may become resident right away and the loads of the
//              previous state and of the norms follow griddepcontrol.wait; true: those loads come first
//              (the caller guarantees that they were written before this kernel could start), `before_wait`
//              runs, and the next kernel is released only after the wait.
//   l1_late  : with late_pdl: the norms come from the kernel right before this one after all (loaded after the wait).
struct SelectRole {
    bool leader = true;
    int32_t* kept_sm = nullptr;
    bool clear_acc = true;
    bool late_pdl = false;
    bool l1_late = false;
};
struct NoHook {
    __device__ void operator()() const {}
};

// One warp: the bin that holds the k-th largest of the keys counted in `h` (1 <= k <= number counted).
__device__ __forceinline__ void find_threshold_bin(const int* h, int k, int lane, int& tbin, int& need, int& cnt)
{
    const int4* h4 = reinterpret_cast<const int4*>(h);
    int mine = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {                                      // bins 32 lane .. 32 lane + 31
        const int4 v = h4[(i << 5) + lane];
        mine += (v.x + v.y) + (v.z + v.w);
    }
    const int inc = warp_incl_scan(mine, lane);
    const unsigned hit = __ballot_sync(0xffffffffu, inc - mine < k && k <= inc);
    const int L = max(__ffs(hit) - 1, 0);
    const int above_l = __shfl_sync(0xffffffffu, inc - mine, L);
    const int c = h[hist_pos(32 * L + lane)];                          // the 32 bins of that lane, one per lane
    const int inc2 = warp_incl_scan(c, lane);
    const int above = above_l + inc2 - c;
    const unsigned hit2 = __ballot_sync(0xffffffffu, above < k && k <= above + c);
    const int i = max(__ffs(hit2) - 1, 0);
    tbin = 32 * L + i;
    need = k - __shfl_sync(0xffffffffu, above, i);
    cnt = __shfl_sync(0xffffffffu, c, i);
}

// `before_wait` runs ahead of the wait for the previous kernel (late_pdl only); `after_list` runs as soon as
// the kept list is written, before the bookkeeping that nobody downstream waits for (smoothed state,
// indicators and diagnostics when the budgets came from the host, optional score outputs).
template <int NT, int CAP = kMaxVis, class Hook = NoHook, class After = NoHook>
__device__ __forceinline__ void select_sample(const SampleDev& s, int b_local, const GateParams& gp, const SelectIO& io,
                                              SelectSmem<NT, CAP>& sm, const SelectRole role = SelectRole(),
                                              Hook before_wait = Hook(), After after_list = After())
{
    constexpr int EPT = CAP / NT;                         // elements per thread, strided by NT
    constexpr int NW = NT / 32;
    static_assert(EPT >= 1 && EPT * NT == CAP, "thread count must divide the capacity");
    static_assert(EPT * NW <= 128, "the emission prefix is taken by one warp, four entries per lane");
    static_assert((2 * kCandMax * 8) % NT == 0 || NT % (2 * kCandMax * 8) == 0, "whole warps rank the listed keys");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n2 = s.n_2d, n3 = s.n_3d, nv = n2 + n3;
    const int b_glob = io.chunk_first + b_local;
    const bool carry = s.c_prev != 0.f;
    const bool leader = role.leader;
    const bool k_fixed = s.k_2d_fixed >= 0;               // budgets decided on the host (FIXED mode, cold start)
    // The modality sums feed the indicators.  With host-decided budgets only the leader needs them (for the
    // smoothed state and the diagnostics), and it takes them after the selection, off everyone's chain.
    const bool want_sums = leader || !k_fixed;

    // prologue that needs nothing from the previous kernel
    if (!role.late_pdl) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int i = tid; i < 2 * kSelBins / 4; i += NT) reinterpret_cast<int4*>(&sm.hist[0][0])[i] = make_int4(0, 0, 0, 0);
    if (tid < 2) {
        sm.ncand[tid] = 0;
        if (k_fixed) sm.ctl[6 + tid] = tid == 0 ? s.k_2d_fixed : s.budget - s.k_2d_fixed;
    }
    float a[EPT], prev[EPT], nrm[EPT];
    unsigned long long fx[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) { a[e] = 0.f; prev[e] = 0.f; nrm[e] = 0.f; fx[e] = 0ull; }
    if (role.late_pdl) {
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (e * NT >= nv) break;
            const int j = tid + e * NT;
            if (j < nv) {
                if (carry) prev[e] = io.ahat_state[s.state_off + j];
                if (gp.has_l1 && want_sums && !role.l1_late) nrm[e] = io.l1[s.vis_off + j];
            }
        }
        before_wait();
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");      // scores come from the kernel before this one

    // ---- 1. all loads first
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        if (e * NT >= nv) break;                           // uniform: nobody owns an element in this slice
        const int j = tid + e * NT;
        if (j < nv) {
            if (io.acc64) fx[e] = __ldcg(io.acc64 + s.vis_off + j);        // written by other CTAs' atomics
            else if (!io.part) a[e] = io.attn[s.vis_off + j];
            if (!role.late_pdl) {
                if (carry) prev[e] = io.ahat_state[s.state_off + j];
                if (gp.has_l1 && want_sums) nrm[e] = io.l1[s.vis_off + j];
            } else if (role.l1_late) {
                if (gp.has_l1 && want_sums) nrm[e] = io.l1[s.vis_off + j];
            }
        }
    }
    if (io.part && !io.acc64) {                            // per-head fp32 partials, summed in head order
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (e * NT >= nv) break;
            const int j = tid + e * NT;
            if (j < nv) {
                float acc = 0.f;
#pragma unroll 8
                for (int h = 0; h < io.n_heads; ++h) acc += io.part[static_cast<int64_t>(h) * io.part_stride + s.vis_off + j];
                a[e] = acc;
            }
        }
    }
    // (no array below is indexed with a run-time value: such an array would live in local memory, and every
    //  first touch of a local-memory line is a round trip to L2 on this latency chain)
    uint32_t key[EPT];
    float sums[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};   // scores 2D, 3D; norms 2D, 3D; smoothed scores 2D, 3D
    uint32_t mn2 = 0xFFFFFFFFu, mn3 = 0xFFFFFFFFu, mx2 = 0u, mx3 = 0u;
#pragma unroll
    for (int e = 0; e < EPT; ++e) key[e] = 0u;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        if (e * NT >= nv) break;
        const int j = tid + e * NT;
        if (j < nv) {
            if (io.acc64) {
                a[e] = __ull2float_rn(fx[e]) * kFixInv;   // one rounding: the exact head sum to fp32
                if (role.clear_acc) io.acc64[s.vis_off + j] = 0ull;    // ready for the next call
            }
            const float smo = carry ? fmaf(s.c_prev, prev[e], s.c_new * a[e]) : a[e];
            key[e] = order_key(smo);
            if (j < n2) {
                sums[0] += a[e]; sums[2] += nrm[e]; sums[4] += smo;
                mn2 = min(mn2, key[e]); mx2 = max(mx2, key[e]);
            } else {
                sums[1] += a[e]; sums[3] += nrm[e]; sums[5] += smo;
                mn3 = min(mn3, key[e]); mx3 = max(mx3, key[e]);
            }
        }
    }
    // Per-warp key extremes, and (where wanted) partial sums with a fixed order of additions, so that every
    // CTA that repeats this selection gets the same bits.
    mn2 = __reduce_min_sync(0xffffffffu, mn2); mx2 = __reduce_max_sync(0xffffffffu, mx2);
    mn3 = __reduce_min_sync(0xffffffffu, mn3); mx3 = __reduce_max_sync(0xffffffffu, mx3);
    if (lane == 0) *reinterpret_cast<uint4*>(sm.ext[warp]) = make_uint4(mn2, mx2, mn3, mx3);
    if (!k_fixed) {                                           // block-uniform: the budgets need the indicators
        const float col = warp_sum8(sums, lane);
        if ((lane & 3) == 0) sm.red[warp][lane >> 2] = col;
    }
    __syncthreads();                                                                       // ---- barrier A

    // range of the keys of each modality; shift < 0: all keys equal (or none)
    uint32_t lo2, lo3;
    int sh2, sh3;
    {
        uint4 x4 = make_uint4(0xFFFFFFFFu, 0u, 0xFFFFFFFFu, 0u);
        if (lane < NW) x4 = *reinterpret_cast<const uint4*>(sm.ext[lane]);
        lo2 = __reduce_min_sync(0xffffffffu, x4.x);
        const uint32_t hi2 = __reduce_max_sync(0xffffffffu, x4.y);
        lo3 = __reduce_min_sync(0xffffffffu, x4.z);
        const uint32_t hi3 = __reduce_max_sync(0xffffffffu, x4.w);
        sh2 = hi2 > lo2 ? max(0, (32 - __clz(hi2 - lo2)) - kSelBinBits) : -1;       // (key - lo) >> shift < 1024
        sh3 = hi3 > lo3 ? max(0, (32 - __clz(hi3 - lo3)) - kSelBinBits) : -1;
    }

    // ---- 2. indicators, gates, budget.  One warp: lane c adds column c of the per-warp partials in warp
    //         order; lane 0 collects the six totals and does the few dozen flops.  With device-decided budgets
    //         this runs now (the threshold search needs the budgets) beside the histogram of the other warps;
    //         with host-decided budgets the leader runs it at the very end.
    auto indicators = [&]() {
        float t = 0.f;
        if (lane < 8)
            for (int w = 0; w < NW; ++w) t += sm.red[w][lane];
        const float t0 = __shfl_sync(0xffffffffu, t, 0), t1 = __shfl_sync(0xffffffffu, t, 1);
        const float t2 = __shfl_sync(0xffffffffu, t, 2), t3 = __shfl_sync(0xffffffffu, t, 3);
        const float t4 = __shfl_sync(0xffffffffu, t, 4), t5 = __shfl_sync(0xffffffffu, t, 5);
        if (lane != 0) return;
        float x[4];
        x[3] = t1 / (t0 + t1);                                            // attention share of 3D (Eq. P2D / P3D); IEEE division: a share of an only modality is exactly 1
        x[2] = 1.f - x[3];
        if (gp.has_l1) {                                          // feature-norm share (Eq. 3-1), mean norms
            const float m2 = n2 > 0 ? t2 / static_cast<float>(n2) : 0.f;
            const float m3 = n3 > 0 ? t3 / static_cast<float>(n3) : 0.f;
            x[1] = m3 / (m2 + m3);
            x[0] = 1.f - x[1];
        } else {
            x[0] = x[1] = 0.5f;
        }
        float mh[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            mh[c] = carry ? fmaf(s.c_prev, io.mhat_state[s.mstate_off * 4 + c], s.c_new * x[c]) : x[c];
            if (s.update_state && leader) io.mhat_state[s.mstate_off_w * 4 + c] = mh[c];
        }
        const int c1 = mh[1] < gp.tau_2d ? MVLA_SET_2D : (mh[1] > gp.tau_3d ? MVLA_SET_3D : (MVLA_SET_2D | MVLA_SET_3D));
        const int c2 = mh[3] < gp.eps_3d ? MVLA_SET_2D : (MVLA_SET_2D | MVLA_SET_3D);
        int cf = c2 & c1;
        if (cf == 0) cf = c2;                                     // conflict resolution (Sec. 4.4)
        int k2, k3;
        if (s.k_2d_fixed >= 0) {
            k2 = s.k_2d_fixed;
            k3 = s.budget - k2;
        } else {
            const float w3 = cf == (MVLA_SET_2D | MVLA_SET_3D) ? mh[3] : (cf == MVLA_SET_2D ? 0.f : 1.f);
            const int lo3k = max(s.kmin_3d, s.budget - n2);
            const int hi3k = min(n3, s.budget - s.kmin_2d);
            k3 = static_cast<int>(floorf(static_cast<float>(s.budget) * w3 + 0.5f));
            k3 = min(max(k3, lo3k), hi3k);
            k2 = s.budget - k3;
            sm.ctl[6] = k2; sm.ctl[7] = k3;
        }
        if (io.z_out) { sm.zf[0] = static_cast<float>(n2) / t4; sm.zf[1] = static_cast<float>(n3) / t5; }
        if (leader) {
            if (io.budgets) {
                io.budgets[b_glob * 2 + 0] = k2;
                io.budgets[b_glob * 2 + 1] = k3;
            }
            if (io.diag) {
                mvla_diag dg;
                dg.t = s.t; dg.c_s1 = c1; dg.c_s2 = c2; dg.c_final = cf;
                dg.budget = s.budget; dg.k_2d = k2; dg.k_3d = k3; dg.reserved = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) { dg.x[c] = x[c]; dg.mhat[c] = mh[c]; }
                io.diag[b_glob] = dg;
            }
            io.out_offsets[b_glob] = s.out_off;
            if (io.write_total && b_local == io.n_in_launch - 1) io.out_offsets[b_glob + 1] = io.total_out;
        }
    };
    if (!k_fixed && warp == NW - 1) indicators();

    // ---- 3./4. threshold bin per modality, refined while the bin is crowded
    // st[e]: 0 dropped, 1 kept, 2 undecided (in the threshold bin, or not yet examined)
    int st[EPT], slot[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) { st[e] = (tid + e * NT) < nv ? 2 : 0; slot[e] = -1; }
    bool act2 = true, act3 = true;            // the modality still has a histogram pass to run
    int mode2 = SEL_NONE, mode3 = SEL_NONE, need2 = 0, need3 = 0, k2 = 0, k3 = 0;
#pragma unroll 1
    for (int level = 0; level < 5; ++level) {
        // count the undecided keys of the active modalities (a modality whose keys are all equal needs no count)
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (e * NT >= nv) break;
            const bool is3 = (tid + e * NT) >= n2;
            const int sh = is3 ? sh3 : sh2;
            if (st[e] == 2 && (is3 ? act3 : act2) && sh >= 0) {
                const int r = kSelBins - 1 - static_cast<int>((key[e] - (is3 ? lo3 : lo2)) >> sh);
                atomicAdd(&sm.hist[is3 ? 1 : 0][hist_pos(r)], 1);
            }
        }
        __syncthreads();                                                                   // ---- barrier B
        if (warp < 2 && (warp == 0 ? act2 : act3)) {
            const int m = warp, n_m = m == 0 ? n2 : n3, sh = m == 0 ? sh2 : sh3;
            const int k = level == 0 ? sm.ctl[6 + m] : sm.krem[m];
            int mode, tbin = 0, need = 0;
            if (level == 0 && k <= 0) mode = SEL_NONE;
            else if (level == 0 && k >= n_m) mode = SEL_ALL;
            else if (sh < 0) { mode = SEL_TIES; need = k; }                // equal keys only: index order decides
            else {
                int cnt;
                find_threshold_bin(sm.hist[m], k, lane, tbin, need, cnt);
                mode = need == cnt ? SEL_BIN_ALL : (cnt <= kCandMax ? SEL_LIST : (sh == 0 ? SEL_TIES : SEL_REFINE));
            }
            if (lane == 0) { sm.ctl[m] = mode; sm.ctl[2 + m] = tbin; sm.ctl[4 + m] = need; sm.krem[m] = need; }
        }
        __syncthreads();                                                                   // ---- barrier C
        const int4 c0 = *reinterpret_cast<const int4*>(&sm.ctl[0]);       // modes, threshold bins
        const int4 c1 = *reinterpret_cast<const int4*>(&sm.ctl[4]);       // keys to take from the bins, budgets
        if (act2) { mode2 = c0.x; need2 = c1.x; }
        if (act3) { mode3 = c0.y; need3 = c1.y; }
        k2 = c1.z; k3 = c1.w;
        const int tb2 = c0.z, tb3 = c0.w;
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (e * NT >= nv) break;
            const bool is3 = (tid + e * NT) >= n2;
            if (st[e] != 2 || !(is3 ? act3 : act2)) continue;
            const int mode = is3 ? mode3 : mode2, sh = is3 ? sh3 : sh2, tbin = is3 ? tb3 : tb2;
            if (mode == SEL_NONE) st[e] = 0;
            else if (mode == SEL_ALL) st[e] = 1;
            else if (sh >= 0) {
                const int r = kSelBins - 1 - static_cast<int>((key[e] - (is3 ? lo3 : lo2)) >> sh);
                if (r < tbin) st[e] = 1;
                else if (r > tbin) st[e] = 0;
                else if (mode == SEL_BIN_ALL) st[e] = 1;
                else if (mode == SEL_LIST) {
                    slot[e] = atomicAdd(&sm.ncand[is3 ? 1 : 0], 1);
                    sm.cand_key[is3 ? 1 : 0][slot[e]] = key[e];
                    sm.cand_idx[is3 ? 1 : 0][slot[e]] = tid + e * NT;
                }
            }
        }
        // a crowded threshold bin becomes the whole range of the next pass
        if (act2 && mode2 == SEL_REFINE) { lo2 += static_cast<uint32_t>(kSelBins - 1 - tb2) << sh2; sh2 = max(0, sh2 - kSelBinBits); }
        else act2 = false;
        if (act3 && mode3 == SEL_REFINE) { lo3 += static_cast<uint32_t>(kSelBins - 1 - tb3) << sh3; sh3 = max(0, sh3 - kSelBinBits); }
        else act3 = false;
        if (!act2 && !act3) break;                             // block-uniform: the modes come from shared memory
        __syncthreads();                                       // the threshold warps are done with the histograms
        for (int i = tid; i < 2 * kSelBins / 4; i += NT) reinterpret_cast<int4*>(&sm.hist[0][0])[i] = make_int4(0, 0, 0, 0);
        __syncthreads();
    }
    if (mode2 == SEL_LIST || mode3 == SEL_LIST) {              // rank the few keys of the threshold bin
        __syncthreads();                                                                   // ---- barrier D
        // All pairs at once: 8 lanes share one listed key c1 and compare it with four others each (one
        // 16-byte load of keys, one of indices); three shuffles add their counts.  No thread loops over
        // the list, so no warp lags behind the others.
        for (int wk = tid; wk < 2 * kCandMax * 8; wk += NT) {      // (modality, key, group of four)
            const int m = wk / (kCandMax * 8), c1 = (wk >> 3) & (kCandMax - 1), g = wk & 7;
            const int n = sm.ncand[m];
            const uint32_t k1 = sm.cand_key[m][c1];
            const int i1 = sm.cand_idx[m][c1];
            const uint4 q = reinterpret_cast<const uint4*>(sm.cand_key[m])[g];
            const int4 ix = reinterpret_cast<const int4*>(sm.cand_idx[m])[g];
            const int c = 4 * g;                               // entries past n are stale: masked
            int cnt = ((c < n) & ((q.x > k1) | ((q.x == k1) & (ix.x < i1)))) ? 1 : 0;
            cnt += ((c + 1 < n) & ((q.y > k1) | ((q.y == k1) & (ix.y < i1)))) ? 1 : 0;
            cnt += ((c + 2 < n) & ((q.z > k1) | ((q.z == k1) & (ix.z < i1)))) ? 1 : 0;
            cnt += ((c + 3 < n) & ((q.w > k1) | ((q.w == k1) & (ix.w < i1)))) ? 1 : 0;
            cnt += __shfl_xor_sync(0xffffffffu, cnt, 1);
            cnt += __shfl_xor_sync(0xffffffffu, cnt, 2);
            cnt += __shfl_xor_sync(0xffffffffu, cnt, 4);
            if (g == 0) sm.cand_rank[m][c1] = cnt;
        }
        __syncthreads();
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (slot[e] < 0) continue;
            const bool is3 = (tid + e * NT) >= n2;
            st[e] = sm.cand_rank[is3 ? 1 : 0][slot[e]] < (is3 ? need3 : need2) ? 1 : 0;
        }
    }

    // ---- 5. emission.  Tokens are ranked in visual order (2D first) by warp ballots; slice e of the
    //         threads' elements covers indices [e NT, (e + 1) NT).  The three segments are contiguous, so
    //         a kept token's output row is the number of rows that the segments lying before its own
    //         contribute plus its rank inside its modality.
    const int base2 = (s.off_txt < s.off_2d ? s.n_txt : 0) + (s.off_3d < s.off_2d ? k3 : 0);
    const int base3 = (s.off_txt < s.off_3d ? s.n_txt : 0) + (s.off_2d < s.off_3d ? k2 : 0);
    const int baset = (s.off_2d < s.off_txt ? k2 : 0) + (s.off_3d < s.off_txt ? k3 : 0);
    int32_t* const kept_sm = role.kept_sm;
    for (int i = tid; i < s.n_txt; i += NT) {
        if (leader) io.kept_idx[s.out_off + baset + i] = s.off_txt + i;
        if (kept_sm) kept_sm[baset + i] = s.off_txt + i;
    }
    // Exclusive prefix of the per-(slice, warp) counts in sm.wtot, for this warp's entry of every slice:
    // one scan per warp (each warp for itself: no further barrier), then one shuffle per slice.
    constexpr int PER = (EPT * NW + 31) / 32;                   // entries per lane
    auto prefixes = [&](int (&pre)[EPT]) {
        int v[PER], mine = 0;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int p = lane * PER + i;
            v[i] = p < EPT * NW ? (&sm.wtot[0][0])[p] : 0;
            mine += v[i];
        }
        const int excl = warp_incl_scan(mine, lane) - mine;
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            const int p = e * NW + warp;
            int r = __shfl_sync(0xffffffffu, excl, p / PER);
#pragma unroll
            for (int i = 0; i < PER - 1; ++i) {
                const int vi = __shfl_sync(0xffffffffu, v[i], p / PER);
                if (i < p % PER) r += vi;
            }
            pre[e] = r;
        }
    };
    const bool ties = mode2 == SEL_TIES || mode3 == SEL_TIES;     // block-uniform
    if (ties) {                                                   // equal keys straddle a budget: lower index wins
        int tlow[EPT], pre[EPT];
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            const int j = tid + e * NT;
            const bool t2 = st[e] == 2 && j < n2, t3 = st[e] == 2 && j >= n2;
            const unsigned b2 = __ballot_sync(0xffffffffu, t2), b3 = __ballot_sync(0xffffffffu, t3);
            const unsigned below = (1u << lane) - 1u;
            tlow[e] = t2 ? __popc(b2 & below) : __popc(b3 & below);
            if (lane == 0) sm.wtot[e][warp] = __popc(b2) | (__popc(b3) << 16);
        }
        __syncthreads();
        prefixes(pre);
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (st[e] != 2) continue;
            const int j = tid + e * NT;
            if (j < n2) st[e] = (pre[e] & 0xFFFF) + tlow[e] < need2 ? 1 : 0;
            else        st[e] = (pre[e] >> 16) + tlow[e] < need3 ? 1 : 0;
        }
        __syncthreads();                                          // sm.wtot is reused below
    }
    int klow[EPT], pre[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        const unsigned b = __ballot_sync(0xffffffffu, st[e] == 1);
        klow[e] = __popc(b & ((1u << lane) - 1u));
        if (lane == 0) sm.wtot[e][warp] = __popc(b);
    }
    __syncthreads();                                                                       // ---- barrier E
    prefixes(pre);
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        if (e * NT >= nv) break;                                  // uniform
        if (st[e] != 1) continue;
        const int j = tid + e * NT, r = pre[e] + klow[e];
        const int pos = j < n2 ? base2 + r : base3 + (r - k2);
        const int val = j < n2 ? s.off_2d + j : s.off_3d + (j - n2);
        if (leader) io.kept_idx[s.out_off + pos] = val;
        if (kept_sm) kept_sm[pos] = val;
    }
    after_list();
    if (role.late_pdl) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- 6. what nobody downstream waits for
    if (leader) {
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (e * NT >= nv) break;
            const int j = tid + e * NT;
            if (j < nv) {
                if (io.attn_out) io.attn_out[s.vis_off + j] = a[e];
                if (s.update_state) io.ahat_state[s.state_off_w + j] = key_to_float(key[e]);
                if (io.ahat_out) io.ahat_out[s.vis_off + j] = key_to_float(key[e]);
            }
        }
    }
    if (k_fixed && leader) {                                  // host-decided budgets: indicators, state, diagnostics
        const float col = warp_sum8(sums, lane);
        if ((lane & 3) == 0) sm.red[warp][lane >> 2] = col;
        __syncthreads();
        if (warp == NW - 1) indicators();
    }
    // optional: the smoothed scores normalised to mean one inside each modality.  The ranking above
    // uses the smoothed scores themselves; a positive per-modality factor cannot change it.
    if (io.z_out && leader) {
        __syncthreads();                                          // sm.zf written by the indicator warp
        const float f2 = sm.zf[0], f3 = sm.zf[1];
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (e * NT >= nv) break;
            const int j = tid + e * NT;
            if (j < nv) io.z_out[s.vis_off + j] = key_to_float(key[e]) * (j < n2 ? f2 : f3);
        }
    }
}

}  // namespace mvla
