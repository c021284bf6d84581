// Carry-over, budget split and top-k selection of ONE sample by one CTA of NT threads
// (Alg. 1 of the paper, steps 1-4; Eqs. 8, 9, 10).
//
// The work is a few KB, so the kernel is a chain of latencies; it is written to keep that chain short:
//   1. every thread issues ALL its global loads (scores, previous state, norms) before any dependent
//      work, then smooths the scores (Eq. 8 / Eq. 9 as  xhat = c_prev xhat + c_new x) and builds
//      order-preserving 32-bit keys, kept in registers and in shared memory;
//   2. modality sums -> the four indicators, smoothed too; dual threshold (Sec. 4.1), target-object
//      rule (Sec. 4.2), fusion (Sec. 4.4), budget split.  One thread does this while the others
//      already build the first radix histogram;
//   3. radix select of the k-th largest key of each modality: up to 4 passes of 8 bits, both
//      modalities at once, one warp-aggregated shared-memory histogram per pass (all cleared up
//      front); a modality is settled early when a digit bin must be taken whole;
//   4. emission merged with all text positions: elements above the threshold plus the first
//      (lowest-index) elements equal to it; one block-wide prefix scan per NT elements ranks the kept
//      ones (one more only when equal keys straddle a budget).
#pragma once

#include "common.cuh"

#include <math_constants.h>

namespace mvla {

constexpr float kFixScale = 1152921504606846976.f;          // 2^60
constexpr float kFixInv = 1.f / 1152921504606846976.f;      // 2^-60, exact

template <int NT>
struct SelectSmem {
    uint32_t key[kMaxVis];
    int hist[4][2][256];          // one histogram per radix pass and modality
    float red[NT / 32][4];        // per-warp partial sums of the instantaneous scores and norms
    float red2[NT / 32][4];       // scratch of the optional normalisation
    float tot[4];
    int scan[NT / 32 + 1];
    uint32_t prefix[2];
    int krem[2];
    int k[2];
    int alltie[2];                // every element equal to the threshold key is kept: no tie ranking needed
    int done[2];                  // the threshold is settled before all 32 bits were examined
    uint32_t cmask[2];            // key bits that the threshold comparison looks at
};

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

// Deterministic block sum of 4 values per thread: fixed shuffle tree inside each warp, then warp 0
// adds the warp partials with the same tree.  Result in sm_tot[0..3] after the trailing barrier.
template <int NT>
__device__ __forceinline__ void block_sum4(float (&x)[4], float (*scratch)[4], float* sm_tot)
{
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) x[c] += __shfl_xor_sync(0xffffffffu, x[c], off);
    if (lane == 0)
#pragma unroll
        for (int c = 0; c < 4; ++c) scratch[warp][c] = x[c];
    __syncthreads();
    if (warp == 0) {
        float y[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            y[c] = lane < NW ? scratch[lane][c] : 0.f;
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) y[c] += __shfl_xor_sync(0xffffffffu, y[c], off);
        }
        if (lane == 0)
#pragma unroll
            for (int c = 0; c < 4; ++c) sm_tot[c] = y[c];
    }
    __syncthreads();
}

// Exclusive block scan of one int per thread.
template <int NT>
__device__ __forceinline__ int block_exscan(int x, int* warp_tot, int* total)
{
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = x;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += n;
    }
    __syncthreads();                                       // previous users of warp_tot are done
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int t = lane < NW ? warp_tot[lane] : 0;
        int winc = t;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, winc, off);
            if (lane >= off) winc += n;
        }
        if (lane < NW) warp_tot[lane] = winc - t;          // exclusive prefix of the warp totals
        if (lane == 31) warp_tot[NW] = winc;               // grand total
    }
    __syncthreads();
    *total = warp_tot[NW];
    return warp_tot[warp] + inc - x;
}

template <int NT>
__device__ void select_sample(const SampleDev& s, int b_local, const GateParams& gp, const SelectIO& io,
                              SelectSmem<NT>& sm)
{
    constexpr int EPT = kMaxVis / NT;                     // elements per thread, strided by NT
    static_assert(EPT >= 1 && EPT * NT == kMaxVis, "thread count must divide the capacity");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n2 = s.n_2d, n3 = s.n_3d, nv = n2 + n3;
    const int b_glob = io.chunk_first + b_local;
    const bool carry = s.c_prev != 0.f;

    // prologue that needs nothing from the previous kernel
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int i = tid; i < 4 * 2 * 256; i += NT) (&sm.hist[0][0][0])[i] = 0;
    const bool k_fixed = s.k_2d_fixed >= 0;               // budgets decided on the host (FIXED mode, cold start)
    if (tid < 2) {
        sm.prefix[tid] = 0u; sm.alltie[tid] = 1; sm.done[tid] = 0; sm.cmask[tid] = 0xFFFFFFFFu;
        if (k_fixed) sm.k[tid] = sm.krem[tid] = tid == 0 ? s.k_2d_fixed : s.budget - s.k_2d_fixed;
    }
    __syncthreads();                                        // histograms are clear before anyone adds to them
    asm volatile("griddepcontrol.wait;" ::: "memory");      // scores come from the kernel before this one

    // ---- 1. all loads first
    float a[EPT], prev[EPT], nrm[EPT];
    unsigned long long fx[EPT];
#pragma unroll
    for (int e = 0; e < EPT; ++e) { a[e] = 0.f; prev[e] = 0.f; nrm[e] = 0.f; fx[e] = 0ull; }
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        if (e * NT >= nv) break;                           // uniform: nobody owns an element in this slice
        const int j = tid + e * NT;
        if (j < nv) {
            if (io.acc64) fx[e] = __ldcg(io.acc64 + s.vis_off + j);        // written by other CTAs' atomics
            else if (!io.part) a[e] = io.attn[s.vis_off + j];
            if (carry) prev[e] = io.ahat_state[s.state_off + j];
            if (gp.has_l1) nrm[e] = io.l1[s.vis_off + j];
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
    uint32_t key[EPT];
    float sums[4] = {0.f, 0.f, 0.f, 0.f};     // sum a over 2D, over 3D, sum l1 over 2D, over 3D
    float ssm[4] = {0.f, 0.f, 0.f, 0.f};      // sums of the smoothed scores per modality (for z)
#pragma unroll
    for (int e = 0; e < EPT; ++e) key[e] = 0u;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        if (e * NT >= nv) break;
        const int j = tid + e * NT;
        if (j < nv) {
            if (io.acc64) {
                a[e] = __ull2float_rn(fx[e]) * kFixInv;   // one rounding: the exact head sum to fp32
                io.acc64[s.vis_off + j] = 0ull;            // ready for the next call
            }
            const float smo = carry ? fmaf(s.c_prev, prev[e], s.c_new * a[e]) : a[e];
            if (io.attn_out) io.attn_out[s.vis_off + j] = a[e];
            if (s.update_state) io.ahat_state[s.state_off + j] = smo;
            if (io.ahat_out) io.ahat_out[s.vis_off + j] = smo;
            key[e] = order_key(smo);
            sm.key[j] = key[e];
            if (j < n2) { sums[0] += a[e]; sums[2] += nrm[e]; ssm[0] += smo; }
            else        { sums[1] += a[e]; sums[3] += nrm[e]; ssm[1] += smo; }
        }
    }
    // Per-warp partial sums (fixed shuffle tree).  The sum over warps is taken later by the one warp that
    // needs it, so that with host-decided budgets nothing below waits for the indicator arithmetic.
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) sums[c] += __shfl_xor_sync(0xffffffffu, sums[c], off);
    if (lane == 0)
#pragma unroll
        for (int c = 0; c < 4; ++c) sm.red[warp][c] = sums[c];

    // optional: the smoothed scores normalised to mean one inside each modality.  The ranking below
    // uses the smoothed scores themselves; a positive per-modality factor cannot change it.
    if (io.z_out) {
        block_sum4<NT>(ssm, sm.red2, sm.tot);
        const float f2 = static_cast<float>(n2) / sm.tot[0], f3 = static_cast<float>(n3) / sm.tot[1];
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            if (e * NT >= nv) break;
            const int j = tid + e * NT;
            if (j < nv) io.z_out[s.vis_off + j] = key_to_float(key[e]) * (j < n2 ? f2 : f3);
        }
    }

    // One radix histogram pass over the keys that still match the prefix found so far.
    auto histogram = [&](int pass, int shift, uint32_t p0, uint32_t p1, bool skip0, bool skip1) {
        const uint32_t himask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
        int* hist = &sm.hist[pass][0][0];
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            const int j = tid + e * NT;
            if (e * NT >= ((nv + 31) & ~31)) break;        // uniform: no warp has work in this slice
            int bin = -1;                                  // -1: not a candidate (any more)
            if (j < nv) {
                const int m = j >= n2;
                if (!(m ? skip1 : skip0) && ((key[e] ^ (m ? p1 : p0)) & himask) == 0u)
                    bin = (m << 8) | static_cast<int>((key[e] >> shift) & 255u);
            }
            // keys share their leading bytes most of the time: one atomic per warp instead of 32
            int same;
            __match_all_sync(0xffffffffu, bin, &same);
            if (same) {
                if (lane == 0 && bin >= 0) atomicAdd(hist + bin, 32);
            } else if (bin >= 0) {
                atomicAdd(hist + bin, 1);
            }
        }
    };
    histogram(0, 24, 0u, 0u, false, false);   // needs no budget yet
    __syncthreads();                          // first histogram and the per-warp sums are complete

    // ---- 2. indicators, gates, budget: the last warp (which rarely owns elements) adds the per-warp sums
    //         with the same fixed tree, its first lane does the few dozen flops.  With host-decided budgets
    //         the other warps go straight on to the digit search and meet this warp at the next barrier.
    if (warp == NT / 32 - 1) {
        float t0, t1, t2, t3;
        {
            float y[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                y[c] = lane < NT / 32 ? sm.red[lane][c] : 0.f;
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) y[c] += __shfl_xor_sync(0xffffffffu, y[c], off);
            }
            t0 = y[0]; t1 = y[1]; t2 = y[2]; t3 = y[3];
        }
      if (lane == 0) {
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
            if (s.update_state) io.mhat_state[s.mstate_off * 4 + c] = mh[c];
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
            const int lo = max(s.kmin_3d, s.budget - n2);
            const int hi = min(n3, s.budget - s.kmin_2d);
            k3 = static_cast<int>(floorf(static_cast<float>(s.budget) * w3 + 0.5f));
            k3 = min(max(k3, lo), hi);
            k2 = s.budget - k3;
        }
        if (!k_fixed) {
            sm.k[0] = k2; sm.k[1] = k3;
            sm.krem[0] = k2; sm.krem[1] = k3;
        }
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
    }
    if (!k_fixed) __syncthreads();            // the digit search needs the budgets (block-uniform branch)

    // ---- 3. radix select, 8 bits per pass, most significant first.  A modality is settled as soon as
    //         the digit bin that holds its k-th largest element must be taken whole (then the bits seen
    //         so far decide membership); otherwise after four passes sm.prefix[m] is the key of the k-th
    //         largest element and sm.krem[m] how many elements equal to it are kept.
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (pass > 0) {
            const bool d0 = sm.done[0] || sm.k[0] == 0, d1 = sm.done[1] || sm.k[1] == 0;
            if (d0 && d1) break;                            // block-uniform
            histogram(pass, shift, sm.prefix[0], sm.prefix[1], d0, d1);
            __syncthreads();
        }
        if (warp < 2 && sm.k[warp] > 0 && !sm.done[warp]) {
            // lane L owns the 8 digits 255-8L .. 248-8L (descending); find the digit where the
            // count of elements with a larger digit first reaches k
            const int m = warp, krem = sm.krem[m];
            int cnt[8], mine = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { cnt[i] = sm.hist[pass][m][255 - 8 * lane - i]; mine += cnt[i]; }
            int inc = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += n;
            }
            int above = inc - mine;                       // elements with digits above this lane's range
            if (above < krem && krem <= inc) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (above < krem && krem <= above + cnt[i]) {
                        sm.prefix[m] |= static_cast<uint32_t>(255 - 8 * lane - i) << shift;
                        sm.krem[m] = krem - above;
                        if (krem - above == cnt[i]) {         // the whole bin is kept: settled
                            sm.done[m] = 1;
                            sm.cmask[m] = 0xFFFFFFFFu << shift;
                        } else if (pass == 3) {
                            sm.alltie[m] = 0;                 // equal keys straddle the budget: rank them by index
                        }
                        break;
                    }
                    above += cnt[i];
                }
            }
        }
        __syncthreads();
    }

    // ---- 4. emission.  Each thread decides its own elements from the keys it holds in registers; one
    //         block scan per slice of NT elements (in visual order: 2D first) ranks the kept ones.  The
    //         three segments are contiguous, so a kept token's output row is the number of rows that the
    //         segments lying before its own contribute plus its rank inside its modality.
    const uint32_t th2 = sm.prefix[0], th3 = sm.prefix[1];
    const uint32_t cm2 = sm.cmask[0], cm3 = sm.cmask[1];
    const int k2 = sm.k[0], k3 = sm.k[1];
    const int need2 = k2 > 0 ? sm.krem[0] : 0, need3 = k3 > 0 ? sm.krem[1] : 0;
    const bool rank_ties = !(sm.alltie[0] && sm.alltie[1]);          // block-uniform
    const int base2 = (s.off_txt < s.off_2d ? s.n_txt : 0) + (s.off_3d < s.off_2d ? k3 : 0);
    const int base3 = (s.off_txt < s.off_3d ? s.n_txt : 0) + (s.off_2d < s.off_3d ? k2 : 0);
    const int baset = (s.off_2d < s.off_txt ? k2 : 0) + (s.off_3d < s.off_txt ? k3 : 0);
    for (int i = tid; i < s.n_txt; i += NT) io.kept_idx[s.out_off + baset + i] = s.off_txt + i;

    int run_kept = 0, run_t2 = 0, run_t3 = 0;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        if (e * NT >= nv) break;                                      // uniform
        const int j = tid + e * NT;
        int c = 0;                                                    // 0 dropped, 1 kept, 2 tie in 2D, 3 tie in 3D
        if (j < nv) {
            if (j < n2) {
                const uint32_t kk = key[e] & cm2;
                c = k2 <= 0 ? 0 : (kk > th2 ? 1 : (kk == th2 ? 2 : 0));
            } else {
                const uint32_t kk = key[e] & cm3;
                c = k3 <= 0 ? 0 : (kk > th3 ? 1 : (kk == th3 ? 3 : 0));
            }
        }
        if (rank_ties) {                                              // equal keys straddle a budget: lower index wins
            int tot = 0;
            const int tr = block_exscan<NT>((c == 2) + ((c == 3) << 16), sm.scan, &tot);
            if (c == 2) c = (run_t2 + (tr & 0xFFFF)) < need2 ? 1 : 0;
            else if (c == 3) c = (run_t3 + (tr >> 16)) < need3 ? 1 : 0;
            run_t2 += tot & 0xFFFF;
            run_t3 += tot >> 16;
        } else if (c >= 2) {
            c = 1;                                                    // every element equal to the threshold is kept
        }
        int tot = 0;
        const int r = run_kept + block_exscan<NT>(c, sm.scan, &tot);
        run_kept += tot;
        if (c) {
            if (j < n2) io.kept_idx[s.out_off + base2 + r] = s.off_2d + j;
            else        io.kept_idx[s.out_off + base3 + (r - k2)] = s.off_3d + (j - n2);
        }
    }
}

}  // namespace mvla
