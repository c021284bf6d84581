// Alg. 1 of the paper taken literally, patch by patch: the work of one CTA on the indicators of a block of
// patches, and of one CTA on the stages after them for a sample.  A patch p of a sample owns visual token
// p (2D) and visual token P + p (3D), P = n_2d = n_3d.
//
// The data is a few KB to a few MB that sits in L2; this is a latency chain, not bandwidth work.
// Every comparison that decides a set is taken in double on the fp32 values, and the K-Means runs in
// double, so that the same fp32 inputs give the same decisions as a double-precision restatement.
#pragma once

#include "common.cuh"
#include "device_utils.cuh"
#include "select_impl.cuh"

#include <math_constants.h>

namespace mvla {

constexpr int kIndThreads = 512;
constexpr int kMaxPatch = kMaxVis / 2;

__device__ __forceinline__ unsigned long long pack2f(float lo, float hi)
{
    return static_cast<unsigned long long>(__float_as_uint(lo)) | (static_cast<unsigned long long>(__float_as_uint(hi)) << 32);
}
__device__ __forceinline__ unsigned long long ld_relaxed_gpu_u64(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// Indicators of a block of PP = 2, 4 or 8 patches (8 floats = one 32-byte sector per (head, query); fewer
// patches per CTA when the batch is too small to fill the SMs otherwise), by a CTA of kIndThreads threads.
// Thread = (patch, group): the group walks the (head, query) pairs with stride 512 / PP, so a CTA has
// all its loads of a pass in flight at once (a few per thread).
// Also writes the per-token scores of the patch's two tokens: a_j = ||alpha_j||_1 / (H n_t).
// The L1 feature norms of the CTA's 2 PP rows (Sec. 3.1.2) are taken here too, 256 / PP threads per row,
// their loads issued before the kernel waits for the attention copy of the kernel before it.
//
// `blk`: which block of PP patches of sample `s`.  `rec`: when not null, the patch's indicators and scores
// also go, as three 8-byte words per patch ({x0, x1}, {x2, x3}, {a_2D, a_3D}; all ones before the launch),
// to the CTA of the same kernel that runs the stages after this one: an aligned 8-byte store is
// indivisible and no result of arithmetic has all 64 bits set, so each word is its own "ready" signal.
template <typename T, int PP>
__device__ __forceinline__ void patch_indicators_block(const SampleDev& s, int blk, int n_heads, const AlphaOut& alpha,
                                                       const T* __restrict__ hidden, int d_model, float* __restrict__ x_out,
                                                       float* __restrict__ attn_out, unsigned long long* __restrict__ rec, bool norms_early)
{
    constexpr int kIndPatches = PP;
    constexpr int kIndGroups = kIndThreads / PP;          // groups of (head, query) pairs
    constexpr int kRowThreads = kIndThreads / (2 * PP);   // threads that share one hidden row
    __shared__ float red[kIndThreads / 32][kIndPatches][4];
    __shared__ float tot[kIndPatches][4];
    __shared__ float rown[kIndThreads / 32];
    const int P = s.n_2d;
    const int p0 = blk * kIndPatches;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p0 >= P) return;                                  // block-uniform
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pl = tid & (kIndPatches - 1), g = tid / kIndPatches;
    const int p = p0 + pl;
    const bool live = p < P;
    const int npairs = n_heads * s.n_txt;
    const float* base = alpha.ptr + static_cast<int64_t>(s.vis_off + p) * alpha.stride_j;   // the patch's 2D token; its 3D token is P rows on
    const int64_t to3 = static_cast<int64_t>(P) * alpha.stride_j;

    // ---- feature norms: row r of the CTA = 2D token p0 + r (r < PP) or 3D token p0 + r - PP.  The first
    //      kNormKeep 16-byte pieces of a thread are loaded here and added up further down, once the loads of
    //      the attention copy are in flight too.  `norms_early`: issue them before the wait for the kernel
    //      before this one (they do not depend on it), else after it -- beside a scoring kernel in the middle
    //      of its own stores the early loads were seen to cost that kernel more than they save here.
    constexpr int kNormKeep = 8;
    constexpr int kVec = 16 / sizeof(T);
    const int nr = tid / kRowThreads, within = tid % kRowThreads;
    const int pr = p0 + (nr & (kIndPatches - 1));
    const int nvec = d_model / kVec;
    const uint4* nsrc = nullptr;
    if (pr < P)
        nsrc = reinterpret_cast<const uint4*>(hidden + static_cast<int64_t>(s.seq_off + (nr < kIndPatches ? s.off_2d : s.off_3d) + pr) * d_model);
    uint4 hv[kNormKeep];
    auto norm_loads = [&]() {
#pragma unroll
        for (int k = 0; k < kNormKeep; ++k) {
            const int i = within + k * kRowThreads;
            hv[k] = (nsrc && i < nvec) ? __ldg(nsrc + i) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    auto abs_sum = [](const uint4& u) {
        if constexpr (sizeof(T) == 2) {
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
            float a = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                a += fabsf(__uint_as_float(w[e] << 16));           // low bf16
                a += fabsf(__uint_as_float(w[e] & 0xFFFF0000u));   // high bf16
            }
            return a;
        } else {
            return fabsf(__uint_as_float(u.x)) + fabsf(__uint_as_float(u.y)) +
                   fabsf(__uint_as_float(u.z)) + fabsf(__uint_as_float(u.w));
        }
    };
    if (norms_early) norm_loads();
    asm volatile("griddepcontrol.wait;" ::: "memory");    // the attention copy comes from the kernel before this one
    if (!norms_early) norm_loads();

    // Sum over the lanes of a warp that hold the same patch (the lane bits above log2 PP), then over the
    // warps in a fixed order: tot[patch][c].
    auto reduce = [&](float (&v)[4], int ncomp) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (c >= ncomp) break;
#pragma unroll
            for (int off = PP; off < 32; off <<= 1) v[c] += __shfl_xor_sync(0xffffffffu, v[c], off);
        }
        __syncthreads();                                  // earlier readers of red / tot are done
        if (lane < kIndPatches)
#pragma unroll
            for (int c = 0; c < 4; ++c) red[warp][lane][c] = v[c];
        __syncthreads();
        if (tid < kIndPatches * 4) {
            const int q = tid >> 2, c = tid & 3;
            float acc = 0.f;
#pragma unroll 8
            for (int w = 0; w < kIndThreads / 32; ++w) acc += red[w][q][c];
            tot[q][c] = acc;
        }
        __syncthreads();
    };

    // pass 1: <a3, a2>, <a2, a2>, ||a2||_1, ||a3||_1.  The first kKeep pairs of a thread stay in registers for
    // pass 2 (all of them at the shapes this path is built for): the attention copy is read once.
    constexpr int kKeep = 16;
    float r2[kKeep], r3[kKeep];
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    const int nq = min(kKeep, (npairs + kIndGroups - 1) / kIndGroups);   // block-uniform: slots in use
    // pair idx = g + q kIndGroups is (head h, query i); stepping q moves (h, i) by a fixed amount
    const int step_h = kIndGroups / s.n_txt, step_i = kIndGroups - step_h * s.n_txt;
    int h = g / s.n_txt, i = g - h * s.n_txt;
#pragma unroll
    for (int q = 0; q < kKeep; ++q) {                     // all loads of the thread in flight at once
        r2[q] = 0.f; r3[q] = 0.f;
        if (q >= nq) continue;                            // uniform
        if (live && g + q * kIndGroups < npairs) {
            const float* a = base + static_cast<int64_t>(h) * alpha.stride_h + i;
            r2[q] = __ldcg(a); r3[q] = __ldcg(a + to3);
        }
        h += step_h; i += step_i;
        if (i >= s.n_txt) { i -= s.n_txt; ++h; }
    }
    {                                                     // the feature norms, now that every load is in flight
        float acc = 0.f;
#pragma unroll
        for (int k = 0; k < kNormKeep; ++k) acc += abs_sum(hv[k]);
        if (nsrc)
            for (int k = within + kNormKeep * kRowThreads; k < nvec; k += kRowThreads) acc += abs_sum(__ldg(nsrc + k));
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) rown[warp] = acc;                  // read after the barriers of the first reduction
    }
#pragma unroll
    for (int q = 0; q < kKeep; ++q) {                     // (a pair that does not exist adds zeros)
        if (q >= nq) break;                               // uniform
        v[0] = fmaf(r3[q], r2[q], v[0]);
        v[1] = fmaf(r2[q], r2[q], v[1]);
        v[2] += fabsf(r2[q]);
        v[3] += fabsf(r3[q]);
    }
    if (live) {
#pragma unroll 4
        for (int idx = g + kKeep * kIndGroups; idx < npairs; idx += kIndGroups) {
            const int hh = idx / s.n_txt, ii = idx - hh * s.n_txt;
            const float* a = base + static_cast<int64_t>(hh) * alpha.stride_h + ii;
            const float a2 = __ldcg(a), a3 = __ldcg(a + to3);
            v[0] = fmaf(a3, a2, v[0]);
            v[1] = fmaf(a2, a2, v[1]);
            v[2] += fabsf(a2);
            v[3] += fabsf(a3);
        }
    }
    reduce(v, 4);
    const float t0 = tot[pl][0], t1 = tot[pl][1], t2 = tot[pl][2], t3 = tot[pl][3];
    const float coef = t1 > 0.f ? t0 / t1 : 0.f;         // projection coefficient of a3 on a2 (Eq. 3-4)

    // pass 2: || a3 - coef a2 ||_1, the part of the 3D token's attention that the 2D token's does not explain
    float o[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int q = 0; q < kKeep; ++q) {
        if (q >= nq) break;                               // uniform
        o[0] += fabsf(fmaf(-coef, r2[q], r3[q]));
    }
    if (live) {
#pragma unroll 4
        for (int idx = g + kKeep * kIndGroups; idx < npairs; idx += kIndGroups) {
            const int hh = idx / s.n_txt, ii = idx - hh * s.n_txt;
            const float* a = base + static_cast<int64_t>(hh) * alpha.stride_h + ii;
            o[0] += fabsf(fmaf(-coef, __ldcg(a), __ldcg(a + to3)));
        }
    }
    reduce(o, 1);
    if (g == 0 && live) {
        constexpr int kRowWarps = kRowThreads / 32;
        float f2 = 0.f, f3 = 0.f;                         // the patch's 2D token, its 3D token
#pragma unroll
        for (int w = 0; w < kRowWarps; ++w) {
            f2 += rown[pl * kRowWarps + w];
            f3 += rown[(kIndPatches + pl) * kRowWarps + w];
        }
        float4 x;
        x.x = f2 / (f2 + f3);                             // Eq. 3-1, the term of this patch
        x.y = f3 / (f2 + f3);
        x.z = t2 / (t2 + t3);                             // Eq. P2D
        x.w = tot[pl][0] / (t2 + t3);                     // Eq. P3D
        reinterpret_cast<float4*>(x_out)[s.vis_off / 2 + p] = x;
        const float inv = 1.f / static_cast<float>(npairs);
        attn_out[s.vis_off + p] = t2 * inv;               // mean over heads and text queries
        attn_out[s.vis_off + P + p] = t3 * inv;
        if (rec) {
            unsigned long long* r = rec + (static_cast<int64_t>(s.vis_off / 2) + p) * 3;
            r[0] = pack2f(x.x, x.y);
            r[1] = pack2f(x.z, x.w);
            r[2] = pack2f(t2 * inv, t3 * inv);
        }
    }
}

template <int NT>
struct PatchSmemT {
    double mass[kMaxPatch];                 // attention mass of every patch (what K-Means clusters)
    uint8_t label[kMaxPatch];
    union {                                 // one after the other in time:
        float massf[kMaxPatch];             //   the masses rounded to fp32 (first look of the K-Means assignment)
        uint8_t keep[2 * kMaxPatch];        //   keep flags in visual order: 2D tokens, then 3D tokens (written after the K-Means)
    };
    float2 share[kMaxPatch];                // smoothed attention shares of every patch (M^S2_2D, M^S2_3D)
    double mu[2];                           // their means over the patches (the baselines of the robot rule)
    float thr[8];                           // the thresholds of stages 2-3 as fp32 numbers that decide like the doubles
    double centre[3];
    int cnt[5];                             // kept 2D, kept 3D, patches per class
    int iters;
    int out_off;
    int scan[NT / 32 + 1];
};

__device__ __forceinline__ double warp_sum_d(double v)
{
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}
__device__ __forceinline__ int ld_volatile_i32(const int* p)
{
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// One CTA per sample: stages 1-4 of Alg. 1 for its patches, then its first output row and the ordered
// kept positions.  A sample's first output row is the sum of the kept rows of the samples before it:
// each CTA publishes its count (value, fence, flag) and reads the counts of the samples before it in this
// launch, which have lower block indices and were therefore dispatched no later than itself; the wait is
// bounded and reports MVLA_ERR_TIMEOUT.  The CTA that finishes last clears the flags for the next launch.
//
// `b_local` of `n_in_launch`: which sample of the launch this CTA has.
// `rec`: null: indicators and scores come from io.x / io.attn, written by the kernel before this one; else
//        they are taken, patch by patch, from the 8-byte words that patch_indicators_block writes in the
//        same kernel (bounded wait for each).
// `list`: when not null, kHandWords + `cap` 4-byte words (all -1 before the launch) for CTAs of the same
//        kernel that copy the rows: in each of the first kHandLines lines of 32 words, word 0 = 1 once the
//        masks are decided (the list follows shortly: time to start polling it), word 1 = first output
//        row of the sample, word 2 = number of rows it keeps (written before word 1 by the same thread;
//        a reader takes word 2 only after it has seen word 1 and re-reads it until it is there); word
//        kHandWords + r = index inside the sample of the token that goes to the sample's output row r.
template <int NT>
__device__ __forceinline__ void patch_select_block(const SampleDev& s, int b_local, int n_in_launch, const PatchParams& pp,
                                                   const PatchIO& io, PatchSmemT<NT>& sm, const unsigned long long* rec,
                                                   int32_t* list)
{
    constexpr int kPPT = kMaxPatch / NT;                  // patches per thread, strided by the block size
    const int b_glob = io.chunk_first + b_local;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = s.n_2d, nv = 2 * P;
    const int pat_off = s.vis_off / 2;
    const bool carry = s.c_prev != 0.f;
    const bool cold = s.t == 1 && pp.cold_start_full_keep;
    float4* state = reinterpret_cast<float4*>(io.xhat_state) + static_cast<int64_t>(s.slot_index) * pp.max_patch;
    if (tid < 5) sm.cnt[tid] = 0;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");    // scores and indicators come from the kernel before this one (or, with `rec`, the hand-over words were re-armed by it)

    // ---- stage 1 (action iteration): X^ = c_prev X^ + c_new X for every patch and indicator (Eqs. 8, 9).
    //      All loads of a thread are issued before anything depends on them.
    float4 x[kPPT], pr[kPPT];
    float a2[kPPT], a3[kPPT], uu[kPPT];
#pragma unroll
    for (int e = 0; e < kPPT; ++e) {
        if (e * NT >= P) break;                        // block-uniform
        const int p = tid + e * NT;
        if (p < P) {
            if (!rec) {
                x[e] = reinterpret_cast<const float4*>(io.x)[pat_off + p];
                a2[e] = io.attn[s.vis_off + p];
                a3[e] = io.attn[s.vis_off + P + p];
            }
            if (carry) pr[e] = state[p];
            uu[e] = io.rand_u[pat_off + p];
        }
    }
    if (rec) {                                            // from the CTAs of this kernel that compute them
        bool ok = true;
        const uint64_t t_start = global_ns();
#pragma unroll
        for (int e = 0; e < kPPT; ++e) {
            if (e * NT >= P) break;
            const int p = tid + e * NT;
            if (p < P) {
                const unsigned long long* r = rec + static_cast<int64_t>(pat_off + p) * 3;
                unsigned long long w0 = ~0ull, w1 = ~0ull, w2 = ~0ull;
                for (uint32_t it = 0; it < kSpinLimit; ++it) {
                    w0 = ld_relaxed_gpu_u64(r); w1 = ld_relaxed_gpu_u64(r + 1); w2 = ld_relaxed_gpu_u64(r + 2);
                    if (w0 != ~0ull && w1 != ~0ull && w2 != ~0ull) break;
                    if ((it & 63u) == 63u && global_ns() - t_start > 1000000000ull) break;
                }
                ok &= w0 != ~0ull && w1 != ~0ull && w2 != ~0ull;
                x[e] = make_float4(__uint_as_float(static_cast<unsigned>(w0)), __uint_as_float(static_cast<unsigned>(w0 >> 32)),
                                   __uint_as_float(static_cast<unsigned>(w1)), __uint_as_float(static_cast<unsigned>(w1 >> 32)));
                a2[e] = __uint_as_float(static_cast<unsigned>(w2));
                a3[e] = __uint_as_float(static_cast<unsigned>(w2 >> 32));
            }
        }
        if (!ok) *reinterpret_cast<volatile int*>(io.status) = MVLA_ERR_TIMEOUT;   // the values are garbage: the caller sees the error
    }
    // Double-precision instructions are scarce on this part (a warp-wide one keeps the unit busy for many
    // cycles), so every thread does as few as it can -- the mass of its patch -- and one warp does the rest.
    float4 xh[kPPT];
#pragma unroll
    for (int e = 0; e < kPPT; ++e) {
        if (e * NT >= P) break;
        const int p = tid + e * NT;
        if (p < P) {
            float4 v = x[e];
            if (carry) {
                v.x = fmaf(s.c_prev, pr[e].x, s.c_new * x[e].x);
                v.y = fmaf(s.c_prev, pr[e].y, s.c_new * x[e].y);
                v.z = fmaf(s.c_prev, pr[e].z, s.c_new * x[e].z);
                v.w = fmaf(s.c_prev, pr[e].w, s.c_new * x[e].w);
            }
            xh[e] = v;
            if (s.update_state) state[p] = v;
            if (io.xhat_out) reinterpret_cast<float4*>(io.xhat_out)[pat_off + p] = v;
            // the patch's attention response: the mass of its two tokens
            const double m = static_cast<double>(a2[e]) + static_cast<double>(a3[e]);
            sm.mass[p] = m;
            sm.massf[p] = static_cast<float>(m);
            sm.label[p] = 255;
            sm.share[p] = make_float2(v.z, v.w);
        }
    }
    __syncthreads();

    // ---- stage 3 preparation by one warp, without block barriers: the baselines (means of the smoothed
    //      shares), then the 1-D K-Means, K = 3 (Sec. 4.2), started from the smallest mass, the mean and the
    //      largest.  A round: assign to the nearest centre (ties to the lower one); unless nothing changed,
    //      move the centres to the class means.
    if (warp == 0) {
        double sum_m = 0.0, sum_z = 0.0, sum_w = 0.0;
        long long mx = 0, mn = 0x7FF0000000000000ll;             // masses are >= 0: their bit patterns order like the values
#pragma unroll 8
        for (int p = lane; p < P; p += 32) {                      // (unrolled: the shared-memory loads of eight patches overlap)
            const double m = sm.mass[p];
            const float2 zw = sm.share[p];
            sum_m += m;
            sum_z += static_cast<double>(zw.x);
            sum_w += static_cast<double>(zw.y);
            mx = max(mx, __double_as_longlong(m));
            mn = min(mn, __double_as_longlong(m));
        }
        sum_m = warp_sum_d(sum_m); sum_z = warp_sum_d(sum_z); sum_w = warp_sum_d(sum_w);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, off));
        }
        // the three means with one division sequence: lane 0 the masses, lane 1 and 2 the shares
        const double mean = (lane == 0 ? sum_m : (lane == 1 ? sum_z : sum_w)) / P;
        const double mu_2d = __shfl_sync(0xffffffffu, mean, 1), mu_3d = __shfl_sync(0xffffffffu, mean, 2);
        if (lane == 0) {
            sm.mu[0] = mu_2d; sm.mu[1] = mu_3d;
            // x < t for an fp32 x and a double t holds exactly when x < (t rounded up to fp32); x > t when
            // x > (t rounded down): the per-patch rules below decide in fp32 what the doubles would decide
            sm.thr[0] = __double2float_ru(pp.tau_2d);        // S1_3D <  tau_2D
            sm.thr[1] = __double2float_rd(pp.tau_3d);        // S1_3D >  tau_3D
            sm.thr[2] = __double2float_ru(pp.bg_prune_prob); // u     <  background pruning probability
            sm.thr[3] = __double2float_rd(mu_3d);            // M_3D  >  its mean
            sm.thr[4] = __double2float_rd(mu_2d);            // M_2D  >  its mean
            sm.thr[5] = __double2float_rd(pp.obj_2d_min);    // M_2D  >  object rule's 2D floor
            sm.thr[6] = __double2float_ru(pp.eps_3d);        // M_3D  <  eps_3D
        }
        double c0 = __longlong_as_double(mn), c1 = __shfl_sync(0xffffffffu, mean, 0), c2 = __longlong_as_double(mx);
        int iters = 0;
        while (iters < pp.kmeans_max_iter) {                      // warp-uniform
            ++iters;
            int changed = 0;
            double s0 = 0.0, s1 = 0.0, s2 = 0.0;
            int n0 = 0, n1 = 0, n2 = 0;
            // Nearest centre.  fp32 decides wherever it can be sure: with m and the centres rounded to fp32
            // a distance is off by at most 2^-23 (m + c), so a comparison of two distances whose fp32 values
            // differ by more than `tol` comes out as in double; anything closer (ties included) is redone
            // in double.  Class sums stay in double.
            const float f0 = static_cast<float>(c0), f1 = static_cast<float>(c1), f2 = static_cast<float>(c2);
#pragma unroll 8
            for (int p = lane; p < P; p += 32) {
                const double m = sm.mass[p];
                const float mf = sm.massf[p];
                const float tol = 4e-7f * (fabsf(mf) + fmaxf(fabsf(f0), fmaxf(fabsf(f1), fabsf(f2))));
                const float e0 = fabsf(mf - f0), e1 = fabsf(mf - f1), e2 = fabsf(mf - f2);
                int best = e1 < e0 ? 1 : 0;
                const float eb = fminf(e0, e1);
                bool sure = fabsf(e1 - e0) > tol && fabsf(e2 - eb) > tol;
                if (e2 < eb) best = 2;
                if (!sure) {
                    best = 0;
                    double bdist = fabs(m - c0);
                    const double d1 = fabs(m - c1), d2 = fabs(m - c2);
                    if (d1 < bdist) { bdist = d1; best = 1; }
                    if (d2 < bdist) { bdist = d2; best = 2; }
                }
                if (sm.label[p] != best) { sm.label[p] = static_cast<uint8_t>(best); changed = 1; }
                s0 += best == 0 ? m : 0.0; n0 += best == 0;
                s1 += best == 1 ? m : 0.0; n1 += best == 1;
                s2 += best == 2 ? m : 0.0; n2 += best == 2;
            }
            if (!__any_sync(0xffffffffu, changed)) break;
            s0 = warp_sum_d(s0); s1 = warp_sum_d(s1); s2 = warp_sum_d(s2);
            n0 = __reduce_add_sync(0xffffffffu, n0); n1 = __reduce_add_sync(0xffffffffu, n1); n2 = __reduce_add_sync(0xffffffffu, n2);
            // the three class means with one division sequence (lane k: class k)
            const int nk = lane == 0 ? n0 : (lane == 1 ? n1 : n2);
            const double ck = (lane == 0 ? s0 : (lane == 1 ? s1 : s2)) / max(nk, 1);
            if (n0 > 0) c0 = __shfl_sync(0xffffffffu, ck, 0);
            if (n1 > 0) c1 = __shfl_sync(0xffffffffu, ck, 1);
            if (n2 > 0) c2 = __shfl_sync(0xffffffffu, ck, 2);
        }
        if (lane == 0) { sm.centre[0] = c0; sm.centre[1] = c1; sm.centre[2] = c2; sm.iters = iters; }
    }
    __syncthreads();

    // ---- stages 2-4 for every patch: C_S1 (dual threshold), C_S2 (semantic rules), fusion, masks
    const int both = MVLA_SET_2D | MVLA_SET_3D;
#pragma unroll
    for (int e = 0; e < kPPT; ++e) {
        if (e * NT >= P) break;
        const int p = tid + e * NT;
        if (p < P) {
            const int label = sm.label[p];
            const float s1_3d = xh[e].y, m2 = xh[e].z, m3 = xh[e].w;
            const int c1 = s1_3d < sm.thr[0] ? MVLA_SET_2D : (s1_3d > sm.thr[1] ? MVLA_SET_3D : both);
            int c2;
            if (label == MVLA_LABEL_BG) c2 = uu[e] < sm.thr[2] ? 0 : both;
            else if (label == MVLA_LABEL_ROB) c2 = m3 > sm.thr[3] ? both : (m2 > sm.thr[4] ? MVLA_SET_2D : 0);
            else c2 = (m2 > sm.thr[5] && m3 < sm.thr[6]) ? MVLA_SET_2D : both;
            int cf = 0;
            if (c2 != 0) {
                cf = c2 & c1;
                if (cf == 0) cf = c2;                             // conflict resolution
            }
            if (cold) cf = both;                                  // cold start: full unpruned tokens
            if (io.info_out) io.info_out[pat_off + p] = label | (c1 << 2) | (c2 << 4) | (cf << 6);
            const int k2 = (cf & MVLA_SET_2D) ? 1 : 0, k3 = (cf & MVLA_SET_3D) ? 1 : 0;
            sm.keep[p] = static_cast<uint8_t>(k2);
            sm.keep[P + p] = static_cast<uint8_t>(k3);
            if (k2) atomicAdd(&sm.cnt[0], 1);                     // integer counts: the order of the adds is immaterial
            if (k3) atomicAdd(&sm.cnt[1], 1);
            atomicAdd(&sm.cnt[2 + label], 1);
        }
    }
    __syncthreads();
    if (list && tid < kHandLines) list[32 * tid] = 1;             // the list follows shortly
    const int k2 = sm.cnt[0], k3 = sm.cnt[1];
    const int n_out = s.n_txt + k2 + k3;

    // ---- first output row: publish this sample's count, add up the counts of the samples before it.
    //      (A sample that is alone in its launch and first in its batch starts at row 0: nothing to wait for.)
    const bool alone = n_in_launch == 1;                          // nobody in this launch to wait for or to tell
    const bool first_row_known = alone && b_glob == 0;
    auto bookkeeping = [&](int off) {                             // lane 0 of warp 0
        io.out_offsets[b_glob] = off;
        if (b_glob == io.batch_total - 1) io.out_offsets[io.batch_total] = off + n_out;
        if (io.counts) { io.counts[b_glob * 2] = k2; io.counts[b_glob * 2 + 1] = k3; }
        if (io.diag) {
            mvla_patch_diag dg;
            dg.t = s.t; dg.iters = sm.iters;
            for (int c = 0; c < 3; ++c) { dg.n_label[c] = sm.cnt[2 + c]; dg.centre[c] = static_cast<float>(sm.centre[c]); }
            dg.k_2d = k2; dg.k_3d = k3; dg.n_out = n_out;
            dg.mu_2d = static_cast<float>(sm.mu[0]); dg.mu_3d = static_cast<float>(sm.mu[1]);
            dg.reserved[0] = dg.reserved[1] = dg.reserved[2] = 0.f;
            io.diag[b_glob] = dg;
        }
    };
    if (first_row_known) {
        if (list && tid < kHandLines) { list[32 * tid + 2] = n_out; list[32 * tid + 1] = 0; }
        if (tid == 0) { sm.out_off = 0; io.nout_ws[b_glob] = n_out; }   // later launches of this call read the count in stream order
    } else {
        if (warp == 0) {
            if (lane == 0) {
                io.nout_ws[b_glob] = n_out;                       // later launches of this call read it in stream order
                if (!alone) {
                    __threadfence();
                    asm volatile("st.volatile.global.s32 [%0], %1;" ::"l"(io.ready_ws + b_glob), "r"(1) : "memory");
                }
            }
            int off = 0;
            bool ok = true;
            for (int b = lane; b < b_glob; b += 32) {
                if (b >= io.chunk_first) {                        // same launch: wait for its flag (bounded)
                    bool got = false;
                    for (uint32_t it = 0; it < kSpinLimit && !got; ++it) {
                        got = ld_volatile_i32(io.ready_ws + b) != 0;
                        if (!got) __nanosleep(64);
                    }
                    ok &= got;
                    __threadfence();
                }
                off += ld_volatile_i32(io.nout_ws + b);           // earlier launches of this call are complete
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
            if (!__all_sync(0xffffffffu, ok) && lane == 0) *reinterpret_cast<volatile int*>(io.status) = MVLA_ERR_TIMEOUT;
            if (list && lane < kHandLines) { list[32 * lane + 2] = n_out; list[32 * lane + 1] = off; }
            if (lane == 0) {
                sm.out_off = off;
                // every wait of this CTA is over: the CTA that gets here last clears the flags of the launch
                if (!alone) __threadfence();
                if (!alone && atomicAdd(io.done_ws, 1) == n_in_launch - 1) {
                    for (int b = 0; b < n_in_launch; ++b) io.ready_ws[io.chunk_first + b] = 0;
                    *io.done_ws = 0;
                    __threadfence();
                }
            }
        }
        __syncthreads();
    }

    // ---- Eq. 10 as an ordered list.  The three segments are contiguous, so a kept token's output row is
    //      the rows of the segments lying before its own plus its rank inside its modality.
    const int out_off = first_row_known ? 0 : sm.out_off;
    const int base2 = (s.off_txt < s.off_2d ? s.n_txt : 0) + (s.off_3d < s.off_2d ? k3 : 0);
    const int base3 = (s.off_txt < s.off_3d ? s.n_txt : 0) + (s.off_2d < s.off_3d ? k2 : 0);
    const int baset = (s.off_2d < s.off_txt ? k2 : 0) + (s.off_3d < s.off_txt ? k3 : 0);
    for (int i = tid; i < s.n_txt; i += NT) {
        io.kept_idx[out_off + baset + i] = s.off_txt + i;
        if (list) list[kHandWords + baset + i] = s.off_txt + i;
    }
    int run = 0;
    for (int j0 = 0; j0 < nv; j0 += NT) {              // block-uniform
        const int j = j0 + tid;
        const int c = j < nv ? sm.keep[j] : 0;
        int tot = 0;
        const int r = run + block_exscan<NT>(c, sm.scan, &tot);
        run += tot;
        if (c) {
            const int pos = j < P ? base2 + r : base3 + (r - k2);
            const int val = j < P ? s.off_2d + j : s.off_3d + (j - P);
            io.kept_idx[out_off + pos] = val;
            if (list) list[kHandWords + pos] = val;
        }
    }
    if (tid == 0) bookkeeping(out_off);                           // nobody in this kernel waits for these
}

}  // namespace mvla
