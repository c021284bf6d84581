// Alg. 1 of the paper taken literally, patch by patch.  A patch p of a sample owns visual token p (2D)
// and visual token P + p (3D), P = n_2d = n_3d.
//
//   patch_indicators_kernel : the four indicators of every patch from the attention copy that the
//                             salience kernel leaves behind (Eq. 3-1, Eq. 3-4, Eq. P2D, Eq. P3D);
//   patch_select_kernel     : temporal predictor (Eqs. 8, 9), dual threshold (Sec. 4.1), 1-D K-Means and
//                             the semantic rules (Sec. 4.2), fusion (Sec. 4.4), then the output offsets
//                             over the batch and the ordered kept-position lists (Eq. 10).
//
// The data is a few KB to a few MB that sits in L2; these kernels are latency chains, not bandwidth work.
// Every comparison that decides a set is taken in double on the fp32 values, and the K-Means runs in
// double, so that the same fp32 inputs give the same decisions as a double-precision restatement.
#include "common.cuh"
#include "select_impl.cuh"

#include <math_constants.h>

namespace mvla {
namespace {

constexpr int kIndThreads = 512;
constexpr int kPatchThreads = 256;
constexpr int kMaxPatch = kMaxVis / 2;
constexpr int kPPT = kMaxPatch / kPatchThreads;      // patches per thread, strided by the block size

// grid = (ceil(max P / PP), samples), PP = 2, 4 or 8 patches per CTA (8 floats = one 32-byte sector per
// (head, query); fewer patches per CTA when the batch is too small to fill the SMs otherwise).
// Thread = (patch, group): the group walks the (head, query) pairs with stride 512 / PP, so a CTA has
// all its loads of a pass in flight at once (a few per thread).
// Also writes the per-token scores of the patch's two tokens: a_j = ||alpha_j||_1 / (H n_t).
// The L1 feature norms of the CTA's 2 PP rows (Sec. 3.1.2) are taken here too, 256 / PP threads per row,
// their loads issued before the kernel waits for the attention copy of the kernel before it.
template <typename T, int PP>
__global__ void __launch_bounds__(kIndThreads, 1)
patch_indicators_kernel(const __grid_constant__ BatchDesc bd, int n_heads, const AlphaOut alpha,
                        const T* __restrict__ hidden, int d_model, float* __restrict__ x_out,
                        float* __restrict__ attn_out)
{
    constexpr int kIndPatches = PP;
    constexpr int kIndGroups = kIndThreads / PP;          // groups of (head, query) pairs
    constexpr int kRowThreads = kIndThreads / (2 * PP);   // threads that share one hidden row
    __shared__ float red[kIndThreads / 32][kIndPatches][4];
    __shared__ float tot[kIndPatches][4];
    __shared__ float rown[kIndThreads / 32];
    const SampleDev& s = bd.s[blockIdx.y];
    const int P = s.n_2d;
    const int p0 = blockIdx.x * kIndPatches;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p0 >= P) return;                                  // block-uniform
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pl = tid & (kIndPatches - 1), g = tid / kIndPatches;
    const int p = p0 + pl;
    const bool live = p < P;
    const int npairs = n_heads * s.n_txt;
    const float* base = alpha.ptr + s.vis_off + p;

    // ---- feature norms: row r of the CTA = 2D token p0 + r (r < PP) or 3D token p0 + r - PP
    {
        const int r = tid / kRowThreads, within = tid % kRowThreads;
        const int pr = p0 + (r & (kIndPatches - 1));
        float acc = 0.f;
        if (pr < P) {
            const int row = s.seq_off + (r < kIndPatches ? s.off_2d : s.off_3d) + pr;
            constexpr int kVec = 16 / sizeof(T);
            const uint4* src = reinterpret_cast<const uint4*>(hidden + static_cast<int64_t>(row) * d_model);
            const int nvec = d_model / kVec;
#pragma unroll 8
            for (int i = within; i < nvec; i += kRowThreads) {
                const uint4 u = __ldg(src + i);
                if constexpr (sizeof(T) == 2) {
                    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        acc += fabsf(__uint_as_float(w[e] << 16));           // low bf16
                        acc += fabsf(__uint_as_float(w[e] & 0xFFFF0000u));   // high bf16
                    }
                } else {
                    acc += fabsf(__uint_as_float(u.x)) + fabsf(__uint_as_float(u.y)) +
                           fabsf(__uint_as_float(u.z)) + fabsf(__uint_as_float(u.w));
                }
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) rown[warp] = acc;                  // read after the barriers of the first reduction
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");    // the attention copy comes from the kernel before this one

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

    // pass 1: <a3, a2>, <a2, a2>, ||a2||_1, ||a3||_1
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (live) {
#pragma unroll 4
        for (int idx = g; idx < npairs; idx += kIndGroups) {
            const int h = idx / s.n_txt, i = idx - h * s.n_txt;
            const float* a = base + static_cast<int64_t>(h) * alpha.stride_h + static_cast<int64_t>(i) * alpha.stride_i;
            const float a2 = __ldcg(a), a3 = __ldcg(a + P);
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
    if (live) {
#pragma unroll 4
        for (int idx = g; idx < npairs; idx += kIndGroups) {
            const int h = idx / s.n_txt, i = idx - h * s.n_txt;
            const float* a = base + static_cast<int64_t>(h) * alpha.stride_h + static_cast<int64_t>(i) * alpha.stride_i;
            o[0] += fabsf(fmaf(-coef, __ldcg(a), __ldcg(a + P)));
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
    }
}

struct PatchSmem {
    double mass[kMaxPatch];                 // attention mass of every patch (what K-Means clusters)
    uint8_t label[kMaxPatch];
    uint8_t keep[2 * kMaxPatch];            // keep flags in visual order: 2D tokens, then 3D tokens
    double red[kPatchThreads / 32][5];
    double tot[5];
    double centre[3];
    int cnt[5];                             // kept 2D, kept 3D, patches per class
    int iters;
    int out_off;
    int scan[kPatchThreads / 32 + 1];
};

// Deterministic block reduction of 5 doubles per thread (fixed shuffle tree, then warp 0 over the warp
// partials).  Component c is a maximum when bit c of `max_mask` is set, else a sum.  Result in sm.tot.
__device__ __forceinline__ void block_reduce5(double (&v)[5], unsigned max_mask, PatchSmem& sm)
{
    constexpr int NW = kPatchThreads / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int c = 0; c < 5; ++c)
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            const double o = __shfl_xor_sync(0xffffffffu, v[c], off);
            v[c] = (max_mask >> c & 1u) ? fmax(v[c], o) : v[c] + o;
        }
    if (lane == 0)
#pragma unroll
        for (int c = 0; c < 5; ++c) sm.red[warp][c] = v[c];
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int c = 0; c < 5; ++c) {
            const bool is_max = (max_mask >> c & 1u) != 0;
            double y = lane < NW ? sm.red[lane][c] : (is_max ? -CUDART_INF : 0.0);
#pragma unroll
            for (int off = NW / 2; off >= 1; off >>= 1) {
                const double o = __shfl_xor_sync(0xffffffffu, y, off);
                y = is_max ? fmax(y, o) : y + o;
            }
            if (lane == 0) sm.tot[c] = y;
        }
    }
    __syncthreads();
}

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
__global__ void __launch_bounds__(kPatchThreads, 1)
patch_select_kernel(const __grid_constant__ BatchDesc bd, const PatchParams pp, const PatchIO io)
{
    __shared__ PatchSmem sm;
    const SampleDev& s = bd.s[blockIdx.x];
    const int b_glob = io.chunk_first + blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int P = s.n_2d, nv = 2 * P;
    const int pat_off = s.vis_off / 2;
    const bool carry = s.c_prev != 0.f;
    const bool cold = s.t == 1 && pp.cold_start_full_keep;
    float4* state = reinterpret_cast<float4*>(io.xhat_state) + static_cast<int64_t>(s.slot_index) * pp.max_patch;
    if (tid < 5) sm.cnt[tid] = 0;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");    // scores and indicators come from the kernel before this one

    // ---- stage 1 (action iteration): X^ = c_prev X^ + c_new X for every patch and indicator (Eqs. 8, 9).
    //      All loads of a thread are issued before anything depends on them.
    float4 x[kPPT], pr[kPPT];
    float a2[kPPT], a3[kPPT], uu[kPPT];
#pragma unroll
    for (int e = 0; e < kPPT; ++e) {
        if (e * kPatchThreads >= P) break;                        // block-uniform
        const int p = tid + e * kPatchThreads;
        if (p < P) {
            x[e] = reinterpret_cast<const float4*>(io.x)[pat_off + p];
            if (carry) pr[e] = state[p];
            a2[e] = io.attn[s.vis_off + p];
            a3[e] = io.attn[s.vis_off + P + p];
            uu[e] = io.rand_u[pat_off + p];
        }
    }
    float4 xh[kPPT];
    double init[5] = {0.0, -CUDART_INF, -CUDART_INF, 0.0, 0.0};   // sum mass, max mass, max -mass, sum M^S2_2D, sum M^S2_3D
#pragma unroll
    for (int e = 0; e < kPPT; ++e) {
        if (e * kPatchThreads >= P) break;
        const int p = tid + e * kPatchThreads;
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
            sm.label[p] = 255;
            init[0] += m;
            init[1] = fmax(init[1], m);
            init[2] = fmax(init[2], -m);
            init[3] += static_cast<double>(v.z);
            init[4] += static_cast<double>(v.w);
        }
    }
    block_reduce5(init, 0x6u, sm);
    const double mu_2d = sm.tot[3] / P, mu_3d = sm.tot[4] / P;    // baselines: means of the smoothed shares

    // ---- stage 3 preparation: 1-D K-Means, K = 3 (Sec. 4.2), by one warp without block barriers.  A round:
    //      assign to the nearest centre (ties to the lower one); unless nothing changed, move the centres
    //      to the class means.
    if (warp == 0) {
        double c0 = -sm.tot[2], c1 = sm.tot[0] / P, c2 = sm.tot[1];   // min, mean, max
        int iters = 0;
        while (iters < pp.kmeans_max_iter) {                      // warp-uniform
            ++iters;
            int changed = 0;
            double s0 = 0.0, s1 = 0.0, s2 = 0.0, n0 = 0.0, n1 = 0.0, n2 = 0.0;
            for (int p = lane; p < P; p += 32) {
                const double m = sm.mass[p];
                int best = 0;
                double bdist = fabs(m - c0);
                const double d1 = fabs(m - c1), d2 = fabs(m - c2);
                if (d1 < bdist) { bdist = d1; best = 1; }
                if (d2 < bdist) { bdist = d2; best = 2; }
                if (sm.label[p] != best) { sm.label[p] = static_cast<uint8_t>(best); changed = 1; }
                s0 += best == 0 ? m : 0.0; n0 += best == 0 ? 1.0 : 0.0;
                s1 += best == 1 ? m : 0.0; n1 += best == 1 ? 1.0 : 0.0;
                s2 += best == 2 ? m : 0.0; n2 += best == 2 ? 1.0 : 0.0;
            }
            if (!__any_sync(0xffffffffu, changed)) break;
            s0 = warp_sum_d(s0); s1 = warp_sum_d(s1); s2 = warp_sum_d(s2);
            n0 = warp_sum_d(n0); n1 = warp_sum_d(n1); n2 = warp_sum_d(n2);
            if (n0 > 0.0) c0 = s0 / n0;
            if (n1 > 0.0) c1 = s1 / n1;
            if (n2 > 0.0) c2 = s2 / n2;
        }
        if (lane == 0) { sm.centre[0] = c0; sm.centre[1] = c1; sm.centre[2] = c2; sm.iters = iters; }
    }
    __syncthreads();

    // ---- stages 2-4 for every patch: C_S1 (dual threshold), C_S2 (semantic rules), fusion, masks
    const int both = MVLA_SET_2D | MVLA_SET_3D;
#pragma unroll
    for (int e = 0; e < kPPT; ++e) {
        if (e * kPatchThreads >= P) break;
        const int p = tid + e * kPatchThreads;
        if (p < P) {
            const int label = sm.label[p];
            const double s1_3d = xh[e].y, m2 = xh[e].z, m3 = xh[e].w;
            const int c1 = s1_3d < pp.tau_2d ? MVLA_SET_2D : (s1_3d > pp.tau_3d ? MVLA_SET_3D : both);
            int c2;
            if (label == MVLA_LABEL_BG) c2 = static_cast<double>(uu[e]) < pp.bg_prune_prob ? 0 : both;
            else if (label == MVLA_LABEL_ROB) c2 = m3 > mu_3d ? both : (m2 > mu_2d ? MVLA_SET_2D : 0);
            else c2 = (m2 > pp.obj_2d_min && m3 < pp.eps_3d) ? MVLA_SET_2D : both;
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
    const int k2 = sm.cnt[0], k3 = sm.cnt[1];
    const int n_out = s.n_txt + k2 + k3;

    // ---- first output row: publish this sample's count, add up the counts of the samples before it
    const bool alone = gridDim.x == 1;                            // nobody in this launch to wait for or to tell
    if (warp == 0) {
        if (lane == 0) {
            io.nout_ws[b_glob] = n_out;                           // later launches of this call read it in stream order
            if (!alone) {
                __threadfence();
                asm volatile("st.volatile.global.s32 [%0], %1;" ::"l"(io.ready_ws + b_glob), "r"(1) : "memory");
            }
        }
        int off = 0;
        bool ok = true;
        for (int b = lane; b < b_glob; b += 32) {
            if (b >= io.chunk_first) {                            // same launch: wait for its flag (bounded)
                bool got = false;
                for (uint32_t it = 0; it < kSpinLimit && !got; ++it) {
                    got = ld_volatile_i32(io.ready_ws + b) != 0;
                    if (!got) __nanosleep(64);
                }
                ok &= got;
                __threadfence();
            }
            off += ld_volatile_i32(io.nout_ws + b);               // earlier launches of this call are complete
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
        if (!__all_sync(0xffffffffu, ok) && lane == 0) *reinterpret_cast<volatile int*>(io.status) = MVLA_ERR_TIMEOUT;
        if (lane == 0) {
            sm.out_off = off;
            io.out_offsets[b_glob] = off;
            if (b_glob == io.batch_total - 1) io.out_offsets[io.batch_total] = off + n_out;
            if (io.counts) { io.counts[b_glob * 2] = k2; io.counts[b_glob * 2 + 1] = k3; }
            if (io.diag) {
                mvla_patch_diag dg;
                dg.t = s.t; dg.iters = sm.iters;
                for (int c = 0; c < 3; ++c) { dg.n_label[c] = sm.cnt[2 + c]; dg.centre[c] = static_cast<float>(sm.centre[c]); }
                dg.k_2d = k2; dg.k_3d = k3; dg.n_out = n_out;
                dg.mu_2d = static_cast<float>(mu_2d); dg.mu_3d = static_cast<float>(mu_3d);
                dg.reserved[0] = dg.reserved[1] = dg.reserved[2] = 0.f;
                io.diag[b_glob] = dg;
            }
            // every wait of this CTA is over: the CTA that gets here last clears the flags of the launch
            if (!alone) __threadfence();
            if (!alone && atomicAdd(io.done_ws, 1) == static_cast<int>(gridDim.x) - 1) {
                for (int b = 0; b < static_cast<int>(gridDim.x); ++b) io.ready_ws[io.chunk_first + b] = 0;
                *io.done_ws = 0;
                __threadfence();
            }
        }
    }
    __syncthreads();

    // ---- Eq. 10 as an ordered list.  The three segments are contiguous, so a kept token's output row is
    //      the rows of the segments lying before its own plus its rank inside its modality.
    const int out_off = sm.out_off;
    const int base2 = (s.off_txt < s.off_2d ? s.n_txt : 0) + (s.off_3d < s.off_2d ? k3 : 0);
    const int base3 = (s.off_txt < s.off_3d ? s.n_txt : 0) + (s.off_2d < s.off_3d ? k2 : 0);
    const int baset = (s.off_2d < s.off_txt ? k2 : 0) + (s.off_3d < s.off_txt ? k3 : 0);
    for (int i = tid; i < s.n_txt; i += kPatchThreads) io.kept_idx[out_off + baset + i] = s.off_txt + i;
    int run = 0;
    for (int j0 = 0; j0 < nv; j0 += kPatchThreads) {              // block-uniform
        const int j = j0 + tid;
        const int c = j < nv ? sm.keep[j] : 0;
        int tot = 0;
        const int r = run + block_exscan<kPatchThreads>(c, sm.scan, &tot);
        run += tot;
        if (c) {
            if (j < P) io.kept_idx[out_off + base2 + r] = s.off_2d + j;
            else       io.kept_idx[out_off + base3 + (r - k2)] = s.off_3d + (j - P);
        }
    }
}

}  // namespace

cudaError_t launch_patch_indicators(const BatchDesc& bd, int n_heads, AlphaOut alpha, int dtype, int d_model,
                                    const void* hidden, float* x_out, float* attn_out, cudaStream_t stream)
{
    int max_p = 0;
    for (int b = 0; b < bd.n; ++b) max_p = max(max_p, bd.s[b].n_2d);
    if (max_p == 0) return cudaSuccess;
    // as many patches per CTA as still give every multiprocessor a CTA
    int pp = 8;
    const int sms = sm_count_of_current_device();
    while (pp > 2 && static_cast<int64_t>(bd.n) * ((max_p + pp - 1) / pp) < sms) pp >>= 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((max_p + pp - 1) / pp, bd.n);
    cfg.blockDim = dim3(kIndThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
#define MVLA_IND(T, PPV)                                                                                  \
    if (pp == PPV)                                                                                        \
        return cudaLaunchKernelEx(&cfg, patch_indicators_kernel<T, PPV>, bd, n_heads, alpha,              \
                                  static_cast<const T*>(hidden), d_model, x_out, attn_out);
    if (dtype == MVLA_DTYPE_BF16) { MVLA_IND(__nv_bfloat16, 8) MVLA_IND(__nv_bfloat16, 4) MVLA_IND(__nv_bfloat16, 2) }
    else { MVLA_IND(float, 8) MVLA_IND(float, 4) MVLA_IND(float, 2) }
#undef MVLA_IND
    return cudaErrorInvalidConfiguration;
}

cudaError_t launch_patch_select(const BatchDesc& bd, const PatchParams& pp, const PatchIO& io, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(bd.n);
    cfg.blockDim = dim3(kPatchThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, patch_select_kernel, bd, pp, io);
}

}  // namespace mvla
