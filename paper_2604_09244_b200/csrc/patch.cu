// Alg. 1 of the paper taken literally, patch by patch.  A patch p of a sample owns visual token p (2D)
// and visual token P + p (3D), P = n_2d = n_3d.
//
//   patch_indicators_kernel : the four indicators of every patch from the attention copy that the
//                             salience kernel leaves behind (Eq. 3-1, Eq. 3-4, Eq. P2D, Eq. P3D);
//   patch_decide_kernel     : temporal predictor (Eqs. 8, 9), dual threshold (Sec. 4.1), 1-D K-Means and
//                             the semantic rules (Sec. 4.2), fusion (Sec. 4.4) -> keep flags and counts;
//   patch_emit_kernel       : output offsets over the batch and the ordered kept-position lists (Eq. 10).
//
// The data is a few KB to a few MB that sits in L2; these kernels are latency chains, not bandwidth work.
// Every comparison that decides a set is taken in double on the fp32 values, and the K-Means runs in
// double, so that the same fp32 inputs give the same decisions as a double-precision restatement.
#include "common.cuh"
#include "select_impl.cuh"

#include <math_constants.h>

namespace mvla {
namespace {

constexpr int kIndThreads = 256;                     // 32 patches x 8 groups of (head, query) pairs
constexpr int kIndGroups = kIndThreads / 32;
constexpr int kPatchThreads = 1024;
constexpr int kMaxPatch = kMaxVis / 2;
constexpr int kPPT = kMaxPatch / kPatchThreads;      // patches per thread, strided by the block size

// grid = (ceil(max P / 32), samples).  Lane = patch (coalesced over the key index), warp = group of pairs.
__global__ void __launch_bounds__(kIndThreads)
patch_indicators_kernel(const __grid_constant__ BatchDesc bd, int n_heads, const AlphaOut alpha,
                        const float* __restrict__ l1, float* __restrict__ x_out)
{
    __shared__ float red[kIndGroups][32][4];
    const SampleDev& s = bd.s[blockIdx.y];
    const int P = s.n_2d;
    const int p0 = blockIdx.x * 32;
    if (p0 >= P) return;                                  // block-uniform
    const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
    const int p = p0 + lane;
    const bool live = p < P;
    const int npairs = n_heads * s.n_txt;
    const float* base = alpha.ptr + s.vis_off + p;

    // pass 1: <a3, a2>, <a2, a2>, ||a2||_1, ||a3||_1
    float d32 = 0.f, d22 = 0.f, n2 = 0.f, n3 = 0.f;
    if (live) {
#pragma unroll 4
        for (int idx = g; idx < npairs; idx += kIndGroups) {
            const int h = idx / s.n_txt, i = idx - h * s.n_txt;
            const float* a = base + static_cast<int64_t>(h) * alpha.stride_h + static_cast<int64_t>(i) * alpha.stride_i;
            const float a2 = __ldg(a), a3 = __ldg(a + P);
            d32 = fmaf(a3, a2, d32);
            d22 = fmaf(a2, a2, d22);
            n2 += fabsf(a2);
            n3 += fabsf(a3);
        }
    }
    red[g][lane][0] = d32; red[g][lane][1] = d22; red[g][lane][2] = n2; red[g][lane][3] = n3;
    __syncthreads();
    float t[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int w = 0; w < kIndGroups; ++w)                  // fixed order: every warp gets the same totals
#pragma unroll
        for (int c = 0; c < 4; ++c) t[c] += red[w][lane][c];
    const float coef = t[1] > 0.f ? t[0] / t[1] : 0.f;   // projection coefficient of a3 on a2 (Eq. 3-4)
    __syncthreads();

    // pass 2: || a3 - coef a2 ||_1, the part of the 3D token's attention that the 2D token's does not explain
    float no = 0.f;
    if (live) {
#pragma unroll 4
        for (int idx = g; idx < npairs; idx += kIndGroups) {
            const int h = idx / s.n_txt, i = idx - h * s.n_txt;
            const float* a = base + static_cast<int64_t>(h) * alpha.stride_h + static_cast<int64_t>(i) * alpha.stride_i;
            no += fabsf(fmaf(-coef, __ldg(a), __ldg(a + P)));
        }
    }
    red[g][lane][0] = no;
    __syncthreads();
    if (g == 0 && live) {
        float o = 0.f;
#pragma unroll
        for (int w = 0; w < kIndGroups; ++w) o += red[w][lane][0];
        const float f2 = l1[s.vis_off + p], f3 = l1[s.vis_off + P + p];
        float4 x;
        x.x = f2 / (f2 + f3);                             // Eq. 3-1, the term of this patch
        x.y = f3 / (f2 + f3);
        x.z = t[2] / (t[2] + t[3]);                       // Eq. P2D
        x.w = o / (t[2] + t[3]);                          // Eq. P3D
        reinterpret_cast<float4*>(x_out)[s.vis_off / 2 + p] = x;
    }
}

struct PatchSmem {
    double red[kPatchThreads / 32][6];
    double tot[6];
    double centre[3];
};

// Deterministic block reduction of N doubles per thread (fixed shuffle tree, then warp 0 over the warp
// partials).  Component c is a maximum when bit c of `max_mask` is set, else a sum.  Result in sm.tot.
template <int N>
__device__ __forceinline__ void block_reduce_d(double (&v)[N], unsigned max_mask, PatchSmem& sm)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int c = 0; c < N; ++c)
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
            const double o = __shfl_xor_sync(0xffffffffu, v[c], off);
            v[c] = (max_mask >> c & 1u) ? fmax(v[c], o) : v[c] + o;
        }
    __syncthreads();                                      // earlier readers of sm.red / sm.tot are done
    if (lane == 0)
#pragma unroll
        for (int c = 0; c < N; ++c) sm.red[warp][c] = v[c];
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int c = 0; c < N; ++c) {
            double y = sm.red[lane][c];                   // kPatchThreads / 32 == 32 warps
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
                const double o = __shfl_xor_sync(0xffffffffu, y, off);
                y = (max_mask >> c & 1u) ? fmax(y, o) : y + o;
            }
            if (lane == 0) sm.tot[c] = y;
        }
    }
    __syncthreads();
}

// One CTA per sample.
__global__ void __launch_bounds__(kPatchThreads, 1)
patch_decide_kernel(const __grid_constant__ BatchDesc bd, const PatchParams pp, const PatchIO io)
{
    static_assert(kPatchThreads / 32 == 32, "the second reduction level is one warp");
    __shared__ PatchSmem sm;
    const SampleDev& s = bd.s[blockIdx.x];
    const int b_glob = io.chunk_first + blockIdx.x;
    const int tid = threadIdx.x;
    const int P = s.n_2d;
    const int pat_off = s.vis_off / 2;
    const bool carry = s.c_prev != 0.f;
    const bool cold = s.t == 1 && pp.cold_start_full_keep;
    float4* state = reinterpret_cast<float4*>(io.xhat_state) + static_cast<int64_t>(s.mstate_off) * pp.max_patch;

    // ---- stage 1 (action iteration): X^ = c_prev X^ + c_new X for every patch and indicator (Eqs. 8, 9)
    float4 xh[kPPT];
    double mass[kPPT], u[kPPT];
    bool live[kPPT];
    double init[5] = {0.0, -CUDART_INF, -CUDART_INF, 0.0, 0.0};   // sum mass, max mass, max -mass, sum M^S2_2D, sum M^S2_3D
#pragma unroll
    for (int e = 0; e < kPPT; ++e) {
        const int p = tid + e * kPatchThreads;
        live[e] = p < P;
        xh[e] = make_float4(0.f, 0.f, 0.f, 0.f);
        mass[e] = 0.0; u[e] = 0.0;
        if (live[e]) {
            const float4 x = reinterpret_cast<const float4*>(io.x)[pat_off + p];
            float4 v = x;
            if (carry) {
                const float4 pr = state[p];
                v.x = fmaf(s.c_prev, pr.x, s.c_new * x.x);
                v.y = fmaf(s.c_prev, pr.y, s.c_new * x.y);
                v.z = fmaf(s.c_prev, pr.z, s.c_new * x.z);
                v.w = fmaf(s.c_prev, pr.w, s.c_new * x.w);
            }
            xh[e] = v;
            if (s.update_state) state[p] = v;
            if (io.xhat_out) reinterpret_cast<float4*>(io.xhat_out)[pat_off + p] = v;
            // the patch's attention response: the mass of its two tokens
            mass[e] = static_cast<double>(io.attn[s.vis_off + p]) + static_cast<double>(io.attn[s.vis_off + P + p]);
            u[e] = static_cast<double>(io.rand_u[pat_off + p]);
            init[0] += mass[e];
            init[1] = fmax(init[1], mass[e]);
            init[2] = fmax(init[2], -mass[e]);
            init[3] += static_cast<double>(v.z);
            init[4] += static_cast<double>(v.w);
        }
    }
    block_reduce_d<5>(init, 0x6u, sm);
    const double mu_2d = sm.tot[3] / P, mu_3d = sm.tot[4] / P;    // baselines: means of the smoothed shares
    if (tid == 0) {
        sm.centre[0] = -sm.tot[2];                                // min
        sm.centre[1] = sm.tot[0] / P;                             // mean
        sm.centre[2] = sm.tot[1];                                 // max
    }
    __syncthreads();

    // ---- stage 3 preparation: 1-D K-Means, K = 3 (Sec. 4.2).  A round: assign to the nearest centre
    //      (ties to the lower one); unless nothing changed, move the centres to the class means.
    int label[kPPT];
#pragma unroll
    for (int e = 0; e < kPPT; ++e) label[e] = -1;
    int iters = 0;
    while (iters < pp.kmeans_max_iter) {                          // block-uniform
        ++iters;
        const double c0 = sm.centre[0], c1 = sm.centre[1], c2 = sm.centre[2];
        int changed = 0;
        double acc[6] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0};           // class sums, class counts
#pragma unroll
        for (int e = 0; e < kPPT; ++e) {
            if (!live[e]) continue;
            int best = 0;
            double bd_ = fabs(mass[e] - c0);
            const double d1 = fabs(mass[e] - c1), d2 = fabs(mass[e] - c2);
            if (d1 < bd_) { bd_ = d1; best = 1; }
            if (d2 < bd_) { bd_ = d2; best = 2; }
            if (best != label[e]) { label[e] = best; changed = 1; }
            acc[best] += mass[e];
            acc[3 + best] += 1.0;
        }
        if (!__syncthreads_or(changed)) break;
        block_reduce_d<6>(acc, 0u, sm);
        if (tid == 0)
#pragma unroll
            for (int c = 0; c < 3; ++c)
                if (sm.tot[3 + c] > 0.0) sm.centre[c] = sm.tot[c] / sm.tot[3 + c];
        __syncthreads();
    }

    // ---- stages 2-4 for every patch: C_S1 (dual threshold), C_S2 (semantic rules), fusion, masks
    const int both = MVLA_SET_2D | MVLA_SET_3D;
    double cnt[5] = {0.0, 0.0, 0.0, 0.0, 0.0};                    // kept 2D, kept 3D, patches per class
#pragma unroll
    for (int e = 0; e < kPPT; ++e) {
        if (!live[e]) continue;
        const int p = tid + e * kPatchThreads;
        const double s1_3d = xh[e].y, m2 = xh[e].z, m3 = xh[e].w;
        const int c1 = s1_3d < pp.tau_2d ? MVLA_SET_2D : (s1_3d > pp.tau_3d ? MVLA_SET_3D : both);
        int c2;
        if (label[e] == MVLA_LABEL_BG) c2 = u[e] < pp.bg_prune_prob ? 0 : both;
        else if (label[e] == MVLA_LABEL_ROB) c2 = m3 > mu_3d ? both : (m2 > mu_2d ? MVLA_SET_2D : 0);
        else c2 = (m2 > pp.obj_2d_min && m3 < pp.eps_3d) ? MVLA_SET_2D : both;
        int cf = 0;
        if (c2 != 0) {
            cf = c2 & c1;
            if (cf == 0) cf = c2;                                 // conflict resolution
        }
        if (cold) cf = both;                                      // cold start: full unpruned tokens
        if (io.info_out) io.info_out[pat_off + p] = label[e] | (c1 << 2) | (c2 << 4) | (cf << 6);
        io.mask_ws[s.vis_off + p] = (cf & MVLA_SET_2D) ? 1 : 0;
        io.mask_ws[s.vis_off + P + p] = (cf & MVLA_SET_3D) ? 1 : 0;
        cnt[0] += (cf & MVLA_SET_2D) ? 1.0 : 0.0;
        cnt[1] += (cf & MVLA_SET_3D) ? 1.0 : 0.0;
        cnt[2 + label[e]] += 1.0;
    }
    block_reduce_d<5>(cnt, 0u, sm);
    if (tid == 0) {
        const int k2 = static_cast<int>(sm.tot[0]), k3 = static_cast<int>(sm.tot[1]);
        io.nout_ws[b_glob * 4 + 0] = s.n_txt + k2 + k3;
        io.nout_ws[b_glob * 4 + 1] = k2;
        io.nout_ws[b_glob * 4 + 2] = k3;
        if (io.counts) { io.counts[b_glob * 2] = k2; io.counts[b_glob * 2 + 1] = k3; }
        if (io.diag) {
            mvla_patch_diag dg;
            dg.t = s.t; dg.iters = iters;
            for (int c = 0; c < 3; ++c) { dg.n_label[c] = static_cast<int>(sm.tot[2 + c]); dg.centre[c] = static_cast<float>(sm.centre[c]); }
            dg.k_2d = k2; dg.k_3d = k3; dg.n_out = s.n_txt + k2 + k3;
            dg.mu_2d = static_cast<float>(mu_2d); dg.mu_3d = static_cast<float>(mu_3d);
            dg.reserved[0] = dg.reserved[1] = dg.reserved[2] = 0.f;
            io.diag[b_glob] = dg;
        }
    }
}

// One CTA per sample: its first output row (the kept rows of the samples before it), then the kept
// positions in sequence order.  The three segments are contiguous, so a kept token's output row is the
// rows of the segments lying before its own plus its rank inside its modality.
__global__ void __launch_bounds__(kPatchThreads, 1)
patch_emit_kernel(const __grid_constant__ BatchDesc bd, const PatchIO io)
{
    __shared__ int scan[kPatchThreads / 32 + 1];
    __shared__ int s_off;
    const SampleDev& s = bd.s[blockIdx.x];
    const int b_glob = io.chunk_first + blockIdx.x;
    const int tid = threadIdx.x;
    const int P = s.n_2d, nv = 2 * P;
    if (tid == 0) {
        int off = 0;
        for (int b = 0; b < b_glob; ++b) off += io.nout_ws[b * 4];
        s_off = off;
        io.out_offsets[b_glob] = off;
        if (b_glob == io.batch_total - 1) io.out_offsets[io.batch_total] = off + io.nout_ws[b_glob * 4];
    }
    __syncthreads();
    const int out_off = s_off;
    const int k2 = io.nout_ws[b_glob * 4 + 1], k3 = io.nout_ws[b_glob * 4 + 2];
    const int base2 = (s.off_txt < s.off_2d ? s.n_txt : 0) + (s.off_3d < s.off_2d ? k3 : 0);
    const int base3 = (s.off_txt < s.off_3d ? s.n_txt : 0) + (s.off_2d < s.off_3d ? k2 : 0);
    const int baset = (s.off_2d < s.off_txt ? k2 : 0) + (s.off_3d < s.off_txt ? k3 : 0);
    for (int i = tid; i < s.n_txt; i += kPatchThreads) io.kept_idx[out_off + baset + i] = s.off_txt + i;
    int run = 0;
    for (int j0 = 0; j0 < nv; j0 += kPatchThreads) {              // block-uniform
        const int j = j0 + tid;
        const int c = j < nv ? io.mask_ws[s.vis_off + j] : 0;
        int tot = 0;
        const int r = run + block_exscan<kPatchThreads>(c, scan, &tot);
        run += tot;
        if (c) {
            if (j < P) io.kept_idx[out_off + base2 + r] = s.off_2d + j;
            else       io.kept_idx[out_off + base3 + (r - k2)] = s.off_3d + (j - P);
        }
    }
}

}  // namespace

cudaError_t launch_patch_indicators(const BatchDesc& bd, int n_heads, AlphaOut alpha, const float* l1,
                                    float* x_out, cudaStream_t stream)
{
    int max_p = 0;
    for (int b = 0; b < bd.n; ++b) max_p = max(max_p, bd.s[b].n_2d);
    if (max_p == 0) return cudaSuccess;
    patch_indicators_kernel<<<dim3((max_p + 31) / 32, bd.n), kIndThreads, 0, stream>>>(bd, n_heads, alpha, l1, x_out);
    return cudaGetLastError();
}

cudaError_t launch_patch_decide(const BatchDesc& bd, const PatchParams& pp, const PatchIO& io, cudaStream_t stream)
{
    patch_decide_kernel<<<bd.n, kPatchThreads, 0, stream>>>(bd, pp, io);
    return cudaGetLastError();
}

cudaError_t launch_patch_emit(const BatchDesc& bd, const PatchIO& io, cudaStream_t stream)
{
    patch_emit_kernel<<<bd.n, kPatchThreads, 0, stream>>>(bd, io);
    return cudaGetLastError();
}

}  // namespace mvla
