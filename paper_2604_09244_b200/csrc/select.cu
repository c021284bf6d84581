// Carry-over, budget split and top-k selection (Alg. 1 of the paper, steps 1-4; Eqs. 8, 9, 10).
//
// One CTA of 1024 threads per sample:
//   1. gather the instantaneous scores a_j (summing the per-head partials in head order),
//      smooth them into the per-token state (Eq. 8 / Eq. 9 as  xhat = c_prev xhat + c_new x),
//   2. reduce the modality sums -> the four indicators, smooth those too, evaluate the dual
//      threshold (Sec. 4.1), the target-object rule (Sec. 4.2) and the fusion (Sec. 4.4),
//      split the budget,
//   3. radix-select the k-th largest smoothed score of each modality (4 passes of 8 bits on an
//      order-preserving 32-bit key, both modalities at once),
//   4. emit the kept positions in sequence order, merged with all text positions: elements above
//      the threshold, plus the first (lowest-index) elements equal to it, via two block-wide
//      ballot / prefix scans.
#include "common.cuh"

#include <math_constants.h>

namespace mvla {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kPerThread = kMaxVis / kSelThreads;          // strided elements per thread (8)
constexpr int kMaxSeq = kMaxVis + kMaxText;
constexpr int kPosPerThread = (kMaxSeq + kSelThreads - 1) / kSelThreads;

// fp32 -> uint32 whose unsigned order is the float order; NaN sorts below everything.
__device__ __forceinline__ uint32_t order_key(float x)
{
    if (x != x) return 0u;
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Deterministic block sum of up to 4 values per thread (fixed shuffle tree, fixed warp order).
struct Sum4 { float v[4]; };
__device__ Sum4 block_sum4(Sum4 x, float (*scratch)[4])
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) x.v[c] += __shfl_xor_sync(0xffffffffu, x.v[c], off);
    __syncthreads();
    if (lane == 0)
#pragma unroll
        for (int c = 0; c < 4; ++c) scratch[warp][c] = x.v[c];
    __syncthreads();
    Sum4 r;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        float acc = 0.f;
        for (int w = 0; w < kSelWarps; ++w) acc += scratch[w][c];
        r.v[c] = acc;
    }
    return r;
}

// Exclusive block scan of one int per thread; returns the exclusive prefix, *total gets the sum.
__device__ int block_exscan(int x, int* warp_tot, int* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = x;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += n;
    }
    __syncthreads();
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int t = warp_tot[lane];
        int winc = t;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, winc, off);
            if (lane >= off) winc += n;
        }
        warp_tot[lane] = winc - t;                 // exclusive prefix of the warp totals
        if (lane == 31) warp_tot[32] = winc;
    }
    __syncthreads();
    if (total) *total = warp_tot[32];
    return warp_tot[warp] + inc - x;
}

__global__ void __launch_bounds__(kSelThreads, 1)
select_kernel(const __grid_constant__ BatchDesc bd, const GateParams gp, const float* __restrict__ attn,
              const float* __restrict__ part, int64_t part_stride, int n_heads,
              const float* __restrict__ l1, float* __restrict__ ahat_state, float* __restrict__ mhat_state,
              int32_t* __restrict__ kept_idx, int32_t* __restrict__ out_offsets, int chunk_first,
              int32_t total_out, int write_total, int32_t* __restrict__ budgets,
              float* __restrict__ attn_out, float* __restrict__ ahat_out, float* __restrict__ z_out,
              mvla_diag* __restrict__ diag)
{
    __shared__ uint32_t s_key[kMaxVis];
    __shared__ float s_red[kSelWarps][4];
    __shared__ int s_hist[2][256];
    __shared__ int s_scan[kSelWarps + 1];
    __shared__ uint32_t s_prefix[2];
    __shared__ int s_krem[2];
    __shared__ int s_k[2];

    const SampleDev& s = bd.s[blockIdx.x];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n2 = s.n_2d, n3 = s.n_3d, nv = n2 + n3;

    // ---- 1. scores, smoothing, modality sums
    float ah[kPerThread];
    Sum4 acc = {{0.f, 0.f, 0.f, 0.f}};      // sum a over 2D, sum a over 3D, sum l1 over 2D, sum l1 over 3D
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) {
        const int j = tid + e * kSelThreads;
        ah[e] = 0.f;
        if (j < nv) {
            float a;
            if (part) {
                a = 0.f;
                for (int h = 0; h < n_heads; ++h) a += part[static_cast<int64_t>(h) * part_stride + s.vis_off + j];
            } else {
                a = attn[s.vis_off + j];
            }
            if (attn_out) attn_out[s.vis_off + j] = a;
            const float prev = s.c_prev != 0.f ? ahat_state[s.state_off + j] : 0.f;
            const float sm = s.c_prev != 0.f ? fmaf(s.c_prev, prev, s.c_new * a) : a;
            ah[e] = sm;
            if (s.update_state) ahat_state[s.state_off + j] = sm;
            if (ahat_out) ahat_out[s.vis_off + j] = sm;
            s_key[j] = order_key(sm);
            const float n = gp.has_l1 ? l1[s.vis_off + j] : 0.f;
            if (j < n2) { acc.v[0] += a; acc.v[2] += n; }
            else        { acc.v[1] += a; acc.v[3] += n; }
        }
    }
    const Sum4 tot = block_sum4(acc, s_red);

    // optional: the smoothed scores normalised to mean one inside each modality.  The ranking
    // below uses the smoothed scores themselves; a positive per-modality factor cannot change it.
    if (z_out) {
        Sum4 sa = {{0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) {
            const int j = tid + e * kSelThreads;
            if (j < nv) sa.v[j >= n2] += ah[e];
        }
        const Sum4 st = block_sum4(sa, s_red);
        const float f2 = static_cast<float>(n2) / st.v[0], f3 = static_cast<float>(n3) / st.v[1];
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) {
            const int j = tid + e * kSelThreads;
            if (j < nv) z_out[s.vis_off + j] = ah[e] * (j < n2 ? f2 : f3);
        }
    }

    // ---- 2. indicators, gates, budget (one thread; a few dozen flops)
    if (tid == 0) {
        float x[4];
        x[3] = tot.v[1] / (tot.v[0] + tot.v[1]);                 // attention share of 3D (Eq. P2D / P3D)
        x[2] = 1.f - x[3];
        if (gp.has_l1) {                                          // feature-norm share (Eq. 3-1), mean norms
            const float m2 = n2 > 0 ? tot.v[2] / static_cast<float>(n2) : 0.f;
            const float m3 = n3 > 0 ? tot.v[3] / static_cast<float>(n3) : 0.f;
            x[1] = m3 / (m2 + m3);
            x[0] = 1.f - x[1];
        } else {
            x[0] = x[1] = 0.5f;
        }
        float mh[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            mh[c] = s.c_prev != 0.f ? fmaf(s.c_prev, mhat_state[s.mstate_off * 4 + c], s.c_new * x[c]) : x[c];
            if (s.update_state) mhat_state[s.mstate_off * 4 + c] = mh[c];
        }
        int c1 = mh[1] < gp.tau_2d ? MVLA_SET_2D : (mh[1] > gp.tau_3d ? MVLA_SET_3D : (MVLA_SET_2D | MVLA_SET_3D));
        int c2 = mh[3] < gp.eps_3d ? MVLA_SET_2D : (MVLA_SET_2D | MVLA_SET_3D);
        int cf = c2 & c1;
        if (cf == 0) cf = c2;
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
        s_k[0] = k2;
        s_k[1] = k3;
        s_krem[0] = k2;
        s_krem[1] = k3;
        s_prefix[0] = s_prefix[1] = 0u;
        if (budgets) {
            budgets[(chunk_first + blockIdx.x) * 2 + 0] = k2;
            budgets[(chunk_first + blockIdx.x) * 2 + 1] = k3;
        }
        if (diag) {
            mvla_diag dg;
            dg.t = s.t; dg.c_s1 = c1; dg.c_s2 = c2; dg.c_final = cf;
            dg.budget = s.budget; dg.k_2d = k2; dg.k_3d = k3; dg.reserved = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) { dg.x[c] = x[c]; dg.mhat[c] = mh[c]; }
            diag[chunk_first + blockIdx.x] = dg;
        }
        out_offsets[chunk_first + blockIdx.x] = s.out_off;
        if (write_total && blockIdx.x == gridDim.x - 1) out_offsets[chunk_first + gridDim.x] = total_out;
    }
    for (int i = tid; i < 512; i += kSelThreads) (&s_hist[0][0])[i] = 0;
    __syncthreads();

    // ---- 3. radix select: after the four passes s_prefix[m] is the key of the k_m-th largest
    //         element of modality m and s_krem[m] how many elements equal to it are kept.
    for (int shift = 24; shift >= 0; shift -= 8) {
        const uint32_t himask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) {
            const int j = tid + e * kSelThreads;
            if (j < nv) {
                const int m = j >= n2;
                const uint32_t key = s_key[j];
                if (((key ^ s_prefix[m]) & himask) == 0u) atomicAdd(&s_hist[m][(key >> shift) & 255u], 1);
            }
        }
        __syncthreads();
        if (warp < 2 && s_k[warp] > 0) {
            // lane L owns the 8 digits 255-8L .. 248-8L (descending); find the digit where the
            // count of elements with a larger digit first reaches k
            const int m = warp, krem = s_krem[m];
            int cnt[8], mine = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { cnt[i] = s_hist[m][255 - 8 * lane - i]; mine += cnt[i]; }
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
                        s_prefix[m] |= static_cast<uint32_t>(255 - 8 * lane - i) << shift;
                        s_krem[m] = krem - above;
                        break;
                    }
                    above += cnt[i];
                }
            }
        }
        __syncthreads();
        for (int i = tid; i < 512; i += kSelThreads) (&s_hist[0][0])[i] = 0;
        __syncthreads();
    }

    // ---- 4. emission in sequence order.  Thread t owns positions [t*P, t*P + P).
    const int seq = s.n_txt + nv;
    const int P = (seq + kSelThreads - 1) / kSelThreads;
    const int p0 = tid * P;
    const uint32_t th2 = s_prefix[0], th3 = s_prefix[1];
    const int need2 = s_k[0] > 0 ? s_krem[0] : 0, need3 = s_k[1] > 0 ? s_krem[1] : 0;
    const bool any2 = s_k[0] > 0, any3 = s_k[1] > 0;

    // class of a position: 0 dropped, 1 kept, 2 tie in 2D, 3 tie in 3D
    int cls[kPosPerThread];
    int ties = 0;                                   // low 16 bits: 2D ties, high 16 bits: 3D ties
#pragma unroll
    for (int i = 0; i < kPosPerThread; ++i) {
        const int p = p0 + i;
        int c = 0;
        if (i < P && p < seq) {
            if (p >= s.off_txt && p < s.off_txt + s.n_txt) c = 1;
            else if (p >= s.off_2d && p < s.off_2d + n2) {
                const uint32_t key = s_key[p - s.off_2d];
                c = !any2 ? 0 : (key > th2 ? 1 : (key == th2 ? 2 : 0));
            } else if (p >= s.off_3d && p < s.off_3d + n3) {
                const uint32_t key = s_key[n2 + p - s.off_3d];
                c = !any3 ? 0 : (key > th3 ? 1 : (key == th3 ? 3 : 0));
            }
        }
        cls[i] = c;
        ties += (c == 2) + ((c == 3) << 16);
    }
    int tie_rank = block_exscan(ties, s_scan, nullptr);
    int r2 = tie_rank & 0xFFFF, r3 = tie_rank >> 16;
    int kept = 0;
#pragma unroll
    for (int i = 0; i < kPosPerThread; ++i) {
        if (cls[i] == 2) cls[i] = (r2++ < need2) ? 1 : 0;        // lower index wins
        else if (cls[i] == 3) cls[i] = (r3++ < need3) ? 1 : 0;
        kept += cls[i];
    }
    int pos = block_exscan(kept, s_scan, nullptr);
#pragma unroll
    for (int i = 0; i < kPosPerThread; ++i)
        if (cls[i]) kept_idx[s.out_off + pos++] = p0 + i;
}

}  // namespace

cudaError_t launch_select(const BatchDesc& bd, const GateParams& gp, const float* attn, const float* part,
                          int64_t part_stride, int n_heads, const float* l1, float* ahat_state,
                          float* mhat_state, int32_t* kept_idx, int32_t* out_offsets, int chunk_first,
                          int32_t total_out, int write_total, int32_t* budgets, float* attn_out,
                          float* ahat_out, float* z_out, mvla_diag* diag, cudaStream_t stream)
{
    select_kernel<<<bd.n, kSelThreads, 0, stream>>>(bd, gp, attn, part, part_stride, n_heads, l1, ahat_state,
                                                    mhat_state, kept_idx, out_offsets, chunk_first, total_out,
                                                    write_total, budgets, attn_out, ahat_out, z_out, diag);
    return cudaGetLastError();
}

}  // namespace mvla
