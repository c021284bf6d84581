// Salience of the visual tokens (Sec. 3.2.1 of the paper): scaled dot-product logits of the text
// queries against the visual keys, softmax over all visual keys, mean over heads and queries.
//
// Work split: one thread-block cluster per (sample, head); each CTA of the cluster owns
// `tiles_per_cta` tiles of 128 keys.  A CTA produces the logits of its keys against all text
// queries (tensor cores for bf16: TMA -> shared memory -> tcgen05.mma -> tensor memory; plain
// FMAs for fp32), reduces a local softmax maximum and denominator per query, exchanges those with
// the other CTAs of the cluster through distributed shared memory, and writes, per key, the
// head's contribution  sum_i softmax(l[h,i,:])_j / (H n_t)  to part[h][j].  Heads are summed
// later in a fixed order so that the result does not depend on scheduling.
#include "common.cuh"
#include "device_utils.cuh"
#include "tmem_plan.h"

#include <math_constants.h>

namespace mvla {
namespace {

constexpr int kThreads = 128;

// ------------------------------------------------------------------ the kernel
// grid = (cluster size, n_heads, samples), cluster = (cluster size, 1, 1), block = 128 threads.
// Thread r owns key r of each tile (tensor-memory lane r).
template <typename T, bool UMMA>
__global__ void __launch_bounds__(kThreads, 1)
salience_kernel(const __grid_constant__ BatchDesc bd, const __grid_constant__ CUtensorMap tmap_q,
                const __grid_constant__ CUtensorMap tmap_k, const T* __restrict__ q,
                const T* __restrict__ k, int n_heads, int kv_group, int head_dim, int esize, int tiles_per_cta, int npad,
                float* __restrict__ part, int64_t part_stride, int* status, const AlphaOut alpha)
{
    extern __shared__ uint8_t dyn_smem_raw[];
    uint8_t* dyn_smem = dyn_smem_raw + ((1024u - (smem_u32(dyn_smem_raw) & 1023u)) & 1023u);   // swizzle atoms are 1 KB
    __shared__ float s_m[kMaxText];          // local max per query (log2 domain), -inf replaced by 0
    __shared__ float s_w[kMaxText];          // final weight per query
    __shared__ float s_peer[kMaxCluster][2][kMaxText];   // (raw local max, local sum) pushed here by every CTA of the cluster
    __shared__ float s_wred[4][kMaxText];
    __shared__ __align__(8) uint64_t s_bar[2];
    __shared__ uint32_t s_tmem;

    cluster_arrive_relaxed();                 // matched by the wait before the first remote store
    const SampleDev& s = bd.s[blockIdx.z];
    const int h = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t crank = cluster_ctarank();
    const uint32_t csize = gridDim.x;
    const int d = head_dim;
    const int64_t row_elems = static_cast<int64_t>(n_heads) * d;
    const int64_t kv_row_elems = static_cast<int64_t>(n_heads / kv_group) * d;   // grouped key heads: K rows are narrower
    const int hk = h / kv_group;                                                 // the key head this query head reads
    // logits are kept in the log2 domain: y = <q, k> * log2(e) / sqrt(d)
    const float cscale = 1.4426950408889634f * rsqrtf(static_cast<float>(d));
    const int tt0 = static_cast<int>(crank) * tiles_per_cta;

    uint32_t tmem_base = 0, tmem_cols = 0;
    const int tcol = npad <= 16 ? 16 : (npad <= 32 ? 32 : 64);   // tensor-memory columns reserved per tile
    float* Ls = nullptr;   // fp32 path: logits [tile][query][key]
    bool ok = true;

    if constexpr (UMMA) {
        const int khalves = (d * esize + 127) / 128;          // 128-byte swizzle rows (64 bf16 or 128 e4m3) per key; a last partial box is zero-filled by TMA
        const int box_elems = 128 / esize;
        uint8_t* Ks = dyn_smem;                               // [tile][khalf][128 rows x 128 B]
        uint8_t* Qs = dyn_smem + static_cast<size_t>(tiles_per_cta) * khalves * 16384;   // [khalf][npad rows x 128 B]
        const uint32_t bar_full = smem_u32(&s_bar[0]), bar_mma = smem_u32(&s_bar[1]);
        tmem_cols = 32;
        while (tmem_cols < static_cast<uint32_t>(tiles_per_cta * tcol)) tmem_cols <<= 1;
        if (tid == 0) {                       // the loads go out first; everything else overlaps with them
            prefetch_tensormap(&tmap_q);
            prefetch_tensormap(&tmap_k);
            mbar_init(bar_full, 1);
            mbar_init(bar_mma, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            int live = 0;
            for (int t = 0; t < tiles_per_cta; ++t) live += tile_info(s, tt0 + t).valid > 0;
            const uint32_t bytes = static_cast<uint32_t>(khalves) * (npad * 128 + live * 16384);
            mbar_expect_tx(bar_full, bytes);
            for (int kh = 0; kh < khalves; ++kh)
                for (int c = 0; c < npad / 16; ++c)
                    tma_load_3d(smem_u32(Qs + kh * npad * 128 + c * 2048), &tmap_q, kh * box_elems, h,
                                s.seq_off + s.off_txt + c * 16, bar_full);
            for (int t = 0; t < tiles_per_cta; ++t) {
                const TileInfo ti = tile_info(s, tt0 + t);
                if (ti.valid <= 0) continue;
                for (int kh = 0; kh < khalves; ++kh)
                    tma_load_3d(smem_u32(Ks + (t * khalves + kh) * 16384), &tmap_k, kh * box_elems, hk, ti.row0, bar_full);
            }
        }
        // blocks until the columns are free: the launcher has made sure that the CTAs resident on a multiprocessor
        // never ask for more than its 512 columns together, so no CTA waits here for one that waits for it
        if (warp == 1) tmem_alloc(smem_u32(&s_tmem), tmem_cols);
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        tmem_base = s_tmem;

        if (tid == 0) {
            bool got = mbar_wait(bar_full, 0);
            if (!got) {                       // report, then give the copies one more bounded chance to land
                *reinterpret_cast<volatile int*>(status) = MVLA_ERR_TIMEOUT;
                got = mbar_wait(bar_full, 0);
            }
            if (got) {
                tc_fence_after();
                const uint32_t idesc = idesc_by_size(esize, npad);
                for (int t = 0; t < tiles_per_cta; ++t) {
                    if (tile_info(s, tt0 + t).valid <= 0) continue;
                    for (int kb = 0; kb < khalves * 4; ++kb) {     // columns past d are zeros
                        const int kh = kb >> 2, kin = kb & 3;      // 4 K-steps of 16 inside a 64-wide half
                        const uint64_t a = smem_desc_sw128(smem_u32(Ks + (t * khalves + kh) * 16384) + kin * 32);
                        const uint64_t b = smem_desc_sw128(smem_u32(Qs + kh * npad * 128) + kin * 32);
                        umma_by_size(esize, tmem_base + t * tcol, a, b, idesc, kb > 0 ? 1u : 0u);
                    }
                }
            }
            umma_commit(bar_mma);             // arrives once every MMA issued above has finished
        }
        __syncwarp();
        if (!mbar_wait(bar_mma, 0)) {
            ok = false;
            *reinterpret_cast<volatile int*>(status) = MVLA_ERR_TIMEOUT;
        }
        ok = __syncthreads_and(ok) != 0;      // block-uniform from here on (aligned instructions follow)
        tc_fence_after();
    } else {
        // fp32 / generic path: stage Q and one key tile in shared memory as fp32, FMA the logits.
        float* Qs = reinterpret_cast<float*>(dyn_smem);               // [npad][d]
        float* Ks = Qs + npad * d;                                    // [128][d + 1]
        Ls = Ks + kKeyTile * (d + 1);                                 // [tile][npad][128]
        const int kp = d + 1;
        for (int idx = tid; idx < npad * d; idx += kThreads) {
            const int i = idx / d, c = idx - i * d;
            Qs[idx] = i < s.n_txt
                ? to_f32(q[static_cast<int64_t>(s.seq_off + s.off_txt + i) * row_elems + static_cast<int64_t>(h) * d + c])
                : 0.f;
        }
        for (int t = 0; t < tiles_per_cta; ++t) {
            const TileInfo ti = tile_info(s, tt0 + t);
            if (ti.valid <= 0) continue;
            __syncthreads();
            for (int idx = tid; idx < kKeyTile * d; idx += kThreads) {
                const int r = idx / d, c = idx - r * d;
                Ks[r * kp + c] = r < ti.valid
                    ? to_f32(k[static_cast<int64_t>(ti.row0 + r) * kv_row_elems + static_cast<int64_t>(hk) * d + c])
                    : 0.f;
            }
            __syncthreads();
            const float* kr = Ks + tid * kp;
            for (int cb = 0; cb < npad; cb += 16) {
                float acc[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] = 0.f;
                for (int c = 0; c < d; c += 4) {
                    const float k0 = kr[c], k1 = kr[c + 1], k2 = kr[c + 2], k3 = kr[c + 3];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float4 q4 = *reinterpret_cast<const float4*>(Qs + (cb + i) * d + c);
                        acc[i] = fmaf(k0, q4.x, acc[i]);
                        acc[i] = fmaf(k1, q4.y, acc[i]);
                        acc[i] = fmaf(k2, q4.z, acc[i]);
                        acc[i] = fmaf(k3, q4.w, acc[i]);
                    }
                }
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    Ls[(t * npad + cb + i) * kKeyTile + tid] = tid < ti.valid ? acc[i] * cscale : -CUDART_INF_F;
            }
        }
        __syncthreads();
    }

    // Loads the 16 logits (log2 domain) of this thread's key for queries [cb, cb+16) of tile t.
    auto load_chunk = [&](int t, int cb, int valid, float (&v)[16]) {
        if constexpr (UMMA) {
            tmem_ld16(tmem_base + (static_cast<uint32_t>(warp * 32) << 16) + static_cast<uint32_t>(t * tcol + cb), v);
            const bool live = tid < valid;
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = live ? v[i] * cscale : -CUDART_INF_F;
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = Ls[(t * npad + cb + i) * kKeyTile + tid];
        }
    };

    // ---- pass 1: local maximum per query over this CTA's keys
    for (int cb = 0; cb < npad; cb += 16) {
        float m[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) m[i] = -CUDART_INF_F;
        for (int t = 0; t < tiles_per_cta; ++t) {
            const int valid = tile_info(s, tt0 + t).valid;
            if (valid <= 0 || !ok) continue;
            float v[16];
            load_chunk(t, cb, valid, v);
#pragma unroll
            for (int i = 0; i < 16; ++i) m[i] = fmaxf(m[i], v[i]);
        }
        const float red = warp_reduce16<true>(m, lane);
        if ((lane & 1) == 0) s_wred[warp][cb + col16(lane)] = red;
    }
    __syncthreads();
    float m_raw = -CUDART_INF_F;
    if (tid < npad) {
        m_raw = fmaxf(fmaxf(s_wred[0][tid], s_wred[1][tid]), fmaxf(s_wred[2][tid], s_wred[3][tid]));
        s_m[tid] = (m_raw == -CUDART_INF_F) ? 0.f : m_raw;
    }
    __syncthreads();

    // ---- pass 2: local softmax denominator per query
    for (int cb = 0; cb < npad; cb += 16) {
        float sum[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) sum[i] = 0.f;
        for (int t = 0; t < tiles_per_cta; ++t) {
            const int valid = tile_info(s, tt0 + t).valid;
            if (valid <= 0 || !ok) continue;
            float v[16];
            load_chunk(t, cb, valid, v);
#pragma unroll
            for (int i = 0; i < 16; ++i) sum[i] += exp2f(v[i] - s_m[cb + i]);
        }
        const float red = warp_reduce16<false>(sum, lane);
        if ((lane & 1) == 0) s_wred[warp][cb + col16(lane)] = red;
    }
    __syncthreads();
    // ---- exchange (max, sum) with the other key tiles of this (sample, head): every CTA pushes its
    //      pair into every CTA's s_peer slot, then one release/acquire cluster barrier publishes them.
    cluster_wait_acquire();                   // pairs with the arrive at kernel entry: all peers are running
    if (tid < npad) {
        const float ssum = (s_wred[0][tid] + s_wred[1][tid]) + (s_wred[2][tid] + s_wred[3][tid]);
        const uint32_t a_m = smem_u32(&s_peer[crank][0][tid]), a_s = smem_u32(&s_peer[crank][1][tid]);
        for (uint32_t r = 0; r < csize; ++r) {
            st_peer_f32(a_m, r, m_raw);
            st_peer_f32(a_s, r, ssum);
        }
    }
    __syncwarp();
    cluster_arrive_release();
    cluster_wait_acquire();
    if (tid < npad) {
        float gmax = -CUDART_INF_F;
        for (uint32_t r = 0; r < csize; ++r) gmax = fmaxf(gmax, s_peer[r][0][tid]);
        float z = 0.f;
        for (uint32_t r = 0; r < csize; ++r) {
            const float mr = s_peer[r][0][tid];
            if (mr > -CUDART_INF_F) z += s_peer[r][1][tid] * exp2f(mr - gmax);
        }
        const float inv_hn = 1.f / (static_cast<float>(n_heads) * static_cast<float>(s.n_txt));
        s_w[tid] = (tid < s.n_txt && z > 0.f) ? exp2f(s_m[tid] - gmax) / z * inv_hn : 0.f;
    }
    __syncthreads();

    // ---- pass 3: per key, sum over queries of the normalised probabilities
    for (int t = 0; t < tiles_per_cta; ++t) {
        const TileInfo ti = tile_info(s, tt0 + t);
        if (ti.valid <= 0) continue;
        float acc = 0.f;
        if (ok) {
            for (int cb = 0; cb < npad; cb += 16) {
                float v[16];
                load_chunk(t, cb, ti.valid, v);
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float e = exp2f(v[i] - s_m[cb + i]);
                    const float pr = (cb + i < s.n_txt) ? e * s_w[cb + i] : 0.f;
                    acc += pr;
                    if (alpha.ptr && cb + i < s.n_txt && tid < ti.valid)   // the attention itself (per-patch indicators)
                        alpha.ptr[static_cast<int64_t>(h) * alpha.stride_h + static_cast<int64_t>(s.vis_off + ti.vis0 + tid) * alpha.stride_j +
                                  cb + i] = pr * (static_cast<float>(n_heads) * static_cast<float>(s.n_txt));
                }
            }
        }
        if (tid < ti.valid)
            part[static_cast<int64_t>(h) * part_stride + s.vis_off + ti.vis0 + tid] = acc;
    }

    // nothing touches a peer's shared memory after the barrier above, so CTAs may exit independently
    if constexpr (UMMA) {
        tc_fence_before();
        __syncthreads();
        if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);    // the warp that allocated
    }
}

// ------------------------------------------------------------------ head reduce, L1 norms
__global__ void head_reduce_kernel(const float* __restrict__ part, int64_t part_stride, int n_heads,
                                   int total_vis, float* __restrict__ attn)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait();                               // launched while the scoring kernel still runs: wait for its partials
    if (j >= total_vis) return;
    float acc = 0.f;
    for (int h = 0; h < n_heads; ++h) acc += part[static_cast<int64_t>(h) * part_stride + j];
    attn[j] = acc;
}

// One warp per visual row; 16-byte loads; fixed reduction order.
// Launched with programmatic serialization: the kernel after it may become resident at once, and this
// kernel itself needs nothing from the kernel before it except that the hidden rows are final, which the
// launch order guarantees (see the callers).  It therefore does its work first and waits for its
// predecessor LAST, only so that "this kernel is complete" keeps implying "its predecessor is complete"
// for whatever follows.
template <typename T>
__global__ void __launch_bounds__(256)
l1norm_kernel(const __grid_constant__ BatchDesc bd, int d_model, const T* __restrict__ hidden,
              float* __restrict__ l1, int early)
{
    if (early) pdl_trigger();
    else pdl_wait();
    const SampleDev& s = bd.s[blockIdx.y];
    const int nv = s.n_2d + s.n_3d;
    const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (j >= nv) {
        if (early) pdl_wait();
        return;
    }
    const int lane = threadIdx.x & 31;
    const int row = s.seq_off + (j < s.n_2d ? s.off_2d + j : s.off_3d + (j - s.n_2d));
    constexpr int kVec = 16 / sizeof(T);
    const uint4* src = reinterpret_cast<const uint4*>(hidden + static_cast<int64_t>(row) * d_model);
    const int nvec = d_model / kVec;
    float acc = 0.f;
    for (int i = lane; i < nvec; i += 32) {
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
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) l1[s.vis_off + j] = acc;
    if (early) pdl_wait();
}

template <typename T, bool UMMA>
cudaError_t launch_salience_t(const BatchDesc& bd, int n_heads, int kv_group, int head_dim, int esize, const void* q, const void* k,
                              const CUtensorMap* tq, const CUtensorMap* tk, int tiles_per_cta, int cluster,
                              int npad, float* part, int64_t part_stride, int* status, AlphaOut alpha,
                              cudaStream_t stream)
{
    size_t smem;
    if (UMMA)
        smem = 1024 + static_cast<size_t>((head_dim * esize + 127) / 128) * (static_cast<size_t>(tiles_per_cta) * 16384 + npad * 128);
    else
        smem = 1024 + sizeof(float) * (static_cast<size_t>(npad) * head_dim + kKeyTile * (head_dim + 1) +
                                static_cast<size_t>(tiles_per_cta) * npad * kKeyTile);
    if (smem > 227 * 1024) return cudaErrorInvalidConfiguration;
    auto kern = salience_kernel<T, UMMA>;
    int tmem_cols = 0;
    if (UMMA) {       // resident CTAs x tensor-memory columns must not exceed the 512 of a multiprocessor
        const int tcol = npad <= 16 ? 16 : (npad <= 32 ? 32 : 64);
        tmem_cols = tmem_cols_for(tiles_per_cta * tcol);
        smem = smem_for_tmem(smem, tmem_cols);
        if (smem == 0) return cudaErrorInvalidConfiguration;
    }
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    if (UMMA) {
        int resident = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kern, kThreads, smem);
        if (e != cudaSuccess) return e;
        if (resident * tmem_cols > kTmemColsPerSm) return cudaErrorInvalidConfiguration;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cluster, n_heads, bd.n);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    static const CUtensorMap zero_map = {};
    return cudaLaunchKernelEx(&cfg, kern, bd, tq ? *tq : zero_map, tk ? *tk : zero_map,
                              static_cast<const T*>(q), static_cast<const T*>(k), n_heads, kv_group, head_dim, esize,
                              tiles_per_cta, npad, part, part_stride, status, alpha);
}

}  // namespace

cudaError_t launch_salience(const BatchDesc& bd, int dtype, int n_heads, int kv_group, int head_dim, const void* q,
                            const void* k, const CUtensorMap* tmap_q, const CUtensorMap* tmap_k,
                            bool use_umma, int tiles_per_cta, int cluster, int npad, float* part,
                            int64_t part_stride, int* status, AlphaOut alpha, cudaStream_t stream)
{
    if (dtype == MVLA_DTYPE_FP8_E4M3) {      // tensor cores only: there is no FMA path for 8-bit inputs
        if (!use_umma) return cudaErrorInvalidConfiguration;
        return launch_salience_t<uint8_t, true>(bd, n_heads, kv_group, head_dim, 1, q, k, tmap_q, tmap_k, tiles_per_cta,
                                                cluster, npad, part, part_stride, status, alpha, stream);
    }
    if (dtype == MVLA_DTYPE_BF16) {
        if (use_umma)
            return launch_salience_t<__nv_bfloat16, true>(bd, n_heads, kv_group, head_dim, 2, q, k, tmap_q, tmap_k, tiles_per_cta,
                                                          cluster, npad, part, part_stride, status, alpha, stream);
        return launch_salience_t<__nv_bfloat16, false>(bd, n_heads, kv_group, head_dim, 2, q, k, nullptr, nullptr, tiles_per_cta,
                                                       cluster, npad, part, part_stride, status, alpha, stream);
    }
    return launch_salience_t<float, false>(bd, n_heads, kv_group, head_dim, 4, q, k, nullptr, nullptr, tiles_per_cta, cluster,
                                           npad, part, part_stride, status, alpha, stream);
}

cudaError_t launch_head_reduce(const float* part, int64_t part_stride, int n_heads, int total_vis, float* attn,
                               cudaStream_t stream)
{
    if (total_vis <= 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((total_vis + 255) / 256);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, head_reduce_kernel, part, part_stride, n_heads, total_vis, attn);
}

cudaError_t launch_l1norm(const BatchDesc& bd, int dtype, int d_model, const void* hidden, float* l1,
                          bool beside_predecessor, cudaStream_t stream)
{
    int max_nv = 0;
    for (int b = 0; b < bd.n; ++b) max_nv = max(max_nv, bd.s[b].n_2d + bd.s[b].n_3d);
    if (max_nv == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((max_nv + 7) / 8, bd.n);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1] = {pdl_attribute()};
    cfg.attrs = attr;
    cfg.numAttrs = beside_predecessor ? 1 : 0;
    const int early = beside_predecessor ? 1 : 0;
    if (dtype == MVLA_DTYPE_BF16)
        return cudaLaunchKernelEx(&cfg, l1norm_kernel<__nv_bfloat16>, bd, d_model, static_cast<const __nv_bfloat16*>(hidden), l1, early);
    return cudaLaunchKernelEx(&cfg, l1norm_kernel<float>, bd, d_model, static_cast<const float*>(hidden), l1, early);
}

}  // namespace mvla
